// Internal declarations shared by the host API and the sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdlib>
#include <utility>

namespace saf {

// Launch with the programmatic-stream-serialization attribute: the kernel may be scheduled while the kernel
// before it in the stream drains, runs its prologue (barrier set-up, TMEM allocation, descriptor prefetch) and
// then blocks in pdl_wait() until that kernel has completed.  Every kernel launched this way calls pdl_wait()
// before it touches global memory, so completion of a kernel still implies completion of all earlier ones.
// SAF_DISABLE_PDL=1 launches the ordinary way.
inline bool pdl_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("SAF_DISABLE_PDL");
    return !(e && std::atoi(e) == 1);
  }();
  return on;
}
// Which kernels are launched that way (SAF_PDL_MASK: bit 0 staging kernels, 1 forward, 2 backward preparation,
// 3 backward).  Measured on the 124M-shaped step (fwd + bwd back to back, no events in between): only the backward
// gains (-0.5 %); an early forward grid costs 3 %, because its CTAs then land on SMs in the order these become
// free and the pairing of a light and a heavy CTA per SM that the scheduler's work lists assume is lost.
inline int pdl_mask() {
  static const int m = [] {
    const char* e = std::getenv("SAF_PDL_MASK");
    return e ? std::atoi(e) : 8;
  }();
  return m;
}
enum { PDL_STAGE = 1, PDL_FWD = 2, PDL_PREP = 4, PDL_BWD = 8 };
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(int which, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pdl_enabled() && (pdl_mask() & which)) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

constexpr int BLK = 128;            // query rows per item and keys per tile
constexpr int KIND_ORDINARY = 0;
constexpr int KIND_FROZEN = 1;

struct WorkItem { int32_t b, h, blk, kind; };

struct FwdParams {
  int B, H, T, Tp;
  int kv_group;                     // query heads per shared key/value head (>= 1)
  int d_real;                       // head dimension of the tensors (96 runs on the 128-wide kernel, zero-padded by TMA)
  const int* qslot;                 // packed Q/K layout: head -> slot among the ordinary heads (NULL: slot = head)
  float scale_log2;                 // softmax_scale * log2(e)
  const float* alpha;               // [H][Tp]
  const float* rho;                 // [H][Tp]
  const float* logZ;                // [H][Tp]
  void* O;                          // bf16 (fp32 if o_f32), strided
  int o_f32;
  int64_t o_strides[3];             // elements: batch, head, seq
  float* LSE;                       // [B][H][T]
  // Tensor-core form of frozen heads (all NULL when the pattern tables are not prepared): band_f is the
  // forward Hankel band table [H][nblkp][2048] fp16, wvec the row scale w(i) [H][Tp], fast_ok[h] != 0
  // where the form may be used, hord[h] the head's ordinal among the frozen heads (-1 otherwise).
  const void* band_f;
  const float* wvec;
  const int* fast_ok;
  const int* hord;
  // ovf[h] == call_id: a staged fp16 value of head h left fp16's range in this call (general path instead)
  const int* ovf;
  int call_id;
  int nblkp;
  const WorkItem* items;            // grouped by CTA
  const int* cta_offsets;           // [grid+1]
  // D = 64 forward: the items in queue order, claimed at run time.  queue[0] = next unclaimed item, queue[1] = CTAs
  // that have finished; the last CTA to finish sets both back to zero for the next launch.
  const WorkItem* order;
  int n_items;
  int* queue;
  int* status;                      // device status word
  unsigned long long wait_limit_ns;
  // Self-test of the give-up path (0 in normal use): the producer of the D = 64 forward leaves out the load of the
  // first key tile of its first ordinary item, so that the waits for it run out.  Set by saf_create from
  // SAF_SELFTEST_DROP_LOAD, and only for grids of at most 16 CTAs with a wait limit of at most 50 ms.
  int selftest_drop_load;
};

struct BwdParams {
  int B, H, T, Tp;
  int kv_group;                     // as in FwdParams; > 1: dK / dV are reduce-added instead of stored
  const int* qslot;                 // packed layout of Q, K, dQ, dK (see FwdParams)
  int d_real;                       // head dimension of the tensors (128-wide kernel: 128 or 96)
  int n_ord;                        // number of ordinary heads (head count of the packed tensors)
  float scale, scale_log2;
  const float* alpha;
  const float* rho;
  const float* logZ;
  // Workspace images of the extra reduction step that folds the row terms into the score MMAs
  // (ordinary heads): per (b,h,128-row block) a 4 KB no-swizzle K-major tile [128 rows][16] bf16 whose
  // first three columns hold a three-way bf16 split of -LSE/scale (q_ext) or of -delta (do_ext).
  const void* q_ext;
  const void* do_ext;
  int nblk;
  void* dK;                         // [B][H][T][D] grad dtype
  void* dV;
  int grad_f32;
  // tensor-core form of frozen heads (see FwdParams): backward band table and the key scale a(j)
  const void* band_b;
  const float* avec;
  const int* fast_ok;
  const int* hord;
  const int* ovf;                   // as in FwdParams
  int call_id;
  int nblkp;
  const WorkItem* items;
  const int* cta_offsets;
  int* status;
  unsigned long long wait_limit_ns;
};

// Gradients of the compact patterns (saf_pgrad.cu).  Items carry the head's ordinal among the frozen heads.
// One unit of work of the pattern-gradient kernel: key block J of frozen head number hf (ordinal among the frozen
// heads), query blocks I0 .. I1-1, accumulated over batch entries b0 .. b1-1 on the tensor core.
struct PgItem {
  int hf, J, I0, I1, b0, b1, pad0, pad1;
};
// Batch entries whose V tile stays in shared memory for the length of an item (the item's batch range is at most this).
inline int pgrad_batch_chunk(int D) { return D == 64 ? 8 : 4; }
// Batch entries (dO tiles) per stage of the kernel's dO ring.
inline int pgrad_stage_entries(int D) { return D == 64 ? 2 : 1; }
struct PgradParams {
  int B, H, T, Tp;
  int kv_group;
  const float* alpha;               // [H][Tp]
  const float* rho;
  const float* logZ;
  const float* delta;               // [batch chunks][H][T]: rowsum(dO o O) summed over a chunk, frozen heads only
  const int* hlist;                 // ordinal -> head
  float* dalpha;                    // [H][Tp], zeroed before the launch; accumulated with atomicAdd
  float* drho;
  const PgItem* items;
  const int* cta_offsets;
  int* status;
  unsigned long long wait_limit_ns;
};
cudaError_t launch_rowdot(const void* O, int o_f32, const void* dO, const int64_t* o_strides, const int* hlist,
                          float* delta, int B, int H, int Hf, int T, int D, cudaStream_t st);
cudaError_t launch_pgrad(int D, const CUtensorMap& mv, const CUtensorMap& mdo, const PgradParams& p, int grid,
                         cudaStream_t st);

// The vectors a call passes against the bits the pattern tables were built from (snapshot: alpha, rho, logZ,
// each [H][Tp] as raw 32-bit words, one after the other).
struct PatternCheck {
  const float* alpha;
  const float* rho;
  const float* logZ;
  const uint32_t* snap;
  size_t vec_elems;                 // H * Tp
};
// Launchers (defined in the .cu files).  All return the launch error.
cudaError_t launch_logz(const float* alpha, const float* rho, float* logZ, const uint8_t* mask_dev, int H,
                        int Tp, cudaStream_t st);
cudaError_t launch_pattern_tables(const float* alpha, const float* rho, const float* logZ, const uint8_t* mask_dev,
                                  int H, int Tp, float* consts, int* fast_ok, float* avec, float* wvec, void* band_f,
                                  void* band_b, cudaStream_t st);
cudaError_t launch_scale_rows(const void* src, const int64_t* strides, const float* vec, float extra, int Tp,
                              const int* hlist, const int* pat_ok, int* ovf, int call_id, void* dst, int B, int Hf,
                              int T, int D, int src_group, const PatternCheck& chk, cudaStream_t st);   // src head = h / src_group
// powers of two that put the fp16 operands of the tensor-core frozen form into fp16's range
constexpr float HK_BAND_SCALE = 16384.0f;        // bands hold 2^14 r
constexpr float HK_A_SCALE = 2048.0f;            // the forward stages 2^11 a V
// mvt: map of the a-scaled V of the frozen heads [B][Hf][T][D] (any valid map when band_f is NULL)
cudaError_t launch_fwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mvt, const CUtensorMap& mo, const FwdParams& p, int grid, cudaStream_t st);
// mdot: map of the w-scaled dO of the frozen heads [B][Hf][T][D] (any valid map when band_b is NULL);
// mdk / mdv: fp32 maps of dK / dV shaped like mdq (only used when grad_f32 is set)
cudaError_t launch_bwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mdo, const CUtensorMap& mdq, const CUtensorMap& mdot, const CUtensorMap& mdk,
                       const CUtensorMap& mdv, const BwdParams& p, int grid, cudaStream_t st);
// Row terms of ordinary heads (q_ext / do_ext images, see BwdParams); also zeroes dQacc (all heads) and
// dK of frozen heads, and (dot_dst != NULL) stages w(i) dO of the frozen heads in fp16 for the tensor-core form.
struct PrepFrozen {
  const float* wvec;                // [H][Tp]
  const int* hord;                  // head -> ordinal among the frozen heads
  const int* pat_ok;                // per-head flag of the pattern
  int* ovf;                         // set to call_id when a staged value leaves fp16's range
  int call_id;
  void* dot_dst;                    // fp16 [B][Hf][T][D], or NULL
  int Hf, Tp;
  PatternCheck chk;
};
cudaError_t launch_bwd_prep(const void* O, int o_f32, const void* dO, const float* LSE, const int64_t* o_strides,
                            const uint8_t* mask_dev, void* q_ext, void* do_ext, float inv_scale, float* dQacc, void* dK,
                            void* dV, int grad_f32, int kv_group, const int* qslot, int n_ord, const PrepFrozen& fz, int B,
                            int H, int T, int D, cudaStream_t st);   // kv_group > 1: zeroes all of dK and dV (fp32) instead
// dQ (grad dtype) = scale-free copy/convert of dQacc (fp32) for the bf16-gradient case.
cudaError_t launch_bwd_finalize(const float* dQacc, void* dQ, size_t n, cudaStream_t st);
// head dimension 64 (saf_fwd64.cu); launch_fwd dispatches to it
cudaError_t launch_fwd64(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mvt,
                         const CUtensorMap& mo, const FwdParams& p, int grid, cudaStream_t st);
int fwd64_smem_bytes();
// head dimension 128 / 96 (saf_bwd128.cu): mqh / mdoh / mdoth are maps with 64-row boxes (half tiles), mdq the fp32 dQ
// accumulator [B][Hq][T][D]; dK / dV are written with plain stores (reduce-adds for shared heads)
cudaError_t launch_bwd128(const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mqh, const CUtensorMap& mdoh,
                          const CUtensorMap& mdoth, const CUtensorMap& mdq, const BwdParams& p, int grid,
                          cudaStream_t st);
int bwd128_smem_bytes();
int fwd_smem_bytes(int D);
int bwd_smem_bytes(int D);

// compact-pattern fitter (saf_fit.cu): per-head state of Fit, all arrays [Hf, T]
struct FitState {
  int T;
  double lr;
  const double* eta_abs;
  const double* eta_rel;
  double* alpha; double* rho;          // fp64 parameters
  double* m_a; double* v_a; double* m_r; double* v_r;   // Adam moments
  float* a2[2]; float* r2[2];          // log2e-scaled fp32 copies, double-buffered over the steps
  float* nz2;                          // -log2 Z(i) of the current parameters
};
int fit_max_T();
cudaError_t launch_fit_marginals(const float* Abar, float floor_v, double* eta_abs, double* eta_rel, double* plogp,
                                 int Hf, int T, int num_sms, cudaStream_t st);
cudaError_t launch_fit(const FitState& s, int Hf, int steps, const double* plogp, float* alpha_out, float* rho_out,
                       float* logZ_out, long long out_stride, double* loss_out, double* kl_out, cudaStream_t st);

// calibration statistics (saf_calib.cu)
struct CalibParams {
  int B, H, T;                      // B = sequences of this call
  int kv_group;
  float scale_log2e;                // softmax scale x log2(e)
  const float* LSE;                 // [B][H][T], natural-log normalisers from the attention forward
  float* mean_sum;                  // [H][T][T]: sum over sequences of the attention maps (causal tiles only)
  double* sumsq;                    // [H] += sum_n ||A_n||_F^2
  double* sum_plogp;                // [H] += sum_n sum A_n log A_n
  int accumulate;                   // 0: overwrite mean_sum tiles, 1: add to them
  int use_tma;                      // T % 4 == 0: tiles leave by TMA; else plain loads / stores
  int n_items, npairs;              // items = H x npairs, npairs = nblk (nblk+1)/2
  int* status;
  unsigned long long wait_limit_ns;
};
cudaError_t launch_calib(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mm,
                         const CalibParams& p, int grid, cudaStream_t st);
cudaError_t launch_calib_finalize(float* mean, const double* sumsq, const double* sum_plogp, double* tmp, int H, int T,
                                  double n_total, double* s_var, double* s_kl, int num_sms, cudaStream_t st);

}  // namespace saf

// Trace builds only: per-CTA first/last time stamps (globaltimer, ns) of a kernel, read back by
// saf_debug_read_span_<name>; regular builds compile these to nothing.
#ifdef SAF_TRACE
#define SAF_SPAN_DEFINE(name)                                                                   \
  __device__ unsigned long long g_saf_span_##name[1024][2];                                     \
  extern "C" int saf_debug_read_span_##name(unsigned long long* out) {                          \
    return static_cast<int>(cudaMemcpyFromSymbol(out, g_saf_span_##name, sizeof(g_saf_span_##name))); \
  }
#define SAF_SPAN(name, k)                                                                       \
  do {                                                                                          \
    if (threadIdx.x == 0) g_saf_span_##name[blockIdx.x & 1023][k] = saf::globaltimer_ns();      \
  } while (0)
#else
#define SAF_SPAN_DEFINE(name)
#define SAF_SPAN(name, k)
#endif

