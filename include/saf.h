/* saf.h - C ABI of the B200 (sm_100a) hybrid causal attention layer of Selective Attention Freezing.
 *
 * One layer call runs ordinary query-key softmax heads and "frozen" heads side by side.
 *   ordinary head (Appendix A, Eq. "standard-head"):  S = Q K^T * scale, A = softmax_causal(S), O = A V
 *   frozen head   (Sec. 3.1; Sec. 3.2, Eq. "compact-prior"):  O = P^ V with
 *        P^(i,j) = exp(alpha(j) + rho(i-j)) / Z(i)  for j <= i,  0 for j > i,
 *        Z(i)    = sum_{k<=i} exp(alpha(k) + rho(i-k)),
 *     rebuilt tile by tile from the two length-Tp vectors; the T x T pattern is never stored.
 *   backward      (Sec. 3.3; Appendix E.2): frozen heads give dV = P^T dO and no query/key gradient
 *     (their dQ/dK slots are written with zeros); ordinary heads give dQ, dK, dV.
 * Indices are 0-based: alpha[j] for key j in [0,T), rho[d] for distance d = i-j in [0,T).
 *
 * Conventions (all entry points):
 *   - "dev" pointers are device pointers owned by the caller; "host" pointers are host pointers.
 *     The library never frees or reallocates caller memory.
 *   - Q, K, V, dO and (unless saf_problem.o_dtype says fp32) O are bf16 tensors indexed [b][h][t][c] through element strides (c has stride 1);
 *     base addresses and strides must be multiples of 8 elements (16 bytes).
 *   - frozen_mask_host is a host array uint8[H]; nonzero = frozen head.  It is read (copied) before the call
 *     returns, whatever kind of host memory it lives in.
 *   - alpha, rho, logZ are fp32 [H][Tp] row-major device arrays; rows of ordinary heads are ignored.
 *     They may be NULL when no head is frozen.  Q/K/LSE rows of frozen heads are never read.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     The return value covers host-side validation and launch errors.  A kernel whose bounded wait
 *     gave up reports through saf_last_device_status() after the stream has been synchronised.
 *   - One context serves one stream at a time; contexts are not thread-safe.
 *   - Every function returns SAF_OK (0) or one of the SAF_ERR_* codes; nothing is launched on error.
 */
#ifndef SAF_H_
#define SAF_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct saf_ctx saf_ctx; /* opaque: workspace, cached work lists, device status word */

enum {
  SAF_OK = 0,
  SAF_ERR_INVALID_ARG = 1,    /* NULL pointer, bad shape, T > Tp, misaligned pointer or stride */
  SAF_ERR_UNSUPPORTED = 2,    /* head dimension or dtype outside the supported set */
  SAF_ERR_CUDA = 3,           /* a CUDA runtime/driver call failed */
  SAF_ERR_DEVICE_TIMEOUT = 4, /* a bounded wait inside a kernel gave up */
  SAF_ERR_ARCH = 5,           /* device is not compute capability 10.x */
  SAF_ERR_NOMEM = 6
};
enum { SAF_BF16 = 0, SAF_F32 = 1 };

typedef struct {
  int32_t B, H, T, D;          /* square causal attention: T queries and T keys; D in {64, 96, 128}
                                  (96 runs on the 128-wide kernels) */
  int32_t Tp;                  /* stored pattern length (row length of alpha/rho/logZ); T <= Tp */
  float softmax_scale;         /* <= 0 selects 1/sqrt(D) (Appendix A) */
  int32_t grad_dtype;          /* dtype of dQ/dK/dV: SAF_F32 or SAF_BF16 */
  int32_t kv_group;            /* grouped-query path (Appendix E.2): query heads per shared key/value head;
                                  K, V, dK, dV then have H / kv_group heads and query head h reads head
                                  h / kv_group.  0 or 1 = multi-head attention.  (Shared heads' gradients are
                                  accumulated in fp32; with bf16 gradients in a context-owned workspace.) */
  int32_t packed_qk;           /* nonzero: Q, K, dQ, dK carry only the ordinary heads, in head order (Appendix E.2:
                                  replaced heads have no query/key slot on the multi-head path); needs
                                  kv_group <= 1.  Not available through saf_hybrid_attn_step_host. */
  int32_t o_dtype;             /* dtype of O: SAF_BF16 (0, the default) or SAF_F32.  dO stays bf16 and uses the same
                                  element strides.  SAF_F32 is not available through saf_hybrid_attn_step_host. */
  int64_t q_strides[3], k_strides[3], v_strides[3], o_strides[3]; /* elements: batch, head, seq */
} saf_problem;                 /* dO uses o_strides (elements; o_strides must be multiples of 8 in both cases);
                                  with bf16 O the backward's row term sum(dO*O) is taken from the rounded O (the
                                  parity tests feed the reference the same rounded O when T < 8), with fp32 O from
                                  the unrounded one; LSE [B][H][T], dQ [B][H][T][D] and dK, dV
                                  [B][H/kv_group][T][D] are contiguous (packed_qk: dQ, dK [B][Ho][T][D]) */

/* Library version (major*100 + minor). */
int saf_version(void);
const char* saf_status_string(int code);

/* Create / destroy a context on CUDA device `device`.  Creation allocates a small status word and
 * queries the device; SAF_ERR_ARCH if it is not sm_100-class. */
int saf_create(saf_ctx** out, int device);
int saf_destroy(saf_ctx* ctx);

/* Row normalisers of the compact pattern (Sec. 3.2, Eq. "compact-prior"; Algorithm 1 stores
 * (alpha, rho, log Z) per replaced head):
 *   logZ_dev_out[h][i] = log sum_{k<=i} exp(alpha[h][k] + rho[h][i-k]),  i in [0,Tp), frozen h only.
 * Row i uses alpha[0..i] and rho[0..i] only, so the result serves every T <= Tp.  alpha_dev, rho_dev,
 * logZ_dev_out: device fp32 [H][Tp].  Call again whenever alpha or rho change.
 * frozen_mask_host (here and in every other entry point) is read before the call returns; the caller may change
 * or free it afterwards.
 * The call also builds the context's tables for the tensor-core form of the frozen heads and remembers the three
 * device pointers and their contents.  A later layer call uses the tables only for heads whose alpha, rho and logZ
 * still hold exactly those bits; a head whose vectors were rewritten in place since (by the caller, by
 * saf_fit_compact, by saf_pattern_logz_static) is computed from the vectors it is given, in the slower general form,
 * until saf_pattern_prepare is called again. */
int saf_pattern_prepare(saf_ctx* ctx, int32_t H, int32_t Tp, const uint8_t* frozen_mask_host,
                        const float* alpha_dev, const float* rho_dev, float* logZ_dev_out, void* stream);

/* Row normalisers without any allocation (the paper has no counterpart: this entry point exists for the
 * host program's sake, not the method's).
 *
 * Some host programs cannot let a library allocate device memory: a serving process that hands all of
 * the GPU's memory to its own pool at start-up (a later cudaMalloc simply fails), or a component that
 * must not block on the allocator inside a latency-critical loop.  saf_pattern_prepare needs a device
 * copy of the frozen-head mask and gets it from memory the context allocates; this variant computes
 * the same logZ with that copy in a fixed array inside the library image.
 *
 *   - No context.  `device` is the CUDA device to run on.  Other arguments as saf_pattern_prepare.
 *   - H must not exceed SAF_STATIC_MAX_HEADS; a larger H returns SAF_ERR_INVALID_ARG and launches nothing.
 *   - The call makes no cudaMalloc / cudaFree and uses no allocating library routine.  It only computes
 *     logZ; the tensor-core pattern tables of saf_pattern_prepare are not built, and tables a context built
 *     earlier from the same buffers are not refreshed: layer calls on that context notice the changed contents
 *     and take the general form for those heads until saf_pattern_prepare runs again.
 *   - The first call on a device resolves the array's device address (one cudaGetSymbolAddress, cached per
 *     device).  Make that first call during set-up, before any stream capture is begun.
 *   - The array (SAF_STATIC_MAX_HEADS bytes per GPU, held until the process exits) is shared by every
 *     call and keeps the previous call's contents; each call overwrites the H bytes it reads.  Two calls
 *     whose GPU work overlaps (different streams, or different threads) race on it: serialise them. */
#define SAF_STATIC_MAX_HEADS 1024
int saf_pattern_logz_static(int32_t device, int32_t H, int32_t Tp, const uint8_t* frozen_mask_host,
                            const float* alpha_dev, const float* rho_dev, float* logZ_dev_out, void* stream);

/* Forward of the hybrid layer (Sec. 3.3 "Fused computation"; Appendix E.2): one persistent launch.
 *   Q, K, V : device bf16, strided as in `p`.
 *   logZ    : device fp32 [H][Tp] from saf_pattern_prepare, or NULL to have it computed into
 *             context-owned memory on every call (slower).
 *   O       : device bf16 (fp32 with p->o_dtype = SAF_F32), strided by p->o_strides, every head in its original slot.
 *   LSE     : device fp32 [B][H][T]; natural-log sum of exp of the scaled causal scores for ordinary
 *             heads, 0 for frozen heads (they have no softmax).  May be NULL if every head is frozen. */
int saf_hybrid_attn_fwd(saf_ctx* ctx, const saf_problem* p, const void* Q, const void* K, const void* V,
                        const uint8_t* frozen_mask_host, const float* alpha, const float* rho,
                        const float* logZ, void* O, float* LSE, void* stream);

/* Backward of the hybrid layer (Sec. 3.3; Appendix E.2).  Inputs as in the forward plus O and LSE as
 * the forward wrote them and dO (device bf16, strided by p->o_strides).
 *   dQ, dK, dV : device, contiguous [B][H][T][D], fp32 or bf16 per p->grad_dtype.
 *                Frozen heads: dV = P^^T dO, dQ and dK written with zeros.
 * dQ is accumulated with floating-point atomics across key blocks, so its low-order bits can vary
 * from run to run.  Head dimensions 64, 96 and 128. */
int saf_hybrid_attn_bwd(saf_ctx* ctx, const saf_problem* p, const void* Q, const void* K, const void* V,
                        const void* O, const void* dO, const float* LSE, const uint8_t* frozen_mask_host,
                        const float* alpha, const float* rho, const float* logZ, void* dQ, void* dK,
                        void* dV, void* stream);

/* Whole step through HOST buffers: copies the inputs to context-owned device memory, runs
 * saf_pattern_prepare (only when `prepare` is nonzero; otherwise the normalisers of the previous
 * call on this context are reused), the forward and - when dO_host is not NULL - the backward, and
 * copies the results back.  Tensors are contiguous [B][H][T][D] (strides in `p` are ignored);
 * alpha_host/rho_host are [H][Tp].  Any output pointer may be NULL to skip its copy.  Synchronous.
 * Large problems are cut into up to eight chunks of whole batch entries on three streams (inputs in, compute,
 * results out), so that the copies of neighbouring chunks overlap the compute and each other in both directions
 * of the link; give pinned host memory for that overlap to happen. */
int saf_hybrid_attn_step_host(saf_ctx* ctx, const saf_problem* p, const void* Q_host, const void* K_host,
                              const void* V_host, const void* dO_host, const uint8_t* frozen_mask_host,
                              const float* alpha_host, const float* rho_host, int32_t prepare, void* O_host,
                              float* LSE_host, void* dQ_host, void* dK_host, void* dV_host);

/* Gradients of the compact patterns of the frozen heads, for the control in which alpha and rho stay trainable
 * (appendix on pattern controls; the paper prints no formula, this is the derivative of Eq. "compact-prior").
 * With b_ij = alpha(j) + rho(i-j), P^ = softmax_causal(b), O = P^ V and L = sum(O o dO):
 *   G = dO V^T,  dL/db_ij = P^_ij (G_ij - dO_i . O_i),
 *   dalpha_out[h][j] = sum_b sum_{i>=j} dL/db_ij,   drho_out[h][d] = sum_b sum_{i-j=d} dL/db_ij.
 * V: bf16 [B][H/kv_group][T][D] (v_strides); O (p->o_dtype), dO (bf16): [B][H][T][D] (o_strides), O as returned by the
 * forward;
 * alpha, rho, logZ: device fp32 [H][Tp] (logZ as from saf_pattern_prepare); dalpha_out, drho_out: device fp32
 * [H][Tp], fully overwritten (rows of ordinary heads and entries beyond T with zeros).
 * After an update of alpha/rho the caller refreshes logZ with saf_pattern_prepare. */
int saf_pattern_grad(saf_ctx* ctx, const saf_problem* problem, const void* V, const void* O, const void* dO,
                     const uint8_t* frozen_mask_host, const float* alpha, const float* rho, const float* logZ,
                     float* dalpha_out, float* drho_out, void* stream);

/* Compact-pattern fitter, step 1: sufficient statistics of the target (Sec. 3.2 "Fitting", text below
 * Eq. "fit-objective"; Algorithm 1, fitting loop).  For each of `Hf` heads the causal entries (j <= i) of the mean
 * attention map are floored at `floor_value` (the paper uses 1e-9) and every row is scaled to sum to one; of that
 * target P the call returns eta_abs(j) = sum_{i>=j} P(i,j), eta_rel(d) = sum_{i-j=d} P(i,j) and sum_{ij} P log P
 * (natural log), which is what the acceptance test needs besides the two marginals.
 *   mean_attn   : device float32 [Hf, T, T] row-major (row = query); entries above the diagonal are never read.
 *                 Read once; not modified.
 *   eta_abs_out, eta_rel_out : device float64 [Hf, T]; plogp_out : device float64 [Hf].  Overwritten.
 * T <= 16384 (SAF_ERR_UNSUPPORTED beyond); Hf = 0 is a no-op; Hf <= 65535.  Asynchronous on `stream`.  The sums are
 * accumulated with floating-point atomics: results agree from run to run to rounding, not bit for bit. */
int saf_fit_marginals(saf_ctx* ctx, int32_t Hf, int32_t T, const float* mean_attn, float floor_value,
                      double* eta_abs_out, double* eta_rel_out, double* plogp_out, void* stream);

/* Compact-pattern fitter, step 2: Fit and acceptance statistic (Eq. "fit-objective"; appendix "Selection, fitting,
 * and installation": alpha = 0, rho(d) = log max(eta_rel(d)/(T-d), 1e-9), then `steps` Adam steps (beta1 0.9,
 * beta2 0.999, eps 1e-8, bias-corrected) at learning rate `lr` on
 * L = (1/T)[sum_i log Z(i) - sum_j eta_abs(j) alpha(j) - sum_d eta_rel(d) rho(d)]; the paper uses 400 steps at 0.05).
 * All heads are fitted together; nothing of size T x T is allocated (state: 68 bytes per head and position, held by
 * the context and reused).  Exponentials are fp32, the sums that feed Adam and Adam itself fp64.
 *   eta_abs, eta_rel : device float64 [Hf, T] (from saf_fit_marginals, or accumulated by the caller)
 *   plogp            : device float64 [Hf] or NULL if kl_out is NULL
 *   alpha_out, rho_out, logZ_out : device float32, row h at offset h*out_stride (out_stride >= T elements): the
 *                      fitted parameters and log Z(i) of Eq. "compact-prior", as saf_pattern_prepare takes them
 *   loss_out         : device float64 [Hf] or NULL: L at the fitted parameters
 *   kl_out           : device float64 [Hf] or NULL: kappa = mean row KL(P || P^) = L + plogp/T; the paper accepts a
 *                      head when kappa <= 0.2 nats (the caller compares)
 * steps = 0 returns the starting point.  T <= 16384 (SAF_ERR_UNSUPPORTED beyond).  Asynchronous on `stream`
 * (2*steps + 3 kernel launches). */
int saf_fit_compact(saf_ctx* ctx, int32_t Hf, int32_t T, const double* eta_abs, const double* eta_rel,
                    const double* plogp, int32_t steps, double lr, float* alpha_out, float* rho_out, float* logZ_out,
                    int64_t out_stride, double* loss_out, double* kl_out, void* stream);

/* Calibration statistics of one layer, streaming part (Sec. 3.1 "Calibration and head selection";
 * Eq. "variance-score", Eq. "forward-kl-score").  For the `problem->B` calibration sequences of this call and every
 * head, the attention maps A^(n) = softmax_causal(Q K^T scale) are formed tile by tile (never stored) and added up:
 *   mean_sum[h][i][j] (+)= sum_n A^(n)(i,j)       device float32 [H, T, T] row-major, 16-byte aligned
 *   sumsq[h]          (+)= sum_n ||A^(n)||_F^2     device float64 [H]
 *   sum_plogp[h]      (+)= sum_n sum_{ij} A^(n) log A^(n)   device float64 [H]  (natural log, 0 log 0 = 0)
 * `accumulate` = 0 overwrites (first call of a layer), non-zero adds to what earlier calls left, so N sequences may
 * arrive in any number of calls.  Of mean_sum only the 128 x 128 tiles that meet the causal triangle are touched
 * (inside them entries above the diagonal get zeros); the tiles strictly above it are never read or written.
 *   Q, K    : device bf16 with problem's q_strides / k_strides; all heads are ordinary here (calibration precedes
 *             replacement); kv_group as in the attention calls; packed_qk must be 0; Tp and the other strides are
 *             ignored.  D in {64, 96, 128}.
 *   LSE     : device float32 [B][H][T]: the row normalisers that saf_hybrid_attn_fwd returned for the same Q, K
 *             (natural-log sum of exp of the scaled causal scores).
 * Asynchronous on `stream`. */
int saf_calib_accumulate(saf_ctx* ctx, const saf_problem* problem, const void* Q, const void* K, const float* LSE,
                         float* mean_sum, double* sumsq, double* sum_plogp, int32_t accumulate, void* stream);

/* Calibration statistics, final part: with `n_total` sequences accumulated, scales the causal part of `mean_inout`
 * by 1/n_total in place (the empirical mean A^, the "post-softmax mean" pattern and the input of saf_fit_marginals)
 * and returns per head
 *   s_var_out[h] = (sumsq[h] - N ||A^||_F^2) / ((N-1) T^2)            = Eq. "variance-score"
 *   s_kl_out[h]  = (sum_plogp[h] - N sum A^ log A^) / (N T)           = Eq. "forward-kl-score"
 * (device float64 [H]; either may be NULL; both are clamped at zero against rounding).  s_var needs n_total >= 2
 * (SAF_ERR_INVALID_ARG otherwise).  Asynchronous on `stream`. */
int saf_calib_finalize(saf_ctx* ctx, int32_t H, int32_t T, int64_t n_total, float* mean_inout, const double* sumsq,
                       const double* sum_plogp, double* s_var_out, double* s_kl_out, void* stream);

/* Device-side status of the most recent launches on this context: SAF_OK or SAF_ERR_DEVICE_TIMEOUT.
 * Synchronises the context's device status word with the host (blocks until the stream used by the
 * last call has drained).  `detail_out` (may be NULL) receives the raw word: site and CTA that gave up. */
int saf_last_device_status(saf_ctx* ctx, int32_t* detail_out);

/* Kernel timing for benchmarks.  With profiling enabled, every kernel the library launches is
 * bracketed by a CUDA event pair on the launching stream.  saf_get_kernel_time() waits for the pairs
 * of kernel `which` recorded since its last call, returns their summed duration and count, and
 * forgets them.  Off by default (the events cost a few microseconds per launch). */
enum {
  SAF_KERNEL_FWD = 0,          /* persistent forward kernel */
  SAF_KERNEL_BWD = 1,          /* persistent backward kernel */
  SAF_KERNEL_BWD_PREP = 2,     /* delta = rowsum(dO o O), zero-fill of dQ and of frozen heads' dK */
  SAF_KERNEL_BWD_FINALIZE = 3, /* fp32 -> bf16 conversion of dQ (bf16 gradients only) */
  SAF_KERNEL_LOGZ = 4,         /* pattern normalisers and tables (saf_pattern_prepare) */
  SAF_KERNEL_SCALE = 5,        /* per-call row scaling of the frozen heads' V (forward) / dO (backward) */
  SAF_KERNEL_PGRAD = 6,        /* pattern-gradient kernel (saf_pattern_grad) */
  SAF_KERNEL_FIT = 7,          /* all launches of one saf_fit_compact call, as one interval */
  SAF_KERNEL_FIT_MARGINALS = 8,/* target marginals (saf_fit_marginals) */
  SAF_KERNEL_CALIB = 9,        /* calibration statistics kernel (saf_calib_accumulate) */
  SAF_KERNEL_CALIB_FINALIZE = 10, /* mean and scores (saf_calib_finalize) */
  SAF_KERNEL_COUNT = 11
};
int saf_set_profiling(saf_ctx* ctx, int32_t enable);
int saf_get_kernel_time(saf_ctx* ctx, int32_t which, float* total_ms_out, int32_t* launches_out);

/* Head scheduler (host only, no GPU needed).  Builds the per-CTA work lists the persistent kernels
 * walk: one item per (batch, head, 128-row block); ordinary and frozen items are packed into the
 * same grid, longest-processing-time first, with a frozen tile weighted `frozen_weight_pct` percent
 * of an ordinary one plus a fixed cost per item (150 % of an ordinary tile forward, 100 % backward:
 * the values the library uses for the 64-wide kernels).  `backward` = 0: block is a query block and
 * costs (block+1) key tiles; 1: block is a key block and costs (nblocks-block) query tiles.
 * The layer calls use measured weights per kernel family (frozen tile 30 / 20 % forward / backward at
 * head dimension 64, 50 / 20 % at 96 and 128; item 150 / 100 % and 300 / 200 %), which the
 * environment variables SAF_FROZEN_WEIGHT_PCT, SAF_FROZEN_WEIGHT_BWD_PCT, SAF_ITEM_OVERHEAD_PCT and
 * SAF_ITEM_OVERHEAD_BWD_PCT (read by saf_create) override.  In a forward grid (two CTAs per SM) the
 * layer calls also charge the second half of the grid 20 % (head dimension 64) or 6 % more for the
 * same work, since the CTA that arrives second on an SM runs slower (SAF_SECOND_WAVE_PCT).
 *   items_out   : host int32[n_items*4] = (b, h, block, kind) with kind 0 ordinary / 1 frozen,
 *                 grouped by CTA; n_items = B*H*ceil(T/128)
 *   offsets_out : host int32[n_ctas+1], CSR offsets into items_out
 * Returns SAF_OK or SAF_ERR_INVALID_ARG. */
int saf_build_worklist(int32_t B, int32_t H, int32_t T, const uint8_t* frozen_mask_host, int32_t backward,
                       int32_t n_ctas, int32_t frozen_weight_pct, int32_t* items_out, int32_t* offsets_out);

#ifdef __cplusplus
}
#endif
#endif /* SAF_H_ */
