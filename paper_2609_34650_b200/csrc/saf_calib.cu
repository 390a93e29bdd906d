// Calibration statistics of one layer (Sec. 3.1 "Calibration and head selection"): from the queries and keys of N
// calibration sequences, for every head
//   A^(n)  = softmax_causal(Q^(n) K^(n)T scale)                       (Appendix A, Eq. "standard-head")
//   A^     = (1/N) sum_n A^(n)                                        (empirical mean; the fitter's input)
//   s_var  = 1/((N-1) T^2) sum_n ||A^(n) - A^||_F^2                   (Eq. "variance-score")
//   s_KL   = 1/(N T) sum_n sum_i KL(A^(n)[i,:i+1] || A^[i,:i+1])      (Eq. "forward-kl-score")
// in one streaming pass: sum_n A^(n) goes to a dense [H,T,T] accumulator, and per head the two scalars
// sum_n ||A^(n)||^2 and sum_n sum A^(n) log A^(n); at the end
//   sum_n ||A^(n) - A^||^2 = sum_n ||A^(n)||^2 - N ||A^||^2,   sum_n KL(.) = sum_n sum A log A - N sum A^ log A^.
// No A^(n) is ever stored.  The row normalisers come from the attention forward of the same sequences (its LSE
// output), so a tile of probabilities is exp2(s c - lse') straight from the score tile.
//
// One persistent kernel, item = (head, query block I, key block J <= I), all items cost the same.  Per item a loop
// over the N sequences: S = Q_I K_J^T on the tensor core (tcgen05, both operands K-major in 128B-swizzled smem via
// TMA, score tiles in four TMEM buffers), then per element in registers p = exp2(s c - lse'), acc += p,
// sq += p^2, ent += p log2 p; the 128 x 128 fp32 accumulator tile lives in the registers of the 16 compute warps
// (thread = query row x 32 keys) and leaves once per item through shared memory as four TMA stores into the dense
// accumulator, which drain while the next item computes; in the calls that add to earlier ones the old tile is
// fetched by TMA into the same boxes during the item and summed there (TMA reduce-adds measured 1.2 TB/s, half of
// what the plain load + store path reaches).
// CTA = 576 threads: warps 0-15 compute (TMEM lane = query row; warp >> 2 picks the 32-key column group), warp 16
// TMA producer, warp 17 tcgen05 issuer and TMEM owner.  Every wait is bounded.
#include <cuda_bf16.h>
#include <algorithm>
#include "ptx.cuh"
#include "saf_internal.h"

namespace saf {

namespace {

constexpr float LOG2E_C = 1.4426950408889634f;
constexpr double LN2_C = 0.6931471805599453094;

template <int D>
struct CalCfg {
  static constexpr int NPANEL = D / 64;                 // 64-column bf16 panels: 128-byte rows
  static constexpr int PANEL_BYTES = 128 * 64 * 2;
  static constexpr int TILE_BYTES = NPANEL * PANEL_BYTES;
  static constexpr int NS = (D == 64) ? 4 : 2;          // (Q, K) ring depth (shared memory allows no more at 128)
  static constexpr int STAGE_BYTES = 2 * TILE_BYTES;    // Q tile then K tile
  static constexpr int OFF_OUT = NS * STAGE_BYTES;      // 4 boxes of 128 rows x 32 fp32 (128-byte rows, swizzled): 64 KB
  static constexpr int OUT_BOX_BYTES = 128 * 128;
  static constexpr int OFF_BAR = OFF_OUT + 4 * OUT_BOX_BYTES;
  static constexpr int NSB = 4;                         // score buffers in TMEM (128 fp32 columns each)
  static constexpr int NBAR = 2 * NS + 2 * NSB + 4;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 128 * NSB;
  static constexpr int NTHREADS = 576;
};

enum CalSite { C_QK_EMPTY = 71, C_QK_FULL, C_S_FREE, C_S_FULL, C_OLD_FULL };

// item index -> (h, I, J) with J <= I; pairs are numbered row by row: q = I (I+1)/2 + J
__device__ __forceinline__ void decode_item(int idx, int npairs, int& h, int& I, int& J) {
  h = idx / npairs;
  const int q = idx - h * npairs;
  int i = static_cast<int>((sqrtf(8.0f * static_cast<float>(q) + 1.0f) - 1.0f) * 0.5f);
  while ((i + 1) * (i + 2) / 2 <= q) ++i;
  while (i * (i + 1) / 2 > q) --i;
  I = i;
  J = q - i * (i + 1) / 2;
}

}  // namespace

template <int D, bool ACC>
__global__ void __launch_bounds__(576, 1)
saf_calib_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mm, const CalibParams p) {
  using C = CalCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* qk_full = bars;                      // [NS]
  uint64_t* qk_empty = bars + C::NS;             // [NS]
  uint64_t* s_full = qk_empty + C::NS;           // [NSB] score buffer b holds a finished tile
  uint64_t* s_free = s_full + C::NSB;            // [NSB] the compute warps have read buffer b (16 warp arrivals)
  uint64_t* old_full = s_free + C::NSB;               // [4] the old accumulator values of output box k have landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(old_full + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(qk_full + s, 1);
      mbar_init(qk_empty + s, 1);
    }
    for (int b = 0; b < C::NSB; ++b) {
      mbar_init(s_full + b, 1);
      mbar_init(s_free + b, 16);
    }
    for (int k = 0; k < 4; ++k) mbar_init(old_full + k, 1);
    mbar_fence_init();
  }
  if (warp == 17) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 16) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mq);
      tma_prefetch_desc(&mk);
      uint32_t nl = 0;
      bool ok = true;
      for (int idx = blockIdx.x; idx < p.n_items && ok; idx += gridDim.x) {
        int h, I, J;
        decode_item(idx, p.npairs, h, I, J);
        for (int n = 0; n < p.B; ++n, ++nl) {
          const int s = nl % C::NS;
          ok = mbar_wait(qk_empty + s, ((nl / C::NS) & 1) ^ 1, wc, C_QK_EMPTY);
          if (!ok) break;
          mbar_expect_tx(qk_full + s, C::STAGE_BYTES);
          uint8_t* st = smem + s * C::STAGE_BYTES;
          for (int pn = 0; pn < C::NPANEL; ++pn) {
            tma_load_4d(st + pn * C::PANEL_BYTES, &mq, qk_full + s, pn * 64, I * BLK, h, n);
            tma_load_4d(st + C::TILE_BYTES + pn * C::PANEL_BYTES, &mk, qk_full + s, pn * 64, J * BLK, h / p.kv_group, n);
          }
        }
      }
    }
  } else if (warp == 17) {
    // ------------------------------------------------------------------ tcgen05 issuer
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);    // S: 128 queries x 128 keys, both K-major
    const uint64_t d_k = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint32_t lo_k = desc_lo(d_k), hi_k = desc_hi(d_k);
    uint32_t nl = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < p.n_items && ok; idx += gridDim.x) {
      for (int n = 0; n < p.B && ok; ++n, ++nl) {
        const uint32_t s = nl % C::NS, gb = nl % C::NSB;
        ok = mbar_wait_warp(qk_full + s, (nl / C::NS) & 1, wc, C_QK_FULL);
        if (!ok) break;
        ok = mbar_wait_warp(s_free + gb, ((nl / C::NSB) & 1) ^ 1, wc, C_S_FREE);
        if (!ok) break;
        tc_fence_after();
        const uint32_t q_lo = lo_k + ((s * C::STAGE_BYTES) >> 4);
        const uint32_t k_lo = q_lo + (C::TILE_BYTES >> 4);
        if (leader) {
#pragma unroll
          for (int kc = 0; kc < D / 16; ++kc) {
            const uint32_t off = ((kc >> 2) * C::PANEL_BYTES + (kc & 3) * 32) >> 4;
            umma_ss2(tmem + 128 * gb, q_lo + off, hi_k, k_lo + off, hi_k, idesc, kc > 0);
          }
          umma_commit(s_full + gb);
          umma_commit(qk_empty + s);
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps (512 threads)
    const int q4 = warp & 3, cq = warp >> 2;
    const int rowl = q4 * 32 + lane;                   // query row within the block = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const float c2 = p.scale_log2e;
    uint32_t nl = 0, nold = 0;
    bool ok = true;
    for (int idx = blockIdx.x; idx < p.n_items; idx += gridDim.x) {
      int h, I, J;
      decode_item(idx, p.npairs, h, I, J);
      const int qi = I * BLK + rowl;
      const int k0 = J * BLK + 32 * cq;                // first key of this thread's 32 columns
      const bool diag = (I == J) || (J * BLK + BLK > p.T);   // tiles that need the per-element mask
      const float* lse_h = p.LSE + static_cast<size_t>(h) * p.T + qi;
      const size_t lse_step = static_cast<size_t>(p.H) * p.T;
      // The four 32-column groups of compute warps hand their output box over independently of one another
      // (thread 128 cq leads group cq): a barrier over all 16 warps would put them back in lockstep at every item.
      const bool box_ok = J * BLK + 32 * cq < p.T;     // the group's box lies inside the matrix
      const bool lead = (tid == 128 * cq);
      uint8_t* const box = smem + C::OFF_OUT + cq * C::OUT_BOX_BYTES;
      if (ACC && p.use_tma && lead) {
        // what earlier calls left in this box is fetched while the sequences are processed (the previous item's
        // store has finished reading the box first)
        bulk_wait_group_read0();
        if (box_ok) {
          mbar_expect_tx(old_full + cq, C::OUT_BOX_BYTES);
          tma_load_4d(box, &mm, old_full + cq, J * BLK + 32 * cq, I * BLK, h, 0);
        }
      }
      uint64_t acc2[16];                               // the thread's 32 accumulators as packed pairs
#pragma unroll
      for (int k = 0; k < 16; ++k) acc2[k] = 0ull;
      uint64_t sq2 = 0ull, ps2 = 0ull;
      float lsum = 0.0f;
      // the normaliser of sequence n+1 is loaded while sequence n is processed and first touched one round later
      // (a use right after the load would stall the warp for the whole memory latency in front of the wait below)
      const bool row_ok = qi < p.T;
      float lse_raw = row_ok ? __ldg(lse_h) : 0.0f;
      for (int n = 0; n < p.B; ++n, ++nl) {
        float lse_raw_next = 0.0f;
        if (n + 1 < p.B && row_ok) lse_raw_next = __ldg(lse_h + (n + 1) * lse_step);
        const uint32_t gb = nl % C::NSB;
        if (ok && !mbar_wait_warp(s_full + gb, (nl / C::NSB) & 1, wc, C_S_FULL)) ok = false;
        if (!ok) continue;                             // (keeps the loop counters in step; nothing is read)
        const float lse2 = row_ok ? lse_raw * LOG2E_C : INFINITY;
        lse_raw = lse_raw_next;
        tc_fence_after();
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + 128 * gb + 32 * cq, r);
        tmem_wait_ld();
        tc_fence_before();
        warp_arrive(s_free + gb);                      // the tensor core may overwrite this buffer
        // p log2 p = p (s c - lse'): the first part is summed per element as p s, the second needs no tile at
        // all because a row of probabilities sums to one: the threads of key block 0, column group 0 add lse'
        // once per row and sequence.
        if (J == 0 && cq == 0 && row_ok) lsum += lse2;
        const uint64_t c2p = pk2(c2, c2), nlse = pk2(-lse2, -lse2);
        if (diag) {
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            const uint64_t s2 = pk2(__uint_as_float(r[2 * k]), __uint_as_float(r[2 * k + 1]));
            float a0, a1;
            upk2(fma2(s2, c2p, nlse), a0, a1);
            if (k0 + 2 * k > qi) a0 = -INFINITY;       // causal mask (also keys beyond T: qi < T there)
            if (k0 + 2 * k + 1 > qi) a1 = -INFINITY;
            const uint64_t p2 = pk2(ex2_approx(a0), ex2_approx(a1));
            acc2[k] = add2(acc2[k], p2);
            sq2 = fma2(p2, p2, sq2);
            ps2 = fma2(p2, s2, ps2);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            const uint64_t s2 = pk2(__uint_as_float(r[2 * k]), __uint_as_float(r[2 * k + 1]));
            float a0, a1;
            upk2(fma2(s2, c2p, nlse), a0, a1);
            const uint64_t p2 = pk2(ex2_approx(a0), ex2_approx(a1));
            acc2[k] = add2(acc2[k], p2);
            sq2 = fma2(p2, p2, sq2);
            ps2 = fma2(p2, s2, ps2);
          }
        }
      }
      float acc[32];
#pragma unroll
      for (int k = 0; k < 16; ++k) upk2(acc2[k], acc[2 * k], acc[2 * k + 1]);
      float sq, ps;
      {
        float x0, x1;
        upk2(sq2, x0, x1);
        sq = x0 + x1;
        upk2(ps2, x0, x1);
        ps = x0 + x1;
      }
      float ent = fmaf(ps, c2, -lsum);                 // sum of p log2 p of this thread's part of the item
      // the item's tile of sum_n A^(n): written, or added to what earlier calls left
      if (p.use_tma) {
        // through shared memory and one TMA store per 32-column box: coalesced, and it drains while the next item
        // computes.  The previous item's box has been read out before it is overwritten; the four warps of the
        // group also agree here whether a wait has been abandoned.
        if (!ACC && lead) bulk_wait_group_read0();
        if (ACC && box_ok) {
          if (ok && !mbar_wait_warp(old_full + cq, nold & 1, wc, C_OLD_FULL)) ok = false;
          ++nold;
        }
        if (named_bar_or(1 + cq, 128, !ok)) break;
        const uint32_t stage_row = smem_u32(box) + rowl * 128;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const uint32_t chunk = static_cast<uint32_t>(g ^ (rowl & 7)) * 16;
          float o0 = 0.0f, o1 = 0.0f, o2 = 0.0f, o3 = 0.0f;
          if (ACC) ld_shared_v4f(stage_row + chunk, o0, o1, o2, o3);
          st_shared_v4w(stage_row + chunk, __float_as_uint(acc[4 * g] + o0), __float_as_uint(acc[4 * g + 1] + o1),
                        __float_as_uint(acc[4 * g + 2] + o2), __float_as_uint(acc[4 * g + 3] + o3));
        }
        fence_proxy_async_smem();
        named_bar_sync(5 + cq, 128);
        if (lead && box_ok) {
          tma_store_4d(&mm, box, J * BLK + 32 * cq, I * BLK, h, 0);
          bulk_commit_group();
        }
      } else {
        // row lengths that are no multiple of four floats cannot be described to TMA: plain loads and stores
        if (!ok) break;
        if (qi < p.T) {
          float* dst = p.mean_sum + (static_cast<size_t>(h) * p.T + qi) * p.T + k0;
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (k0 + e < p.T) dst[e] = ACC ? dst[e] + acc[e] : acc[e];
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sq += __shfl_xor_sync(0xffffffffu, sq, o);
        ent += __shfl_xor_sync(0xffffffffu, ent, o);
      }
      if (lane == 0) {
        atomicAdd(p.sumsq + h, static_cast<double>(sq));
        atomicAdd(p.sum_plogp + h, static_cast<double>(ent) * LN2_C);
      }
    }
    if ((tid & 127) == 0) bulk_wait_group0();          // every store has landed before the kernel ends
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 17) tmem_dealloc(tmem, C::TMEM_COLS);
}

namespace {

// Mean and its two sums: one CTA walks rows blockIdx.x, blockIdx.x + gridDim.x, ... of head blockIdx.y; the causal
// part of each row is scaled by 1/N in place and contributes m^2 and m log m.
__global__ void __launch_bounds__(256)
saf_calib_mean_kernel(float* __restrict__ mean, double inv_n, double* __restrict__ tmp, int T) {
  __shared__ double red[2][8];
  const int h = blockIdx.y, tid = threadIdx.x;
  float* M = mean + static_cast<size_t>(h) * T * T;
  double s2 = 0.0, sl = 0.0;
  const float invf = static_cast<float>(inv_n);
  for (int i = blockIdx.x; i < T; i += gridDim.x) {
    float* row = M + static_cast<size_t>(i) * T;
    float a2 = 0.0f, al = 0.0f;
    for (int j0 = tid; j0 <= i; j0 += 1024) {        // four independent loads in flight per thread
      float v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = (j0 + 256 * u <= i) ? row[j0 + 256 * u] : 0.0f;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (j0 + 256 * u <= i) {
          const float m = v[u] * invf;
          row[j0 + 256 * u] = m;
          a2 = fmaf(m, m, a2);
          if (m > 0.0f) al = fmaf(m, __log2f(m), al);
        }
      }
    }
    s2 += static_cast<double>(a2);
    sl += static_cast<double>(al);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    sl += __shfl_xor_sync(0xffffffffu, sl, o);
  }
  if ((tid & 31) == 0) {
    red[0][tid >> 5] = s2;
    red[1][tid >> 5] = sl;
  }
  __syncthreads();
  if (tid == 0) {
    double a = 0.0, b = 0.0;
    for (int w = 0; w < 8; ++w) {
      a += red[0][w];
      b += red[1][w];
    }
    atomicAdd(tmp + 2 * h, a);
    atomicAdd(tmp + 2 * h + 1, b * LN2_C);
  }
}

// s_var = (sum_n ||A_n||^2 - N ||A^||^2) / ((N-1) T^2),  s_KL = (sum_n sum A_n log A_n - N sum A^ log A^) / (N T);
// both are non-negative by definition, so rounding residue below zero is clamped.
__global__ void saf_calib_scores_kernel(const double* __restrict__ sumsq, const double* __restrict__ sum_plogp,
                                        const double* __restrict__ tmp, double n_total, int T, int H,
                                        double* __restrict__ s_var, double* __restrict__ s_kl) {
  const int h = blockIdx.x * blockDim.x + threadIdx.x;
  if (h >= H) return;
  const double t = static_cast<double>(T);
  if (s_var) s_var[h] = fmax(sumsq[h] - n_total * tmp[2 * h], 0.0) / ((n_total - 1.0) * t * t);
  if (s_kl) s_kl[h] = fmax(sum_plogp[h] - n_total * tmp[2 * h + 1], 0.0) / (n_total * t);
}

}  // namespace

int calib_smem_bytes(int D) { return D == 64 ? CalCfg<64>::SMEM : CalCfg<128>::SMEM; }

template <int D, bool ACC>
static cudaError_t launch_calib_t(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mm,
                                  const CalibParams& p, int grid, cudaStream_t st) {
  cudaError_t e = cudaFuncSetAttribute(saf_calib_kernel<D, ACC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       CalCfg<D>::SMEM);
  if (e != cudaSuccess) return e;
  saf_calib_kernel<D, ACC><<<grid, CalCfg<D>::NTHREADS, CalCfg<D>::SMEM, st>>>(mq, mk, mm, p);
  return cudaGetLastError();
}

cudaError_t launch_calib(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mm,
                         const CalibParams& p, int grid, cudaStream_t st) {
  if (D == 64) return p.accumulate ? launch_calib_t<64, true>(mq, mk, mm, p, grid, st)
                                   : launch_calib_t<64, false>(mq, mk, mm, p, grid, st);
  return p.accumulate ? launch_calib_t<128, true>(mq, mk, mm, p, grid, st)
                      : launch_calib_t<128, false>(mq, mk, mm, p, grid, st);
}

cudaError_t launch_calib_finalize(float* mean, const double* sumsq, const double* sum_plogp, double* tmp, int H, int T,
                                  double n_total, double* s_var, double* s_kl, int num_sms, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(tmp, 0, static_cast<size_t>(H) * 2 * sizeof(double), st);
  if (e != cudaSuccess) return e;
  int nb = std::max(1, std::min((8 * num_sms + H - 1) / H, T));
  saf_calib_mean_kernel<<<dim3(nb, H), 256, 0, st>>>(mean, 1.0 / n_total, tmp, T);
  saf_calib_scores_kernel<<<(H + 127) / 128, 128, 0, st>>>(sumsq, sum_plogp, tmp, n_total, T, H, s_var, s_kl);
  return cudaGetLastError();
}

}  // namespace saf
