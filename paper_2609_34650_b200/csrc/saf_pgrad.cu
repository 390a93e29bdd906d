// Gradients of the compact pattern of the frozen heads (the control in which alpha and rho stay trainable;
// appendix on pattern controls).  The paper prints no formula; this is the derivative of Eq. "compact-prior":
// with the bias b_ij = alpha(j) + rho(i-j), P^ = softmax_causal(b), O = P^ V and L = sum(O o dO),
//   G = dO V^T,  dL/db_ij = P^_ij (G_ij - delta_i),  delta_i = sum_k P^_ik G_ik = dO_i . O_i,
//   dL/dalpha(j) = sum_{i >= j} dL/db_ij,   dL/drho(d) = sum_{i-j = d} dL/db_ij,   both summed over the batch.
//
// One persistent kernel, item = (batch, frozen head, 128-key block J), loop over query blocks I >= J:
//   G^T tile [128 keys x 128 queries] = V_J dO_I^T on the tensor core (tcgen05, both operands K-major in
//   128B-swizzled smem via TMA, accumulator double-buffered in TMEM), then per element in registers
//   p = exp2(alpha'(j) + rho'(i-j) - logZ'(i)) (primes: log2e-scaled; distances < 0 and rows/keys beyond T carry
//   -inf, which is the causal mask), db = p (G - delta_i).
//   dalpha(j): the thread that owns key row j sums its db over the whole item and adds once (atomicAdd).
//   drho(d):   within a warp the 32 lanes hold 32 consecutive keys; a lane that fetches column e from lane
//              (l' + e) mod 32 always lands on the same two diagonals, so the 95 diagonal sums of a warp's
//              32 x 64 sub-tile come out of independent shuffles (three registers per lane) and are added to drho
//              with atomicAdd (combining the warps in shared memory first measured slower).
// CTA = 320 threads: warps 0-7 compute (TMEM lane = key row; warps 0-3 query columns 0-63, warps 4-7 columns 64-127),
// warp 8 TMA producer, warp 9 tcgen05 issuer and TMEM owner.  Every wait is bounded.
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

namespace saf {

namespace {

constexpr float LOG2E_P = 1.4426950408889634f;

template <int D>
struct PgCfg {
  static constexpr int NPANEL = D / 64;                 // 64-column bf16 panels: 128-byte rows
  static constexpr int PANEL_BYTES = 128 * 64 * 2;
  static constexpr int TILE_BYTES = NPANEL * PANEL_BYTES;
  static constexpr int NS = 2;                          // dO ring depth
  static constexpr int OFF_V = 0;
  static constexpr int OFF_DO = TILE_BYTES;
  static constexpr int OFF_TAB = OFF_DO + NS * TILE_BYTES;
  // floats: r2raw[256] z2s[128] dl[128]
  static constexpr int TAB_FLOATS = 256 + 128 + 128;
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  static constexpr int NBAR = 2 + 2 * NS + 2 + 2;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 256;                 // two G^T buffers of 128 fp32 columns
  static constexpr int NTHREADS = 320;
};

enum PgSite { G_V_EMPTY = 61, G_DO_EMPTY, G_V_FULL, G_DO_FULL, G_G_FREE, G_G_FULL };

}  // namespace

template <int D>
__global__ void __launch_bounds__(320, 2)
saf_pgrad_kernel(const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mdo, const PgradParams p) {
  using C = PgCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* v_full = bars;
  uint64_t* v_empty = bars + 1;
  uint64_t* do_full = bars + 2;                  // [NS]
  uint64_t* do_empty = do_full + C::NS;          // [NS]
  uint64_t* g_full = do_empty + C::NS;           // [2] G^T buffer b holds a finished tile
  uint64_t* g_free = g_full + 2;                 // [2] the compute warps have read buffer b (8 warp arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(g_free + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* tab = reinterpret_cast<float*>(smem + C::OFF_TAB);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  const int nblk = (p.T + BLK - 1) / BLK;

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(v_full, 1);
    mbar_init(v_empty, 1);
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(do_full + s, 1);
      mbar_init(do_empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(g_full + b, 1);
      mbar_init(g_free + b, 8);
    }
    mbar_fence_init();
  }
  if (warp == 9) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int it_begin = p.cta_offsets[blockIdx.x], it_end = p.cta_offsets[blockIdx.x + 1];

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mdo);
      uint32_t nv = 0, ndo = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const WorkItem w = p.items[it];                  // w.h = ordinal among the frozen heads
        const int h = p.hlist[w.h];
        ok = mbar_wait(v_empty, (nv & 1) ^ 1, wc, G_V_EMPTY);
        if (!ok) break;
        mbar_expect_tx(v_full, C::TILE_BYTES);
        for (int pn = 0; pn < C::NPANEL; ++pn)
          tma_load_4d(smem + C::OFF_V + pn * C::PANEL_BYTES, &mv, v_full, pn * 64, w.blk * BLK, h / p.kv_group, w.b);
        ++nv;
        for (int I = w.blk; I < nblk; ++I) {
          const int s = ndo % C::NS;
          ok = mbar_wait(do_empty + s, ((ndo / C::NS) & 1) ^ 1, wc, G_DO_EMPTY);
          if (!ok) break;
          mbar_expect_tx(do_full + s, C::TILE_BYTES);
          for (int pn = 0; pn < C::NPANEL; ++pn)
            tma_load_4d(smem + C::OFF_DO + s * C::TILE_BYTES + pn * C::PANEL_BYTES, &mdo, do_full + s, pn * 64, I * BLK,
                        h, w.b);
          ++ndo;
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ tcgen05 issuer
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t idesc = umma_idesc_bf16(128, 128, 0, 0);    // G^T: 128 keys x 128 queries, both K-major
    const uint64_t d_k = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint32_t lo_k = desc_lo(d_k), hi_k = desc_hi(d_k);
    const uint32_t v_lo = lo_k + (C::OFF_V >> 4);
    uint32_t nv = 0, ndo = 0, ng = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end && ok; ++it) {
      const WorkItem w = p.items[it];
      const int ntiles = nblk - w.blk;
      ok = mbar_wait_warp(v_full, nv & 1, wc, G_V_FULL);
      if (!ok) break;
      ++nv;
      for (int t = 0; t < ntiles && ok; ++t, ++ng) {
        const uint32_t s = ndo % C::NS, gb = ng & 1;
        ok = mbar_wait_warp(do_full + s, (ndo / C::NS) & 1, wc, G_DO_FULL);
        if (!ok) break;
        ++ndo;
        ok = mbar_wait_warp(g_free + gb, ((ng >> 1) & 1) ^ 1, wc, G_G_FREE);
        if (!ok) break;
        tc_fence_after();
        const uint32_t do_lo = lo_k + ((C::OFF_DO + s * C::TILE_BYTES) >> 4);
        if (leader) {
#pragma unroll
          for (int kc = 0; kc < D / 16; ++kc) {
            const uint32_t off = ((kc >> 2) * C::PANEL_BYTES + (kc & 3) * 32) >> 4;
            umma_ss2(tmem + 128 * gb, v_lo + off, hi_k, do_lo + off, hi_k, idesc, kc > 0);
          }
          umma_commit(g_full + gb);
          umma_commit(do_empty + s);
          if (t == ntiles - 1) umma_commit(v_empty);
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps (256 threads)
    const int q4 = warp & 3, hh = warp >> 2;
    const int rowl = q4 * 32 + lane;                   // key row within the block = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    float* r2raw = tab;                                // [256] rho' over the tile's band of distances
    float* z2s = tab + 256;                            // [128] logZ' of the tile's queries
    float* dl = tab + 384;                             // [128] delta of the tile's queries
    uint32_t ng = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end; ++it) {
      const WorkItem w = p.items[it];
      const int h = p.hlist[w.h];
      const int ntiles = nblk - w.blk;
      const int key = w.blk * BLK + rowl;
      const float* alpha_h = p.alpha + static_cast<size_t>(h) * p.Tp;
      const float* rho_h = p.rho + static_cast<size_t>(h) * p.Tp;
      const float* logz_h = p.logZ + static_cast<size_t>(h) * p.Tp;
      const float* delta_bh = p.delta + (static_cast<size_t>(w.b) * p.H + h) * p.T;
      const float a2 = (key < p.T) ? alpha_h[key] * LOG2E_P : -INFINITY;
      float dacc = 0.0f;                               // dalpha(key) of this item (this thread's query half)
      bool leave = false;
      for (int t = 0; t < ntiles; ++t, ++ng) {
        // the previous tile's table readers are done; the warps also agree whether to go on
        if (named_bar_or(1, 256, !ok)) {
          ok = false;
          leave = true;
          break;
        }
        const int I = w.blk + t;
        const int d0 = t * BLK - 127;                  // band: distances d0 .. d0+254, index x = q - row + 127
        {
          const int d = d0 + tid;
          r2raw[tid] = (tid < 255 && d >= 0 && d < p.T) ? rho_h[d] * LOG2E_P : -INFINITY;
          if (tid < 128) {
            const int qi = I * BLK + tid;
            z2s[tid] = (qi < p.T) ? logz_h[qi] * LOG2E_P : INFINITY;
            dl[tid] = (qi < p.T) ? delta_bh[qi] : 0.0f;
          }
        }
        named_bar_sync(2, 256);
        const uint32_t gb = ng & 1;
        if (!mbar_wait_warp(g_full + gb, (ng >> 1) & 1, wc, G_G_FULL)) ok = false;
        tc_fence_after();
        const uint32_t t_g = tmem + lane_base + 128 * gb + 64 * hh;
        // Diagonal sums without a serial chain: the entry of column e that lane l' fetches from lane (l' + e) mod 32
        // lies on diagonal x = 32 cc + 31 - l' (no wrap) or 32 cc + 63 - l' (wrap), whatever e is, so every lane
        // sums two diagonals per 32-column chunk with independent shuffles.
        float dg[2][2] = {{0.0f, 0.0f}, {0.0f, 0.0f}};
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t r[32];
          tmem_ld32(t_g + 32 * cc, r);
          tmem_wait_ld();
          if (cc == 1) {
            tc_fence_before();
            warp_arrive(g_free + gb);                  // the tensor core may overwrite this buffer
          }
          const int q0 = 64 * hh + 32 * cc;
          const float* rb = r2raw + (q0 - rowl + 127);
#pragma unroll
          for (int e4 = 0; e4 < 8; ++e4) {
            const float4 z4 = *reinterpret_cast<const float4*>(z2s + q0 + 4 * e4);
            const float4 d4 = *reinterpret_cast<const float4*>(dl + q0 + 4 * e4);
            const float zz[4] = {z4.x, z4.y, z4.z, z4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int e = 4 * e4 + k;
              const float pij = ex2_approx(a2 + rb[e] - zz[k]);
              const float db = pij * (__uint_as_float(r[e]) - dd[k]);
              dacc += db;
              const float got = __shfl_sync(0xffffffffu, db, lane + e);      // (the source lane is taken modulo 32)
              if (lane + e < 32) dg[cc][0] += got;
              else dg[cc][1] += got;
            }
          }
        }
        if (ok) {
          // lane l' holds the diagonals x = 31 - l', 63 - l', 95 - l' (x = column - key lane + 31 within this warp's
          // 32 keys x 64 queries); distance d = (I - J) 128 + 64 hh - 32 q4 + x - 31
          float* drho_h = p.drho + static_cast<size_t>(h) * p.Tp;
          const int dbase = t * BLK + 64 * hh - 32 * q4 - lane;
          const float v3[3] = {dg[0][0], dg[0][1] + dg[1][0], dg[1][1]};
#pragma unroll
          for (int k = 0; k < 3; ++k) {
            const int d = dbase + 32 * k;
            if (d >= 0 && d < p.T && (k < 2 || lane > 0)) atomicAdd(drho_h + d, v3[k]);
          }
        }
      }
      if (leave) break;
      if (ok && key < p.T) atomicAdd(p.dalpha + static_cast<size_t>(h) * p.Tp + key, dacc);
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, C::TMEM_COLS);
}

// delta[b][h][t] = sum_c dO[b][h][t][c] * O[b][h][t][c] for the frozen heads (hlist); TPR threads per row, eight
// features each (16 threads with four idle ones at D = 96, so that a row stays inside a warp).
template <int D, int TPR>
__global__ void __launch_bounds__(256) saf_rowdot_kernel(const __nv_bfloat16* __restrict__ O,
                                                         const __nv_bfloat16* __restrict__ dO, int64_t s0, int64_t s1,
                                                         int64_t s2, const int* __restrict__ hlist,
                                                         float* __restrict__ delta, int B, int H, int Hf, int T) {
  const long long gid = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long rowid = gid / TPR;               // over [B][Hf][T]
  const int part = static_cast<int>(gid % TPR);
  const bool inrange = rowid < static_cast<long long>(B) * Hf * T;
  float acc = 0.0f;
  int b = 0, h = 0, t = 0;
  if (inrange) {
    t = static_cast<int>(rowid % T);
    h = hlist[(rowid / T) % Hf];
    b = static_cast<int>(rowid / (static_cast<long long>(T) * Hf));
  }
  if (inrange && part * 8 < D) {
    const int64_t off = b * s0 + h * s1 + static_cast<int64_t>(t) * s2 + part * 8;
    const uint4 o4 = *reinterpret_cast<const uint4*>(O + off);
    const uint4 d4 = *reinterpret_cast<const uint4*>(dO + off);
    const __nv_bfloat162* o2 = reinterpret_cast<const __nv_bfloat162*>(&o4);
    const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&d4);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 of = __bfloat1622float2(o2[e]), df = __bfloat1622float2(d2[e]);
      acc = fmaf(of.x, df.x, acc);
      acc = fmaf(of.y, df.y, acc);
    }
  }
#pragma unroll
  for (int o = TPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (inrange && part == 0) delta[(static_cast<size_t>(b) * H + h) * T + t] = acc;
}

cudaError_t launch_rowdot(const void* O, const void* dO, const int64_t* os, const int* hlist, float* delta, int B, int H,
                          int Hf, int T, int D, cudaStream_t st) {
  const int tpr = D == 96 ? 16 : D / 8;
  const long long nthreads = static_cast<long long>(B) * Hf * T * tpr;
  const unsigned grid = static_cast<unsigned>((nthreads + 255) / 256);
#define SAF_ROWDOT_ARGS \
  static_cast<const __nv_bfloat16*>(O), static_cast<const __nv_bfloat16*>(dO), os[0], os[1], os[2], hlist, delta, B, H, Hf, T
  if (D == 64) saf_rowdot_kernel<64, 8><<<grid, 256, 0, st>>>(SAF_ROWDOT_ARGS);
  else if (D == 96) saf_rowdot_kernel<96, 16><<<grid, 256, 0, st>>>(SAF_ROWDOT_ARGS);
  else saf_rowdot_kernel<128, 16><<<grid, 256, 0, st>>>(SAF_ROWDOT_ARGS);
#undef SAF_ROWDOT_ARGS
  return cudaGetLastError();
}

cudaError_t launch_pgrad(int D, const CUtensorMap& mv, const CUtensorMap& mdo, const PgradParams& p, int grid,
                         cudaStream_t st) {
  cudaError_t e;
  if (D == 64) {
    e = cudaFuncSetAttribute(saf_pgrad_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, PgCfg<64>::SMEM);
    if (e != cudaSuccess) return e;
    saf_pgrad_kernel<64><<<grid, PgCfg<64>::NTHREADS, PgCfg<64>::SMEM, st>>>(mv, mdo, p);
  } else {
    e = cudaFuncSetAttribute(saf_pgrad_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, PgCfg<128>::SMEM);
    if (e != cudaSuccess) return e;
    saf_pgrad_kernel<128><<<grid, PgCfg<128>::NTHREADS, PgCfg<128>::SMEM, st>>>(mv, mdo, p);
  }
  return cudaGetLastError();
}

}  // namespace saf
