// Gradients of the compact pattern of the frozen heads (the control in which alpha and rho stay trainable;
// appendix on pattern controls).  The paper prints no formula; this is the derivative of Eq. "compact-prior":
// with the bias b_ij = alpha(j) + rho(i-j), P^ = softmax_causal(b), O = P^ V and L = sum(O o dO),
//   G = dO V^T,  dL/db_ij = P^_ij (G_ij - delta_i),  delta_i = sum_k P^_ik G_ik = dO_i . O_i,
//   dL/dalpha(j) = sum_{i >= j} dL/db_ij,   dL/drho(d) = sum_{i-j = d} dL/db_ij,   both summed over the batch.
//
// P^ does not depend on the batch entry, so the batch sum moves inside the contraction:
//   sum_b dL/db_ij = P^_ij (Gs_ij - Ds_i),  Gs = sum_b dO_b V_b^T (one contraction over batch and features),
//   Ds_i = sum_b delta_b,i,
// and the per-element work (one exponential each) is done once per head, not once per head and batch entry.
//
// One persistent kernel, item = (frozen head, 128-key block J, a run of query blocks I >= J, a run of batch
// entries of at most VB); the V_J tiles of the item's batch entries stay in shared memory, per query block:
//   Gs^T tile [128 keys x 128 queries] = sum_b V_J,b dO_I,b^T on the tensor core (tcgen05, both operands K-major in
//   128B-swizzled smem via TMA, dO streamed through a ring of stages of SB batch entries each, accumulator
//   double-buffered in TMEM), then per element
//   in registers p = exp2(alpha'(j) + rho'(i-j) - logZ'(i)) (primes: log2e-scaled; distances < 0 and rows/keys
//   beyond T carry -inf, which is the causal mask), db = p (Gs - Ds_i).
//   dalpha(j): the thread that owns key row j sums its db over the whole item and adds once (atomicAdd).
//   drho(d):   within a warp the 32 lanes hold 32 consecutive keys; a lane that fetches column e from lane
//              (l' + e) mod 32 always lands on the same two diagonals, so the 63 diagonal sums of a warp's
//              32 x 32 sub-tile come out of independent shuffles (two registers per lane) and are added to drho
//              with atomicAdd (combining the warps in shared memory first measured slower).
// CTA = 576 threads, one per SM: warps 0-15 compute (TMEM lane = key row; warp w owns keys 32 (w mod 4) .. +31 and
// query columns 32 (w / 4) .. +31), warp 16 TMA producer, warp 17 tcgen05 issuer and TMEM owner.  Every wait is
// bounded.
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
  static constexpr int VB = (D == 64) ? 8 : 4;          // resident V tiles = batch entries per item (pgrad_batch_chunk)
  static constexpr int SB = (D == 64) ? 2 : 1;          // batch entries (dO tiles) per ring stage (pgrad_stage_entries)
  static constexpr int NS = (D == 64) ? 4 / SB : 2;     // dO ring depth (five single-tile stages measured the same)
  static constexpr int STAGE_BYTES = SB * TILE_BYTES;
  static constexpr int OFF_V = 0;
  static constexpr int OFF_DO = VB * TILE_BYTES;
  static constexpr int OFF_TAB = OFF_DO + NS * STAGE_BYTES;
  // floats, two sets (tile parity): r2raw[256] z2s[128] dl[128]
  static constexpr int TAB_FLOATS = 2 * (256 + 128 + 128);
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  static constexpr int NBAR = 2 + 2 * NS + 2 + 2;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 256;                 // two G^T buffers of 128 fp32 columns
  static constexpr int NCW = 16;                        // compute warps: 4 lane quarters x 4 column quarters
  static constexpr int NTHREADS = (NCW + 2) * 32;
};

enum PgSite { G_V_EMPTY = 61, G_DO_EMPTY, G_V_FULL, G_DO_FULL, G_G_FREE, G_G_FULL };

}  // namespace

template <int D>
__global__ void __launch_bounds__(PgCfg<D>::NTHREADS, 1)
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
      mbar_init(g_free + b, C::NCW);
    }
    mbar_fence_init();
  }
  if (warp == C::NCW + 1) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int it_begin = p.cta_offsets[blockIdx.x], it_end = p.cta_offsets[blockIdx.x + 1];

  if (warp == C::NCW) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mdo);
      uint32_t nv = 0, ndo = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const PgItem w = p.items[it];
        const int h = p.hlist[w.hf];
        ok = mbar_wait(v_empty, (nv & 1) ^ 1, wc, G_V_EMPTY);
        if (!ok) break;
        if constexpr (C::NPANEL == 1) {
          // one copy for the whole batch run (the map's box spans VB batch entries; entries beyond B arrive as zeros)
          mbar_expect_tx(v_full, C::VB * C::TILE_BYTES);
          tma_load_4d(smem + C::OFF_V, &mv, v_full, 0, w.J * BLK, h / p.kv_group, w.b0);
        } else {
          mbar_expect_tx(v_full, (w.b1 - w.b0) * C::TILE_BYTES);
          for (int b = w.b0; b < w.b1; ++b)
            for (int pn = 0; pn < C::NPANEL; ++pn)
              tma_load_4d(smem + C::OFF_V + (b - w.b0) * C::TILE_BYTES + pn * C::PANEL_BYTES, &mv, v_full, pn * 64,
                          w.J * BLK, h / p.kv_group, b);
        }
        ++nv;
        for (int I = w.I0; I < w.I1 && ok; ++I) {
          for (int b = w.b0; b < w.b1; b += C::SB) {
            const int s = ndo % C::NS;
            const int nb = min(C::SB, w.b1 - b);
            ok = mbar_wait(do_empty + s, ((ndo / C::NS) & 1) ^ 1, wc, G_DO_EMPTY);
            if (!ok) break;
            if constexpr (C::NPANEL == 1) {
              mbar_expect_tx(do_full + s, C::STAGE_BYTES);   // (the map's box spans the stage's SB batch entries)
              tma_load_4d(smem + C::OFF_DO + s * C::STAGE_BYTES, &mdo, do_full + s, 0, I * BLK, h, b);
            } else {
              mbar_expect_tx(do_full + s, nb * C::TILE_BYTES);
              for (int e = 0; e < nb; ++e)
                for (int pn = 0; pn < C::NPANEL; ++pn)
                  tma_load_4d(smem + C::OFF_DO + s * C::STAGE_BYTES + e * C::TILE_BYTES + pn * C::PANEL_BYTES, &mdo,
                              do_full + s, pn * 64, I * BLK, h, b + e);
            }
            ++ndo;
          }
        }
      }
    }
  } else if (warp == C::NCW + 1) {
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
      const PgItem w = p.items[it];
      const int ntiles = w.I1 - w.I0, nb = w.b1 - w.b0;
      ok = mbar_wait_warp(v_full, nv & 1, wc, G_V_FULL);
      if (!ok) break;
      ++nv;
      for (int t = 0; t < ntiles && ok; ++t, ++ng) {
        const uint32_t gb = ng & 1;
        ok = mbar_wait_warp(g_free + gb, ((ng >> 1) & 1) ^ 1, wc, G_G_FREE);
        if (!ok) break;
        for (int b = 0; b < nb; b += C::SB) {
          const uint32_t s = ndo % C::NS;
          const int ne = min(C::SB, nb - b);
          ok = mbar_wait_warp(do_full + s, (ndo / C::NS) & 1, wc, G_DO_FULL);
          if (!ok) break;
          ++ndo;
          tc_fence_after();
          if (leader) {
            for (int e = 0; e < ne; ++e) {
              const uint32_t do_lo = lo_k + ((C::OFF_DO + s * C::STAGE_BYTES + e * C::TILE_BYTES) >> 4);
              const uint32_t vb_lo = v_lo + (((b + e) * C::TILE_BYTES) >> 4);
#pragma unroll
              for (int kc = 0; kc < D / 16; ++kc) {
                const uint32_t off = ((kc >> 2) * C::PANEL_BYTES + (kc & 3) * 32) >> 4;
                umma_ss2(tmem + 128 * gb, vb_lo + off, hi_k, do_lo + off, hi_k, idesc, (kc > 0) || (b + e > 0));
              }
            }
            umma_commit(do_empty + s);
            if (b + ne >= nb) {
              umma_commit(g_full + gb);
              if (t == ntiles - 1) umma_commit(v_empty);
            }
          }
          __syncwarp();
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps (512 threads)
    constexpr int NCT = C::NCW * 32;
    const int q4 = warp & 3, hq = warp >> 2;           // lane quarter (32 keys), column quarter (32 queries)
    const int rowl = q4 * 32 + lane;                   // key row within the block = TMEM lane
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    // Tables of a tile, two sets used in turn: r2raw[256] rho' over the tile's band of distances, z2s[128] logZ' and
    // dl[128] the batch-summed delta of the tile's queries.  A tile's set is fetched into registers while the tile
    // before it is computed and stored after it, so that the global-load latency stays off the tile's path.
    uint32_t ng = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end; ++it) {
      const PgItem w = p.items[it];
      const int h = p.hlist[w.hf];
      const int ntiles = w.I1 - w.I0;
      const int key = w.J * BLK + rowl;
      const float* alpha_h = p.alpha + static_cast<size_t>(h) * p.Tp;
      const float* rho_h = p.rho + static_cast<size_t>(h) * p.Tp;
      const float* logz_h = p.logZ + static_cast<size_t>(h) * p.Tp;
      const float* delta_ch = p.delta + (static_cast<size_t>(w.b0 / C::VB) * p.H + h) * p.T;
      const float a2 = (key < p.T) ? alpha_h[key] * LOG2E_P : -INFINITY;
      float dacc = 0.0f;                               // dalpha(key) of this item (this thread's query quarter)
      bool leave = false;
      // what this thread contributes to the tables of query block I (threads 0-255: r2raw; 256-383: z2s and dl)
      auto fetch = [&](int I, float& v0, float& v1) {
        if (tid < 256) {
          const int d = (I - w.J) * BLK - 127 + tid;   // band: distances d0 .. d0+254, index x = q - row + 127
          v0 = (tid < 255 && d >= 0 && d < p.T) ? rho_h[d] * LOG2E_P : -INFINITY;
        } else if (tid < 384) {
          const int qi = I * BLK + tid - 256;
          v0 = (qi < p.T) ? logz_h[qi] * LOG2E_P : INFINITY;
          v1 = (qi < p.T) ? delta_ch[qi] : 0.0f;
        }
      };
      auto put = [&](uint32_t set, float v0, float v1) {
        float* t0 = tab + set * 512;
        if (tid < 256) {
          t0[tid] = v0;
        } else if (tid < 384) {
          t0[tid] = v0;                                // z2s = t0 + 256
          t0[tid + 128] = v1;                          // dl = t0 + 384
        }
      };
      float n0 = 0.0f, n1 = 0.0f;
      fetch(w.I0, n0, n1);
      put(ng & 1, n0, n1);
      for (int t = 0; t < ntiles; ++t, ++ng) {
        // this tile's tables are written and the other set's readers are done; the warps also agree whether to go on
        if (named_bar_or(1, NCT, !ok)) {
          ok = false;
          leave = true;
          break;
        }
        const int I = w.I0 + t;
        const int tj = I - w.J;                        // tile's distance from the diagonal, in blocks
        if (t + 1 < ntiles) fetch(I + 1, n0, n1);
        const float* r2raw = tab + (ng & 1) * 512;
        const float* z2s = r2raw + 256;
        const float* dl = r2raw + 384;
        const uint32_t gb = ng & 1;
        if (!mbar_wait_warp(g_full + gb, (ng >> 1) & 1, wc, G_G_FULL)) ok = false;
        tc_fence_after();
        const uint32_t t_g = tmem + lane_base + 128 * gb + 32 * hq;
        // Diagonal sums without a serial chain: the entry of column e that lane l' fetches from lane (l' + e) mod 32
        // lies on diagonal x = 31 - l' (no wrap) or 63 - l' (wrap) of the warp's 32 x 32 sub-tile, whatever e is, so
        // every lane sums two diagonals with independent shuffles.
        float dg[2] = {0.0f, 0.0f};
        {
          uint32_t r[32];
          tmem_ld32(t_g, r);
          tmem_wait_ld();
          tc_fence_before();
          warp_arrive(g_free + gb);                    // the tensor core may overwrite this buffer
          const int q0 = 32 * hq;
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
              if (lane + e < 32) dg[0] += got;
              else dg[1] += got;
            }
          }
        }
        if (ok) {
          // lane l' holds the diagonals x = 31 - l' and 63 - l' (x = column - key lane + 31 within this warp's
          // 32 keys x 32 queries); distance d = (I - J) 128 + 32 hq - 32 q4 + x - 31
          float* drho_h = p.drho + static_cast<size_t>(h) * p.Tp;
          const int dbase = tj * BLK + 32 * hq - 32 * q4 - lane;
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const int d = dbase + 32 * k;
            if (d >= 0 && d < p.T && (k < 1 || lane > 0)) atomicAdd(drho_h + d, dg[k]);
          }
        }
        if (t + 1 < ntiles) put((ng + 1) & 1, n0, n1);
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
  if (warp == C::NCW + 1) tmem_dealloc(tmem, C::TMEM_COLS);
}

// delta[c][h][t] = sum over the batch entries b of chunk c (VB consecutive entries) of sum_f dO[b][h][t][f] O[b][h][t][f]
// for the frozen heads (hlist); TPR threads per row, eight features each (16 threads with four idle ones at D = 96, so
// that a row stays inside a warp).
template <int D, int TPR, bool OF32>
__global__ void __launch_bounds__(256) saf_rowdot_kernel(const void* __restrict__ O,
                                                         const __nv_bfloat16* __restrict__ dO, int64_t s0, int64_t s1,
                                                         int64_t s2, const int* __restrict__ hlist,
                                                         float* __restrict__ delta, int B, int H, int Hf, int T, int VB) {
  const long long gid = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long rowid = gid / TPR;               // over [chunks][Hf][T]
  const int part = static_cast<int>(gid % TPR);
  const int nbc = (B + VB - 1) / VB;
  const bool inrange = rowid < static_cast<long long>(nbc) * Hf * T;
  float acc = 0.0f;
  int c = 0, h = 0, t = 0;
  if (inrange) {
    t = static_cast<int>(rowid % T);
    h = hlist[(rowid / T) % Hf];
    c = static_cast<int>(rowid / (static_cast<long long>(T) * Hf));
  }
  if (inrange && part * 8 < D) {
    const int b1 = min(B, (c + 1) * VB);
#pragma unroll 4
    for (int b = c * VB; b < b1; ++b) {
      const int64_t off = b * s0 + h * s1 + static_cast<int64_t>(t) * s2 + part * 8;
      const uint4 d4 = *reinterpret_cast<const uint4*>(dO + off);
      const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&d4);
      if constexpr (OF32) {
        const float* of = static_cast<const float*>(O) + off;
        const float4 oa = *reinterpret_cast<const float4*>(of), ob = *reinterpret_cast<const float4*>(of + 4);
        const float ov[8] = {oa.x, oa.y, oa.z, oa.w, ob.x, ob.y, ob.z, ob.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 df = __bfloat1622float2(d2[e]);
          acc = fmaf(ov[2 * e], df.x, acc);
          acc = fmaf(ov[2 * e + 1], df.y, acc);
        }
      } else {
        const uint4 o4 = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(O) + off);
        const __nv_bfloat162* o2 = reinterpret_cast<const __nv_bfloat162*>(&o4);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 of = __bfloat1622float2(o2[e]), df = __bfloat1622float2(d2[e]);
          acc = fmaf(of.x, df.x, acc);
          acc = fmaf(of.y, df.y, acc);
        }
      }
    }
  }
#pragma unroll
  for (int o = TPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (inrange && part == 0) delta[(static_cast<size_t>(c) * H + h) * T + t] = acc;
}

cudaError_t launch_rowdot(const void* O, int o_f32, const void* dO, const int64_t* os, const int* hlist, float* delta,
                          int B, int H, int Hf, int T, int D, cudaStream_t st) {
  const int tpr = D == 96 ? 16 : D / 8;
  const int vb = pgrad_batch_chunk(D);
  const long long nthreads = static_cast<long long>((B + vb - 1) / vb) * Hf * T * tpr;
  const unsigned grid = static_cast<unsigned>((nthreads + 255) / 256);
#define SAF_ROWDOT(DD, TT, FF) \
  saf_rowdot_kernel<DD, TT, FF><<<grid, 256, 0, st>>>(O, static_cast<const __nv_bfloat16*>(dO), os[0], os[1], os[2], \
                                                      hlist, delta, B, H, Hf, T, vb)
  if (D == 64) { if (o_f32) SAF_ROWDOT(64, 8, true); else SAF_ROWDOT(64, 8, false); }
  else if (D == 96) { if (o_f32) SAF_ROWDOT(96, 16, true); else SAF_ROWDOT(96, 16, false); }
  else { if (o_f32) SAF_ROWDOT(128, 16, true); else SAF_ROWDOT(128, 16, false); }
#undef SAF_ROWDOT
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
