// Forward of the hybrid causal attention layer on sm_100a: one persistent kernel for ordinary
// (flash-style online softmax) and frozen (pattern rebuilt from alpha/rho/logZ) heads.
//
// Per CTA (320 threads): warps 0-7 = compute, warp 8 = TMA producer, warp 9 = tcgen05 issuer and TMEM
// owner.  Two compute threads share a query row (= TMEM lane): warps 0-3 own key columns 0-63 of a
// tile, warps 4-7 columns 64-127; row maxima and row sums are exchanged through shared memory.  Two
// CTAs share an SM, so one CTA's softmax and bookkeeping overlap the other's MMAs.
// TMEM columns: [0,128) S (fp32) / P (bf16 pairs in [0,32) and [64,96): each warp writes into the
// columns it has consumed itself), [128,128+D) O accumulator.
//
// Ordinary item (b,h,I): for J = 0..I: S = Q_I K_J^T (tcgen05, operands in 128B-swizzled smem via TMA),
//   row max / lazy rescale / exp2 / row sum in registers, P -> TMEM as bf16, O += P V_J (A from TMEM,
//   V as MN-major B); epilogue O / l and LSE.
// Frozen item (b,h,I): for J = 0..I: P^(i,j) = exp(alpha(j) + rho(i-j) - logZ(i)) for j <= i
//   (Eq. "compact-prior" with the stored normaliser) generated into TMEM, O += P^ V_J.  No Q/K loads,
//   no score MMA, no max/sum.  The exponential is factorised per tile as
//   w(i) * a(j) * r(i-j) with a = exp(alpha - max_tile alpha), r = exp(rho - max_band rho),
//   w = exp(max alpha + max rho - logZ(i)); a tile whose exponent range would leave fp32 falls back to
//   one exp per element.
// Frozen item, tensor-core form (pattern tables prepared and the head's flag set): with global maxima,
//   O = diag(w) R (diag(a) V), R(i,j) = r(i-j).  A tile of R with reversed rows is a Hankel matrix that the
//   tensor core reads straight from a 4 KB band table (no-swizzle descriptor, both strides 128 bytes), so
//   a tile is one bulk copy of the band, one TMA load of the a-scaled V tile and 8 MMAs; the compute warps
//   only scale the finished rows by w(i) (TMEM lane m holds query 127-m of the block).
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

#define TRF(role, id)

SAF_SPAN_DEFINE(fwd128)

namespace saf {

constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;

template <int D>
struct FwdCfg {
  static constexpr int NPANEL = D / 64;                 // 64-column bf16 panels: 128-byte rows, one swizzle atom
  static constexpr int PANEL_BYTES = 128 * 64 * 2;      // 16 KB
  static constexpr int TILE_BYTES = NPANEL * PANEL_BYTES;
  static constexpr int NS = (D == 64) ? 2 : 1;          // K and V ring depth
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = TILE_BYTES;
  static constexpr int OFF_V = OFF_K + NS * TILE_BYTES;
  static constexpr int OFF_TAB = OFF_V + NS * TILE_BYTES;
  // floats: aJ[128] rband[256] a2raw[128] r2raw[256] red[32] xch[2][2][128] lx[2][128]
  static constexpr int TAB_FLOATS = 128 + 256 + 128 + 256 + 32 + 512 + 256;
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  static constexpr int NBAR = 2 + 4 * NS + 4;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;   // + slack for 1024-byte alignment
  static constexpr int TMEM_COLS = 256;
  static constexpr int COL_S = 0, COL_P = 0, COL_O = 128;
  static constexpr int NTHREADS = 320;
  // A thread keeps its 64 scores in registers between the max and the exp pass (reading them from TMEM
  // twice instead measured almost twice as slow at D = 128).
  static constexpr bool SCORES_IN_REGS = true;
};

enum FwdSite { SITE_Q_EMPTY = 1, SITE_K_EMPTY, SITE_V_EMPTY, SITE_Q_FULL, SITE_K_FULL, SITE_P_FULL, SITE_V_FULL,
               SITE_O_FREE, SITE_S_FULL, SITE_PV_DONE };

template <int D>
__global__ void __launch_bounds__(320, 2)
saf_fwd_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
               const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mvt, const FwdParams p) {
  using C = FwdCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* q_full = bars;
  uint64_t* q_empty = bars + 1;
  uint64_t* k_full = bars + 2;
  uint64_t* k_empty = k_full + C::NS;
  uint64_t* v_full = k_empty + C::NS;
  uint64_t* v_empty = v_full + C::NS;
  uint64_t* s_full = v_empty + C::NS;
  uint64_t* p_full = s_full + 1;
  uint64_t* pv_done = p_full + 1;
  uint64_t* o_free = pv_done + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_free + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* tab = reinterpret_cast<float*>(smem + C::OFF_TAB);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  SAF_SPAN(fwd128, 0);
  int tr_n = 0;
  (void)tr_n;

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(q_full, 1);
    mbar_init(q_empty, 1);
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(k_full + s, 1);
      mbar_init(k_empty + s, 1);
      mbar_init(v_full + s, 1);
      mbar_init(v_empty + s, 1);
    }
    mbar_init(s_full, 1);
    mbar_init(p_full, 8);                        // one arrival per compute warp
    mbar_init(pv_done, 1);
    mbar_init(o_free, 8);
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
  // the prologue above overlapped the previous kernel's tail; global memory is touched only from here on
  pdl_launch_dependents();
  pdl_wait();

  const int it_begin = p.cta_offsets[blockIdx.x], it_end = p.cta_offsets[blockIdx.x + 1];

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mq);
      tma_prefetch_desc(&mk);
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mvt);
      uint32_t nq = 0, nk = 0, nv = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const WorkItem w = p.items[it];
        const int ntiles = w.blk + 1;
        if (w.kind == KIND_FROZEN && p.band_f != nullptr && p.fast_ok[w.h] != 0 && p.ovf[w.h] != p.call_id) {
          // tensor-core form: per tile the Hankel band of distance block (I - J) and the scaled V tile
          const int ord = p.hord[w.h];
          const uint8_t* bands = static_cast<const uint8_t*>(p.band_f) + static_cast<size_t>(w.h) * p.nblkp * 4096;
          for (int j = 0; j < ntiles; ++j) {
            const int sk = nk % C::NS;
            ok = mbar_wait(k_empty + sk, ((nk / C::NS) & 1) ^ 1, wc, SITE_K_EMPTY);
            if (!ok) break;
            mbar_expect_tx(k_full + sk, 4096);
            bulk_load(smem + C::OFF_K + sk * C::TILE_BYTES, bands + static_cast<size_t>(w.blk - j) * 4096, 4096,
                      k_full + sk);
            ++nk;
            const int sv = nv % C::NS;
            ok = mbar_wait(v_empty + sv, ((nv / C::NS) & 1) ^ 1, wc, SITE_V_EMPTY);
            if (!ok) break;
            mbar_expect_tx(v_full + sv, C::TILE_BYTES);
            for (int pn = 0; pn < C::NPANEL; ++pn)
              tma_load_4d(smem + C::OFF_V + sv * C::TILE_BYTES + pn * C::PANEL_BYTES, &mvt, v_full + sv, pn * 64,
                          j * BLK, ord, w.b);
            ++nv;
          }
          continue;
        }
        if (w.kind == KIND_ORDINARY) {
          ok = mbar_wait(q_empty, (nq & 1) ^ 1, wc, SITE_Q_EMPTY);
          if (!ok) break;
          mbar_expect_tx(q_full, C::TILE_BYTES);
          for (int pn = 0; pn < C::NPANEL; ++pn)
            tma_load_4d(smem + C::OFF_Q + pn * C::PANEL_BYTES, &mq, q_full, pn * 64, w.blk * BLK,
                        p.qslot ? p.qslot[w.h] : w.h, w.b);
          ++nq;
        }
        for (int j = 0; j < ntiles && ok; ++j) {
          if (w.kind == KIND_ORDINARY) {
            const int s = nk % C::NS;
            ok = mbar_wait(k_empty + s, ((nk / C::NS) & 1) ^ 1, wc, SITE_K_EMPTY);
            if (!ok) break;
            mbar_expect_tx(k_full + s, C::TILE_BYTES);
            for (int pn = 0; pn < C::NPANEL; ++pn)
              tma_load_4d(smem + C::OFF_K + s * C::TILE_BYTES + pn * C::PANEL_BYTES, &mk, k_full + s, pn * 64,
                          j * BLK, p.qslot ? p.qslot[w.h] : w.h / p.kv_group, w.b);
            ++nk;
          }
          const int s = nv % C::NS;
          ok = mbar_wait(v_empty + s, ((nv / C::NS) & 1) ^ 1, wc, SITE_V_EMPTY);
          if (!ok) break;
          mbar_expect_tx(v_full + s, C::TILE_BYTES);
          for (int pn = 0; pn < C::NPANEL; ++pn)
            tma_load_4d(smem + C::OFF_V + s * C::TILE_BYTES + pn * C::PANEL_BYTES, &mv, v_full + s, pn * 64,
                        j * BLK, w.h / p.kv_group, w.b);
          ++nv;
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ tcgen05 issuer
    // The whole warp walks the loops (warp-uniform operands); one elected lane issues.
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t idesc_s = umma_idesc_bf16(128, 128, 0, 0);
    // (head dimension 96 runs here with features 96..127 zero-filled by TMA: its MMAs skip the two empty k-steps of
    // the scores and produce only 96 output columns)
    const uint32_t idesc_o = umma_idesc_bf16(128, p.d_real, 0, 1);
    const int nk16 = p.d_real / 16;
    const uint32_t idesc_hk = umma_idesc_f16(128, p.d_real, 0, 1);  // tensor-core frozen form: fp16 band x fp16 scaled V
    uint32_t nq = 0, nk = 0, nv = 0, np = 0, nitem = 0;
    bool ok = true;
    // descriptor halves for smem offset 0: K-major tiles (k-step +32 B within a 64-column panel) and
    // the MN-major V tile (k-step +2048 B, LBO = panel stride)
    const uint64_t d_kmaj = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_mn = umma_smem_desc(sb, C::PANEL_BYTES, 1024, UMMA_LAYOUT_SW128);
    const uint32_t lo_k = desc_lo(d_kmaj), hi_k = desc_hi(d_kmaj), lo_m = desc_lo(d_mn), hi_m = desc_hi(d_mn);
    const uint32_t q_lo = lo_k + (C::OFF_Q >> 4);
    // Hankel band: no-swizzle K-major, core matrices 128 bytes apart in both directions
    const uint64_t d_band = umma_smem_desc(sb, 128, 128, UMMA_LAYOUT_NONE);
    const uint32_t lo_b = desc_lo(d_band), hi_b = desc_hi(d_band);
    for (int it = it_begin; it < it_end && ok; ++it, ++nitem) {
      const WorkItem w = p.items[it];
      const int ntiles = w.blk + 1;
      const bool ord = w.kind == KIND_ORDINARY;
      if (w.kind == KIND_FROZEN && p.band_f != nullptr && p.fast_ok[w.h] != 0 && p.ovf[w.h] != p.call_id) {
        for (int j = 0; j < ntiles && ok; ++j) {
          const uint32_t sk = nk % C::NS, sv = nv % C::NS;
          ok = mbar_wait_warp(k_full + sk, (nk / C::NS) & 1, wc, SITE_K_FULL);
          if (!ok) break;
          ++nk;
          ok = mbar_wait_warp(v_full + sv, (nv / C::NS) & 1, wc, SITE_V_FULL);
          if (!ok) break;
          ++nv;
          if (j == 0) {
            ok = mbar_wait_warp(o_free, (nitem & 1) ^ 1, wc, SITE_O_FREE);
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t band_lo = lo_b + ((C::OFF_K + sk * C::TILE_BYTES) >> 4);
          const uint32_t v_lo = lo_m + ((C::OFF_V + sv * C::TILE_BYTES) >> 4);
          const uint32_t acc0 = j > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ss2(tmem + C::COL_O, band_lo + 16 * kc, hi_b, v_lo + 128 * kc, hi_m, idesc_hk, kc > 0 ? 1u : acc0);
            umma_commit(k_empty + sk);
            umma_commit(v_empty + sv);
            if (j == ntiles - 1) umma_commit(pv_done);
          }
          __syncwarp();
        }
        continue;
      }
      if (ord) {
        ok = mbar_wait_warp(q_full, nq & 1, wc, SITE_Q_FULL);
        if (!ok) break;
        ++nq;
      }
      for (int j = 0; j < ntiles && ok; ++j) {
        if (ord) {
          const uint32_t s = nk % C::NS;
          TRF(0, 1);
          ok = mbar_wait_warp(k_full + s, (nk / C::NS) & 1, wc, SITE_K_FULL);
          if (!ok) break;
          ++nk;
          tc_fence_after();
          TRF(0, 2);
          const uint32_t k_lo = lo_k + ((C::OFF_K + s * C::TILE_BYTES) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < D / 16; ++kc) {
              if (kc >= nk16) break;
              const uint32_t off = ((kc >> 2) * C::PANEL_BYTES + (kc & 3) * 32) >> 4;
              umma_ss2(tmem + C::COL_S, q_lo + off, hi_k, k_lo + off, hi_k, idesc_s, kc > 0);
            }
            umma_commit(s_full);
            umma_commit(k_empty + s);
            if (j == ntiles - 1) umma_commit(q_empty);
          }
          __syncwarp();
          TRF(0, 3);
        }
        ok = mbar_wait_warp(p_full, np & 1, wc, SITE_P_FULL);
        if (!ok) break;
        ++np;
        TRF(0, 4);
        const uint32_t s = nv % C::NS;
        ok = mbar_wait_warp(v_full + s, (nv / C::NS) & 1, wc, SITE_V_FULL);
        if (!ok) break;
        ++nv;
        if (j == 0) {
          ok = mbar_wait_warp(o_free, (nitem & 1) ^ 1, wc, SITE_O_FREE);
          if (!ok) break;
        }
        tc_fence_after();
        TRF(0, 5);
        const uint32_t v_lo = lo_m + ((C::OFF_V + s * C::TILE_BYTES) >> 4);
        const uint32_t acc0 = j > 0 ? 1u : 0u;
        if (leader) {
          // bf16 P pairs: keys 0-63 in columns [0,32), keys 64-127 in columns [64,96)
#pragma unroll
          for (int kc = 0; kc < 8; ++kc)
            umma_ts2(tmem + C::COL_O, tmem + C::COL_P + 8 * kc + (kc >= 4 ? 32u : 0u), v_lo + 128 * kc, hi_m, idesc_o,
                     kc > 0 ? 1u : acc0);
          umma_commit(v_empty + s);
          umma_commit(pv_done);
        }
        __syncwarp();
        TRF(0, 6);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps (256 threads)
    const int q4 = warp & 3, hh = warp >> 2;
    const int rowl = q4 * 32 + lane;                   // query row within the tile = TMEM lane
    const int pair_bar = 1 + q4;                       // named barrier of the two warps sharing this lane quarter
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const uint32_t t_s = tmem + lane_base + C::COL_S + 64 * hh;       // this thread's 64 score columns
    const uint32_t t_p = tmem + lane_base + C::COL_P + 64 * hh;       // ... and where its bf16 pairs go
    const uint32_t t_o = tmem + lane_base + C::COL_O + (D / 2) * hh;  // this thread's half of the O row
    float* aJ = tab;
    float* rband = tab + 128;
    float* a2raw = tab + 384;
    float* r2raw = tab + 512;
    float* red = tab + 768;
    float* xch = tab + 800;                            // [tile parity][hh][row]
    float* lx = tab + 1312;                            // [hh][row]
    uint32_t ns = 0, npv = 0;
    bool ok = true;
    const int trr = 1 + hh;
    (void)trr;
    // A compute warp whose wait was abandoned keeps walking (without storing) until the next
    // agreement barrier, where all eight leave together; none is ever left alone at a barrier.
    for (int it = it_begin; it < it_end; ++it) {
      const WorkItem w = p.items[it];
      const int ntiles = w.blk + 1;
      int row = w.blk * BLK + rowl;
      float inv_l = 1.0f, lse = 0.0f;
      if (named_bar_or(5, 256, !ok)) break;
      if (w.kind == KIND_FROZEN && p.band_f != nullptr && p.fast_ok[w.h] != 0 && p.ovf[w.h] != p.call_id) {
        // tensor-core form: nothing to do per tile; lane m holds query 127-m, scaled by w(i) below
        row = w.blk * BLK + 127 - rowl;
        inv_l = (row < p.T) ? p.wvec[static_cast<size_t>(w.h) * p.Tp + row] * (1.0f / (HK_BAND_SCALE * HK_A_SCALE)) : 0.0f;
      } else if (w.kind == KIND_ORDINARY) {
        float m_ref = -INFINITY, l = 0.0f;
        const float c = p.scale_log2;
        for (int j = 0; j < ntiles; ++j) {
          TRF(trr, 11);
          if (!mbar_wait_warp(s_full, ns & 1, wc, SITE_S_FULL)) ok = false;
          ++ns;
          if (j > 0) {
            if (!mbar_wait_warp(pv_done, npv & 1, wc, SITE_PV_DONE)) ok = false;
            ++npv;
          }
          tc_fence_after();
          TRF(trr, 12);
          const bool diag = (j == w.blk);
          uint32_t r0[C::SCORES_IN_REGS ? 32 : 1], r1[C::SCORES_IN_REGS ? 32 : 1];
          float mx;
          if constexpr (C::SCORES_IN_REGS) {
            tmem_ld32(t_s, r0);
            tmem_ld32(t_s + 32, r1);
            tmem_wait_ld();
            if (diag) {
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                if (64 * hh + e > rowl) r0[e] = 0xff800000u;        // -inf above the diagonal
                if (64 * hh + 32 + e > rowl) r1[e] = 0xff800000u;
              }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              mx0 = fmaxf(mx0, __uint_as_float(r0[e]));
              mx1 = fmaxf(mx1, __uint_as_float(r1[e]));
            }
            mx = fmaxf(mx0, mx1);
          } else {
            mx = -INFINITY;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              uint32_t r[32];
              tmem_ld32(t_s + 32 * cc, r);
              tmem_wait_ld();
              float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                float s0 = __uint_as_float(r[2 * e]), s1 = __uint_as_float(r[2 * e + 1]);
                if (diag) {
                  if (64 * hh + 32 * cc + 2 * e > rowl) s0 = -INFINITY;
                  if (64 * hh + 32 * cc + 2 * e + 1 > rowl) s1 = -INFINITY;
                }
                m0 = fmaxf(m0, s0);
                m1 = fmaxf(m1, s1);
              }
              mx = fmaxf(mx, fmaxf(m0, m1));
            }
          }
          TRF(trr, 13);
          // row maximum over both column halves
          float* xs = xch + (j & 1) * 256;
          xs[hh * 128 + rowl] = mx;
          named_bar_sync(pair_bar, 64);
          mx = fmaxf(mx, xs[(hh ^ 1) * 128 + rowl]);
          TRF(trr, 14);
          const float m_new = fmaxf(m_ref, mx * c);
          if (j == 0) {
            m_ref = m_new;
          } else {
            const bool need = (m_new - m_ref) > 8.0f;
            if (__any_sync(0xffffffffu, need)) {
              const float f = need ? ex2_approx(m_ref - m_new) : 1.0f;
              l *= f;
              if (need) m_ref = m_new;
#pragma unroll
              for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t r[16];
                tmem_ld16(t_o + 16 * cc, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
                tmem_st16(t_o + 16 * cc, r);
              }
            }
          }
          const float neg_m = -m_ref;
          float l0 = 0.0f, l1 = 0.0f;
          if constexpr (C::SCORES_IN_REGS) {
            uint32_t pk0[16], pk1[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float a0 = ex2_approx(fmaf(__uint_as_float(r0[2 * e]), c, neg_m));
              const float a1 = ex2_approx(fmaf(__uint_as_float(r0[2 * e + 1]), c, neg_m));
              const float b0 = ex2_approx(fmaf(__uint_as_float(r1[2 * e]), c, neg_m));
              const float b1 = ex2_approx(fmaf(__uint_as_float(r1[2 * e + 1]), c, neg_m));
              l0 += a0 + a1;
              l1 += b0 + b1;
              pk0[e] = pack_bf16x2(a0, a1);
              pk1[e] = pack_bf16x2(b0, b1);
            }
            tmem_st16(t_p, pk0);
            tmem_st16(t_p + 16, pk1);
          } else {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
              uint32_t r[32];
              tmem_ld32(t_s + 32 * cc, r);
              tmem_wait_ld();
              uint32_t pk[16];
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                float a0 = ex2_approx(fmaf(__uint_as_float(r[2 * e]), c, neg_m));
                float a1 = ex2_approx(fmaf(__uint_as_float(r[2 * e + 1]), c, neg_m));
                if (diag) {
                  if (64 * hh + 32 * cc + 2 * e > rowl) a0 = 0.0f;
                  if (64 * hh + 32 * cc + 2 * e + 1 > rowl) a1 = 0.0f;
                }
                l0 += a0;
                l1 += a1;
                pk[e] = pack_bf16x2(a0, a1);
              }
              tmem_st16(t_p + 16 * cc, pk);
            }
          }
          l += l0 + l1;
          TRF(trr, 15);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(p_full);
          TRF(trr, 16);
        }
        // row sum over both column halves
        lx[hh * 128 + rowl] = l;
        named_bar_sync(pair_bar, 64);
        l += lx[(hh ^ 1) * 128 + rowl];
        inv_l = 1.0f / l;
        lse = (m_ref + log2f(l)) * LN2_F;
      } else {
        // ---------------- frozen head: generate P^ tiles
        const float* alpha_h = p.alpha + static_cast<size_t>(w.h) * p.Tp;
        const float* rho_h = p.rho + static_cast<size_t>(w.h) * p.Tp;
        const float z2 = (row < p.T) ? p.logZ[static_cast<size_t>(w.h) * p.Tp + row] * LOG2E_F : INFINITY;
        bool leave = false;
        for (int j = 0; j < ntiles; ++j) {
          // previous tile's table readers are done; the compute warps also agree whether to go on
          if (named_bar_or(5, 256, !ok)) {
            ok = false;
            leave = true;
            break;
          }
          const int d0 = (w.blk - j) * BLK - 127;      // band covers distances d0 .. d0+254
          float a2 = -INFINITY, r2 = -INFINITY;
          if (tid < 128) {
            const int key = j * BLK + tid;
            if (key < p.T) a2 = alpha_h[key] * LOG2E_F;
            a2raw[tid] = a2;
          }
          {
            const int d = d0 + tid;                    // one band entry per compute thread (255 used)
            if (tid < 255 && d >= 0 && d < p.T) r2 = rho_h[d] * LOG2E_F;
            r2raw[tid] = r2;
          }
          float ma = a2, mr = r2;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, o));
            mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o));
          }
          if (lane == 0) {
            red[warp] = ma;                            // warps 4-7 contribute -inf
            red[8 + warp] = mr;
          }
          named_bar_sync(6, 256);
          ma = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
          mr = fmaxf(fmaxf(fmaxf(red[8], red[9]), fmaxf(red[10], red[11])),
                     fmaxf(fmaxf(red[12], red[13]), fmaxf(red[14], red[15])));
          const float ew = ma + mr - z2;               // -inf for rows beyond T
          const unsigned anybad = __any_sync(0xffffffffu, ew > 100.0f);   // factorised form would overflow / flush
          if (lane == 0) red[16 + warp] = anybad ? 1.0f : 0.0f;
          if (tid < 128) aJ[tid] = ex2_approx(a2 - ma);
          rband[tid] = ex2_approx(r2 - mr);
          named_bar_sync(7, 256);
          const bool exact = (red[16] + red[17] + red[18] + red[19] + red[20] + red[21] + red[22] + red[23]) > 0.0f;
          if (j > 0) {
            if (!mbar_wait_warp(pv_done, npv & 1, wc, SITE_PV_DONE)) ok = false;   // previous P^ tile consumed
            ++npv;
            tc_fence_after();
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int k0c = 64 * hh + 32 * cc;         // first key column of this chunk
            uint32_t pk[16];
            if (!exact) {
              const float wv = ex2_approx(ew);
              const float* rb = rband + rowl + 127;    // rb[-k] = r(distance of key k in this tile)
#pragma unroll
              for (int e4 = 0; e4 < 8; ++e4) {
                const int k0 = k0c + 4 * e4;
                const float4 a4 = *reinterpret_cast<const float4*>(aJ + k0);
                const float p0 = wv * a4.x * rb[-k0], p1 = wv * a4.y * rb[-k0 - 1];
                const float p2 = wv * a4.z * rb[-k0 - 2], p3 = wv * a4.w * rb[-k0 - 3];
                pk[2 * e4] = pack_bf16x2(p0, p1);
                pk[2 * e4 + 1] = pack_bf16x2(p2, p3);
              }
            } else {
              const float* rb = r2raw + rowl + 127;
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                const int k0 = k0c + 2 * e;
                const float p0 = ex2_approx(a2raw[k0] + rb[-k0] - z2);
                const float p1 = ex2_approx(a2raw[k0 + 1] + rb[-k0 - 1] - z2);
                pk[e] = pack_bf16x2(p0, p1);
              }
            }
            tmem_st16(t_p + 16 * cc, pk);
          }
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(p_full);
        }
        if (leave) break;
      }
      // ---------------- epilogue: wait for the last P V, scale, store this thread's half of the row
      if (!mbar_wait_warp(pv_done, npv & 1, wc, SITE_PV_DONE)) ok = false;
      ++npv;
      tc_fence_after();
      __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.O) + w.b * p.o_strides[0] + w.h * p.o_strides[1] +
                            static_cast<int64_t>(row) * p.o_strides[2] + (D / 2) * hh;
#pragma unroll
      for (int cc = 0; cc < D / 64; ++cc) {
        uint32_t r[32];
        tmem_ld32(t_o + 32 * cc, r);
        tmem_wait_ld();
        if (row < p.T && ok && p.o_f32) {
          float* orow32 = static_cast<float*>(p.O) + w.b * p.o_strides[0] + w.h * p.o_strides[1] +
                          static_cast<int64_t>(row) * p.o_strides[2] + (D / 2) * hh + 32 * cc;
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if ((D / 2) * hh + 32 * cc + 4 * g < p.d_real)
              *reinterpret_cast<float4*>(orow32 + 4 * g) =
                  make_float4(__uint_as_float(r[4 * g + 0]) * inv_l, __uint_as_float(r[4 * g + 1]) * inv_l,
                              __uint_as_float(r[4 * g + 2]) * inv_l, __uint_as_float(r[4 * g + 3]) * inv_l);
        } else if (row < p.T && ok) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            uint4 o;
            o.x = pack_bf16x2(__uint_as_float(r[8 * g + 0]) * inv_l, __uint_as_float(r[8 * g + 1]) * inv_l);
            o.y = pack_bf16x2(__uint_as_float(r[8 * g + 2]) * inv_l, __uint_as_float(r[8 * g + 3]) * inv_l);
            o.z = pack_bf16x2(__uint_as_float(r[8 * g + 4]) * inv_l, __uint_as_float(r[8 * g + 5]) * inv_l);
            o.w = pack_bf16x2(__uint_as_float(r[8 * g + 6]) * inv_l, __uint_as_float(r[8 * g + 7]) * inv_l);
            if ((D / 2) * hh + 32 * cc + 8 * g < p.d_real) *reinterpret_cast<uint4*>(orow + 32 * cc + 8 * g) = o;
          }
        }
      }
      if (p.LSE != nullptr && hh == 0 && row < p.T && ok)
        p.LSE[(static_cast<size_t>(w.b) * p.H + w.h) * p.T + row] = lse;
      tc_fence_before();
      warp_arrive(o_free);
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  if (*abort_flag) {
    // A wait gave up: let copies and MMAs that are still in flight land before the CTA's
    // shared memory and TMEM are released.
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  SAF_SPAN(fwd128, 1);
  if (warp == 9) tmem_dealloc(tmem, C::TMEM_COLS);
}

int fwd_smem_bytes(int D) { return D == 64 ? fwd64_smem_bytes() : FwdCfg<128>::SMEM; }

cudaError_t launch_fwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mvt, const CUtensorMap& mo, const FwdParams& p, int grid, cudaStream_t st) {
  cudaError_t e;
  if (D == 64) {
    return launch_fwd64(mq, mk, mv, mvt, mo, p, grid, st);   // head dimension 64 has its own kernel
  } else {
    e = cudaFuncSetAttribute(saf_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<128>::SMEM);
    if (e != cudaSuccess) return e;
    return launch_pdl(PDL_FWD, saf_fwd_kernel<128>, dim3(grid), dim3(320), FwdCfg<128>::SMEM, st, mq, mk, mv, mvt, p);
  }
}

}  // namespace saf
