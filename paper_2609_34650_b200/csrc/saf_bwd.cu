// Backward of the hybrid causal attention layer on sm_100a (head dimension 64): one persistent
// kernel, one work item per (batch, head, 128-key block J), looping over query blocks I >= J.
//
// CTA = 320 threads: warps 0-7 compute (TMEM lane = key row; warps 0-3 own query columns 0-63 of a
// tile, warps 4-7 columns 64-127), warp 8 TMA producer, warp 9 tcgen05 issuer / TMEM owner.
//
// Ordinary item, per tile (Appendix E.2: key-block programs accumulate dV and dK; dQ here is produced
// by the same tile loop and accumulated across key blocks with fp32 atomics instead of a second pass):
//   S^T  = K_J Q_I^T,  dP^T = V_J dO_I^T                       (tcgen05, smem operands)
//   P^T  = exp(S^T * scale - LSE_i),  dS^T = P^T o (dP^T - delta_i)   (registers; bf16 to TMEM, dS^T also to smem)
//   dV_J += P^T dO_I,  dK_J += dS^T Q_I                        (A from TMEM, dO / Q as MN-major B)
//   dQ_I  = dS K_J                                             (A = dS^T tile in smem read M-major, B = K_J)
// Frozen item, per tile (Sec. 3.3: dV = P^^T dO, no query/key gradients):
//   P^^T(j,i) = exp(alpha(j) + rho(i-j) - logZ(i)) for i >= j, generated into TMEM (factorised as in
//   the forward), dV_J += P^^T dO_I.
//
// TMEM columns: [0,128) S^T / P^T (bf16 pairs in [0,64); frozen P^^T double-buffered in [0,64),[64,128)),
// [128,256) dP^T / dS^T (bf16 pairs in [128,192)), [256,320) dV, [320,384) dK, [384,448) dQ.
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

namespace saf {

namespace {

constexpr float LOG2E_B = 1.4426950408889634f;

struct BwdCfg {
  static constexpr int PANEL = 128 * 64 * 2;         // one [128][64] bf16 tile, 128-byte rows, 16 KB
  static constexpr int NS = 2;                       // Q/dO ring depth
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = PANEL;
  static constexpr int OFF_Q = 2 * PANEL;            // NS stages
  static constexpr int OFF_DO = OFF_Q + NS * PANEL;  // NS stages
  static constexpr int OFF_DS = OFF_DO + NS * PANEL; // two panels: queries 0-63, 64-127
  static constexpr int OFF_TAB = OFF_DS + 2 * PANEL;
  // floats: lse2[128] delta[128] wq[128] z2s[128] rband[256] r2raw[256] red[32]
  static constexpr int TAB_FLOATS = 128 * 4 + 256 * 2 + 32;
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  static constexpr int NBAR = 2 + 2 * NS + 6 + 2;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 512;
  static constexpr int COL_S = 0, COL_DP = 128, COL_DV = 256, COL_DK = 320, COL_DQ = 384;
  static constexpr int NCT = 256;                    // compute threads
};

enum BwdSite { B_KV_EMPTY = 21, B_QDO_EMPTY, B_KV_FULL, B_QDO_FULL, B_PDS_FULL, B_ACC_FREE, B_DQ_FREE, B_SDP_FULL,
               B_DQ_FULL, B_ACC_FULL, B_PFREE };

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

}  // namespace

__global__ void __launch_bounds__(320, 1)
saf_bwd_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
               const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mdo, const BwdParams p) {
  using C = BwdCfg;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* kv_full = bars;
  uint64_t* kv_empty = bars + 1;
  uint64_t* qdo_full = bars + 2;
  uint64_t* qdo_empty = qdo_full + C::NS;
  uint64_t* sdp_full = qdo_empty + C::NS;
  uint64_t* pds_full = sdp_full + 1;
  uint64_t* dq_full = pds_full + 1;
  uint64_t* dq_free = dq_full + 1;
  uint64_t* acc_full = dq_free + 1;
  uint64_t* acc_free = acc_full + 1;
  uint64_t* pfree = acc_free + 1;   // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pfree + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* tab = reinterpret_cast<float*>(smem + C::OFF_TAB);
  float* lse2s = tab;
  float* dels = tab + 128;
  float* wq = tab + 256;
  float* z2s = tab + 384;
  float* rband = tab + 512;
  float* r2raw = tab + 768;
  float* red = tab + 1024;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  const int nblk = (p.T + BLK - 1) / BLK;

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(kv_full, 1);
    mbar_init(kv_empty, 1);
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(qdo_full + s, 1);
      mbar_init(qdo_empty + s, 1);
    }
    mbar_init(sdp_full, 1);
    mbar_init(pds_full, C::NCT);
    mbar_init(dq_full, 1);
    mbar_init(dq_free, C::NCT);
    mbar_init(acc_full, 1);
    mbar_init(acc_free, C::NCT);
    mbar_init(pfree, 1);
    mbar_init(pfree + 1, 1);
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
      tma_prefetch_desc(&mq);
      tma_prefetch_desc(&mk);
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mdo);
      uint32_t nkv = 0, nqdo = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it) {
        const WorkItem w = p.items[it];
        const bool ord = w.kind == KIND_ORDINARY;
        if (ord) {
          ok = mbar_wait(kv_empty, (nkv & 1) ^ 1, wc, B_KV_EMPTY);
          if (!ok) break;
          mbar_expect_tx(kv_full, 2 * C::PANEL);
          tma_load_4d(smem + C::OFF_K, &mk, kv_full, 0, w.blk * BLK, w.h, w.b);
          tma_load_4d(smem + C::OFF_V, &mv, kv_full, 0, w.blk * BLK, w.h, w.b);
          ++nkv;
        }
        for (int I = w.blk; I < nblk; ++I) {
          const int s = nqdo % C::NS;
          ok = mbar_wait(qdo_empty + s, ((nqdo / C::NS) & 1) ^ 1, wc, B_QDO_EMPTY);
          if (!ok) break;
          mbar_expect_tx(qdo_full + s, ord ? 2 * C::PANEL : C::PANEL);
          if (ord) tma_load_4d(smem + C::OFF_Q + s * C::PANEL, &mq, qdo_full + s, 0, I * BLK, w.h, w.b);
          tma_load_4d(smem + C::OFF_DO + s * C::PANEL, &mdo, qdo_full + s, 0, I * BLK, w.h, w.b);
          ++nqdo;
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ tcgen05 issuer
    if (lane == 0) {
      const uint32_t sb = smem_u32(smem);
      constexpr uint32_t id_s = umma_idesc_bf16(128, 128, 0, 0);     // S^T, dP^T: both operands K-major
      constexpr uint32_t id_acc = umma_idesc_bf16(128, 64, 0, 1);    // dV, dK: A from TMEM, B MN-major
      constexpr uint32_t id_dq = umma_idesc_bf16(128, 64, 1, 1);     // dQ: A (dS^T tile) M-major, B MN-major
      uint32_t nkv = 0, nqdo = 0, npds = 0, nitem = 0, ndq = 0;
      bool ok = true;
      for (int it = it_begin; it < it_end && ok; ++it, ++nitem) {
        const WorkItem w = p.items[it];
        const bool ord = w.kind == KIND_ORDINARY;
        if (ord) {
          ok = mbar_wait(kv_full, nkv & 1, wc, B_KV_FULL);
          if (!ok) break;
          ++nkv;
        }
        int t = 0;
        for (int I = w.blk; I < nblk; ++I, ++t) {
          const int s = nqdo % C::NS;
          ok = mbar_wait(qdo_full + s, (nqdo / C::NS) & 1, wc, B_QDO_FULL);
          if (!ok) break;
          ++nqdo;
          tc_fence_after();
          const uint32_t q_s = sb + C::OFF_Q + s * C::PANEL, do_s = sb + C::OFF_DO + s * C::PANEL;
          if (ord) {
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ss(tmem + C::COL_S, umma_smem_desc(sb + C::OFF_K + 32 * kc, 16, 1024, UMMA_LAYOUT_SW128),
                      umma_smem_desc(q_s + 32 * kc, 16, 1024, UMMA_LAYOUT_SW128), id_s, kc > 0);
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ss(tmem + C::COL_DP, umma_smem_desc(sb + C::OFF_V + 32 * kc, 16, 1024, UMMA_LAYOUT_SW128),
                      umma_smem_desc(do_s + 32 * kc, 16, 1024, UMMA_LAYOUT_SW128), id_s, kc > 0);
            umma_commit(sdp_full);
          }
          ok = mbar_wait(pds_full, npds & 1, wc, B_PDS_FULL);
          if (!ok) break;
          ++npds;
          if (t == 0) {
            ok = mbar_wait(acc_free, (nitem & 1) ^ 1, wc, B_ACC_FREE);
            if (!ok) break;
          }
          tc_fence_after();
          // ordinary: P^T pairs sit in columns [0,32) and [64,96); frozen: contiguous in buffer t&1
          const uint32_t pcol = ord ? C::COL_S : (t & 1) * 64;
          const uint32_t hstep = ord ? 32u : 0u;     // extra column offset of k-steps 4..7
#pragma unroll
          for (int kc = 0; kc < 8; ++kc)
            umma_ts(tmem + C::COL_DV, tmem + pcol + 8 * kc + (kc >= 4 ? hstep : 0u),
                    umma_smem_desc(do_s + 2048 * kc, C::PANEL, 1024, UMMA_LAYOUT_SW128), id_acc,
                    (t > 0 || kc > 0) ? 1u : 0u);
          if (ord) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ts(tmem + C::COL_DK, tmem + C::COL_DP + 8 * kc + (kc >= 4 ? 32u : 0u),
                      umma_smem_desc(q_s + 2048 * kc, C::PANEL, 1024, UMMA_LAYOUT_SW128), id_acc,
                      (t > 0 || kc > 0) ? 1u : 0u);
            umma_commit(qdo_empty + s);
            ok = mbar_wait(dq_free, (ndq & 1) ^ 1, wc, B_DQ_FREE);
            if (!ok) break;
            ++ndq;
            tc_fence_after();
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ss(tmem + C::COL_DQ, umma_smem_desc(sb + C::OFF_DS + 2048 * kc, C::PANEL, 1024, UMMA_LAYOUT_SW128),
                      umma_smem_desc(sb + C::OFF_K + 2048 * kc, C::PANEL, 1024, UMMA_LAYOUT_SW128), id_dq, kc > 0);
            umma_commit(dq_full);
          } else {
            umma_commit(qdo_empty + s);
            umma_commit(pfree + (t & 1));
          }
        }
        if (!ok) break;
        if (ord) umma_commit(kv_empty);
        umma_commit(acc_full);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute warps (256 threads)
    const int q4 = warp & 3, half = warp >> 2;
    const int rowl = q4 * 32 + lane;                     // TMEM lane: key row (tile loop) / query row (dQ drain)
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    uint32_t nsdp = 0, ndq = 0, nacc = 0, npf0 = 0, npf1 = 0;
    bool ok = true;
    for (int it = it_begin; it < it_end; ++it) {
      const WorkItem w = p.items[it];
      const bool ord = w.kind == KIND_ORDINARY;
      const int ntiles = nblk - w.blk;
      const int key = w.blk * BLK + rowl;
      const size_t bh = static_cast<size_t>(w.b) * p.H + w.h;
      bool leave = false;
      if (ord) {
        const float c = p.scale_log2;
        for (int t = 0; t < ntiles; ++t) {
          const int I = w.blk + t;
          if (named_bar_or(1, C::NCT, !ok)) {   // uniform over the compute warps: leave together
            ok = false;
            leave = true;
            break;
          }
          if (tid < 128) {
            const int qi = I * BLK + tid;
            lse2s[tid] = (qi < p.T) ? p.LSE[bh * p.T + qi] * LOG2E_B : INFINITY;
            dels[tid] = (qi < p.T) ? p.delta[bh * p.Tpad + qi] : 0.0f;
          }
          // drain dQ of the previous tile while the tensor core works on this tile's S^T / dP^T
          if (t > 0) {
            if (mbar_wait_warp(dq_full, ndq & 1, wc, B_DQ_FULL)) {
              ++ndq;
              tc_fence_after();
              uint32_t r[32];
              tmem_ld32(tmem + lane_base + C::COL_DQ + 32 * half, r);
              tmem_wait_ld();
              const int qi = (I - 1) * BLK + rowl;
              if (qi < p.T && ok) {
                float* dst = p.dQacc + (bh * p.T + qi) * 64 + 32 * half;
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  red_add_v4(dst + 4 * e, __uint_as_float(r[4 * e]) * p.scale, __uint_as_float(r[4 * e + 1]) * p.scale,
                             __uint_as_float(r[4 * e + 2]) * p.scale, __uint_as_float(r[4 * e + 3]) * p.scale);
              }
              tc_fence_before();
              mbar_arrive(dq_free);
            } else {
              ok = false;
            }
          }
          named_bar_sync(1, C::NCT);
          if (!mbar_wait_warp(sdp_full, nsdp & 1, wc, B_SDP_FULL)) ok = false;
          ++nsdp;
          tc_fence_after();
          const bool diag = (t == 0);
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int q0 = 64 * half + 32 * cc;          // first query column of this chunk
            uint32_t rs[32], rd[32];
            tmem_ld32(tmem + lane_base + C::COL_S + q0, rs);
            tmem_ld32(tmem + lane_base + C::COL_DP + q0, rd);
            tmem_wait_ld();
            uint32_t pk[16], dk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int qa = q0 + 2 * e;
              const float2 l2 = *reinterpret_cast<const float2*>(lse2s + qa);
              const float2 de = *reinterpret_cast<const float2*>(dels + qa);
              float p0 = ex2_approx(fmaf(__uint_as_float(rs[2 * e]), c, -l2.x));
              float p1 = ex2_approx(fmaf(__uint_as_float(rs[2 * e + 1]), c, -l2.y));
              if (diag) {                                // causal: query index >= key index
                if (qa < rowl) p0 = 0.0f;
                if (qa + 1 < rowl) p1 = 0.0f;
              }
              const float d0 = p0 * (__uint_as_float(rd[2 * e]) - de.x);
              const float d1 = p1 * (__uint_as_float(rd[2 * e + 1]) - de.y);
              pk[e] = pack_bf16x2(p0, p1);
              dk[e] = pack_bf16x2(d0, d1);
            }
            // bf16 pairs go where this warp has already consumed the fp32 values: queries 0-63 in
            // columns +[0,32), queries 64-127 in columns +[64,96) (the other half's columns are still live)
            tmem_st16(tmem + lane_base + C::COL_S + 64 * half + 16 * cc, pk);
            tmem_st16(tmem + lane_base + C::COL_DP + 64 * half + 16 * cc, dk);
            // dS^T row (this key) -> smem panel `half`, 128-byte swizzle: 16-byte chunk index ^= row & 7
            const uint32_t rowaddr = smem_u32(smem + C::OFF_DS + half * C::PANEL + rowl * 128);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const uint32_t chunk = static_cast<uint32_t>((4 * cc + g) ^ (rowl & 7));
              st_shared_v4(rowaddr + chunk * 16, dk[4 * g], dk[4 * g + 1], dk[4 * g + 2], dk[4 * g + 3]);
            }
          }
          tmem_wait_st();
          fence_proxy_async_smem();
          tc_fence_before();
          mbar_arrive(pds_full);
        }
        // last tile's dQ
        {
          if (!mbar_wait_warp(dq_full, ndq & 1, wc, B_DQ_FULL)) ok = false;
          ++ndq;
          tc_fence_after();
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + C::COL_DQ + 32 * half, r);
          tmem_wait_ld();
          const int qi = (nblk - 1) * BLK + rowl;
          if (qi < p.T && ok) {
            float* dst = p.dQacc + (bh * p.T + qi) * 64 + 32 * half;
#pragma unroll
            for (int e = 0; e < 8; ++e)
              red_add_v4(dst + 4 * e, __uint_as_float(r[4 * e]) * p.scale, __uint_as_float(r[4 * e + 1]) * p.scale,
                         __uint_as_float(r[4 * e + 2]) * p.scale, __uint_as_float(r[4 * e + 3]) * p.scale);
          }
          tc_fence_before();
          mbar_arrive(dq_free);
        }
      } else {
        // ---------------- frozen head: P^^T tiles
        const float* alpha_h = p.alpha + static_cast<size_t>(w.h) * p.Tp;
        const float* rho_h = p.rho + static_cast<size_t>(w.h) * p.Tp;
        const float* logz_h = p.logZ + static_cast<size_t>(w.h) * p.Tp;
        const float a2 = (key < p.T) ? alpha_h[key] * LOG2E_B : -INFINITY;
        float ma = a2;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, o));
        // block maximum of alpha over the 128 keys: exchanged once per item through `red`
        if (named_bar_or(1, C::NCT, !ok)) {
          ok = false;
          break;
        }
        if (lane == 0 && half == 0) red[16 + q4] = ma;
        named_bar_sync(1, C::NCT);
        ma = fmaxf(fmaxf(red[16], red[17]), fmaxf(red[18], red[19]));
        const float aj = ex2_approx(a2 - ma);
        for (int t = 0; t < ntiles; ++t) {
          const int I = w.blk + t;
          if (named_bar_or(1, C::NCT, !ok)) {   // uniform over the compute warps: leave together
            ok = false;
            leave = true;
            break;
          }
          const int d0 = t * BLK - 127;                // band: distances d0 .. d0+254, index x = q - row + 127
          float r2v = -INFINITY;
          {
            const int d = d0 + tid;                    // tid in [0,256): one band entry per compute thread
            if (tid < 255 && d >= 0 && d < p.T) r2v = rho_h[d] * LOG2E_B;
            r2raw[tid] = r2v;
            float mr = r2v;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o));
            if (lane == 0) red[warp] = mr;
          }
          float z2 = INFINITY;
          if (tid < 128) {
            const int qi = I * BLK + tid;
            if (qi < p.T) z2 = logz_h[qi] * LOG2E_B;
            z2s[tid] = z2;
          }
          named_bar_sync(1, C::NCT);
          float mr = red[0];
#pragma unroll
          for (int k = 1; k < 8; ++k) mr = fmaxf(mr, red[k]);
          rband[tid] = ex2_approx(r2v - mr);
          bool bad = false;
          if (tid < 128) {
            const float ew = ma + mr - z2;
            bad = ew > 100.0f;
            wq[tid] = ex2_approx(ew);
          }
          const unsigned anybad = __any_sync(0xffffffffu, bad);
          if (lane == 0) red[8 + warp] = anybad ? 1.0f : 0.0f;
          named_bar_sync(1, C::NCT);
          bool exact = false;
#pragma unroll
          for (int k = 0; k < 4; ++k) exact |= red[8 + k] > 0.0f;
          // buffer (t&1) must have been consumed by the dV MMA of tile t-2
          if (t >= 2) {
            uint32_t& n = (t & 1) ? npf1 : npf0;
            if (!mbar_wait_warp(pfree + (t & 1), n & 1, wc, B_PFREE)) ok = false;
            ++n;
            tc_fence_after();
          }
          const uint32_t t_p = tmem + lane_base + (t & 1) * 64;
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int q0 = 64 * half + 32 * cc;
            uint32_t pk[16];
            if (!exact) {
              const float* rb = rband + (q0 - rowl + 127);
#pragma unroll
              for (int e4 = 0; e4 < 8; ++e4) {
                const float4 w4 = *reinterpret_cast<const float4*>(wq + q0 + 4 * e4);
                const float p0 = aj * w4.x * rb[4 * e4], p1 = aj * w4.y * rb[4 * e4 + 1];
                const float p2 = aj * w4.z * rb[4 * e4 + 2], p3 = aj * w4.w * rb[4 * e4 + 3];
                pk[2 * e4] = pack_bf16x2(p0, p1);
                pk[2 * e4 + 1] = pack_bf16x2(p2, p3);
              }
            } else {
              const float* rb = r2raw + (q0 - rowl + 127);
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                const float p0 = ex2_approx(a2 + rb[2 * e] - z2s[q0 + 2 * e]);
                const float p1 = ex2_approx(a2 + rb[2 * e + 1] - z2s[q0 + 2 * e + 1]);
                pk[e] = pack_bf16x2(p0, p1);
              }
            }
            tmem_st16(t_p + (q0 >> 1), pk);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(pds_full);
        }
      }
      if (leave) break;
      // ---------------- epilogue: dV (warps 0-3) and dK (warps 4-7) of this key block
      // (a warp whose wait was abandoned keeps walking - without storing - to the next agreement
      // barrier, so that no other compute warp is left waiting for it)
      if (!mbar_wait_warp(acc_full, nacc & 1, wc, B_ACC_FULL)) ok = false;
      ++nacc;
      tc_fence_after();
      if (!ord) {
        // keep the double-buffer barriers in step: absorb the completions not waited for in the loop
        const int left0 = (ntiles + 1) / 2 - ((ntiles > 2) ? (ntiles - 1) / 2 : 0);   // buffer 0: tiles 0,2,4,..
        const int left1 = ntiles / 2 - ((ntiles > 3) ? (ntiles - 2) / 2 : 0);          // buffer 1: tiles 1,3,5,..
        for (int k = 0; k < left0; ++k) {
          if (!mbar_wait_warp(pfree, npf0 & 1, wc, B_PFREE)) ok = false;
          ++npf0;
        }
        for (int k = 0; k < left1; ++k) {
          if (!mbar_wait_warp(pfree + 1, npf1 & 1, wc, B_PFREE)) ok = false;
          ++npf1;
        }
      }
      if (half == 0 || ord) {
        const uint32_t col = half == 0 ? C::COL_DV : C::COL_DK;
        const float mul = half == 0 ? 1.0f : p.scale;
        void* base = half == 0 ? p.dV : p.dK;
        const size_t off = (bh * p.T + key) * 64;
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + col + 32 * cc, r);
          tmem_wait_ld();
          if (key < p.T && ok) {
            if (p.grad_f32) {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(base) + off + 32 * cc);
#pragma unroll
              for (int e = 0; e < 8; ++e)
                dst[e] = make_float4(__uint_as_float(r[4 * e]) * mul, __uint_as_float(r[4 * e + 1]) * mul,
                                     __uint_as_float(r[4 * e + 2]) * mul, __uint_as_float(r[4 * e + 3]) * mul);
            } else {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off + 32 * cc);
#pragma unroll
              for (int e = 0; e < 4; ++e)
                dst[e] = make_uint4(pack_bf16x2(__uint_as_float(r[8 * e]) * mul, __uint_as_float(r[8 * e + 1]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 2]) * mul, __uint_as_float(r[8 * e + 3]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 4]) * mul, __uint_as_float(r[8 * e + 5]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 6]) * mul, __uint_as_float(r[8 * e + 7]) * mul));
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acc_free);
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

int bwd_smem_bytes(int) { return BwdCfg::SMEM; }

cudaError_t launch_bwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mdo, const BwdParams& p, int grid, cudaStream_t st) {
  if (D != 64) return cudaErrorNotSupported;
  cudaError_t e = cudaFuncSetAttribute(saf_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg::SMEM);
  if (e != cudaSuccess) return e;
  saf_bwd_kernel<<<grid, 320, BwdCfg::SMEM, st>>>(mq, mk, mv, mdo, p);
  return cudaGetLastError();
}

}  // namespace saf
