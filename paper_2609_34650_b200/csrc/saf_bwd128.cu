// Backward of the hybrid causal attention layer on sm_100a, head dimension 128 (96 runs here too: TMA zero-fills
// features 96..127): one persistent kernel, one work item per (batch, head, 128-key block J), looping over
// 64-query half tiles u of the query blocks I >= J.
//
// With 128 features the two gradient accumulators of a key block take half of TMEM, so there is room for one
// S^T / dP^T buffer only (64 query columns) and the half tiles go through it one after the other:
//   A(u):       S'^T = K_J Q_u^T + 1 (-LSE/scale)^T,  dP'^T = V_J dO_u^T + 1 (-delta)^T      (operands in smem; the
//               row terms ride on one extra 16-wide reduction step, as at head dimension 64)
//   compute(u): P^T = exp2(c S'^T), dS^T = P^T o dP'^T (bf16 back into the buffer's own columns; dS^T also to smem)
//   B(u):       dV_J += P^T dO_u,  dK_J += dS^T Q_u       (A from TMEM, 128-wide MMAs), then A(u+1) right behind it
//   C(t):       dQ_t = dS K_J once per full tile           (A = the smem dS^T tile read M-major, B = K_J MN-major)
// Appendix E.2 (key-block programs accumulate dV and dK; dQ here comes out of the same loop and is accumulated
// across key blocks with TMA reduce-adds).  Frozen items (Sec. 3.3: dV = P^^T dO, no query/key gradients) use the
// tensor-core form (Hankel band x scaled dO, see the forward) or generate P^^T half tiles with one exponential per
// element.
//
// CTA = 704 threads: warps 0-15 compute (TMEM lane = key row; four warps per lane quarter, 16 query columns each),
// warps 16-19 dQ drain, warp 20 TMA producer, warp 21 tcgen05 issuer and TMEM owner.
// TMEM columns: [0,128) dV, [128,256) dK, [256,320) S^T / P^T, [320,384) dP^T / dS^T, [384,512) dQ.
// Q and dO travel as 64-row half tiles through a ring of two stages, so the next half tile loads while the
// current one is in the tensor core.  Every wait is bounded.
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

SAF_SPAN_DEFINE(bwd128)

namespace saf {

namespace {

constexpr float LOG2E_W = 1.4426950408889634f;

struct W128 {
  static constexpr int PANEL = 128 * 64 * 2;         // [128 rows][64 cols] bf16, 16 KB
  static constexpr int HP = 64 * 64 * 2;             // half-tile panel [64 rows][64 cols], 8 KB
  static constexpr int NS = 2;                       // half-tile stages of Q / dO
  static constexpr int OFF_K = 0;                    // 2 panels
  static constexpr int OFF_V = 2 * PANEL;            // 2 panels
  static constexpr int OFF_QH = 4 * PANEL;           // NS x 2 half panels
  static constexpr int OFF_DOH = OFF_QH + NS * 2 * HP;
  static constexpr int OFF_DS = OFF_DOH + NS * 2 * HP;   // 2 panels: [query half][128 key rows][64 queries]
  static constexpr int OFF_DQ = OFF_DS + 2 * PANEL;      // fp32 staging box [128 rows][32 floats]
  static constexpr int OFF_AUX = OFF_DQ + PANEL;         // NS x 4 KB: row-term images of Q | dO (2 KB each), or a band
  static constexpr int OFF_ONES = OFF_AUX + NS * 4096;   // 4 KB constant tile: columns 0..2 one, rest zero
  static constexpr int OFF_TAB = OFF_ONES + 4096;
  static constexpr int TAB_FLOATS = 256 + 128;           // r2raw[256] z2s[128]
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  static constexpr int NBAR = 2 + 2 * NS + 9;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 512;
  static constexpr int COL_DV = 0, COL_DK = 128, COL_S = 256, COL_DP = 320, COL_DQ = 384;
  static constexpr int NTHREADS = 704;
};

enum W128Site { W_KV_EMPTY = 81, W_H_EMPTY, W_KV_FULL, W_H_FULL, W_PDS_FULL, W_ACC_FREE, W_DQ_FREE, W_S_FULL,
                W_SDP_FULL, W_DQ_FULL, W_ACC_FULL, W_PFREE, W_C_DONE };

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Work item `it` and whether it takes the tensor-core frozen form, fetched one item ahead of its use.
struct ItemW {
  WorkItem w;
  bool fast;
};
__device__ __forceinline__ ItemW load_item_w(const BwdParams& p, int it, int it_end) {
  ItemW v;
  v.w = WorkItem{0, 0, 0, KIND_ORDINARY};
  v.fast = false;
  if (it < it_end) {
    const int4 raw = __ldg(reinterpret_cast<const int4*>(p.items + it));
    v.w = WorkItem{raw.x, raw.y, raw.z, raw.w};
    v.fast = raw.w != KIND_ORDINARY && p.band_b != nullptr && __ldg(p.fast_ok + raw.y) != 0 &&
             __ldg(p.ovf + raw.y) != p.call_id;
  }
  return v;
}

}  // namespace

__global__ void __launch_bounds__(W128::NTHREADS, 1)
saf_bwd128_kernel(const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv,
                  const __grid_constant__ CUtensorMap mqh, const __grid_constant__ CUtensorMap mdoh,
                  const __grid_constant__ CUtensorMap mdoth, const __grid_constant__ CUtensorMap mdq,
                  const BwdParams p) {
  using C = W128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* kv_full = bars;
  uint64_t* kv_empty = bars + 1;
  uint64_t* h_full = bars + 2;                   // [NS] a half tile of Q / dO (or band + scaled dO) has landed
  uint64_t* h_empty = h_full + C::NS;            // [NS]
  uint64_t* s_full = h_empty + C::NS;            // S'^T is complete
  uint64_t* sdp_full = s_full + 1;               // ... and dP'^T
  uint64_t* pds_full = sdp_full + 1;             // the compute warps have written P^T / dS^T (16 warp arrivals)
  uint64_t* dq_full = pds_full + 1;
  uint64_t* dq_free = dq_full + 1;               // 4 drain warps
  uint64_t* acc_full = dq_free + 1;
  uint64_t* acc_free = acc_full + 1;             // 16 compute warps
  uint64_t* pfree = acc_free + 1;                // generic frozen form: the P^^T half tile has been consumed
  uint64_t* c_done = pfree + 1;                  // the dQ MMAs have read the smem dS^T tile
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(c_done + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  SAF_SPAN(bwd128, 0);
  const int nblk = p.nblk;

  if (tid == 0) {
    *abort_flag = 0;
    mbar_init(kv_full, 1);
    mbar_init(kv_empty, 1);
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(h_full + s, 1);
      mbar_init(h_empty + s, 1);
    }
    mbar_init(s_full, 1);
    mbar_init(sdp_full, 1);
    mbar_init(pds_full, 16);
    mbar_init(dq_full, 1);
    mbar_init(dq_free, 4);
    mbar_init(acc_full, 1);
    mbar_init(acc_free, 16);
    mbar_init(pfree, 1);
    mbar_init(c_done, 1);
    mbar_fence_init();
  }
  // constant tile of ones (columns 0..2) in the no-swizzle K-major core-matrix layout
  for (int i = tid; i < 256; i += C::NTHREADS) {
    const int k8 = (i >> 3) & 1;                 // 16-byte unit i: row group i>>4, k-half k8, row-in-group i&7
    uint4 v = make_uint4(0, 0, 0, 0);
    if (k8 == 0) {
      v.x = 0x3F803F80u;                         // bf16 1.0, 1.0
      v.y = 0x00003F80u;                         // bf16 1.0, 0
    }
    reinterpret_cast<uint4*>(smem + C::OFF_ONES)[i] = v;
  }
  if (warp == 21) {
    tmem_alloc(tmem_slot, C::TMEM_COLS);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // the prologue above overlapped the previous kernel's tail; global memory is touched only from here on
  pdl_launch_dependents();
  pdl_wait();
  const int it_begin = p.cta_offsets[blockIdx.x], it_end = p.cta_offsets[blockIdx.x + 1];

  if (warp == 20) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mk);
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mqh);
      tma_prefetch_desc(&mdoh);
      tma_prefetch_desc(&mdoth);
      uint32_t nkv = 0, nh = 0;
      bool ok = true;
      ItemW nxt = load_item_w(p, it_begin, it_end);
      for (int it = it_begin; it < it_end && ok; ++it) {
        const WorkItem w = nxt.w;
        const bool fast = nxt.fast;
        nxt = load_item_w(p, it + 1, it_end);
        const bool ord = w.kind == KIND_ORDINARY;
        const size_t bh = static_cast<size_t>(w.b) * p.H + w.h;
        const int qh = (ord && p.qslot) ? p.qslot[w.h] : w.h;          // head index in the Q tensor
        if (ord) {
          const int kh = p.qslot ? p.qslot[w.h] : w.h / p.kv_group;    // ... in the K tensor
          ok = mbar_wait(kv_empty, (nkv & 1) ^ 1, wc, W_KV_EMPTY);
          if (!ok) break;
          mbar_expect_tx(kv_full, 4 * C::PANEL);
          for (int pn = 0; pn < 2; ++pn) {
            tma_load_4d(smem + C::OFF_K + pn * C::PANEL, &mk, kv_full, pn * 64, w.blk * BLK, kh, w.b);
            tma_load_4d(smem + C::OFF_V + pn * C::PANEL, &mv, kv_full, pn * 64, w.blk * BLK, w.h / p.kv_group, w.b);
          }
          ++nkv;
        }
        const int fo = fast ? p.hord[w.h] : 0;
        const uint8_t* bands = static_cast<const uint8_t*>(p.band_b) + static_cast<size_t>(w.h) * p.nblkp * 4096;
        const int U = 2 * (nblk - w.blk);
        for (int u = 0; u < U; ++u, ++nh) {
          const int I = w.blk + (u >> 1), row0 = I * BLK + 64 * (u & 1);
          const uint32_t s = nh % C::NS;
          ok = mbar_wait(h_empty + s, ((nh / C::NS) & 1) ^ 1, wc, W_H_EMPTY);
          if (!ok) break;
          uint8_t* qdst = smem + C::OFF_QH + s * 2 * C::HP;
          uint8_t* ddst = smem + C::OFF_DOH + s * 2 * C::HP;
          uint8_t* aux = smem + C::OFF_AUX + s * 4096;
          if (fast) {
            // tensor-core form: the Hankel band of distance block (I - J) and the scaled dO half tile
            mbar_expect_tx(h_full + s, 2 * C::HP + 4096);
            bulk_load(aux, bands + static_cast<size_t>(I - w.blk) * 4096, 4096, h_full + s);
            for (int pn = 0; pn < 2; ++pn) tma_load_4d(ddst + pn * C::HP, &mdoth, h_full + s, pn * 64, row0, fo, w.b);
          } else if (ord) {
            mbar_expect_tx(h_full + s, 4 * C::HP + 4096);
            const size_t img = (bh * nblk + I) * 4096 + (u & 1) * 2048;
            bulk_load(aux, static_cast<const uint8_t*>(p.q_ext) + img, 2048, h_full + s);
            bulk_load(aux + 2048, static_cast<const uint8_t*>(p.do_ext) + img, 2048, h_full + s);
            for (int pn = 0; pn < 2; ++pn) {
              tma_load_4d(qdst + pn * C::HP, &mqh, h_full + s, pn * 64, row0, qh, w.b);
              tma_load_4d(ddst + pn * C::HP, &mdoh, h_full + s, pn * 64, row0, w.h, w.b);
            }
          } else {
            mbar_expect_tx(h_full + s, 2 * C::HP);
            for (int pn = 0; pn < 2; ++pn) tma_load_4d(ddst + pn * C::HP, &mdoh, h_full + s, pn * 64, row0, w.h, w.b);
          }
        }
      }
    }
  }
  else if (warp == 21) {
    // ------------------------------------------------------------------ tcgen05 issuer
    // The whole warp walks the loops (warp-uniform operands); one elected lane issues.  MMAs issued by one thread
    // execute in issue order: A(u+1) is queued right behind B(u), which reads the bf16 contents of the same buffer.
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t id_s = umma_idesc_bf16(128, 64, 0, 0);      // S^T, dP^T half tiles: both operands K-major
    // (head dimension 96 runs here with features 96..127 zero-filled by TMA: the gradient MMAs produce only 96
    // columns and the score MMAs skip the two empty k-steps)
    const uint32_t id_acc = umma_idesc_bf16(128, p.d_real, 0, 1);  // dV, dK: A from TMEM, B MN-major
    const uint32_t id_dq = umma_idesc_bf16(128, p.d_real, 1, 1);   // dQ: A (dS^T tile) M-major, B MN-major
    const uint32_t id_hk = umma_idesc_f16(128, p.d_real, 0, 1);    // fp16 band x fp16 scaled dO
    const int nk16 = p.d_real / 16;
    // descriptor halves for smem offset 0: 128B-swizzled K-major (k-step +32 B inside a 64-feature panel), the
    // no-swizzle K-major row-term tiles (LBO 128 B, SBO 256 B), 128B-swizzled MN-major tiles whose two 64-wide
    // halves are a half panel (Q / dO stages) or a panel (K_J, dS^T) apart, and the Hankel band
    const uint64_t d_k = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_x = umma_smem_desc(sb, 128, 256, UMMA_LAYOUT_NONE);
    const uint64_t d_mh = umma_smem_desc(sb, C::HP, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_m = umma_smem_desc(sb, C::PANEL, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_band = umma_smem_desc(sb, 128, 128, UMMA_LAYOUT_NONE);
    const uint32_t lo_k = desc_lo(d_k), hi_k = desc_hi(d_k), lo_x = desc_lo(d_x), hi_x = desc_hi(d_x);
    const uint32_t lo_mh = desc_lo(d_mh), hi_mh = desc_hi(d_mh), lo_m = desc_lo(d_m), hi_m = desc_hi(d_m);
    const uint32_t lo_b = desc_lo(d_band), hi_b = desc_hi(d_band);
    const uint32_t ones_lo = lo_x + (C::OFF_ONES >> 4);
    const uint32_t k_lo = lo_k + (C::OFF_K >> 4), v_lo = lo_k + (C::OFF_V >> 4);
    const uint32_t km_lo = lo_m + (C::OFF_K >> 4), ds_lo = lo_m + (C::OFF_DS >> 4);
    const uint32_t t_s = tmem + C::COL_S, t_dp = tmem + C::COL_DP;
    uint32_t nkv = 0, nh = 0, nitem = 0, ndq = 0, npds = 0;
    bool ok = true;
    ItemW nxt = load_item_w(p, it_begin, it_end);
    for (int it = it_begin; it < it_end && ok; ++it, ++nitem) {
      const WorkItem w = nxt.w;
      const bool fast = nxt.fast;
      nxt = load_item_w(p, it + 1, it_end);
      const bool ord = w.kind == KIND_ORDINARY;
      const int U = 2 * (nblk - w.blk);
      if (ord) {
        ok = mbar_wait_warp(kv_full, nkv & 1, wc, W_KV_FULL);
        if (!ok) break;
        ++nkv;
        // score MMAs of the half tile in ring position pos
        auto issue_A = [&](uint32_t pos) {
          const uint32_t s = pos % C::NS;
          const uint32_t q_lo = lo_k + ((C::OFF_QH + s * 2 * C::HP) >> 4);
          const uint32_t do_lo = lo_k + ((C::OFF_DOH + s * 2 * C::HP) >> 4);
          const uint32_t qx_lo = lo_x + ((C::OFF_AUX + s * 4096) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc) {
              if (kc >= nk16) break;
              const uint32_t ok_ = ((kc >> 2) * C::PANEL + (kc & 3) * 32) >> 4;
              const uint32_t oh_ = ((kc >> 2) * C::HP + (kc & 3) * 32) >> 4;
              umma_ss2(t_s, k_lo + ok_, hi_k, q_lo + oh_, hi_k, id_s, kc > 0);
            }
            umma_ss2(t_s, ones_lo, hi_x, qx_lo, hi_x, id_s, 1);
            umma_commit(s_full);                         // the exponentials start while dP'^T is computed
#pragma unroll
            for (int kc = 0; kc < 8; ++kc) {
              if (kc >= nk16) break;
              const uint32_t ok_ = ((kc >> 2) * C::PANEL + (kc & 3) * 32) >> 4;
              const uint32_t oh_ = ((kc >> 2) * C::HP + (kc & 3) * 32) >> 4;
              umma_ss2(t_dp, v_lo + ok_, hi_k, do_lo + oh_, hi_k, id_s, kc > 0);
            }
            umma_ss2(t_dp, ones_lo, hi_x, qx_lo + (2048 >> 4), hi_x, id_s, 1);
            umma_commit(sdp_full);
          }
          __syncwarp();
        };
        ok = mbar_wait_warp(h_full + nh % C::NS, (nh / C::NS) & 1, wc, W_H_FULL);
        if (!ok) break;
        tc_fence_after();
        issue_A(nh);
        for (int u = 0; u < U && ok; ++u) {
          const uint32_t pos = nh + u, s = pos % C::NS;
          ok = mbar_wait_warp(pds_full, npds & 1, wc, W_PDS_FULL);
          ++npds;
          if (ok && u == 0) ok = mbar_wait_warp(acc_free, (nitem & 1) ^ 1, wc, W_ACC_FREE);
          if (!ok) break;
          tc_fence_after();
          const uint32_t doh_lo = lo_mh + ((C::OFF_DOH + s * 2 * C::HP) >> 4);
          const uint32_t qh_lo = lo_mh + ((C::OFF_QH + s * 2 * C::HP) >> 4);
          const uint32_t acc0 = u > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ts2(tmem + C::COL_DV, t_s + 16 * kc, doh_lo + 128 * kc, hi_mh, id_acc, kc > 0 ? 1u : acc0);
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ts2(tmem + C::COL_DK, t_dp + 16 * kc, qh_lo + 128 * kc, hi_mh, id_acc, kc > 0 ? 1u : acc0);
            umma_commit(h_empty + s);
          }
          __syncwarp();
          if (u + 1 < U) {
            ok = mbar_wait_warp(h_full + (pos + 1) % C::NS, ((pos + 1) / C::NS) & 1, wc, W_H_FULL);
            if (!ok) break;
            tc_fence_after();
            issue_A(pos + 1);
          }
          if (u & 1) {
            // full tile done: dQ of the tile
            ok = mbar_wait_warp(dq_free, (ndq & 1) ^ 1, wc, W_DQ_FREE);
            if (!ok) break;
            ++ndq;
            tc_fence_after();
            if (leader) {
#pragma unroll
              for (int kc = 0; kc < 8; ++kc)
                umma_ss2(tmem + C::COL_DQ, ds_lo + 128 * kc, hi_m, km_lo + 128 * kc, hi_m, id_dq, kc > 0);
              umma_commit(dq_full);
              umma_commit(c_done);
            }
            __syncwarp();
          }
        }
        if (!ok) break;
        nh += U;
        if (leader) umma_commit(kv_empty);
      } else {
        // frozen item: dV only.  Tensor-core form: A = Hankel band rows of this query half, B = scaled dO half tile;
        // general form: A = the P^^T half tile the compute warps wrote into the S^T buffer.
        for (int u = 0; u < U && ok; ++u, ++nh) {
          const uint32_t s = nh % C::NS;
          ok = mbar_wait_warp(h_full + s, (nh / C::NS) & 1, wc, W_H_FULL);
          if (ok && !fast) {
            ok = mbar_wait_warp(pds_full, npds & 1, wc, W_PDS_FULL);
            ++npds;
          }
          if (ok && u == 0) ok = mbar_wait_warp(acc_free, (nitem & 1) ^ 1, wc, W_ACC_FREE);
          if (!ok) break;
          tc_fence_after();
          const uint32_t doh_lo = lo_mh + ((C::OFF_DOH + s * 2 * C::HP) >> 4);
          const uint32_t band_lo = lo_b + ((C::OFF_AUX + s * 4096) >> 4) + 16 * 4 * (u & 1);
          const uint32_t acc0 = u > 0 ? 1u : 0u;
          if (leader) {
            if (fast) {
#pragma unroll
              for (int kc = 0; kc < 4; ++kc)
                umma_ss2(tmem + C::COL_DV, band_lo + 16 * kc, hi_b, doh_lo + 128 * kc, hi_mh, id_hk, kc > 0 ? 1u : acc0);
            } else {
#pragma unroll
              for (int kc = 0; kc < 4; ++kc)
                umma_ts2(tmem + C::COL_DV, t_s + 16 * kc, doh_lo + 128 * kc, hi_mh, id_acc, kc > 0 ? 1u : acc0);
              umma_commit(pfree);
            }
            umma_commit(h_empty + s);
          }
          __syncwarp();
        }
        if (!ok) break;
      }
      if (leader) umma_commit(acc_full);
      __syncwarp();
    }
  }
  else if (warp >= 16 && warp < 20) {
    // ------------------------------------------------------------------ dQ drain warps (128 threads)
    // dQ of a tile (128 queries x 128 features, fp32) leaves in four [128][32] boxes through one staging box.
    const int q4 = warp & 3;
    const int rowl = q4 * 32 + lane;                    // query row within the tile
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const uint32_t stage_row = smem_u32(smem + C::OFF_DQ) + rowl * 128;
    const int nbox = p.d_real > 96 ? 4 : 3;             // head dimension 96: the fourth box does not exist
    uint32_t ndq = 0;
    bool ok = true, leave = false;
    for (int it = it_begin; it < it_end && !leave; ++it) {
      const WorkItem w = p.items[it];
      if (w.kind != KIND_ORDINARY) continue;
      const int qh = p.qslot ? p.qslot[w.h] : w.h;      // head index in the dQ accumulator
      for (int I = w.blk; I < nblk && !leave; ++I) {
        for (int k = 0; k < 4; ++k) {
          // the previous reduce has finished reading the staging box (thread 512 waits for it before arriving
          // here); the drain warps also agree here whether a wait has been abandoned
          if (named_bar_or(2, 128, !ok)) {
            leave = true;
            break;
          }
          if (k == 0) {
            if (!mbar_wait_warp(dq_full, ndq & 1, wc, W_DQ_FULL)) ok = false;
            ++ndq;
            tc_fence_after();
          }
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + C::COL_DQ + 32 * k, r);
          tmem_wait_ld();
          if (k == 3) {
            tc_fence_before();
            warp_arrive(dq_free);                       // the tensor core may overwrite dQ
          }
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint32_t chunk = static_cast<uint32_t>(g ^ (rowl & 7)) * 16;
            st_shared_v4w(stage_row + chunk, __float_as_uint(__uint_as_float(r[4 * g]) * p.scale),
                          __float_as_uint(__uint_as_float(r[4 * g + 1]) * p.scale),
                          __float_as_uint(__uint_as_float(r[4 * g + 2]) * p.scale),
                          __float_as_uint(__uint_as_float(r[4 * g + 3]) * p.scale));
          }
          fence_proxy_async_smem();
          named_bar_sync(3, 128);
          if (tid == 512 && ok && k < nbox) {
            tma_reduce_add_4d(&mdq, smem + C::OFF_DQ, 32 * k, I * BLK, qh, w.b);
            bulk_commit_group();
            bulk_wait_group_read0();
          }
        }
      }
    }
    if (tid == 512) bulk_wait_group0();                 // all reduce-adds have landed before the kernel ends
  }
  else {
    // ------------------------------------------------------------------ compute warps (16 x 32 threads)
    // warp = 4 cq + q4: lane quarter q4 (TMEM lane = key row), 16 query columns cq of the 64-column half tile
    const int q4 = warp & 3, cq = warp >> 2;
    const int rowl = q4 * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const uint32_t t_s = tmem + lane_base + C::COL_S + 16 * cq;
    const uint32_t t_dp = tmem + lane_base + C::COL_DP + 16 * cq;
    float* r2raw = reinterpret_cast<float*>(smem + C::OFF_TAB);   // [256] rho' over the tile's band of distances
    float* z2s = r2raw + 256;                                      // [128] logZ' of the tile's queries
    uint32_t nsdp = 0, nacc = 0, gt = 0, npf = 0;
    bool ok = true;
    // A warp whose wait was abandoned keeps walking (without storing) to the next agreement barrier, where all
    // sixteen leave together; none is ever left alone at a named barrier.
    ItemW nxt = load_item_w(p, it_begin, it_end);
    for (int it = it_begin; it < it_end; ++it) {
      const WorkItem w = nxt.w;
      const bool fast = nxt.fast;                        // (the next item is fetched under the epilogue's wait)
      const bool ord = w.kind == KIND_ORDINARY;
      const int U = 2 * (nblk - w.blk);
      int key = w.blk * BLK + rowl;
      float dv_mul = 1.0f;
      if (named_bar_or(1, 512, !ok)) break;
      if (fast) {
        // tensor-core form: nothing to do per tile; lane m holds key 127-m, scaled by a(j) below
        key = w.blk * BLK + 127 - rowl;
        dv_mul = (key < p.T) ? p.avec[static_cast<size_t>(w.h) * p.Tp + key] * (1.0f / HK_BAND_SCALE) : 0.0f;
      } else if (ord) {
        const float c = p.scale_log2;
        for (int u = 0; u < U; ++u) {
          const int b = u & 1;
          if (!mbar_wait_warp(s_full, nsdp & 1, wc, W_S_FULL)) ok = false;
          tc_fence_after();
          // P^T of this warp's 16 query columns from S'^T alone; dP'^T is still on the tensor core
          uint32_t rs[16];
          tmem_ld16(t_s, rs);
          tmem_wait_ld();
          {
            uint32_t pk[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float p0 = ex2_approx(__uint_as_float(rs[2 * e]) * c);
              float p1 = ex2_approx(__uint_as_float(rs[2 * e + 1]) * c);
              if (u < 2) {                                 // diagonal tile: query index >= key index
                const int qa = 64 * b + 16 * cq + 2 * e;
                if (qa < rowl) p0 = 0.0f;
                if (qa + 1 < rowl) p1 = 0.0f;
              }
              rs[2 * e] = __float_as_uint(p0);
              rs[2 * e + 1] = __float_as_uint(p1);
              pk[e] = pack_bf16x2(p0, p1);
            }
            tmem_st8(t_s, pk);                             // bf16 pairs re-use columns this warp has consumed
          }
          if (!mbar_wait_warp(sdp_full, nsdp & 1, wc, W_SDP_FULL)) ok = false;
          ++nsdp;
          tc_fence_after();
          if (b == 0) {
            // the dQ MMAs of the previous tile have read the smem dS^T tile
            if (!mbar_wait_warp(c_done, (gt & 1) ^ 1, wc, W_C_DONE)) ok = false;
          }
          uint32_t rd[16], dk[8];
          tmem_ld16(t_dp, rd);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 8; ++e)
            dk[e] = pack_bf16x2(__uint_as_float(rs[2 * e]) * __uint_as_float(rd[2 * e]),
                                __uint_as_float(rs[2 * e + 1]) * __uint_as_float(rd[2 * e + 1]));
          tmem_st8(t_dp, dk);
          // dS^T row (this key) -> smem panel of this query half, 128-byte swizzle (chunk ^= row & 7)
          const uint32_t rowaddr = smem_u32(smem + C::OFF_DS + b * C::PANEL) + rowl * 128;
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            const uint32_t chunk = static_cast<uint32_t>((2 * cq + g) ^ (rowl & 7));
            st_shared_v4w(rowaddr + chunk * 16, dk[4 * g], dk[4 * g + 1], dk[4 * g + 2], dk[4 * g + 3]);
          }
          tmem_wait_st();
          fence_proxy_async_smem();
          tc_fence_before();
          warp_arrive(pds_full);
          if (b == 1) ++gt;
        }
      } else {
        // ---------------- frozen head, general form: P^^T half tiles, one exponential per element
        const float* alpha_h = p.alpha + static_cast<size_t>(w.h) * p.Tp;
        const float* rho_h = p.rho + static_cast<size_t>(w.h) * p.Tp;
        const float* logz_h = p.logZ + static_cast<size_t>(w.h) * p.Tp;
        const float a2 = (key < p.T) ? alpha_h[key] * LOG2E_W : -INFINITY;
        bool leave = false;
        for (int u = 0; u < U; ++u) {
          const int b = u & 1, t = u >> 1;
          if (b == 0) {
            if (named_bar_or(1, 512, !ok)) {               // previous tile's table readers are done; agree to go on
              ok = false;
              leave = true;
              break;
            }
            const int d = t * BLK - 127 + tid;             // band entry x = tid: distance of (query - key + 127)
            if (tid < 256) r2raw[tid] = (tid < 255 && d >= 0 && d < p.T) ? rho_h[d] * LOG2E_W : -INFINITY;
            if (tid < 128) {
              const int qi = (w.blk + t) * BLK + tid;
              z2s[tid] = (qi < p.T) ? logz_h[qi] * LOG2E_W : INFINITY;
            }
            named_bar_sync(2, 512);
          }
          if (u > 0) {                                     // the previous P^^T half tile has been consumed
            if (!mbar_wait_warp(pfree, npf & 1, wc, W_PFREE)) ok = false;
            ++npf;
            tc_fence_after();
          }
          const int q0 = 64 * b + 16 * cq;
          const float* rb = r2raw + (q0 - rowl + 127);
          uint32_t pk[8];
#pragma unroll
          for (int e = 0; e < 8; ++e)
            pk[e] = pack_bf16x2(ex2_approx(a2 + rb[2 * e] - z2s[q0 + 2 * e]),
                                ex2_approx(a2 + rb[2 * e + 1] - z2s[q0 + 2 * e + 1]));
          tmem_st8(t_s, pk);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(pds_full);
        }
        if (leave) break;
        // keep the barrier in step: absorb the completion of the last half tile
        if (!mbar_wait_warp(pfree, npf & 1, wc, W_PFREE)) ok = false;
        ++npf;
      }
      // ---------------- epilogue: this warp's 32 feature columns of dV and (ordinary items) dK
      nxt = load_item_w(p, it + 1, it_end);              // its load latency passes under the wait for the last MMAs
      if (!mbar_wait_warp(acc_full, nacc & 1, wc, W_ACC_FULL)) ok = false;
      ++nacc;
      tc_fence_after();
      const int ncol = p.d_real;                           // 128, or 96 (row length of the gradient tensors)
      const int kvh = w.h / p.kv_group;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        if (which == 1 && !ord) break;
        uint32_t r[32];
        tmem_ld32(tmem + lane_base + (which == 0 ? C::COL_DV : C::COL_DK) + 32 * cq, r);
        tmem_wait_ld();
        if (which == 1 || !ord) {
          tc_fence_before();
          warp_arrive(acc_free);                           // the accumulators may be overwritten
        }
        const float mul = which == 0 ? dv_mul : p.scale;
        const int hk = (which == 1 && p.qslot) ? p.qslot[w.h] : kvh;
        const int nhk = (which == 1 && p.qslot) ? p.n_ord : p.H / p.kv_group;
        const size_t off = ((static_cast<size_t>(w.b) * nhk + hk) * p.T + key) * ncol + 32 * cq;
        void* base = which == 0 ? p.dV : p.dK;
        if (key < p.T && ok && 32 * cq < ncol) {
          if (p.grad_f32) {
            float* dst = static_cast<float*>(base) + off;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float x0 = __uint_as_float(r[4 * e]) * mul, x1 = __uint_as_float(r[4 * e + 1]) * mul;
              const float x2 = __uint_as_float(r[4 * e + 2]) * mul, x3 = __uint_as_float(r[4 * e + 3]) * mul;
              if (p.kv_group > 1) red_add_v4(dst + 4 * e, x0, x1, x2, x3);     // shared head: sum over its query heads
              else *reinterpret_cast<float4*>(dst + 4 * e) = make_float4(x0, x1, x2, x3);
            }
          } else {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off);
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
  SAF_SPAN(bwd128, 1);
  if (warp == 21) tmem_dealloc(tmem, C::TMEM_COLS);
}

int bwd128_smem_bytes() { return W128::SMEM; }

cudaError_t launch_bwd128(const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mqh, const CUtensorMap& mdoh,
                          const CUtensorMap& mdoth, const CUtensorMap& mdq, const BwdParams& p, int grid,
                          cudaStream_t st) {
  cudaError_t e =
      cudaFuncSetAttribute(saf_bwd128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, W128::SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(PDL_BWD, saf_bwd128_kernel, dim3(grid), dim3(W128::NTHREADS), W128::SMEM, st, mk, mv, mqh, mdoh, mdoth, mdq, p);
}

}  // namespace saf
