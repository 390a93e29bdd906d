// Backward of the hybrid causal attention layer on sm_100a (head dimension 64): one persistent
// kernel, one work item per (batch, head, 128-key block J), looping over query blocks I >= J.
//
// CTA = 704 threads:
//   warps 0-7   compute group 0: even 64-query half tiles (TMEM buffer 0); TMEM lane = key row, two warps
//               per lane quarter, each on 32 of the half tile's 64 query columns
//   warps 8-15  compute group 1: odd half tiles (TMEM buffer 1)
//   warps 16-19 dQ drain: TMEM -> swizzled smem -> TMA reduce-add into the fp32 dQ accumulator
//   warp 20     TMA producer
//   warp 21     tcgen05 issuer of every MMA (A(u), B(u), C(t) below) and TMEM owner.  MMAs of one thread execute
//               in issue order, which the schedule relies on; splitting the issue over two warps measured slower.
// The per-tile critical path is a chain (scores -> exponentials -> gradient MMAs -> next scores on the
// same buffer), so the exponential step is spread over as many warps as the register file allows.
//
// Ordinary item (Appendix E.2: key-block programs accumulate dV and dK; dQ here comes out of the same
// tile loop and is accumulated across key blocks by reduce-adds instead of a second pass).  The tile
// loop is software-pipelined over half tiles u with S^T/dP^T double-buffered in TMEM:
//   A(u): S'^T[u&1]  = K_J Q_u^T  + 1 (-LSE_i/scale)^T,   dP'^T[u&1] = V_J dO_u^T + 1 (-delta_i)^T
//         (the row terms ride on one extra 16-wide reduction step: a constant tile of ones times a
//          three-way bf16 split of the fp32 row value, so S' and dP' leave the tensor core ready)
//   compute(u): P^T = exp2(c S'^T) = exp(scale S - LSE),  dS^T = P^T o dP'^T   (bf16 to TMEM; dS^T also to smem)
//   B(u): dV_J += P^T dO_u,  dK_J += dS^T Q_u                  (A from TMEM, dO / Q rows as MN-major B)
//   C(t), once per full tile: dQ_t = dS K_J                    (A = smem dS^T tile read M-major, B = K_J)
// Frozen item (Sec. 3.3: dV = P^^T dO, no query/key gradients), full tiles alternating between the
// two compute groups:
//   P^^T(j,i) = exp(alpha(j) + rho(i-j) - logZ(i)) for i >= j, generated into TMEM (factorised as in
//   the forward), dV_J += P^^T dO_I.
//
// Frozen item, tensor-core form (pattern tables prepared and the head's flag set):
//   dV = diag(a) R^T (diag(w) dO).  A tile of R^T with reversed rows is a Hankel matrix read by the tensor
//   core from a 4 KB band table; per tile one bulk copy of the band, one TMA load of the w-scaled dO tile
//   and 8 MMAs.  The compute warps only scale the finished rows by a(j) (lane m holds key 127-m).
//
// TMEM columns: [0,64) dV, [64,128) dK, [128,192)/[192,256) S^T buffers (bf16 P^T pairs re-use the
// columns their own warp consumed: [0,16) and [32,48) of the buffer; frozen P^^T tiles use the two 64-column buffers whole), [256,320)/[320,384) dP^T
// buffers (bf16 dS^T likewise), [384,448) dQ, [448,480) K_J and [480,512) V_J as bf16 pairs (copied once
// per item from their smem tiles, so that the score MMAs read their A operand from TMEM instead of
// re-reading 4 KB of shared memory per instruction: the kernel is shared-memory-bandwidth bound).
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

#ifdef SAF_TRACE
__device__ unsigned long long g_saf_trace[24][4096];
#define TR(role, id)                                                                                   \
  do {                                                                                                 \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && tr_n < 4090)                                    \
      g_saf_trace[role][tr_n++] = (static_cast<unsigned long long>(id) << 48) | (clock64() & 0xffffffffffffULL); \
  } while (0)
extern "C" int saf_debug_read_trace(unsigned long long* out) {
  return static_cast<int>(cudaMemcpyFromSymbol(out, g_saf_trace, sizeof(g_saf_trace)));
}
#else
#define TR(role, id)
#endif
SAF_SPAN_DEFINE(bwd)

namespace saf {

namespace {

constexpr float LOG2E_B = 1.4426950408889634f;

struct BwdCfg {
  static constexpr int PANEL = 128 * 64 * 2;         // one [128][64] bf16 tile, 128-byte rows, 16 KB
  static constexpr int NS = 2;                       // Q/dO ring depth
  static constexpr int OFF_K = 0;                    // 2 slots: the next item's K_J is prefetched
  static constexpr int OFF_V = 2 * PANEL;            // 1 slot: V_J is only staged here on its way to TMEM
  static constexpr int OFF_Q = 3 * PANEL;            // NS stages
  static constexpr int OFF_DO = OFF_Q + NS * PANEL;  // NS stages
  static constexpr int OFF_DS = OFF_DO + NS * PANEL; // 2 buffers x 2 panels (queries 0-63, 64-127)
  static constexpr int OFF_DQ = OFF_DS + 4 * PANEL;  // fp32 staging: one box [128 rows][32 floats], 128B swizzle
  static constexpr int OFF_QX = OFF_DQ + PANEL;      // NS x 4 KB row-term images of Q
  static constexpr int OFF_DOX = OFF_QX + NS * 4096; // NS x 4 KB row-term images of dO
  static constexpr int OFF_ONES = OFF_DOX + NS * 4096;   // 4 KB constant tile: columns 0..2 one, rest zero
  static constexpr int OFF_TAB = OFF_ONES + 4096;
  // per compute group: wq[128] z2s[128] rband[256] r2raw[256] red[16]
  static constexpr int TAB_FLOATS = 128 * 2 + 256 * 2 + 16;
  static constexpr int OFF_BAR = OFF_TAB + 2 * TAB_FLOATS * 4;
  // slot k of the tensor-core frozen ring
  __host__ __device__ static constexpr int fz_do(int k) { return (k < 2 ? OFF_DO : OFF_Q) + (k & 1) * PANEL; }
  __host__ __device__ static constexpr int fz_band(int k) { return (k < 2 ? OFF_QX : OFF_DOX) + (k & 1) * 4096; }
  static constexpr int NFZ = 4;                       // ring depth of the tensor-core frozen form (see the producer)
  static constexpr int NBAR = 4 + 2 * NS + 2 + 2 + 4 + 2 + 1 + 2 * NFZ + 2 + 2;
  static constexpr int SMEM = OFF_BAR + NBAR * 8 + 16 + 1024;
  static constexpr int TMEM_COLS = 512;
  static constexpr int COL_DV = 0, COL_DK = 64, COL_S = 128, COL_DP = 256, COL_DQ = 384, COL_KT = 448, COL_VT = 480;
  static constexpr int NTHREADS = 704;
};

enum BwdSite { B_KV_EMPTY = 21, B_QDO_EMPTY, B_KV_FULL, B_QDO_FULL, B_PDS_FULL, B_ACC_FREE, B_DQ_FREE, B_SDP_FULL,
               B_DQ_FULL, B_ACC_FULL, B_PFREE };

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Work item `it` and whether it takes the tensor-core frozen form, fetched one item ahead of its use so
// that the two dependent global loads stay off the item-to-item critical path.
struct ItemView {
  WorkItem w;
  bool fast;
};
__device__ __forceinline__ ItemView load_item(const BwdParams& p, int it, int it_end) {
  ItemView v;
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

__global__ void __launch_bounds__(BwdCfg::NTHREADS, 1)
saf_bwd_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
               const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mdo,
               const __grid_constant__ CUtensorMap mdq, const __grid_constant__ CUtensorMap mdot,
               const __grid_constant__ CUtensorMap mdk, const __grid_constant__ CUtensorMap mdv,
               const BwdParams p) {
  using C = BwdCfg;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* kv_full = bars;                      // [2] K_J / V_J of an item have landed (index = K slot)
  uint64_t* kv_empty = bars + 2;                 // [2] the item's MMAs have finished with K slot s
  uint64_t* qdo_full = bars + 4;                 // [NS]
  uint64_t* qdo_empty = qdo_full + C::NS;        // [NS]
  uint64_t* sdp_full = qdo_empty + C::NS;        // [2]
  uint64_t* pds_full = sdp_full + 2;             // [2]
  uint64_t* dq_full = pds_full + 2;
  uint64_t* dq_free = dq_full + 1;
  uint64_t* acc_full = dq_free + 1;
  uint64_t* acc_free = acc_full + 1;
  uint64_t* pfree = acc_free + 1;                // [2]
  uint64_t* kvt_full = pfree + 2;                // K_J / V_J have been copied into TMEM
  uint64_t* fz_full = kvt_full + 1;              // [NFZ] band + scaled dO tile of a tensor-core frozen tile
  uint64_t* fz_empty = fz_full + C::NFZ;         // [NFZ]
  uint64_t* s_full = fz_empty + C::NFZ;          // [2] S'^T of buffer b is complete (dP'^T follows: sdp_full)
  // [2] ordinary tiles: group b has written P^T / dS^T of its half tile.  The barrier of buffer 1 also counts the four
  // drain warps, which arrive once they have read the previous tile's dQ out of TMEM: the issuer's one wait in front
  // of a tile's second half then covers the accumulator that the tile's dQ MMAs (issued behind it) overwrite.
  uint64_t* pds_ord = s_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pds_ord + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  const int nblk = p.nblk;
  SAF_SPAN(bwd, 0);

  if (tid == 0) {
    *abort_flag = 0;
    for (int k = 0; k < 2; ++k) {
      mbar_init(kv_full + k, 1);
      mbar_init(kv_empty + k, 1);
    }
    for (int s = 0; s < C::NS; ++s) {
      mbar_init(qdo_full + s, 1);
      mbar_init(qdo_empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(sdp_full + b, 1);
      mbar_init(s_full + b, 1);
      mbar_init(pds_full + b, 8);                // one arrival per warp of the group
      mbar_init(pfree + b, 1);
      mbar_init(pds_ord + b, b == 0 ? 8 : 12);
    }
    mbar_init(kvt_full, 16);
    for (int k = 0; k < C::NFZ; ++k) {
      mbar_init(fz_full + k, 1);
      mbar_init(fz_empty + k, 1);
    }
    mbar_init(dq_full, 1);
    mbar_init(dq_free, 4);
    mbar_init(acc_full, 1);
    mbar_init(acc_free, 16);
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
      tma_prefetch_desc(&mq);
      tma_prefetch_desc(&mk);
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mdo);
      tma_prefetch_desc(&mdot);
      uint32_t nkv = 0, nqdo = 0, nfz = 0;
      bool ok = true, fz_open = false;
#ifdef SAF_TRACE
      int tr_n = 0;
#endif
      // K_J / V_J of the ordinary items run one item ahead of the tile loads: K into the other K slot (free
      // once the item before the current one has finished), V into the single V slot (free once the
      // current item's V has been copied to TMEM).
      int next_kv = it_begin;
      auto load_next_kv = [&]() {
        while (next_kv < it_end && p.items[next_kv].kind != KIND_ORDINARY) ++next_kv;
        if (next_kv >= it_end) return;
        const WorkItem w2 = p.items[next_kv++];
        const uint32_t ks = nkv & 1;
        ok = mbar_wait(kv_empty + ks, ((nkv >> 1) & 1) ^ 1, wc, B_KV_EMPTY);
        if (ok && nkv > 0) ok = mbar_wait(kvt_full, (nkv - 1) & 1, wc, B_KV_EMPTY);
        if (!ok) return;
        TR(2, 31);
        mbar_expect_tx(kv_full + ks, 2 * C::PANEL);
        tma_load_4d(smem + C::OFF_K + ks * C::PANEL, &mk, kv_full + ks, 0, w2.blk * BLK,
                    p.qslot ? p.qslot[w2.h] : w2.h / p.kv_group, w2.b);
        tma_load_4d(smem + C::OFF_V, &mv, kv_full + ks, 0, w2.blk * BLK, w2.h / p.kv_group, w2.b);
        ++nkv;
      };
      load_next_kv();
      for (int it = it_begin; it < it_end && ok; ++it) {
        const WorkItem w = p.items[it];
        const bool ord = w.kind == KIND_ORDINARY;
        const size_t bh = static_cast<size_t>(w.b) * p.H + w.h;
        const int qh = (ord && p.qslot) ? p.qslot[w.h] : w.h;     // head index in the Q tensor
        const bool fast = !ord && p.band_b != nullptr && p.fast_ok[w.h] != 0 && p.ovf[w.h] != p.call_id;
        if (fast) {
          // tensor-core form: per tile the Hankel band of distance block (I - J) and the scaled dO tile.  These
          // tiles have no compute step to hide the load latency behind, so they run a ring of their own, four
          // deep, laid over the idle Q/dO stages and row-term images: slot k keeps its dO tile in dO stage k
          // (k < 2) or Q stage k-2, its band in the Q (k < 2) or dO row-term image of stage k & 1.
          if (!fz_open) {
            // the stages' last ordinary / general tiles must have been consumed
            for (uint32_t n = nqdo > 1 ? nqdo - 2 : 0; n < nqdo && ok; ++n)
              ok = mbar_wait(qdo_empty + n % C::NS, (n / C::NS) & 1, wc, B_QDO_EMPTY);
            if (!ok) break;
            fz_open = true;
          }
          const int fo = p.hord[w.h];
          const uint8_t* bands = static_cast<const uint8_t*>(p.band_b) + static_cast<size_t>(w.h) * p.nblkp * 4096;
          for (int I = w.blk; I < nblk; ++I) {
            const uint32_t k = nfz % C::NFZ;
            ok = mbar_wait(fz_empty + k, ((nfz / C::NFZ) & 1) ^ 1, wc, B_QDO_EMPTY);
            if (!ok) break;
            mbar_expect_tx(fz_full + k, C::PANEL + 4096);
            bulk_load(smem + C::fz_band(k), bands + static_cast<size_t>(I - w.blk) * 4096, 4096, fz_full + k);
            tma_load_4d(smem + C::fz_do(k), &mdot, fz_full + k, 0, I * BLK, fo, w.b);
            ++nfz;
          }
          continue;
        }
        if (fz_open) {
          // back to the shared stages: the frozen ring's tiles in flight must have been consumed
          for (uint32_t n = nfz > C::NFZ ? nfz - C::NFZ : 0; n < nfz && ok; ++n)
            ok = mbar_wait(fz_empty + n % C::NFZ, (n / C::NFZ) & 1, wc, B_QDO_EMPTY);
          if (!ok) break;
          fz_open = false;
        }
        for (int I = w.blk; I < nblk; ++I) {
          const int s = nqdo % C::NS;
          ok = mbar_wait(qdo_empty + s, ((nqdo / C::NS) & 1) ^ 1, wc, B_QDO_EMPTY);
          if (!ok) break;
          TR(2, I == w.blk ? 33 : 32);
          mbar_expect_tx(qdo_full + s, ord ? 2 * C::PANEL + 8192 : C::PANEL);
          if (ord) {
            tma_load_4d(smem + C::OFF_Q + s * C::PANEL, &mq, qdo_full + s, 0, I * BLK, qh, w.b);
            const size_t img = (bh * nblk + I) * 4096;
            bulk_load(smem + C::OFF_QX + s * 4096, static_cast<const uint8_t*>(p.q_ext) + img, 4096, qdo_full + s);
            bulk_load(smem + C::OFF_DOX + s * 4096, static_cast<const uint8_t*>(p.do_ext) + img, 4096, qdo_full + s);
          }
          tma_load_4d(smem + C::OFF_DO + s * C::PANEL, &mdo, qdo_full + s, 0, I * BLK, w.h, w.b);
          ++nqdo;
          // with this item's first tiles under way, fetch K_J / V_J of the next ordinary item
          if (ord && I == min(w.blk + 1, nblk - 1)) {
            load_next_kv();
            if (!ok) break;
          }
        }
      }
    }
  } else if (warp == 21) {
    // ------------------------------------------------------------------ tcgen05 issuer
    // The whole warp walks the loops (warp-uniform operands); one elected lane issues.  MMAs issued by one
    // thread execute in issue order, which is what lets A(u+2) follow B(u) on the same TMEM buffer with
    // no completion round trip in between.
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t id_s = umma_idesc_bf16(128, 64, 0, 0);      // S^T, dP^T half tiles: both operands K-major
    constexpr uint32_t id_acc = umma_idesc_bf16(128, 64, 0, 1);    // dV, dK: A from TMEM, B MN-major
    constexpr uint32_t id_dq = umma_idesc_bf16(128, 64, 1, 1);     // dQ: A (dS^T tile) M-major, B MN-major
    // descriptor halves for smem offset 0: 128B-swizzled K-major (k-step +32 B), the no-swizzle K-major
    // row-term tiles (LBO 128 B, SBO 256 B) and 128B-swizzled MN-major tiles (k-step +2048 B, LBO = panel)
    const uint64_t d_k = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_x = umma_smem_desc(sb, 128, 256, UMMA_LAYOUT_NONE);
    const uint64_t d_m = umma_smem_desc(sb, C::PANEL, 1024, UMMA_LAYOUT_SW128);
    const uint32_t lo_k = desc_lo(d_k), hi_k = desc_hi(d_k), lo_x = desc_lo(d_x), hi_x = desc_hi(d_x);
    const uint32_t lo_m = desc_lo(d_m), hi_m = desc_hi(d_m);
    const uint32_t ones_lo = lo_x + (C::OFF_ONES >> 4);
    uint32_t nqdo = 0, nitem = 0, ndq = 0, ntile_ord = 0, nkv = 0, nfz = 0;
    uint32_t npds0 = 0, npds1 = 0;
#ifdef SAF_TRACE
    int tr_n = 0;
#endif
    bool ok = true;
    ItemView nxt = load_item(p, it_begin, it_end);
    for (int it = it_begin; it < it_end && ok; ++it, ++nitem) {
      const WorkItem w = nxt.w;
      const bool fast = nxt.fast;
      nxt = load_item(p, it + 1, it_end);
      const bool ord = w.kind == KIND_ORDINARY;
      const int ntiles = nblk - w.blk;
      if (ord) {
        // K_J / V_J are read from TMEM (copied there by the compute warps); K_J's smem slot feeds dQ
        const uint32_t km_lo = lo_m + ((C::OFF_K + (nkv & 1) * C::PANEL) >> 4);
        uint64_t* const kv_done = kv_empty + (nkv & 1);
        ok = mbar_wait_warp(kvt_full, nkv & 1, wc, B_KV_FULL);
        if (!ok) break;
        ++nkv;
        TR(3, 7);
        // score MMAs of half tile u into buffer u & 1, in two parts (issuing lane only): S'^T, whose completion
        // starts the exponentials, and dP'^T
        auto issue_S = [&](int u) {
          const uint32_t s = (nqdo + (u >> 1)) % C::NS;
          const uint32_t b = u & 1;
          const uint32_t q_lo = lo_k + ((C::OFF_Q + s * C::PANEL + b * 8192) >> 4);
          const uint32_t qx_lo = lo_x + ((C::OFF_QX + s * 4096 + b * 2048) >> 4);
          const uint32_t t_s = tmem + C::COL_S + 64 * b;
#pragma unroll
          for (int kc = 0; kc < 4; ++kc)
            umma_ts2(t_s, tmem + C::COL_KT + 8 * kc, q_lo + 2 * kc, hi_k, id_s, kc > 0);
          umma_ss2(t_s, ones_lo, hi_x, qx_lo, hi_x, id_s, 1);
          umma_commit(s_full + b);                       // the exponentials start while dP'^T is computed
        };
        auto issue_dP = [&](int u) {
          const uint32_t s = (nqdo + (u >> 1)) % C::NS;
          const uint32_t b = u & 1;
          const uint32_t do_lo = lo_k + ((C::OFF_DO + s * C::PANEL + b * 8192) >> 4);
          const uint32_t dox_lo = lo_x + ((C::OFF_DOX + s * 4096 + b * 2048) >> 4);
          const uint32_t t_dp = tmem + C::COL_DP + 64 * b;
#pragma unroll
          for (int kc = 0; kc < 4; ++kc)
            umma_ts2(t_dp, tmem + C::COL_VT + 8 * kc, do_lo + 2 * kc, hi_k, id_s, kc > 0);
          umma_ss2(t_dp, ones_lo, hi_x, dox_lo, hi_x, id_s, 1);
          umma_commit(sdp_full + b);
        };
        auto issue_A = [&](int u) {
          if (leader) {
            issue_S(u);
            issue_dP(u);
          }
          __syncwarp();
        };
        ok = mbar_wait_warp(qdo_full + nqdo % C::NS, (nqdo / C::NS) & 1, wc, B_QDO_FULL);
        if (!ok) break;
        tc_fence_after();
        TR(3, 1);
        issue_A(0);
        TR(3, 2);
        issue_A(1);
        TR(3, 3);
        // Per tile: first what the compute warps wait for - for each buffer, dV of its half tile and right behind
        // it the buffer's next S'^T (MMAs execute in issue order, so S'^T may overwrite P^T once the dV MMAs that
        // read it are queued) - then what they need only after their exponentials: dK and the next dP'^T of both
        // buffers (dP'^T follows the dK MMAs that read dS^T), the release of the Q/dO stage, and dQ of the tile.
        for (int t = 0; t < ntiles && ok; ++t) {
          const uint32_t pos = nqdo + t;
          const uint32_t s = pos % C::NS;
          const bool more = t + 1 < ntiles;
          const uint32_t acc0 = t > 0 ? 1u : 0u;
#pragma unroll
          for (int b = 0; b < 2; ++b) {
            TR(0, 4);
            ok = mbar_wait_warp(pds_ord + b, ntile_ord & 1, wc, B_PDS_FULL);
            if (!ok) break;
            TR(0, 5);
            if (t == 0 && b == 0) {
              ok = mbar_wait_warp(acc_free, (nitem & 1) ^ 1, wc, B_ACC_FREE);
              if (!ok) break;
            }
            if (more && b == 0) {
              // Q / dO of the next tile (its first half tile goes into this buffer below)
              ok = mbar_wait_warp(qdo_full + (pos + 1) % C::NS, ((pos + 1) / C::NS) & 1, wc, B_QDO_FULL);
              if (!ok) break;
            }
            tc_fence_after();
            const uint32_t do_lo = lo_m + ((C::OFF_DO + s * C::PANEL + b * 8192) >> 4);
            const uint32_t t_p = tmem + C::COL_S + 64 * b;
            if (leader) {
#pragma unroll
              for (int kc = 0; kc < 4; ++kc)
                umma_ts2(tmem + C::COL_DV, t_p + 8 * kc + (kc >= 2 ? 16 : 0), do_lo + 128 * kc, hi_m, id_acc,
                         (kc > 0 || b > 0) ? 1u : acc0);
              if (more) issue_S(2 * t + 2 + b);
              // dK of this half tile and the buffer's next dP'^T follow at once (rather than after the other buffer's
              // dV and S'^T): the second group's scores are then issued a good 700 clk after the first group's, which
              // keeps the two groups' exponential phases apart - in phase, they halve each other's rate on the
              // 16-per-clock special-function unit
              const uint32_t q_lo = lo_m + ((C::OFF_Q + s * C::PANEL + b * 8192) >> 4);
              const uint32_t t_ds = tmem + C::COL_DP + 64 * b;
#pragma unroll
              for (int kc = 0; kc < 4; ++kc)
                umma_ts2(tmem + C::COL_DK, t_ds + 8 * kc + (kc >= 2 ? 16 : 0), q_lo + 128 * kc, hi_m, id_acc,
                         (kc > 0 || b > 0) ? 1u : acc0);
              // full tile done: its Q/dO stage can be refilled
              if (b == 1) umma_commit(qdo_empty + s);
              if (more) issue_dP(2 * t + 2 + b);
            }
            __syncwarp();
            TR(0, 10 + b);
          }
          if (!ok) break;
          __syncwarp();
          TR(0, 6);
          // (no wait for the dQ accumulator: the drain warps' arrivals were part of this tile's pds_ord[1] phase)
          const uint32_t ds_lo = lo_m + ((C::OFF_DS + (ntile_ord & 1) * 2 * C::PANEL) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ss2(tmem + C::COL_DQ, ds_lo + 128 * kc, hi_m, km_lo + 128 * kc, hi_m, id_dq, kc > 0);
            umma_commit(dq_full);
          }
          TR(0, 9);
          ++ntile_ord;
          __syncwarp();
          TR(0, 14);
        }
        if (!ok) break;
        nqdo += ntiles;
        if (leader) umma_commit(kv_done);
      } else if (fast) {
        // tensor-core form of a frozen head: A = Hankel band (no-swizzle, both strides 128 B), B = scaled dO
        constexpr uint32_t id_hk = umma_idesc_f16(128, 64, 0, 1);   // fp16 band x fp16 scaled dO
        const uint64_t d_band = umma_smem_desc(sb, 128, 128, UMMA_LAYOUT_NONE);
        const uint32_t lo_b = desc_lo(d_band), hi_b = desc_hi(d_band);
        for (int t = 0; t < ntiles; ++t) {
          const uint32_t k = nfz % C::NFZ;
          TR(0, 20);
          ok = mbar_wait_warp(fz_full + k, (nfz / C::NFZ) & 1, wc, B_QDO_FULL);
          if (!ok) break;
          ++nfz;
          TR(0, 21);
          if (t == 0) {
            ok = mbar_wait_warp(acc_free, (nitem & 1) ^ 1, wc, B_ACC_FREE);
            if (!ok) break;
            TR(0, 23);
          }
          tc_fence_after();
          const uint32_t band_lo = lo_b + (static_cast<uint32_t>(C::fz_band(k)) >> 4);
          const uint32_t do_lo = lo_m + (static_cast<uint32_t>(C::fz_do(k)) >> 4);
          const uint32_t acc0 = t > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ss2(tmem + C::COL_DV, band_lo + 16 * kc, hi_b, do_lo + 128 * kc, hi_m, id_hk, kc > 0 ? 1u : acc0);
            umma_commit(fz_empty + k);
          }
          __syncwarp();
          TR(0, 22);
        }
        if (!ok) break;
      } else {
        for (int t = 0; t < ntiles; ++t) {
          const uint32_t s = nqdo % C::NS;
          ok = mbar_wait_warp(qdo_full + s, (nqdo / C::NS) & 1, wc, B_QDO_FULL);
          if (!ok) break;
          ++nqdo;
          const uint32_t b = t & 1;
          if (b == 0) {
            ok = mbar_wait_warp(pds_full, npds0 & 1, wc, B_PDS_FULL);
            ++npds0;
          } else {
            ok = mbar_wait_warp(pds_full + 1, npds1 & 1, wc, B_PDS_FULL);
            ++npds1;
          }
          if (!ok) break;
          if (t == 0) {
            ok = mbar_wait_warp(acc_free, (nitem & 1) ^ 1, wc, B_ACC_FREE);
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t do_lo = lo_m + ((C::OFF_DO + s * C::PANEL) >> 4);
          const uint32_t acc0 = t > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ts2(tmem + C::COL_DV, tmem + C::COL_S + 64 * b + 8 * kc, do_lo + 128 * kc, hi_m, id_acc,
                       kc > 0 ? 1u : acc0);
            umma_commit(qdo_empty + s);
            umma_commit(pfree + b);
          }
          __syncwarp();
        }
        if (!ok) break;
      }
      if (leader) umma_commit(acc_full);
      __syncwarp();
    }
  } else if (warp >= 16 && warp < 20) {
    // ------------------------------------------------------------------ dQ drain warps (128 threads)
    const int q4 = warp & 3;                            // TMEM lane quarter of this warp
    const int rowl = q4 * 32 + lane;                    // query row within the tile
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    uint32_t ndq = 0;
    bool ok = true;
#ifdef SAF_TRACE
    int tr_n = 0;
#endif
    // Each drain warp moves the 32 query rows of its TMEM lane quarter on its own, through its own 4 KB of the staging
    // area: TMEM -> registers -> [32 rows][32 floats] box (128-byte swizzle: 16-byte chunk index ^= row & 7) -> tiled
    // TMA reduce-add, two boxes (feature halves) per tile.  A warp waits for its previous reduce-add to have read
    // the box only when it is about to write it again, so four small reduce-adds are in flight per CTA while the
    // warps stage the next ones (one 16 KB box per half, staged and reduced in turn by all four warps together,
    // kept these warps busy 90 % of a tile's time: they, not the tensor pipe, set the tile period).
    uint8_t* const my_box = smem + C::OFF_DQ + q4 * 4096;
    const uint32_t my_row = smem_u32(my_box) + lane * 128;
    (void)rowl;
    warp_arrive(pds_ord + 1);                           // the first tile finds the dQ accumulator free
    for (int it = it_begin; it < it_end && ok; ++it) {
      const WorkItem w = p.items[it];
      if (w.kind != KIND_ORDINARY) continue;
      const int qh = p.qslot ? p.qslot[w.h] : w.h;       // head index in the dQ accumulator
      for (int I = w.blk; I < nblk; ++I) {
        TR(4 + warp, 40);
        if (!mbar_wait_warp(dq_full, ndq & 1, wc, B_DQ_FULL)) {
          ok = false;
          break;
        }
        ++ndq;
        TR(4 + warp, 41);
        tc_fence_after();
        uint32_t r0[32], r1[32];
        tmem_ld32(tmem + lane_base + C::COL_DQ, r0);
        tmem_ld32(tmem + lane_base + C::COL_DQ + 32, r1);
        tmem_wait_ld();
        tc_fence_before();
        warp_arrive(pds_ord + 1);                       // the tensor core may overwrite dQ (counted in the next tile's phase)
        const int row_first = I * BLK + 32 * q4;         // sequence position of this warp's first row
#pragma unroll
        for (int box = 0; box < 2; ++box) {
          if (lane == 0) bulk_wait_group_read0();       // this warp's previous reduce-add has read the box
          __syncwarp();
          const uint32_t* r = box ? r1 : r0;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const uint32_t chunk = static_cast<uint32_t>(g ^ (lane & 7)) * 16;
            st_shared_v4(my_row + chunk, __float_as_uint(__uint_as_float(r[4 * g]) * p.scale),
                         __float_as_uint(__uint_as_float(r[4 * g + 1]) * p.scale),
                         __float_as_uint(__uint_as_float(r[4 * g + 2]) * p.scale),
                         __float_as_uint(__uint_as_float(r[4 * g + 3]) * p.scale));
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && row_first < p.T) {           // (rows beyond T inside the box are clipped by the map)
            tma_reduce_add_4d(&mdq, my_box, 32 * box, row_first, qh, w.b);
            bulk_commit_group();
          }
        }
        TR(4 + warp, 42);
      }
    }
    if (lane == 0) bulk_wait_group0();                  // the reduce-adds have landed before the kernel ends
  } else {
    // ------------------------------------------------------------------ compute groups (2 x 256 threads)
    // warp = 8 grp + 4 sub + q4: two warps per TMEM lane quarter, `sub` picks the 32-column half
    const int grp = warp >> 3, sub = (warp >> 2) & 1, q4 = warp & 3;
    const int gtid = tid & 255;                          // thread index within the group
    const int rowl = q4 * 32 + lane;                     // TMEM lane = key row of the block
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    float* tab = reinterpret_cast<float*>(smem + C::OFF_TAB) + grp * C::TAB_FLOATS;
    float* wq = tab;
    float* z2s = tab + 128;
    float* rband = tab + 256;
    float* r2raw = tab + 512;
    float* red = tab + 768;
    const int bar_id = 4 + grp;                          // named barrier of this group
    uint32_t nacc = 0, ntile_ord = 0, nsdp = 0, npf = 0, nkvc = 0;
    bool ok = true;
#ifdef SAF_TRACE
    int tr_n = 0;
#endif
    // K_J (group 0) / V_J (group 1) of the next ordinary item: this thread's half row from the swizzled
    // smem tile into TMEM as the A operand of the score MMAs (bf16 pairs, feature index = reduction index)
    // The fp32 epilogue leaves through TMA stores that read this group's dS^T panels; before the group
    // writes those panels again (dS^T of a first tile, or the next epilogue) the stores must have read them.
    // The two panels leave as separate bulk groups, the one that the next item's first tile writes first,
    // so that that tile only waits for half of the store.
    int store_pending = 0;                               // bulk groups possibly unread; uniform over the group
    auto staging_free = [&](int allow) {
      if (store_pending <= allow) return;
      if (gtid == 0) {
        if (allow == 0) bulk_wait_group_read0();
        else asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      }
      named_bar_sync(bar_id, 256);
      store_pending = allow;
    };
    bool kv_in_tmem = false;
    auto copy_kv = [&]() {
      const uint32_t ks = nkvc & 1;
      if (!mbar_wait_warp(kv_full + ks, (nkvc >> 1) & 1, wc, B_KV_FULL)) ok = false;
      ++nkvc;
      const uint32_t src = smem_u32(smem + (grp == 0 ? C::OFF_K + ks * C::PANEL : C::OFF_V)) + rowl * 128;
      uint32_t kvr[16];
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t a = src + static_cast<uint32_t>((4 * sub + g) ^ (rowl & 7)) * 16;
        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(kvr[4 * g]), "=r"(kvr[4 * g + 1]), "=r"(kvr[4 * g + 2]), "=r"(kvr[4 * g + 3])
                     : "r"(a)
                     : "memory");
      }
      tmem_st16(tmem + lane_base + (grp == 0 ? C::COL_KT : C::COL_VT) + 16 * sub, kvr);
      tmem_wait_st();
      tc_fence_before();
      warp_arrive(kvt_full);
    };
    // A warp whose wait was abandoned keeps walking (without storing) to the next agreement barrier,
    // where the warps of its group leave together; none is ever left alone at a named barrier.
    ItemView nxt = load_item(p, it_begin, it_end);
    for (int it = it_begin; it < it_end; ++it) {
      const WorkItem w = nxt.w;
      const bool fast = nxt.fast;                        // (the next item is fetched below, under the wait for the
                                                         // item's last MMAs, where its load latency costs nothing)
      const bool ord = w.kind == KIND_ORDINARY;
      const int ntiles = nblk - w.blk;
      int key = w.blk * BLK + rowl;
      const size_t bh = static_cast<size_t>(w.b) * p.H + w.h;
      float dv_mul = 1.0f;
      bool rev = false;                                  // tensor-core frozen form: lane m holds key 127-m
      bool stored = false;                               // this group staged an fp32 block for a TMA store
      if (named_bar_or(bar_id, 256, !ok)) break;

      if (fast) {
        // tensor-core form: nothing to do per tile; lane m holds key 127-m, scaled by a(j) below
        key = w.blk * BLK + 127 - rowl;
        rev = true;
        dv_mul = (key < p.T) ? p.avec[static_cast<size_t>(w.h) * p.Tp + key] * (1.0f / HK_BAND_SCALE) : 0.0f;
      } else if (ord) {
        const float c = p.scale_log2;
        if (!kv_in_tmem) copy_kv();                  // first ordinary item of this CTA
        for (int t = 0; t < ntiles; ++t) {
          // this group's half tile of tile t: queries 64*grp .. 64*grp+63; this warp's 32 of them
          TR(4 + warp, 11);
          if (!mbar_wait_warp(s_full + grp, nsdp & 1, wc, B_SDP_FULL)) ok = false;
          tc_fence_after();
          TR(4 + warp, 12);
          const uint32_t t_s = tmem + lane_base + C::COL_S + 64 * grp;
          const uint32_t t_dp = tmem + lane_base + C::COL_DP + 64 * grp;
          const uint32_t rowaddr =
              smem_u32(smem + C::OFF_DS + ((ntile_ord + t) & 1) * 2 * C::PANEL + grp * C::PANEL) + rowl * 128;
          const bool diag = (t == 0);
          // P^T of this warp's 32 query columns from S'^T alone; dP'^T is still on the tensor core
          uint32_t rs[32];
          tmem_ld32(t_s + 32 * sub, rs);
          tmem_wait_ld();
          {
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              float p0 = ex2_approx(__uint_as_float(rs[2 * e]) * c);
              float p1 = ex2_approx(__uint_as_float(rs[2 * e + 1]) * c);
              if (diag) {                                  // causal: query index >= key index
                const int qa = 64 * grp + 32 * sub + 2 * e;
                if (qa < rowl) p0 = 0.0f;
                if (qa + 1 < rowl) p1 = 0.0f;
              }
              rs[2 * e] = __float_as_uint(p0);
              rs[2 * e + 1] = __float_as_uint(p1);
              pk[e] = pack_bf16x2(p0, p1);
            }
            // bf16 pairs re-use columns this warp has already consumed
            tmem_st16(t_s + 32 * sub, pk);
          }
          if (!mbar_wait_warp(sdp_full + grp, nsdp & 1, wc, B_SDP_FULL)) ok = false;
          ++nsdp;
          tc_fence_after();
          if (t <= 1) staging_free(1 - t);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            uint32_t rd[16], dk[8];
            tmem_ld16(t_dp + 32 * sub + 16 * hh, rd);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e)
              dk[e] = pack_bf16x2(__uint_as_float(rs[16 * hh + 2 * e]) * __uint_as_float(rd[2 * e]),
                                  __uint_as_float(rs[16 * hh + 2 * e + 1]) * __uint_as_float(rd[2 * e + 1]));
            tmem_st8(t_dp + 32 * sub + 8 * hh, dk);
            // dS^T row (this key) -> smem panel of this half tile, 128-byte swizzle (chunk ^= row & 7)
#pragma unroll
            for (int g = 0; g < 2; ++g) {
              const uint32_t chunk = static_cast<uint32_t>((4 * sub + 2 * hh + g) ^ (rowl & 7));
              st_shared_v4(rowaddr + chunk * 16, dk[4 * g], dk[4 * g + 1], dk[4 * g + 2], dk[4 * g + 3]);
            }
          }
          tmem_wait_st();
          fence_proxy_async_smem();
          tc_fence_before();
          warp_arrive(pds_ord + grp);
          TR(4 + warp, 16);
        }
        ntile_ord += ntiles;
        // K_J / V_J of the next ordinary item go to TMEM now, ahead of this item's epilogue, so that its
        // score MMAs can start while the epilogue runs.  The last score MMAs of this item (both buffers)
        // must have read the old copies first.
        kv_in_tmem = false;
        for (int nx = it + 1; nx < it_end; ++nx)
          if (p.items[nx].kind == KIND_ORDINARY) {
            kv_in_tmem = true;
            break;
          }
        if (kv_in_tmem) {
          TR(4 + warp, 21);
          if (!mbar_wait_warp(sdp_full + (grp ^ 1), (nsdp - 1) & 1, wc, B_SDP_FULL)) ok = false;
          tc_fence_after();
          copy_kv();
          TR(4 + warp, 22);
        }
      } else {
        // ---------------- frozen head: P^^T tiles; group g generates tiles t = g, g+2, ...
        const float* alpha_h = p.alpha + static_cast<size_t>(w.h) * p.Tp;
        const float* rho_h = p.rho + static_cast<size_t>(w.h) * p.Tp;
        const float* logz_h = p.logZ + static_cast<size_t>(w.h) * p.Tp;
        const float a2 = (key < p.T) ? alpha_h[key] * LOG2E_B : -INFINITY;
        float ma = a2;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, o));
        // block maximum of alpha over the 128 keys: exchanged once per item through `red`
        if (lane == 0 && sub == 0) red[12 + q4] = ma;
        named_bar_sync(bar_id, 256);
        ma = fmaxf(fmaxf(red[12], red[13]), fmaxf(red[14], red[15]));
        const float aj = ex2_approx(a2 - ma);
        bool leave = false;
        int nmine = 0;
        for (int t = grp; t < ntiles; t += 2, ++nmine) {
          const int I = w.blk + t;
          if (named_bar_or(bar_id, 256, !ok)) {          // uniform over the group: leave together
            ok = false;
            leave = true;
            break;
          }
          const int d0 = t * BLK - 127;                  // band: distances d0 .. d0+254, index x = q - row + 127
          // band entry x = gtid (255 of them); the query terms are built by the first 128 threads
          const int da = d0 + gtid;
          const float r2a = (gtid < 255 && da >= 0 && da < p.T) ? rho_h[da] * LOG2E_B : -INFINITY;
          r2raw[gtid] = r2a;
          float mr = r2a;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o));
          if (lane == 0) red[4 * sub + q4] = mr;
          const int qi = I * BLK + (gtid & 127);
          const float z2 = (qi < p.T) ? logz_h[qi] * LOG2E_B : INFINITY;
          if (sub == 0) z2s[gtid] = z2;
          named_bar_sync(bar_id, 256);
          mr = fmaxf(fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3])),
                     fmaxf(fmaxf(red[4], red[5]), fmaxf(red[6], red[7])));
          rband[gtid] = ex2_approx(r2a - mr);
          const float ew = ma + mr - z2;
          if (sub == 0) wq[gtid] = ex2_approx(ew);
          const unsigned anybad = __any_sync(0xffffffffu, ew > 100.0f);
          if (lane == 0 && sub == 0) red[8 + q4] = anybad ? 1.0f : 0.0f;
          named_bar_sync(bar_id, 256);
          const bool exact = (red[8] + red[9] + red[10] + red[11]) > 0.0f;
          // this group's buffer must have been consumed by the dV MMA of its previous tile
          if (nmine > 0) {
            if (!mbar_wait_warp(pfree + grp, npf & 1, wc, B_PFREE)) ok = false;
            ++npf;
            tc_fence_after();
          }
          const uint32_t t_p = tmem + lane_base + C::COL_S + grp * 64;
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            const int cc = 2 * sub + ch;                  // this warp's 32-query chunks of the tile
            const int q0 = 32 * cc;
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
            tmem_st16(t_p + 16 * cc, pk);
          }
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(pds_full + grp);
        }
        if (leave) break;
        // keep the buffer barrier in step: absorb the completion of this group's last tile
        if (nmine > 0) {
          if (!mbar_wait_warp(pfree + grp, npf & 1, wc, B_PFREE)) ok = false;
          ++npf;
        }
      }
      // ---------------- epilogue: dV (group 0) and dK (group 1) of this key block
      nxt = load_item(p, it + 1, it_end);
      if (!mbar_wait_warp(acc_full, nacc & 1, wc, B_ACC_FULL)) ok = false;
      ++nacc;
      tc_fence_after();
      TR(4 + warp, 23);
      if (grp == 0 || ord) {
        const uint32_t col = grp == 0 ? C::COL_DV : C::COL_DK;
        const float mul = grp == 0 ? dv_mul : p.scale;
        void* base = grp == 0 ? p.dV : p.dK;
        const size_t bho = (grp == 1 && p.qslot) ? static_cast<size_t>(w.b) * p.n_ord + p.qslot[w.h] : bh;
        const size_t off = (bho * p.T + key) * 64;
        {
          const int cc = sub;                             // this warp's 32 feature columns
          uint32_t r[32];
          tmem_ld32(tmem + lane_base + col + 32 * cc, r);
          tmem_wait_ld();
          tc_fence_before();
          warp_arrive(acc_free);                          // the accumulators may be overwritten
          TR(4 + warp, 25);
          if (p.grad_f32) {
            staging_free(0);
            // fp32 rows go through the (idle) dS^T buffers as two 128-byte-swizzled [128][32] boxes and
            // leave with tiled TMA stores (rows beyond T are clipped).  A group stages inside the panels
            // it writes dS^T to itself, since the other group may already be in the next item.
            const int srow_i = rev ? 127 - rowl : rowl;
            const uint32_t srow =
                smem_u32(smem + C::OFF_DS + (2 * sub + grp) * C::PANEL) + static_cast<uint32_t>(srow_i) * 128;
#pragma unroll
            for (int g = 0; g < 8; ++g)
              st_shared_v4(srow + static_cast<uint32_t>(g ^ (srow_i & 7)) * 16,
                           __float_as_uint(__uint_as_float(r[4 * g]) * mul),
                           __float_as_uint(__uint_as_float(r[4 * g + 1]) * mul),
                           __float_as_uint(__uint_as_float(r[4 * g + 2]) * mul),
                           __float_as_uint(__uint_as_float(r[4 * g + 3]) * mul));
            TR(4 + warp, 26);
            fence_proxy_async_smem();
            TR(4 + warp, 27);
            stored = true;
          } else if (key < p.T && ok) {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + off + 32 * cc);
#pragma unroll
              for (int e = 0; e < 4; ++e)
                dst[e] = make_uint4(pack_bf16x2(__uint_as_float(r[8 * e]) * mul, __uint_as_float(r[8 * e + 1]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 2]) * mul, __uint_as_float(r[8 * e + 3]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 4]) * mul, __uint_as_float(r[8 * e + 5]) * mul),
                                    pack_bf16x2(__uint_as_float(r[8 * e + 6]) * mul, __uint_as_float(r[8 * e + 7]) * mul));
          }
        }
      } else {
        tc_fence_before();
        warp_arrive(acc_free);
      }
      if (stored) {                                      // uniform over the group
        named_bar_sync(bar_id, 256);
        TR(4 + warp, 28);
        if (gtid == 0 && ok) {
          const CUtensorMap* m = grp == 0 ? &mdv : &mdk;
          const int first = ntile_ord & 1;              // dS^T buffer of the next ordinary tile
          const uint8_t* src0 = smem + C::OFF_DS + (2 * first + grp) * C::PANEL;
          const uint8_t* src1 = smem + C::OFF_DS + (2 * (first ^ 1) + grp) * C::PANEL;
          if (p.kv_group > 1) {
            // grouped-query path: the query heads of a group add into their shared head's gradient
            const int kvh = w.h / p.kv_group;
            tma_reduce_add_4d(m, src0, 32 * first, w.blk * BLK, kvh, w.b);
            bulk_commit_group();
            tma_reduce_add_4d(m, src1, 32 * (first ^ 1), w.blk * BLK, kvh, w.b);
            bulk_commit_group();
          } else {
            // (packed layout: dK has the ordinary heads only)
            const int oh = (grp == 1 && p.qslot) ? p.qslot[w.h] : w.h;
            tma_store_4d(m, src0, 32 * first, w.blk * BLK, oh, w.b);
            bulk_commit_group();
            tma_store_4d(m, src1, 32 * (first ^ 1), w.blk * BLK, oh, w.b);
            bulk_commit_group();
          }
        }
        store_pending = 2;
      }
      TR(4 + warp, 24);
    }
    if (gtid == 0) bulk_wait_group0();                   // the stores have landed before the kernel ends
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
  SAF_SPAN(bwd, 1);
  if (warp == 21) tmem_dealloc(tmem, C::TMEM_COLS);
}

int bwd_smem_bytes(int) { return BwdCfg::SMEM; }

cudaError_t launch_bwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mdo, const CUtensorMap& mdq, const CUtensorMap& mdot, const CUtensorMap& mdk,
                       const CUtensorMap& mdv, const BwdParams& p, int grid, cudaStream_t st) {
  if (D != 64) return cudaErrorNotSupported;
  cudaError_t e = cudaFuncSetAttribute(saf_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg::SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(PDL_BWD, saf_bwd_kernel, dim3(grid), dim3(BwdCfg::NTHREADS), BwdCfg::SMEM, st, mq, mk, mv, mdo,
                    mdq, mdot, mdk, mdv, p);
}

}  // namespace saf
