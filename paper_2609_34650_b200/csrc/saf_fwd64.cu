// Forward of the hybrid causal attention layer on sm_100a, head dimension 64: one persistent kernel for
// ordinary (flash-style online softmax) and frozen (pattern rebuilt from alpha/rho/logZ) heads.
//
// The softmax of a tile is a serial chain (score MMA -> row max -> exponentials -> P V MMA) whose
// exponentials are bound by the 16-per-clock special-function unit; to keep that unit busy the kernel runs
// four such chains per SM: two CTAs per SM, and in each CTA two compute groups that split every 128-key
// tile into its two 64-key halves.  A group keeps its own running maximum, row sum and output accumulator
// for its key half; the two partial results are merged once per item in the epilogue
// (O = (f0 O_0 + f1 O_1) / (f0 l_0 + f1 l_1), f_g = 2^(m_g - max(m_0, m_1))).
//
// Per CTA (320 threads): warps 0-3 = compute group 0 (keys 0-63 of a tile), warps 4-7 = group 1 (keys
// 64-127), one thread per query row (= TMEM lane) in each group; warp 8 = TMA producer; warp 9 = tcgen05
// issuer and TMEM owner.  TMEM columns: [0,64) S_0, [64,128) S_1 (fp32 scores; the bf16 P pairs of a group
// re-use the first 32 columns of its own S buffer), [128,192) O_0, [192,256) O_1.
//
// Ordinary item (b,h,I): for J = 0..I: S_g = Q_I K_J[64g..]^T (operands in 128B-swizzled smem via TMA),
//   row max / lazy rescale / exp2 / row sum in registers, P_g -> TMEM as bf16, O_g += P_g V_J[64g..]
//   (A from TMEM, V as MN-major B).  The issuer queues the next tile's score MMA of a group right behind
//   its P V MMA: MMAs of one thread execute in issue order, so no completion round trip is needed.
// Frozen item (b,h,I): for J = 0..I: P^(i,j) = exp(alpha(j) + rho(i-j) - logZ(i)) for j <= i
//   (Eq. "compact-prior" with the stored normaliser) generated into TMEM, O_g += P^_g V_J[64g..].  No Q/K
//   loads, no score MMA, no max/sum.  The exponential is factorised per tile as w(i) * a(j) * r(i-j) with
//   a = exp(alpha - max_tile alpha), r = exp(rho - max_band rho), w = exp(max alpha + max rho - logZ(i));
//   a tile whose exponent range would leave fp32 falls back to one exp per element.
// Frozen item, tensor-core form (pattern tables prepared and the head's flag set): with global maxima,
//   O = diag(w) R (diag(a) V), R(i,j) = r(i-j).  A tile of R with reversed rows is a Hankel matrix that the
//   tensor core reads straight from a 4 KB band table (no-swizzle descriptor, both strides 128 bytes), so
//   a tile is one bulk copy of the band, one TMA load of the a-scaled V tile and 8 MMAs into O_0; the compute
//   warps only scale the finished rows by w(i) (TMEM lane m holds query 127-m of the block).  These tiles run
//   a ring of their own, three deep, laid over the K and V stages and the Q tile.
// Epilogue of every item: the merged, scaled O tile is written into a swizzled staging tile and leaves by one
//   TMA store (rows beyond T are clipped by the tensor map).
#include <cuda_bf16.h>
#include "ptx.cuh"
#include "saf_internal.h"

#ifdef SAF_TRACE
__device__ unsigned long long g_saf_trace_fwd[4][16384];
#define TRF(role, id)                                                                                  \
  do {                                                                                                 \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && tr_n < 16380)                                    \
      g_saf_trace_fwd[role][tr_n++] = (static_cast<unsigned long long>(id) << 48) | (clock64() & 0xffffffffffffULL); \
  } while (0)
extern "C" int saf_debug_read_trace_fwd(unsigned long long* out) {
  return static_cast<int>(cudaMemcpyFromSymbol(out, g_saf_trace_fwd, sizeof(g_saf_trace_fwd)));
}
#else
#define TRF(role, id)
#endif

SAF_SPAN_DEFINE(fwd64)

namespace saf {

namespace {

constexpr float LOG2E_G = 1.4426950408889634f;
constexpr float LN2_G = 0.6931471805599453f;

struct Fwd64Cfg {
  static constexpr int TILE_BYTES = 128 * 64 * 2;       // one [128][64] bf16 tile, 128-byte rows, 16 KB
  static constexpr int HALF_BYTES = TILE_BYTES / 2;     // its rows 64..127
  static constexpr int NS = 2;                          // K and V ring depth
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = TILE_BYTES;
  static constexpr int OFF_V = OFF_K + NS * TILE_BYTES;
  static constexpr int OFF_OST = OFF_V + NS * TILE_BYTES;   // O tile staged for its TMA store (128-byte swizzle)
  static constexpr int OFF_TAB = OFF_OST + TILE_BYTES;
  // floats: aJ[128] rband[256] a2raw[128] r2raw[256] red[32] ml[2][2][128]
  static constexpr int TAB_FLOATS = 128 + 256 + 128 + 256 + 32 + 512;
  static constexpr int OFF_BAR = OFF_TAB + TAB_FLOATS * 4;
  // Ring of the tensor-core frozen form, three deep (its tiles have no compute step to hide the load latency
  // behind): slot k keeps its scaled V tile in V stage k (k < 2) or in the Q tile (k = 2) and its 4 KB band in the
  // K ring's area.
  static constexpr int NFZ = 3;
  __host__ __device__ static constexpr int fz_v(int k) { return k < 2 ? OFF_V + k * TILE_BYTES : OFF_Q; }
  __host__ __device__ static constexpr int fz_band(int k) { return OFF_K + k * 4096; }
  // Work items are claimed at run time (atomic counter in global memory) by the producer thread, which hands them
  // to the other roles through a ring of NRING records in shared memory.
  static constexpr int NRING = 4;
  static constexpr int NBAR = 2 + 4 * NS + 2 + 2 + 2 + 1 + 2 * NFZ + 2 * NRING;
  static constexpr int OFF_RING = (OFF_BAR + NBAR * 8 + 16 + 15) / 16 * 16;   // int4 records (after the barriers, the TMEM slot
                                                                // and the abort flag)
  static constexpr int SMEM = OFF_RING + NRING * 16 + 1024;     // + slack for 1024-byte alignment
  static constexpr int TMEM_COLS = 256;
  static constexpr int COL_S = 0, COL_O = 128;          // + 64 g
  static constexpr int NTHREADS = 320;
};

enum Fwd64Site { F_Q_EMPTY = 41, F_K_EMPTY, F_V_EMPTY, F_Q_FULL, F_K_FULL, F_P_FULL, F_V_FULL, F_O_FREE, F_S_FULL,
                 F_PV_DONE, F_RING_EMPTY, F_RING_FULL };

// A work item as the roles see it: the record of the scheduler's list plus whether a frozen item takes the
// tensor-core form.  kind < 0 marks the end of the queue.
struct ItemView64 {
  WorkItem w;
  bool fast;
};
constexpr int RING_FAST = 1 << 8;
constexpr int RING_END = -1;

// Consumer side of the item ring (warp-uniform): wait for record n, copy it, release the slot at once (the copy is
// all a role needs).  Returns false when the wait was abandoned.
__device__ __forceinline__ bool ring_take(const int4* ring, uint64_t* ring_full, uint64_t* ring_empty, uint32_t n,
                                          const WaitCtx& wc, ItemView64& v) {
  const uint32_t slot = n % Fwd64Cfg::NRING;
  if (!mbar_wait_warp(ring_full + slot, (n / Fwd64Cfg::NRING) & 1, wc, F_RING_FULL)) return false;
  const int4 raw = ring[slot];
  warp_arrive(ring_empty + slot);
  v.w = WorkItem{raw.x, raw.y, raw.z, raw.w < 0 ? RING_END : (raw.w & 0xff)};
  v.fast = raw.w >= 0 && (raw.w & RING_FAST) != 0;
  return true;
}

}  // namespace

template <bool OF32>
__global__ void __launch_bounds__(320, 2)
saf_fwd64_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                 const __grid_constant__ CUtensorMap mv, const __grid_constant__ CUtensorMap mvt,
                 const __grid_constant__ CUtensorMap mo, const FwdParams p) {
  using C = Fwd64Cfg;
  constexpr int D = 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  uint64_t* q_full = bars;
  uint64_t* q_empty = bars + 1;
  uint64_t* k_full = bars + 2;
  uint64_t* k_empty = k_full + C::NS;
  uint64_t* v_full = k_empty + C::NS;
  uint64_t* v_empty = v_full + C::NS;
  uint64_t* s_full = v_empty + C::NS;            // [2] the score MMA of group g's key half has completed
  uint64_t* p_full = s_full + 2;                 // [2] group g has written its P pairs (4 warp arrivals)
  uint64_t* pv_done = p_full + 2;                // [2] P V MMAs of group g have completed (see the issuer)
  uint64_t* o_free = pv_done + 2;
  uint64_t* fz_full = o_free + 1;                // [NFZ] band + scaled V tile of a tensor-core frozen tile
  uint64_t* fz_empty = fz_full + C::NFZ;         // [NFZ]
  uint64_t* ring_full = fz_empty + C::NFZ;       // [NRING] record n has been published by the producer
  uint64_t* ring_empty = ring_full + C::NRING;   // [NRING] issuer + 8 compute warps have copied it
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ring_empty + C::NRING);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int4* ring = reinterpret_cast<int4*>(smem + C::OFF_RING);
  float* tab = reinterpret_cast<float*>(smem + C::OFF_TAB);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{abort_flag, p.status, p.wait_limit_ns};
  SAF_SPAN(fwd64, 0);
#ifdef SAF_TRACE
  int tr_n = 0;
#endif

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
    for (int g = 0; g < 2; ++g) {
      mbar_init(s_full + g, 1);
      mbar_init(p_full + g, 4);                  // one arrival per warp of the group
      mbar_init(pv_done + g, 1);
    }
    mbar_init(o_free, 8);
    for (int k = 0; k < C::NFZ; ++k) {
      mbar_init(fz_full + k, 1);
      mbar_init(fz_empty + k, 1);
    }
    for (int k = 0; k < C::NRING; ++k) {
      mbar_init(ring_full + k, 1);
      mbar_init(ring_empty + k, 9);
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
  // the prologue above overlapped the previous kernel's tail; global memory is touched only from here on
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&mq);
      tma_prefetch_desc(&mk);
      tma_prefetch_desc(&mv);
      tma_prefetch_desc(&mvt);
      uint32_t nq = 0, nk = 0, nv = 0, nfz = 0;
      bool ok = true, fz_open = false;
      bool drop_load = p.selftest_drop_load != 0;        // self-test of the give-up path: see FwdParams
      for (uint32_t nclaim = 0; ok; ++nclaim) {
        // claim the next item of the queue and publish it to the other roles
        const uint32_t slot = nclaim % C::NRING;
        ok = mbar_wait(ring_empty + slot, ((nclaim / C::NRING) & 1) ^ 1, wc, F_RING_EMPTY);
        if (!ok) break;
        const int idx = atomicAdd(p.queue, 1);
        int4 rec = make_int4(0, 0, 0, RING_END);
        bool fast = false;
        if (idx < p.n_items) {
          rec = __ldg(reinterpret_cast<const int4*>(p.order + idx));
          fast = rec.w != KIND_ORDINARY && p.band_f != nullptr && __ldg(p.fast_ok + rec.y) != 0 &&
                 __ldg(p.ovf + rec.y) != p.call_id;
          if (fast) rec.w |= RING_FAST;
        }
        ring[slot] = rec;
        mbar_arrive(ring_full + slot);                   // (release: the record is visible to whoever sees the phase)
        if (idx >= p.n_items) break;
        const WorkItem w = WorkItem{rec.x, rec.y, rec.z, rec.w & 0xff};
        const int ntiles = w.blk + 1;
        if (fast) {
          // tensor-core form: per tile the Hankel band of distance block (I - J) and the scaled V tile, in a ring of
          // their own laid over the K and V stages and the Q tile
          if (!fz_open) {
            // the last tiles that went through those stages must have been consumed
            for (uint32_t n = nk > C::NS ? nk - C::NS : 0; n < nk && ok; ++n)
              ok = mbar_wait(k_empty + n % C::NS, (n / C::NS) & 1, wc, F_K_EMPTY);
            for (uint32_t n = nv > C::NS ? nv - C::NS : 0; n < nv && ok; ++n)
              ok = mbar_wait(v_empty + n % C::NS, (n / C::NS) & 1, wc, F_V_EMPTY);
            if (ok && nq > 0) ok = mbar_wait(q_empty, (nq - 1) & 1, wc, F_Q_EMPTY);
            if (!ok) break;
            fz_open = true;
          }
          const int ord = p.hord[w.h];
          const uint8_t* bands = static_cast<const uint8_t*>(p.band_f) + static_cast<size_t>(w.h) * p.nblkp * 4096;
          for (int j = 0; j < ntiles; ++j) {
            const uint32_t k = nfz % C::NFZ;
            ok = mbar_wait(fz_empty + k, ((nfz / C::NFZ) & 1) ^ 1, wc, F_V_EMPTY);
            if (!ok) break;
            mbar_expect_tx(fz_full + k, C::TILE_BYTES + 4096);
            bulk_load(smem + C::fz_band(k), bands + static_cast<size_t>(w.blk - j) * 4096, 4096, fz_full + k);
            tma_load_4d(smem + C::fz_v(k), &mvt, fz_full + k, 0, j * BLK, ord, w.b);
            ++nfz;
          }
          continue;
        }
        if (fz_open) {
          // back to the ordinary stages: the frozen ring's tiles in flight must have been consumed
          for (uint32_t n = nfz > C::NFZ ? nfz - C::NFZ : 0; n < nfz && ok; ++n)
            ok = mbar_wait(fz_empty + n % C::NFZ, (n / C::NFZ) & 1, wc, F_V_EMPTY);
          if (!ok) break;
          fz_open = false;
        }
        const bool ord = w.kind == KIND_ORDINARY;
        const int kh = !ord ? 0 : (p.qslot ? p.qslot[w.h] : w.h / p.kv_group);   // head index in the K tensor
        if (ord) {
          ok = mbar_wait(q_empty, (nq & 1) ^ 1, wc, F_Q_EMPTY);
          if (!ok) break;
          mbar_expect_tx(q_full, C::TILE_BYTES);
          tma_load_4d(smem + C::OFF_Q, &mq, q_full, 0, w.blk * BLK, p.qslot ? p.qslot[w.h] : w.h, w.b);
          ++nq;
        }
        for (int j = 0; j < ntiles && ok; ++j) {
          if (ord) {
            const int s = nk % C::NS;
            ok = mbar_wait(k_empty + s, ((nk / C::NS) & 1) ^ 1, wc, F_K_EMPTY);
            if (!ok) break;
            if (!drop_load) {
              mbar_expect_tx(k_full + s, C::TILE_BYTES);
              tma_load_4d(smem + C::OFF_K + s * C::TILE_BYTES, &mk, k_full + s, 0, j * BLK, kh, w.b);
            }
            drop_load = false;
            ++nk;
          }
          const int s = nv % C::NS;
          ok = mbar_wait(v_empty + s, ((nv / C::NS) & 1) ^ 1, wc, F_V_EMPTY);
          if (!ok) break;
          mbar_expect_tx(v_full + s, C::TILE_BYTES);
          tma_load_4d(smem + C::OFF_V + s * C::TILE_BYTES, &mv, v_full + s, 0, j * BLK, w.h / p.kv_group, w.b);
          ++nv;
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ tcgen05 issuer
    // The whole warp walks the loops (warp-uniform operands); one elected lane issues.
    const bool leader = elect_one() != 0;
    const uint32_t sb = smem_u32(smem);
    constexpr uint32_t idesc_s = umma_idesc_bf16(128, 64, 0, 0);   // S_g: 128 queries x 64 keys, both K-major
    constexpr uint32_t idesc_o = umma_idesc_bf16(128, D, 0, 1);    // O_g: A = P_g from TMEM, B = V rows MN-major
    constexpr uint32_t idesc_hk = umma_idesc_f16(128, D, 0, 1);    // tensor-core frozen form: fp16 band x fp16 scaled V
    uint32_t nq = 0, nk = 0, nv = 0, nitem = 0, nfz = 0;
    uint32_t np0 = 0, np1 = 0;
    bool ok = true;
    // descriptor halves for smem offset 0: K-major tiles (k-step +32 B) and the MN-major V tile (k-step
    // +2048 B); rows 64.. of either tile start 8 KB in
    const uint64_t d_kmaj = umma_smem_desc(sb, 16, 1024, UMMA_LAYOUT_SW128);
    const uint64_t d_mn = umma_smem_desc(sb, C::TILE_BYTES, 1024, UMMA_LAYOUT_SW128);
    const uint32_t lo_k = desc_lo(d_kmaj), hi_k = desc_hi(d_kmaj), lo_m = desc_lo(d_mn), hi_m = desc_hi(d_mn);
    const uint32_t q_lo = lo_k + (C::OFF_Q >> 4);
    // Hankel band: no-swizzle K-major, core matrices 128 bytes apart in both directions
    const uint64_t d_band = umma_smem_desc(sb, 128, 128, UMMA_LAYOUT_NONE);
    const uint32_t lo_b = desc_lo(d_band), hi_b = desc_hi(d_band);
    for (uint32_t nrec = 0; ok; ++nrec, ++nitem) {
      ItemView64 cur;
      ok = ring_take(ring, ring_full, ring_empty, nrec, wc, cur);
      if (!ok || cur.w.kind == RING_END) break;
      const WorkItem w = cur.w;
      const bool fast = cur.fast;
      const int ntiles = w.blk + 1;
      const bool ord = w.kind == KIND_ORDINARY;
      if (fast) {
        for (int j = 0; j < ntiles && ok; ++j) {
          const uint32_t k = nfz % C::NFZ;
          ok = mbar_wait_warp(fz_full + k, (nfz / C::NFZ) & 1, wc, F_V_FULL);
          if (!ok) break;
          ++nfz;
          if (j == 0) {
            ok = mbar_wait_warp(o_free, (nitem & 1) ^ 1, wc, F_O_FREE);
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t band_lo = lo_b + (static_cast<uint32_t>(C::fz_band(k)) >> 4);
          const uint32_t v_lo = lo_m + (static_cast<uint32_t>(C::fz_v(k)) >> 4);
          const uint32_t acc0 = j > 0 ? 1u : 0u;
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 8; ++kc)
              umma_ss2(tmem + C::COL_O, band_lo + 16 * kc, hi_b, v_lo + 128 * kc, hi_m, idesc_hk, kc > 0 ? 1u : acc0);
            umma_commit(fz_empty + k);
            if (j == ntiles - 1) {
              umma_commit(pv_done);
              umma_commit(pv_done + 1);
            }
          }
          __syncwarp();
        }
        continue;
      }
      if (ord) {
        // score MMA of group g for the tile in K stage s; P V MMA of group g for the tile in V stage s
        auto issue_qk = [&](uint32_t g, uint32_t s) {
          const uint32_t k_lo = lo_k + ((C::OFF_K + s * C::TILE_BYTES + g * C::HALF_BYTES) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ss2(tmem + C::COL_S + 64 * g, q_lo + 2 * kc, hi_k, k_lo + 2 * kc, hi_k, idesc_s, kc > 0);
            umma_commit(s_full + g);
          }
          __syncwarp();
        };
        auto issue_pv = [&](uint32_t g, uint32_t s, uint32_t acc0) {
          const uint32_t v_lo = lo_m + ((C::OFF_V + s * C::TILE_BYTES + g * C::HALF_BYTES) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ts2(tmem + C::COL_O + 64 * g, tmem + C::COL_S + 64 * g + 8 * kc, v_lo + 128 * kc, hi_m, idesc_o,
                       kc > 0 ? 1u : acc0);
          }
          __syncwarp();
        };
        ok = mbar_wait_warp(q_full, nq & 1, wc, F_Q_FULL);
        if (!ok) break;
        ++nq;
        {
          const uint32_t s = nk % C::NS;
          ok = mbar_wait_warp(k_full + s, (nk / C::NS) & 1, wc, F_K_FULL);
          if (!ok) break;
          ++nk;
          tc_fence_after();
          issue_qk(0, s);
          issue_qk(1, s);
          if (leader) umma_commit(k_empty + s);
          __syncwarp();
        }
        for (int j = 0; j < ntiles && ok; ++j) {
          const uint32_t sv = nv % C::NS;
          const bool more = j + 1 < ntiles;
          const uint32_t sk = nk % C::NS;                 // stage of tile j+1's K (if any)
          const uint32_t acc0 = j > 0 ? 1u : 0u;
          // ---- group 0
          // the tiles' loads land long before P is ready: test their barriers first, so that only one test
          // stands between "P is ready" and the MMAs that wait for it
          ok = mbar_wait_warp(v_full + sv, (nv / C::NS) & 1, wc, F_V_FULL);
          if (!ok) break;
          ++nv;
          if (more) {
            ok = mbar_wait_warp(k_full + sk, (nk / C::NS) & 1, wc, F_K_FULL);
            if (!ok) break;
            ++nk;
          }
          if (j == 0) {
            ok = mbar_wait_warp(o_free, (nitem & 1) ^ 1, wc, F_O_FREE);
            if (!ok) break;
          }
          ok = mbar_wait_warp(p_full, np0 & 1, wc, F_P_FULL);
          if (!ok) break;
          ++np0;
          tc_fence_after();
          issue_pv(0, sv, acc0);
          if (more) issue_qk(0, sk);                      // executes after P V_0: same thread, in order
          // ---- group 1
          ok = mbar_wait_warp(p_full + 1, np1 & 1, wc, F_P_FULL);
          if (!ok) break;
          ++np1;
          tc_fence_after();
          TRF(0, 4);
          issue_pv(1, sv, acc0);
          TRF(0, 5);
          if (leader) umma_commit(v_empty + sv);
          if (more) {
            issue_qk(1, sk);
            if (leader) umma_commit(k_empty + sk);
            TRF(0, 6);
          } else if (leader) {
            umma_commit(q_empty);
            umma_commit(pv_done);
            umma_commit(pv_done + 1);
          }
          __syncwarp();
        }
        continue;
      }
      // generic frozen item: P^ halves written by the groups, one P V MMA per group and tile
      for (int j = 0; j < ntiles && ok; ++j) {
        const uint32_t sv = nv % C::NS;
        ok = mbar_wait_warp(v_full + sv, (nv / C::NS) & 1, wc, F_V_FULL);
        if (!ok) break;
        ++nv;
        if (j == 0) {
          ok = mbar_wait_warp(o_free, (nitem & 1) ^ 1, wc, F_O_FREE);
          if (!ok) break;
        }
        const uint32_t acc0 = j > 0 ? 1u : 0u;
        for (uint32_t g = 0; g < 2 && ok; ++g) {
          if (g == 0) {
            ok = mbar_wait_warp(p_full, np0 & 1, wc, F_P_FULL);
            ++np0;
          } else {
            ok = mbar_wait_warp(p_full + 1, np1 & 1, wc, F_P_FULL);
            ++np1;
          }
          if (!ok) break;
          tc_fence_after();
          const uint32_t v_lo = lo_m + ((C::OFF_V + sv * C::TILE_BYTES + g * C::HALF_BYTES) >> 4);
          if (leader) {
#pragma unroll
            for (int kc = 0; kc < 4; ++kc)
              umma_ts2(tmem + C::COL_O + 64 * g, tmem + C::COL_S + 64 * g + 8 * kc, v_lo + 128 * kc, hi_m, idesc_o,
                       kc > 0 ? 1u : acc0);
            umma_commit(pv_done + g);                    // the group may overwrite its P^ half
            if (g == 1) umma_commit(v_empty + sv);
          }
          __syncwarp();
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ compute groups (2 x 128 threads)
    const int q4 = warp & 3, g = warp >> 2;
    const int rowl = q4 * 32 + lane;                   // query row within the tile = TMEM lane
    const int pair_bar = 1 + q4;                       // named barrier of the two warps sharing this lane quarter
    const uint32_t lane_base = static_cast<uint32_t>(q4 * 32) << 16;
    const uint32_t t_s = tmem + lane_base + C::COL_S + 64 * g;        // this group's score columns / P pairs
    const uint32_t t_o = tmem + lane_base + C::COL_O + 64 * g;        // this group's accumulator
    float* aJ = tab;
    float* rband = tab + 128;
    float* a2raw = tab + 384;
    float* r2raw = tab + 512;
    float* red = tab + 768;
    float* ml = tab + 800;                             // [g][m, l][row]
    uint32_t ns = 0, npv = 0;
    bool ok = true;
    const int trr = 1 + g;
    (void)trr;
    // A compute warp whose wait was abandoned keeps walking (without storing) until the next
    // agreement barrier, where all eight leave together; none is ever left alone at a barrier.
    for (uint32_t nrec = 0;; ++nrec) {
      ItemView64 cur;
      if (!ring_take(ring, ring_full, ring_empty, nrec, wc, cur)) {
        ok = false;                                      // keep walking to the agreement barrier below
        cur.w = WorkItem{0, 0, 0, KIND_ORDINARY};
        cur.fast = false;
      }
      const bool at_end = cur.w.kind == RING_END;
      const WorkItem w = cur.w;
      const bool fast = cur.fast;
      const int ntiles = w.blk + 1;
      int row = w.blk * BLK + rowl;
      // epilogue weights of the two accumulators and the common row factor
      float f0 = 1.0f, f1 = 1.0f, inv_l = 1.0f, lse = 0.0f;
      bool use1 = true;
      if (tid == 0) bulk_wait_group_read0();             // the previous item's O tile has left the staging tile
      if (named_bar_or(5, 256, !ok) || at_end) break;    // (the end record reaches all eight warps alike)
      if (q4 == 0) TRF(trr, 19);
      if (fast) {
        // tensor-core form: nothing to do per tile; lane m holds query 127-m, scaled by w(i) below
        row = w.blk * BLK + 127 - rowl;
        inv_l = (row < p.T) ? p.wvec[static_cast<size_t>(w.h) * p.Tp + row] * (1.0f / (HK_BAND_SCALE * HK_A_SCALE)) : 0.0f;
        use1 = false;
      } else if (w.kind == KIND_ORDINARY) {
        float m_ref = -INFINITY, l = 0.0f;
        const float c = p.scale_log2;
        for (int j = 0; j < ntiles; ++j) {
          if (q4 == 0) TRF(trr, 11);
          // (the completion of this score MMA also covers the group's previous P V MMA, issued before it)
          if (!mbar_wait_warp(s_full + g, ns & 1, wc, F_S_FULL)) ok = false;
          ++ns;
          tc_fence_after();
          if (q4 == 0) TRF(trr, 12);
          const bool diag = (j == w.blk);
          uint32_t r0[32], r1[32];
          tmem_ld32(t_s, r0);
          tmem_ld32(t_s + 32, r1);
          tmem_wait_ld();
          if (diag) {
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              if (64 * g + e > rowl) r0[e] = 0xff800000u;          // -inf above the diagonal
              if (64 * g + 32 + e > rowl) r1[e] = 0xff800000u;
            }
          }
          float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            mx0 = fmaxf(mx0, __uint_as_float(r0[e]));
            mx1 = fmaxf(mx1, __uint_as_float(r1[e]));
          }
          const float mx = fmaxf(mx0, mx1);
          if (q4 == 0) TRF(trr, 13);
          const float m_new = fmaxf(m_ref, mx * c);      // stays -inf while every key so far is masked
          if (j == 0) {
            m_ref = m_new;
          } else {
            const bool need = (m_new - m_ref) > 8.0f;    // false when both are -inf (NaN compares false)
            if (__any_sync(0xffffffffu, need)) {
              const float f = need ? ex2_approx(m_ref - m_new) : 1.0f;
              l *= f;
              if (need) m_ref = m_new;
#pragma unroll
              for (int cc = 0; cc < 4; ++cc) {
                uint32_t r[16];
                tmem_ld16(t_o + 16 * cc, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 16; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * f);
                tmem_st16(t_o + 16 * cc, r);
              }
            }
          }
          const float neg_m = (m_ref == -INFINITY) ? 0.0f : -m_ref;   // all-masked rows: exp2(-inf) = 0
          float l0 = 0.0f, l1 = 0.0f;
          {
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float a0 = ex2_approx(fmaf(__uint_as_float(r0[2 * e]), c, neg_m));
              const float a1 = ex2_approx(fmaf(__uint_as_float(r0[2 * e + 1]), c, neg_m));
              l0 += a0;
              l1 += a1;
              pk[e] = pack_bf16x2(a0, a1);
            }
            tmem_st16(t_s, pk);
          }
          {
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float b0 = ex2_approx(fmaf(__uint_as_float(r1[2 * e]), c, neg_m));
              const float b1 = ex2_approx(fmaf(__uint_as_float(r1[2 * e + 1]), c, neg_m));
              l0 += b0;
              l1 += b1;
              pk[e] = pack_bf16x2(b0, b1);
            }
            tmem_st16(t_s + 16, pk);
          }
          l += l0 + l1;
          if (q4 == 0) TRF(trr, 15);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(p_full + g);
          if (q4 == 0) TRF(trr, 16);
        }
        // merge the two key halves: common maximum, weights, row sum
        ml[g * 256 + rowl] = m_ref;
        ml[g * 256 + 128 + rowl] = l;
        named_bar_sync(pair_bar, 64);
        const float m0 = ml[rowl], l0s = ml[128 + rowl], m1 = ml[256 + rowl], l1s = ml[256 + 128 + rowl];
        const float m = fmaxf(m0, m1);                  // finite: key 0 is visible to every row
        f0 = ex2_approx(m0 - m);
        f1 = ex2_approx(m1 - m);                        // 0 for a half that was masked throughout
        const float lt = l0s * f0 + l1s * f1;
        inv_l = 1.0f / lt;
        lse = (m + log2f(lt)) * LN2_G;
      } else {
        // ---------------- frozen head: generate P^ tiles (this group's 64 keys of each)
        const float* alpha_h = p.alpha + static_cast<size_t>(w.h) * p.Tp;
        const float* rho_h = p.rho + static_cast<size_t>(w.h) * p.Tp;
        const float z2 = (row < p.T) ? p.logZ[static_cast<size_t>(w.h) * p.Tp + row] * LOG2E_G : INFINITY;
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
            if (key < p.T) a2 = alpha_h[key] * LOG2E_G;
            a2raw[tid] = a2;
          }
          {
            const int d = d0 + tid;                    // one band entry per compute thread (255 used)
            if (tid < 255 && d >= 0 && d < p.T) r2 = rho_h[d] * LOG2E_G;
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
            // previous P^ tile consumed (both halves: a thread follows every phase of both barriers, so that
            // the parity it waits for in the epilogue can never be one phase pair behind)
            if (!mbar_wait_warp(pv_done, npv & 1, wc, F_PV_DONE)) ok = false;
            if (!mbar_wait_warp(pv_done + 1, npv & 1, wc, F_PV_DONE)) ok = false;
            ++npv;
            tc_fence_after();
          }
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            const int k0c = 64 * g + 32 * cc;          // first key column of this chunk
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
            tmem_st16(t_s + 16 * cc, pk);
          }
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(p_full + g);
        }
        if (leave) break;
      }
      // ---------------- epilogue: wait for the last P V of both groups, merge, scale, store 32 columns each
      {
        const uint32_t par = npv & 1;
        if (!mbar_wait_warp(pv_done, par, wc, F_PV_DONE)) ok = false;
        if (!mbar_wait_warp(pv_done + 1, par, wc, F_PV_DONE)) ok = false;
        ++npv;
      }
      tc_fence_after();
      if (q4 == 0) TRF(trr, 17);
      if constexpr (OF32) {
        // fp32 output: every thread writes its 32 columns of its row straight to global memory
        const float s0 = f0 * inv_l, s1 = f1 * inv_l;
        float* orow = static_cast<float*>(p.O) + w.b * p.o_strides[0] + w.h * p.o_strides[1] +
                      static_cast<int64_t>(row) * p.o_strides[2] + 32 * g;
#pragma unroll
        for (int hc = 0; hc < 2; ++hc) {
          uint32_t ra[16], rb2[16];
          tmem_ld16(tmem + lane_base + C::COL_O + 32 * g + 16 * hc, ra);
          if (use1) tmem_ld16(tmem + lane_base + C::COL_O + 64 + 32 * g + 16 * hc, rb2);
          tmem_wait_ld();
          if (hc == 1) {
            tc_fence_before();
            warp_arrive(o_free);                          // the accumulators may be overwritten
          }
          if (row < p.T && ok) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float v[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                v[e] = __uint_as_float(ra[4 * q + e]) * s0;
                if (use1) v[e] = fmaf(__uint_as_float(rb2[4 * q + e]), s1, v[e]);
              }
              *reinterpret_cast<float4*>(orow + 16 * hc + 4 * q) = make_float4(v[0], v[1], v[2], v[3]);
            }
          }
        }
      } else {
        // The O tile goes through a swizzled staging tile and leaves by one TMA store: a row per thread written
        // straight to global memory touches 32 lines per store instruction and kept the load/store unit busy for
        // ~1800 clk per item.  The staging tile is free once the previous item's store has read it, which the
        // agreement barrier at the top of the item has made known to all compute warps.
        {
          const int rl = row - w.blk * BLK;                 // row within the tile (reversed in the tensor-core form)
          const uint32_t strow = smem_u32(smem + C::OFF_OST) + static_cast<uint32_t>(rl) * 128;
          const float s0 = f0 * inv_l, s1 = f1 * inv_l;
  #pragma unroll
          for (int hc = 0; hc < 2; ++hc) {
            uint32_t ra[16], rb2[16];
            tmem_ld16(tmem + lane_base + C::COL_O + 32 * g + 16 * hc, ra);
            if (use1) tmem_ld16(tmem + lane_base + C::COL_O + 64 + 32 * g + 16 * hc, rb2);
            tmem_wait_ld();
            if (hc == 1) {
              tc_fence_before();
              warp_arrive(o_free);                          // the accumulators may be overwritten
            }
  #pragma unroll
            for (int q = 0; q < 2; ++q) {
              float v[8];
  #pragma unroll
              for (int e = 0; e < 8; ++e) {
                v[e] = __uint_as_float(ra[8 * q + e]) * s0;
                if (use1) v[e] = fmaf(__uint_as_float(rb2[8 * q + e]), s1, v[e]);
              }
              const uint32_t chunk = static_cast<uint32_t>((4 * g + 2 * hc + q) ^ (rl & 7));
              st_shared_v4w(strow + chunk * 16, pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                            pack_bf16x2(v[6], v[7]));
            }
          }
        }
        fence_proxy_async_smem();
        const bool all_ok = !named_bar_or(8, 256, !ok);
        if (tid == 0 && all_ok) {
          tma_store_4d(&mo, smem + C::OFF_OST, 0, w.blk * BLK, w.h, w.b);
          bulk_commit_group();
        }
      }
      if (p.LSE != nullptr && g == 0 && row < p.T && ok)
        p.LSE[(static_cast<size_t>(w.b) * p.H + w.h) * p.T + row] = lse;
      if (q4 == 0) TRF(trr, 18);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (tid == 0) bulk_wait_group0();               // the last O tile has left the staging tile
  __syncwarp();
  if (*abort_flag) {
    // A wait gave up: let copies and MMAs that are still in flight land before the CTA's
    // shared memory and TMEM are released.
    for (int i = 0; i < 64; ++i) __nanosleep(20000);
  }
  tc_fence_before();
  __syncthreads();
  SAF_SPAN(fwd64, 1);
  if (warp == 9) tmem_dealloc(tmem, C::TMEM_COLS);
  if (tid == 0) {
    // this CTA claims nothing more; the last CTA to get here rewinds the queue for the next launch
    __threadfence();
    if (atomicAdd(p.queue + 1, 1) == static_cast<int>(gridDim.x) - 1) {
      p.queue[0] = 0;
      p.queue[1] = 0;
      __threadfence();
    }
  }
}

int fwd64_smem_bytes() { return Fwd64Cfg::SMEM; }

cudaError_t launch_fwd64(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mvt,
                         const CUtensorMap& mo, const FwdParams& p, int grid, cudaStream_t st) {
  cudaError_t e;
  if (p.o_f32) {
    e = cudaFuncSetAttribute(saf_fwd64_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fwd64Cfg::SMEM);
    if (e != cudaSuccess) return e;
    return launch_pdl(PDL_FWD, saf_fwd64_kernel<true>, dim3(grid), dim3(Fwd64Cfg::NTHREADS), Fwd64Cfg::SMEM, st, mq, mk, mv,
                      mvt, mo, p);
  }
  e = cudaFuncSetAttribute(saf_fwd64_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Fwd64Cfg::SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(PDL_FWD, saf_fwd64_kernel<false>, dim3(grid), dim3(Fwd64Cfg::NTHREADS), Fwd64Cfg::SMEM, st, mq, mk, mv,
                    mvt, mo, p);
}

}  // namespace saf
