// Host side of the C ABI: argument validation, context (workspace, cached work lists, device status
// word), TMA tensor maps, the head scheduler and the launches.
#include <algorithm>
#include <array>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <queue>
#include <vector>

#include "../../include/saf.h"
#include "saf_internal.h"

using namespace saf;

#define SAF_VERSION_NUM 100

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct WorklistEntry {
  int B, H, T, backward, grid, wide;
  std::vector<uint8_t> mask;
  std::vector<WorkItem> items_host;       // kept alive: the upload is asynchronous on the caller's stream
  std::vector<int> offsets_host;
  WorkItem* items_dev = nullptr;
  int* offsets_dev = nullptr;
  WorkItem* order_dev = nullptr;          // the same items in queue order (kernels that take work dynamically)
  std::vector<WorkItem> order_host;
  int n_items = 0;
};

struct DevBuf {
  void* ptr = nullptr;
  size_t bytes = 0;
};

// Which (alpha, rho, logZ) the context's tensor-core pattern tables were built from.
struct PatternCache {
  bool valid = false;
  const float* alpha = nullptr;
  const float* rho = nullptr;
  const float* logZ = nullptr;
  int H = 0, Tp = 0, Hf = 0;
  std::vector<uint8_t> mask;
};

struct TimedLaunch {
  int which;
  cudaEvent_t beg, end;
};

}  // namespace

struct saf_ctx {
  int device = 0;
  int num_sms = 0;
  int* status_dev = nullptr;
  int* queue_dev = nullptr;                // work-queue counters: {next item, CTAs done} per kernel that uses one
  cudaStream_t last_stream = nullptr;
  EncodeTiledFn encode = nullptr;
  unsigned long long wait_limit_ns = 2000000000ull;
  // Scheduler cost model, in percent of an ordinary tile: a frozen tile (forward, backward) and the fixed cost of a
  // work item (prologue, epilogue, pipeline refill).  0 = the measured default of the kernel family
  // (sched_defaults); set by the SAF_FROZEN_WEIGHT_* / SAF_ITEM_OVERHEAD_* environment variables.
  int frozen_weight_pct = 0;
  int frozen_weight_bwd_pct = 0;
  int item_overhead_pct = 0;
  int item_overhead_bwd_pct = 0;
  // Forward grid = two CTAs per SM: the CTA that arrives second on an SM (block index >= grid / 2) runs slower
  // than the first (measured 13 % at head dimension 64, 2 % on the 128-wide kernel; best settings 20 and 6) and gets that much less
  // work.  -1 = the measured default; SAF_SECOND_WAVE_PCT overrides.
  int second_wave_pct = -1;
  int call_counter = 0;                    // ids of the calls that stage fp16 operands (overflow marks)
  std::vector<WorklistEntry> worklists;
  DevBuf mask_buf, logz_buf, delta_buf, dqacc_buf, dkacc_buf, dvacc_buf, qslot_buf;
  // what mask_buf / qslot_buf currently hold (host copies) and the stream that wrote them
  std::vector<uint8_t> mask_host, mask_staging, qslot_mask_host;
  std::vector<int> qslot_host;
  cudaStream_t mask_stream = nullptr, qslot_stream = nullptr;
  // tensor-core form of frozen heads: tables built by saf_pattern_prepare, scaled V / dO per call
  PatternCache pat;
  bool tensor_pattern = true;              // SAF_DISABLE_TENSOR_PATTERN=1 turns the form off
  bool selftest_drop_load = false;         // SAF_SELFTEST_DROP_LOAD=1: see FwdParams::selftest_drop_load
  DevBuf pat_consts, pat_ok, pat_avec, pat_wvec, pat_bandf, pat_bandb, pat_hord, pat_hlist, pat_snap, vt_buf, dot_buf, ok_fwd, ok_bwd, pg_hlist, pg_delta, pg_items, pg_offsets, fit_buf, calib_tmp;
  std::vector<int> pg_hlist_host, pg_offsets_host;   // host copies of the pattern-gradient tables (upload sources)
  std::vector<PgItem> pg_items_host;
  std::array<int, 5> pg_key = {0, 0, 0, 0, 0};      // (B, frozen heads, T, D, grid) the work list was built for
  bool profiling = false;
  std::vector<TimedLaunch> timed;          // event pairs recorded since the last query
  std::vector<cudaEvent_t> event_pool;
  // staging for the host-buffer entry point
  DevBuf hq, hk, hv, hdo, ho, hlse, hdq, hdk, hdv, halpha, hrho, hlogz;
  // host-buffer step: compute stream, copy stream and the events that order them
  static constexpr int HS_CHUNKS = 8;
  cudaStream_t hs_main = nullptr, hs_copy = nullptr, hs_outs = nullptr;
  cudaEvent_t hs_in[HS_CHUNKS] = {}, hs_do[HS_CHUNKS] = {}, hs_fwd[HS_CHUNKS] = {}, hs_cmp[HS_CHUNKS] = {};
};

namespace {

int ensure(DevBuf& b, size_t bytes) {
  if (b.bytes >= bytes && b.ptr) return SAF_OK;
  if (b.ptr) cudaFree(b.ptr);
  b.ptr = nullptr;
  b.bytes = 0;
  if (cudaMalloc(&b.ptr, bytes) != cudaSuccess) {
    cudaGetLastError();
    return SAF_ERR_NOMEM;
  }
  b.bytes = bytes;
  return SAF_OK;
}
void release(DevBuf& b) {
  if (b.ptr) cudaFree(b.ptr);
  b.ptr = nullptr;
  b.bytes = 0;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// [B][H][T][D] bf16 tensor with element strides (batch, head, seq); box = 64 features x 128 rows,
// 128-byte swizzle; rows beyond T read as zero.
int make_map(saf_ctx* ctx, CUtensorMap* out, const void* base, const saf_problem* p, const int64_t* strides,
             CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, int heads = 0, int box_rows = BLK,
             int box_batch = 1) {
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(p->D), static_cast<cuuint64_t>(p->T),
                        static_cast<cuuint64_t>(heads > 0 ? heads : p->H), static_cast<cuuint64_t>(p->B)};
  cuuint64_t gs[3] = {static_cast<cuuint64_t>(strides[2]) * 2, static_cast<cuuint64_t>(strides[1]) * 2,
                      static_cast<cuuint64_t>(strides[0]) * 2};
  // (box_batch > 1: one copy brings the same tile of several consecutive batch entries, laid out one after the other)
  cuuint32_t box[4] = {64, static_cast<cuuint32_t>(box_rows), 1, static_cast<cuuint32_t>(box_batch)};
  cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = ctx->encode(out, dtype, 4, const_cast<void*>(base), dims, gs, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SAF_OK : SAF_ERR_CUDA;
}

// The tables in the context describe exactly these vectors and this mask.
bool pattern_matches(const saf_ctx* ctx, const saf_problem* p, const uint8_t* mask, const float* alpha,
                     const float* rho, const float* logZ) {
  const PatternCache& c = ctx->pat;
  return ctx->tensor_pattern && c.valid && c.alpha == alpha && c.rho == rho && c.logZ == logZ && c.H == p->H &&
         c.Tp == p->Tp && std::memcmp(c.mask.data(), mask, p->H) == 0;
}

PatternCheck pattern_check(const saf_ctx* ctx, const float* alpha, const float* rho, const float* logZ) {
  return PatternCheck{alpha, rho, logZ, static_cast<const uint32_t*>(ctx->pat_snap.ptr),
                      static_cast<size_t>(ctx->pat.H) * ctx->pat.Tp};
}

// map of a contiguous [B][Hn][T][D] fp16 workspace
int make_map_contig(saf_ctx* ctx, CUtensorMap* out, const void* base, const saf_problem* p, int Hn,
                    int box_rows = BLK) {
  saf_problem q = *p;
  q.H = Hn;
  const int64_t st[3] = {static_cast<int64_t>(Hn) * p->T * p->D, static_cast<int64_t>(p->T) * p->D, p->D};
  return make_map(ctx, out, base, &q, st, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 0, box_rows);
}

int check_strides(const int64_t* s, int D) {
  for (int i = 0; i < 3; ++i)
    if (s[i] <= 0 || (s[i] % 8) != 0) return SAF_ERR_INVALID_ARG;
  if (s[2] < D) return SAF_ERR_INVALID_ARG;
  return SAF_OK;
}

int validate(const saf_problem* p, const uint8_t* mask, int* n_frozen) {
  if (!p || !mask) return SAF_ERR_INVALID_ARG;
  if (p->B < 1 || p->H < 1 || p->T < 1 || p->Tp < 1) return SAF_ERR_INVALID_ARG;
  if (p->T > p->Tp) return SAF_ERR_INVALID_ARG;
  if (p->D != 64 && p->D != 96 && p->D != 128) return SAF_ERR_UNSUPPORTED;   // 96 runs padded on the 128-wide kernels
  if (p->grad_dtype != SAF_F32 && p->grad_dtype != SAF_BF16) return SAF_ERR_UNSUPPORTED;
  if (p->o_dtype != SAF_F32 && p->o_dtype != SAF_BF16) return SAF_ERR_UNSUPPORTED;
  if (p->kv_group < 0 || (p->kv_group > 1 && p->H % p->kv_group != 0)) return SAF_ERR_INVALID_ARG;
  if (p->packed_qk && p->kv_group > 1) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  for (int h = 0; h < p->H; ++h) nf += mask[h] ? 1 : 0;
  *n_frozen = nf;
  return SAF_OK;
}

inline int kv_group_of(const saf_problem* p) { return p->kv_group > 1 ? p->kv_group : 1; }

// Packed Q/K layout: device table head -> slot among the ordinary heads (-1 for frozen heads).  The table is
// uploaded only when the mask differs from the one it was built from (a layer's mask is static), from a vector
// owned by the context, so the caller's array is read before the call returns whatever memory it lives in.
int upload_qslot(saf_ctx* ctx, const uint8_t* mask, int H, cudaStream_t st, const int** out) {
  const void* before = ctx->qslot_buf.ptr;
  int rc = ensure(ctx->qslot_buf, static_cast<size_t>(std::max(H, 64)) * sizeof(int));
  if (rc) return rc;
  if (ctx->qslot_buf.ptr != before) ctx->qslot_mask_host.clear();
  *out = static_cast<const int*>(ctx->qslot_buf.ptr);
  if (ctx->qslot_mask_host.size() == static_cast<size_t>(H) && ctx->qslot_stream == st &&
      std::memcmp(ctx->qslot_mask_host.data(), mask, H) == 0)
    return SAF_OK;
  ctx->qslot_host.resize(H);
  int n = 0;
  for (int h = 0; h < H; ++h) ctx->qslot_host[h] = mask[h] ? -1 : n++;
  ctx->qslot_mask_host.clear();
  if (cudaMemcpyAsync(ctx->qslot_buf.ptr, ctx->qslot_host.data(), static_cast<size_t>(H) * sizeof(int),
                      cudaMemcpyHostToDevice, st) != cudaSuccess)
    return SAF_ERR_CUDA;
  ctx->qslot_mask_host.assign(mask, mask + H);
  ctx->qslot_stream = st;
  return SAF_OK;
}

// Device copy of the frozen-head mask, uploaded only when it changes (see upload_qslot).
int upload_mask(saf_ctx* ctx, const uint8_t* mask, int H, cudaStream_t st) {
  const void* before = ctx->mask_buf.ptr;
  int rc = ensure(ctx->mask_buf, std::max(H, 256));
  if (rc) return rc;
  if (ctx->mask_buf.ptr != before) ctx->mask_host.clear();
  if (ctx->mask_host.size() == static_cast<size_t>(H) && ctx->mask_stream == st &&
      std::memcmp(ctx->mask_host.data(), mask, H) == 0)
    return SAF_OK;
  ctx->mask_staging.assign(mask, mask + H);
  ctx->mask_host.clear();
  if (cudaMemcpyAsync(ctx->mask_buf.ptr, ctx->mask_staging.data(), H, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return SAF_ERR_CUDA;
  ctx->mask_host.assign(mask, mask + H);
  ctx->mask_stream = st;
  return SAF_OK;
}

// Work lists of the persistent kernels.  Items of one (batch, head) unit are kept close in time, so that
// what they share stays in L2 while it is needed: in the backward every key block of a unit adds into
// the unit's dQ rows and re-reads its Q/dO tiles; in the forward every query block re-reads its K/V
// tiles.  Units are walked in order, the blocks of a unit alternately from the expensive and the cheap
// end, and each item goes to the CTA that becomes free first (list scheduling, which is what a dynamic
// queue would do); only the last items are ordered longest-first so that the tail stays short.
void build_worklist_host(int B, int H, int T, const uint8_t* mask, int backward, int n_ctas, int frozen_pct,
                         int overhead_pct, int overhead_frozen_pct, int second_wave_pct, std::vector<WorkItem>& items,
                         std::vector<int>& offsets, std::vector<WorkItem>* order = nullptr) {
  const int nblk = (T + BLK - 1) / BLK;
  struct Cand { WorkItem w; long long cost; };
  std::vector<Cand> cand;
  cand.reserve(static_cast<size_t>(B) * H * nblk);
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h) {
      const int kind = mask[h] ? KIND_FROZEN : KIND_ORDINARY;
      for (int z = 0; z < nblk; ++z) {
        // zig-zag over the blocks: most expensive, cheapest, second most expensive, ...
        const int r = (z & 1) ? (nblk - 1 - z / 2) : (z / 2);        // rank by cost, 0 = most expensive
        const int k = backward ? r : (nblk - 1 - r);
        const long long tiles = backward ? (nblk - k) : (k + 1);
        // + fixed per-item overhead
        const long long cost = tiles * (kind == KIND_FROZEN ? frozen_pct : 100) +
                               (kind == KIND_FROZEN ? overhead_frozen_pct : overhead_pct);
        cand.push_back({{b, h, k, kind}, cost});
      }
    }
  // the tail (about two items per CTA) longest-first
  const size_t tail = std::min(cand.size(), static_cast<size_t>(2) * n_ctas);
  std::stable_sort(cand.end() - tail, cand.end(), [](const Cand& a, const Cand& b) { return a.cost > b.cost; });
  if (order) {
    // the sequence itself is the work queue of the kernels that claim items at run time
    order->clear();
    for (const Cand& c : cand) order->push_back(c.w);
  }
  typedef std::pair<long long, int> Load;   // (load, cta)
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < n_ctas; ++c) heap.push({0, c});
  std::vector<std::vector<WorkItem>> per(n_ctas);
  for (const Cand& c : cand) {
    Load l = heap.top();
    heap.pop();
    per[l.second].push_back(c.w);
    // CTAs of the second half of the grid (the second CTA of each SM when the grid is two per SM) run slower
    const long long scaled = l.second >= n_ctas / 2 ? c.cost * (100 + second_wave_pct) : c.cost * 100;
    heap.push({l.first + scaled, l.second});
  }
  items.clear();
  offsets.assign(n_ctas + 1, 0);
  for (int c = 0; c < n_ctas; ++c) {
    offsets[c] = static_cast<int>(items.size());
    items.insert(items.end(), per[c].begin(), per[c].end());
  }
  offsets[n_ctas] = static_cast<int>(items.size());
}

// Measured cost-model defaults: `wide` = the 128-wide kernels (head dimension 96 or 128), else the 64-wide ones.
void sched_defaults(int wide, int backward, int* frozen_pct, int* overhead_pct, int* overhead_frozen_pct) {
  if (backward) {
    *frozen_pct = 20;
    *overhead_pct = wide ? 200 : 150;   // (a trace puts the item boundary of the 64-wide backward at ~1.6 tiles)
    *overhead_frozen_pct = wide ? 200 : 100;   // (a frozen item ends with half the epilogue: dV only)
  } else {
    *frozen_pct = wide ? 50 : 30;
    *overhead_pct = *overhead_frozen_pct = 150;   // (re-fitted: the 128-wide forward measured 1-1.6 % slower with 300)
  }
}

int get_worklist(saf_ctx* ctx, int B, int H, int T, const uint8_t* mask, int backward, int grid, int wide,
                 cudaStream_t st, const WorklistEntry** out) {
  for (const WorklistEntry& e : ctx->worklists)
    if (e.B == B && e.H == H && e.T == T && e.backward == backward && e.grid == grid && e.wide == wide &&
        std::memcmp(e.mask.data(), mask, H) == 0) {
      *out = &e;
      return SAF_OK;
    }
  if (ctx->worklists.size() >= 32) {   // bounded cache: drop the oldest
    cudaStreamSynchronize(st);
    cudaFree(ctx->worklists.front().items_dev);
    cudaFree(ctx->worklists.front().offsets_dev);
    cudaFree(ctx->worklists.front().order_dev);
    ctx->worklists.erase(ctx->worklists.begin());
  }
  std::vector<WorkItem> items;
  std::vector<int> offsets;
  int frozen_pct, overhead_pct, overhead_frozen_pct;
  sched_defaults(wide, backward, &frozen_pct, &overhead_pct, &overhead_frozen_pct);
  const int fw = backward ? ctx->frozen_weight_bwd_pct : ctx->frozen_weight_pct;
  const int ov = backward ? ctx->item_overhead_bwd_pct : ctx->item_overhead_pct;
  if (fw > 0) frozen_pct = fw;
  if (ov > 0) overhead_pct = overhead_frozen_pct = ov;   // (the override sets both kinds)
  const int second_wave = backward ? 0 : (ctx->second_wave_pct >= 0 ? ctx->second_wave_pct : (wide ? 6 : 20));
  WorklistEntry e;
  build_worklist_host(B, H, T, mask, backward, grid, frozen_pct, overhead_pct, overhead_frozen_pct, second_wave, items,
                      offsets, &e.order_host);
  e.B = B; e.H = H; e.T = T; e.backward = backward; e.grid = grid; e.wide = wide;
  e.mask.assign(mask, mask + H);
  e.n_items = static_cast<int>(items.size());
  if (cudaMalloc(&e.items_dev, items.size() * sizeof(WorkItem)) != cudaSuccess) return SAF_ERR_NOMEM;
  if (cudaMalloc(&e.offsets_dev, offsets.size() * sizeof(int)) != cudaSuccess) {
    cudaFree(e.items_dev);
    return SAF_ERR_NOMEM;
  }
  if (cudaMalloc(&e.order_dev, e.order_host.size() * sizeof(WorkItem)) != cudaSuccess) {
    cudaFree(e.items_dev);
    cudaFree(e.offsets_dev);
    return SAF_ERR_NOMEM;
  }
  // uploaded on the stream the kernel will run on (a non-blocking stream does not order with the legacy stream);
  // the source vectors live as long as the entry
  e.items_host = std::move(items);
  e.offsets_host = std::move(offsets);
  if (cudaMemcpyAsync(e.items_dev, e.items_host.data(), e.items_host.size() * sizeof(WorkItem), cudaMemcpyHostToDevice,
                      st) != cudaSuccess ||
      cudaMemcpyAsync(e.offsets_dev, e.offsets_host.data(), e.offsets_host.size() * sizeof(int),
                      cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(e.order_dev, e.order_host.data(), e.order_host.size() * sizeof(WorkItem), cudaMemcpyHostToDevice,
                      st) != cudaSuccess) {
    cudaFree(e.order_dev);
    cudaFree(e.items_dev);
    cudaFree(e.offsets_dev);
    return SAF_ERR_CUDA;
  }
  ctx->worklists.push_back(std::move(e));
  *out = &ctx->worklists.back();
  return SAF_OK;
}

// Kernel timing (opt-in): an event pair on the launching stream around one kernel.
cudaEvent_t take_event(saf_ctx* ctx) {
  if (!ctx->event_pool.empty()) {
    cudaEvent_t e = ctx->event_pool.back();
    ctx->event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
struct ScopedTimer {
  saf_ctx* ctx;
  cudaStream_t st;
  TimedLaunch t{};
  bool on;
  ScopedTimer(saf_ctx* c, int which, cudaStream_t s) : ctx(c), st(s), on(c->profiling && c->timed.size() < 65536) {
    if (!on) return;
    t.which = which;
    t.beg = take_event(ctx);
    t.end = take_event(ctx);
    cudaEventRecord(t.beg, st);
  }
  ~ScopedTimer() {
    if (!on) return;
    cudaEventRecord(t.end, st);
    ctx->timed.push_back(t);
  }
};

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

}  // namespace

extern "C" {

int saf_version(void) { return SAF_VERSION_NUM; }

const char* saf_status_string(int code) {
  switch (code) {
    case SAF_OK: return "ok";
    case SAF_ERR_INVALID_ARG: return "invalid argument";
    case SAF_ERR_UNSUPPORTED: return "unsupported head dimension or dtype";
    case SAF_ERR_CUDA: return "CUDA call failed";
    case SAF_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel gave up";
    case SAF_ERR_ARCH: return "device is not sm_100-class";
    case SAF_ERR_NOMEM: return "out of device memory";
    default: return "unknown status";
  }
}

int saf_create(saf_ctx** out, int device) {
  if (!out) return SAF_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    cudaGetLastError();
    return SAF_ERR_CUDA;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SAF_ERR_CUDA;
  if (prop.major != 10) return SAF_ERR_ARCH;
  DeviceGuard g(device);
  if (!g.ok) return SAF_ERR_CUDA;
  saf_ctx* ctx = new saf_ctx();
  ctx->device = device;
  ctx->num_sms = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult q;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) {
    delete ctx;
    return SAF_ERR_CUDA;
  }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&ctx->queue_dev, 8 * sizeof(int)) != cudaSuccess ||
      cudaMemset(ctx->queue_dev, 0, 8 * sizeof(int)) != cudaSuccess) {
    delete ctx;
    return SAF_ERR_NOMEM;
  }
  if (cudaMalloc(&ctx->status_dev, sizeof(int)) != cudaSuccess || cudaMemset(ctx->status_dev, 0, sizeof(int)) != cudaSuccess) {
    delete ctx;
    return SAF_ERR_NOMEM;
  }
  if (const char* e = std::getenv("SAF_WAIT_LIMIT_MS")) {
    long v = std::atol(e);
    if (v > 0) ctx->wait_limit_ns = static_cast<unsigned long long>(v) * 1000000ull;
  }
  if (const char* e = std::getenv("SAF_DISABLE_TENSOR_PATTERN")) ctx->tensor_pattern = std::atoi(e) == 0;
  if (const char* e = std::getenv("SAF_SELFTEST_DROP_LOAD")) ctx->selftest_drop_load = std::atoi(e) == 1;
  if (const char* e = std::getenv("SAF_FROZEN_WEIGHT_PCT")) {
    long v = std::atol(e);
    if (v > 0 && v <= 400) ctx->frozen_weight_pct = static_cast<int>(v);
  }
  if (const char* e = std::getenv("SAF_FROZEN_WEIGHT_BWD_PCT")) {
    long v = std::atol(e);
    if (v > 0 && v <= 400) ctx->frozen_weight_bwd_pct = static_cast<int>(v);
  }
  if (const char* e = std::getenv("SAF_SECOND_WAVE_PCT")) {
    long v = std::atol(e);
    if (v >= 0 && v <= 100) ctx->second_wave_pct = static_cast<int>(v);
  }
  if (const char* e = std::getenv("SAF_ITEM_OVERHEAD_PCT")) {
    long v = std::atol(e);
    if (v > 0 && v <= 2000) ctx->item_overhead_pct = static_cast<int>(v);
  }
  if (const char* e = std::getenv("SAF_ITEM_OVERHEAD_BWD_PCT")) {
    long v = std::atol(e);
    if (v > 0 && v <= 2000) ctx->item_overhead_bwd_pct = static_cast<int>(v);
  }
  *out = ctx;
  return SAF_OK;
}

int saf_destroy(saf_ctx* ctx) {
  if (!ctx) return SAF_OK;
  DeviceGuard g(ctx->device);
  cudaDeviceSynchronize();
  for (WorklistEntry& e : ctx->worklists) {
    cudaFree(e.items_dev);
    cudaFree(e.offsets_dev);
    cudaFree(e.order_dev);
  }
  DevBuf* pbufs[] = {&ctx->pat_consts, &ctx->pat_ok, &ctx->pat_avec, &ctx->pat_wvec, &ctx->pat_bandf, &ctx->pat_bandb,
                     &ctx->pat_hord, &ctx->pat_hlist, &ctx->pat_snap, &ctx->vt_buf, &ctx->dot_buf, &ctx->ok_fwd, &ctx->ok_bwd, &ctx->pg_hlist, &ctx->pg_delta, &ctx->pg_items, &ctx->pg_offsets, &ctx->fit_buf, &ctx->calib_tmp};
  for (DevBuf* b : pbufs) release(*b);
  DevBuf* bufs[] = {&ctx->mask_buf, &ctx->logz_buf, &ctx->delta_buf, &ctx->dqacc_buf, &ctx->dkacc_buf, &ctx->dvacc_buf, &ctx->qslot_buf, &ctx->hq, &ctx->hk, &ctx->hv,
                    &ctx->hdo, &ctx->ho, &ctx->hlse, &ctx->hdq, &ctx->hdk, &ctx->hdv, &ctx->halpha, &ctx->hrho,
                    &ctx->hlogz};
  for (DevBuf* b : bufs) release(*b);
  if (ctx->status_dev) cudaFree(ctx->status_dev);
  if (ctx->queue_dev) cudaFree(ctx->queue_dev);
  if (ctx->hs_main) cudaStreamDestroy(ctx->hs_main);
  if (ctx->hs_copy) cudaStreamDestroy(ctx->hs_copy);
  if (ctx->hs_outs) cudaStreamDestroy(ctx->hs_outs);
  for (int c = 0; c < saf_ctx::HS_CHUNKS; ++c)
    for (cudaEvent_t e : {ctx->hs_in[c], ctx->hs_do[c], ctx->hs_fwd[c], ctx->hs_cmp[c]})
    if (e) cudaEventDestroy(e);
  for (TimedLaunch& t : ctx->timed) {
    cudaEventDestroy(t.beg);
    cudaEventDestroy(t.end);
  }
  for (cudaEvent_t e : ctx->event_pool) cudaEventDestroy(e);
  delete ctx;
  return SAF_OK;
}

int saf_pattern_prepare(saf_ctx* ctx, int32_t H, int32_t Tp, const uint8_t* frozen_mask_host, const float* alpha_dev,
                        const float* rho_dev, float* logZ_dev_out, void* stream) {
  if (!ctx || !frozen_mask_host || H < 1 || Tp < 1) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  for (int h = 0; h < H; ++h) nf += frozen_mask_host[h] ? 1 : 0;
  if (nf == 0) return SAF_OK;
  if (!alpha_dev || !rho_dev || !logZ_dev_out) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = upload_mask(ctx, frozen_mask_host, H, st);
  if (rc) return rc;
  ctx->last_stream = st;
  {
    ScopedTimer timer(ctx, SAF_KERNEL_LOGZ, st);
    if (launch_logz(alpha_dev, rho_dev, logZ_dev_out, static_cast<const uint8_t*>(ctx->mask_buf.ptr), H, Tp, st) !=
        cudaSuccess)
      return SAF_ERR_CUDA;
  }
  ctx->pat.valid = false;
  if (!ctx->tensor_pattern) return SAF_OK;
  // tables of the tensor-core form (Hankel bands of exp(rho), key scale a, row scale w, per-head flag)
  const int nblkp = (Tp + 127) / 128;
  const size_t vecb = static_cast<size_t>(H) * Tp * sizeof(float);
  const size_t bandb = static_cast<size_t>(H) * nblkp * 4096;
  if ((rc = ensure(ctx->pat_consts, static_cast<size_t>(H) * 2 * sizeof(float))) ||
      (rc = ensure(ctx->pat_ok, static_cast<size_t>(H) * sizeof(int))) || (rc = ensure(ctx->pat_avec, vecb)) ||
      (rc = ensure(ctx->pat_wvec, vecb)) || (rc = ensure(ctx->pat_bandf, bandb)) ||
      (rc = ensure(ctx->pat_bandb, bandb)) || (rc = ensure(ctx->pat_hord, static_cast<size_t>(H) * sizeof(int))) ||
      (rc = ensure(ctx->pat_hlist, static_cast<size_t>(H) * sizeof(int))) || (rc = ensure(ctx->pat_snap, 3 * vecb)) ||
      (rc = ensure(ctx->ok_fwd, static_cast<size_t>(H) * sizeof(int))) ||
      (rc = ensure(ctx->ok_bwd, static_cast<size_t>(H) * sizeof(int))))
    return rc;
  // per-head overflow marks of the forward / backward staging kernels (a mark is the id of the call that set it)
  if (cudaMemsetAsync(ctx->ok_fwd.ptr, 0, static_cast<size_t>(H) * sizeof(int), st) != cudaSuccess ||
      cudaMemsetAsync(ctx->ok_bwd.ptr, 0, static_cast<size_t>(H) * sizeof(int), st) != cudaSuccess)
    return SAF_ERR_CUDA;
  std::vector<int> hord(H, -1), hlist(H, 0);
  int ord = 0;
  for (int h = 0; h < H; ++h)
    if (frozen_mask_host[h]) {
      hlist[ord] = h;
      hord[h] = ord++;
    }
  if (cudaMemcpyAsync(ctx->pat_hord.ptr, hord.data(), static_cast<size_t>(H) * sizeof(int), cudaMemcpyHostToDevice, st) !=
          cudaSuccess ||
      cudaMemcpyAsync(ctx->pat_hlist.ptr, hlist.data(), static_cast<size_t>(H) * sizeof(int), cudaMemcpyHostToDevice,
                      st) != cudaSuccess)
    return SAF_ERR_CUDA;
  {
    ScopedTimer timer(ctx, SAF_KERNEL_LOGZ, st);
    if (launch_pattern_tables(alpha_dev, rho_dev, logZ_dev_out, static_cast<const uint8_t*>(ctx->mask_buf.ptr), H, Tp,
                              static_cast<float*>(ctx->pat_consts.ptr), static_cast<int*>(ctx->pat_ok.ptr),
                              static_cast<float*>(ctx->pat_avec.ptr), static_cast<float*>(ctx->pat_wvec.ptr),
                              ctx->pat_bandf.ptr, ctx->pat_bandb.ptr, st) != cudaSuccess)
      return SAF_ERR_CUDA;
  }
  // Snapshot of the three vectors: the tables are matched to a later call by these pointers, and the staging kernels
  // compare the bits, so a head whose vectors were rewritten in place since (by the caller, by the fitter, by the
  // allocation-free normaliser entry point) falls back to the general form instead of using stale tables.
  {
    uint8_t* snap = static_cast<uint8_t*>(ctx->pat_snap.ptr);
    if (cudaMemcpyAsync(snap, alpha_dev, vecb, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(snap + vecb, rho_dev, vecb, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(snap + 2 * vecb, logZ_dev_out, vecb, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return SAF_ERR_CUDA;
  }
  ctx->pat.valid = true;
  ctx->pat.alpha = alpha_dev;
  ctx->pat.rho = rho_dev;
  ctx->pat.logZ = logZ_dev_out;
  ctx->pat.H = H;
  ctx->pat.Tp = Tp;
  ctx->pat.Hf = nf;
  ctx->pat.mask.assign(frozen_mask_host, frozen_mask_host + H);
  return SAF_OK;
}

int saf_hybrid_attn_fwd(saf_ctx* ctx, const saf_problem* p, const void* Q, const void* K, const void* V,
                        const uint8_t* frozen_mask_host, const float* alpha, const float* rho, const float* logZ,
                        void* O, float* LSE, void* stream) {
  if (!ctx) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  int rc = validate(p, frozen_mask_host, &nf);
  if (rc) return rc;
  const int no = p->H - nf;
  if (!V || !O) return SAF_ERR_INVALID_ARG;
  if (no > 0 && (!Q || !K || !LSE)) return SAF_ERR_INVALID_ARG;
  if (nf > 0 && (!alpha || !rho)) return SAF_ERR_INVALID_ARG;
  if (!aligned16(V) || !aligned16(O) || (no > 0 && (!aligned16(Q) || !aligned16(K)))) return SAF_ERR_INVALID_ARG;
  if (check_strides(p->v_strides, p->D) || check_strides(p->o_strides, p->D)) return SAF_ERR_INVALID_ARG;
  if (no > 0 && (check_strides(p->q_strides, p->D) || check_strides(p->k_strides, p->D))) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;

  if (nf > 0 && !logZ) {
    rc = ensure(ctx->logz_buf, static_cast<size_t>(p->H) * p->Tp * sizeof(float));
    if (rc) return rc;
    rc = saf_pattern_prepare(ctx, p->H, p->Tp, frozen_mask_host, alpha, rho, static_cast<float*>(ctx->logz_buf.ptr),
                             stream);
    if (rc) return rc;
    logZ = static_cast<const float*>(ctx->logz_buf.ptr);
  }
  const int nblk = (p->T + BLK - 1) / BLK;
  const long long n_items = static_cast<long long>(p->B) * p->H * nblk;
  const int grid = static_cast<int>(std::min<long long>(2LL * ctx->num_sms, n_items));
  const WorklistEntry* wl = nullptr;
  rc = get_worklist(ctx, p->B, p->H, p->T, frozen_mask_host, 0, grid, p->D != 64, st, &wl);
  if (rc) return rc;

  CUtensorMap mq, mk, mv;
  // frozen-only layers never touch Q/K: any valid map will do
  const int kvg = kv_group_of(p);
  rc = make_map(ctx, &mv, V, p, p->v_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->H / kvg);
  if (rc) return rc;
  if (no > 0) {
    rc = make_map(ctx, &mq, Q, p, p->q_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->packed_qk ? no : p->H);
    if (rc) return rc;
    rc = make_map(ctx, &mk, K, p, p->k_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->packed_qk ? no : p->H / kvg);
    if (rc) return rc;
  } else {
    mq = mv;
    mk = mv;
  }
  FwdParams fp;
  CUtensorMap mvt = mv;
  fp.band_f = nullptr; fp.wvec = nullptr; fp.fast_ok = nullptr; fp.hord = nullptr; fp.ovf = nullptr; fp.call_id = 0; fp.nblkp = (p->Tp + 127) / 128;
  if (nf > 0 && pattern_matches(ctx, p, frozen_mask_host, alpha, rho, logZ)) {
    // tensor-core form: V of the frozen heads scaled by a(j) once per call
    const size_t vtb = static_cast<size_t>(p->B) * nf * p->T * p->D * 2;
    rc = ensure(ctx->vt_buf, vtb);
    if (rc) return rc;
    // the scaling kernel marks a head whose values leave fp16's range with this call's id
    fp.call_id = ++ctx->call_counter;
    {
      ScopedTimer timer(ctx, SAF_KERNEL_SCALE, st);
      if (launch_scale_rows(V, p->v_strides, static_cast<const float*>(ctx->pat_avec.ptr), HK_A_SCALE, p->Tp,
                            static_cast<const int*>(ctx->pat_hlist.ptr), static_cast<const int*>(ctx->pat_ok.ptr),
                            static_cast<int*>(ctx->ok_fwd.ptr), fp.call_id, ctx->vt_buf.ptr, p->B, nf, p->T, p->D,
                            kvg, pattern_check(ctx, alpha, rho, logZ), st) != cudaSuccess)
        return SAF_ERR_CUDA;
    }
    rc = make_map_contig(ctx, &mvt, ctx->vt_buf.ptr, p, nf);
    if (rc) return rc;
    fp.band_f = ctx->pat_bandf.ptr;
    fp.wvec = static_cast<const float*>(ctx->pat_wvec.ptr);
    fp.fast_ok = static_cast<const int*>(ctx->pat_ok.ptr);
    fp.ovf = static_cast<const int*>(ctx->ok_fwd.ptr);
    fp.hord = static_cast<const int*>(ctx->pat_hord.ptr);
  }
  fp.B = p->B; fp.H = p->H; fp.T = p->T; fp.Tp = p->Tp;
  fp.kv_group = kvg;
  fp.d_real = p->D;
  fp.qslot = nullptr;
  if (p->packed_qk && no > 0 && (rc = upload_qslot(ctx, frozen_mask_host, p->H, st, &fp.qslot))) return rc;
  const float scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(p->D));
  fp.scale_log2 = scale * 1.4426950408889634f;
  fp.alpha = alpha; fp.rho = rho; fp.logZ = logZ;
  fp.O = O;
  fp.o_f32 = p->o_dtype == SAF_F32 ? 1 : 0;
  for (int i = 0; i < 3; ++i) fp.o_strides[i] = p->o_strides[i];
  fp.LSE = LSE;
  fp.items = wl->items_dev;
  fp.cta_offsets = wl->offsets_dev;
  fp.order = wl->order_dev;
  fp.n_items = wl->n_items;
  fp.queue = ctx->queue_dev;
  fp.status = ctx->status_dev;
  fp.wait_limit_ns = ctx->wait_limit_ns;
  fp.selftest_drop_load =
      (ctx->selftest_drop_load && grid <= 16 && ctx->wait_limit_ns <= 50000000ull && p->D == 64) ? 1 : 0;
  ScopedTimer timer(ctx, SAF_KERNEL_FWD, st);
  // head dimension 96 runs on the 128-wide kernel: TMA zero-fills features 96..127 of every operand tile
  // bf16 O leaves the D = 64 kernel as whole tiles by TMA stores (rows beyond T are clipped by the map); with fp32 O
  // the kernel stores rows itself and never touches this map
  CUtensorMap mo;
  rc = make_map(ctx, &mo, O, p, p->o_strides);
  if (rc) return rc;
  if (launch_fwd(p->D == 96 ? 128 : p->D, mq, mk, mv, mvt, mo, fp, grid, st) != cudaSuccess) return SAF_ERR_CUDA;
  return SAF_OK;
}

int saf_hybrid_attn_bwd(saf_ctx* ctx, const saf_problem* p, const void* Q, const void* K, const void* V,
                        const void* O, const void* dO, const float* LSE, const uint8_t* frozen_mask_host,
                        const float* alpha, const float* rho, const float* logZ, void* dQ, void* dK, void* dV,
                        void* stream) {
  if (!ctx) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  int rc = validate(p, frozen_mask_host, &nf);
  if (rc) return rc;
  const int no = p->H - nf;
  const bool no_qk_out = p->packed_qk && no == 0;        // packed layout of a frozen-only layer: no dQ / dK at all
  if (!dO || !dV || (!no_qk_out && (!dQ || !dK))) return SAF_ERR_INVALID_ARG;
  if (no > 0 && (!Q || !K || !V || !O || !LSE)) return SAF_ERR_INVALID_ARG;
  if (nf > 0 && (!alpha || !rho)) return SAF_ERR_INVALID_ARG;
  if (!aligned16(dO) || !aligned16(dQ) || !aligned16(dK) || !aligned16(dV)) return SAF_ERR_INVALID_ARG;
  if (no > 0 && (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O))) return SAF_ERR_INVALID_ARG;
  if (check_strides(p->o_strides, p->D)) return SAF_ERR_INVALID_ARG;
  if (no > 0 && (check_strides(p->q_strides, p->D) || check_strides(p->k_strides, p->D) ||
                 check_strides(p->v_strides, p->D)))
    return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;

  if (nf > 0 && !logZ) {
    rc = ensure(ctx->logz_buf, static_cast<size_t>(p->H) * p->Tp * sizeof(float));
    if (rc) return rc;
    rc = saf_pattern_prepare(ctx, p->H, p->Tp, frozen_mask_host, alpha, rho, static_cast<float*>(ctx->logz_buf.ptr),
                             stream);
    if (rc) return rc;
    logZ = static_cast<const float*>(ctx->logz_buf.ptr);
  }
  rc = upload_mask(ctx, frozen_mask_host, p->H, st);
  if (rc) return rc;

  const int nblk = (p->T + BLK - 1) / BLK;
  const int nqh = p->packed_qk ? no : p->H;                  // heads of Q, K, dQ (and of dK when packed)
  const size_t nelem = static_cast<size_t>(p->B) * nqh * p->T * p->D;
  const size_t ext_bytes = static_cast<size_t>(p->B) * p->H * nblk * 4096;   // one 4 KB image per 128-row block
  rc = ensure(ctx->delta_buf, 2 * ext_bytes);                 // q_ext images followed by do_ext images
  if (rc) return rc;
  uint8_t* q_ext = static_cast<uint8_t*>(ctx->delta_buf.ptr);
  uint8_t* do_ext = q_ext + ext_bytes;
  const float scale_v = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(p->D));
  const int grad_f32 = p->grad_dtype == SAF_F32;
  const int kvg = kv_group_of(p);
  float* dqacc = static_cast<float*>(dQ);
  if (!grad_f32 || no_qk_out) {
    rc = ensure(ctx->dqacc_buf, std::max<size_t>(nelem, 64) * sizeof(float));
    if (rc) return rc;
    dqacc = static_cast<float*>(ctx->dqacc_buf.ptr);
  }
  // Shared key/value heads accumulate their gradients in fp32 (reduce-adds); with bf16 gradients that happens in
  // a workspace that is converted at the end, and the kernels see fp32 targets.
  const bool kv_acc = kvg > 1 && !grad_f32;
  const size_t nkv = static_cast<size_t>(p->B) * (p->H / kvg) * p->T * p->D;
  void* dK_k = dK;
  void* dV_k = dV;
  if (kv_acc) {
    if ((rc = ensure(ctx->dkacc_buf, nkv * sizeof(float))) || (rc = ensure(ctx->dvacc_buf, nkv * sizeof(float))))
      return rc;
    dK_k = ctx->dkacc_buf.ptr;
    dV_k = ctx->dvacc_buf.ptr;
  }
  const int kern_f32 = (grad_f32 || kv_acc) ? 1 : 0;
  const int* qslot = nullptr;
  if (p->packed_qk && (rc = upload_qslot(ctx, frozen_mask_host, p->H, st, &qslot))) return rc;
  // tensor-core form of the frozen heads: the preparation kernel also stages w(i) dO in fp16
  const bool tensor_form = nf > 0 && pattern_matches(ctx, p, frozen_mask_host, alpha, rho, logZ);
  PrepFrozen fz{};
  if (tensor_form) {
    rc = ensure(ctx->dot_buf, static_cast<size_t>(p->B) * nf * p->T * p->D * 2);
    if (rc) return rc;
    fz.wvec = static_cast<const float*>(ctx->pat_wvec.ptr);
    fz.hord = static_cast<const int*>(ctx->pat_hord.ptr);
    fz.pat_ok = static_cast<const int*>(ctx->pat_ok.ptr);
    fz.ovf = static_cast<int*>(ctx->ok_bwd.ptr);
    fz.call_id = ++ctx->call_counter;
    fz.dot_dst = ctx->dot_buf.ptr;
    fz.Hf = nf;
    fz.Tp = p->Tp;
    fz.chk = pattern_check(ctx, alpha, rho, logZ);
  }
  // O is only read for ordinary heads; a frozen-only layer may pass O = NULL
  {
    ScopedTimer timer(ctx, SAF_KERNEL_BWD_PREP, st);
    if (launch_bwd_prep(O, p->o_dtype == SAF_F32, dO, LSE, p->o_strides, static_cast<const uint8_t*>(ctx->mask_buf.ptr), q_ext, do_ext,
                        1.0f / scale_v, dqacc, dK_k, dV_k, kern_f32, kvg, qslot, no, fz, p->B, p->H, p->T, p->D, st) !=
        cudaSuccess)
      return SAF_ERR_CUDA;
  }

  const long long n_items = static_cast<long long>(p->B) * p->H * nblk;
  const int grid = static_cast<int>(std::min<long long>(ctx->num_sms, n_items));
  const WorklistEntry* wl = nullptr;
  rc = get_worklist(ctx, p->B, p->H, p->T, frozen_mask_host, 1, grid, p->D != 64, st, &wl);
  if (rc) return rc;

  CUtensorMap mq, mk, mv, mdo;
  rc = make_map(ctx, &mdo, dO, p, p->o_strides);
  if (rc) return rc;
  if (no > 0) {
    if ((rc = make_map(ctx, &mq, Q, p, p->q_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, nqh))) return rc;
    if ((rc = make_map(ctx, &mk, K, p, p->k_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->packed_qk ? no : p->H / kvg)))
      return rc;
    if ((rc = make_map(ctx, &mv, V, p, p->v_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->H / kvg))) return rc;
  } else {
    mq = mdo; mk = mdo; mv = mdo;
  }
  if (p->D != 64) {
    // ---- 128-wide kernel: Q / dO travel as 64-row half tiles, dK / dV leave with plain stores
    CUtensorMap mqh = mdo, mdoh, mdoth, mdq128;
    if ((rc = make_map(ctx, &mdoh, dO, p, p->o_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 0, 64))) return rc;
    if (no > 0 && (rc = make_map(ctx, &mqh, Q, p, p->q_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, nqh, 64))) return rc;
    mdoth = mdoh;
    {
      const cuuint64_t Dd = static_cast<cuuint64_t>(p->D), Tt = static_cast<cuuint64_t>(p->T);
      const cuuint64_t Hq = static_cast<cuuint64_t>(std::max(nqh, 1));
      cuuint64_t dims[4] = {Dd, Tt, Hq, static_cast<cuuint64_t>(p->B)};
      cuuint64_t gs[3] = {Dd * 4, Tt * Dd * 4, Tt * Dd * 4 * Hq};
      cuuint32_t box[4] = {32, BLK, 1, 1};
      cuuint32_t es[4] = {1, 1, 1, 1};
      if (ctx->encode(&mdq128, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, dqacc, dims, gs, box, es,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return SAF_ERR_CUDA;
    }
    BwdParams bp;
    bp.band_b = nullptr; bp.avec = nullptr; bp.fast_ok = nullptr; bp.hord = nullptr; bp.ovf = nullptr; bp.call_id = 0;
    bp.nblkp = (p->Tp + 127) / 128;
    if (tensor_form) {
      if ((rc = make_map_contig(ctx, &mdoth, ctx->dot_buf.ptr, p, nf, 64))) return rc;
      bp.band_b = ctx->pat_bandb.ptr;
      bp.avec = static_cast<const float*>(ctx->pat_avec.ptr);
      bp.fast_ok = fz.pat_ok;
      bp.hord = fz.hord;
      bp.ovf = fz.ovf;
      bp.call_id = fz.call_id;
    }
    bp.B = p->B; bp.H = p->H; bp.T = p->T; bp.Tp = p->Tp;
    bp.kv_group = kvg;
    bp.qslot = qslot;
    bp.n_ord = no;
    bp.d_real = p->D;
    bp.scale = scale_v;
    bp.scale_log2 = scale_v * 1.4426950408889634f;
    bp.alpha = alpha; bp.rho = rho; bp.logZ = logZ;
    bp.q_ext = q_ext;
    bp.do_ext = do_ext;
    bp.nblk = nblk;
    bp.dK = dK_k; bp.dV = dV_k;
    bp.grad_f32 = kern_f32;
    bp.items = wl->items_dev;
    bp.cta_offsets = wl->offsets_dev;
    bp.status = ctx->status_dev;
    bp.wait_limit_ns = ctx->wait_limit_ns;
    {
      ScopedTimer timer(ctx, SAF_KERNEL_BWD, st);
      if (launch_bwd128(mk, mv, mqh, mdoh, mdoth, mdq128, bp, grid, st) != cudaSuccess) return SAF_ERR_CUDA;
    }
    if (!grad_f32) {
      ScopedTimer timer(ctx, SAF_KERNEL_BWD_FINALIZE, st);
      if (nelem > 0 && launch_bwd_finalize(dqacc, dQ, nelem, st) != cudaSuccess) return SAF_ERR_CUDA;
      if (kv_acc && (launch_bwd_finalize(static_cast<const float*>(dK_k), dK, nkv, st) != cudaSuccess ||
                     launch_bwd_finalize(static_cast<const float*>(dV_k), dV, nkv, st) != cudaSuccess))
        return SAF_ERR_CUDA;
    }
    return SAF_OK;
  }
  // fp32 dQ accumulator [B][H][T][64] as a 4-D tensor for tiled reduce-adds: box = 32 floats x 128 rows
  // (dK and dV get maps of the same shape for the tiled stores of the fp32 epilogue)
  CUtensorMap mdq, mdk, mdv;
  {
    // dQ: [B][H][T][64], or [B][Ho][T][64] in the packed layout
    cuuint64_t dims[4] = {64, static_cast<cuuint64_t>(p->T), static_cast<cuuint64_t>(std::max(nqh, 1)),
                          static_cast<cuuint64_t>(p->B)};
    cuuint64_t gs[3] = {64 * 4, static_cast<cuuint64_t>(p->T) * 64 * 4,
                        static_cast<cuuint64_t>(p->T) * 64 * 4 * std::max(nqh, 1)};
    cuuint32_t box[4] = {32, BLK, 1, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    auto enc = [&](CUtensorMap* m, void* base) {
      return ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, base, dims, gs, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    // (the dQ boxes are 32 rows high: every drain warp reduces the rows of its own TMEM lane quarter)
    box[1] = 32;
    if (!enc(&mdq, dqacc)) return SAF_ERR_CUDA;
    box[1] = BLK;
    if (!enc(&mdk, dqacc)) return SAF_ERR_CUDA;
    mdv = mdk;
    // dK: like dQ when packed, else [B][H/kv_group][T][64]; dV: [B][H/kv_group][T][64]
    if (kern_f32 && p->packed_qk && nqh > 0 && !enc(&mdk, dK_k)) return SAF_ERR_CUDA;
    dims[2] = static_cast<cuuint64_t>(p->H / kvg);
    gs[2] = static_cast<cuuint64_t>(p->T) * 64 * 4 * (p->H / kvg);
    if (kern_f32 && ((!p->packed_qk && !enc(&mdk, dK_k)) || !enc(&mdv, dV_k))) return SAF_ERR_CUDA;
  }
  BwdParams bp;
  CUtensorMap mdot = mdo;
  bp.band_b = nullptr; bp.avec = nullptr; bp.fast_ok = nullptr; bp.hord = nullptr; bp.ovf = nullptr; bp.call_id = 0; bp.nblkp = (p->Tp + 127) / 128;
  if (tensor_form) {
    rc = make_map_contig(ctx, &mdot, ctx->dot_buf.ptr, p, nf);
    if (rc) return rc;
    bp.band_b = ctx->pat_bandb.ptr;
    bp.avec = static_cast<const float*>(ctx->pat_avec.ptr);
    bp.fast_ok = fz.pat_ok;
    bp.hord = fz.hord;
    bp.ovf = fz.ovf;
    bp.call_id = fz.call_id;
  }
  bp.B = p->B; bp.H = p->H; bp.T = p->T; bp.Tp = p->Tp;
  bp.kv_group = kvg;
  bp.qslot = qslot;
  bp.n_ord = no;
  bp.d_real = p->D;
  bp.scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(p->D));
  bp.scale_log2 = bp.scale * 1.4426950408889634f;
  bp.alpha = alpha; bp.rho = rho; bp.logZ = logZ;
  bp.q_ext = q_ext;
  bp.do_ext = do_ext;
  bp.nblk = nblk;
  bp.dK = dK_k; bp.dV = dV_k;
  bp.grad_f32 = kern_f32;
  bp.items = wl->items_dev;
  bp.cta_offsets = wl->offsets_dev;
  bp.status = ctx->status_dev;
  bp.wait_limit_ns = ctx->wait_limit_ns;
  {
    ScopedTimer timer(ctx, SAF_KERNEL_BWD, st);
    if (launch_bwd(p->D, mq, mk, mv, mdo, mdq, mdot, mdk, mdv, bp, grid, st) != cudaSuccess) return SAF_ERR_CUDA;
  }
  if (!grad_f32) {
    ScopedTimer timer(ctx, SAF_KERNEL_BWD_FINALIZE, st);
    if (nelem > 0 && launch_bwd_finalize(dqacc, dQ, nelem, st) != cudaSuccess) return SAF_ERR_CUDA;
    if (kv_acc && (launch_bwd_finalize(static_cast<const float*>(dK_k), dK, nkv, st) != cudaSuccess ||
                   launch_bwd_finalize(static_cast<const float*>(dV_k), dV, nkv, st) != cudaSuccess))
      return SAF_ERR_CUDA;
  }
  return SAF_OK;
}

int saf_hybrid_attn_step_host(saf_ctx* ctx, const saf_problem* p, const void* Q_host, const void* K_host,
                              const void* V_host, const void* dO_host, const uint8_t* frozen_mask_host,
                              const float* alpha_host, const float* rho_host, int32_t prepare, void* O_host,
                              float* LSE_host, void* dQ_host, void* dK_host, void* dV_host) {
  if (!ctx) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  int rc = validate(p, frozen_mask_host, &nf);
  if (rc) return rc;
  const int no = p->H - nf;
  if (p->packed_qk || p->o_dtype != SAF_BF16) return SAF_ERR_UNSUPPORTED;
  if (!V_host || (no > 0 && (!Q_host || !K_host)) || (nf > 0 && (!alpha_host || !rho_host))) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  const int kvg = kv_group_of(p);
  const size_t nelem = static_cast<size_t>(p->B) * p->H * p->T * p->D;
  const size_t tb = nelem * 2;
  const size_t gb = nelem * (p->grad_dtype == SAF_F32 ? 4 : 2);
  const size_t pb = static_cast<size_t>(p->H) * p->Tp * sizeof(float);
  const size_t lb = static_cast<size_t>(p->B) * p->H * p->T * sizeof(float);
  const bool bwd = dO_host != nullptr;
  if ((rc = ensure(ctx->hq, tb)) || (rc = ensure(ctx->hk, tb)) || (rc = ensure(ctx->hv, tb)) ||
      (rc = ensure(ctx->ho, tb)) || (rc = ensure(ctx->hlse, lb)) || (rc = ensure(ctx->halpha, pb)) ||
      (rc = ensure(ctx->hrho, pb)) || (rc = ensure(ctx->hlogz, pb)))
    return rc;
  if (bwd && ((rc = ensure(ctx->hdo, tb)) || (rc = ensure(ctx->hdq, gb)) || (rc = ensure(ctx->hdk, gb)) ||
              (rc = ensure(ctx->hdv, gb))))
    return rc;
  // Three streams: inputs in, compute, results out.  The batch is cut into chunks; chunk c+1 is on its way in and
  // chunk c-1 on its way out (the link is full duplex) while chunk c computes.
  if (!ctx->hs_main) {
    if (cudaStreamCreateWithFlags(&ctx->hs_main, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&ctx->hs_copy, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&ctx->hs_outs, cudaStreamNonBlocking) != cudaSuccess)
      return SAF_ERR_CUDA;
    for (int c = 0; c < saf_ctx::HS_CHUNKS; ++c)
      for (cudaEvent_t* e : {&ctx->hs_in[c], &ctx->hs_do[c], &ctx->hs_fwd[c], &ctx->hs_cmp[c]})
        if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return SAF_ERR_CUDA;
  }
  cudaStream_t st = ctx->hs_main, sc = ctx->hs_copy, so = ctx->hs_outs;
  // chunks of whole batches; small problems go in one piece (a chunk should keep the link busy for a while)
  int nchunks = 1;
  if (tb >= (8u << 20)) nchunks = std::min<int>(saf_ctx::HS_CHUNKS, p->B);
  const int bc_max = (p->B + nchunks - 1) / nchunks;
  saf_problem q = *p;
  const int64_t s2 = p->D, s1 = static_cast<int64_t>(p->T) * p->D, s0 = s1 * p->H;
  int64_t* sets[4] = {q.q_strides, q.k_strides, q.v_strides, q.o_strides};
  for (int64_t* s : sets) { s[0] = s0; s[1] = s1; s[2] = s2; }
  q.k_strides[0] = q.v_strides[0] = s0 / kvg;
  bool okc = true;
  if (nf > 0 && prepare) {
    okc &= cudaMemcpyAsync(ctx->halpha.ptr, alpha_host, pb, cudaMemcpyHostToDevice, st) == cudaSuccess;
    okc &= cudaMemcpyAsync(ctx->hrho.ptr, rho_host, pb, cudaMemcpyHostToDevice, st) == cudaSuccess;
  }
  if (!okc) return SAF_ERR_CUDA;
  const float* a = static_cast<const float*>(ctx->halpha.ptr);
  const float* r = static_cast<const float*>(ctx->hrho.ptr);
  float* z = static_cast<float*>(ctx->hlogz.ptr);
  if (nf > 0 && prepare && (rc = saf_pattern_prepare(ctx, p->H, p->Tp, frozen_mask_host, a, r, z, st))) return rc;
  const size_t esz = 2, gsz = (p->grad_dtype == SAF_F32 ? 4 : 2);
  const size_t per_b = static_cast<size_t>(p->H) * p->T * p->D;          // elements of one batch entry, H heads
  const size_t per_b_kv = per_b / kvg;
  const size_t per_b_lse = static_cast<size_t>(p->H) * p->T;
  auto off = [](const void* base, size_t bytes) { return static_cast<const char*>(base) + bytes; };
  auto offw = [](void* base, size_t bytes) { return static_cast<char*>(base) + bytes; };
  int ci = 0;
  for (int b0 = 0; b0 < p->B; b0 += bc_max, ++ci) {
    const int bc = std::min(bc_max, p->B - b0);
    q.B = bc;
    const size_t o_q = b0 * per_b, o_kv = b0 * per_b_kv, o_l = b0 * per_b_lse;
    // ---- in: Q, K, V, then dO
    if (no > 0) {
      okc &= cudaMemcpyAsync(offw(ctx->hq.ptr, o_q * esz), off(Q_host, o_q * esz), bc * per_b * esz,
                             cudaMemcpyHostToDevice, sc) == cudaSuccess;
      okc &= cudaMemcpyAsync(offw(ctx->hk.ptr, o_kv * esz), off(K_host, o_kv * esz), bc * per_b_kv * esz,
                             cudaMemcpyHostToDevice, sc) == cudaSuccess;
    }
    okc &= cudaMemcpyAsync(offw(ctx->hv.ptr, o_kv * esz), off(V_host, o_kv * esz), bc * per_b_kv * esz,
                           cudaMemcpyHostToDevice, sc) == cudaSuccess;
    okc &= cudaEventRecord(ctx->hs_in[ci], sc) == cudaSuccess;
    if (bwd) {
      okc &= cudaMemcpyAsync(offw(ctx->hdo.ptr, o_q * esz), off(dO_host, o_q * esz), bc * per_b * esz,
                             cudaMemcpyHostToDevice, sc) == cudaSuccess;
      okc &= cudaEventRecord(ctx->hs_do[ci], sc) == cudaSuccess;
    }
    // ---- compute
    okc &= cudaStreamWaitEvent(st, ctx->hs_in[ci], 0) == cudaSuccess;
    if (!okc) return SAF_ERR_CUDA;
    void* Oc = offw(ctx->ho.ptr, o_q * esz);
    float* Lc = static_cast<float*>(ctx->hlse.ptr) + o_l;
    rc = saf_hybrid_attn_fwd(ctx, &q, offw(ctx->hq.ptr, o_q * esz), offw(ctx->hk.ptr, o_kv * esz),
                             offw(ctx->hv.ptr, o_kv * esz), frozen_mask_host, a, r, z, Oc, Lc, st);
    if (rc) return rc;
    // O and LSE leave as soon as the forward of the chunk is done
    okc &= cudaEventRecord(ctx->hs_fwd[ci], st) == cudaSuccess;
    okc &= cudaStreamWaitEvent(so, ctx->hs_fwd[ci], 0) == cudaSuccess;
    if (O_host) okc &= cudaMemcpyAsync(offw(O_host, o_q * esz), Oc, bc * per_b * esz, cudaMemcpyDeviceToHost, so) == cudaSuccess;
    if (LSE_host)
      okc &= cudaMemcpyAsync(LSE_host + o_l, Lc, bc * per_b_lse * sizeof(float), cudaMemcpyDeviceToHost, so) == cudaSuccess;
    if (bwd) {
      // (dO was queued behind the chunk's Q, K, V on the inbound stream)
      okc &= cudaStreamWaitEvent(st, ctx->hs_do[ci], 0) == cudaSuccess;
      if (!okc) return SAF_ERR_CUDA;
      void* dQc = offw(ctx->hdq.ptr, o_q * gsz);
      void* dKc = offw(ctx->hdk.ptr, o_kv * gsz);
      void* dVc = offw(ctx->hdv.ptr, o_kv * gsz);
      rc = saf_hybrid_attn_bwd(ctx, &q, offw(ctx->hq.ptr, o_q * esz), offw(ctx->hk.ptr, o_kv * esz),
                               offw(ctx->hv.ptr, o_kv * esz), Oc, offw(ctx->hdo.ptr, o_q * esz), Lc, frozen_mask_host,
                               a, r, z, dQc, dKc, dVc, st);
      if (rc) return rc;
      okc &= cudaEventRecord(ctx->hs_cmp[ci], st) == cudaSuccess;
      okc &= cudaStreamWaitEvent(so, ctx->hs_cmp[ci], 0) == cudaSuccess;
      if (dQ_host) okc &= cudaMemcpyAsync(offw(dQ_host, o_q * gsz), dQc, bc * per_b * gsz, cudaMemcpyDeviceToHost, so) == cudaSuccess;
      if (dK_host) okc &= cudaMemcpyAsync(offw(dK_host, o_kv * gsz), dKc, bc * per_b_kv * gsz, cudaMemcpyDeviceToHost, so) == cudaSuccess;
      if (dV_host) okc &= cudaMemcpyAsync(offw(dV_host, o_kv * gsz), dVc, bc * per_b_kv * gsz, cudaMemcpyDeviceToHost, so) == cudaSuccess;
    }
    if (!okc) return SAF_ERR_CUDA;
  }
  if (cudaStreamSynchronize(sc) != cudaSuccess || cudaStreamSynchronize(so) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return SAF_ERR_CUDA;
  return saf_last_device_status(ctx, nullptr);
}

int saf_pattern_grad(saf_ctx* ctx, const saf_problem* p, const void* V, const void* O, const void* dO,
                     const uint8_t* frozen_mask_host, const float* alpha, const float* rho, const float* logZ,
                     float* dalpha_out, float* drho_out, void* stream) {
  if (!ctx || !dalpha_out || !drho_out) return SAF_ERR_INVALID_ARG;
  int nf = 0;
  int rc = validate(p, frozen_mask_host, &nf);
  if (rc) return rc;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;
  const size_t pbytes = static_cast<size_t>(p->H) * p->Tp * sizeof(float);
  if (cudaMemsetAsync(dalpha_out, 0, pbytes, st) != cudaSuccess || cudaMemsetAsync(drho_out, 0, pbytes, st) != cudaSuccess)
    return SAF_ERR_CUDA;
  if (nf == 0) return SAF_OK;
  if (!V || !O || !dO || !alpha || !rho || !logZ) return SAF_ERR_INVALID_ARG;
  if (!aligned16(V) || !aligned16(O) || !aligned16(dO)) return SAF_ERR_INVALID_ARG;
  if (check_strides(p->v_strides, p->D) || check_strides(p->o_strides, p->D)) return SAF_ERR_INVALID_ARG;
  const int kvg = kv_group_of(p);
  // ordinal -> head table of the frozen heads, and delta = rowsum(dO o O) of their rows
  std::vector<int> hlist;
  for (int h = 0; h < p->H; ++h)
    if (frozen_mask_host[h]) hlist.push_back(h);
  const void* const hlist_dev_before = ctx->pg_hlist.ptr;
  if ((rc = ensure(ctx->pg_hlist, static_cast<size_t>(p->H) * sizeof(int))) ||
      (rc = ensure(ctx->pg_delta, static_cast<size_t>(p->B) * p->H * p->T * sizeof(float))))
    return rc;
  if (ctx->pg_hlist.ptr != hlist_dev_before) ctx->pg_hlist_host.clear();   // a new buffer holds nothing yet
  // The tables are uploaded on the caller's stream from vectors the context owns, and only when they change (an
  // earlier launch may still be reading the device copy: stream order keeps the two apart).
  if (hlist != ctx->pg_hlist_host) {
    ctx->pg_hlist_host = hlist;
    if (cudaMemcpyAsync(ctx->pg_hlist.ptr, ctx->pg_hlist_host.data(), hlist.size() * sizeof(int), cudaMemcpyHostToDevice,
                        st) != cudaSuccess)
      return SAF_ERR_CUDA;
  }
  {
    ScopedTimer timer(ctx, SAF_KERNEL_BWD_PREP, st);
    if (launch_rowdot(O, p->o_dtype == SAF_F32, dO, p->o_strides, static_cast<const int*>(ctx->pg_hlist.ptr),
                      static_cast<float*>(ctx->pg_delta.ptr), p->B, p->H, nf, p->T, p->D, st) != cudaSuccess)
      return SAF_ERR_CUDA;
  }
  // Work list: (frozen-head ordinal, key block J, run of query blocks, run of batch entries), dealt longest first to
  // the least loaded CTA.  An item costs its tiles plus about 0.7 of a tile for loading its V tiles (which cannot
  // start before the item in front of it has finished), so longer runs are cheaper but balance worse: the run
  // length is the one of 1 .. 16 whose dealt list has the shortest longest CTA under that cost.
  const int nblk = (p->T + BLK - 1) / BLK;
  const int vb = pgrad_batch_chunk(p->D);
  const int nbc = (p->B + vb - 1) / vb;
  const long long total_tiles = static_cast<long long>(nf) * nbc * nblk * (nblk + 1) / 2;
  const int grid = static_cast<int>(std::min<long long>(ctx->num_sms, total_tiles));
  const std::array<int, 5> key = {p->B, nf, p->T, p->D, grid};
  if (key != ctx->pg_key) {
    auto cost = [](const PgItem& w) { return 10 * (w.I1 - w.I0) + 7; };
    auto deal = [&](int run, std::vector<std::vector<PgItem>>* out) {
      std::vector<PgItem> items;
      for (int hf = 0; hf < nf; ++hf)
        for (int c = 0; c < nbc; ++c)
          for (int J = 0; J < nblk; ++J)
            for (int I0 = J; I0 < nblk; I0 += run)
              items.push_back(PgItem{hf, J, I0, std::min(nblk, I0 + run), c * vb, std::min(p->B, (c + 1) * vb), 0, 0});
      std::stable_sort(items.begin(), items.end(), [&](const PgItem& a, const PgItem& b) { return cost(a) > cost(b); });
      std::priority_queue<std::pair<long long, int>, std::vector<std::pair<long long, int>>, std::greater<>> load;
      for (int c = 0; c < grid; ++c) load.push({0, c});
      if (out) out->assign(grid, {});
      long long longest = 0;
      for (const PgItem& w : items) {
        auto [l, c] = load.top();
        load.pop();
        if (out) (*out)[c].push_back(w);
        load.push({l + cost(w), c});
        longest = std::max(longest, l + cost(w));
      }
      return longest;
    };
    int run = 1;
    long long best = -1;
    for (int r = 1; r <= std::min(16, nblk); ++r) {
      const long long m = deal(r, nullptr);
      if (best < 0 || m < best) {
        best = m;
        run = r;
      }
    }
    std::vector<std::vector<PgItem>> per_cta;
    deal(run, &per_cta);
    ctx->pg_items_host.clear();
    ctx->pg_offsets_host.assign(1, 0);
    for (int c = 0; c < grid; ++c) {
      ctx->pg_items_host.insert(ctx->pg_items_host.end(), per_cta[c].begin(), per_cta[c].end());
      ctx->pg_offsets_host.push_back(static_cast<int>(ctx->pg_items_host.size()));
    }
    if ((rc = ensure(ctx->pg_items, ctx->pg_items_host.size() * sizeof(PgItem))) ||
        (rc = ensure(ctx->pg_offsets, ctx->pg_offsets_host.size() * sizeof(int))))
      return rc;
    if (cudaMemcpyAsync(ctx->pg_items.ptr, ctx->pg_items_host.data(), ctx->pg_items_host.size() * sizeof(PgItem),
                        cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ctx->pg_offsets.ptr, ctx->pg_offsets_host.data(), ctx->pg_offsets_host.size() * sizeof(int),
                        cudaMemcpyHostToDevice, st) != cudaSuccess)
      return SAF_ERR_CUDA;
    ctx->pg_key = key;
  }
  CUtensorMap mv, mdo;
  // at D = 64 a tile is one 64-column panel, so one copy can bring the tiles of a whole batch run (V) or ring stage (dO)
  const int vbox = p->D == 64 ? vb : 1, dobox = p->D == 64 ? pgrad_stage_entries(p->D) : 1;
  if ((rc = make_map(ctx, &mv, V, p, p->v_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->H / kvg, BLK, vbox))) return rc;
  if ((rc = make_map(ctx, &mdo, dO, p, p->o_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 0, BLK, dobox))) return rc;
  PgradParams gp;
  gp.B = p->B; gp.H = p->H; gp.T = p->T; gp.Tp = p->Tp;
  gp.kv_group = kvg;
  gp.alpha = alpha; gp.rho = rho; gp.logZ = logZ;
  gp.delta = static_cast<const float*>(ctx->pg_delta.ptr);
  gp.hlist = static_cast<const int*>(ctx->pg_hlist.ptr);
  gp.dalpha = dalpha_out;
  gp.drho = drho_out;
  gp.items = static_cast<const PgItem*>(ctx->pg_items.ptr);
  gp.cta_offsets = static_cast<const int*>(ctx->pg_offsets.ptr);
  gp.status = ctx->status_dev;
  gp.wait_limit_ns = ctx->wait_limit_ns;
  {
    ScopedTimer timer(ctx, SAF_KERNEL_PGRAD, st);
    // (head dimension 96 runs on the 128-wide kernel: TMA zero-fills features 96..127)
    if (launch_pgrad(p->D == 96 ? 128 : p->D, mv, mdo, gp, grid, st) != cudaSuccess) return SAF_ERR_CUDA;
  }
  return SAF_OK;
}

int saf_fit_marginals(saf_ctx* ctx, int32_t Hf, int32_t T, const float* mean_attn, float floor_value,
                      double* eta_abs_out, double* eta_rel_out, double* plogp_out, void* stream) {
  if (!ctx || !eta_abs_out || !eta_rel_out || !plogp_out) return SAF_ERR_INVALID_ARG;
  if (Hf < 0 || T < 1 || !(floor_value > 0.0f)) return SAF_ERR_INVALID_ARG;
  if (T > fit_max_T()) return SAF_ERR_UNSUPPORTED;
  if (Hf == 0) return SAF_OK;
  if (!mean_attn || Hf > 65535) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;
  const size_t vb = static_cast<size_t>(Hf) * T * sizeof(double);
  if (cudaMemsetAsync(eta_abs_out, 0, vb, st) != cudaSuccess || cudaMemsetAsync(eta_rel_out, 0, vb, st) != cudaSuccess ||
      cudaMemsetAsync(plogp_out, 0, static_cast<size_t>(Hf) * sizeof(double), st) != cudaSuccess)
    return SAF_ERR_CUDA;
  ScopedTimer timer(ctx, SAF_KERNEL_FIT_MARGINALS, st);
  if (launch_fit_marginals(mean_attn, floor_value, eta_abs_out, eta_rel_out, plogp_out, Hf, T, ctx->num_sms, st) !=
      cudaSuccess)
    return SAF_ERR_CUDA;
  return SAF_OK;
}

int saf_fit_compact(saf_ctx* ctx, int32_t Hf, int32_t T, const double* eta_abs, const double* eta_rel,
                    const double* plogp, int32_t steps, double lr, float* alpha_out, float* rho_out, float* logZ_out,
                    int64_t out_stride, double* loss_out, double* kl_out, void* stream) {
  if (!ctx || Hf < 0 || T < 1 || steps < 0 || !(lr > 0.0) || out_stride < T) return SAF_ERR_INVALID_ARG;
  if (T > fit_max_T()) return SAF_ERR_UNSUPPORTED;
  if (Hf == 0) return SAF_OK;
  if (!eta_abs || !eta_rel || !alpha_out || !rho_out || !logZ_out || Hf > 65535) return SAF_ERR_INVALID_ARG;
  if (kl_out && !plogp) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;
  // state: 6 fp64 and 5 fp32 arrays of [Hf, T]
  const size_t n = static_cast<size_t>(Hf) * T;
  int rc = ensure(ctx->fit_buf, n * (6 * sizeof(double) + 5 * sizeof(float)));
  if (rc) return rc;
  FitState s;
  s.T = T;
  s.lr = lr;
  s.eta_abs = eta_abs;
  s.eta_rel = eta_rel;
  double* d = static_cast<double*>(ctx->fit_buf.ptr);
  s.alpha = d; s.rho = d + n; s.m_a = d + 2 * n; s.v_a = d + 3 * n; s.m_r = d + 4 * n; s.v_r = d + 5 * n;
  float* f = reinterpret_cast<float*>(d + 6 * n);
  s.a2[0] = f; s.a2[1] = f + n; s.r2[0] = f + 2 * n; s.r2[1] = f + 3 * n; s.nz2 = f + 4 * n;
  ScopedTimer timer(ctx, SAF_KERNEL_FIT, st);
  if (launch_fit(s, Hf, steps, plogp, alpha_out, rho_out, logZ_out, out_stride, loss_out, kl_out, st) != cudaSuccess)
    return SAF_ERR_CUDA;
  return SAF_OK;
}

int saf_calib_accumulate(saf_ctx* ctx, const saf_problem* p, const void* Q, const void* K, const float* LSE,
                         float* mean_sum, double* sumsq, double* sum_plogp, int32_t accumulate, void* stream) {
  if (!ctx || !p || !mean_sum || !sumsq || !sum_plogp) return SAF_ERR_INVALID_ARG;
  if (p->B < 1 || p->H < 1 || p->T < 1) return SAF_ERR_INVALID_ARG;
  if (p->D != 64 && p->D != 96 && p->D != 128) return SAF_ERR_UNSUPPORTED;
  if (p->kv_group < 0 || (p->kv_group > 1 && p->H % p->kv_group != 0) || p->packed_qk) return SAF_ERR_INVALID_ARG;
  if (!Q || !K || !LSE || !aligned16(Q) || !aligned16(K) || !aligned16(mean_sum)) return SAF_ERR_INVALID_ARG;
  if (check_strides(p->q_strides, p->D) || check_strides(p->k_strides, p->D)) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;
  const int kvg = kv_group_of(p);
  if (!accumulate) {
    const size_t hb = static_cast<size_t>(p->H) * sizeof(double);
    if (cudaMemsetAsync(sumsq, 0, hb, st) != cudaSuccess || cudaMemsetAsync(sum_plogp, 0, hb, st) != cudaSuccess)
      return SAF_ERR_CUDA;
  }
  CUtensorMap mq, mk;
  int rc;
  if ((rc = make_map(ctx, &mq, Q, p, p->q_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->H))) return rc;
  if ((rc = make_map(ctx, &mk, K, p, p->k_strides, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p->H / kvg))) return rc;
  // the dense accumulator as a [1][H][T][T] fp32 tensor, boxes of 128 rows x 32 columns (128-byte rows, swizzled)
  CUtensorMap mm = mq;
  const bool use_tma = (p->T % 4) == 0;
  if (use_tma) {
    const cuuint64_t Tt = static_cast<cuuint64_t>(p->T);
    cuuint64_t dims[4] = {Tt, Tt, static_cast<cuuint64_t>(p->H), 1};
    cuuint64_t gs[3] = {Tt * 4, Tt * Tt * 4, Tt * Tt * 4 * static_cast<cuuint64_t>(p->H)};
    cuuint32_t box[4] = {32, BLK, 1, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    if (ctx->encode(&mm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, mean_sum, dims, gs, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SAF_ERR_CUDA;
  }
  const int nblk = (p->T + BLK - 1) / BLK;
  CalibParams cp;
  cp.use_tma = use_tma ? 1 : 0;
  cp.B = p->B; cp.H = p->H; cp.T = p->T;
  cp.kv_group = kvg;
  const float scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / std::sqrt(static_cast<float>(p->D));
  cp.scale_log2e = scale * 1.4426950408889634f;
  cp.LSE = LSE;
  cp.mean_sum = mean_sum;
  cp.sumsq = sumsq;
  cp.sum_plogp = sum_plogp;
  cp.accumulate = accumulate ? 1 : 0;
  cp.npairs = nblk * (nblk + 1) / 2;
  const long long n_items = static_cast<long long>(p->H) * cp.npairs;
  if (n_items > 0x7fffffffLL) return SAF_ERR_INVALID_ARG;
  cp.n_items = static_cast<int>(n_items);
  cp.status = ctx->status_dev;
  cp.wait_limit_ns = ctx->wait_limit_ns;
  const int grid = static_cast<int>(std::min<long long>(ctx->num_sms, n_items));
  ScopedTimer timer(ctx, SAF_KERNEL_CALIB, st);
  // (head dimension 96 runs on the 128-wide kernel: TMA zero-fills features 96..127)
  if (launch_calib(p->D == 64 ? 64 : 128, mq, mk, mm, cp, grid, st) != cudaSuccess) return SAF_ERR_CUDA;
  return SAF_OK;
}

int saf_calib_finalize(saf_ctx* ctx, int32_t H, int32_t T, int64_t n_total, float* mean_inout, const double* sumsq,
                       const double* sum_plogp, double* s_var_out, double* s_kl_out, void* stream) {
  if (!ctx || H < 1 || T < 1 || n_total < 1 || !mean_inout || !sumsq || !sum_plogp) return SAF_ERR_INVALID_ARG;
  if (s_var_out && n_total < 2) return SAF_ERR_INVALID_ARG;   // the sample variance needs two sequences
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->last_stream = st;
  int rc = ensure(ctx->calib_tmp, static_cast<size_t>(H) * 2 * sizeof(double));
  if (rc) return rc;
  ScopedTimer timer(ctx, SAF_KERNEL_CALIB_FINALIZE, st);
  if (launch_calib_finalize(mean_inout, sumsq, sum_plogp, static_cast<double*>(ctx->calib_tmp.ptr), H, T,
                            static_cast<double>(n_total), s_var_out, s_kl_out, ctx->num_sms, st) != cudaSuccess)
    return SAF_ERR_CUDA;
  return SAF_OK;
}

int saf_last_device_status(saf_ctx* ctx, int32_t* detail_out) {
  if (!ctx) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  if (cudaStreamSynchronize(ctx->last_stream) != cudaSuccess) return SAF_ERR_CUDA;
  int word = 0;
  if (cudaMemcpy(&word, ctx->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SAF_ERR_CUDA;
  if (detail_out) *detail_out = word;
  if (word != 0) {
    cudaMemset(ctx->status_dev, 0, sizeof(int));
    return SAF_ERR_DEVICE_TIMEOUT;
  }
  return SAF_OK;
}

int saf_set_profiling(saf_ctx* ctx, int32_t enable) {
  if (!ctx) return SAF_ERR_INVALID_ARG;
  ctx->profiling = enable != 0;
  return SAF_OK;
}

int saf_get_kernel_time(saf_ctx* ctx, int32_t which, float* total_ms_out, int32_t* launches_out) {
  if (!ctx || !total_ms_out || !launches_out || which < 0 || which >= SAF_KERNEL_COUNT) return SAF_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SAF_ERR_CUDA;
  double total = 0.0;
  int n = 0;
  std::vector<TimedLaunch> keep;
  for (const TimedLaunch& t : ctx->timed) {
    if (t.which != which) {
      keep.push_back(t);
      continue;
    }
    float ms = 0.0f;
    if (cudaEventSynchronize(t.end) != cudaSuccess || cudaEventElapsedTime(&ms, t.beg, t.end) != cudaSuccess)
      return SAF_ERR_CUDA;
    total += ms;
    ++n;
    ctx->event_pool.push_back(t.beg);
    ctx->event_pool.push_back(t.end);
  }
  ctx->timed.swap(keep);
  *total_ms_out = static_cast<float>(total);
  *launches_out = n;
  return SAF_OK;
}

int saf_build_worklist(int32_t B, int32_t H, int32_t T, const uint8_t* frozen_mask_host, int32_t backward,
                       int32_t n_ctas, int32_t frozen_weight_pct, int32_t* items_out, int32_t* offsets_out) {
  if (B < 1 || H < 1 || T < 1 || n_ctas < 1 || !frozen_mask_host || !items_out || !offsets_out ||
      frozen_weight_pct < 1)
    return SAF_ERR_INVALID_ARG;
  std::vector<WorkItem> items;
  std::vector<int> offsets;
  int fp_unused, ov, ovf;
  sched_defaults(0, backward ? 1 : 0, &fp_unused, &ov, &ovf);      // the 64-wide kernels' per-item overheads
  build_worklist_host(B, H, T, frozen_mask_host, backward ? 1 : 0, n_ctas, frozen_weight_pct, ov, ovf, 0, items, offsets);
  std::memcpy(items_out, items.data(), items.size() * sizeof(WorkItem));
  std::memcpy(offsets_out, offsets.data(), offsets.size() * sizeof(int));
  return SAF_OK;
}

}  // extern "C"
