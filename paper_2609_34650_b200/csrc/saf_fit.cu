// The compact-pattern fitter (Sec. 3.2 "Fitting", Eq. "fit-objective"; Algorithm 1's fitting loop; appendix
// "Selection, fitting, and installation" and "Compact fitting and storage").
//
//   target     P = rows of the mean attention map, causal entries floored at 1e-9, each row scaled to sum one
//   marginals  eta_abs(j) = sum_{i>=j} P(i,j),  eta_rel(d) = sum_{i-j=d} P(i,j),  and sum_{ij} P log P
//   Fit        alpha = 0, rho(d) = log max(eta_rel(d)/(T-d), 1e-9); J Adam steps on
//              L = (1/T)[sum_i log Z(i) - eta_abs.alpha - eta_rel.rho],  whose gradient is
//              (fitted marginal - target marginal)/T
//   accept     kappa = mean row KL(P || P^) = L + (1/T) sum P log P   (rows of P sum to one)
//
// Nothing of size T x T is formed after the target has been read once.  Every Adam step is two launches:
//   pass A   rows:      S(i) = sum_{d<=i} exp2(r'(d) + a'(i-d) - z'(i)),  z'(i) += log2 S(i)
//   pass B   marginals: c(j) = sum_d exp2(r'(d) - z'(j+d) + a'(j))  and  g(d) = sum_j exp2(a'(j) - z'(j+d) + r'(d)),
//            followed in the same thread by the Adam update of alpha(j) / rho(d) (fp64 state)
// (primes: scaled by log2 e; z' is log2 Z).  All three sums have the same shape
//   out(x) = sum_y exp2(u[y] + win[x -/+ y] + c[x]),
// one lane per x, the operand u uniform over the warp, the window operand contiguous over the lanes, so one kernel
// serves them.  The reference point of the exponentials is the previous step's z' (one Adam step moves every
// parameter by a fraction of a unit), so no running maximum is needed; the first pass starts from the upper bound
// max r' (alpha = 0).  The special-function unit (one exp2 per causal pair and pass) bounds the kernel.
#include <cuda_runtime.h>
#include <cstdint>
#include <cmath>
#include <algorithm>
#include "saf_internal.h"

namespace saf {

namespace {

constexpr double LOG2E_D = 1.4426950408889634074;
constexpr double LN2_D = 0.6931471805599453094;
constexpr int XB = 32;             // x values per CTA of the pass kernel (one per lane)
constexpr int PASS_WARPS = 8;      // warps of a pass CTA; they split the y range in chunks of 32
constexpr int YC = 4096;           // y values staged in shared memory at a time

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ------------------------------------------------------------------------------------------------ target marginals
// One CTA of NT threads walks rows blockIdx.x, blockIdx.x + gridDim.x, ... of head blockIdx.y.  Thread t owns the
// columns t, t + NT, ...: their column sums stay in registers over all rows of the CTA; the diagonal sums live in
// shared memory (for a given row every thread touches different distances, rows are separated by the CTA barrier of
// the row-sum reduction).  256 threads with up to 32 columns each measured fastest (loading the next row ahead of
// the reduction costs registers, hence resident CTAs, and measured slower).
// Row pieces specialised on the number KK of column chunks that reach the diagonal, so that the chunks above it
// cost nothing and the loads of a row still issue back to back.
template <int NT, int KK>
__device__ __forceinline__ void marg_load(const float* __restrict__ r, int row, int tid, float floor_v, float* dst) {
#pragma unroll
  for (int k = 0; k < KK; ++k) {
    const int j = tid + k * NT;
    dst[k] = (j <= row) ? fmaxf(__ldg(r + j), floor_v) : 0.0f;
  }
}
template <int KK>
__device__ __forceinline__ float marg_sum(const float* cur) {
  float s = 0.0f;
#pragma unroll
  for (int k = 0; k < KK; ++k) s += cur[k];
  return s;
}
template <int NT, int KK>
__device__ __forceinline__ void marg_consume(const float* cur, float inv, float* col, float* dg, float& ent, int i,
                                             int tid) {
#pragma unroll
  for (int k = 0; k < KK; ++k) {
    if (tid + k * NT <= i) {
      const float p = cur[k] * inv;
      col[k] += p;
      dg[-k * NT] += p;
      ent = fmaf(p, __log2f(p), ent);
    }
  }
}
// (quarters of the NCH chunks: case q serves rows whose last chunk index is below (q+1) NCH/4; one case per chunk
// count measured slower: more registers, fewer resident CTAs)
#define SAF_MARG_DISPATCH(q, CALL)                         \
  switch (q) {                                             \
    case 0: { constexpr int KK = G; CALL; } break;         \
    case 1: { constexpr int KK = 2 * G; CALL; } break;     \
    case 2: { constexpr int KK = 3 * G; CALL; } break;     \
    default: { constexpr int KK = NCH; CALL; } break;      \
  }

template <int NT, int NCH>
__global__ void __launch_bounds__(NT)
saf_fit_marginals_kernel(const float* __restrict__ Abar, float floor_v, double* __restrict__ eta_abs,
                         double* __restrict__ eta_rel, double* __restrict__ plogp, int T) {
  extern __shared__ float sm_f[];
  float* diag = sm_f;                          // [T]
  constexpr int NW = NT / 32;
  constexpr int G = (NCH >= 4) ? NCH / 4 : NCH;
  __shared__ float red[2][NW];
  __shared__ double redd[NW];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.y;
  const float* A = Abar + static_cast<size_t>(h) * T * T;
  for (int d = tid; d < T; d += NT) diag[d] = 0.0f;
  float col[NCH];
#pragma unroll
  for (int k = 0; k < NCH; ++k) col[k] = 0.0f;
  float ent = 0.0f;                            // sum p log2 p of this thread (scaled to nats at the end)
  double ent_d = 0.0;
  float cur[NCH];
  int i = blockIdx.x;
  if (i < T) {
    SAF_MARG_DISPATCH((i / NT) / G, (marg_load<NT, KK>(A + static_cast<size_t>(i) * T, i, tid, floor_v, cur)));
  }
  __syncthreads();
  int par = 0, nrow = 0;
  for (; i < T; i += gridDim.x, par ^= 1, ++nrow) {
    const int q = (i / NT) / G;
    float s = 0.0f;
    SAF_MARG_DISPATCH(q, (s = marg_sum<KK>(cur)));
    s = warp_sum(s);
    if (lane == 0) red[par][warp] = s;
    __syncthreads();                           // also: the previous row's diagonal updates are complete
    float tot = 0.0f;
#pragma unroll
    for (int w = 0; w < NW; ++w) tot += red[par][w];
    const float inv = 1.0f / tot;
    float* dg = diag + (i - tid);
    SAF_MARG_DISPATCH(q, (marg_consume<NT, KK>(cur, inv, col, dg, ent, i, tid)));
    if ((nrow & 63) == 63) {                   // keep the fp32 partial short
      ent_d += static_cast<double>(ent);
      ent = 0.0f;
    }
    const int inext = i + gridDim.x;
    if (inext < T) {
      SAF_MARG_DISPATCH((inext / NT) / G, (marg_load<NT, KK>(A + static_cast<size_t>(inext) * T, inext, tid, floor_v, cur)));
    }
  }
  ent_d += static_cast<double>(ent);
  __syncthreads();
  double* ea = eta_abs + static_cast<size_t>(h) * T;
  double* er = eta_rel + static_cast<size_t>(h) * T;
#pragma unroll
  for (int k = 0; k < NCH; ++k) {
    const int j = tid + k * NT;
    if (j < T && col[k] != 0.0f) atomicAdd(ea + j, static_cast<double>(col[k]));
  }
  for (int d = tid; d < T; d += NT)
    if (diag[d] != 0.0f) atomicAdd(er + d, static_cast<double>(diag[d]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ent_d += __shfl_xor_sync(0xffffffffu, ent_d, o);
  if (lane == 0) redd[warp] = ent_d;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < NW; ++w) t += redd[w];
    atomicAdd(plogp + h, t * LN2_D);
  }
}
#undef SAF_MARG_DISPATCH

// ------------------------------------------------------------------------------------------------ Fit: start
// One CTA per head: alpha = 0, rho(d) = log max(eta_rel(d)/(T-d), 1e-9), Adam moments zero, and the first
// reference point of the exponentials: every row starts from the upper bound max_d r'(d) (alpha = 0).
__global__ void __launch_bounds__(256)
saf_fit_init_kernel(FitState s) {
  __shared__ float redm[8];
  const int h = blockIdx.x, tid = threadIdx.x, T = s.T;
  const size_t o = static_cast<size_t>(h) * T;
  float mx = -INFINITY;
  for (int d = tid; d < T; d += 256) {
    const double r = log(fmax(s.eta_rel[o + d] / static_cast<double>(T - d), 1e-9));
    s.rho[o + d] = r;
    s.alpha[o + d] = 0.0;
    s.m_a[o + d] = 0.0; s.v_a[o + d] = 0.0; s.m_r[o + d] = 0.0; s.v_r[o + d] = 0.0;
    const float r2 = static_cast<float>(r * LOG2E_D);
    s.r2[0][o + d] = r2;
    s.a2[0][o + d] = 0.0f;
    mx = fmaxf(mx, r2);
  }
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, k));
  if ((tid & 31) == 0) redm[tid >> 5] = mx;
  __syncthreads();
  mx = redm[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) mx = fmaxf(mx, redm[w]);
  for (int i = tid; i < T; i += 256) s.nz2[o + i] = -mx;
}

// ------------------------------------------------------------------------------------------------ Fit: the passes
// MODE 0 (pass A): x = query i, y = distance d <= i:   u = r', window = a'[i-d],  c = -z'(i)   -> z'(i) += log2 S
// MODE 1 (pass B): blockIdx.z = 0: x = key j, y = d <= T-1-j:  u = r', window = -z'[j+d], c = a'(j) -> Adam on alpha(j)
//                  blockIdx.z = 1: x = d,     y = j <= T-1-d:  u = a', window = -z'[d+j], c = r'(d) -> Adam on rho(d)
// CTA = 32 consecutive x (one per lane) x 8 warps that take the 32-wide chunks of y in turn.  Both operands are
// staged in shared memory, 4096 values of y at a time; window entries outside the causal range are -inf, which is the
// mask.
template <int MODE>
__global__ void __launch_bounds__(PASS_WARPS * 32)
saf_fit_pass_kernel(FitState s, int cur, double bc1, double bc2) {
  extern __shared__ float sm_f[];
  const int T = s.T;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h = blockIdx.y;
  const size_t o = static_cast<size_t>(h) * T;
  const int nxb = (T + XB - 1) / XB;
  // the longest blocks first: pass A's work grows with x, pass B's shrinks
  const int xb = (MODE == 0) ? nxb - 1 - static_cast<int>(blockIdx.x) : static_cast<int>(blockIdx.x);
  const int x0 = xb * XB;
  const int which = (MODE == 0) ? 0 : static_cast<int>(blockIdx.z);
  const int ny = (MODE == 0) ? min(T, x0 + XB) : T - x0;          // y = 0 .. ny-1 covers every lane's range
  const int nyp = (ny + 31) & ~31;
  const int ycap = min(YC, (T + 31) & ~31);
  float* us = sm_f;                       // [ycap]
  float* ws = sm_f + ycap;                // [ycap + 32]
  const float* a2c = cur ? s.a2[1] : s.a2[0];
  const float* r2c = cur ? s.r2[1] : s.r2[0];
  const float* u_g = (MODE == 1 && which == 1) ? a2c + o : r2c + o;
  const float* w_g = (MODE == 0) ? a2c + o : s.nz2 + o;
  const int x = x0 + lane;
  float c = -INFINITY;
  if (x < T) c = (MODE == 0) ? s.nz2[o + x] : (which == 0 ? a2c[o + x] : r2c[o + x]);
  float acc0 = 0.0f, acc1 = 0.0f;
  // the y range in chunks of YC: shared memory per CTA stays at 33 KB whatever T is (six CTAs per SM)
  for (int yb = 0; yb < nyp; yb += YC) {
    const int nyc = min(YC, nyp - yb);                 // a multiple of 32
    if (yb > 0) __syncthreads();                       // the previous chunk has been read
    for (int y = tid; y < nyc; y += PASS_WARPS * 32) us[y] = (yb + y < ny) ? u_g[yb + y] : -INFINITY;
    if (MODE == 0) {
      // lane x at distance y reads a'[x - y]: the chunk's window starts at g0 = x0 - (yb + nyc - 1), and
      // ws[k] = a'[g0 + k] (-inf below index 0); the lane's entry for y is ws[lane + (yb + nyc - 1 - y)]
      const int g0 = x0 - (yb + nyc - 1);
      for (int k = tid; k < nyc + 32; k += PASS_WARPS * 32) {
        const int g = g0 + k;
        ws[k] = (g >= 0 && g < ny) ? w_g[g] : -INFINITY;
      }
    } else {
      // lane x at offset y reads -z'[x + y]: ws[k] = -z'[x0 + yb + k] (-inf beyond T); the lane's entry is
      // ws[lane + (y - yb)]
      for (int k = tid; k < nyc + 32; k += PASS_WARPS * 32) ws[k] = (x0 + yb + k < T) ? w_g[x0 + yb + k] : -INFINITY;
    }
    __syncthreads();
    for (int y0 = warp * 32; y0 < nyc; y0 += PASS_WARPS * 32) {
      const float4* u4 = reinterpret_cast<const float4*>(us + y0);
      const float* wp = (MODE == 0) ? ws + (lane + nyc - 1 - y0) : ws + (lane + y0);
#pragma unroll
      for (int t4 = 0; t4 < 8; ++t4) {
        const float4 u = u4[t4];
        const int t = 4 * t4;
        const float w0 = (MODE == 0) ? wp[-t] : wp[t];
        const float w1 = (MODE == 0) ? wp[-t - 1] : wp[t + 1];
        const float w2 = (MODE == 0) ? wp[-t - 2] : wp[t + 2];
        const float w3 = (MODE == 0) ? wp[-t - 3] : wp[t + 3];
        acc0 += ex2f((u.x + c) + w0);
        acc1 += ex2f((u.y + c) + w1);
        acc0 += ex2f((u.z + c) + w2);
        acc1 += ex2f((u.w + c) + w3);
      }
    }
  }
  __shared__ float red[PASS_WARPS][32];
  red[warp][lane] = acc0 + acc1;
  __syncthreads();
  if (warp != 0 || x >= T) return;
  float S = 0.0f;
#pragma unroll
  for (int w = 0; w < PASS_WARPS; ++w) S += red[w][lane];
  if (MODE == 0) {
    s.nz2[o + x] = c - __log2f(S);
  } else {
    // gradient of Eq. "fit-objective": (fitted marginal - target marginal) / T, then one Adam step in fp64
    const double eta = (which == 0) ? s.eta_abs[o + x] : s.eta_rel[o + x];
    double* par = (which == 0) ? s.alpha : s.rho;
    double* mm = (which == 0) ? s.m_a : s.m_r;
    double* vv = (which == 0) ? s.v_a : s.v_r;
    const double g = (static_cast<double>(S) - eta) / static_cast<double>(T);
    const double m = 0.9 * mm[o + x] + 0.1 * g;
    const double v = 0.999 * vv[o + x] + 0.001 * g * g;
    mm[o + x] = m;
    vv[o + x] = v;
    const double pnew = par[o + x] - s.lr * (m / bc1) / (sqrt(v / bc2) + 1e-8);
    par[o + x] = pnew;
    float* dst = (which == 0) ? (cur ? s.a2[0] : s.a2[1]) : (cur ? s.r2[0] : s.r2[1]);
    dst[o + x] = static_cast<float>(pnew * LOG2E_D);
  }
}

// ------------------------------------------------------------------------------------------------ Fit: results
// One CTA per head, fp64: L = (1/T)[sum_i log Z(i) - eta_abs.alpha - eta_rel.rho], kappa = L + (1/T) sum P log P,
// and the fp32 copies of alpha, rho, log Z that the attention kernels take.
__global__ void __launch_bounds__(256)
saf_fit_final_kernel(FitState s, const double* __restrict__ plogp, float* __restrict__ alpha_out,
                     float* __restrict__ rho_out, float* __restrict__ logZ_out, long long out_stride,
                     double* __restrict__ loss_out, double* __restrict__ kl_out) {
  __shared__ double redd[8];
  const int h = blockIdx.x, tid = threadIdx.x, T = s.T;
  const size_t o = static_cast<size_t>(h) * T;
  const size_t oo = static_cast<size_t>(h) * static_cast<size_t>(out_stride);
  double acc = 0.0;
  for (int k = tid; k < T; k += 256) {
    const double a = s.alpha[o + k], r = s.rho[o + k];
    const double lz = -static_cast<double>(s.nz2[o + k]) * LN2_D;
    acc += lz - s.eta_abs[o + k] * a - s.eta_rel[o + k] * r;
    alpha_out[oo + k] = static_cast<float>(a);
    rho_out[oo + k] = static_cast<float>(r);
    logZ_out[oo + k] = static_cast<float>(lz);
  }
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, k);
  if ((tid & 31) == 0) redd[tid >> 5] = acc;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += redd[w];
    const double loss = t / static_cast<double>(T);
    if (loss_out) loss_out[h] = loss;
    if (kl_out) kl_out[h] = loss + plogp[h] / static_cast<double>(T);
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------------ launchers
int fit_max_T() { return 16384; }

cudaError_t launch_fit_marginals(const float* Abar, float floor_v, double* eta_abs, double* eta_rel, double* plogp,
                                 int Hf, int T, int num_sms, cudaStream_t st) {
  // CTAs per head: one resident wave over all heads, but at least 32 rows each so that the final flush
  // (2T atomics per CTA) stays small beside the rows read
  const size_t smem = static_cast<size_t>(T) * sizeof(float);
#define SAF_MARG(NT, N)                                                                                          \
  do {                                                                                                           \
    auto kern = saf_fit_marginals_kernel<NT, N>;                                                                 \
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,                      \
                                         static_cast<int>(smem));                                                \
    if (e != cudaSuccess) return e;                                                                              \
    int occ = 1;                                                                                                 \
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NT, smem);                                     \
    if (e != cudaSuccess) return e;                                                                              \
    int nb = (std::max(occ, 1) * num_sms) / Hf;             /* one resident wave over all heads */               \
    nb = std::max(1, std::min(nb, (T + 31) / 32));                                                               \
    kern<<<dim3(nb, Hf), NT, smem, st>>>(Abar, floor_v, eta_abs, eta_rel, plogp, T);                             \
  } while (0)
  if (T <= 128 * 2) SAF_MARG(128, 2);
  else if (T <= 256 * 4) SAF_MARG(256, 4);
  else if (T <= 256 * 8) SAF_MARG(256, 8);
  else if (T <= 256 * 16) SAF_MARG(256, 16);
  else if (T <= 256 * 32) SAF_MARG(256, 32);
  else if (T <= 512 * 32) SAF_MARG(512, 32);
  else return cudaErrorInvalidValue;
#undef SAF_MARG
  return cudaGetLastError();
}

cudaError_t launch_fit(const FitState& s, int Hf, int steps, const double* plogp, float* alpha_out, float* rho_out,
                       float* logZ_out, long long out_stride, double* loss_out, double* kl_out, cudaStream_t st) {
  const int T = s.T;
  const int nxb = (T + XB - 1) / XB;
  const size_t smem = (2 * static_cast<size_t>(std::min((T + 31) & ~31, YC)) + 32) * sizeof(float);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(saf_fit_pass_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(smem))) != cudaSuccess)
    return e;
  if ((e = cudaFuncSetAttribute(saf_fit_pass_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(smem))) != cudaSuccess)
    return e;
  saf_fit_init_kernel<<<Hf, 256, 0, st>>>(s);
  int cur = 0;
  double p1 = 1.0, p2 = 1.0;
  for (int t = 1; t <= steps; ++t) {
    p1 *= 0.9;
    p2 *= 0.999;
    saf_fit_pass_kernel<0><<<dim3(nxb, Hf, 1), PASS_WARPS * 32, smem, st>>>(s, cur, 1.0, 1.0);
    saf_fit_pass_kernel<1><<<dim3(nxb, Hf, 2), PASS_WARPS * 32, smem, st>>>(s, cur, 1.0 - p1, 1.0 - p2);
    cur ^= 1;
  }
  saf_fit_pass_kernel<0><<<dim3(nxb, Hf, 1), PASS_WARPS * 32, smem, st>>>(s, cur, 1.0, 1.0);
  saf_fit_final_kernel<<<Hf, 256, 0, st>>>(s, plogp, alpha_out, rho_out, logZ_out, out_stride, loss_out, kl_out);
  return cudaGetLastError();
}

}  // namespace saf
