// Small memory-bound helper kernels: the pattern's row normalisers, the backward's delta / zero-fill
// pass and the fp32 -> bf16 conversion of the accumulated query gradient.
#include <cuda_bf16.h>
#include "saf_internal.h"

namespace saf {

// logZ[h][i] = log sum_{k<=i} exp(alpha[h][k] + rho[h][i-k])   (Eq. "compact-prior", the normaliser Z(i)).
// One warp per row; two passes (row maximum, then the sum of exponentials); lane partials in fp32,
// the 32 partials and the logarithm in fp64.
__global__ void __launch_bounds__(256) saf_logz_kernel(const float* __restrict__ alpha, const float* __restrict__ rho,
                                                       float* __restrict__ logZ, const uint8_t* __restrict__ mask,
                                                       int Tp) {
  const int h = blockIdx.y;
  if (!mask[h]) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // heavy (late) rows first so that the tail of the grid is cheap
  const int i = Tp - 1 - (blockIdx.x * 8 + warp);
  if (i < 0) return;
  const float* a = alpha + static_cast<size_t>(h) * Tp;
  const float* r = rho + static_cast<size_t>(h) * Tp;
  float m = -INFINITY;
  for (int k = lane; k <= i; k += 32) m = fmaxf(m, a[k] + r[i - k]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float s0 = 0.0f, s1 = 0.0f;
  int k = lane;
  for (; k + 32 <= i; k += 64) {
    s0 += __expf(a[k] + r[i - k] - m);
    s1 += __expf(a[k + 32] + r[i - k - 32] - m);
  }
  if (k <= i) s0 += __expf(a[k] + r[i - k] - m);
  double s = static_cast<double>(s0) + static_cast<double>(s1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) logZ[static_cast<size_t>(h) * Tp + i] = static_cast<float>(static_cast<double>(m) + log(s));
}

cudaError_t launch_logz(const float* alpha, const float* rho, float* logZ, const uint8_t* mask_dev, int H, int Tp,
                        cudaStream_t st) {
  dim3 grid((Tp + 7) / 8, H);
  saf_logz_kernel<<<grid, 256, 0, st>>>(alpha, rho, logZ, mask_dev, Tp);
  return cudaGetLastError();
}

// Backward preparation.  Eight threads per (b,h,row) with D = 64 (sixteen with D = 128), each owning
// eight consecutive features:
//   ordinary head: delta[b][h][row] = sum_c dO*O  (the row term of the softmax Jacobian)
//   every head   : dQacc row = 0 (it is accumulated atomically by the main kernel)
//   frozen head  : dK row = 0 (no key gradient; Sec. 3.3)
template <int D>
__global__ void __launch_bounds__(256) saf_bwd_prep_kernel(const __nv_bfloat16* __restrict__ O,
                                                           const __nv_bfloat16* __restrict__ dO, int64_t os0, int64_t os1,
                                                           int64_t os2, const uint8_t* __restrict__ mask,
                                                           float* __restrict__ delta, int Tpad, float* __restrict__ dQacc,
                                                           void* __restrict__ dK, int grad_f32, int B, int H, int T) {
  constexpr int TPR = D / 8;                       // threads per row
  const long long gid = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long rowid = gid / TPR;
  const int part = static_cast<int>(gid % TPR);
  const long long nrows = static_cast<long long>(B) * H * T;
  const bool valid = rowid < nrows;
  float acc = 0.0f;
  int b = 0, h = 0, t = 0;
  bool frozen = false;
  if (valid) {
    t = static_cast<int>(rowid % T);
    h = static_cast<int>((rowid / T) % H);
    b = static_cast<int>(rowid / (static_cast<long long>(T) * H));
    frozen = mask[h] != 0;
    const size_t grow = static_cast<size_t>(rowid) * D + part * 8;
    float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<float4*>(dQacc + grow) = z;
    *reinterpret_cast<float4*>(dQacc + grow + 4) = z;
    if (frozen) {
      if (grad_f32) {
        *reinterpret_cast<float4*>(static_cast<float*>(dK) + grow) = z;
        *reinterpret_cast<float4*>(static_cast<float*>(dK) + grow + 4) = z;
      } else {
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dK) + grow) = make_uint4(0, 0, 0, 0);
      }
    } else {
      const int64_t off = b * os0 + h * os1 + static_cast<int64_t>(t) * os2 + part * 8;
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
  }
#pragma unroll
  for (int o = TPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (valid && part == 0 && !frozen) delta[(static_cast<size_t>(b) * H + h) * Tpad + t] = acc;
}

cudaError_t launch_bwd_prep(const void* O, const void* dO, const int64_t* os, const uint8_t* mask_dev, float* delta,
                            int Tpad, float* dQacc, void* dK, int grad_f32, int B, int H, int T, int D,
                            cudaStream_t st) {
  const long long nthreads = static_cast<long long>(B) * H * T * (D / 8);
  const unsigned grid = static_cast<unsigned>((nthreads + 255) / 256);
  if (D == 64)
    saf_bwd_prep_kernel<64><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(O),
                                                  static_cast<const __nv_bfloat16*>(dO), os[0], os[1], os[2], mask_dev,
                                                  delta, Tpad, dQacc, dK, grad_f32, B, H, T);
  else
    saf_bwd_prep_kernel<128><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(O),
                                                   static_cast<const __nv_bfloat16*>(dO), os[0], os[1], os[2], mask_dev,
                                                   delta, Tpad, dQacc, dK, grad_f32, B, H, T);
  return cudaGetLastError();
}

__global__ void __launch_bounds__(256) saf_f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst,
                                                              size_t n8) {
  const size_t i = static_cast<size_t>(blockIdx.x) * 256 + threadIdx.x;
  if (i >= n8) return;
  const float4 a = *reinterpret_cast<const float4*>(src + i * 8);
  const float4 b = *reinterpret_cast<const float4*>(src + i * 8 + 4);
  __nv_bfloat162 r[4];
  r[0] = __floats2bfloat162_rn(a.x, a.y);
  r[1] = __floats2bfloat162_rn(a.z, a.w);
  r[2] = __floats2bfloat162_rn(b.x, b.y);
  r[3] = __floats2bfloat162_rn(b.z, b.w);
  *reinterpret_cast<uint4*>(dst + i * 8) = *reinterpret_cast<uint4*>(r);
}

cudaError_t launch_bwd_finalize(const float* dQacc, void* dQ, size_t n, cudaStream_t st) {
  const size_t n8 = n / 8;
  saf_f32_to_bf16_kernel<<<static_cast<unsigned>((n8 + 255) / 256), 256, 0, st>>>(
      dQacc, static_cast<__nv_bfloat16*>(dQ), n8);
  return cudaGetLastError();
}

}  // namespace saf
