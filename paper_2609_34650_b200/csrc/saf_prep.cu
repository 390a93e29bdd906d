// Small memory-bound helper kernels: the pattern's row normalisers, the backward's delta / zero-fill
// pass and the fp32 -> bf16 conversion of the accumulated query gradient.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cstring>
#include <mutex>

#include "../../include/saf.h"
#include "ptx.cuh"
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

// ------------------------------------------------------------------------------------------------
// Tables of the tensor-core form of a frozen head.  With c_a = max alpha, c_r = max rho,
//   a(j) = exp(alpha(j) - c_a),  r(d) = exp(rho(d) - c_r),  w(i) = exp(c_a + c_r - logZ(i)),
// Eq. "compact-prior" reads  P^(i,j) = w(i) r(i-j) a(j):  O = diag(w) R (diag(a) V) with the Toeplitz
// matrix R(i,j) = r(i-j) [j <= i], and dV = diag(a) R^T (diag(w) dO).  A 128x128 tile of R (or R^T)
// with its rows in reverse order is a Hankel matrix g[m + k]; stored as 31 overlapping 8x8 core
// matrices (chunk c, row ri, element e = g[8c + ri + e], 128 bytes per chunk) it is a valid no-swizzle
// K-major UMMA operand with both descriptor strides equal to 128 bytes, so the tensor core reads the
// pattern tile straight from a 4 KB band of the relative-distance vector.
//   band_f[h][D][x] : g[x] = r(128 D + 127 - x)   (forward,  rows = queries reversed)
//   band_b[h][D][x] : g[x] = r(128 D - 127 + x)   (backward, rows = keys reversed)
// The band and the scaled V / dO tiles are fp16 (the tensor core needs one 16-bit type for both operands;
// fp16 keeps 11 significant bits, so the form adds less rounding than the bf16 pattern tile of the
// general path).  To use fp16's range, the bands hold 2^14 r and the forward stages 2^11 a V; the
// epilogues undo the powers of two.  A value below fp16's normal range is then off by at most 2^-25 in
// scaled units, i.e. the pattern entry w a r by at most w 2^-39: the form is used for a head only if
// max_i (c_a + c_r - logZ(i)) <= 9 (fast_ok), which keeps that below 1e-8 and leaves w dO room in fp16
// (the scaling kernel checks the staged values against fp16's range on every call).
__global__ void __launch_bounds__(256) saf_pattern_consts_kernel(const float* __restrict__ alpha,
                                                                 const float* __restrict__ rho,
                                                                 const float* __restrict__ logZ,
                                                                 const uint8_t* __restrict__ mask, int Tp,
                                                                 float* __restrict__ consts, int* __restrict__ fast_ok) {
  const int h = blockIdx.x;
  if (!mask[h]) {
    if (threadIdx.x == 0) fast_ok[h] = 0;
    return;
  }
  __shared__ float red[3][8];
  const float* a = alpha + static_cast<size_t>(h) * Tp;
  const float* r = rho + static_cast<size_t>(h) * Tp;
  const float* z = logZ + static_cast<size_t>(h) * Tp;
  float ma = -INFINITY, mr = -INFINITY, mz = INFINITY;
  for (int t = threadIdx.x; t < Tp; t += 256) {
    ma = fmaxf(ma, a[t]);
    mr = fmaxf(mr, r[t]);
    mz = fminf(mz, z[t]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ma = fmaxf(ma, __shfl_xor_sync(0xffffffffu, ma, o));
    mr = fmaxf(mr, __shfl_xor_sync(0xffffffffu, mr, o));
    mz = fminf(mz, __shfl_xor_sync(0xffffffffu, mz, o));
  }
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
    red[0][warp] = ma;
    red[1][warp] = mr;
    red[2][warp] = mz;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < 8; ++k) {
      ma = fmaxf(ma, red[0][k]);
      mr = fmaxf(mr, red[1][k]);
      mz = fminf(mz, red[2][k]);
    }
    consts[2 * h] = ma;
    consts[2 * h + 1] = mr;
    const float wmax = ma + mr - mz;
    fast_ok[h] = (wmax <= 9.0f && wmax > -1e30f && ma < 1e30f && mr < 1e30f) ? 1 : 0;
  }
}

__global__ void __launch_bounds__(256) saf_pattern_tables_kernel(const float* __restrict__ alpha,
                                                                 const float* __restrict__ rho,
                                                                 const float* __restrict__ logZ,
                                                                 const uint8_t* __restrict__ mask, int Tp,
                                                                 const float* __restrict__ consts,
                                                                 float* __restrict__ avec, float* __restrict__ wvec,
                                                                 __half* __restrict__ band_f,
                                                                 __half* __restrict__ band_b, int nblkp) {
  const int h = blockIdx.y, dblk = blockIdx.x;
  if (!mask[h]) return;
  const float ca = consts[2 * h], cr = consts[2 * h + 1];
  const size_t row = static_cast<size_t>(h) * Tp;
  const int t = dblk * 128 + threadIdx.x;
  if (threadIdx.x < 128 && t < Tp) {
    avec[row + t] = __expf(alpha[row + t] - ca);
    wvec[row + t] = __expf(ca + cr - logZ[row + t]);
  }
  const size_t band = (static_cast<size_t>(h) * nblkp + dblk) * 2048;
  for (int idx = threadIdx.x; idx < 2048; idx += 256) {
    const int c = idx >> 6, ri = (idx >> 3) & 7, e = idx & 7;
    const int x = 8 * c + ri + e;
    const int df = dblk * 128 + 127 - x, db = dblk * 128 - 127 + x;
    const bool used = c < 31;
    const float vf = (used && df >= 0 && df < Tp) ? 16384.0f * __expf(rho[row + df] - cr) : 0.0f;
    const float vb = (used && db >= 0 && db < Tp) ? 16384.0f * __expf(rho[row + db] - cr) : 0.0f;
    band_f[band + idx] = __float2half_rn(vf);
    band_b[band + idx] = __float2half_rn(vb);
  }
}

cudaError_t launch_pattern_tables(const float* alpha, const float* rho, const float* logZ, const uint8_t* mask_dev, int H,
                                  int Tp, float* consts, int* fast_ok, float* avec, float* wvec, void* band_f,
                                  void* band_b, cudaStream_t st) {
  const int nblkp = (Tp + 127) / 128;
  saf_pattern_consts_kernel<<<H, 256, 0, st>>>(alpha, rho, logZ, mask_dev, Tp, consts, fast_ok);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  saf_pattern_tables_kernel<<<dim3(nblkp, H), 256, 0, st>>>(alpha, rho, logZ, mask_dev, Tp, consts, avec, wvec,
                                                            static_cast<__half*>(band_f),
                                                            static_cast<__half*>(band_b), nblkp);
  return cudaGetLastError();
}

// dst[b][ord][t][:] = fp16(extra * vec[h][t] * src[b][h][t][:]), h = hlist[ord], for the frozen heads whose tensor-core form is
// enabled (V scaled by a, or dO scaled by w).  Eight features per thread.  A product that leaves fp16's range
// marks the head (ovf[h] = call_id), which sends it down the general path in the kernel that follows; the
// mark of an earlier call has another id and needs no reset.  The same mark is raised when alpha, rho or logZ of the
// head no longer hold the bits the tables were built from (another call may have rewritten the vectors in place):
// the threads of batch entry 0 compare their row's three values with the snapshot taken at preparation.
__device__ __forceinline__ bool pattern_row_changed(const PatternCheck& c, size_t i) {
  const size_t n = c.vec_elems;
  return __float_as_uint(c.alpha[i]) != c.snap[i] || __float_as_uint(c.rho[i]) != c.snap[n + i] ||
         __float_as_uint(c.logZ[i]) != c.snap[2 * n + i];
}

template <int D>
__global__ void __launch_bounds__(256) saf_scale_rows_kernel(const __nv_bfloat16* __restrict__ src, int64_t s0, int64_t s1,
                                                             int64_t s2, const float* __restrict__ vec, float extra,
                                                             int Tp, const int* __restrict__ hlist,
                                                             const int* __restrict__ pat_ok, int* __restrict__ ovf,
                                                             int call_id, __half* __restrict__ dst, int B, int Hf,
                                                             int T, int src_group, const PatternCheck chk) {
  constexpr int TPR = D / 8;
  pdl_launch_dependents();
  pdl_wait();                                      // (launched with programmatic stream serialization)
  const long long gid = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long rowid = gid / TPR;               // over [B][Hf][T]: frozen heads only
  const int part = static_cast<int>(gid % TPR);
  if (rowid >= static_cast<long long>(B) * Hf * T) return;
  const int t = static_cast<int>(rowid % T);
  const int ord = static_cast<int>((rowid / T) % Hf);
  const int b = static_cast<int>(rowid / (static_cast<long long>(T) * Hf));
  const int h = hlist[ord];
  if (!pat_ok[h]) return;
  const float f = vec[static_cast<size_t>(h) * Tp + t] * extra;
  const uint4 v4 =
      *reinterpret_cast<const uint4*>(src + b * s0 + (h / src_group) * s1 + static_cast<int64_t>(t) * s2 + part * 8);
  const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&v4);
  __half2 o[4];
  bool bad = false;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 x = __bfloat1622float2(v2[e]);
    const float y0 = x.x * f, y1 = x.y * f;
    bad |= !(fabsf(y0) <= 65504.0f) || !(fabsf(y1) <= 65504.0f);     // also catches NaN
    o[e] = __floats2half2_rn(y0, y1);
  }
  if (b == 0 && part == 0) bad |= pattern_row_changed(chk, static_cast<size_t>(h) * Tp + t);
  if (bad) ovf[h] = call_id;
  *reinterpret_cast<uint4*>(dst + (static_cast<size_t>(rowid)) * D + part * 8) = *reinterpret_cast<uint4*>(o);
}

cudaError_t launch_scale_rows(const void* src, const int64_t* strides, const float* vec, float extra, int Tp,
                              const int* hlist, const int* pat_ok, int* ovf, int call_id, void* dst, int B, int Hf,
                              int T, int D, int src_group, const PatternCheck& chk, cudaStream_t st) {
  const long long nthreads = static_cast<long long>(B) * Hf * T * (D / 8);
  const unsigned grid = static_cast<unsigned>((nthreads + 255) / 256);
  cudaError_t e;
  if (D == 96)
    e = launch_pdl(PDL_STAGE, saf_scale_rows_kernel<96>, dim3(grid), dim3(256), 0, st, static_cast<const __nv_bfloat16*>(src), strides[0], strides[1],
                                                    strides[2], vec, extra, Tp, hlist, pat_ok, ovf, call_id,
                                                    static_cast<__half*>(dst), B, Hf, T, src_group, chk);
  else if (D == 64)
    e = launch_pdl(PDL_STAGE, saf_scale_rows_kernel<64>, dim3(grid), dim3(256), 0, st, static_cast<const __nv_bfloat16*>(src), strides[0], strides[1],
                                                    strides[2], vec, extra, Tp, hlist, pat_ok, ovf, call_id,
                                                    static_cast<__half*>(dst), B, Hf, T, src_group, chk);
  else
    e = launch_pdl(PDL_STAGE, saf_scale_rows_kernel<128>, dim3(grid), dim3(256), 0, st, static_cast<const __nv_bfloat16*>(src), strides[0], strides[1],
                                                     strides[2], vec, extra, Tp, hlist, pat_ok, ovf, call_id,
                                                     static_cast<__half*>(dst), B, Hf, T, src_group, chk);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Three-way bf16 split of an fp32 value: hi + mid + lo reproduces x to ~24 bits.
__device__ __forceinline__ uint4 split3_bf16(float x) {
  const __nv_bfloat16 hi = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
  uint4 v = make_uint4(0, 0, 0, 0);
  v.x = static_cast<uint32_t>(__bfloat16_as_ushort(hi)) | (static_cast<uint32_t>(__bfloat16_as_ushort(mid)) << 16);
  v.y = static_cast<uint32_t>(__bfloat16_as_ushort(lo));
  return v;
}

// Backward preparation.  Eight threads per (b,h,row) with D = 64 (sixteen with D = 128), each owning
// eight consecutive features; rows run to a multiple of 128 so that the row-term images are complete:
//   ordinary head: delta = sum_c dO*O (the row term of the softmax Jacobian);
//                  q_ext row  = split3(-LSE/scale)  (so that S - LSE/scale comes out of the score MMA),
//                  do_ext row = split3(-delta)      (so that dP - delta comes out of the dP MMA);
//                  rows beyond T: q_ext = most negative bf16 (their probabilities become 0), do_ext = 0
//   every head   : dQacc row = 0 (it is accumulated by reduce-adds of the main kernel)
//   frozen head  : dK row = 0 (no key gradient; Sec. 3.3); with the tensor-core form, the row w(i) dO in fp16
// Image layout per 128-row block (4 KB): byte (n/8)*256 + (k/8)*128 + (n%8)*16 + (k%8)*2 for row n, column k < 16.
// (TPR threads per row: D / 8, or 16 with four idle ones at D = 96 so that a row stays inside a warp)
// (OF32: O is fp32 instead of bf16, same element strides)
template <int D, int TPR, bool OF32>
__global__ void __launch_bounds__(256, 8) saf_bwd_prep_kernel(const void* __restrict__ O,
                                                           const __nv_bfloat16* __restrict__ dO,
                                                           const float* __restrict__ LSE, int64_t os0, int64_t os1,
                                                           int64_t os2, const uint8_t* __restrict__ mask,
                                                           uint8_t* __restrict__ q_ext, uint8_t* __restrict__ do_ext,
                                                           float inv_scale, float* __restrict__ dQacc,
                                                           void* __restrict__ dK, void* __restrict__ dV,
                                                           int grad_f32, int kv_group,
                                                           const int* __restrict__ qslot, int n_ord,
                                                           const PrepFrozen fz, int B, int H, int T) {
  const int Tpad = (T + 127) / 128 * 128;
  pdl_launch_dependents();
  pdl_wait();                                      // (launched with programmatic stream serialization)
  const long long gid = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  const long long rowid = gid / TPR;               // over [B][H][Tpad]
  const int part = static_cast<int>(gid % TPR);
  const long long nrows = static_cast<long long>(B) * H * Tpad;
  const bool inrange = rowid < nrows;
  float acc = 0.0f;
  int b = 0, h = 0, t = 0;
  bool frozen = false, valid = false;
  if (inrange) {
    t = static_cast<int>(rowid % Tpad);
    h = static_cast<int>((rowid / Tpad) % H);
    b = static_cast<int>(rowid / (static_cast<long long>(Tpad) * H));
    frozen = mask[h] != 0;
    valid = t < T;
  }
  if (valid && part * 8 < D) {
    const size_t grow = ((static_cast<size_t>(b) * H + h) * T + t) * D + part * 8;
    float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
    if (qslot == nullptr) {
      *reinterpret_cast<float4*>(dQacc + grow) = z;
      *reinterpret_cast<float4*>(dQacc + grow + 4) = z;
    } else if (!frozen) {
      // packed layout: dQ has the ordinary heads only
      const size_t prow = ((static_cast<size_t>(b) * n_ord + qslot[h]) * T + t) * D + part * 8;
      *reinterpret_cast<float4*>(dQacc + prow) = z;
      *reinterpret_cast<float4*>(dQacc + prow + 4) = z;
    }
    if (kv_group > 1 && h % kv_group == 0) {
      // grouped-query path: the shared heads' gradients are accumulated by reduce-adds of the main kernel
      const size_t krow = ((static_cast<size_t>(b) * (H / kv_group) + h / kv_group) * T + t) * D + part * 8;
      *reinterpret_cast<float4*>(static_cast<float*>(dK) + krow) = z;
      *reinterpret_cast<float4*>(static_cast<float*>(dK) + krow + 4) = z;
      *reinterpret_cast<float4*>(static_cast<float*>(dV) + krow) = z;
      *reinterpret_cast<float4*>(static_cast<float*>(dV) + krow + 4) = z;
    }
    if (frozen) {
      if (kv_group > 1 || qslot != nullptr) {
        // nothing to zero per frozen head (shared heads are zeroed above; the packed dK has no such row)
      } else if (grad_f32) {
        *reinterpret_cast<float4*>(static_cast<float*>(dK) + grow) = z;
        *reinterpret_cast<float4*>(static_cast<float*>(dK) + grow + 4) = z;
      } else {
        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dK) + grow) = make_uint4(0, 0, 0, 0);
      }
      if (fz.dot_dst != nullptr && fz.pat_ok[h] != 0) {
        const float f = fz.wvec[static_cast<size_t>(h) * fz.Tp + t];
        const uint4 d4 =
            *reinterpret_cast<const uint4*>(dO + b * os0 + h * os1 + static_cast<int64_t>(t) * os2 + part * 8);
        const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&d4);
        __half2 o[4];
        bool bad = false;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 x = __bfloat1622float2(d2[e]);
          const float y0 = x.x * f, y1 = x.y * f;
          bad |= !(fabsf(y0) <= 65504.0f) || !(fabsf(y1) <= 65504.0f);     // also catches NaN
          o[e] = __floats2half2_rn(y0, y1);
        }
        if (b == 0 && part == 0) bad |= pattern_row_changed(fz.chk, static_cast<size_t>(h) * fz.Tp + t);
        if (bad) fz.ovf[h] = fz.call_id;
        const size_t drow = (static_cast<size_t>(b) * fz.Hf + fz.hord[h]) * T + t;
        *reinterpret_cast<uint4*>(static_cast<__half*>(fz.dot_dst) + drow * D + part * 8) =
            *reinterpret_cast<uint4*>(o);
      }
    } else {
      const int64_t off = b * os0 + h * os1 + static_cast<int64_t>(t) * os2 + part * 8;
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
  if (inrange && part == 0 && !frozen) {
    const size_t bh = static_cast<size_t>(b) * H + h;
    const size_t img = (bh * (Tpad / 128) + t / 128) * 4096 + ((t % 128) / 8) * 256 + (t % 8) * 16;
    uint4 qv, dv;
    if (valid) {
      qv = split3_bf16(-LSE[bh * T + t] * inv_scale);
      dv = split3_bf16(-acc);
    } else {
      qv = make_uint4(0xFF7Fu, 0, 0, 0);           // bf16 0xFF7F = -3.39e38
      dv = make_uint4(0, 0, 0, 0);
    }
    const uint4 zero = make_uint4(0, 0, 0, 0);
    *reinterpret_cast<uint4*>(q_ext + img) = qv;
    *reinterpret_cast<uint4*>(q_ext + img + 128) = zero;
    *reinterpret_cast<uint4*>(do_ext + img) = dv;
    *reinterpret_cast<uint4*>(do_ext + img + 128) = zero;
  }
}

cudaError_t launch_bwd_prep(const void* O, int o_f32, const void* dO, const float* LSE, const int64_t* os,
                            const uint8_t* mask_dev, void* q_ext, void* do_ext, float inv_scale, float* dQacc, void* dK,
                            void* dV, int grad_f32, int kv_group, const int* qslot, int n_ord, const PrepFrozen& fz, int B,
                            int H, int T, int D, cudaStream_t st) {
  const int Tpad = (T + 127) / 128 * 128;
  const int tpr = D == 96 ? 16 : D / 8;
  const long long nthreads = static_cast<long long>(B) * H * Tpad * tpr;
  const unsigned grid = static_cast<unsigned>((nthreads + 255) / 256);
#define SAF_PREP_ARGS                                                                                                  \
  O, static_cast<const __nv_bfloat16*>(dO), LSE, os[0], os[1], os[2], mask_dev, static_cast<uint8_t*>(q_ext),          \
      static_cast<uint8_t*>(do_ext), inv_scale, dQacc, dK, dV, grad_f32, kv_group, qslot, n_ord, fz, B, H, T
#define SAF_PREP_LAUNCH(DD, TT, FF) \
  launch_pdl(PDL_PREP, saf_bwd_prep_kernel<DD, TT, FF>, dim3(grid), dim3(256), 0, st, SAF_PREP_ARGS)
  cudaError_t e;
  if (D == 64) e = o_f32 ? SAF_PREP_LAUNCH(64, 8, true) : SAF_PREP_LAUNCH(64, 8, false);
  else if (D == 96) e = o_f32 ? SAF_PREP_LAUNCH(96, 16, true) : SAF_PREP_LAUNCH(96, 16, false);
  else e = o_f32 ? SAF_PREP_LAUNCH(128, 16, true) : SAF_PREP_LAUNCH(128, 16, false);
#undef SAF_PREP_LAUNCH
#undef SAF_PREP_ARGS
  return e != cudaSuccess ? e : cudaGetLastError();
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

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the normaliser computation.
//
// saf_logz_kernel needs the frozen-head mask in device memory.  saf_pattern_prepare keeps that copy in
// memory it allocates through the context; here it lives in a fixed array that is part of the library
// image, so the call path contains no allocation at all.  Every GPU that loads the library carries
// these SAF_STATIC_MAX_HEADS bytes until the process exits.
namespace {

static __device__ __align__(256) uint8_t g_static_mask_scratch[SAF_STATIC_MAX_HEADS];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
uint8_t* g_static_mask_ptr[kMaxDevices] = {};   // device address of the array, per device, resolved once
// The caller's mask is copied here first (under the mutex) and uploaded from here: the upload then never reads the
// caller's array after the call has returned, whatever kind of host memory that array lives in.
uint8_t g_static_mask_host[SAF_STATIC_MAX_HEADS];

}  // namespace

extern "C" int saf_pattern_logz_static(int32_t device, int32_t H, int32_t Tp, const uint8_t* frozen_mask_host,
                                       const float* alpha_dev, const float* rho_dev, float* logZ_dev_out,
                                       void* stream) {
  if (device < 0 || device >= kMaxDevices || H < 1 || Tp < 1 || !frozen_mask_host) return SAF_ERR_INVALID_ARG;
  if (H > SAF_STATIC_MAX_HEADS) return SAF_ERR_INVALID_ARG;   // beyond the built-in scratch: use saf_pattern_prepare
  int nf = 0;
  for (int h = 0; h < H; ++h) nf += frozen_mask_host[h] ? 1 : 0;
  if (nf == 0) return SAF_OK;
  if (!alpha_dev || !rho_dev || !logZ_dev_out) return SAF_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return SAF_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return SAF_ERR_CUDA;
  int rc = SAF_OK;
  uint8_t* scratch = nullptr;
  {
    // In host code the array's name is only a handle; the address a kernel can use has to be asked
    // for, once per device, with that device current.
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_mask_ptr[device]) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_mask_scratch) != cudaSuccess || !ptr) {
        cudaGetLastError();
        rc = SAF_ERR_CUDA;
      } else {
        g_static_mask_ptr[device] = static_cast<uint8_t*>(ptr);
      }
    }
    scratch = g_static_mask_ptr[device];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (rc == SAF_OK) {
    // The array keeps whatever the previous call left; the first H bytes are all this call reads,
    // and they are overwritten here.
    std::lock_guard<std::mutex> lock(g_static_mutex);
    std::memcpy(g_static_mask_host, frozen_mask_host, static_cast<size_t>(H));
    // (pageable source: the runtime stages the bytes before this call returns)
    if (cudaMemcpyAsync(scratch, g_static_mask_host, static_cast<size_t>(H), cudaMemcpyHostToDevice, st) != cudaSuccess)
      rc = SAF_ERR_CUDA;
  }
  if (rc == SAF_OK && saf::launch_logz(alpha_dev, rho_dev, logZ_dev_out, scratch, H, Tp, st) != cudaSuccess)
    rc = SAF_ERR_CUDA;
  if (prev != device) cudaSetDevice(prev);
  return rc;
}

