// Internal declarations shared by the host API and the sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

namespace saf {

constexpr int BLK = 128;            // query rows per item and keys per tile
constexpr int KIND_ORDINARY = 0;
constexpr int KIND_FROZEN = 1;

struct WorkItem { int32_t b, h, blk, kind; };

struct FwdParams {
  int B, H, T, Tp;
  float scale_log2;                 // softmax_scale * log2(e)
  const float* alpha;               // [H][Tp]
  const float* rho;                 // [H][Tp]
  const float* logZ;                // [H][Tp]
  void* O;                          // bf16, strided
  int64_t o_strides[3];             // elements: batch, head, seq
  float* LSE;                       // [B][H][T]
  const WorkItem* items;            // grouped by CTA
  const int* cta_offsets;           // [grid+1]
  int* status;                      // device status word
  unsigned long long wait_limit_ns;
};

struct BwdParams {
  int B, H, T, Tp;
  float scale, scale_log2;
  const float* alpha;
  const float* rho;
  const float* logZ;
  const float* LSE;                 // [B][H][T]
  const float* delta;               // [B][H][Tpad] workspace, rowsum(dO o O) for ordinary heads
  int Tpad;
  float* dQacc;                     // fp32 [B][H][T][D], zeroed before the launch (atomically accumulated)
  void* dK;                         // [B][H][T][D] grad dtype
  void* dV;
  int grad_f32;
  const WorkItem* items;
  const int* cta_offsets;
  int* status;
  unsigned long long wait_limit_ns;
};

// Launchers (defined in the .cu files).  All return the launch error.
cudaError_t launch_logz(const float* alpha, const float* rho, float* logZ, const uint8_t* mask_dev, int H,
                        int Tp, cudaStream_t st);
cudaError_t launch_fwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const FwdParams& p, int grid, cudaStream_t st);
cudaError_t launch_bwd(int D, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                       const CUtensorMap& mdo, const BwdParams& p, int grid, cudaStream_t st);
// delta = rowsum(dO o O) for ordinary heads; also zeroes dQacc (all heads) and dK of frozen heads.
cudaError_t launch_bwd_prep(const void* O, const void* dO, const int64_t* o_strides, const uint8_t* mask_dev,
                            float* delta, int Tpad, float* dQacc, void* dK, int grad_f32, int B, int H, int T,
                            int D, cudaStream_t st);
// dQ (grad dtype) = scale-free copy/convert of dQacc (fp32) for the bf16-gradient case.
cudaError_t launch_bwd_finalize(const float* dQacc, void* dQ, size_t n, cudaStream_t st);
int fwd_smem_bytes(int D);
int bwd_smem_bytes(int D);

}  // namespace saf
