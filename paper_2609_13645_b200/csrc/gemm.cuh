// Host-side interface of the tcgen05 GEMM family.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace fs {

enum GemmEpilogue : int {
  EPI_BF16 = 0,        // C bf16 = R(acc)
  EPI_BF16_RESID = 1,  // C bf16 = R(resid + acc), resid bf16 with C's shape and row stride
  EPI_F32 = 2,         // C fp32 = acc
  EPI_F32_ACC = 3,     // C fp32 += acc
  EPI_ROPE = 4,        // C bf16 = R(rope(acc)) for columns < rope_cols (heads of head_dim columns), R(acc) beyond
  EPI_SWIGLU = 5       // acc columns alternate 16 gate / 16 up: writes gate|up to gu bf16 [M, 2f] and a = R(silu(G) U) to C [M, f]
};

struct GemmArgs {
  const bf16* A = nullptr;  // a_mn = 0: [M, lda] row-major (k contiguous); a_mn = 1: [K, lda] row-major (m contiguous)
  int a_mn = 0;
  int64_t lda = 0;
  const bf16* B = nullptr;  // b_mn = 0: [N, ldb]; b_mn = 1: [K, ldb]
  int b_mn = 0;
  int64_t ldb = 0;
  void* C = nullptr;
  int64_t ldc = 0;
  const bf16* resid = nullptr;
  int epi = EPI_BF16;
  int M = 0, N = 0, K = 0;
  // EPI_ROPE
  const float* rope_cos = nullptr;  // fp32 [seq, head_dim/2]
  const float* rope_sin = nullptr;
  int seq = 1, head_dim = 64, rope_cols = 0;
  // EPI_SWIGLU
  bf16* gu = nullptr;  // [M, 2f] gate | up
  int d_ffn = 0;
  int* err = nullptr;  // device status word
  // Optional fp32 scratch for split-K: weight-gradient GEMMs with few output tiles split their (long) contraction over
  // several CTA pairs, write partial tiles here and add them in a fixed order.  Unused when null or too small.
  float* splitk_scratch = nullptr;
  size_t splitk_bytes = 0;
};

// Enqueues the contraction on `stream`.  Returns cudaErrorInvalidValue for shapes it does not take.
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t stream);

extern int g_gemm_force_bn;
extern int g_gemm_pairs;

}  // namespace fs
