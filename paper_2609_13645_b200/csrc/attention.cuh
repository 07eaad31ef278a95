// Host-side interface of the causal flash-attention kernels (tcgen05 tensor cores, accumulators in TMEM, TMA loads).
#pragma once
#include <cuda_runtime.h>

#include "common.cuh"

namespace fs {

// qkv bf16 [B*S, (n_h + 2 n_kv) d] packed q heads | k heads | v heads (q, k rotated); o bf16 [B*S, n_h d];
// lse fp32 [B, n_h, S] in natural log.  d in {64, 128}.  err: device status word.  One kernel launch.
cudaError_t attention_fwd(const bf16* qkv, bf16* o, float* lse, int B, int S, int n_heads, int n_kv, int d, int* err,
                          cudaStream_t st);

// Three kernel launches (delta pre-pass, dQ, dK/dV).  delta: fp32 scratch [B, n_h, S].  dqkv has qkv's layout.
// cos/sin: fp32 [S, d/2] or both null (then dq, dk are left in the rotated frame).
cudaError_t attention_bwd(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                          const float* cos, const float* sin, int B, int S, int n_heads, int n_kv, int d, int* err,
                          cudaStream_t st);

// The same with a scratch array for dS^T (B n_h S^2 bf16 in 32-query chunks, attention_bwd_ds_bytes() bytes, 128-byte aligned): the
// dK/dV kernel leaves its rounded dS tiles there and dQ becomes one causally truncated batched contraction over them
// (delta pre-pass, dK/dV, dQ: three launches, five tile products per block pair instead of seven).  Needs S % 128 == 0;
// with ds == nullptr, too small a scratch or another S this is attention_bwd().
size_t attention_bwd_ds_bytes(int B, int S, int n_heads);
cudaError_t attention_bwd_ws(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                             const float* cos, const float* sin, bf16* ds, size_t ds_bytes, int B, int S, int n_heads,
                             int n_kv, int d, int* err, cudaStream_t st);

// dQ from stored dS^T (the last launch of attention_bwd_ws).
cudaError_t attention_dq_from_ds(const bf16* ds, const bf16* qkv, bf16* dqkv, const float* cos, const float* sin, int B, int S,
                                 int n_heads, int n_kv, int d, int* err, cudaStream_t st);

// delta[b, n, i] = sum_k dO[b,i,n,k] O[b,i,n,k] (the backward pre-pass; one launch)
cudaError_t attention_delta(const bf16* o, const bf16* d_o, float* delta, int B, int S, int n_heads, int d, cudaStream_t st);

// Device status word used by the single-kernel entry points (address on the current device).
int* attention_status_word();

}  // namespace fs
