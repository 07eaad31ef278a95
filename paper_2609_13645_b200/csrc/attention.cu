// Attention pieces that do not run on the tensor cores: the backward pre-pass (delta) and the single-kernel entry point
// that brings its own scratch.  The flash-attention kernels themselves are in attention_tc.cu.
#include "attention.cuh"

#include <math.h>

#include <mutex>

#include "../../include/forgestep.h"

namespace fs {
namespace {

// ============================================================================ backward pre-pass
// delta[b, n, i] = sum_k dO[b,i,n,k] O[b,i,n,k]; one warp per (token, head).
template <int D>
__global__ void attn_delta_kernel(const bf16* __restrict__ o, const bf16* __restrict__ d_o, float* __restrict__ delta,
                                  int B, int S, int n_heads) {
  const long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long total = (long long)B * S * n_heads;
  if (w >= total) return;
  const int n = (int)(w % n_heads);
  const long long tok = w / n_heads;
  const bf16* po = o + (tok * n_heads + n) * D;
  const bf16* pd = d_o + (tok * n_heads + n) * D;
  float acc = 0.f;
#pragma unroll
  for (int c = lane * 2; c < D; c += 64) {
    const uint32_t a = *reinterpret_cast<const uint32_t*>(po + c);
    const uint32_t d = *reinterpret_cast<const uint32_t*>(pd + c);
    acc += bf16_lo(a) * bf16_lo(d) + bf16_hi(a) * bf16_hi(d);
  }
  acc = warp_sum(acc);
  if (lane == 0) {
    const int b = (int)(tok / S), i = (int)(tok % S);
    delta[((long long)b * n_heads + n) * S + i] = acc;
  }
}

}  // namespace

cudaError_t attention_delta(const bf16* o, const bf16* d_o, float* delta, int B, int S, int nh, int d, cudaStream_t st) {
  const long long warps = (long long)B * S * nh;
  const int blocks = (int)((warps * 32 + 255) / 256);
  if (d == 64) attn_delta_kernel<64><<<blocks, 256, 0, st>>>(o, d_o, delta, B, S, nh);
  else if (d == 128) attn_delta_kernel<128><<<blocks, 256, 0, st>>>(o, d_o, delta, B, S, nh);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

}  // namespace fs

// =============================================================================== entry point that allocates nothing
// Scratch for the backward pre-pass (delta = rowsum(dO * O), one float per (batch, head, position)) that lives in the
// library image instead of in caller-provided memory.  4 MiB per GPU that loads the library, held until exit.
namespace {
constexpr long long kStaticDeltaFloats = 1ll << 20;
static __device__ __align__(256) float g_static_delta[kStaticDeltaFloats];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_delta_addr[kMaxDevices] = {nullptr};

// Device address of g_static_delta on the CURRENT device.  In host code the symbol's name is only a handle, not a
// device pointer, so the address is asked for once per device (with that device current) and remembered.
cudaError_t static_delta_ptr(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_delta_addr[dev] == nullptr) {
    float* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_delta);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_static_delta_addr[dev] = p;
  }
  *out = g_static_delta_addr[dev];
  return cudaSuccess;
}
}  // namespace

extern "C" ft_status ft_k_attention_bwd_noalloc(const void* dev_qkv, const void* dev_o, const void* dev_do,
                                                const float* dev_lse, void* dev_dqkv, const float* dev_cos,
                                                const float* dev_sin, int32_t B, int32_t S, int32_t n_heads,
                                                int32_t n_kv_heads, int32_t head_dim, void* stream) {
  if (!dev_qkv || !dev_o || !dev_do || !dev_lse || !dev_dqkv) return FT_EINVAL;
  if (B <= 0 || S <= 0 || n_heads <= 0) return FT_EINVAL;
  if ((long long)B * n_heads * S > kStaticDeltaFloats) return FT_ENOMEM;  // beyond the built-in scratch
  float* delta = nullptr;
  if (static_delta_ptr(&delta) != cudaSuccess) return FT_ECUDA;
  // every element of delta that the two main kernels read is written by the pre-pass of this same call,
  // so nothing has to start at zero
  // same kernels as ft_k_attention_bwd, so the same bits
  int* status = fs::attention_status_word();
  if (!status) return FT_ECUDA;
  cudaError_t e = fs::attention_bwd(reinterpret_cast<const fs::bf16*>(dev_qkv), reinterpret_cast<const fs::bf16*>(dev_o),
                                    reinterpret_cast<const fs::bf16*>(dev_do), dev_lse, delta,
                                    reinterpret_cast<fs::bf16*>(dev_dqkv), dev_cos, dev_sin, B, S, n_heads, n_kv_heads,
                                    head_dim, status, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}
