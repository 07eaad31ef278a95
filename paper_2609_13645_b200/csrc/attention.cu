// Attention pieces that do not run on the tensor cores: the backward pre-pass (delta) and the single-kernel entry point
// that brings its own scratch.  The flash-attention kernels themselves are in attention_tc.cu.
#include "attention.cuh"

#include <math.h>

#include <mutex>

#include "../../include/forgestep.h"

namespace fs {
namespace {

// ============================================================================ backward pre-pass
// delta[b, n, i] = sum_k dO[b,i,n,k] O[b,i,n,k].  D/8 lanes share one (token, head) row with one 16-byte load per
// tensor each; every warp keeps two groups of rows in flight and walks the rows grid-strided.  The D products of a
// row are added in a fixed order (8 per lane, then a butterfly over the row's lanes).
template <int D>
__global__ void __launch_bounds__(256)
attn_delta_kernel(const bf16* __restrict__ o, const bf16* __restrict__ d_o, float* __restrict__ delta, int B, int S,
                  int n_heads) {
  pdl_trigger();
  pdl_wait();
  constexpr int LPR = D / 8;    // lanes per row
  constexpr int RPW = 32 / LPR;  // rows per warp and load
  const int lane = threadIdx.x & 31, sub = lane / LPR, l = lane % LPR;
  const long long total = (long long)B * S * n_heads;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long base = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * (2 * RPW); base < total;
       base += nwarps * (2 * RPW)) {
    uint4 a[2], d[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const long long w = base + u * RPW + sub;
      const bool ok = w < total;
      a[u] = ok ? *reinterpret_cast<const uint4*>(o + w * D + l * 8) : make_uint4(0, 0, 0, 0);
      d[u] = ok ? *reinterpret_cast<const uint4*>(d_o + w * D + l * 8) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      float acc = bf16_lo(a[u].x) * bf16_lo(d[u].x) + bf16_hi(a[u].x) * bf16_hi(d[u].x);
      acc += bf16_lo(a[u].y) * bf16_lo(d[u].y) + bf16_hi(a[u].y) * bf16_hi(d[u].y);
      acc += bf16_lo(a[u].z) * bf16_lo(d[u].z) + bf16_hi(a[u].z) * bf16_hi(d[u].z);
      acc += bf16_lo(a[u].w) * bf16_lo(d[u].w) + bf16_hi(a[u].w) * bf16_hi(d[u].w);
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
      const long long w = base + u * RPW + sub;
      if (l == 0 && w < total) {
        const int n = (int)(w % n_heads);
        const long long tok = w / n_heads;
        const int b = (int)(tok / S), i = (int)(tok % S);
        delta[((long long)b * n_heads + n) * S + i] = acc;
      }
    }
  }
}

}  // namespace

cudaError_t attention_delta(const bf16* o, const bf16* d_o, float* delta, int B, int S, int nh, int d, cudaStream_t st) {
  const long long rows = (long long)B * S * nh;
  const long long want = (rows * (d / 8) + 2 * 256 - 1) / (2 * 256);  // blocks if every thread took one load pair
  const int blocks = (int)(want < 148 * 8 ? (want > 0 ? want : 1) : 148 * 8);
  if (d == 64) return launch_pdl(attn_delta_kernel<64>, blocks, 256, 0, st, o, d_o, delta, B, S, nh);
  if (d == 128) return launch_pdl(attn_delta_kernel<128>, blocks, 256, 0, st, o, d_o, delta, B, S, nh);
  return cudaErrorInvalidValue;
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
