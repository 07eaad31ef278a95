// Causal flash attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands by TMA).
//
// Forward, one CTA per (128 query rows, head, batch row), two CTAs per SM so that one CTA's softmax overlaps the
// other's matrix work:
//   warp 0      TMA producer: Q once, then K/V blocks of 64 keys through a 2-stage ring
//   warp 1      MMA issuer:   S_j = Q K_j^T (two S buffers in TMEM), O += P_j V_j
//   warps 2..5  softmax: one query row per thread (TMEM lane = row), P written to shared memory as the next
//               MMA's A operand, O rescaled in TMEM only when the row's integer reference moves
// The row reference is an integer power of two (ceil of the running maximum in the log2 domain), so rescaling is
// exact and commutes with the bf16 rounding of P: the result does not depend on the key-block size or order.
#include <math.h>

#include "attention.cuh"
#include "tmap.cuh"

namespace fs {
namespace {

constexpr float kLn2 = 0.6931471805599453f;
constexpr int ATT_THREADS = 192;

// barrier slots of the forward kernel
enum { B_QFULL = 0, B_KVFULL = 1, B_KVEMPTY = 3, B_SFULL = 5, B_SEMPTY = 7, B_PFULL = 9, B_ODONE = 10, B_COUNT = 11 };

template <int D>
struct FwdCfg {
  static constexpr int BQ = 128, BK = 64, KC = D / 64;
  static constexpr int Q_BYTES = BQ * D * 2;
  static constexpr int KV_BYTES = BK * D * 2;  // one K or one V block
  static constexpr int P_BYTES = BQ * BK * 2;
  static constexpr int OFF_K = Q_BYTES;
  static constexpr int OFF_V = OFF_K + 2 * KV_BYTES;
  static constexpr int OFF_P = OFF_V + 2 * KV_BYTES;
  static constexpr int OFF_BAR = OFF_P + P_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 128;
  static constexpr int TMEM_COLS = 256;  // S0 [0,64) S1 [64,128) O [128, 128+D)
  static constexpr int O_COL = 128;
};

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 2)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                   bf16* __restrict__ o, float* __restrict__ lse, int S, int n_heads, int n_kv, float scale_log2,
                   int* err) {
  using C = FwdCfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  const uint32_t bar0 = sbase + C::OFF_BAR;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if ((sbase & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base: refuse rather than compute garbage
    if (threadIdx.x == 0) atomicExch(err, (int)ERR_BAD_ALIGNMENT);
    return;
  }
  const int qb = gridDim.x - 1 - blockIdx.x;  // heaviest blocks first
  const int n = blockIdx.y, b = blockIdx.z;
  const int kvh = n / (n_heads / n_kv);
  const int hq = n_heads * D, hkv = n_kv * D;
  const int q0 = qb * C::BQ;
  const int kv_end = min(S, q0 + C::BQ);
  const int nb = (kv_end + C::BK - 1) / C::BK;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_QFULL), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_KVFULL + i), 1);
      mbar_init(bar(B_KVEMPTY + i), 1);
      mbar_init(bar(B_SFULL + i), 1);
      mbar_init(bar(B_SEMPTY + i), 4);
    }
    mbar_init(bar(B_PFULL), 4);
    mbar_init(bar(B_ODONE), 1);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmKV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), C::Q_BYTES);
#pragma unroll
      for (int kc = 0; kc < C::KC; ++kc)
        tma_load_3d(sbase + kc * (C::BQ * 128), &tmQ, bar(B_QFULL), n * D + kc * 64, q0, b);
      for (int j = 0; j < nb; ++j) {
        const int st = j & 1;
        if (!mbar_wait(bar(B_KVEMPTY + st), (((uint32_t)j >> 1) & 1u) ^ 1u, abort_flag, err)) break;
        mbar_expect_tx(bar(B_KVFULL + st), 2 * C::KV_BYTES);
#pragma unroll
        for (int kc = 0; kc < C::KC; ++kc) {
          tma_load_3d(sbase + C::OFF_K + st * C::KV_BYTES + kc * (C::BK * 128), &tmKV, bar(B_KVFULL + st),
                      hq + kvh * D + kc * 64, j * C::BK, b);
          tma_load_3d(sbase + C::OFF_V + st * C::KV_BYTES + kc * (C::BK * 128), &tmKV, bar(B_KVFULL + st),
                      hq + hkv + kvh * D + kc * 64, j * C::BK, b);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(C::BQ >> 4) << 24);
      const uint32_t idesc_s = idesc_base | ((uint32_t)(C::BK >> 3) << 17);            // N = 64 keys, both K-major
      const uint32_t idesc_pv = idesc_base | (1u << 16) | ((uint32_t)(D >> 3) << 17);  // N = D, B (V) mn-major
      auto issue_s = [&](int j) {
        const int st = j & 1;
        const uint32_t d_tmem = tmem_base + (uint32_t)((j & 1) * C::BK);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint32_t a = sbase + (k >> 2) * (C::BQ * 128) + (k & 3) * 32;
          const uint32_t bb = sbase + C::OFF_K + st * C::KV_BYTES + (k >> 2) * (C::BK * 128) + (k & 3) * 32;
          umma_bf16(d_tmem, umma_desc_sw128(a, 0, 1024), umma_desc_sw128(bb, 0, 1024), idesc_s, k > 0 ? 1u : 0u);
        }
        umma_commit(bar(B_SFULL + (j & 1)));
      };
      bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, err) && mbar_wait(bar(B_KVFULL), 0, abort_flag, err);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; j < nb && ok; ++j) {
        if (j + 1 < nb) {
          const int s1 = (j + 1) & 1;
          if (!mbar_wait(bar(B_KVFULL + s1), ((uint32_t)(j + 1) >> 1) & 1u, abort_flag, err)) { ok = false; break; }
          if (!mbar_wait(bar(B_SEMPTY + s1), (((uint32_t)(j + 1) >> 1) & 1u) ^ 1u, abort_flag, err)) { ok = false; break; }
          tc_fence_after();
          issue_s(j + 1);
        }
        if (!mbar_wait(bar(B_PFULL), (uint32_t)j & 1u, abort_flag, err)) { ok = false; break; }
        tc_fence_after();
        const int st = j & 1;
#pragma unroll
        for (int k = 0; k < C::BK / 16; ++k) {
          const uint32_t a = sbase + C::OFF_P + k * 32;
          const uint32_t bb = sbase + C::OFF_V + st * C::KV_BYTES + k * 2048;
          umma_bf16(tmem_base + C::O_COL, umma_desc_sw128(a, 0, 1024), umma_desc_sw128(bb, C::BK * 128, 1024), idesc_pv,
                    (j > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(bar(B_KVEMPTY + st));
        umma_commit(bar(B_ODONE));
      }
    }
  } else {
    const int q = warp & 3;
    const int rloc = q * 32 + lane;  // row within the tile = TMEM lane
    const int row = q0 + rloc;
    const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
    float mref = -INFINITY, lsum = 0.f;
    bool ok = true;
    for (int j = 0; j < nb; ++j) {
      ok = mbar_wait(bar(B_SFULL + (j & 1)), ((uint32_t)j >> 1) & 1u, abort_flag, err);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t r0[32], r1[32];
      tmem_ld32(tlane + (uint32_t)((j & 1) * C::BK), r0);
      tmem_ld32(tlane + (uint32_t)((j & 1) * C::BK + 32), r1);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SEMPTY + (j & 1)));

      const int k0 = j * C::BK;
      const bool need_mask = k0 + C::BK - 1 > q0 + q * 32;  // warp-uniform
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        float a = __uint_as_float(r0[i]) * scale_log2;
        float c = __uint_as_float(r1[i]) * scale_log2;
        if (need_mask) {
          if (k0 + i > row) a = -INFINITY;
          if (k0 + 32 + i > row) c = -INFINITY;
        }
        r0[i] = __float_as_uint(a);
        r1[i] = __float_as_uint(c);
        mx = fmaxf(mx, fmaxf(a, c));
      }
      const float mnew = fmaxf(mref, ceilf(mx));
      const float alpha = exp2f(mref - mnew);  // exact power of two; 0 on the first block
      float psum = 0.f;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float a = exp2f(__uint_as_float(r0[i]) - mnew);
        const float c = exp2f(__uint_as_float(r1[i]) - mnew);
        psum += a + c;
        r0[i] = __float_as_uint(a);
        r1[i] = __float_as_uint(c);
      }
      lsum = lsum * alpha + psum;
      mref = mnew;

      if (j > 0) {
        // P_{j-1} has been consumed and O holds blocks 0..j-1: both needed before touching P or O
        ok = mbar_wait(bar(B_ODONE), (uint32_t)(j - 1) & 1u, abort_flag, err);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll 1
          for (int c = 0; c < D; c += 32) {
            uint32_t t[32];
            tmem_ld32(tlane + (uint32_t)(C::O_COL + c), t);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
            tmem_st32(tlane + (uint32_t)(C::O_COL + c), t);
          }
          tmem_st_wait();
        }
      }
      // P (bf16) into the 128-byte-swizzled K-major tile [128 rows x 64 keys]
      uint8_t* prow = smem + C::OFF_P + rloc * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint32_t* src = c < 4 ? &r0[c * 8] : &r1[(c - 4) * 8];
        uint4 v;
        v.x = pack_bf16(__uint_as_float(src[0]), __uint_as_float(src[1]));
        v.y = pack_bf16(__uint_as_float(src[2]), __uint_as_float(src[3]));
        v.z = pack_bf16(__uint_as_float(src[4]), __uint_as_float(src[5]));
        v.w = pack_bf16(__uint_as_float(src[6]), __uint_as_float(src[7]));
        *reinterpret_cast<uint4*>(prow + ((c ^ (rloc & 7)) << 4)) = v;
      }
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL));
    }
    if (ok) {
      ok = mbar_wait(bar(B_ODONE), (uint32_t)(nb - 1) & 1u, abort_flag, err);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = 1.0f / lsum;
      bf16* orow = o + ((long long)b * S + row) * hq + n * D;
#pragma unroll 1
      for (int c = 0; c < D; c += 32) {
        uint32_t t[32];
        tmem_ld32(tlane + (uint32_t)(C::O_COL + c), t);
        tmem_ld_wait();
        if (row < S) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(t[i]) * inv, __uint_as_float(t[i + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(t[i + 2]) * inv, __uint_as_float(t[i + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(t[i + 4]) * inv, __uint_as_float(t[i + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(t[i + 6]) * inv, __uint_as_float(t[i + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + c + i) = v;
          }
        }
      }
      if (row < S) lse[((long long)b * n_heads + n) * S + row] = (mref + log2f(lsum)) * kLn2;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int D>
cudaError_t attention_fwd_tc_t(const bf16* qkv, bf16* o, float* lse, int B, int S, int nh, int nkv, int* err,
                               cudaStream_t st) {
  using C = FwdCfg<D>;
  static bool once = false;
  if (!once) {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    once = true;
  }
  const int nqkv = (nh + 2 * nkv) * D;
  CUtensorMap tmQ, tmKV;
  if (!make_tmap_3d(&tmQ, qkv, nqkv, S, B, nqkv, C::BQ) || !make_tmap_3d(&tmKV, qkv, nqkv, S, B, nqkv, C::BK))
    return cudaErrorInvalidValue;
  const float scale_log2 = (float)((1.0 / sqrt((double)D)) * 1.4426950408889634);
  dim3 grid((S + C::BQ - 1) / C::BQ, nh, B);
  attn_fwd_tc_kernel<D><<<grid, ATT_THREADS, C::SMEM_BYTES, st>>>(tmQ, tmKV, o, lse, S, nh, nkv, scale_log2, err);
  return cudaGetLastError();
}

static __device__ int g_attn_status;

}  // namespace

int g_attention_impl = 1;

int* attention_status_word() {
  static int* addr[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!addr[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_attn_status) != cudaSuccess) return nullptr;
    addr[dev] = p;
  }
  return addr[dev];
}

cudaError_t attention_fwd_tc(const bf16* qkv, bf16* o, float* lse, int B, int S, int nh, int nkv, int d, int* err,
                             cudaStream_t st) {
  if (B <= 0 || S <= 0 || nh <= 0 || nkv <= 0 || nh % nkv || !err) return cudaErrorInvalidValue;
  if (d == 64) return attention_fwd_tc_t<64>(qkv, o, lse, B, S, nh, nkv, err, st);
  if (d == 128) return attention_fwd_tc_t<128>(qkv, o, lse, B, S, nh, nkv, err, st);
  return cudaErrorInvalidValue;
}

}  // namespace fs
