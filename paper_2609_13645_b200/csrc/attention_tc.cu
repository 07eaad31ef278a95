// Causal flash attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands by TMA).
//
// Forward, one CTA per (128 query rows, head, batch row), two CTAs per SM so that one CTA's softmax overlaps the
// other's matrix work:
//   warp 0      TMA producer: Q once, then K blocks of 64 keys through a 3-stage ring
//   warp 6      TMA producer: V blocks through a 2-stage ring (V is needed a block later than K)
//   warp 1      MMA issuer:   S_j = Q K_j^T (two S buffers in TMEM), O += P_j V_j with P read from TMEM
//   warps 2..5  softmax: one query row per thread (TMEM lane = row), bf16 P written back over the S columns it came
//               from, O rescaled in TMEM only when the row's integer reference moves
// The row reference is an integer power of two (ceil of the running maximum in the log2 domain), so rescaling is
// exact and commutes with the bf16 rounding of P: the result does not depend on the key-block size or order.
#include <math.h>

#include "attention.cuh"

#include <mutex>
#include "tmap.cuh"

namespace fs {
namespace {

constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRefSlack = 8.0f;

// barrier slots of the forward kernel
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 4, B_VFULL = 7, B_VEMPTY = 9, B_SFULL = 11, B_PFULL = 13, B_ODONE = 15,
       B_OFINAL = 16, B_COUNT = 17 };
constexpr int ATT_THREADS = 224;  // K producer, MMA issuer, 4 softmax warps, V producer

template <int D>
struct FwdCfg {
  static constexpr int BQ = 128, BK = 64, KC = D / 64;
  static constexpr int NK = 3, NV = 2;  // K is needed one block ahead of V, so it gets the deeper ring
  static constexpr int Q_BYTES = BQ * D * 2;
  static constexpr int KV_BYTES = BK * D * 2;  // one K or one V block
  static constexpr int OFF_K = Q_BYTES;
  static constexpr int OFF_V = OFF_K + NK * KV_BYTES;
  static constexpr int OFF_BAR = OFF_V + NV * KV_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 160;
  static constexpr int TMEM_COLS = 256;  // S0 [0,64) S1 [64,128) (bf16 P overwrites the first 32 columns) O [128, 128+D)
  static constexpr int O_COL = 128;
};

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 2)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                   bf16* __restrict__ o, float* __restrict__ lse, int S, int n_heads, int n_kv, int n_batch, int n_qblocks,
                   float scale_log2, int* err) {
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
  // Thread blocks are started in index order, so the index runs over the query blocks from the heaviest (last) to the
  // lightest across ALL heads and batch rows: the blocks still running at the end of the launch are the short ones.  (With
  // the query block as the fastest grid dimension the heaviest block of the last head started last and ran alone.)
  const int groups = n_heads * n_batch;
  const int qb = n_qblocks - 1 - (int)blockIdx.x / groups;
  const int grp = (int)blockIdx.x % groups;
  const int n = grp % n_heads, b = grp / n_heads;
  const int kvh = n / (n_heads / n_kv);
  const int hq = n_heads * D, hkv = n_kv * D;
  const int q0 = qb * C::BQ;
  const int kv_end = min(S, q0 + C::BQ);
  const int nb = (kv_end + C::BK - 1) / C::BK;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_QFULL), 1);
    for (int i = 0; i < C::NK; ++i) {
      mbar_init(bar(B_KFULL + i), 1);
      mbar_init(bar(B_KEMPTY + i), 1);
    }
    for (int i = 0; i < C::NV; ++i) {
      mbar_init(bar(B_VFULL + i), 1);
      mbar_init(bar(B_VEMPTY + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_SFULL + i), 1);
      // two P barriers: a softmax warp that does not have to rescale O may run one block ahead of a slower warp, and
      // its arrival for block j+1 must not be counted for block j
      mbar_init(bar(B_PFULL + i), 4);
    }
    mbar_init(bar(B_ODONE), 1);
    mbar_init(bar(B_OFINAL), 1);
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
  pdl_trigger();
  pdl_wait();  // set-up done; from here on the kernel touches what its predecessor wrote

  if (warp == 0) {
    // ------------------------------------------------------------------ Q and K producer
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), C::Q_BYTES);
#pragma unroll
      for (int kc = 0; kc < C::KC; ++kc)
        tma_load_3d(sbase + kc * (C::BQ * 128), &tmQ, bar(B_QFULL), n * D + kc * 64, q0, b);
      for (int j = 0; j < nb; ++j) {
        const int st = j % C::NK;
        if (!mbar_wait(bar(B_KEMPTY + st), ((uint32_t)(j / C::NK) & 1u) ^ 1u, abort_flag, err, kWaitLimitCycles, 0x31)) break;
        mbar_expect_tx(bar(B_KFULL + st), C::KV_BYTES);
#pragma unroll
        for (int kc = 0; kc < C::KC; ++kc)
          tma_load_3d(sbase + C::OFF_K + st * C::KV_BYTES + kc * (C::BK * 128), &tmKV, bar(B_KFULL + st),
                      hq + kvh * D + kc * 64, j * C::BK, b);
      }
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ V producer
    if (lane == 0) {
      for (int j = 0; j < nb; ++j) {
        const int st = j % C::NV;
        if (!mbar_wait(bar(B_VEMPTY + st), ((uint32_t)(j / C::NV) & 1u) ^ 1u, abort_flag, err, kWaitLimitCycles, 0x32)) break;
        mbar_expect_tx(bar(B_VFULL + st), C::KV_BYTES);
#pragma unroll
        for (int kc = 0; kc < C::KC; ++kc)
          tma_load_3d(sbase + C::OFF_V + st * C::KV_BYTES + kc * (C::BK * 128), &tmKV, bar(B_VFULL + st),
                      hq + hkv + kvh * D + kc * 64, j * C::BK, b);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(C::BQ >> 4) << 24);
      const uint32_t idesc_s = idesc_base | ((uint32_t)(C::BK >> 3) << 17);            // N = 64 keys, both K-major
      const uint32_t idesc_pv = idesc_base | (1u << 16) | ((uint32_t)(D >> 3) << 17);  // N = D, B (V) mn-major
      const uint64_t dq = umma_desc_sw128(sbase, 0, 1024);
      // S_j overwrites the TMEM buffer that held P_{j-2}; PV_{j-2} was issued earlier by this thread, so it is ordered
      auto issue_s = [&](int j) -> bool {
        const int st = j % C::NK;
        if (!mbar_wait(bar(B_KFULL + st), (uint32_t)(j / C::NK) & 1u, abort_flag, err, kWaitLimitCycles, 0x33)) return false;
        tc_fence_after();
        const uint64_t dk = umma_desc_sw128(sbase + C::OFF_K + st * C::KV_BYTES, 0, 1024);
        const uint32_t d_tmem = tmem_base + (uint32_t)((j & 1) * C::BK);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t qo = (uint64_t)(((k >> 2) * (C::BQ * 128) + (k & 3) * 32) >> 4);
          const uint64_t ko = (uint64_t)(((k >> 2) * (C::BK * 128) + (k & 3) * 32) >> 4);
          umma_bf16(d_tmem, dq + qo, dk + ko, idesc_s, k > 0 ? 1u : 0u);
        }
        umma_commit(bar(B_SFULL + (j & 1)));
        umma_commit(bar(B_KEMPTY + st));  // K_j is free as soon as S_j is done
        return true;
      };
      bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, err, kWaitLimitCycles, 0x34);
      if (ok) ok = issue_s(0);
      for (int j = 0; j < nb && ok; ++j) {
        if (j + 1 < nb && !issue_s(j + 1)) { ok = false; break; }
        const int st = j % C::NV;
        if (!mbar_wait(bar(B_VFULL + st), (uint32_t)(j / C::NV) & 1u, abort_flag, err, kWaitLimitCycles, 0x35)) { ok = false; break; }
        if (!mbar_wait(bar(B_PFULL + (j & 1)), ((uint32_t)j >> 1) & 1u, abort_flag, err, kWaitLimitCycles, 0x36)) { ok = false; break; }
        tc_fence_after();
        const uint64_t dv = umma_desc_sw128(sbase + C::OFF_V + st * C::KV_BYTES, C::BK * 128, 1024);
        const uint32_t tp = tmem_base + (uint32_t)((j & 1) * C::BK);  // bf16 P: 16 keys = 8 columns per K step
#pragma unroll
        for (int k = 0; k < C::BK / 16; ++k)
          umma_bf16_ts(tmem_base + C::O_COL, tp + (uint32_t)(k * 8), dv + (uint64_t)((k * 2048) >> 4), idesc_pv,
                       (j > 0 || k > 0) ? 1u : 0u);
        umma_commit(bar(B_VEMPTY + st));
        umma_commit(bar(B_ODONE));
      }
      if (ok) umma_commit(bar(B_OFINAL));  // every product of this tile is done: a barrier of its own, one phase
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (2..5)
    const int q = warp & 3;
    const int rloc = q * 32 + lane;  // row within the tile = TMEM lane
    const int row = q0 + rloc;
    const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
    float mref = -INFINITY, lsum = 0.f;
    bool ok = true;
    for (int j = 0; j < nb; ++j) {
      ok = mbar_wait(bar(B_SFULL + (j & 1)), ((uint32_t)j >> 1) & 1u, abort_flag, err, kWaitLimitCycles, 0x37);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t r0[32], r1[32];
      tmem_ld32(tlane + (uint32_t)((j & 1) * C::BK), r0);
      tmem_ld32(tlane + (uint32_t)((j & 1) * C::BK + 32), r1);
      tmem_ld_wait();

      const int k0 = j * C::BK;
      const bool need_mask = k0 + C::BK - 1 > q0 + q * 32;  // warp-uniform
      if (need_mask) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (k0 + i > row) r0[i] = 0xff800000u;       // -inf
          if (k0 + 32 + i > row) r1[i] = 0xff800000u;
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fmaxf(__uint_as_float(r0[i]), __uint_as_float(r1[i])));
      // scale_log2 > 0, so the maximum commutes with the scaling.  The reference only moves once the block maximum
      // has passed it by more than 2^kRefSlack (P stays below that, far from overflow): with 32 rows per warp some
      // row's maximum crosses an integer in almost every block, and each move costs the whole warp a wait for the
      // previous P V product and a pass over O.  Powers of two commute with the roundings, so nothing else changes.
      const float mcand = ceilf(mx * scale_log2);
      const float mnew = mcand > mref + kRefSlack ? mcand : mref;
      const float alpha = fast_exp2(mref - mnew);  // exact power of two; 0 on the first block
      float psum = 0.f;
      uint32_t pw[32];  // bf16 pairs: keys 2c, 2c+1 in word c
#pragma unroll
      for (int i = 0; i < 32; i += 2) {
        const float a0 = fast_exp2(fmaf(__uint_as_float(r0[i]), scale_log2, -mnew));
        const float a1 = fast_exp2(fmaf(__uint_as_float(r0[i + 1]), scale_log2, -mnew));
        const float c0 = fast_exp2(fmaf(__uint_as_float(r1[i]), scale_log2, -mnew));
        const float c1 = fast_exp2(fmaf(__uint_as_float(r1[i + 1]), scale_log2, -mnew));
        psum += (a0 + a1) + (c0 + c1);
        pw[i >> 1] = pack_bf16(a0, a1);
        pw[16 + (i >> 1)] = pack_bf16(c0, c1);
      }
      lsum = lsum * alpha + psum;
      mref = mnew;

      // O has to be rescaled only when this row's integer reference moved (rare after the first blocks); only then
      // does the softmax wait for the previous P V product
      if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
        ok = mbar_wait(bar(B_ODONE), (uint32_t)(j - 1) & 1u, abort_flag, err, kWaitLimitCycles, 0x38);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < D; c += 32) {
          uint32_t t[32];
          tmem_ld32(tlane + (uint32_t)(C::O_COL + c), t);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) t[i] = __float_as_uint(__uint_as_float(t[i]) * alpha);
          tmem_st32(tlane + (uint32_t)(C::O_COL + c), t);
        }
      }
      // bf16 P back into TMEM over the first 32 of the 64 fp32 columns it was computed from
      tmem_st32(tlane + (uint32_t)((j & 1) * C::BK), pw);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL + (j & 1)));
    }
    // The end of the last P V product is signalled on a barrier of its own.  (B_ODONE cannot serve: a parity wait only
    // tells two consecutive phases apart, and a warp that is slow to get here after its last arrival can find that
    // barrier two phases on, products nb-2 AND nb-1 both done, which reads like "nb-2 still running": waiting for the
    // two in turn ran into its time limit about once in 10^7 thread blocks.)
    if (ok) {
      ok = mbar_wait(bar(B_OFINAL), 0, abort_flag, err, kWaitLimitCycles, 0x39);
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
  static unsigned long long smem_set = 0;
  cudaError_t e0 = ensure_dynamic_smem(attn_fwd_tc_kernel<D>, C::SMEM_BYTES, smem_set);
  if (e0 != cudaSuccess) return e0;
  const int nqkv = (nh + 2 * nkv) * D;
  CUtensorMap tmQ, tmKV;
  if (!make_tmap_3d(&tmQ, qkv, nqkv, S, B, nqkv, C::BQ) || !make_tmap_3d(&tmKV, qkv, nqkv, S, B, nqkv, C::BK))
    return cudaErrorInvalidValue;
  const float scale_log2 = (float)((1.0 / sqrt((double)D)) * 1.4426950408889634);
  const int nqb = (S + C::BQ - 1) / C::BQ;
  dim3 grid((unsigned)(nqb * nh * B), 1, 1);
  cudaError_t el = launch_pdl(attn_fwd_tc_kernel<D>, grid, ATT_THREADS, C::SMEM_BYTES, st, tmQ, tmKV, o, lse, S, nh, nkv, B, nqb, scale_log2, err);
  if (el != cudaSuccess) return el;
  return cudaGetLastError();
}

// ============================================================================ backward
// One kernel template for both halves of the deterministic backward.  A CTA keeps a "resident" pair of [128 x D]
// tiles (X1, X2) and streams pairs of [64 x D] tiles (Y1, Y2):
//   MODE_DQ : X = (Q, dO) of 128 queries, Y = (K, V) blocks          -> dQ  += dS  K
//   MODE_DKV: X = (K, V) of 128 keys,     Y = (Q, dO) blocks, all the query heads of the GQA group in a fixed order
//                                                                     -> dV += P^T dO,  dK += dS^T Q
// Per streamed block:  S = X1 Y1^T and dP = X2 Y2^T (two tcgen05 GEMMs into one of two TMEM buffers); the compute
// warps (one X row per thread) turn them into P = exp2(S c - LSE) and dS = P (dP - delta), write them as bf16
// A-operand tiles to shared memory, and the accumulating GEMMs read the SAME streamed tiles again as mn-major B
// operands.  warp 0 = TMA producer, warp 1 = MMA issuer, warps 2..9 = compute (two warps per TMEM lane quarter, each
// taking half of the 64 streamed columns).
enum { MODE_DQ = 0, MODE_DKV = 1 };
// barrier slots: Y ring (up to 4 stages) first, then the double-buffered TMEM / operand-tile handshakes
enum { BB_XFULL = 0, BB_YFULL = 1, BB_YEMPTY = 5, BB_SDPFULL = 9, BB_SDPEMPTY = 11, BB_TFULL = 13, BB_TEMPTY = 15,
       BB_ACCDONE = 17, BB_COUNT = 18 };
constexpr int BWD_THREADS = 352;  // producer, MMA issuer A, 8 compute warps, MMA issuer B

template <int D, int MODE>
struct BwdCfg {
  static constexpr int KC = D / 64;
  static constexpr int X_BYTES = 128 * D * 2;
  static constexpr int Y_BYTES = 64 * D * 2;
  static constexpr int NST = 4;  // stages of the streamed-tile ring
  static constexpr int OFF_X1 = 0, OFF_X2 = X_BYTES, OFF_Y = 2 * X_BYTES;
  static constexpr int OFF_STAT = OFF_Y + NST * 2 * Y_BYTES;
  static constexpr int OFF_BAR = OFF_STAT + 2048;
  static constexpr int SMEM_BYTES = OFF_BAR + 256;
  static constexpr int TMEM_COLS = 512;  // buffer b: S at b*128, dP at b*128+64; accumulators from column 256
  static constexpr int ACC0 = 256, ACC1 = 256 + D;
};

__device__ __forceinline__ void store8_b32(void* dst, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
               "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

template <int W>
__device__ __forceinline__ void tmem_load_cols(uint32_t taddr, float (&out)[W]) {
  static_assert(W == 32 || W == 16, "chunk width");
  if constexpr (W == 32) {
    uint32_t t[32];
    tmem_ld32(taddr, t);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) out[i] = __uint_as_float(t[i]);
  } else {
    uint32_t t[16];
    tmem_ld16(taddr, t);
    tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] = __uint_as_float(t[i]);
  }
}

template <int W>
__device__ __forceinline__ void store_bf16_row(bf16* dst, const float (&v)[W]) {
#pragma unroll
  for (int i = 0; i < W; i += 8) {
    uint4 o;
    o.x = pack_bf16(v[i], v[i + 1]);
    o.y = pack_bf16(v[i + 2], v[i + 3]);
    o.z = pack_bf16(v[i + 4], v[i + 5]);
    o.w = pack_bf16(v[i + 6], v[i + 7]);
    *reinterpret_cast<uint4*>(dst + i) = o;
  }
}

template <int D, int MODE>
__global__ void __launch_bounds__(BWD_THREADS, 1)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap tm_qkv128, const __grid_constant__ CUtensorMap tm_qkv64,
                   const __grid_constant__ CUtensorMap tm_do128, const __grid_constant__ CUtensorMap tm_do64,
                   const float* __restrict__ lse, const float* __restrict__ delta, bf16* __restrict__ dqkv,
                   bf16* __restrict__ ds_out, const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, int S,
                   int n_heads, int n_kv, int n_batch, int n_xblocks, float scale, float scale_log2, int* err) {
  using C = BwdCfg<D, MODE>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  const uint32_t bar0 = sbase + C::OFF_BAR;
  auto bar = [&](int i) { return bar0 + 8u * i; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + BB_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* s_stat = reinterpret_cast<float*>(smem + C::OFF_STAT);  // [stage][0: lse*log2e, 1: delta][64]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if ((sbase & 1023u) != 0u) {
    if (threadIdx.x == 0) atomicExch(err, (int)ERR_BAD_ALIGNMENT);
    return;
  }
  const int n_rep = n_heads / n_kv;
  const int hq = n_heads * D, hkv = n_kv * D;
  const long long ld = hq + 2 * hkv;
  // one-dimensional grid, heaviest blocks first across all heads and batch rows (see the forward kernel)
  const int groups = (MODE == MODE_DQ ? n_heads : n_kv) * n_batch;
  const int xrank = (int)blockIdx.x / groups, grp = (int)blockIdx.x % groups;
  const int heads_here = MODE == MODE_DQ ? n_heads : n_kv;
  const int b = grp / heads_here;
  int x0, kvh, n_q = 0, iters, qb0 = 0, per_head = 1;
  if constexpr (MODE == MODE_DQ) {
    x0 = (n_xblocks - 1 - xrank) * 128;  // the last query blocks see the most keys
    n_q = grp % heads_here;
    kvh = n_q / n_rep;
    iters = (min(S, x0 + 128) + 63) / 64;
  } else {
    x0 = xrank * 128;  // the first key blocks see the most queries
    kvh = grp % heads_here;
    qb0 = x0 / 64;
    per_head = (S + 63) / 64 - qb0;
    iters = per_head * n_rep;
  }

  if (threadIdx.x == 0) {
    mbar_init(bar(BB_XFULL), 1);
    for (int i = 0; i < C::NST; ++i) {
      mbar_init(bar(BB_YFULL + i), MODE == MODE_DKV ? 2 : 1);
      mbar_init(bar(BB_YEMPTY + i), 2);   // one commit from each MMA-issuing warp
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(BB_SDPFULL + i), 2);
      mbar_init(bar(BB_TFULL + i), 8);
    }
    mbar_init(bar(BB_ACCDONE), 2);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_qkv128);
    tma_prefetch_desc(&tm_qkv64);
    tma_prefetch_desc(&tm_do128);
    tma_prefetch_desc(&tm_do64);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();
  pdl_wait();  // set-up done; from here on the kernel touches what its predecessor wrote

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      mbar_expect_tx(bar(BB_XFULL), 2 * C::X_BYTES);
#pragma unroll
      for (int kc = 0; kc < C::KC; ++kc) {
        if constexpr (MODE == MODE_DQ) {
          tma_load_3d(sbase + C::OFF_X1 + kc * 16384, &tm_qkv128, bar(BB_XFULL), n_q * D + kc * 64, x0, b);
          tma_load_3d(sbase + C::OFF_X2 + kc * 16384, &tm_do128, bar(BB_XFULL), n_q * D + kc * 64, x0, b);
        } else {
          tma_load_3d(sbase + C::OFF_X1 + kc * 16384, &tm_qkv128, bar(BB_XFULL), hq + kvh * D + kc * 64, x0, b);
          tma_load_3d(sbase + C::OFF_X2 + kc * 16384, &tm_qkv128, bar(BB_XFULL), hq + hkv + kvh * D + kc * 64, x0, b);
        }
      }
    }
    for (int it = 0; it < iters; ++it) {
      const int st = it % C::NST;
      bool ok = mbar_wait(bar(BB_YEMPTY + st), (((uint32_t)(it / C::NST)) & 1u) ^ 1u, abort_flag, err, kWaitLimitCycles, 0x41);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t ydst = sbase + C::OFF_Y + st * 2 * C::Y_BYTES;
      if constexpr (MODE == MODE_DQ) {
        if (lane == 0) {
          mbar_expect_tx(bar(BB_YFULL + st), 2 * C::Y_BYTES);
#pragma unroll
          for (int kc = 0; kc < C::KC; ++kc) {
            tma_load_3d(ydst + kc * 8192, &tm_qkv64, bar(BB_YFULL + st), hq + kvh * D + kc * 64, it * 64, b);
            tma_load_3d(ydst + C::Y_BYTES + kc * 8192, &tm_qkv64, bar(BB_YFULL + st), hq + hkv + kvh * D + kc * 64,
                        it * 64, b);
          }
        }
      } else {
        const int rep = it / per_head, qb = qb0 + it % per_head;
        const int n = kvh * n_rep + rep;
        if (lane == 0) {
          mbar_expect_tx(bar(BB_YFULL + st), 2 * C::Y_BYTES);
#pragma unroll
          for (int kc = 0; kc < C::KC; ++kc) {
            tma_load_3d(ydst + kc * 8192, &tm_qkv64, bar(BB_YFULL + st), n * D + kc * 64, qb * 64, b);
            tma_load_3d(ydst + C::Y_BYTES + kc * 8192, &tm_do64, bar(BB_YFULL + st), n * D + kc * 64, qb * 64, b);
          }
        }
        const long long stat = ((long long)b * n_heads + n) * S;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int qq = qb * 64 + lane * 2 + e;
          s_stat[st * 128 + lane * 2 + e] = qq < S ? lse[stat + qq] * 1.4426950408889634f : 0.f;
          s_stat[st * 128 + 64 + lane * 2 + e] = qq < S ? delta[stat + qq] : 0.f;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BB_YFULL + st));
      }
    }
  } else if (warp == 1 || warp == 10) {
    // ------------------------------------------------------------------ MMA issuers
    // A single thread cannot issue the small (N = 64 / 128) MMAs of this kernel fast enough to keep the tensor pipe
    // fed, so two warps issue independent accumulator chains: side 0 owns S (and dV, which reads P^T from the S
    // columns), side 1 owns dP (and dK / dQ, which read dS from the dP columns).  Each chain stays in issue order.
    if (lane == 0) {
      const int side = warp == 1 ? 0 : 1;
      const uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t idesc_sdp = idesc_base | ((uint32_t)(64 >> 3) << 17);            // N = 64, both K-major
      const uint32_t idesc_acc = idesc_base | (1u << 16) | ((uint32_t)(D >> 3) << 17);  // N = D, B mn-major
      // descriptors are built once per tile; a K step of 16 elements moves the start-address field (units of 16 B)
      // by 2 inside a 64-element chunk of a K-major tile and by 128 for an mn-major tile
      const uint64_t dx = umma_desc_sw128(sbase + (side == 0 ? C::OFF_X1 : C::OFF_X2), 0, 1024);
      auto issue_sdp = [&](int it) {
        const int st = it % C::NST;
        const uint32_t y = sbase + C::OFF_Y + st * 2 * C::Y_BYTES + side * C::Y_BYTES;
        const uint64_t dy = umma_desc_sw128(y, 0, 1024);
        const uint32_t d_t = tmem_base + (uint32_t)((it & 1) * 128 + side * 64);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t xo = (uint64_t)(((k >> 2) * 16384 + (k & 3) * 32) >> 4);
          const uint64_t yo = (uint64_t)(((k >> 2) * 8192 + (k & 3) * 32) >> 4);
          umma_bf16(d_t, dx + xo, dy + yo, idesc_sdp, k > 0 ? 1u : 0u);
        }
        umma_commit(bar(BB_SDPFULL + (it & 1)));
      };
      bool ok = mbar_wait(bar(BB_XFULL), 0, abort_flag, err, kWaitLimitCycles, 0x42) && mbar_wait(bar(BB_YFULL), 0, abort_flag, err, kWaitLimitCycles, 0x43);
      if (ok) {
        tc_fence_after();
        issue_sdp(0);
      }
      for (int it = 0; it < iters && ok; ++it) {
        if (it + 1 < iters) {
          const int y1s = (it + 1) % C::NST;
          if (!mbar_wait(bar(BB_YFULL + y1s), ((uint32_t)((it + 1) / C::NST)) & 1u, abort_flag, err, kWaitLimitCycles, 0x44)) { ok = false; break; }
          // the TMEM columns this writes were last read by this same thread's accumulating MMAs of block it-1: in order
          tc_fence_after();
          issue_sdp(it + 1);
        }
        const int bf = it & 1;
        if (!mbar_wait(bar(BB_TFULL + bf), ((uint32_t)it >> 1) & 1u, abort_flag, err, kWaitLimitCycles, 0x45)) { ok = false; break; }
        tc_fence_after();
        const int yst = it % C::NST;
        const uint32_t y1 = sbase + C::OFF_Y + yst * 2 * C::Y_BYTES, y2 = y1 + C::Y_BYTES;
        // A operands (bf16 P^T / dS^T) sit in TMEM where S / dP were: 16 queries (K = 16) = 8 columns; the two
        // compute warps of a lane quarter each wrote their 32 queries at the start of their own 32 fp32 columns
        const uint32_t ta = tmem_base + (uint32_t)(bf * 128 + side * 64);
        const uint32_t first = it > 0 ? 1u : 0u;
        if (MODE == MODE_DKV || side == 1) {
          // side 0: dV += P^T dO;  side 1: dK += dS^T Q  (or dQ += dS K)
          const uint64_t by = umma_desc_sw128((MODE == MODE_DKV && side == 0) ? y2 : y1, 8192, 1024);
          const uint32_t dacc = tmem_base + (uint32_t)((MODE == MODE_DKV && side == 1) ? C::ACC1 : C::ACC0);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint32_t acol = (uint32_t)((k >> 1) * 32 + (k & 1) * 8);
            umma_bf16_ts(dacc, ta + acol, by + (uint64_t)((k * 2048) >> 4), idesc_acc, k > 0 ? 1u : first);
          }
        }
        umma_commit(bar(BB_YEMPTY + yst));
      }
      if (ok) umma_commit(bar(BB_ACCDONE));
    }
  } else {
    // ------------------------------------------------------------------ compute warps
    const int q = warp & 3, ch = (warp - 2) >> 2;
    const int rloc = q * 32 + lane;
    const int row = x0 + rloc;  // query (MODE_DQ) or key (MODE_DKV) position
    const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
    float lse2_row = 0.f, delta_row = 0.f;
    if constexpr (MODE == MODE_DQ) {
      if (row < S) {
        const long long stat = ((long long)b * n_heads + n_q) * S;
        lse2_row = lse[stat + row] * 1.4426950408889634f;
        delta_row = delta[stat + row];
      }
    }
    bool ok = true;
    for (int it = 0; it < iters; ++it) {
      const int bf = it & 1;
      ok = mbar_wait(bar(BB_SDPFULL + bf), ((uint32_t)it >> 1) & 1u, abort_flag, err, kWaitLimitCycles, 0x46);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      uint32_t rs[32], rp[32];
      tmem_ld32(tlane + (uint32_t)(bf * 128 + ch * 32), rs);
      tmem_ld32(tlane + (uint32_t)(bf * 128 + 64 + ch * 32), rp);
      tmem_ld_wait();

      int y0;
      const int yst = it % C::NST;
      const float* st_lse = s_stat + yst * 128 + ch * 32;
      const float* st_dl = st_lse + 64;
      if constexpr (MODE == MODE_DQ) {
        y0 = it * 64;
      } else {
        y0 = (qb0 + it % per_head) * 64;
        ok = mbar_wait(bar(BB_YFULL + yst), ((uint32_t)(it / C::NST)) & 1u, abort_flag, err, kWaitLimitCycles, 0x47);  // acquire the staged statistics
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      // masking is only needed where the block touches the diagonal (or the end of the sequence): warp-uniform
      const int cmin = y0 + ch * 32, rmin = x0 + q * 32;
      bool full;
      if constexpr (MODE == MODE_DQ) full = cmin + 31 <= rmin;            // every key <= every query of this warp
      else full = cmin >= rmin + 31 && cmin + 32 <= S;                    // every query >= every key, and in range
      if constexpr (MODE == MODE_DQ) {
        const float nl = -lse2_row;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float p = fast_exp2(fmaf(__uint_as_float(rs[i]), scale_log2, nl));
          if (!full && cmin + i > row) p = 0.f;
          rs[i] = __float_as_uint(p);
          rp[i] = __float_as_uint(p * (__uint_as_float(rp[i]) - delta_row));
        }
      } else {
        if (full) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(st_lse + i);
            const float4 d4 = *reinterpret_cast<const float4*>(st_dl + i);
            const float ll[4] = {l4.x, l4.y, l4.z, l4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              const float p = fast_exp2(fmaf(__uint_as_float(rs[i + u]), scale_log2, -ll[u]));
              rs[i + u] = __float_as_uint(p);
              rp[i + u] = __float_as_uint(p * (__uint_as_float(rp[i + u]) - dd[u]));
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            const float4 l4 = *reinterpret_cast<const float4*>(st_lse + i);
            const float4 d4 = *reinterpret_cast<const float4*>(st_dl + i);
            const float ll[4] = {l4.x, l4.y, l4.z, l4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              float p = fast_exp2(fmaf(__uint_as_float(rs[i + u]), scale_log2, -ll[u]));
              if (cmin + i + u < row || cmin + i + u >= S) p = 0.f;
              rs[i + u] = __float_as_uint(p);
              rp[i + u] = __float_as_uint(p * (__uint_as_float(rp[i + u]) - dd[u]));
            }
          }
        }
      }
      // bf16 pairs back into TMEM, over this warp's own (already loaded) fp32 columns
      uint32_t wp[16], wd[16];
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        wp[c] = pack_bf16(__uint_as_float(rs[2 * c]), __uint_as_float(rs[2 * c + 1]));
        wd[c] = pack_bf16(__uint_as_float(rp[2 * c]), __uint_as_float(rp[2 * c + 1]));
      }
      if constexpr (MODE == MODE_DKV) tmem_st16(tlane + (uint32_t)(bf * 128 + ch * 32), wp);
      tmem_st16(tlane + (uint32_t)(bf * 128 + 64 + ch * 32), wd);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BB_TFULL + bf));
      if constexpr (MODE == MODE_DKV) {
        // after the arrival, off the MMA chain's critical path: the same rounded dS also goes to the dS^T scratch
        // of the dQ contraction that follows (S % 128 == 0 there)
        if (ds_out != nullptr) {
          const int n = kvh * n_rep + it / per_head;
          // 32-query chunks [b n_h + n][query / 32][key][query % 32]: one contiguous 64-byte row per thread
          bf16* dsp = ds_out + ((((long long)b * n_heads + n) * (S >> 5) + (cmin >> 5)) * S + row) * 32;
          store8_b32(dsp, wd);
          store8_b32(dsp + 16, wd + 8);
        }
      }
    }
    if (ok) {
      ok = mbar_wait(bar(BB_ACCDONE), 0, abort_flag, err, kWaitLimitCycles, 0x48);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      // rotated output (dQ or dK): this warp owns columns [i0, i0+W) and their partners D/2 further
      constexpr int W = D / 4, H = D / 2;
      const int i0 = ch * W;
      const uint32_t racc = tlane + (uint32_t)(MODE == MODE_DQ ? C::ACC0 : C::ACC1);
      float lo[W], hi[W];
      tmem_load_cols<W>(racc + (uint32_t)i0, lo);
      tmem_load_cols<W>(racc + (uint32_t)(H + i0), hi);
#pragma unroll
      for (int i = 0; i < W; ++i) { lo[i] *= scale; hi[i] *= scale; }
      if (rope_cos != nullptr) {
        const int pos = min(row, S - 1);
        const float* cs = rope_cos + (long long)pos * H + i0;
        const float* sn = rope_sin + (long long)pos * H + i0;
#pragma unroll
        for (int i = 0; i < W; i += 4) {
          const float4 c4 = *reinterpret_cast<const float4*>(cs + i);
          const float4 s4 = *reinterpret_cast<const float4*>(sn + i);
          const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float y1 = lo[i + u], y2 = hi[i + u];
            lo[i + u] = y1 * cc[u] + y2 * ss[u];
            hi[i + u] = y2 * cc[u] - y1 * ss[u];
          }
        }
      }
      const int colbase = MODE == MODE_DQ ? n_q * D : hq + kvh * D;
      if (row < S) {
        bf16* dst = dqkv + ((long long)b * S + row) * ld + colbase;
        store_bf16_row<W>(dst + i0, lo);
        store_bf16_row<W>(dst + H + i0, hi);
      }
      if constexpr (MODE == MODE_DKV) {
        bf16* dstv = dqkv + ((long long)b * S + row) * ld + hq + hkv + kvh * D;
#pragma unroll 1
        for (int c = ch * H; c < (ch + 1) * H; c += 32) {
          float v[32];
          tmem_load_cols<32>(tlane + (uint32_t)(C::ACC0 + c), v);
          if (row < S) store_bf16_row<32>(dstv + c, v);
        }
      }
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
cudaError_t attention_bwd_tc_t(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                               const float* cs, const float* sn, bf16* ds, int B, int S, int nh, int nkv, int* err,
                               cudaStream_t st) {
  using CQ = BwdCfg<D, MODE_DQ>;
  using CK = BwdCfg<D, MODE_DKV>;
  static unsigned long long smem_set_q = 0, smem_set_k = 0;
  cudaError_t e0 = ensure_dynamic_smem(attn_bwd_tc_kernel<D, MODE_DQ>, CQ::SMEM_BYTES, smem_set_q);
  if (e0 != cudaSuccess) return e0;
  e0 = ensure_dynamic_smem(attn_bwd_tc_kernel<D, MODE_DKV>, CK::SMEM_BYTES, smem_set_k);
  if (e0 != cudaSuccess) return e0;
  const int hq = nh * D, nqkv = (nh + 2 * nkv) * D;
  CUtensorMap tq128, tq64, td128, td64;
  if (!make_tmap_3d(&tq128, qkv, nqkv, S, B, nqkv, 128) || !make_tmap_3d(&tq64, qkv, nqkv, S, B, nqkv, 64) ||
      !make_tmap_3d(&td128, d_o, hq, S, B, hq, 128) || !make_tmap_3d(&td64, d_o, hq, S, B, hq, 64))
    return cudaErrorInvalidValue;
  const float scale = (float)(1.0 / sqrt((double)D));
  const float scale_log2 = (float)((1.0 / sqrt((double)D)) * 1.4426950408889634);
  cudaError_t e = attention_delta(o, d_o, delta, B, S, nh, D, st);
  if (e != cudaSuccess) return e;
  const int nxb = (S + 127) / 128;
  dim3 gq((unsigned)(nxb * nh * B), 1, 1), gk((unsigned)(nxb * nkv * B), 1, 1);
  bf16* none = nullptr;
  if (ds != nullptr) {
    // dK/dV first, leaving dS^T behind; dQ is then one causally truncated batched contraction over it
    e = launch_pdl(attn_bwd_tc_kernel<D, MODE_DKV>, gk, BWD_THREADS, CK::SMEM_BYTES, st, tq128, tq64, td128, td64, lse, delta,
                   dqkv, ds, cs, sn, S, nh, nkv, B, nxb, scale, scale_log2, err);
    if (e != cudaSuccess) return e;
    return attention_dq_from_ds(ds, qkv, dqkv, cs, sn, B, S, nh, nkv, D, err, st);
  }
  e = launch_pdl(attn_bwd_tc_kernel<D, MODE_DQ>, gq, BWD_THREADS, CQ::SMEM_BYTES, st, tq128, tq64, td128, td64, lse, delta,
                 dqkv, none, cs, sn, S, nh, nkv, B, nxb, scale, scale_log2, err);
  if (e != cudaSuccess) return e;
  return launch_pdl(attn_bwd_tc_kernel<D, MODE_DKV>, gk, BWD_THREADS, CK::SMEM_BYTES, st, tq128, tq64, td128, td64, lse, delta,
                    dqkv, none, cs, sn, S, nh, nkv, B, nxb, scale, scale_log2, err);
}

static __device__ int g_attn_status;

}  // namespace

int* attention_status_word() {
  static int* addr[64] = {nullptr};
  static std::mutex mu;  // the per-device address is looked up once; callers may come from several host threads
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_attn_status) != cudaSuccess) return nullptr;
    addr[dev] = p;
  }
  return addr[dev];
}

cudaError_t attention_fwd(const bf16* qkv, bf16* o, float* lse, int B, int S, int nh, int nkv, int d, int* err,
                             cudaStream_t st) {
  if (B <= 0 || S <= 0 || nh <= 0 || nkv <= 0 || nh % nkv || !err) return cudaErrorInvalidValue;
  if (d == 64) return attention_fwd_tc_t<64>(qkv, o, lse, B, S, nh, nkv, err, st);
  if (d == 128) return attention_fwd_tc_t<128>(qkv, o, lse, B, S, nh, nkv, err, st);
  return cudaErrorInvalidValue;
}

size_t attention_bwd_ds_bytes(int B, int S, int nh) {
  if (B <= 0 || S <= 0 || nh <= 0 || S % 128 != 0) return 0;
  return (size_t)B * nh * S * S * sizeof(bf16);
}

cudaError_t attention_bwd_ws(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                             const float* cs, const float* sn, bf16* ds, size_t ds_bytes, int B, int S, int nh, int nkv, int d,
                             int* err, cudaStream_t st) {
  if (B <= 0 || S <= 0 || nh <= 0 || nkv <= 0 || nh % nkv || !err) return cudaErrorInvalidValue;
  if ((cs == nullptr) != (sn == nullptr)) return cudaErrorInvalidValue;
  const size_t need = attention_bwd_ds_bytes(B, S, nh);
  if (ds != nullptr && (need == 0 || ds_bytes < need || (reinterpret_cast<uintptr_t>(ds) & 127u) != 0)) ds = nullptr;
  if (d == 64) return attention_bwd_tc_t<64>(qkv, o, d_o, lse, delta, dqkv, cs, sn, ds, B, S, nh, nkv, err, st);
  if (d == 128) return attention_bwd_tc_t<128>(qkv, o, d_o, lse, delta, dqkv, cs, sn, ds, B, S, nh, nkv, err, st);
  return cudaErrorInvalidValue;
}

cudaError_t attention_bwd(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                          const float* cs, const float* sn, int B, int S, int nh, int nkv, int d, int* err, cudaStream_t st) {
  return attention_bwd_ws(qkv, o, d_o, lse, delta, dqkv, cs, sn, nullptr, 0, B, S, nh, nkv, d, err, st);
}

}  // namespace fs
