// dQ of the attention backward as one batched, causally truncated contraction over the stored dS^T tiles:
//   dQ[b, h, i, :] = scale * sum_{j <= i} dS[b, h, i, j] K[b, kv(h), j, :]
// The dK/dV kernel computes dS (bf16) anyway; when it also writes its tiles to a scratch array, dQ needs neither S nor
// dP again: 5 tile products per (query block, key block) pair in the whole backward pass instead of 7, and every dS
// value is rounded exactly once for both of its uses.  Each dQ element is the sum of one CTA's MMAs in a fixed order,
// so the result is deterministic without atomics.
//
// Scratch layout: element (z = b n_h + h, key j, query i) at ((z * S/32 + i / 32) * S + j) * 32 + i % 32, i.e. 32-query
// chunks [z][i / 32][j][32].  A thread of the dK/dV kernel (one key, 32 queries) then stores one contiguous 64-byte
// row, its warp a 2 KiB run, and a TMA box of 64 keys x 4 chunks lands in shared memory as the MN-major operand layout
// of the 64-byte swizzle (4 blocks of [64 keys][64 bytes]).  Measured against the alternatives at B 4, S 2048, 16/8
// heads of 128: row-major dS^T (128-byte swizzle) costs the dK/dV kernel 40 us of scattered 32-byte stores; 16-query
// chunks (32-byte swizzle) give back those 40 us but slow this kernel's TMA loads by 15 us; this layout loses neither.
//
// Persistent, warp-specialised like the GEMM: warp 0 TMA producer, warp 1 MMA issuer, warps 2..5 epilogue (scale,
// inverse rotation, one rounding to bf16).  A tile is 128 queries of one (batch, head); its K range ends at the diagonal.
// Both operands are MN-major in memory (the contraction index j is the row index of dS^T and of K), as in a weight
// gradient.  Accumulators are double-buffered in TMEM.
#include "attention.cuh"

#include "tmap.cuh"

namespace fs {

namespace {

constexpr int DQ_THREADS = 192;
constexpr int DQ_BM = 128;  // queries per tile
constexpr int DQ_BK = 64;   // keys per pipeline stage

template <int D>
struct DqCfg {
  static constexpr int A_BYTES = DQ_BK * DQ_BM * 2;  // one box of dS^T: 4 chunks of [64 keys][32 queries]
  static constexpr int B_BYTES = DQ_BK * D * 2;      // D / 64 boxes of K
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = 3;
  static constexpr int OFF_BAR = STAGES * STAGE_BYTES;
  static constexpr int SMEM_BYTES = OFF_BAR + 128;
  static constexpr int TMEM_COLS = 2 * D;
};

template <int D>
__global__ void __launch_bounds__(DQ_THREADS, 2)
attn_dq_gemm_kernel(const __grid_constant__ CUtensorMap tm_ds, const __grid_constant__ CUtensorMap tm_qkv,
                    bf16* __restrict__ dqkv, const float* __restrict__ rope_cos, const float* __restrict__ rope_sin, int B,
                    int S, int n_heads, int n_kv, float scale, int* err) {
  using C = DqCfg<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
  const uint32_t bar0 = sbase + C::OFF_BAR;
  // barrier slots: [0,S) full, [S,2S) empty, 2S+{0,1} accumulator full, 2S+{2,3} accumulator empty
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if ((sbase & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicExch(err, (int)ERR_BAD_ALIGNMENT);
    return;
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_ds);
    tma_prefetch_desc(&tm_qkv);
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

  const int tiles_q = S / DQ_BM;
  const int nz = B * n_heads;
  const int ntiles = tiles_q * nz;
  const int n_rep = n_heads / n_kv;
  const int hq = n_heads * D;
  const long long ld = (long long)(n_heads + 2 * n_kv) * D;
  // tile t: the longest K ranges (last query blocks) first; neighbouring CTAs take the same query block of different heads
  auto tile_of = [&](int t, int& qt, int& z) {
    qt = tiles_q - 1 - t / nz;
    z = t % nz;
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        int qt, z;
        tile_of(t, qt, z);
        const int b = z / n_heads, h = z % n_heads, kvh = h / n_rep;
        const int q0 = qt * DQ_BM, kblocks = (q0 + DQ_BM) / DQ_BK;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, err, kWaitLimitCycles, 0x51)) { ok = false; break; }
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, C::STAGE_BYTES);
          const uint32_t a_dst = sbase + stage * C::STAGE_BYTES;
          const uint32_t b_dst = a_dst + C::A_BYTES;
          tma_load_4d(a_dst, &tm_ds, fb, 0, kb * DQ_BK, q0 / 32, z);  // 4 chunks of [64 keys][32 queries]
#pragma unroll
          for (int j = 0; j < D / 64; ++j) tma_load_3d(b_dst + j * 8192, &tm_qkv, fb, hq + kvh * D + 64 * j, kb * DQ_BK, b);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // fp32 accumulate, bf16 operands, both MN-major, N = D, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(D >> 3) << 17) |
                             ((uint32_t)(DQ_BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        int qt, z;
        tile_of(t, qt, z);
        const int kblocks = (qt * DQ_BM + DQ_BM) / DQ_BK;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, err, kWaitLimitCycles, 0x52)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * D);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, err, kWaitLimitCycles, 0x53)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = sbase + stage * C::STAGE_BYTES;
          const uint32_t b_addr = a_addr + C::A_BYTES;
#pragma unroll
          for (int k = 0; k < DQ_BK / 16; ++k) {
            const uint64_t adesc = umma_desc_sw64(a_addr + k * 1024, 4096, 512);
            const uint64_t bdesc = umma_desc_sw128(b_addr + k * 2048, 8192, 1024);
            umma_bf16(d_tmem, adesc, bdesc, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    constexpr int H = D / 2;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
      int qt, z;
      tile_of(t, qt, z);
      const int b = z / n_heads, h = z % n_heads;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, err, kWaitLimitCycles, 0x54);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = qt * DQ_BM + q * 32 + lane;  // query position (S is a multiple of 128: always in range)
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * D);
      bf16* dst = dqkv + ((long long)b * S + row) * ld + h * D;
      for (int i0 = 0; i0 < H; i0 += 32) {
        uint32_t r1[32], r2[32];
        tmem_ld32(taddr + (uint32_t)i0, r1);
        tmem_ld32(taddr + (uint32_t)(H + i0), r2);
        tmem_ld_wait();
        float lo[32], hi[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          lo[i] = __uint_as_float(r1[i]) * scale;
          hi[i] = __uint_as_float(r2[i]) * scale;
        }
        if (rope_cos != nullptr) {  // backward of the rotation: its transpose, on the unrounded sums
          const float* cs = rope_cos + (long long)row * H + i0;
          const float* sn = rope_sin + (long long)row * H + i0;
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
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
#pragma unroll
        for (int i = 0; i < 32; i += 8) {
          uint4 o1, o2;
          o1.x = pack_bf16(lo[i], lo[i + 1]); o1.y = pack_bf16(lo[i + 2], lo[i + 3]);
          o1.z = pack_bf16(lo[i + 4], lo[i + 5]); o1.w = pack_bf16(lo[i + 6], lo[i + 7]);
          o2.x = pack_bf16(hi[i], hi[i + 1]); o2.y = pack_bf16(hi[i + 2], hi[i + 3]);
          o2.z = pack_bf16(hi[i + 4], hi[i + 5]); o2.w = pack_bf16(hi[i + 6], hi[i + 7]);
          *reinterpret_cast<uint4*>(dst + i0 + i) = o1;
          *reinterpret_cast<uint4*>(dst + H + i0 + i) = o2;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  // teardown: everyone meets here, also after a wait that ran out
  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM are released
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
cudaError_t launch_dq(const bf16* ds, const bf16* qkv, bf16* dqkv, const float* cs, const float* sn, int B, int S, int nh,
                      int nkv, int* err, cudaStream_t st) {
  using C = DqCfg<D>;
  static unsigned long long smem_set = 0;
  cudaError_t e0 = ensure_dynamic_smem(attn_dq_gemm_kernel<D>, C::SMEM_BYTES, smem_set);
  if (e0 != cudaSuccess) return e0;
  const int nqkv = (nh + 2 * nkv) * D;
  CUtensorMap tm_ds, tm_qkv;
  if (!make_tmap_ds_chunked(&tm_ds, ds, S, (uint64_t)B * nh) || !make_tmap_3d(&tm_qkv, qkv, nqkv, S, B, nqkv, 64))
    return cudaErrorInvalidValue;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int ntiles = (S / DQ_BM) * B * nh;
  const int grid = ntiles < 2 * sms ? ntiles : 2 * sms;
  const float scale = (float)(1.0 / sqrt((double)D));
  return launch_pdl(attn_dq_gemm_kernel<D>, grid, DQ_THREADS, C::SMEM_BYTES, st, tm_ds, tm_qkv, dqkv, cs, sn, B, S, nh, nkv,
                    scale, err);
}

}  // namespace

cudaError_t attention_dq_from_ds(const bf16* ds, const bf16* qkv, bf16* dqkv, const float* rope_cos, const float* rope_sin,
                                 int B, int S, int nh, int nkv, int d, int* err, cudaStream_t st) {
  if (S % DQ_BM != 0 || nh % nkv != 0) return cudaErrorInvalidValue;
  if (d == 64) return launch_dq<64>(ds, qkv, dqkv, rope_cos, rope_sin, B, S, nh, nkv, err, st);
  if (d == 128) return launch_dq<128>(ds, qkv, dqkv, rope_cos, rope_sin, B, S, nh, nkv, err, st);
  return cudaErrorInvalidValue;
}

}  // namespace fs
