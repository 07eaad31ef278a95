// Causal flash attention, forward and backward, on a packed qkv buffer.
//
// Forward: online softmax over key blocks with the row reference kept as an INTEGER power of two
// (ceil of the running maximum in the log2 domain).  Rescaling by exact powers of two commutes with the
// bf16 rounding of the probabilities, so the result does not depend on the order or size of key blocks.
// LSE (natural log) is kept for the backward.
//
// Backward is deterministic (no floating-point atomics): one kernel owns query rows and accumulates dQ
// over key blocks, a second owns key rows and accumulates dK and dV over query blocks and over the query
// heads of a GQA group; a small pre-pass computes delta_i = sum_k dO_ik O_ik.  Both recompute
// P = exp(S - LSE) from the stored LSE.  dQ and dK are rotated back (RoPE backward) before their single
// rounding when tables are given.
//
// Tensor-core path of these kernels: warp-level mma.sync m16n8k16 bf16 with fp32 accumulation; all
// intermediate tiles stay in registers (S / P / dS never touch shared memory).
#include "attention.cuh"

#include <math.h>

#include <mutex>

#include "../../include/forgestep.h"

namespace fs {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  return (uint32_t)(row * (D * 2) + (((chunk) ^ (row & 7)) << 4));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// rows [row0, row0+ROWS) of a [*, D] slice (row stride ld elements) -> swizzled shared tile; rows >= row_limit are zero.
template <int D, int ROWS, int THREADS>
__device__ __forceinline__ void load_tile(uint32_t sbase, const bf16* g, long long ld, int row0, int row_limit, int tid) {
  constexpr int CH = D / 8;
#pragma unroll
  for (int i = tid; i < ROWS * CH; i += THREADS) {
    const int r = i / CH, c = i % CH;
    const int gr = row0 + r;
    const bool v = gr < row_limit;
    const bf16* src = g + (long long)(v ? gr : 0) * ld + c * 8;
    cp_async16(sbase + tile_off<D>(r, c), src, v);
  }
}

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A fragment (16 rows x 16 k) of a row-major [rows, D] tile: rows row0.., k-step ks.
template <int D>
__device__ __forceinline__ void load_a(uint32_t tile, int row0, int ks, int lane, uint32_t (&a)[4]) {
  ldsm_x4(tile + tile_off<D>(row0 + (lane & 15), ks * 2 + (lane >> 4)), a[0], a[1], a[2], a[3]);
}
// B fragments for two n-tiles (16 n) x 16 k from a tile stored [n, k] (k contiguous): {b0,b1} of n-tile 0, then of n-tile 1.
template <int D>
__device__ __forceinline__ void load_b_nk(uint32_t tile, int n0, int ks, int lane, uint32_t (&b)[4]) {
  ldsm_x4(tile + tile_off<D>(n0 + (lane & 7) + ((lane >> 4) << 3), ks * 2 + ((lane >> 3) & 1)), b[0], b[1], b[2], b[3]);
}
// B fragments for two n-tiles x 16 k from a tile stored [k, n] (n contiguous): rows k0.., column chunks 2*np, 2*np+1.
template <int D>
__device__ __forceinline__ void load_b_kn(uint32_t tile, int k0, int np, int lane, uint32_t (&b)[4]) {
  ldsm_x4_t(tile + tile_off<D>(k0 + (lane & 15), np * 2 + (lane >> 4)), b[0], b[1], b[2], b[3]);
}

// acc[NT][4] += A(rows row0.. of tile_a, all D) * B^T where B is tile_b rows n0.. (stored [n, D])
template <int D, int NT>
__device__ __forceinline__ void gemm_a_smem_b_nk(float (&acc)[NT][4], uint32_t tile_a, int row0, uint32_t tile_b, int n0,
                                                 int lane) {
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    uint32_t a[4];
    load_a<D>(tile_a, row0, ks, lane, a);
#pragma unroll
    for (int np = 0; np < NT / 2; ++np) {
      uint32_t b[4];
      load_b_nk<D>(tile_b, n0 + np * 16, ks, lane, b);
      mma16816(acc[2 * np], a, b[0], b[1]);
      mma16816(acc[2 * np + 1], a, b[2], b[3]);
    }
  }
}

// out[D/8][4] += P(16 x 16*KS, bf16 fragments pf) * B where B is tile_b rows k0.. stored [k, D]
template <int D, int KS>
__device__ __forceinline__ void gemm_a_reg_b_kn(float (&out)[D / 8][4], const uint32_t (&pf)[KS][4], uint32_t tile_b,
                                                int k0, int lane) {
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
    for (int np = 0; np < D / 16; ++np) {
      uint32_t b[4];
      load_b_kn<D>(tile_b, k0 + kk * 16, np, lane, b);
      mma16816(out[2 * np], pf[kk], b[0], b[1]);
      mma16816(out[2 * np + 1], pf[kk], b[2], b[3]);
    }
  }
}

// write a warp's 16 x D accumulator (already scaled) as bf16 into its 16 rows of a swizzled tile
template <int D>
__device__ __forceinline__ void stage_rows(uint8_t* tile, int row0, const float (&acc)[D / 8][4], int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int nt = 0; nt < D / 8; ++nt) {
    *reinterpret_cast<uint32_t*>(tile + tile_off<D>(row0 + g, nt) + t * 4) = pack_bf16(acc[nt][0], acc[nt][1]);
    *reinterpret_cast<uint32_t*>(tile + tile_off<D>(row0 + g + 8, nt) + t * 4) = pack_bf16(acc[nt][2], acc[nt][3]);
  }
}
// copy a warp's 16 staged rows to global memory, 16 bytes per lane, rows >= row_limit skipped
template <int D>
__device__ __forceinline__ void copy_rows_out(const uint8_t* tile, int row0, bf16* g, long long ld, int grow0,
                                              int row_limit, int lane) {
  constexpr int CH = D / 8;
#pragma unroll
  for (int i = lane; i < 16 * CH; i += 32) {
    const int r = i / CH, c = i % CH;
    if (grow0 + r < row_limit)
      *reinterpret_cast<uint4*>(g + (long long)(grow0 + r) * ld + c * 8) =
          *reinterpret_cast<const uint4*>(tile + tile_off<D>(row0 + r, c));
  }
}

// rotate a 16 x D accumulator by the negative RoPE angle of its rows (positions pos_g, pos_g8)
template <int D>
__device__ __forceinline__ void rope_transpose(float (&acc)[D / 8][4], const float* cs, const float* sn, int pos_g,
                                               int pos_g8, int lane) {
  const int t = lane & 3;
  constexpr int H = D / 2;
#pragma unroll
  for (int nt = 0; nt < D / 16; ++nt) {
    const int c = nt * 8 + t * 2;
    const float2 c0 = *reinterpret_cast<const float2*>(cs + (long long)pos_g * H + c);
    const float2 s0 = *reinterpret_cast<const float2*>(sn + (long long)pos_g * H + c);
    const float2 c1 = *reinterpret_cast<const float2*>(cs + (long long)pos_g8 * H + c);
    const float2 s1 = *reinterpret_cast<const float2*>(sn + (long long)pos_g8 * H + c);
    float (&lo)[4] = acc[nt];
    float (&hi)[4] = acc[nt + D / 16];
    float y1, y2;
    y1 = lo[0]; y2 = hi[0]; lo[0] = y1 * c0.x + y2 * s0.x; hi[0] = y2 * c0.x - y1 * s0.x;
    y1 = lo[1]; y2 = hi[1]; lo[1] = y1 * c0.y + y2 * s0.y; hi[1] = y2 * c0.y - y1 * s0.y;
    y1 = lo[2]; y2 = hi[2]; lo[2] = y1 * c1.x + y2 * s1.x; hi[2] = y2 * c1.x - y1 * s1.x;
    y1 = lo[3]; y2 = hi[3]; lo[3] = y1 * c1.y + y2 * s1.y; hi[3] = y2 * c1.y - y1 * s1.y;
  }
}

// ============================================================================ forward
// grid (q blocks, n_heads, B), 256 threads: 8 warps x 16 query rows; key blocks of 64.
template <int D>
__global__ void __launch_bounds__(256, 1)
attn_fwd_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ o, float* __restrict__ lse, int S, int n_heads,
                int n_kv, float scale_log2) {
  constexpr int BMQ = 128, BNK = 64, TILE_Q = BMQ * D * 2, TILE_K = BNK * D * 2;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* sQ = smem;
  uint8_t* sK = smem + TILE_Q;               // two buffers
  uint8_t* sV = smem + TILE_Q + 2 * TILE_K;  // two buffers
  const uint32_t uQ = smem_u32(sQ), uK = smem_u32(sK), uV = smem_u32(sV);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int qb = gridDim.x - 1 - blockIdx.x;  // heaviest blocks first
  const int n = blockIdx.y, b = blockIdx.z;
  const int kvh = n / (n_heads / n_kv);
  const int hq = n_heads * D, hkv = n_kv * D;
  const long long ld = hq + 2 * hkv;
  const bf16* qbase = qkv + (long long)b * S * ld + n * D;
  const bf16* kbase = qkv + (long long)b * S * ld + hq + kvh * D;
  const bf16* vbase = kbase + hkv;
  const int q0 = qb * BMQ;
  const int kv_end = min(S, q0 + BMQ);
  const int nb = (kv_end + BNK - 1) / BNK;

  load_tile<D, BMQ, 256>(uQ, qbase, ld, q0, S, tid);
  load_tile<D, BNK, 256>(uK, kbase, ld, 0, S, tid);
  load_tile<D, BNK, 256>(uV, vbase, ld, 0, S, tid);
  cp_async_commit();

  uint32_t qf[D / 16][4];
  float oacc[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float mref[2] = {-INFINITY, -INFINITY};  // integer reference (log2 domain) of rows g, g+8
  float lsum[2] = {0.f, 0.f};              // this thread's share of the row sums
  const int row_g = q0 + warp * 16 + g;

  for (int j = 0; j < nb; ++j) {
    cp_async_wait_all();
    __syncthreads();
    if (j == 0) {
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) load_a<D>(uQ, warp * 16, ks, lane, qf[ks]);
    }
    if (j + 1 < nb) {
      load_tile<D, BNK, 256>(uK + ((j + 1) & 1) * TILE_K, kbase, ld, (j + 1) * BNK, S, tid);
      load_tile<D, BNK, 256>(uV + ((j + 1) & 1) * TILE_K, vbase, ld, (j + 1) * BNK, S, tid);
      cp_async_commit();
    }
    const int k0 = j * BNK;
    if (k0 > q0 + warp * 16 + 15) continue;  // every key of this block is in the future of this warp's rows
    const uint32_t tK = uK + (j & 1) * TILE_K, tV = uV + (j & 1) * TILE_K;

    float s[BNK / 8][4];
#pragma unroll
    for (int i = 0; i < BNK / 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < BNK / 16; ++np) {
        uint32_t bfr[4];
        load_b_nk<D>(tK, np * 16, ks, lane, bfr);
        mma16816(s[2 * np], qf[ks], bfr[0], bfr[1]);
        mma16816(s[2 * np + 1], qf[ks], bfr[2], bfr[3]);
      }
    }
    const bool need_mask = k0 + BNK - 1 > q0 + warp * 16;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < BNK / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float v = s[nt][e] * scale_log2;
        if (need_mask) {
          const int key = k0 + nt * 8 + t * 2 + (e & 1);
          const int row = row_g + ((e >> 1) << 3);
          if (key > row) v = -INFINITY;
        }
        s[nt][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float alpha[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      const float mnew = fmaxf(mref[r], ceilf(mx[r]));
      alpha[r] = exp2f(mref[r] - mnew);  // exact power of two (0 on the first block)
      mref[r] = mnew;
      lsum[r] *= alpha[r];
    }
    uint32_t pf[BNK / 16][4];
#pragma unroll
    for (int nt = 0; nt < BNK / 8; ++nt) {
      const float p0 = exp2f(s[nt][0] - mref[0]);
      const float p1 = exp2f(s[nt][1] - mref[0]);
      const float p2 = exp2f(s[nt][2] - mref[1]);
      const float p3 = exp2f(s[nt][3] - mref[1]);
      lsum[0] += p0 + p1;
      lsum[1] += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
      oacc[i][0] *= alpha[0]; oacc[i][1] *= alpha[0];
      oacc[i][2] *= alpha[1]; oacc[i][3] *= alpha[1];
    }
    gemm_a_reg_b_kn<D, BNK / 16>(oacc, pf, tV, 0, lane);
  }

#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 1);
    lsum[r] += __shfl_xor_sync(0xffffffffu, lsum[r], 2);
  }
  const float inv0 = 1.0f / lsum[0], inv1 = 1.0f / lsum[1];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    oacc[i][0] *= inv0; oacc[i][1] *= inv0;
    oacc[i][2] *= inv1; oacc[i][3] *= inv1;
  }
  if (t == 0) {
    float* l = lse + ((long long)b * n_heads + n) * S;
    if (row_g < S) l[row_g] = (mref[0] + log2f(lsum[0])) * kLn2;
    if (row_g + 8 < S) l[row_g + 8] = (mref[1] + log2f(lsum[1])) * kLn2;
  }
  __syncwarp();
  stage_rows<D>(sQ, warp * 16, oacc, lane);  // the Q tile is dead: every warp holds its fragments in registers
  __syncwarp();
  copy_rows_out<D>(sQ, warp * 16, o + (long long)b * S * hq + n * D, hq, q0 + warp * 16, S, lane);
}

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

// ============================================================================ backward: dQ
// grid (q blocks, n_heads, B), 256 threads: 8 warps x 16 query rows; key blocks of 64.
template <int D>
__global__ void __launch_bounds__(256, 1)
attn_bwd_dq_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ d_o, const float* __restrict__ lse,
                   const float* __restrict__ delta, bf16* __restrict__ dqkv, const float* __restrict__ rope_cos,
                   const float* __restrict__ rope_sin, int S, int n_heads, int n_kv, float scale, float scale_log2) {
  constexpr int BMQ = 128, BNK = 64, TILE_Q = BMQ * D * 2, TILE_K = BNK * D * 2;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* sQ = smem;
  const uint32_t uQ = smem_u32(smem), uDO = uQ + TILE_Q, uK = uDO + TILE_Q, uV = uK + 2 * TILE_K;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int qb = gridDim.x - 1 - blockIdx.x;
  const int n = blockIdx.y, b = blockIdx.z;
  const int kvh = n / (n_heads / n_kv);
  const int hq = n_heads * D, hkv = n_kv * D;
  const long long ld = hq + 2 * hkv;
  const bf16* qbase = qkv + (long long)b * S * ld + n * D;
  const bf16* kbase = qkv + (long long)b * S * ld + hq + kvh * D;
  const bf16* vbase = kbase + hkv;
  const bf16* dobase = d_o + (long long)b * S * hq + n * D;
  const int q0 = qb * BMQ;
  const int kv_end = min(S, q0 + BMQ);
  const int nb = (kv_end + BNK - 1) / BNK;

  load_tile<D, BMQ, 256>(uQ, qbase, ld, q0, S, tid);
  load_tile<D, BMQ, 256>(uDO, dobase, hq, q0, S, tid);
  load_tile<D, BNK, 256>(uK, kbase, ld, 0, S, tid);
  load_tile<D, BNK, 256>(uV, vbase, ld, 0, S, tid);
  cp_async_commit();

  const int row_g = q0 + warp * 16 + g;
  const long long stat = ((long long)b * n_heads + n) * S;
  float lse2[2], dl[2];
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row_g + 8 * r;
    lse2[r] = row < S ? lse[stat + row] * kLog2e : 0.f;
    dl[r] = row < S ? delta[stat + row] : 0.f;
  }
  float dq[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f;

  for (int j = 0; j < nb; ++j) {
    cp_async_wait_all();
    __syncthreads();
    if (j + 1 < nb) {
      load_tile<D, BNK, 256>(uK + ((j + 1) & 1) * TILE_K, kbase, ld, (j + 1) * BNK, S, tid);
      load_tile<D, BNK, 256>(uV + ((j + 1) & 1) * TILE_K, vbase, ld, (j + 1) * BNK, S, tid);
      cp_async_commit();
    }
    const int k0 = j * BNK;
    if (k0 > q0 + warp * 16 + 15) continue;
    const uint32_t tK = uK + (j & 1) * TILE_K, tV = uV + (j & 1) * TILE_K;

    float s[BNK / 8][4], dp[BNK / 8][4];
#pragma unroll
    for (int i = 0; i < BNK / 8; ++i) {
      s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
      dp[i][0] = dp[i][1] = dp[i][2] = dp[i][3] = 0.f;
    }
    gemm_a_smem_b_nk<D, BNK / 8>(s, uQ, warp * 16, tK, 0, lane);
    gemm_a_smem_b_nk<D, BNK / 8>(dp, uDO, warp * 16, tV, 0, lane);
    const bool need_mask = k0 + BNK - 1 > q0 + warp * 16;
    uint32_t dsf[BNK / 16][4];
#pragma unroll
    for (int nt = 0; nt < BNK / 8; ++nt) {
      float ds[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = e >> 1;
        float p = exp2f(s[nt][e] * scale_log2 - lse2[r]);
        if (need_mask) {
          const int key = k0 + nt * 8 + t * 2 + (e & 1);
          if (key > row_g + 8 * r) p = 0.f;
        }
        ds[e] = p * (dp[nt][e] - dl[r]);
      }
      dsf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(ds[0], ds[1]);
      dsf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(ds[2], ds[3]);
    }
    gemm_a_reg_b_kn<D, BNK / 16>(dq, dsf, tK, 0, lane);
  }

#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    dq[i][0] *= scale; dq[i][1] *= scale; dq[i][2] *= scale; dq[i][3] *= scale;
  }
  if (rope_cos != nullptr)
    rope_transpose<D>(dq, rope_cos, rope_sin, min(row_g, S - 1), min(row_g + 8, S - 1), lane);
  __syncwarp();
  stage_rows<D>(sQ, warp * 16, dq, lane);  // each warp only ever read its own 16 rows of the Q tile
  __syncwarp();
  copy_rows_out<D>(sQ, warp * 16, dqkv + (long long)b * S * ld + n * D, ld, q0 + warp * 16, S, lane);
}

// ============================================================================ backward: dK, dV
// grid (key blocks of 64, n_kv, B), 128 threads: 4 warps x 16 key rows; query blocks of 64, visited for every
// query head of the group in a fixed order.
template <int D>
__global__ void __launch_bounds__(128, 1)
attn_bwd_dkv_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ d_o, const float* __restrict__ lse,
                    const float* __restrict__ delta, bf16* __restrict__ dqkv, const float* __restrict__ rope_cos,
                    const float* __restrict__ rope_sin, int S, int n_heads, int n_kv, float scale, float scale_log2) {
  constexpr int BNK = 64, BMQ = 64, TILE = 64 * D * 2;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* sK = smem;
  uint8_t* sV = smem + TILE;
  const uint32_t uK = smem_u32(smem), uV = uK + TILE, uQ = uV + TILE, uDO = uQ + 2 * TILE;
  float* s_lse = reinterpret_cast<float*>(smem + 6 * TILE);  // [2][64]
  float* s_dl = s_lse + 2 * BMQ;                             // [2][64]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int kb = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int n_rep = n_heads / n_kv;
  const int hq = n_heads * D, hkv = n_kv * D;
  const long long ld = hq + 2 * hkv;
  const bf16* kbase = qkv + (long long)b * S * ld + hq + kvh * D;
  const bf16* vbase = kbase + hkv;
  const int k0 = kb * BNK;
  const int nqb = (S + BMQ - 1) / BMQ;
  const int per_head = nqb - kb;  // query blocks kb .. nqb-1 see these keys
  const int iters = per_head * n_rep;

  auto issue = [&](int it) {
    const int rep = it / per_head, qb = kb + it % per_head;
    const int n = kvh * n_rep + rep;
    const int buf = it & 1;
    load_tile<D, BMQ, 128>(uQ + buf * TILE, qkv + (long long)b * S * ld + n * D, ld, qb * BMQ, S, tid);
    load_tile<D, BMQ, 128>(uDO + buf * TILE, d_o + (long long)b * S * hq + n * D, hq, qb * BMQ, S, tid);
    if (tid < BMQ) {
      const int row = qb * BMQ + tid;
      const long long stat = ((long long)b * n_heads + n) * S;
      s_lse[buf * BMQ + tid] = row < S ? lse[stat + row] * kLog2e : 0.f;
      s_dl[buf * BMQ + tid] = row < S ? delta[stat + row] : 0.f;
    }
  };

  load_tile<D, BNK, 128>(uK, kbase, ld, k0, S, tid);
  load_tile<D, BNK, 128>(uV, vbase, ld, k0, S, tid);
  issue(0);
  cp_async_commit();

  float dk[D / 8][4], dv[D / 8][4];
#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
    dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
  }
  const int key_g = k0 + warp * 16 + g;

  for (int it = 0; it < iters; ++it) {
    cp_async_wait_all();
    __syncthreads();
    if (it + 1 < iters) {
      issue(it + 1);
      cp_async_commit();
    }
    const int qb = kb + it % per_head;
    const int qrow0 = qb * BMQ;
    const int buf = it & 1;
    const uint32_t tQ = uQ + buf * TILE, tDO = uDO + buf * TILE;
    const float* lq = s_lse + buf * BMQ;
    const float* dlq = s_dl + buf * BMQ;
    const bool diag = qb == kb;

#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int c0 = half * 32;  // first query of this half within the tile
      if (diag && qrow0 + c0 + 31 < k0 + warp * 16) continue;  // all 32 queries precede this warp's keys
      float st[4][4], dpt[4][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        st[i][0] = st[i][1] = st[i][2] = st[i][3] = 0.f;
        dpt[i][0] = dpt[i][1] = dpt[i][2] = dpt[i][3] = 0.f;
      }
      gemm_a_smem_b_nk<D, 4>(st, uK, warp * 16, tQ, c0, lane);     // S^T = K Q^T
      gemm_a_smem_b_nk<D, 4>(dpt, uV, warp * 16, tDO, c0, lane);   // dP^T = V dO^T
      uint32_t pf[2][4], dsf[2][4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        float p[4], ds[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int qc = c0 + nt * 8 + t * 2 + (e & 1);  // query column within the tile
          const int query = qrow0 + qc;
          const int key = key_g + ((e >> 1) << 3);
          float pv = exp2f(st[nt][e] * scale_log2 - lq[qc]);
          if (query < key || query >= S) pv = 0.f;
          p[e] = pv;
          ds[e] = pv * (dpt[nt][e] - dlq[qc]);
        }
        pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p[0], p[1]);
        pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p[2], p[3]);
        dsf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(ds[0], ds[1]);
        dsf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(ds[2], ds[3]);
      }
      gemm_a_reg_b_kn<D, 2>(dv, pf, tDO, c0, lane);  // dV += P^T dO
      gemm_a_reg_b_kn<D, 2>(dk, dsf, tQ, c0, lane);  // dK += dS^T Q
    }
  }

#pragma unroll
  for (int i = 0; i < D / 8; ++i) {
    dk[i][0] *= scale; dk[i][1] *= scale; dk[i][2] *= scale; dk[i][3] *= scale;
  }
  if (rope_cos != nullptr)
    rope_transpose<D>(dk, rope_cos, rope_sin, min(key_g, S - 1), min(key_g + 8, S - 1), lane);
  __syncthreads();  // all warps are done reading K and V tiles (as A operands) before they are overwritten
  stage_rows<D>(sK, warp * 16, dk, lane);
  stage_rows<D>(sV, warp * 16, dv, lane);
  __syncwarp();
  bf16* dkbase = dqkv + (long long)b * S * ld + hq + kvh * D;
  copy_rows_out<D>(sK, warp * 16, dkbase, ld, k0 + warp * 16, S, lane);
  copy_rows_out<D>(sV, warp * 16, dkbase + hkv, ld, k0 + warp * 16, S, lane);
}

template <int D>
cudaError_t set_smem(const void* fn, int bytes) {
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

}  // namespace


template <int D>
static cudaError_t attention_fwd_t(const bf16* qkv, bf16* o, float* lse, int B, int S, int nh, int nkv, cudaStream_t st) {
  constexpr int smem = 128 * D * 2 + 4 * 64 * D * 2;
  static bool once = false;
  if (!once) {
    cudaError_t e = set_smem<D>((const void*)attn_fwd_kernel<D>, smem);
    if (e != cudaSuccess) return e;
    once = true;
  }
  const float scale_log2 = (float)((1.0 / sqrt((double)D)) * 1.4426950408889634);
  dim3 grid((S + 127) / 128, nh, B);
  attn_fwd_kernel<D><<<grid, 256, smem, st>>>(qkv, o, lse, S, nh, nkv, scale_log2);
  return cudaGetLastError();
}

cudaError_t attention_fwd(const bf16* qkv, bf16* o, float* lse, int B, int S, int nh, int nkv, int d, cudaStream_t st) {
  if (B <= 0 || S <= 0 || nh <= 0 || nkv <= 0 || nh % nkv) return cudaErrorInvalidValue;
  if (d == 64) return attention_fwd_t<64>(qkv, o, lse, B, S, nh, nkv, st);
  if (d == 128) return attention_fwd_t<128>(qkv, o, lse, B, S, nh, nkv, st);
  return cudaErrorInvalidValue;
}

template <int D>
static cudaError_t attention_bwd_t(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta,
                                   bf16* dqkv, const float* cs, const float* sn, int B, int S, int nh, int nkv,
                                   cudaStream_t st) {
  constexpr int smem_dq = 2 * 128 * D * 2 + 4 * 64 * D * 2;
  constexpr int smem_dkv = 6 * 64 * D * 2 + 4 * 64 * 4;
  static bool once = false;
  if (!once) {
    cudaError_t e = set_smem<D>((const void*)attn_bwd_dq_kernel<D>, smem_dq);
    if (e != cudaSuccess) return e;
    e = set_smem<D>((const void*)attn_bwd_dkv_kernel<D>, smem_dkv);
    if (e != cudaSuccess) return e;
    once = true;
  }
  const float scale = (float)(1.0 / sqrt((double)D));
  const float scale_log2 = (float)((1.0 / sqrt((double)D)) * 1.4426950408889634);
  const long long warps = (long long)B * S * nh;
  const int blocks = (int)((warps * 32 + 255) / 256);
  attn_delta_kernel<D><<<blocks, 256, 0, st>>>(o, d_o, delta, B, S, nh);
  dim3 gq((S + 127) / 128, nh, B);
  attn_bwd_dq_kernel<D><<<gq, 256, smem_dq, st>>>(qkv, d_o, lse, delta, dqkv, cs, sn, S, nh, nkv, scale, scale_log2);
  dim3 gk((S + 63) / 64, nkv, B);
  attn_bwd_dkv_kernel<D><<<gk, 128, smem_dkv, st>>>(qkv, d_o, lse, delta, dqkv, cs, sn, S, nh, nkv, scale, scale_log2);
  return cudaGetLastError();
}

cudaError_t attention_bwd(const bf16* qkv, const bf16* o, const bf16* d_o, const float* lse, float* delta, bf16* dqkv,
                          const float* cs, const float* sn, int B, int S, int nh, int nkv, int d, cudaStream_t st) {
  if (B <= 0 || S <= 0 || nh <= 0 || nkv <= 0 || nh % nkv) return cudaErrorInvalidValue;
  if ((cs == nullptr) != (sn == nullptr)) return cudaErrorInvalidValue;
  if (d == 64) return attention_bwd_t<64>(qkv, o, d_o, lse, delta, dqkv, cs, sn, B, S, nh, nkv, st);
  if (d == 128) return attention_bwd_t<128>(qkv, o, d_o, lse, delta, dqkv, cs, sn, B, S, nh, nkv, st);
  return cudaErrorInvalidValue;
}

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
  cudaError_t e;
  if (fs::g_attention_impl) {
    int* status = fs::attention_status_word();
    if (!status) return FT_ECUDA;
    e = fs::attention_bwd_tc(reinterpret_cast<const fs::bf16*>(dev_qkv), reinterpret_cast<const fs::bf16*>(dev_o),
                             reinterpret_cast<const fs::bf16*>(dev_do), dev_lse, delta,
                             reinterpret_cast<fs::bf16*>(dev_dqkv), dev_cos, dev_sin, B, S, n_heads, n_kv_heads, head_dim,
                             status, reinterpret_cast<cudaStream_t>(stream));
  } else {
    e = fs::attention_bwd(reinterpret_cast<const fs::bf16*>(dev_qkv), reinterpret_cast<const fs::bf16*>(dev_o),
                          reinterpret_cast<const fs::bf16*>(dev_do), dev_lse, delta,
                          reinterpret_cast<fs::bf16*>(dev_dqkv), dev_cos, dev_sin, B, S, n_heads, n_kv_heads, head_dim,
                          reinterpret_cast<cudaStream_t>(stream));
  }
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}
