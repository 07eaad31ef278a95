// bf16 GEMM family on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM, operands staged in
// shared memory by TMA with the 128-byte swizzle).  One persistent, warp-specialised kernel:
//   warp 0      : TMA producer (one elected thread)
//   warp 1      : TMEM allocator + MMA issuer (one elected thread)
//   warps 2..5  : epilogue, one TMEM lane quarter each; the accumulator is double-buffered in TMEM so the
//                 epilogue of tile i overlaps the main loop of tile i+1.
// Computes C[M,N] = sum_k A[m,k] B[n,k] for the three operand layouts a training step needs
// (forward: both k-contiguous; data gradient: B mn-contiguous; weight gradient: both mn-contiguous, i.e. the
// contraction runs over the rows of the stored activations) without materialising any transpose.
#include "gemm.cuh"

#include "adamw_math.cuh"
#include "elementwise.cuh"
#include "tmap.cuh"

namespace fs {

int g_pdl = 1;
int g_gemm_balanced = 1;  // development knob: 0 = always the round-robin tile schedule
int g_gemm_swiglu_tma = 1;  // development knob: 0 = SwiGLU-backward epilogue with per-thread loads and stores
int g_gemm_group = 1;       // development knob: 0 = never two weight gradients in one launch
int g_gemm_tma_out = 1;     // development knob: 0 = plain bf16 epilogue with per-thread stores

namespace {

constexpr size_t kScratchFlagFloats = 256;

constexpr int BM = 128;
constexpr int BK = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int A_BYTES = BM * BK * 2;
constexpr int CHUNK_BYTES = 64 * BK * 2;  // one 64 x 64 box of an mn-major operand
constexpr int GEMM_THREADS = 192;

// Per epilogue warp, a 32 x 32 fp32 staging tile that turns "one thread per output row" into coalesced 128-byte row
// segments.  The 16-byte column group j of row r sits at group j ^ (r & 7): conflict-free both for a thread writing
// its row and for 8 lanes reading one row.
constexpr int EPI_STAGE_FLOATS = 32 * 32;
constexpr int EPI_WARPS_MAX = 8;
constexpr int EPI_STAGE_BYTES = EPI_WARPS_MAX * EPI_STAGE_FLOATS * 4;

template <int BN>
struct Cfg {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : 6;
  static constexpr int TMEM_COLS = 2 * BN;
  static constexpr int BAR_BYTES = 256;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + BAR_BYTES + EPI_STAGE_BYTES + 1024;  // + slack to align to 1024
};

struct GemmDev {
  void* C;
  const bf16* resid;
  bf16* gu;
  const float* rope_cos;
  const float* rope_sin;
  int* err;
  long long ldc;
  int M, N, K;
  int epi;
  int seq, head_dim, rope_cols, d_ffn;
  long long rope_ld;
  int panel;               // tile numbering (see tile_coords)
  float alpha;             // accumulator scale (1: off)
  int wide_store;          // 1: C, ldc and N allow 32-byte stores (bf16 output)
  int swiglu_tma;          // SwiGLU-backward epilogue of the pair kernel: gate/up in and d_gate/d_up out as TMA tiles
  int tma_out;             // plain bf16 epilogue of the pair kernel: output tiles leave as TMA stores (AuxMaps::m1 = C)
  // grouped launch (pair kernel, weight gradients): tiles [0, g_tiles0) are this problem's, the tiles after them belong to
  // a second output with the same K whose operand maps travel in AuxMaps and whose fields below replace C, ldc, M, N,
  // panel, alpha and the AdamW pointers in its tiles' loads and epilogues (g_tiles0 = 0: one problem)
  int g_tiles0;
  int g_M, g_N, g_panel;
  long long g_ldc;
  void* g_C;
  float g_alpha;
  float* g_adam_p;
  float* g_adam_m;
  float* g_adam_v;
  bf16* g_adam_pb;
  float* qk_r;             // per-head QK-Norm in the RoPE epilogue (null: off)
  const bf16* qk_gain_q;
  const bf16* qk_gain_k;
  int n_q_heads;
  float qk_eps;
  int ksplit;              // > 1: the K blocks are divided over ksplit work units per output tile
  long long split_stride;  // elements between the partial outputs of consecutive K parts
  int balanced;            // 1: the last partial wave of tiles is divided along K and runs first (see WorkIter)
  int sw_first;            // balanced: first tile of the divided wave (tiles before it run whole, round-robin)
  int sw_parts;            // balanced: K parts per tile of the divided wave
  int sw_kpb;              // balanced: K blocks per part
  int* flags;              // balanced: one arrival counter per pair (zero between launches)
  float* slots;            // balanced: one fp32 partial tile [256][256] per pair
  // fused AdamW (null adam_p: off)
  float* adam_p;
  float* adam_m;
  float* adam_v;
  bf16* adam_pb;
  const StepScalars* adam_sc;
  float* adam_sq;
  float adam_lr, adam_beta1, adam_beta2, adam_eps, adam_wd;
  // streaming cross-entropy (CE instantiation of the pair kernel only)
  int ce_mode, ce_tiles;
  float2* ce_part;
  float* ce_zy;
  const float* ce_lse;
  const int32_t* ce_labels;
  const StepScalars* ce_sc;
  float ce_scale;
};

__device__ __forceinline__ AdamCoef adam_coef(const GemmDev& p) {
  return make_adam_coef(p.adam_lr, p.adam_beta1, p.adam_beta2, p.adam_eps, p.adam_sc->bc1, p.adam_sc->bc2);
}

// Fused AdamW: the epilogue streams master, moments (and, when accumulating, the earlier gradient) of its block with
// few loads in flight, too few to cover DRAM latency.  Each lane therefore asks L2, one 32-column chunk ahead, for the
// 128-byte line of every stream at (its row, that chunk).  (Plain prefetch instructions: bulk prefetches go through
// the TMA unit and were measured to slow the operand loads of the main loop.)
__device__ __forceinline__ void adam_prefetch_chunk(const GemmDev& p, const void* cptr, int row, int gc) {
  if (row >= p.M || gc >= p.N) return;
  const long long o = (long long)row * p.ldc + gc;
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p.adam_p + o));
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p.adam_m + o));
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p.adam_v + o));
  if (p.epi == EPI_F32_ACC) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const float*>(cptr) + o));
}

// Tile index -> (row tile, column tile).  panel = 0: row-fastest.  The ~74 tiles in flight then span every row tile and
// two or three column tiles, so each wave re-reads the whole row operand A: fine while A stays in L2 (a wave then streams
// very little of B).  panel = 1, chosen by the launcher when A is too large for that (> 48 MB): column-fastest inside
// panels of kPanel column tiles, so the tiles in flight form a block of about 9 x 8 and a wave streams 17 tile-widths of
// operand rows per K block instead of 34 (measured on a data-gradient GEMM with a 184 MB operand: DRAM reads down from
// 900 to 380 MB, 6.5 % faster; on the gate/up GEMM, whose operands fit in L2, the row-fastest order is 1 % faster).
constexpr int kPanel = 8;
// SwiGLU-backward epilogue: ask for this thread's row of gate and up, columns [gc, gc + ncols), to be brought into L2
// while the tile's contraction still runs (they were written a whole forward pass ago and come from HBM).
__device__ __forceinline__ void swiglu_bwd_prefetch(const GemmDev& p, int row, int gc, int ncols) {
  if (row >= p.M) return;
  const bf16* g = p.gu + (long long)row * (2LL * p.d_ffn) + gc;
  for (int c = 0; c < ncols && gc + c < p.N; c += 64) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(g + c));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(g + p.d_ffn + c));
  }
}

__device__ __forceinline__ void tile_coords(int panel, int tile, int tiles_m, int tiles_n, int& mi, int& ni) {
  if (!panel) {
    ni = tile / tiles_m;
    mi = tile - ni * tiles_m;
    return;
  }
  const int per_panel = kPanel * tiles_m;
  const int pn = tile / per_panel, r = tile - pn * per_panel;
  const int w = min(kPanel, tiles_n - pn * kPanel);
  mi = r / w;
  ni = pn * kPanel + (r - mi * w);
}

// The work of one CTA pair as a sequence of pieces (output tile, K blocks [kb0, kb1), K part).
// Round-robin schedule: piece i is unit pair + i * npairs of (tile, K part).
// Balanced schedule, for a tile count that leaves a last wave with at most half of the pairs busy: the tiles of that
// wave are divided into sw_parts K parts each and run FIRST, pair q taking part q % sw_parts of tile sw_first +
// q / sw_parts.  All parts but the last leave their accumulator in the pair's scratch slot; the pair with the LAST
// part (the highest-numbered pair of the group) adds them in pair order in its epilogue (which overlaps its next
// tile's main loop).  All pairs then walk the remaining tiles round-robin, in step with one another as in the plain
// schedule, which keeps concurrent CTAs on the same K blocks of shared operands.
// Forward progress: the only wait between CTAs of a grid is the reducing pair's wait for its group's arrival counters,
// and it waits only for LOWER-numbered pairs.  Thread blocks of a grid are handed to SMs in index order, so those pairs
// were started before the waiter; they never wait for another CTA (their pieces of the divided wave come first, then
// whole tiles), so they reach their arrival whatever else shares the GPU: a second grid on another stream (the weight
// gradients) can delay them but cannot hold them back, and the waiter never depends on a block that is not yet
// resident.  Nothing therefore requires the whole grid, let alone two grids, to be co-resident.
struct WorkIter {
  int tiles_mn, kblocks, kpb, nunits, npairs, t;
  int sw_tile, sw_kb0, sw_kb1, sw_part;  // this pair's piece of the divided wave (sw_tile < 0: none)
  __device__ WorkIter(const GemmDev& p, int tiles, int kb, int pair, int np)
      : tiles_mn(tiles), kblocks(kb), kpb((kb + p.ksplit - 1) / p.ksplit), nunits(tiles * p.ksplit), npairs(np), t(pair),
        sw_tile(-1), sw_kb0(0), sw_kb1(0), sw_part(0) {
    if (p.balanced) {
      nunits = p.sw_first;
      const int j = pair / p.sw_parts;
      if (p.sw_first + j < tiles) {
        sw_tile = p.sw_first + j;
        sw_part = pair % p.sw_parts;
        sw_kb0 = sw_part * p.sw_kpb;
        sw_kb1 = min(kb, sw_kb0 + p.sw_kpb);
      }
    }
  }
  // split: the piece belongs to the divided wave
  __device__ bool next(int& tile, int& kb0, int& kb1, int& part, bool& split) {
    if (sw_tile >= 0) {
      tile = sw_tile; kb0 = sw_kb0; kb1 = sw_kb1; part = sw_part; split = true;
      sw_tile = -1;
      return true;
    }
    split = false;
    if (t >= nunits) return false;
    tile = t % tiles_mn;
    part = t / tiles_mn;
    kb0 = part * kpb;
    kb1 = min(kblocks, kb0 + kpb);
    t += npairs;
    return true;
  }
};

// Bounded wait for `flag` to reach `target` (acquire).  One lane calls it.
__device__ __forceinline__ bool flag_wait(const int* flag, int target, volatile int* abort_flag, int* err) {
  const long long t0 = clock64();
  for (uint32_t it = 1;; ++it) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v >= target) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag != 0) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        atomicExch(err, (int)ERR_WAIT_TIMEOUT | (0x25 << 8));
        return false;
      }
    }
    __nanosleep(64);
  }
}

// 16 bf16 = 32 bytes in one store (256-bit stores exist from sm_100 on): one full 32-byte sector per request instead of
// two half-sector requests
__device__ __forceinline__ void store16_bf16(bf16* dst, const float* v) {
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
               "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

__device__ __forceinline__ void store8_f32(float* dst, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
               "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}
__device__ __forceinline__ void load8_b32(const void* src, uint32_t* w) {
  asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
               : "l"(src)
               : "memory");
}

__device__ __forceinline__ void store8_bf16(bf16* dst, const float* v) {
  uint4 o;
  o.x = pack_bf16(v[0], v[1]);
  o.y = pack_bf16(v[2], v[3]);
  o.z = pack_bf16(v[4], v[5]);
  o.w = pack_bf16(v[6], v[7]);
  *reinterpret_cast<uint4*>(dst) = o;
}

constexpr int SLOT_FLOATS = 256 * 256;  // one fp32 partial tile of a CTA pair

// Partial accumulators of the same output tile that other CTA pairs left in scratch.  A slot holds a pair's 256 x 256
// fp32 accumulator in the order the epilogue threads touch it, so that every warp access is one contiguous 512 bytes:
// float4 index = ((cta * 4 + lane quarter) * 64 + (column / 32) * 8 + j) * 32 + lane for columns 32 * (column / 32) +
// 4 j .. + 3 of the row held by `lane`.  `base` points at this thread's first float4 of the first partial.
constexpr int SLOT_F4 = SLOT_FLOATS / 4;
struct Fixup {
  const float4* base = nullptr;
  int n = 0;
};
__device__ __forceinline__ int slot_thread_f4(int cta, int quarter, int lane) { return (cta * 4 + quarter) * 2048 + lane; }

// 32 accumulator columns of this thread's row from TMEM (+ the partials of the same columns, added in index order)
__device__ __forceinline__ void scale32(uint32_t (&r)[32], float alpha) {
  if (alpha != 1.0f) {
#pragma unroll
    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
  }
}

__device__ __forceinline__ void ld_acc32(uint32_t taddr, int coloff, uint32_t (&r)[32], const Fixup& fx, float alpha) {
  tmem_ld32(taddr + coloff, r);
  if (fx.n == 0) {
    tmem_ld_wait();
    scale32(r, alpha);
    return;
  }
  // one round trip to L2 per partial: the trips, not the bytes, bound this loop (the launcher limits their number)
  const float4* src = fx.base + (coloff >> 5) * 256;
  float4 v[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = __ldcg(src + j * 32);
  tmem_ld_wait();
  for (int s = 0;;) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      r[4 * j + 0] = __float_as_uint(__uint_as_float(r[4 * j + 0]) + v[j].x);
      r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + v[j].y);
      r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + v[j].z);
      r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + v[j].w);
    }
    if (++s >= fx.n) break;
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = __ldcg(src + (long long)s * SLOT_F4 + j * 32);
  }
  scale32(r, alpha);
}

// Epilogue of one accumulator tile for one thread: `row` is the global output row held by this thread's TMEM lane,
// taddr the TMEM address of (its lane quarter, first column of the tile), n0 the tile's first output column.
// Every tcgen05.ld is executed by all 32 lanes (rows past M only skip the stores).
template <int BN, int MODE = 0>  // MODE 1: streaming cross-entropy, 2: SwiGLU backward (instantiations of their own)
__device__ __forceinline__ void epilogue_tile(const GemmDev& p, void* cptr, uint32_t taddr, int row, int n0, float& sq,
                                              float* stage, int cb, int ce, const Fixup fx = Fixup()) {
  const bool row_ok = row < p.M;
  uint32_t r[32];
  if constexpr (MODE == 1) {
    // Streaming cross-entropy: this thread holds row `row` of a 256-column tile of logits.
    const int y = row_ok ? p.ce_labels[row] : -1;
    if (p.ce_mode == 1) {
      float m = -INFINITY, s = 0.f, zy = 0.f;
      for (int c = cb; c < ce; c += 32) {
        const int gc = n0 + c;
        if (gc >= p.N) break;
        ld_acc32(taddr, c, r, fx, p.alpha);
        float cm = -INFINITY;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if (gc + j >= p.N) r[j] = 0xff800000u;  // -inf past the last column
          cm = fmaxf(cm, __uint_as_float(r[j]));
        }
        const float mn = fmaxf(m, cm);
        float cs = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) cs += __expf(__uint_as_float(r[j]) - mn);
        s = s * __expf(m - mn) + cs;  // m = -inf on the first chunk: e^(-inf) = 0
        m = mn;
        if (y >= gc && y < gc + 32) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (gc + j == y) zy = __uint_as_float(r[j]);
        }
      }
      if (row_ok) {
        p.ce_part[(long long)row * p.ce_tiles + n0 / BN] = make_float2(m, s);
        if (y >= n0 && y < n0 + BN && y < p.N) p.ce_zy[row] = zy;
      }
    } else {
      const float lse = row_ok ? p.ce_lse[row] : 0.f;
      const float w = (row_ok && y >= 0 && y < p.N) ? p.ce_sc->inv_count * p.ce_scale : 0.f;
      bf16* crow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc;
      for (int c = cb; c < ce; c += 32) {
        const int gc = n0 + c;
        if (gc >= p.N) break;
        ld_acc32(taddr, c, r, fx, p.alpha);
        if (row_ok) {
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float pj = __expf(__uint_as_float(r[j]) - lse);
            if (gc + j == y) pj -= 1.0f;
            v[j] = pj * w;
          }
          if (p.wide_store) {
            if (gc < p.N) store16_bf16(crow + gc, v);
            if (gc + 16 < p.N) store16_bf16(crow + gc + 16, v + 16);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 8)
              if (gc + j < p.N) store8_bf16(crow + gc + j, v + j);
          }
        }
      }
    }
    return;
  }
  if constexpr (MODE == 2) {
    // SwiGLU backward: the accumulator is d_a (logical ffn columns); gate and up of the same (row, column) come from the
    // forward pass' gu, one 32-column chunk ahead like the residual below (the kernel asked for the row's lines to be
    // brought into L2 before it waited for the accumulator).  The 32 columns of a chunk land in 64 contiguous output
    // columns: [16 d_gate | 16 d_up] twice.  (Tried: 8 lanes per row through the staging tile, so that every store is
    // a full line: a third slower; the loads' latency, not the number of requests, is what this epilogue waits for.)
    const int f = p.d_ffn;
    const bf16* grow = p.gu + (long long)row * (2LL * f);
    bf16* drow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc;
    uint4 nG[4], nU[4];
    auto fetch = [&](int gc) {
      if (p.wide_store) {  // 32-byte loads
#pragma unroll
        for (int j = 0; j < 4; j += 2) {
          if (row_ok && gc + 8 * j < p.N) {
            uint32_t w[8];
            load8_b32(grow + gc + 8 * j, w);
            nG[j] = make_uint4(w[0], w[1], w[2], w[3]);
            nG[j + 1] = make_uint4(w[4], w[5], w[6], w[7]);
            load8_b32(grow + f + gc + 8 * j, w);
            nU[j] = make_uint4(w[0], w[1], w[2], w[3]);
            nU[j + 1] = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            nG[j] = nG[j + 1] = nU[j] = nU[j + 1] = make_uint4(0, 0, 0, 0);
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const bool ok = row_ok && gc + 8 * j < p.N;
          nG[j] = ok ? *reinterpret_cast<const uint4*>(grow + gc + 8 * j) : make_uint4(0, 0, 0, 0);
          nU[j] = ok ? *reinterpret_cast<const uint4*>(grow + f + gc + 8 * j) : make_uint4(0, 0, 0, 0);
        }
      }
    };
    fetch(n0 + cb);
    for (int c = cb; c < ce; c += 32) {
      const int gc = n0 + c;
      if (gc >= p.N) break;
      uint4 cG[4], cU[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) { cG[j] = nG[j]; cU[j] = nU[j]; }
      if (c + 32 < ce) fetch(gc + 32);
      ld_acc32(taddr, c, r, fx, p.alpha);
      if (row_ok) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {  // the chunk's two groups of 16 logical columns
          if (gc + 16 * hh < p.N) {
            float dG[16], dU[16];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const uint4 g4 = cG[2 * hh + q], u4 = cU[2 * hh + q];
              const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w}, uw[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int j = 16 * hh + 8 * q + 2 * e;
                swiglu_bwd_elem(round_bf16(__uint_as_float(r[j])), bf16_lo(gw[e]), bf16_lo(uw[e]), dG[8 * q + 2 * e], dU[8 * q + 2 * e]);
                swiglu_bwd_elem(round_bf16(__uint_as_float(r[j + 1])), bf16_hi(gw[e]), bf16_hi(uw[e]), dG[8 * q + 2 * e + 1],
                                dU[8 * q + 2 * e + 1]);
              }
            }
            bf16* dst = drow + 2 * gc + 32 * hh;
            if (p.wide_store) {
              store16_bf16(dst, dG);
              store16_bf16(dst + 16, dU);
            } else {
              store8_bf16(dst, dG);
              store8_bf16(dst + 8, dG + 8);
              store8_bf16(dst + 16, dU);
              store8_bf16(dst + 24, dU + 8);
            }
          }
        }
      }
    }
    return;
  }
  if (p.adam_p != nullptr) {
    // Weight gradient consumed in place: g = accumulator (+ the gradient of earlier chunks for EPI_F32_ACC), then
    // AdamW on master, moments and bf16 copy at the same position.  The 32 x 32 chunk goes through the warp's staging
    // tile so that 8 lanes cover 128 contiguous bytes of one row: all seven streams are read and written coalesced.
    const AdamCoef c = adam_coef(p);
    const int lane = threadIdx.x & 31;
    const int row0 = row - lane;                 // first row of this warp's 32
    const int sub = lane >> 3, col4 = (lane & 7) * 4;
    for (int c0 = cb; c0 < ce; c0 += 32) {
      const int gc = n0 + c0;
      if (gc >= p.N) break;
      if (c0 + 32 < ce) adam_prefetch_chunk(p, cptr, row, gc + 32);
      ld_acc32(taddr, c0, r, fx, p.alpha);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *reinterpret_cast<float4*>(stage + lane * 32 + 4 * (j ^ (lane & 7))) =
            make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                        __uint_as_float(r[4 * j + 3]));
      __syncwarp();
      if (gc + col4 < p.N) {
        // all loads of the chunk are issued before the first store (the compiler cannot prove the streams distinct,
        // so it would otherwise serialise one row's loads behind the previous row's stores)
        // Rolling window over the chunk's 8 row groups: the loads of group i + 4 are issued before group i is updated
        // and stored, so four groups of loads stay in flight behind the arithmetic.  (Loads are placed explicitly: the
        // compiler cannot prove the streams distinct and would not move them above earlier stores.)
        float4 P4[8], M4[8], V4[8], O4[8];
        auto fetch = [&](int i) {
          const int rr = i * 4 + sub;
          const bool okr = row0 + rr < p.M;
          const long long o = (long long)(row0 + rr) * p.ldc + gc + col4;
          const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
          P4[i] = okr ? *reinterpret_cast<const float4*>(p.adam_p + o) : z;
          M4[i] = okr ? *reinterpret_cast<const float4*>(p.adam_m + o) : z;
          V4[i] = okr ? *reinterpret_cast<const float4*>(p.adam_v + o) : z;
          O4[i] = (okr && p.epi == EPI_F32_ACC) ? *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(cptr) + o) : z;
        };
#pragma unroll
        for (int i = 0; i < 4; ++i) fetch(i);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (i + 4 < 8) fetch(i + 4);
          const int rr = i * 4 + sub;
          if (row0 + rr < p.M) {
            const long long o = (long long)(row0 + rr) * p.ldc + gc + col4;
            const float4 g4 = *reinterpret_cast<const float4*>(stage + rr * 32 + 4 * ((col4 >> 2) ^ (rr & 7)));
            float g[4] = {g4.x, g4.y, g4.z, g4.w};
            if (p.epi == EPI_F32_ACC) { g[0] += O4[i].x; g[1] += O4[i].y; g[2] += O4[i].z; g[3] += O4[i].w; }
            float pp[4] = {P4[i].x, P4[i].y, P4[i].z, P4[i].w}, mm[4] = {M4[i].x, M4[i].y, M4[i].z, M4[i].w},
                  vv[4] = {V4[i].x, V4[i].y, V4[i].z, V4[i].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              sq += g[e] * g[e];
              adamw_elem(g[e], p.adam_wd, c, pp[e], mm[e], vv[e]);
            }
            *reinterpret_cast<float4*>(p.adam_p + o) = make_float4(pp[0], pp[1], pp[2], pp[3]);
            *reinterpret_cast<float4*>(p.adam_m + o) = make_float4(mm[0], mm[1], mm[2], mm[3]);
            *reinterpret_cast<float4*>(p.adam_v + o) = make_float4(vv[0], vv[1], vv[2], vv[3]);
            uint2 ob;
            ob.x = pack_bf16(pp[0], pp[1]);
            ob.y = pack_bf16(pp[2], pp[3]);
            *reinterpret_cast<uint2*>(p.adam_pb + o) = ob;
          }
        }
      }
      __syncwarp();
    }
  } else if (p.epi == EPI_ROPE) {
    const int d = p.head_dim;
    const int half = d >> 1;
    const int pos = row_ok ? (row % p.seq) : 0;
    bf16* crow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc;
    for (int hc = cb; hc < ce; hc += d) {
      const int g0 = n0 + hc;
      if (g0 >= p.N) break;
      if (g0 >= p.rope_cols) {
        for (int c = 0; c < d; c += 32) {
          ld_acc32(taddr, hc + c, r, fx, 1.0f);
          if (row_ok) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
            if (p.wide_store) {
#pragma unroll
              for (int j = 0; j < 32; j += 16) store16_bf16(crow + g0 + c + j, v + j);
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 8) store8_bf16(crow + g0 + c + j, v + j);
            }
          }
        }
      } else {
        uint32_t r2[32];
        // per-head QK-Norm: a first pass over the head's accumulators for r, which is applied (with the gain) in the
        // rotation pass below
        float qr = 1.0f;
        const bf16* gain = nullptr;
        if (p.qk_r != nullptr) {
          float ss = 0.f;
          for (int c = 0; c < d; c += 32) {
            ld_acc32(taddr, hc + c, r, fx, 1.0f);
#pragma unroll
            for (int j = 0; j < 32; ++j) ss = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ss);
          }
          qr = 1.0f / sqrtf(ss / (float)d + p.qk_eps);
          const int head = g0 / d;
          gain = head < p.n_q_heads ? p.qk_gain_q : p.qk_gain_k;
          if (row_ok) p.qk_r[(long long)row * (p.rope_cols / d) + head] = qr;
        }
        for (int i0 = 0; i0 < half; i0 += 32) {
          if (fx.n == 0) {
            tmem_ld32(taddr + hc + i0, r);
            tmem_ld32(taddr + hc + i0 + half, r2);
            tmem_ld_wait();
          } else {
            ld_acc32(taddr, hc + i0, r, fx, 1.0f);
            ld_acc32(taddr, hc + i0 + half, r2, fx, 1.0f);
          }
          if (row_ok) {
            const float* cs = p.rope_cos + (long long)i0 * p.rope_ld + pos;
            const float* sn = p.rope_sin + (long long)i0 * p.rope_ld + pos;
            float lo[32], hi[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float cc = cs[(long long)j * p.rope_ld], ss = sn[(long long)j * p.rope_ld];
              float x1 = __uint_as_float(r[j]);
              float x2 = __uint_as_float(r2[j]);
              if (gain != nullptr) {
                x1 = x1 * qr * __bfloat162float(gain[i0 + j]);
                x2 = x2 * qr * __bfloat162float(gain[i0 + half + j]);
              }
              lo[j] = x1 * cc - x2 * ss;
              hi[j] = x2 * cc + x1 * ss;
            }
            if (p.wide_store) {
#pragma unroll
              for (int j = 0; j < 32; j += 16) {
                store16_bf16(crow + g0 + i0 + j, lo + j);
                store16_bf16(crow + g0 + i0 + half + j, hi + j);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 8) {
                store8_bf16(crow + g0 + i0 + j, lo + j);
                store8_bf16(crow + g0 + i0 + half + j, hi + j);
              }
            }
          }
        }
      }
    }
  } else if (p.epi == EPI_SWIGLU) {
    // physical columns alternate 16 gate / 16 up of the same 16 logical ffn columns
    const int f = p.d_ffn;
    bf16* arow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc;
    bf16* gurow = p.gu + (long long)row * (2LL * f);
    for (int c = cb; c < ce; c += 32) {
      const int gc = n0 + c;
      if (gc >= p.N) break;
      ld_acc32(taddr, c, r, fx, p.alpha);
      if (row_ok) {
        const int lc = gc >> 1;  // logical ffn column of this 16-wide group
        float g[16], u[16], a[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          g[j] = round_bf16(__uint_as_float(r[j]));
          u[j] = round_bf16(__uint_as_float(r[16 + j]));
          a[j] = __fdividef(g[j], 1.0f + __expf(-g[j])) * u[j];
        }
        if (p.wide_store) {
          store16_bf16(gurow + lc, g);
          store16_bf16(gurow + f + lc, u);
          store16_bf16(arow + lc, a);
        } else {
          store8_bf16(gurow + lc, g);
          store8_bf16(gurow + lc + 8, g + 8);
          store8_bf16(gurow + f + lc, u);
          store8_bf16(gurow + f + lc + 8, u + 8);
          store8_bf16(arow + lc, a);
          store8_bf16(arow + lc + 8, a + 8);
        }
      }
    }
  } else if (p.epi == EPI_BF16_RESID) {
    // the residual row is read one 32-column chunk ahead of the accumulator it is added to, so its latency overlaps
    // the TMEM load and the stores of the previous chunk
    bf16* crow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc;
    const bf16* rrow = p.resid + (long long)row * p.ldc;
    uint4 nxt[4];
    auto fetch = [&](int gc) {
      if (p.wide_store) {  // two 32-byte loads
#pragma unroll
        for (int j = 0; j < 4; j += 2) {
          if (row_ok && gc + 8 * j < p.N) {
            uint32_t w[8];
            load8_b32(rrow + gc + 8 * j, w);
            nxt[j] = make_uint4(w[0], w[1], w[2], w[3]);
            nxt[j + 1] = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            nxt[j] = make_uint4(0, 0, 0, 0);
            nxt[j + 1] = make_uint4(0, 0, 0, 0);
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          nxt[j] = (row_ok && gc + 8 * j < p.N) ? *reinterpret_cast<const uint4*>(rrow + gc + 8 * j) : make_uint4(0, 0, 0, 0);
      }
    };
    fetch(n0 + cb);
    for (int c = cb; c < ce; c += 32) {
      const int gc = n0 + c;
      if (gc >= p.N) break;
      uint4 cur[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) cur[j] = nxt[j];
      if (c + 32 < ce) fetch(gc + 32);
      ld_acc32(taddr, c, r, fx, p.alpha);
      if (row_ok) {
        float v[32];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[8 * j + 0] = __uint_as_float(r[8 * j + 0]) + bf16_lo(cur[j].x); v[8 * j + 1] = __uint_as_float(r[8 * j + 1]) + bf16_hi(cur[j].x);
          v[8 * j + 2] = __uint_as_float(r[8 * j + 2]) + bf16_lo(cur[j].y); v[8 * j + 3] = __uint_as_float(r[8 * j + 3]) + bf16_hi(cur[j].y);
          v[8 * j + 4] = __uint_as_float(r[8 * j + 4]) + bf16_lo(cur[j].z); v[8 * j + 5] = __uint_as_float(r[8 * j + 5]) + bf16_hi(cur[j].z);
          v[8 * j + 6] = __uint_as_float(r[8 * j + 6]) + bf16_lo(cur[j].w); v[8 * j + 7] = __uint_as_float(r[8 * j + 7]) + bf16_hi(cur[j].w);
        }
        if (p.wide_store) {
#pragma unroll
          for (int j = 0; j < 32; j += 16)
            if (gc + j < p.N) store16_bf16(crow + gc + j, v + j);
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 8)
            if (gc + j < p.N) store8_bf16(crow + gc + j, v + j);
        }
      }
    }
  } else if (p.epi == EPI_F32_ACC) {
    float* crow = reinterpret_cast<float*>(cptr) + (long long)row * p.ldc;
    uint32_t nxt[32];
    auto fetch = [&](int gc) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        if (row_ok && gc + j < p.N) {
          if (p.wide_store) {
            load8_b32(crow + gc + j, nxt + j);
          } else {
            const float4 a = *reinterpret_cast<const float4*>(crow + gc + j);
            const float4 b4 = (gc + j + 4 < p.N) ? *reinterpret_cast<const float4*>(crow + gc + j + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
            nxt[j] = __float_as_uint(a.x); nxt[j + 1] = __float_as_uint(a.y); nxt[j + 2] = __float_as_uint(a.z); nxt[j + 3] = __float_as_uint(a.w);
            nxt[j + 4] = __float_as_uint(b4.x); nxt[j + 5] = __float_as_uint(b4.y); nxt[j + 6] = __float_as_uint(b4.z); nxt[j + 7] = __float_as_uint(b4.w);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) nxt[j + e] = 0u;
        }
      }
    };
    fetch(n0 + cb);
    for (int c = cb; c < ce; c += 32) {
      const int gc = n0 + c;
      if (gc >= p.N) break;
      uint32_t cur[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) cur[j] = nxt[j];
      if (c + 32 < ce) fetch(gc + 32);
      ld_acc32(taddr, c, r, fx, p.alpha);
      if (row_ok) {
#pragma unroll
        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(cur[j]) + __uint_as_float(r[j]));
        if (p.wide_store) {
#pragma unroll
          for (int j = 0; j < 32; j += 8)
            if (gc + j < p.N) store8_f32(crow + gc + j, r + j);
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            if (gc + j < p.N)
              *reinterpret_cast<float4*>(crow + gc + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                      __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
        }
      }
    }
  } else {
    for (int c = cb; c < ce; c += 32) {
      const int gc = n0 + c;
      if (gc >= p.N) break;
      ld_acc32(taddr, c, r, fx, p.alpha);
      if (row_ok) {
        if (p.epi == EPI_BF16) {
          bf16* crow = reinterpret_cast<bf16*>(cptr) + (long long)row * p.ldc + gc;
          if (p.wide_store) {
#pragma unroll
            for (int j = 0; j < 32; j += 16) {
              if (gc + j < p.N) {
                float v[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = __uint_as_float(r[j + e]);
                store16_bf16(crow + j, v);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              if (gc + j < p.N) {
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(r[j + e]);
                store8_bf16(crow + j, v);
              }
            }
          }
        } else {
          float* crow = reinterpret_cast<float*>(cptr) + (long long)row * p.ldc + gc;
          if (p.wide_store) {
#pragma unroll
            for (int j = 0; j < 32; j += 8)
              if (gc + j < p.N) store8_f32(crow + j, r + j);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              if (gc + j < p.N)
                *reinterpret_cast<float4*>(crow + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                   __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
            }
          }
        }
      }
    }
  }
}

template <int BN, bool A_MN, bool B_MN, int MODE = 0>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmDev p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::STAGES * C::STAGE_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  // barrier slots: [0,S) full, [S,2S) empty, 2S+{0,1} accumulator full, 2S+{2,3} accumulator empty
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

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
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
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
  pdl_wait();  // barriers, TMEM and descriptors are set up; everything from here on touches the predecessor's data

  const int tiles_m = (p.M + BM - 1) / BM;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int ntiles = tiles_m * tiles_n;
  const int kblocks = (p.K + BK - 1) / BK;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        int mi, ni;
        tile_coords(p.panel, t, tiles_m, tiles_n, mi, ni);
        const int m0 = mi * BM, n0 = ni * BN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.err, kWaitLimitCycles, 0x11)) { ok = false; break; }
          const uint32_t fb = full_bar(stage);
          mbar_expect_tx(fb, C::STAGE_BYTES);
          const uint32_t a_dst = smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t b_dst = a_dst + A_BYTES;
          if constexpr (!A_MN) {
            tma_load_2d(a_dst, &tmA, fb, kb * BK, m0);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d(a_dst + j * CHUNK_BYTES, &tmA, fb, m0 + 64 * j, kb * BK);
          }
          if constexpr (!B_MN) {
            tma_load_2d(b_dst, &tmB, fb, kb * BK, n0);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(b_dst + j * CHUNK_BYTES, &tmB, fb, n0 + 64 * j, kb * BK);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, bf16 A and B, majors, N/8, M/16
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.err, kWaitLimitCycles, 0x12)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.err, kWaitLimitCycles, 0x13)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t adesc = A_MN ? umma_desc_sw128(a_addr + k * 2048, CHUNK_BYTES, 1024)
                                        : umma_desc_sw128(a_addr + k * 32, 0, 1024);
            const uint64_t bdesc = B_MN ? umma_desc_sw128(b_addr + k * 2048, CHUNK_BYTES, 1024)
                                        : umma_desc_sw128(b_addr + k * 32, 0, 1024);
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
    float sq = 0.f;  // fused AdamW: this thread's share of the squared gradient norm
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
      int mi, ni;
      tile_coords(p.panel, t, tiles_m, tiles_n, mi, ni);
      const int m0 = mi * BM, n0 = ni * BN;
      if (p.adam_p != nullptr) adam_prefetch_chunk(p, p.C, m0 + q * 32 + lane, n0);
      if constexpr (MODE == 2) swiglu_bwd_prefetch(p, m0 + q * 32 + lane, n0, BN);
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.err, kWaitLimitCycles, 0x14);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + q * 32 + lane;
      epilogue_tile<BN, MODE>(p, p.C, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), row, n0, sq,
                        reinterpret_cast<float*>(smem + C::STAGES * C::STAGE_BYTES + C::BAR_BYTES) + q * EPI_STAGE_FLOATS, 0, BN);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (p.adam_p != nullptr) {
      sq = warp_sum(sq);
      if (lane == 0) p.adam_sq[blockIdx.x * 4 + q] = sq;
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

// Two more tensor maps of a launch.  SwiGLU backward (its epilogue moves tiles through the TMA unit): m0 = the forward
// pass' gate | up [T, 2f] in boxes of 32 rows x 32 columns, m1 = the output d_gate / d_up (interleaved 16 | 16) in boxes
// of 32 x 64.  Grouped weight gradients: m0, m1 = operands A and B of the second problem.
struct AuxMaps {
  CUtensorMap m0;
  CUtensorMap m1;
};

// One warp's load of the gate and up tiles (32 rows x 32 logical columns from column gc) into its staging buffer
__device__ __forceinline__ void swiglu_bwd_tma_fetch(const GemmDev& p, const AuxMaps& em, uint32_t buf, uint32_t bar, int gc,
                                                     int row0) {
  mbar_expect_tx(bar, 4096);
  tma_load_2d(buf, &em.m0, bar, gc, row0);
  tma_load_2d(buf + 2048, &em.m0, bar, p.d_ffn + gc, row0);
}

// SwiGLU backward with the epilogue's memory traffic on the TMA unit.  The register path above reads gate and up and
// writes d_gate and d_up with one row per thread, four times the bytes of a plain bf16 epilogue in 32-byte requests that
// each are a wavefront of their own in the load/store pipe (half of that pipe's peak over the whole kernel).  Here a
// warp's 32 rows x 32 columns of gate and of up arrive as two TMA boxes (64-byte rows, 64-byte swizzle) on the warp's own
// mbarrier, the threads read their row from shared memory without bank conflicts, and the 32 x 64 output tile (128-byte
// rows, 128-byte swizzle) leaves as one TMA store.  The load of chunk c + 1 is issued as soon as chunk c sits in
// registers; the store of chunk c drains while chunk c + 1 is computed.  Same element function, same roundings:
// bit-identical to the register path.  Measured at 8192 x 5632 x 2048: 176 -> 168 us alone, 210 -> 199 us inside the c3_1b
// step; the load/store pipe falls to 13 % of its peak, and what remains over the plain data gradient (124 us) is the
// epilogue's bytes themselves on the L2-to-SM path that the operand loads already fill.
// buf: 8 KB, 1024-byte aligned: gate, up, output tile.  Returns false when a bounded wait ran out.
__device__ __forceinline__ bool epilogue_swiglu_bwd_tma(const GemmDev& p, const AuxMaps& em, uint32_t taddr, int row0, int n0,
                                                        int cb, int ce, const Fixup& fx, uint32_t buf, uint32_t bar,
                                                        uint32_t& phase, volatile int* abort_flag) {
  const int lane = threadIdx.x & 31;
  const uint32_t in_row = buf + (uint32_t)lane * 64u, sw_in = (uint32_t)((lane >> 1) & 3);
  const uint32_t out_row = buf + 4096u + (uint32_t)lane * 128u, sw_out = (uint32_t)(lane & 7);
  uint32_t r[32];
  for (int c = cb; c < ce; c += 32) {
    const int gc = n0 + c;
    if (gc >= p.N) break;
    bool ok = mbar_wait(bar, phase, abort_flag, p.err, kWaitLimitCycles, 0x26);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) return false;
    phase ^= 1u;
    uint4 cG[4], cU[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      cG[j] = ld_shared_v4(in_row + (((uint32_t)j ^ sw_in) << 4));
      cU[j] = ld_shared_v4(in_row + 2048u + (((uint32_t)j ^ sw_in) << 4));
    }
    __syncwarp();
    if (lane == 0 && c + 32 < ce && gc + 32 < p.N) swiglu_bwd_tma_fetch(p, em, buf, bar, gc + 32, row0);
    ld_acc32(taddr, c, r, fx, p.alpha);
    uint32_t o[32];  // the thread's 128-byte output row: [16 d_gate | 16 d_up] twice
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      float dG[16], dU[16];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint4 g4 = cG[2 * hh + q], u4 = cU[2 * hh + q];
        const uint32_t gw[4] = {g4.x, g4.y, g4.z, g4.w}, uw[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = 16 * hh + 8 * q + 2 * e;
          swiglu_bwd_elem(round_bf16(__uint_as_float(r[j])), bf16_lo(gw[e]), bf16_lo(uw[e]), dG[8 * q + 2 * e], dU[8 * q + 2 * e]);
          swiglu_bwd_elem(round_bf16(__uint_as_float(r[j + 1])), bf16_hi(gw[e]), bf16_hi(uw[e]), dG[8 * q + 2 * e + 1],
                          dU[8 * q + 2 * e + 1]);
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        o[16 * hh + i] = pack_bf16(dG[2 * i], dG[2 * i + 1]);
        o[16 * hh + 8 + i] = pack_bf16(dU[2 * i], dU[2 * i + 1]);
      }
    }
    if (lane == 0) bulk_wait_group_read0();  // the previous chunk's store has read the output tile
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 8; ++j)
      st_shared_v4(out_row + (((uint32_t)j ^ sw_out) << 4), make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]));
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      tma_store_2d(&em.m1, buf + 4096u, 2 * gc, row0);
      bulk_commit_group();
    }
  }
  return true;
}

// Plain bf16 output through the TMA unit: a warp packs 32 rows x 64 columns of its accumulator into a 4 KB tile
// (128-byte rows, 128-byte swizzle: no bank conflicts with one row per thread) and one lane sends it off as a tensor
// store of full 128-byte lines, alternating between two tiles so that the store of one drains while the next is packed.
// One row per thread with 32-byte global stores is bound by L2 store requests, which shows wherever the epilogue is not
// hidden behind a main loop (short contractions, the last wave of any launch).  Same values, same rounding.
// buf: 8 KB, 1024-byte aligned.
__device__ __forceinline__ void epilogue_bf16_tma(const GemmDev& p, const AuxMaps& em, uint32_t taddr, int row0, int n0,
                                                  int cb, int ce, const Fixup& fx, uint32_t buf) {
  const int lane = threadIdx.x & 31;
  const uint32_t sw = (uint32_t)(lane & 7);
  uint32_t r[32];
  int b = 0;
  for (int c = cb; c < ce; c += 64) {
    const int gc = n0 + c;
    if (gc >= p.N) break;
    uint32_t o[32];
    ld_acc32(taddr, c, r, fx, p.alpha);
#pragma unroll
    for (int i = 0; i < 16; ++i) o[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
    if (gc + 32 < p.N) {
      ld_acc32(taddr, c + 32, r, fx, p.alpha);
#pragma unroll
      for (int i = 0; i < 16; ++i) o[16 + i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) o[16 + i] = 0u;  // columns past N: dropped by the store
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");  // the store that last read this tile
    __syncwarp();
    const uint32_t tile = buf + (uint32_t)b * 4096u, trow = tile + (uint32_t)lane * 128u;
#pragma unroll
    for (int j = 0; j < 8; ++j)
      st_shared_v4(trow + (((uint32_t)j ^ sw) << 4), make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]));
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      tma_store_2d(&em.m1, tile, gc, row0);
      bulk_commit_group();
    }
    b ^= 1;
  }
}

// ---------------------------------------------------------------- CTA-pair variant
// Two CTAs on neighbouring SMs (a cluster of 2) share one 256 x 256 output tile: each loads its own 128 rows of A and
// its own 128 of the 256 rows of B, the leader issues tcgen05.mma.cta_group::2 (M = 256), and each CTA's TMEM ends up
// with its 128 rows x 256 columns of the accumulator.  Per flop this moves a third less operand data through L2 and
// shared memory than the single-CTA 128 x 256 tile.  Every CTA fetches its own operands with its own TMA copies.
struct PairCfg {
  static constexpr int BN = 256;                 // output columns of the pair's tile
  static constexpr int HALF_B = 128;             // rows of B (output columns) each CTA loads
  static constexpr int A_BYTES_ = BM * BK * 2;   // 16 KB
  static constexpr int B_BYTES = HALF_B * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES_ + B_BYTES;
  static constexpr int STAGES = 6;
  static constexpr int EPI_BYTES = EPI_STAGE_BYTES;
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 256 + EPI_BYTES + 1024;
};

// Warps: TMA producer, MMA issuer, then the epilogue warps.  Launched with 192 threads there are four (one per TMEM lane
// quarter, all 256 columns of the tile each); with 320 there are eight (two per quarter, 128 columns each), which the
// fused AdamW epilogue needs to keep enough loads in flight.  (Eight warps cost the plain epilogues about 4 % of tensor
// activity, measured on the gate/up shape, so they are used only where the epilogue is the heavy part.)
constexpr int PAIR_THREADS = 320;

template <bool A_MN, bool B_MN, int MODE = 0>
__global__ void __launch_bounds__(PAIR_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ AuxMaps em, const __grid_constant__ GemmDev p,
                    const __grid_constant__ GemmDev p2) {
  // p2 (grouped launch, MODE 3): p with C, ldc, M, N, panel, alpha and the AdamW pointers of the second problem; a copy
  // of p otherwise.  Both live in parameter space, so the epilogue's reads of either cost what they cost in the other modes.
  using C = PairCfg;
  constexpr int BN = C::BN;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // operand stages, then the epilogue warps' staging area (1024-byte aligned, as swizzled TMA tiles need), then barriers
  uint8_t* epi_stage = smem + C::STAGES * C::STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(epi_stage + C::EPI_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (C::STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * C::STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  auto epi_ld_bar = [&](int w) { return bar0 + 8u * (2 * C::STAGES + 6 + w); };  // one per epilogue warp (TMA epilogue loads)

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(full_bar(s), 1);   // the leader's expect_tx arrival; both CTAs' bytes are counted on the leader's barrier
      mbar_init(empty_bar(s), 1);  // one commit, arriving in both CTAs
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);   // one commit, arriving in both CTAs
      mbar_init(tempty_bar(b), 2 * (blockDim.x / 32 - 2));  // the epilogue warps of both CTAs, all arriving at the leader
    }
    if constexpr (MODE == 2)
      for (int w = 0; w < 4; ++w) mbar_init(epi_ld_bar(w), 1);
    if constexpr (MODE == 3) {
      tma_prefetch_desc(&em.m0);
      tma_prefetch_desc(&em.m1);
    }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if constexpr (MODE == 2) {
      if (p.swiglu_tma) { tma_prefetch_desc(&em.m0); tma_prefetch_desc(&em.m1); }
    }
    if constexpr (MODE == 0) {
      if (p.tma_out) tma_prefetch_desc(&em.m1);
    }
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), C::TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();
  pdl_wait();  // barriers, TMEM and descriptors are set up; everything from here on touches the predecessor's data

  const int tiles_m = (p.M + 255) / 256;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int tiles0 = tiles_m * tiles_n;
  constexpr bool grouped = MODE == 3;  // tiles from tiles0 on belong to the second problem
  const int g_tiles_m = grouped ? (p.g_M + 255) / 256 : 0;
  const int g_tiles_n = grouped ? (p.g_N + BN - 1) / BN : 0;
  const int tiles_mn = tiles0 + g_tiles_m * g_tiles_n;
  const int kblocks_all = (p.K + BK - 1) / BK;
  WorkIter work(p, tiles_mn, kblocks_all, pair, npairs);
  int tile, kb0, kb1, part;
  bool split;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      while (ok && work.next(tile, kb0, kb1, part, split)) {
        int mi, ni;
        const bool second = grouped && tile >= tiles0;
        if (second) tile_coords(p.g_panel, tile - tiles0, g_tiles_m, g_tiles_n, mi, ni);
        else tile_coords(p.panel, tile, tiles_m, tiles_n, mi, ni);
        const CUtensorMap* mapA = second ? &em.m0 : &tmA;
        const CUtensorMap* mapB = second ? &em.m1 : &tmB;
        const int m0 = mi * 256 + (int)rank * BM;        // this CTA's rows of A / of the output
        const int nb0 = ni * BN + (int)rank * C::HALF_B;  // this CTA's rows of B
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.err, kWaitLimitCycles, 0x21 | (MODE << 8))) { ok = false; break; }
          const uint32_t fb = full_bar(stage);
          if (rank == 0) mbar_expect_tx(fb, 2 * C::STAGE_BYTES);
          const uint32_t a_dst = smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t b_dst = a_dst + C::A_BYTES_;
          if constexpr (!A_MN) {
            tma_load_2d_pair(a_dst, mapA, fb, kb * BK, m0);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(a_dst + j * CHUNK_BYTES, mapA, fb, m0 + 64 * j, kb * BK);
          }
          if constexpr (!B_MN) {
            tma_load_2d_pair(b_dst, mapB, fb, kb * BK, nb0);
          } else {
#pragma unroll
            for (int j = 0; j < C::HALF_B / 64; ++j)
              tma_load_2d_pair(b_dst + j * CHUNK_BYTES, mapB, fb, nb0 + 64 * j, kb * BK);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // M = 256 over the pair, N = 256
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) | ((B_MN ? 1u : 0u) << 16) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      while (ok && work.next(tile, kb0, kb1, part, split)) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.err, kWaitLimitCycles, 0x22 | (MODE << 8))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.err, kWaitLimitCycles, 0x23 | (MODE << 8))) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t b_addr = a_addr + C::A_BYTES_;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t adesc = A_MN ? umma_desc_sw128(a_addr + k * 2048, CHUNK_BYTES, 1024)
                                        : umma_desc_sw128(a_addr + k * 32, 0, 1024);
            const uint64_t bdesc = B_MN ? umma_desc_sw128(b_addr + k * 2048, CHUNK_BYTES, 1024)
                                        : umma_desc_sw128(b_addr + k * 32, 0, 1024);
            umma_bf16_pair(d_tmem, adesc, bdesc, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(stage));  // frees the stage in both CTAs
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(tfull_bar(acc));  // wakes the epilogue warps of both CTAs
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int ncols = blockDim.x == PAIR_THREADS ? 128 : 256;  // columns of the tile per epilogue warp
    const int cb = ((warp - 2) >> 2) * ncols;
    const int ce = cb + ncols;
    float* stage = reinterpret_cast<float*>(epi_stage) + (warp - 2) * EPI_STAGE_FLOATS;
    // SwiGLU backward through the TMA unit: four epilogue warps, 8 KB of the staging area and one load barrier each.
    // (Eight warps with 8 KB each, paid for with one of the six operand stages, were no faster: 206 against 199 us per
    // launch at c3_1b.  What this epilogue costs is its bytes on the L2-to-SM path, which the operand loads fill.)
    [[maybe_unused]] const bool tma_epi = MODE == 2 && p.swiglu_tma != 0 && blockDim.x == GEMM_THREADS;
    [[maybe_unused]] const uint32_t tbuf = smem_u32(epi_stage) + (uint32_t)((warp - 2) & 3) * 8192u;
    [[maybe_unused]] const uint32_t tbar = epi_ld_bar((warp - 2) & 3);
    [[maybe_unused]] uint32_t tphase = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    float sq = 0.f;  // fused AdamW: this thread's share of the squared gradient norm
    while (work.next(tile, kb0, kb1, part, split)) {
      int mi, ni;
      const bool second = grouped && tile >= tiles0;
      if (second) tile_coords(p.g_panel, tile - tiles0, g_tiles_m, g_tiles_n, mi, ni);
      else tile_coords(p.panel, tile, tiles_m, tiles_n, mi, ni);
      const int pe_N = second ? p2.N : p.N;   // of the problem this tile belongs to
      void* const pe_C = second ? p2.C : p.C;
      const int m0 = mi * 256 + (int)rank * BM;
      const int n0 = ni * BN;
      const bool reducer = !split || part == p.sw_parts - 1;  // this piece ends in the tile's epilogue
      if (p.adam_p != nullptr && reducer) {
        if (second) adam_prefetch_chunk(p2, p2.C, m0 + q * 32 + lane, n0 + cb);
        else adam_prefetch_chunk(p, p.C, m0 + q * 32 + lane, n0 + cb);
      }
      // (asking one piece earlier instead, from the previous piece's epilogue, was slower: 219 us against 201 at c3_1b)
      [[maybe_unused]] const bool tma_tile = tma_epi && reducer && m0 + q * 32 < p.M && n0 + cb < p.N;
      if constexpr (MODE == 2) {
        if (reducer) swiglu_bwd_prefetch(p, m0 + q * 32 + lane, n0 + cb, ncols);
        if (tma_tile && lane == 0) swiglu_bwd_tma_fetch(p, em, tbuf, tbar, n0 + cb, m0 + q * 32);
      }
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.err, kWaitLimitCycles, 0x24 | (MODE << 8));
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + q * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
      const int slot_f4 = slot_thread_f4((int)rank, q, lane);
      if (!reducer) {
        // an earlier K part of a divided tile: leave this partial accumulator in the pair's slot
        float4* dst = reinterpret_cast<float4*>(p.slots) + (long long)pair * SLOT_F4 + slot_f4;
        uint32_t r[32];
        for (int c = cb; c < ce && n0 + c < pe_N; c += 32) {
          tmem_ld32(taddr + c, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            __stcg(dst + (c >> 5) * 256 + j * 32,
                   make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                               __uint_as_float(r[4 * j + 3])));
        }
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(p.flags + pair, 1);
      } else {
        Fixup fx;
        void* cptr = pe_C;
        if (split && p.sw_parts > 1) {
          // last part of a divided tile: wait for the other parts (they run at the same time on the pairs just below
          // this one, which were started earlier) and add them in pair order
          fx.n = p.sw_parts - 1;
          const int first = pair - fx.n;
          fx.base = reinterpret_cast<const float4*>(p.slots) + (long long)first * SLOT_F4 + slot_f4;
          int got = 1;
          if (lane == 0)
            for (int s = 0; s < fx.n && got; ++s) got = flag_wait(p.flags + first + s, 2 * ((int)blockDim.x / 32 - 2), abort_flag, p.err) ? 1 : 0;
          got = __shfl_sync(0xffffffffu, got, 0);
          if (!got) break;
        } else if (p.ksplit > 1) {
          cptr = reinterpret_cast<float*>(p.C) + (long long)part * p.split_stride;  // this K part's own fp32 partial output
        }
        if constexpr (MODE == 2) {
          if (tma_epi) {
            if (tma_tile && !epilogue_swiglu_bwd_tma(p, em, taddr, m0 + q * 32, n0, cb, ce, fx, tbuf, tbar, tphase, abort_flag)) break;
          } else {
            epilogue_tile<BN, MODE>(p, cptr, taddr, row, n0, sq, stage, cb, ce, fx);
          }
        } else if constexpr (MODE == 3) {
          if (second) epilogue_tile<BN, 0>(p2, cptr, taddr, row, n0, sq, stage, cb, ce, fx);
          else epilogue_tile<BN, 0>(p, cptr, taddr, row, n0, sq, stage, cb, ce, fx);
        } else if constexpr (MODE == 0) {
          if (p.tma_out) {
            if (m0 + q * 32 < p.M) epilogue_bf16_tma(p, em, taddr, m0 + q * 32, n0, cb, ce, fx, tbuf);
          } else {
            epilogue_tile<BN, MODE>(p, cptr, taddr, row, n0, sq, stage, cb, ce, fx);
          }
        } else {
          epilogue_tile<BN, MODE>(p, cptr, taddr, row, n0, sq, stage, cb, ce, fx);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(tempty_bar(acc));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (p.adam_p != nullptr) {
      sq = warp_sum(sq);
      if (lane == 0) p.adam_sq[blockIdx.x * 8 + (warp - 2)] = sq;
    }
    if constexpr (MODE == 2) {
      if (tma_epi && lane == 0) bulk_wait_group0();  // this warp's tensor stores have landed before the kernel ends
    }
    if constexpr (MODE == 0) {
      if (p.tma_out && lane == 0) bulk_wait_group0();
    }
  }

  // teardown: both CTAs meet before either releases shared memory or TMEM the other may still be using
  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync_all();
  if (p.balanced && rank == 0 && threadIdx.x == 0) {
    // every warp of the pair has consumed the partials: clear the arrival counters this pair waited on for the next launch
    WorkIter mine(p, tiles_mn, kblocks_all, pair, npairs);
    if (mine.sw_tile >= 0 && mine.sw_part == p.sw_parts - 1)
      for (int s2 = 1; s2 < p.sw_parts; ++s2) p.flags[pair - s2] = 0;
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

// out[r, c] (+)= sum over K parts of partial[s][r, c], parts added in index order (deterministic).  ADAM: the sum is
// the finished gradient and goes straight into the AdamW update at (r, c) instead of being stored.
template <bool ADAM>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ partial, int nsplit, long long stride, float* __restrict__ out, long long ldc,
                     int M, int N, int accumulate, const GemmDev p) {
  __shared__ float s_sq[8];
  pdl_trigger();
  pdl_wait();
  float sq = 0.f;
  AdamCoef cf = {};
  if (ADAM) cf = adam_coef(p);
  const long long n4 = (long long)M * (N / 4);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / (N / 4);
    const int c = (int)(i % (N / 4)) * 4;
    float4 a = accumulate ? *reinterpret_cast<const float4*>(out + r * ldc + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nsplit; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(partial + s * stride + r * N + c);
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    if (!ADAM) {
      *reinterpret_cast<float4*>(out + r * ldc + c) = a;
    } else {
      const long long o = r * ldc + c;
      const float g[4] = {a.x, a.y, a.z, a.w};
      const float4 p4 = *reinterpret_cast<const float4*>(p.adam_p + o);
      const float4 m4 = *reinterpret_cast<const float4*>(p.adam_m + o);
      const float4 v4 = *reinterpret_cast<const float4*>(p.adam_v + o);
      float pp[4] = {p4.x, p4.y, p4.z, p4.w}, mm[4] = {m4.x, m4.y, m4.z, m4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        sq += g[e] * g[e];
        adamw_elem(g[e], p.adam_wd, cf, pp[e], mm[e], vv[e]);
      }
      *reinterpret_cast<float4*>(p.adam_p + o) = make_float4(pp[0], pp[1], pp[2], pp[3]);
      *reinterpret_cast<float4*>(p.adam_m + o) = make_float4(mm[0], mm[1], mm[2], mm[3]);
      *reinterpret_cast<float4*>(p.adam_v + o) = make_float4(vv[0], vv[1], vv[2], vv[3]);
      uint2 ob;
      ob.x = pack_bf16(pp[0], pp[1]);
      ob.y = pack_bf16(pp[2], pp[3]);
      *reinterpret_cast<uint2*>(p.adam_pb + o) = ob;
    }
  }
  if (ADAM) {
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) s_sq[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int w = 0; w < 8; ++w) tot += s_sq[w];
      p.adam_sq[blockIdx.x] = tot;
    }
  }
}

// ---------------------------------------------------------------- host side
void set_adam(GemmDev& p, const GemmArgs& a) {
  p.adam_p = nullptr; p.adam_m = nullptr; p.adam_v = nullptr; p.adam_pb = nullptr; p.adam_sc = nullptr; p.adam_sq = nullptr;
  p.adam_lr = p.adam_beta1 = p.adam_beta2 = p.adam_eps = p.adam_wd = 0.f;
  if (!a.adam) return;
  p.adam_p = a.adam->p; p.adam_m = a.adam->m; p.adam_v = a.adam->v; p.adam_pb = a.adam->pb;
  p.adam_sc = reinterpret_cast<const StepScalars*>(a.adam->scalars); p.adam_sq = a.adam->sq_slots;
  p.adam_lr = a.adam->lr; p.adam_beta1 = a.adam->beta1; p.adam_beta2 = a.adam->beta2; p.adam_eps = a.adam->eps;
  p.adam_wd = a.adam->wd;
}

int sm_count() {
  static int cache[64] = {0};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < 64 && cache[dev] > 0) return cache[dev];
  cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  if (n <= 0) n = 148;
  if (dev >= 0 && dev < 64) cache[dev] = n;
  return n;
}

template <int BN, bool A_MN, bool B_MN, int MODE = 0>
cudaError_t launch_variant(const GemmArgs& a, cudaStream_t stream) {
  using C = Cfg<BN>;
  auto kern = gemm_tc_kernel<BN, A_MN, B_MN, MODE>;
  static unsigned long long smem_set = 0;
  cudaError_t e0 = ensure_dynamic_smem(kern, C::SMEM_BYTES, smem_set);
  if (e0 != cudaSuccess) return e0;
  CUtensorMap tmA, tmB;
  bool ok = A_MN ? make_tmap_2d(&tmA, a.A, a.M, a.K, a.lda, 64) : make_tmap_2d(&tmA, a.A, a.K, a.M, a.lda, BM);
  ok = ok && (B_MN ? make_tmap_2d(&tmB, a.B, a.N, a.K, a.ldb, 64) : make_tmap_2d(&tmB, a.B, a.K, a.N, a.ldb, BN));
  if (!ok) return cudaErrorInvalidValue;
  GemmDev p;
  p.C = a.C; p.resid = a.resid; p.gu = a.gu; p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin; p.err = a.err;
  p.ldc = a.ldc; p.M = a.M; p.N = a.N; p.K = a.K; p.epi = a.epi;
  p.seq = a.seq; p.head_dim = a.head_dim; p.rope_cols = a.rope_cols; p.d_ffn = a.d_ffn; p.rope_ld = a.rope_ld;
  set_adam(p, a);
  p.alpha = a.alpha;
  {
    const bool f32out = a.epi == EPI_F32 || a.epi == EPI_F32_ACC;
    const int m = f32out ? 7 : 15;  // elements per 32 bytes, minus one
    bool ok32 = (reinterpret_cast<uintptr_t>(a.C) & 31) == 0 && (a.ldc & m) == 0 && (a.N & m) == 0;
    if (a.epi == EPI_BF16_RESID) ok32 = ok32 && (reinterpret_cast<uintptr_t>(a.resid) & 31) == 0;
    if (a.epi == EPI_SWIGLU || a.epi == EPI_SWIGLU_BWD) ok32 = ok32 && (reinterpret_cast<uintptr_t>(a.gu) & 31) == 0;
    p.wide_store = ok32 ? 1 : 0;
  }
  p.qk_r = a.qk_r; p.qk_gain_q = a.qk_gain_q; p.qk_gain_k = a.qk_gain_k; p.n_q_heads = a.n_q_heads; p.qk_eps = a.qk_eps;
  p.panel = (size_t)a.M * a.K * sizeof(bf16) > (48u << 20) ? 1 : 0;
  p.ksplit = 1; p.split_stride = 0; p.balanced = 0; p.sw_first = 0; p.sw_parts = 1; p.sw_kpb = 0; p.flags = nullptr; p.slots = nullptr;
  p.swiglu_tma = 0; p.tma_out = 0;
  p.g_tiles0 = 0; p.g_M = 0; p.g_N = 0; p.g_panel = 0; p.g_ldc = 0; p.g_C = nullptr; p.g_alpha = 1.0f;
  p.g_adam_p = nullptr; p.g_adam_m = nullptr; p.g_adam_v = nullptr; p.g_adam_pb = nullptr;
  p.ce_mode = 0; p.ce_tiles = 0; p.ce_part = nullptr; p.ce_zy = nullptr; p.ce_lse = nullptr; p.ce_labels = nullptr;
  p.ce_sc = nullptr; p.ce_scale = 1.0f;
  const int tiles = ((a.M + BM - 1) / BM) * ((a.N + BN - 1) / BN);
  const int grid = tiles < sm_count() ? tiles : sm_count();
  return launch_pdl(kern, grid, GEMM_THREADS, C::SMEM_BYTES, stream, tmA, tmB, p);
}

// b2: the second problem of a grouped launch (MODE 3 only; validated by gemm_group2_ok)
template <bool A_MN, bool B_MN, int MODE = 0>
cudaError_t launch_pair_variant(const GemmArgs& a, cudaStream_t stream, int* launches, const GemmArgs* b2 = nullptr) {
  using C = PairCfg;
  if ((MODE == 3) != (b2 != nullptr)) return cudaErrorInvalidValue;
  auto kern = gemm_tc_pair_kernel<A_MN, B_MN, MODE>;
  static unsigned long long smem_set = 0;
  cudaError_t e0 = ensure_dynamic_smem(kern, C::SMEM_BYTES, smem_set);
  if (e0 != cudaSuccess) return e0;
  CUtensorMap tmA, tmB;
  bool ok = A_MN ? make_tmap_2d(&tmA, a.A, a.M, a.K, a.lda, 64) : make_tmap_2d(&tmA, a.A, a.K, a.M, a.lda, BM);
  ok = ok && (B_MN ? make_tmap_2d(&tmB, a.B, a.N, a.K, a.ldb, 64) : make_tmap_2d(&tmB, a.B, a.K, a.N, a.ldb, C::HALF_B));
  if (!ok) return cudaErrorInvalidValue;
  GemmDev p;
  p.C = a.C; p.resid = a.resid; p.gu = a.gu; p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin; p.err = a.err;
  p.ldc = a.ldc; p.M = a.M; p.N = a.N; p.K = a.K; p.epi = a.epi;
  p.seq = a.seq; p.head_dim = a.head_dim; p.rope_cols = a.rope_cols; p.d_ffn = a.d_ffn; p.rope_ld = a.rope_ld;
  set_adam(p, a);
  p.alpha = a.alpha;
  {
    const bool f32out = a.epi == EPI_F32 || a.epi == EPI_F32_ACC;
    const int m = f32out ? 7 : 15;  // elements per 32 bytes, minus one
    bool ok32 = (reinterpret_cast<uintptr_t>(a.C) & 31) == 0 && (a.ldc & m) == 0 && (a.N & m) == 0;
    if (a.epi == EPI_BF16_RESID) ok32 = ok32 && (reinterpret_cast<uintptr_t>(a.resid) & 31) == 0;
    if (a.epi == EPI_SWIGLU || a.epi == EPI_SWIGLU_BWD) ok32 = ok32 && (reinterpret_cast<uintptr_t>(a.gu) & 31) == 0;
    p.wide_store = ok32 ? 1 : 0;
  }
  p.qk_r = a.qk_r; p.qk_gain_q = a.qk_gain_q; p.qk_gain_k = a.qk_gain_k; p.n_q_heads = a.n_q_heads; p.qk_eps = a.qk_eps;
  p.panel = (size_t)a.M * a.K * sizeof(bf16) > (48u << 20) ? 1 : 0;
  int tiles = ((a.M + 255) / 256) * ((a.N + 255) / 256);
  AuxMaps em;
  memset(&em, 0, sizeof(em));
  p.g_tiles0 = 0; p.g_M = 0; p.g_N = 0; p.g_panel = 0; p.g_ldc = 0; p.g_C = nullptr; p.g_alpha = 1.0f;
  p.g_adam_p = nullptr; p.g_adam_m = nullptr; p.g_adam_v = nullptr; p.g_adam_pb = nullptr;
  if (b2) {
    const GemmArgs& b = *b2;
    ok = A_MN ? make_tmap_2d(&em.m0, b.A, b.M, b.K, b.lda, 64) : make_tmap_2d(&em.m0, b.A, b.K, b.M, b.lda, BM);
    ok = ok && (B_MN ? make_tmap_2d(&em.m1, b.B, b.N, b.K, b.ldb, 64) : make_tmap_2d(&em.m1, b.B, b.K, b.N, b.ldb, C::HALF_B));
    if (!ok) return cudaErrorInvalidValue;
    p.g_tiles0 = tiles;
    p.g_M = b.M; p.g_N = b.N; p.g_ldc = b.ldc; p.g_C = b.C; p.g_alpha = b.alpha;
    p.g_panel = (size_t)b.M * b.K * sizeof(bf16) > (48u << 20) ? 1 : 0;
    if (b.adam) { p.g_adam_p = b.adam->p; p.g_adam_m = b.adam->m; p.g_adam_v = b.adam->v; p.g_adam_pb = b.adam->pb; }
    if ((reinterpret_cast<uintptr_t>(b.C) & 31) != 0 || (b.ldc & 7) != 0 || (b.N & 7) != 0) p.wide_store = 0;
    tiles += ((b.M + 255) / 256) * ((b.N + 255) / 256);
  }
  const int max_pairs = sm_count() / 2;
  // scratch layout: 256 arrival counters (kept zero between launches), then fp32 partial tiles
  int* flags = reinterpret_cast<int*>(a.scratch);
  float* data = a.scratch ? a.scratch + kScratchFlagFloats : nullptr;
  const size_t data_bytes = a.scratch_bytes > kScratchFlagFloats * sizeof(float) ? a.scratch_bytes - kScratchFlagFloats * sizeof(float) : 0;
  const int kblocks = (a.K + BK - 1) / BK;
  // split-K for weight gradients whose output has too few tiles to occupy the machine
  int ksplit = 1;
  if (A_MN && B_MN && !b2 && (a.epi == EPI_F32 || a.epi == EPI_F32_ACC) && data && tiles * 2 <= max_pairs) {
    int want = max_pairs / tiles;
    if (want > 8) want = 8;
    if (want > kblocks / 8) want = kblocks / 8;  // at least 8 K blocks per part
    if (want >= 2) {
      const int kpb = (kblocks + want - 1) / want;
      want = (kblocks + kpb - 1) / kpb;  // every part non-empty
      if (want >= 2 && (size_t)want * a.M * a.N * sizeof(float) <= data_bytes) ksplit = want;
    }
  }
  p.ksplit = ksplit;
  p.split_stride = (long long)a.M * a.N;
  if (ksplit > 1) { p.C = data; p.ldc = a.N; p.epi = EPI_F32; p.adam_p = nullptr; }  // the reduction applies AdamW instead
  // balanced schedule: a last wave that would keep at most half of the pairs busy is divided along K
  p.balanced = 0; p.sw_first = tiles; p.sw_parts = 1; p.sw_kpb = kblocks; p.flags = flags; p.slots = data;
  const int left = tiles % max_pairs;
  p.ce_mode = MODE == 1 ? a.ce_mode : 0; p.ce_tiles = a.ce_tiles; p.ce_part = a.ce_part; p.ce_zy = a.ce_zy; p.ce_lse = a.ce_lse;
  p.ce_labels = a.ce_labels; p.ce_sc = a.ce_scalars; p.ce_scale = a.ce_scale;
  // Only for contractions of at least 40 K blocks: a divided tile costs its pairs a pass of the fp32 partial through
  // scratch (4.6 us written, then read by the reducing pair) before the whole tiles start.  Against a 3 us main loop
  // (K 768) that makes the launch slower (8192 x 768 x 768: 37 against 29 us), at K 2048 it is a wash to a loss
  // (8192 x 2048 x 2048: 67.5 against 62.6 us), from K 4096 on it wins (8192 x 2048 x 11264: 230 against 249 us).
  if (MODE != 1 && g_gemm_balanced && ksplit == 1 && data && tiles > max_pairs && left > 0 && max_pairs <= 256 && kblocks >= 40 &&
      (size_t)max_pairs * SLOT_FLOATS * sizeof(float) <= data_bytes) {
    int parts = max_pairs / left;
    // The pair with part 0 adds the other parts' tiles while its next tile's main loop runs; the longer that loop (K),
    // the more partials fit into it without delaying the tile after.
    const int cap = kblocks < 48 ? 2 : (kblocks < 80 ? 3 : (kblocks < 112 ? 5 : 8));
    if (parts > cap) parts = cap;
    if (parts > kblocks / 4) parts = kblocks / 4;  // at least 4 K blocks per part
    const int waves = (tiles + max_pairs - 1) / max_pairs;
    if (parts >= 2 && (parts - 1) * 50 < parts * waves) parts = 1;  // saves under 2 % of the kernel: not worth the traffic
    if (parts >= 2) {
      const int kpb = (kblocks + parts - 1) / parts;
      parts = (kblocks + kpb - 1) / kpb;  // every part non-empty
      if (parts >= 2) { p.balanced = 1; p.sw_first = tiles - left; p.sw_parts = parts; p.sw_kpb = kpb; }
    }
  }
  const int work = tiles * ksplit;
  const int pairs = p.balanced ? max_pairs : (work < max_pairs ? work : max_pairs);
  if (p.balanced && a.scratch_reset) {
    cudaError_t e0 = cudaMemsetAsync(flags, 0, kScratchFlagFloats * sizeof(float), stream);
    if (e0 != cudaSuccess) return e0;
  }
  p.tma_out = 0;
  if (MODE == 0 && a.epi == EPI_BF16 && !a.adam && ksplit == 1 && g_gemm_tma_out && (reinterpret_cast<uintptr_t>(a.C) & 15) == 0 &&
      a.ldc % 8 == 0) {
    if (make_tmap_2d_rows32(&em.m1, reinterpret_cast<const bf16*>(a.C), a.N, a.M, a.ldc, 64)) p.tma_out = 1;
  }
  p.swiglu_tma = 0;
  if (MODE == 2 && a.epi == EPI_SWIGLU_BWD && !a.adam && g_gemm_swiglu_tma && (reinterpret_cast<uintptr_t>(a.gu) & 15) == 0 &&
      (reinterpret_cast<uintptr_t>(a.C) & 15) == 0 && a.ldc % 8 == 0) {
    // gate | up of the forward pass [M, 2 f] and the output d_gate / d_up [M, 2 f] (row stride ldc) as TMA tiles
    if (make_tmap_2d_rows32(&em.m0, a.gu, 2ULL * a.d_ffn, a.M, 2ULL * a.d_ffn, 32) &&
        make_tmap_2d_rows32(&em.m1, reinterpret_cast<const bf16*>(a.C), 2ULL * a.d_ffn, a.M, a.ldc, 64))
      p.swiglu_tma = 1;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  // eight epilogue warps only for the fused update (for short contractions, whose epilogue is the long pole too, they
  // changed nothing: that epilogue is bound by L2 store requests, not by warps)
  cfg.blockDim = dim3(a.adam ? PAIR_THREADS : GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = g_pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (launches) *launches = ksplit > 1 ? 2 : 1;
  GemmDev p2 = p;
  if (b2) {
    p2.M = p.g_M; p2.N = p.g_N; p2.ldc = p.g_ldc; p2.C = p.g_C; p2.panel = p.g_panel; p2.alpha = p.g_alpha;
    p2.adam_p = p.g_adam_p; p2.adam_m = p.g_adam_m; p2.adam_v = p.g_adam_v; p2.adam_pb = p.g_adam_pb;
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, em, p, p2);
  if (e != cudaSuccess || ksplit == 1) return e;
  const long long n4 = (long long)a.M * (a.N / 4);
  if (a.adam) {
    GemmDev pa = p;
    set_adam(pa, a);
    const int blocks = (int)((n4 + 255) / 256 < kAdamFuseSlots ? (n4 + 255) / 256 : kAdamFuseSlots);
    return launch_pdl(splitk_reduce_kernel<true>, blocks, 256, 0, stream, data, ksplit, p.split_stride,
                      reinterpret_cast<float*>(a.C), a.ldc, a.M, a.N, a.epi == EPI_F32_ACC ? 1 : 0, pa);
  } else {
    const int blocks = (int)((n4 + 255) / 256 < 1184 ? (n4 + 255) / 256 : 1184);
    return launch_pdl(splitk_reduce_kernel<false>, blocks, 256, 0, stream, data, ksplit, p.split_stride,
                      reinterpret_cast<float*>(a.C), a.ldc, a.M, a.N, a.epi == EPI_F32_ACC ? 1 : 0, p);
  }
  return cudaGetLastError();
}

}  // namespace

int g_gemm_force_bn = 0;
int g_gemm_pairs = 1;  // development knob: 1 = CTA-pair kernel for outputs of at least 256 x 256, 0 = single-CTA kernel only  // development knob: 0 = choose by tile count, 128 or 256 = force that tile width

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t stream, int* launches) {
  if (launches) *launches = 1;
  if (a.M <= 0 || a.N <= 0 || a.K <= 0 || !a.A || !a.B || !a.C || !a.err) return cudaErrorInvalidValue;
  if ((a.N & 7) || (a.lda & 7) || (a.ldb & 7) || (a.ldc & 3)) return cudaErrorInvalidValue;
  if ((a.a_mn ? a.M : a.K) & 7) return cudaErrorInvalidValue;
  if ((a.b_mn ? a.N : a.K) & 7) return cudaErrorInvalidValue;
  if ((reinterpret_cast<uintptr_t>(a.A) | reinterpret_cast<uintptr_t>(a.B) | reinterpret_cast<uintptr_t>(a.C)) & 15)
    return cudaErrorInvalidValue;
  if (a.epi == EPI_BF16_RESID && !a.resid) return cudaErrorInvalidValue;
  if (a.alpha != 1.0f && (a.epi == EPI_ROPE || a.epi == EPI_SWIGLU)) return cudaErrorInvalidValue;
  if (a.qk_r && (a.epi != EPI_ROPE || !a.qk_gain_q || !a.qk_gain_k)) return cudaErrorInvalidValue;
  if (a.adam && ((a.epi != EPI_F32 && a.epi != EPI_F32_ACC) || !a.adam->p || !a.adam->m || !a.adam->v || !a.adam->pb ||
                 !a.adam->scalars || !a.adam->sq_slots))
    return cudaErrorInvalidValue;
  if (a.epi == EPI_ROPE && (!a.rope_cos || !a.rope_sin || a.rope_ld < a.seq || (a.head_dim != 64 && a.head_dim != 128) || a.seq <= 0 ||
                            a.rope_cols % a.head_dim || a.N % a.head_dim))
    return cudaErrorInvalidValue;
  if (a.epi == EPI_SWIGLU && (!a.gu || a.d_ffn <= 0 || a.d_ffn % 16 || a.N != 2 * a.d_ffn)) return cudaErrorInvalidValue;
  if (a.epi == EPI_SWIGLU_BWD && (!a.gu || a.d_ffn <= 0 || a.d_ffn % 16 || a.N != a.d_ffn || a.ldc < 2LL * a.d_ffn ||
                                  (reinterpret_cast<uintptr_t>(a.gu) & 15)))
    return cudaErrorInvalidValue;
  // 128 x 256 tiles move 96 B of operands per tensor-core cycle through shared memory, 128 x 128 tiles 128 B: the
  // wide tile is faster even when it leaves SMs idle (measured), so the narrow one only serves N <= 128
  const bool wide = g_gemm_force_bn ? g_gemm_force_bn == 256 : a.N > 128;
  if (a.ce_mode != 0) {
    // streaming cross-entropy: the CTA-pair kernel's own instantiation; the caller pads nothing, rows and columns may be ragged
    if (a.a_mn || a.b_mn || a.adam || a.M < 1 || (a.ce_mode != 1 && a.ce_mode != 2) || !a.ce_labels ||
        a.ce_tiles != (a.N + 255) / 256)
      return cudaErrorInvalidValue;
    if (a.ce_mode == 1 && (!a.ce_part || !a.ce_zy)) return cudaErrorInvalidValue;
    if (a.ce_mode == 2 && (!a.ce_lse || !a.ce_scalars || a.epi != EPI_BF16)) return cudaErrorInvalidValue;
    return launch_pair_variant<false, false, 1>(a, stream, launches);
  }
  if (a.epi == EPI_SWIGLU_BWD) {
    // instantiations of their own (the epilogue's register needs stay out of the other kernels); data-gradient layout only
    if (a.a_mn || !a.b_mn || a.adam) return cudaErrorInvalidValue;
    if (g_gemm_pairs && !g_gemm_force_bn && a.M >= 256 && a.N >= 256) return launch_pair_variant<false, true, 2>(a, stream, launches);
    return wide ? launch_variant<256, false, true, 2>(a, stream) : launch_variant<128, false, true, 2>(a, stream);
  }
  if (g_gemm_pairs && !g_gemm_force_bn && a.M >= 256 && a.N >= 256) {
    if (!a.a_mn && !a.b_mn) return launch_pair_variant<false, false>(a, stream, launches);
    if (!a.a_mn && a.b_mn) return launch_pair_variant<false, true>(a, stream, launches);
    if (a.a_mn && a.b_mn) return launch_pair_variant<true, true>(a, stream, launches);
    return cudaErrorInvalidValue;
  }
  if (!a.a_mn && !a.b_mn) return wide ? launch_variant<256, false, false>(a, stream) : launch_variant<128, false, false>(a, stream);
  if (!a.a_mn && a.b_mn) return wide ? launch_variant<256, false, true>(a, stream) : launch_variant<128, false, true>(a, stream);
  if (a.a_mn && a.b_mn) return wide ? launch_variant<256, true, true>(a, stream) : launch_variant<128, true, true>(a, stream);
  return cudaErrorInvalidValue;  // (mn-major A with k-major B) is not needed by the train step
}

bool gemm_group2_ok(const GemmArgs& a, const GemmArgs& b) {
  if (!g_gemm_group || !g_gemm_pairs || g_gemm_force_bn) return false;
  if (!a.a_mn || !a.b_mn || !b.a_mn || !b.b_mn) return false;  // weight gradients only
  if (a.K != b.K || a.K <= 0 || a.M < 256 || a.N < 256 || b.M < 256 || b.N < 256) return false;
  if (a.epi != b.epi || (a.epi != EPI_F32 && a.epi != EPI_F32_ACC)) return false;
  if (a.ce_mode || b.ce_mode || a.err != b.err || !a.err) return false;
  if (a.scratch != b.scratch || a.scratch_bytes != b.scratch_bytes) return false;
  if ((a.adam == nullptr) != (b.adam == nullptr)) return false;
  if (a.adam) {
    const AdamFuse &x = *a.adam, &y = *b.adam;
    if (x.scalars != y.scalars || x.lr != y.lr || x.beta1 != y.beta1 || x.beta2 != y.beta2 || x.eps != y.eps || x.wd != y.wd)
      return false;
    if (!y.p || !y.m || !y.v || !y.pb) return false;
  }
  // the second problem's operands and output must pass the checks launch_gemm makes for the first
  if ((b.N & 7) || (b.lda & 7) || (b.ldb & 7) || (b.ldc & 3) || (b.M & 7)) return false;
  if (!b.A || !b.B || !b.C) return false;
  if ((reinterpret_cast<uintptr_t>(b.A) | reinterpret_cast<uintptr_t>(b.B) | reinterpret_cast<uintptr_t>(b.C)) & 15) return false;
  return true;
}

cudaError_t launch_gemm_group2(const GemmArgs& a, const GemmArgs& b, cudaStream_t stream, int* launches) {
  if (launches) *launches = 1;
  if (!gemm_group2_ok(a, b)) return cudaErrorInvalidValue;
  if (a.M <= 0 || a.N <= 0 || !a.A || !a.B || !a.C) return cudaErrorInvalidValue;
  if ((a.N & 7) || (a.lda & 7) || (a.ldb & 7) || (a.ldc & 3) || (a.M & 7)) return cudaErrorInvalidValue;
  if ((reinterpret_cast<uintptr_t>(a.A) | reinterpret_cast<uintptr_t>(a.B) | reinterpret_cast<uintptr_t>(a.C)) & 15)
    return cudaErrorInvalidValue;
  if (a.adam && (!a.adam->p || !a.adam->m || !a.adam->v || !a.adam->pb || !a.adam->scalars || !a.adam->sq_slots))
    return cudaErrorInvalidValue;
  return launch_pair_variant<true, true, 3>(a, stream, launches, &b);
}

}  // namespace fs
