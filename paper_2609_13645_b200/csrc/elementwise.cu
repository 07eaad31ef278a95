// Bandwidth-bound kernels of the train step.  All reductions run in a fixed order (no floating-point
// atomics), so results are bit-identical from run to run; all global accesses are 16-byte vectors.
#include "elementwise.cuh"

#include "adamw_math.cuh"

#include <math.h>

namespace fs {
namespace {

constexpr int kNormMaxChunks = 16;  // d_model <= 16 * 256

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 o;
  o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]); o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
  return o;
}

// ---------------------------------------------------------------- embedding forward
__global__ void embed_fwd_kernel(const int32_t* __restrict__ tok, const bf16* __restrict__ E, bf16* __restrict__ x,
                                 long long total_chunks, int chunks_per_row, int h, int vocab, float scale) {
  pdl_trigger();
  pdl_wait();
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_chunks;
       i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / chunks_per_row;
    const int c = (int)(i % chunks_per_row) * 8;
    int id = tok[t];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
    uint4 v = *reinterpret_cast<const uint4*>(E + (long long)id * h + c);
    if (scale != 1.0f) {  // x_0 = R(scale * E[token])
      float f[8];
      unpack8(v, f);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] *= scale;
      v = pack8(f);
    }
    *reinterpret_cast<uint4*>(x + t * h + c) = v;
  }
}

// ---------------------------------------------------------------- RMSNorm forward: one warp per row
__global__ void rmsnorm_fwd_kernel(const bf16* __restrict__ x, const bf16* __restrict__ g, bf16* __restrict__ y,
                                   float* __restrict__ r, int T, int h, float eps) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= T) return;
  const bf16* xr = x + (long long)row * h;
  float ss = 0.f;
  for (int c = lane * 8; c < h; c += 256) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + c), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) ss += f[e] * f[e];
  }
  ss = warp_sum(ss);
  const float rr = 1.0f / sqrtf(ss / (float)h + eps);
  if (lane == 0) r[row] = rr;
  bf16* yr = y + (long long)row * h;
  for (int c = lane * 8; c < h; c += 256) {
    float f[8], gg[8];
    unpack8(*reinterpret_cast<const uint4*>(xr + c), f);
    unpack8(*reinterpret_cast<const uint4*>(g + c), gg);
#pragma unroll
    for (int e = 0; e < 8; ++e) f[e] = f[e] * rr * gg[e];
    *reinterpret_cast<uint4*>(yr + c) = pack8(f);
  }
}

// ---------------------------------------------------------------- RMSNorm backward
// dx_k = r g_k dy_k - x_k r^3 (1/h) sum_j g_j dy_j x_j (+ resid_k);  dg_k = sum_t dy_tk x_tk r_t.
// WPR warps share a row (1 for h <= 2048, 2 above), rows strided over the grid.  A warp loads its whole share of the
// row with all 16-byte loads in flight at once, keeps it in registers for both the dot product and the update, and
// keeps the dg of its columns in registers; warps owning the same columns are then added in warp order, and a second
// kernel adds the block partials in block order (no floating-point atomics anywhere).
template <int NCHW, int WPR>
__global__ void __launch_bounds__(256)
rmsnorm_bwd_kernel(const bf16* __restrict__ dy, const bf16* __restrict__ x, const float* __restrict__ r,
                   const bf16* __restrict__ g, const bf16* __restrict__ resid, bf16* __restrict__ dx,
                   float* __restrict__ partial, int T, int h) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float s_dg[];  // [h]
  __shared__ float s_dot[2][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = warp % WPR;            // which part of the row this warp owns
  const int slot = warp / WPR;           // which of the block's concurrent rows
  constexpr int ROWS = 8 / WPR;          // rows in flight per block
  float dg[NCHW][8];
#pragma unroll
  for (int i = 0; i < NCHW; ++i)
#pragma unroll
    for (int e = 0; e < 8; ++e) dg[i][e] = 0.f;
  const float inv_h = 1.0f / (float)h;
  int parity = 0;
  const int nrows_iter = (T + gridDim.x * ROWS - 1) / (gridDim.x * ROWS);
  for (int it = 0; it < nrows_iter; ++it) {
    const int row = (it * gridDim.x + blockIdx.x) * ROWS + slot;
    const bool live = row < T;
    uint4 vdy[NCHW], vx[NCHW], vrs[NCHW];
#pragma unroll
    for (int i = 0; i < NCHW; ++i) {
      const int c = (sub * NCHW + i) * 256 + lane * 8;
      const bool okc = live && c < h;
      const long long off = (long long)row * h + c;
      vdy[i] = okc ? *reinterpret_cast<const uint4*>(dy + off) : make_uint4(0, 0, 0, 0);
      vx[i] = okc ? *reinterpret_cast<const uint4*>(x + off) : make_uint4(0, 0, 0, 0);
      vrs[i] = (okc && resid != nullptr) ? *reinterpret_cast<const uint4*>(resid + off) : make_uint4(0, 0, 0, 0);
    }
    const float rr = live ? r[row] : 0.f;
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < NCHW; ++i) {
      const int c = (sub * NCHW + i) * 256 + lane * 8;
      float a[8], b[8], gg[8];
      unpack8(vdy[i], a);
      unpack8(vx[i], b);
      unpack8(c < h ? *reinterpret_cast<const uint4*>(g + c) : make_uint4(0, 0, 0, 0), gg);  // gains stay in L1
#pragma unroll
      for (int e = 0; e < 8; ++e) dot += gg[e] * a[e] * b[e];
    }
    dot = warp_sum(dot);
    if (WPR == 2) {
      // the two warps of a row swap their halves of the dot product (added in a fixed order)
      if (lane == 0) s_dot[parity][warp] = dot;
      __syncthreads();
      const float d0 = s_dot[parity][slot * 2], d1 = s_dot[parity][slot * 2 + 1];
      dot = d0 + d1;
      parity ^= 1;
    }
    const float coef = rr * rr * rr * dot * inv_h;
#pragma unroll
    for (int i = 0; i < NCHW; ++i) {
      const int c = (sub * NCHW + i) * 256 + lane * 8;
      float a[8], b[8], gg[8], rs[8], o[8];
      unpack8(vdy[i], a);
      unpack8(vx[i], b);
      unpack8(c < h ? *reinterpret_cast<const uint4*>(g + c) : make_uint4(0, 0, 0, 0), gg);
      unpack8(vrs[i], rs);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        o[e] = rr * gg[e] * a[e] - b[e] * coef + rs[e];
        dg[i][e] += a[e] * b[e] * rr;
      }
      if (live && c < h) *reinterpret_cast<uint4*>(dx + (long long)row * h + c) = pack8(o);
    }
  }
  for (int w = 0; w < ROWS; ++w) {
    if (slot == w) {
#pragma unroll
      for (int i = 0; i < NCHW; ++i) {
        const int c = (sub * NCHW + i) * 256 + lane * 8;
        if (c < h) {
#pragma unroll
          for (int e = 0; e < 8; ++e) s_dg[c + e] = (w == 0 ? 0.f : s_dg[c + e]) + dg[i][e];
        }
      }
    }
    __syncthreads();
  }
  for (int c = threadIdx.x; c < h; c += blockDim.x) partial[(long long)blockIdx.x * h + c] = s_dg[c];
}

// Column sums of block partials, in block order: 32 columns x 8 row groups per CTA, the 8 groups (each a fixed strided
// subset of the blocks) are then added in group order.
// Many partial buffers at once: blockIdx.y selects slot y ([nblk][h] partials at partial + y * slot_floats) and
// the gradient tensor out[y] it sums into.  One launch at the end of the backward pass replaces one per norm.
__global__ void colsum_many_kernel(const float* __restrict__ partial, float* const* __restrict__ out, int nblk, int h,
                                   long long slot_floats) {
  pdl_trigger();
  pdl_wait();
  __shared__ float s[8][33];
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + cx;
  const float* src = partial + (long long)blockIdx.y * slot_floats;
  float a = 0.f;
  if (c < h)
    for (int b = ry; b < nblk; b += 8) a += src[(long long)b * h + c];
  s[ry][cx] = a;
  __syncthreads();
  if (ry == 0 && c < h) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s[w][cx];
    out[blockIdx.y][c] = tot;
  }
}

// the same for a partial buffer of 2 d columns whose halves belong to two output tensors (query gain | key gain);
// 32 row groups per block (the buffer has up to 1184 rows), added in group order
__global__ void __launch_bounds__(1024)
colsum2_kernel(const float* __restrict__ partial, float* __restrict__ out_a, float* __restrict__ out_b, int nblk, int d) {
  pdl_trigger();
  pdl_wait();
  __shared__ float s[32][33];
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + cx;
  float a = 0.f;
  if (c < 2 * d)
    for (int b = ry; b < nblk; b += 32) a += partial[(long long)b * 2 * d + c];
  s[ry][cx] = a;
  __syncthreads();
  if (ry == 0 && c < 2 * d) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 32; ++w) tot += s[w][cx];
    if (c < d) out_a[c] = tot; else out_b[c - d] = tot;
  }
}

// ---------------------------------------------------------------- SwiGLU backward
__global__ void swiglu_bwd_kernel(const bf16* __restrict__ d_a, const bf16* __restrict__ gu, bf16* __restrict__ d_gu,
                                  long long total_chunks, int chunks_per_row, int f) {
  pdl_trigger();
  pdl_wait();
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total_chunks;
       i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / chunks_per_row;
    const int c = (int)(i % chunks_per_row) * 8;
    float da[8], G[8], U[8], dG[8], dU[8];
    unpack8(*reinterpret_cast<const uint4*>(d_a + t * f + c), da);
    unpack8(*reinterpret_cast<const uint4*>(gu + t * 2 * f + c), G);
    unpack8(*reinterpret_cast<const uint4*>(gu + t * 2 * f + f + c), U);
#pragma unroll
    for (int e = 0; e < 8; ++e) swiglu_bwd_elem(da[e], G[e], U[e], dG[e], dU[e]);
    const int phys = ((c >> 4) << 5) + (c & 15);
    *reinterpret_cast<uint4*>(d_gu + t * 2 * f + phys) = pack8(dG);
    *reinterpret_cast<uint4*>(d_gu + t * 2 * f + phys + 16) = pack8(dU);
  }
}

// ---------------------------------------------------------------- loss
// Counts the labels that enter the loss, with the predicate the loss and its gradient use (0 <= label < vocab), and
// checks the ids: a label >= vocab or a token id outside [0, vocab) raises ERR_BAD_INDEX in *err (the step still runs,
// with such labels ignored and such ids clamped, and the next synchronising call reports the error).
__global__ void count_labels_kernel(const int32_t* __restrict__ labels, const int32_t* __restrict__ tok, int T, int vocab,
                                    StepScalars* sc, int* err, long long denom_override,
                                    const long long* __restrict__ denom_dev) {
  __shared__ int s[32];
  int c = 0;
  bool bad = false;
  for (int i = threadIdx.x; i < T; i += blockDim.x) {
    const int y = labels[i];
    c += (y >= 0 && y < vocab) ? 1 : 0;
    bad |= y >= vocab;
    if (tok != nullptr) { const int id = tok[i]; bad |= id < 0 || id >= vocab; }
  }
  if (bad && err != nullptr) atomicExch(err, (int)ERR_BAD_INDEX);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int tot = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += s[w];
    sc->count = tot;
    // data parallelism: the mean runs over the labels of all ranks, whose number the caller provides
    if (denom_dev != nullptr) denom_override = *denom_dev;  // the count of all ranks, reduced on the device
    const long long denom = denom_override > 0 ? denom_override : (long long)(tot > 0 ? tot : 1);
    sc->inv_count = 1.0f / (float)denom;
  }
}

// one block per row of logits
__global__ void __launch_bounds__(256)
cross_entropy_kernel(const float* __restrict__ z, const int32_t* __restrict__ labels, float* __restrict__ lse_out,
                     float* __restrict__ loss_row, bf16* __restrict__ dz, int V, const StepScalars* __restrict__ sc,
                     float dz_scale) {
  pdl_trigger();
  pdl_wait();
  __shared__ float s_m[8], s_s[8];
  __shared__ float s_lse;
  const int row = blockIdx.x;
  const float* zr = z + (long long)row * V;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float m = -INFINITY, s = 0.f;
  for (int c = threadIdx.x * 4; c < V; c += 1024) {
    const float4 v = *reinterpret_cast<const float4*>(zr + c);
    const float m4 = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
    if (m4 > m) {
      s *= expf(m - m4);
      m = m4;
    }
    s += expf(v.x - m) + expf(v.y - m) + expf(v.z - m) + expf(v.w - m);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
    const float mm = fmaxf(m, m2);
    // symmetric in (m,s) and (m2,s2) up to the commutative add, so both partners get the same bits
    const float a = (m == -INFINITY) ? 0.f : s * expf(m - mm);
    const float b = (m2 == -INFINITY) ? 0.f : s2 * expf(m2 - mm);
    s = (m >= m2) ? a + b : b + a;
    m = mm;
  }
  if (lane == 0) { s_m[warp] = m; s_s[warp] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float mm = s_m[0];
    for (int w = 1; w < 8; ++w) mm = fmaxf(mm, s_m[w]);
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += (s_m[w] == -INFINITY) ? 0.f : s_s[w] * expf(s_m[w] - mm);
    const float lse = mm + logf(tot);
    s_lse = lse;
    lse_out[row] = lse;
    const int y = labels[row];
    loss_row[row] = (y >= 0 && y < V) ? lse - zr[y] : 0.f;
  }
  __syncthreads();
  if (dz == nullptr) return;
  const float lse = s_lse;
  const int y = labels[row];
  const bool counted = y >= 0 && y < V;
  const float w = counted ? sc->inv_count * dz_scale : 0.f;  // dz_scale: the logit factor, folded into the one rounding
  bf16* dr = dz + (long long)row * V;
  for (int c = threadIdx.x * 4; c < V; c += 1024) {
    const float4 v = *reinterpret_cast<const float4*>(zr + c);
    float p0 = expf(v.x - lse), p1 = expf(v.y - lse), p2 = expf(v.z - lse), p3 = expf(v.w - lse);
    if (y == c) p0 -= 1.f;
    if (y == c + 1) p1 -= 1.f;
    if (y == c + 2) p2 -= 1.f;
    if (y == c + 3) p3 -= 1.f;
    uint2 o;
    o.x = pack_bf16(p0 * w, p1 * w);
    o.y = pack_bf16(p2 * w, p3 * w);
    *reinterpret_cast<uint2*>(dr + c) = o;
  }
}

// Streaming cross-entropy, second stage: one warp per row combines the (max, sum of e^(z - max)) pairs that the
// logits GEMM left per 256-column tile, in a fixed order, into the row's log-sum-exp and loss.
__global__ void __launch_bounds__(256)
ce_combine_kernel(const float2* __restrict__ part, int tiles, const float* __restrict__ zy, const int32_t* __restrict__ labels,
                  float* __restrict__ lse_out, float* __restrict__ loss_row, int rows, int V) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  float m = -INFINITY, s = 0.f;
  for (int t = lane; t < tiles; t += 32) {
    const float2 ps = part[(long long)row * tiles + t];
    const float mn = fmaxf(m, ps.x);
    const float a = (m == -INFINITY) ? 0.f : s * expf(m - mn);
    const float b = (ps.x == -INFINITY) ? 0.f : ps.y * expf(ps.x - mn);
    s = a + b;
    m = mn;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
    const float mm = fmaxf(m, m2);
    const float a = (m == -INFINITY) ? 0.f : s * expf(m - mm);
    const float b = (m2 == -INFINITY) ? 0.f : s2 * expf(m2 - mm);
    s = (m >= m2) ? a + b : b + a;  // both partners add in the same order
    m = mm;
  }
  if (lane == 0) {
    const float lse = m + logf(s);
    lse_out[row] = lse;
    const int y = labels[row];
    loss_row[row] = (y >= 0 && y < V) ? lse - zy[row] : 0.f;
  }
}

// MTP head inputs: inside every sequence the ids move up by one (the last position keeps its own id) and the labels
// move up by one (the last position gets -1: no successor, not counted)
__global__ void mtp_shift_kernel(const int32_t* __restrict__ tok, const int32_t* __restrict__ lab, int32_t* __restrict__ tok2,
                                 int32_t* __restrict__ lab2, int T, int S) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T) return;
  const bool last = (i % S) == S - 1;
  tok2[i] = last ? tok[i] : tok[i + 1];
  lab2[i] = last ? -1 : lab[i + 1];
}

// loss <- loss + weight * (the MTP head's mean cross-entropy)
__global__ void add_loss_kernel(StepScalars* sc, const StepScalars* sc2, float weight) {
  const float loss = sc->loss + weight * sc2->loss;
  sc->loss = loss;
  sc->nonfinite = isfinite(loss) ? 0 : 1;
}

__global__ void reduce_loss_kernel(const float* __restrict__ loss_row, int T, StepScalars* sc) {
  __shared__ float s[1024];
  float a = 0.f;
  for (int i = threadIdx.x; i < T; i += blockDim.x) a += loss_row[i];
  s[threadIdx.x] = a;
  __syncthreads();
  for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float loss = s[0] * sc->inv_count;
    sc->loss = loss;
    sc->nonfinite = isfinite(loss) ? 0 : 1;
  }
}

// ---------------------------------------------------------------- embedding backward (sort + ordered segment sums)
constexpr int kSortChunk = 4096;
constexpr int kSortThreads = 512;

__global__ void make_keys_kernel(const int32_t* __restrict__ tok, unsigned long long* __restrict__ keys, int T, int n_pad,
                                 int vocab) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pad) return;
  if (i < T) {
    int id = tok[i];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
    keys[i] = ((unsigned long long)(unsigned)id << 32) | (unsigned)i;
  } else {
    keys[i] = ~0ull;
  }
}

__device__ __forceinline__ void cmp_swap(unsigned long long& a, unsigned long long& b, bool up) {
  if ((a > b) == up) {
    const unsigned long long t = a;
    a = b;
    b = t;
  }
}

// sorts (k_lo == 2) or merges (k_lo == k_hi) one chunk in shared memory: runs the network steps (k, j) for
// k = k_lo..k_hi and j = min(k/2, chunk/2)..1
__global__ void __launch_bounds__(kSortThreads)
bitonic_chunk_kernel(unsigned long long* __restrict__ keys, int k_lo, int k_hi) {
  __shared__ unsigned long long s[kSortChunk];
  const int base = blockIdx.x * kSortChunk;
  for (int i = threadIdx.x; i < kSortChunk; i += kSortThreads) s[i] = keys[base + i];
  __syncthreads();
  for (int k = k_lo; k <= k_hi; k <<= 1) {
    for (int j = min(k >> 1, kSortChunk >> 1); j > 0; j >>= 1) {
      for (int p = threadIdx.x; p < kSortChunk / 2; p += kSortThreads) {
        const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));  // index with bit j clear
        const bool up = ((base + i) & k) == 0;
        cmp_swap(s[i], s[i | j], up);
      }
      __syncthreads();
    }
  }
  for (int i = threadIdx.x; i < kSortChunk; i += kSortThreads) keys[base + i] = s[i];
}

__global__ void bitonic_global_kernel(unsigned long long* __restrict__ keys, int n_pad, int k, int j) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= n_pad / 2) return;
  const int i = ((p & ~(j - 1)) << 1) | (p & (j - 1));
  const bool up = (i & k) == 0;
  unsigned long long a = keys[i], b = keys[i | j];
  if ((a > b) == up) {
    keys[i] = b;
    keys[i | j] = a;
  }
}

// block (i, y) works only if sorted position i starts a run of equal tokens; it owns columns [256 y, 256 y + 256) of
// that token's gradient row.  Its 8 warps take contiguous eighths of the run (position order, four rows in flight,
// added in position order), and the eight partial rows are added in warp order.  A token as frequent as id 0 of a
// Zipf stream (14 % of the positions) is thus spread over h / 256 blocks instead of one.
__global__ void __launch_bounds__(256)
embed_bwd_kernel(const unsigned long long* __restrict__ keys, const bf16* __restrict__ dx, float* __restrict__ dE, int T,
                 int h, float scale, int accumulate) {
  __shared__ int s_end;
  __shared__ float s_part[8][256];
  const int i = blockIdx.x;
  const unsigned long long key = keys[i];
  const unsigned tokid = (unsigned)(key >> 32);
  if (i > 0 && (unsigned)(keys[i - 1] >> 32) == tokid) return;
  if (threadIdx.x == 0) {
    const unsigned long long bound = ((unsigned long long)tokid + 1ull) << 32;  // first key of the next token
    int lo = i + 1, hi = T;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (keys[mid] < bound) lo = mid + 1; else hi = mid;
    }
    s_end = lo;
  }
  __syncthreads();
  const int len = s_end - i;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r0 = i + (int)(((long long)len * warp) / 8), r1 = i + (int)(((long long)len * (warp + 1)) / 8);
  const int slab = blockIdx.y * 256;
  const int c = slab + lane * 8;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c < h) {
    int rpos = r0;
    for (; rpos + 4 <= r1; rpos += 4) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const unsigned pos = (unsigned)(keys[rpos + u] & 0xffffffffull);
        v[u] = *reinterpret_cast<const uint4*>(dx + (long long)pos * h + c);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float f[8];
        unpack8(v[u], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += f[e];
      }
    }
    for (; rpos < r1; ++rpos) {
      const unsigned pos = (unsigned)(keys[rpos] & 0xffffffffull);
      float f[8];
      unpack8(*reinterpret_cast<const uint4*>(dx + (long long)pos * h + c), f);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += f[e];
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) s_part[warp][lane * 8 + e] = acc[e];
  __syncthreads();
  const int col = slab + threadIdx.x;
  if (col < h) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_part[w][threadIdx.x];
    // tied embeddings: the table's gradient already holds the output head's part, this row's sum is added to it
    float* dst = dE + (long long)tokid * h + col;
    *dst = accumulate ? *dst + scale * tot : scale * tot;
  }
}

// ---------------------------------------------------------------- gradient norm, step scalars, AdamW
__global__ void __launch_bounds__(256)
sqnorm_partial_kernel(const float* __restrict__ g, size_t n4, float* __restrict__ partial) {
  __shared__ float s[8];
  float a = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 v = reinterpret_cast<const float4*>(g)[i];
    a += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  a = warp_sum(a);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int w = 0; w < 8; ++w) tot += s[w];
    partial[blockIdx.x] = tot;
  }
}

__global__ void sqnorm_final_kernel(const float* __restrict__ partial, int nblk, StepScalars* sc, AdamHyper hp) {
  __shared__ float s[256];
  float a = 0.f;
  for (int i = threadIdx.x; i < nblk; i += 256) a += partial[i];
  s[threadIdx.x] = a;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float gn = sqrtf(fmaxf(s[0], 0.f));
    sc->gnorm = gn;
    sc->clip = hp.max_grad_norm > 0.f ? fminf(1.0f, hp.max_grad_norm / (gn + 1e-6f)) : 1.0f;
  }
}

// sum of the block partials in index order -> *out (one block)
__global__ void sqnorm_sum_kernel(const float* __restrict__ partial, int nblk, float* __restrict__ out) {
  __shared__ float s[256];
  float a = 0.f;
  for (int i = threadIdx.x; i < nblk; i += 256) a += partial[i];
  s[threadIdx.x] = a;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = s[0];
}

// norm and clip coefficient from a sum of squares that was formed elsewhere (over all ranks' shards)
__global__ void clip_from_sq_kernel(const float* __restrict__ sq_total, StepScalars* sc, AdamHyper hp) {
  const float gn = sqrtf(fmaxf(*sq_total, 0.f));
  sc->gnorm = gn;
  sc->clip = hp.max_grad_norm > 0.f ? fminf(1.0f, hp.max_grad_norm / (gn + 1e-6f)) : 1.0f;
}

__global__ void advance_step_kernel(StepScalars* sc, AdamHyper hp) {
  const long long t = sc->step + 1;
  sc->step = t;
  sc->bc1 = (float)(1.0 - pow((double)hp.beta1, (double)t));
  sc->bc2 = (float)(1.0 - pow((double)hp.beta2, (double)t));
}

// WITH_NORM: clipping is off (coefficient 1), so the squared gradient norm is summed in the same pass and written
// as one partial per block (fixed order: thread-strided, warp shuffle, warp order).
template <bool WITH_NORM>
__global__ void __launch_bounds__(256)
adamw_kernel(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v, const float* __restrict__ g,
             bf16* __restrict__ pb, size_t n4, size_t n4_decay, const StepScalars* __restrict__ sc, AdamHyper hp,
             float* __restrict__ sq_partial) {
  __shared__ float s_sq[8];
  const float clip = WITH_NORM ? 1.0f : sc->clip;
  const AdamCoef c = make_adam_coef(hp.lr, hp.beta1, hp.beta2, hp.eps, sc->bc1, sc->bc2);
  float sq = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float wd = i < n4_decay ? hp.wd : 0.f;
    const float4 g4 = reinterpret_cast<const float4*>(g)[i];
    float4 p4 = reinterpret_cast<float4*>(p)[i];
    float4 m4 = reinterpret_cast<float4*>(m)[i];
    float4 v4 = reinterpret_cast<float4*>(v)[i];
    float gg[4] = {g4.x, g4.y, g4.z, g4.w};
    float pp[4] = {p4.x, p4.y, p4.z, p4.w};
    float mm[4] = {m4.x, m4.y, m4.z, m4.w};
    float vv[4] = {v4.x, v4.y, v4.z, v4.w};
    if (WITH_NORM) sq += g4.x * g4.x + g4.y * g4.y + g4.z * g4.z + g4.w * g4.w;
#pragma unroll
    for (int e = 0; e < 4; ++e) adamw_elem(__fmul_rn(gg[e], clip), wd, c, pp[e], mm[e], vv[e]);
    reinterpret_cast<float4*>(p)[i] = make_float4(pp[0], pp[1], pp[2], pp[3]);
    reinterpret_cast<float4*>(m)[i] = make_float4(mm[0], mm[1], mm[2], mm[3]);
    reinterpret_cast<float4*>(v)[i] = make_float4(vv[0], vv[1], vv[2], vv[3]);
    uint2 o;
    o.x = pack_bf16(pp[0], pp[1]);
    o.y = pack_bf16(pp[2], pp[3]);
    reinterpret_cast<uint2*>(pb)[i] = o;
  }
  if (WITH_NORM) {
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) s_sq[threadIdx.x >> 5] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
      float tot = 0.f;
      for (int w = 0; w < 8; ++w) tot += s_sq[w];
      sq_partial[blockIdx.x] = tot;
    }
  }
}

// ---------------------------------------------------------------- per-head QK-Norm backward
// D/8 lanes per (token, head) row of D entries of dqkv (query heads, then key heads), in place.  dy = the row as the
// attention backward left it (gradient with respect to the normalised, gained, un-rotated head).  The unit-RMS value
// x_hat = x r is rebuilt from the stored rotated head: x_hat = rotate^-1(q) / gain.  Then
//   dx = r (gain dy - x_hat mean_k(gain dy x_hat)),   dgain_k += dy_k x_hat_k.
// Rows are dealt to warps in a fixed grid-strided order and every warp keeps its dgain sums in registers; warps are
// added in warp order into one partial row per block ([block][2][D]: query gain, key gain), blocks by colsum.
template <int D>
__global__ void __launch_bounds__(256)
qknorm_bwd_kernel(bf16* __restrict__ dqkv, const bf16* __restrict__ qkv, const float* __restrict__ rr,
                  const bf16* __restrict__ gain_q, const bf16* __restrict__ gain_k, const float* __restrict__ cosT,
                  const float* __restrict__ sinT, float* __restrict__ partial, float inv_mscale2, int T, int S, int nh,
                  int nkv) {
  pdl_trigger();
  pdl_wait();
  constexpr int HALF = D / 2;
  constexpr int LPR = D / 8;     // lanes per row: each owns columns 4 l .. 4 l + 3 and the same + D/2 (8-byte accesses)
  constexpr int RPW = 32 / LPR;  // rows a warp handles at once
  __shared__ float s_dg[8][2][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int sub = lane / LPR, l = lane % LPR, c0 = 4 * l;
  const int heads = nh + nkv, nqkv = (nh + 2 * nkv) * D;
  float dgq[8], dgk[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) { dgq[e] = 0.f; dgk[e] = 0.f; }
  auto load4 = [](const bf16* p, float* f) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
  };
  // this lane's eight gains of either kind and their reciprocals (rounded once), the same for every row
  float gq[8], gk[8], rgq[8], rgk[8];
  load4(gain_q + c0, gq); load4(gain_q + c0 + HALF, gq + 4);
  load4(gain_k + c0, gk); load4(gain_k + c0 + HALF, gk + 4);
#pragma unroll
  // the tables carry a magnitude factor m (LongRoPE form): rotating back with them gives m^2 x, hence inv_mscale2
  for (int e = 0; e < 8; ++e) { rgq[e] = __frcp_rn(gq[e]) * inv_mscale2; rgk[e] = __frcp_rn(gk[e]) * inv_mscale2; }
  const int rows = T * heads;  // at most 2^24 tokens x heads: fits
  const int stride = (int)gridDim.x * 8 * RPW;
  for (int base = ((int)blockIdx.x * 8 + warp) * RPW; base < rows; base += stride) {
    const int row = base + sub;
    const bool live = row < rows;
    const int rw = live ? row : 0;
    const int t = rw / heads, hd = rw - t * heads;
    const bool is_q = hd < nh;
    const long long off = (long long)t * nqkv + (is_q ? hd * D : nh * D + (hd - nh) * D) + c0;
    const int pos = t % S;
    float q1[4], q2[4], dy[8], gn[8], rg[8], xh[8];
    load4(qkv + off, q1);
    load4(qkv + off + HALF, q2);
    load4(dqkv + off, dy);
    load4(dqkv + off + HALF, dy + 4);
#pragma unroll
    for (int e = 0; e < 8; ++e) { gn[e] = is_q ? gq[e] : gk[e]; rg[e] = is_q ? rgq[e] : rgk[e]; }
    const float4 cs4 = *reinterpret_cast<const float4*>(cosT + (long long)pos * HALF + c0);
    const float4 sn4 = *reinterpret_cast<const float4*>(sinT + (long long)pos * HALF + c0);
    const float cs[4] = {cs4.x, cs4.y, cs4.z, cs4.w}, sn[4] = {sn4.x, sn4.y, sn4.z, sn4.w};
    float dot = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      xh[e] = (q1[e] * cs[e] + q2[e] * sn[e]) * rg[e];          // inverse rotation, then the gain divided out
      xh[4 + e] = (q2[e] * cs[e] - q1[e] * sn[e]) * rg[4 + e];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) dot += gn[e] * dy[e] * xh[e];
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
    dot *= 1.0f / (float)D;
    const float r = live ? rr[row] : 0.f;
    if (live) {
      float o[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) o[e] = r * (gn[e] * dy[e] - xh[e] * dot);
      uint2 w0, w1;
      w0.x = pack_bf16(o[0], o[1]); w0.y = pack_bf16(o[2], o[3]);
      w1.x = pack_bf16(o[4], o[5]); w1.y = pack_bf16(o[6], o[7]);
      *reinterpret_cast<uint2*>(dqkv + off) = w0;
      *reinterpret_cast<uint2*>(dqkv + off + HALF) = w1;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        if (is_q) dgq[e] += dy[e] * xh[e]; else dgk[e] += dy[e] * xh[e];
      }
    }
  }
  // the RPW row groups of a warp, added in group order (lane sub 0 collects), then warps in warp order
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    float aq = 0.f, ak = 0.f;
#pragma unroll
    for (int u = 0; u < RPW; ++u) {
      aq += __shfl_sync(0xffffffffu, dgq[e], u * LPR + l);
      ak += __shfl_sync(0xffffffffu, dgk[e], u * LPR + l);
    }
    if (sub == 0) {
      const int c = (e < 4) ? c0 + e : HALF + c0 + (e - 4);
      s_dg[warp][0][c] = aq;
      s_dg[warp][1][c] = ak;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 2 * D; i += blockDim.x) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_dg[w][i / D][i % D];
    partial[(long long)blockIdx.x * 2 * D + i] = tot;
  }
}

// ---------------------------------------------------------------- initialisation
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// wgu_cols > 0: the tensor is the gate|up matrix [2f, wgu_cols] stored with rows interleaved 16 gate / 16 up; position i
// of the stored tensor then holds the draw of its LOGICAL element (gate rows 0..f-1, then up rows 0..f-1)
__global__ void init_normal_kernel(float* __restrict__ p, size_t n, unsigned long long seed, unsigned long long tensor_id,
                                   double stddev, int wgu_cols, int f) {
  for (size_t pos = (size_t)blockIdx.x * blockDim.x + threadIdx.x; pos < n; pos += (size_t)gridDim.x * blockDim.x) {
    size_t i = pos;
    if (wgu_cols > 0) {
      const size_t pr = pos / (size_t)wgu_cols, c = pos - pr * (size_t)wgu_cols;
      const size_t blk = pr >> 5, within = pr & 31;
      const size_t lr = within < 16 ? blk * 16 + within : (size_t)f + blk * 16 + (within - 16);
      i = lr * (size_t)wgu_cols + c;
    }
    const unsigned long long k = seed ^ ((tensor_id + 1ull) * 0xD1B54A32D192ED03ull) ^ ((unsigned long long)i * 0x8CB92BA72F3D8DD7ull);
    const unsigned long long r = splitmix64(k);
    const double u1 = ((double)(r >> 40) + 1.0) / 16777216.0;
    const double u2 = (double)((r >> 16) & 0xFFFFFFull) / 16777216.0;
    const double z = sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925286766559 * u2);
    p[pos] = (float)(z * stddev);
  }
}

__global__ void fill_kernel(float* __restrict__ p, size_t n, float v) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) p[i] = v;
}

__global__ void cast_bf16_kernel(const float* __restrict__ src, bf16* __restrict__ dst, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}

inline int grid_for(size_t work_items, int threads, int max_blocks = 148 * 16) {
  size_t b = (work_items + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > (size_t)max_blocks) b = max_blocks;
  return (int)b;
}
inline int ok(int launches) { return cudaGetLastError() == cudaSuccess ? launches : -1; }

}  // namespace

int elementwise_blocks_for_norm(int T) {
  const int need = (T + 7) / 8;
  return need < 296 ? need : 296;  // two resident CTAs per SM
}

size_t sort_pad(size_t n) {
  size_t p = kSortChunk;
  while (p < n) p <<= 1;
  return p;
}

int embed_fwd(const int32_t* tok, const bf16* E, bf16* x, int T, int h, int vocab, float scale, cudaStream_t st) {
  const long long total = (long long)T * (h / 8);
  if (launch_pdl(embed_fwd_kernel, grid_for(total, 256), 256, 0, st, tok, E, x, total, h / 8, h, vocab, scale) != cudaSuccess) return -1;
  return ok(1);
}

int rmsnorm_fwd(const bf16* x, const bf16* g, bf16* y, float* r, int T, int h, float eps, cudaStream_t st) {
  if (launch_pdl(rmsnorm_fwd_kernel, (T + 7) / 8, 256, 0, st, x, g, y, r, T, h, eps) != cudaSuccess) return -1;
  return ok(1);
}

template <int NCHW, int WPR>
static void launch_rmsnorm_bwd(int nblk, const bf16* dy, const bf16* x, const float* r, const bf16* g, const bf16* resid,
                               bf16* dx, float* partial, int T, int h, cudaStream_t st) {
  launch_pdl(rmsnorm_bwd_kernel<NCHW, WPR>, nblk, 256, h * sizeof(float), st, dy, x, r, g, resid, dx, partial, T, h);
}

int rmsnorm_bwd(const bf16* dy, const bf16* x, const float* r, const bf16* g, const bf16* resid, bf16* dx,
                float* partial, int T, int h, cudaStream_t st) {
  if ((h & 255) || h > 256 * kNormMaxChunks) return -1;
  const int nblk = elementwise_blocks_for_norm(T);
  const int nch = h >> 8;
#define FS_NORM_CASE(N, W) launch_rmsnorm_bwd<N, W>(nblk, dy, x, r, g, resid, dx, partial, T, h, st); break
  if (nch <= 4) {
    switch (nch) {
      case 1: FS_NORM_CASE(1, 1); case 2: FS_NORM_CASE(2, 1); case 3: FS_NORM_CASE(3, 1); case 4: FS_NORM_CASE(4, 1);
      default: FS_NORM_CASE(4, 1);
    }
  } else {
    // two warps per row from h = 1280 up: half the registers per thread, so two CTAs fit on an SM
    switch ((nch + 1) / 2) {
      case 3: FS_NORM_CASE(3, 2); case 4: FS_NORM_CASE(4, 2); case 5: FS_NORM_CASE(5, 2); case 6: FS_NORM_CASE(6, 2); case 7: FS_NORM_CASE(7, 2); default: FS_NORM_CASE(8, 2);
    }
  }
#undef FS_NORM_CASE
  return ok(1);
}

int colsum_many(const float* partial, float* const* out, int nslots, size_t slot_floats, int T, int h, cudaStream_t st) {
  if (nslots <= 0) return 0;
  const int nblk = elementwise_blocks_for_norm(T);
  if (launch_pdl(colsum_many_kernel, dim3((h + 31) / 32, nslots), 256, 0, st, partial, out, nblk, h, (long long)slot_floats) != cudaSuccess) return -1;
  return ok(1);
}

int qknorm_bwd(bf16* dqkv, const bf16* qkv, const float* r, const bf16* gain_q, const bf16* gain_k, const float* cosT,
               const float* sinT, float* dgain_q, float* dgain_k, float* partial, size_t partial_floats, float inv_mscale2,
               int T, int S, int nh, int nkv, int d, cudaStream_t st) {
  // many small blocks: the kernel is a chain of short dependent loads per row, so it lives on blocks in flight
  const long long rows = (long long)T * (nh + nkv);
  long long want = (rows + 8 * (32 / (d / 8)) - 1) / (8 * (32 / (d / 8)));
  const long long cap = (long long)(partial_floats / (2 * (size_t)d));
  if (want > 148 * 8) want = 148 * 8;
  if (want > cap) want = cap;
  if (want < 1) return -1;
  const int nblk = (int)want;
  cudaError_t e;
  if (d == 64) e = launch_pdl(qknorm_bwd_kernel<64>, nblk, 256, 0, st, dqkv, qkv, r, gain_q, gain_k, cosT, sinT, partial, inv_mscale2, T, S, nh, nkv);
  else if (d == 128) e = launch_pdl(qknorm_bwd_kernel<128>, nblk, 256, 0, st, dqkv, qkv, r, gain_q, gain_k, cosT, sinT, partial, inv_mscale2, T, S, nh, nkv);
  else return -1;
  if (e != cudaSuccess) return -1;
  // partial is [nblk][2 d]: column sums give dgain_q | dgain_k side by side; they land in two gradient tensors
  if (launch_pdl(colsum2_kernel, (2 * d + 31) / 32, 1024, 0, st, partial, dgain_q, dgain_k, nblk, d) != cudaSuccess) return -1;
  return ok(2);
}

int swiglu_bwd(const bf16* d_a, const bf16* gu, bf16* d_gu, int T, int f, cudaStream_t st) {
  const long long total = (long long)T * (f / 8);
  if (launch_pdl(swiglu_bwd_kernel, grid_for(total, 256), 256, 0, st, d_a, gu, d_gu, total, f / 8, f) != cudaSuccess) return -1;
  return ok(1);
}

int count_labels(const int32_t* labels, const int32_t* tok, int T, int vocab, StepScalars* sc, int* err,
                 long long denom_override, const long long* denom_dev, cudaStream_t st) {
  count_labels_kernel<<<1, 1024, 0, st>>>(labels, tok, T, vocab, sc, err, denom_override, denom_dev);
  return ok(1);
}

int cross_entropy_rows(const float* z, const int32_t* labels, float* lse, float* loss_row, bf16* dz, int rows, int V,
                       const StepScalars* sc, float dz_scale, cudaStream_t st) {
  if (launch_pdl(cross_entropy_kernel, rows, 256, 0, st, z, labels, lse, loss_row, dz, V, sc, dz_scale) != cudaSuccess) return -1;
  return ok(1);
}

int ce_combine(const float2* part, int tiles, const float* zy, const int32_t* labels, float* lse, float* loss_row, int rows,
               int V, cudaStream_t st) {
  if (launch_pdl(ce_combine_kernel, (rows + 7) / 8, 256, 0, st, part, tiles, zy, labels, lse, loss_row, rows, V) != cudaSuccess) return -1;
  return ok(1);
}

int mtp_shift(const int32_t* tok, const int32_t* lab, int32_t* tok2, int32_t* lab2, int T, int S, cudaStream_t st) {
  mtp_shift_kernel<<<(T + 255) / 256, 256, 0, st>>>(tok, lab, tok2, lab2, T, S);
  return ok(1);
}

int add_loss(StepScalars* sc, const StepScalars* sc2, float weight, cudaStream_t st) {
  add_loss_kernel<<<1, 1, 0, st>>>(sc, sc2, weight);
  return ok(1);
}

int reduce_loss(const float* loss_row, int T, StepScalars* sc, cudaStream_t st) {
  reduce_loss_kernel<<<1, 1024, 0, st>>>(loss_row, T, sc);
  return ok(1);
}

int embed_bwd(const int32_t* tok, const bf16* dx, float* dE, unsigned long long* keys, int T, int h, int vocab,
              float scale, bool accumulate, cudaStream_t st) {
  const int n_pad = (int)sort_pad((size_t)T);
  int launches = 0;
  make_keys_kernel<<<(n_pad + 255) / 256, 256, 0, st>>>(tok, keys, T, n_pad, vocab);
  ++launches;
  const int nchunks = n_pad / kSortChunk;
  bitonic_chunk_kernel<<<nchunks, kSortThreads, 0, st>>>(keys, 2, kSortChunk);
  ++launches;
  for (int k = kSortChunk * 2; k <= n_pad; k <<= 1) {
    for (int j = k >> 1; j >= kSortChunk; j >>= 1) {
      bitonic_global_kernel<<<(n_pad / 2 + 255) / 256, 256, 0, st>>>(keys, n_pad, k, j);
      ++launches;
    }
    bitonic_chunk_kernel<<<nchunks, kSortThreads, 0, st>>>(keys, k, k);
    ++launches;
  }
  if (!accumulate && cudaMemsetAsync(dE, 0, (size_t)vocab * h * sizeof(float), st) != cudaSuccess) return -1;
  embed_bwd_kernel<<<dim3(T, (h + 255) / 256), 256, 0, st>>>(keys, dx, dE, T, h, scale, accumulate ? 1 : 0);
  ++launches;
  return ok(launches);
}

int grad_norm_and_clip(const float* g, size_t n, float* partial, StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  sqnorm_partial_kernel<<<kSqnormBlocks, 256, 0, st>>>(g, n / 4, partial);
  sqnorm_final_kernel<<<1, 256, 0, st>>>(partial, kSqnormBlocks, sc, hp);
  return ok(2);
}

int sqnorm_to(const float* g, size_t n, float* partial, float* out, cudaStream_t st) {
  sqnorm_partial_kernel<<<kSqnormBlocks, 256, 0, st>>>(g, n / 4, partial);
  sqnorm_sum_kernel<<<1, 256, 0, st>>>(partial, kSqnormBlocks, out);
  return ok(2);
}

int clip_from_sq(const float* sq_total, StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  clip_from_sq_kernel<<<1, 1, 0, st>>>(sq_total, sc, hp);
  return ok(1);
}

int advance_step(StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  advance_step_kernel<<<1, 1, 0, st>>>(sc, hp);
  return ok(1);
}

int adamw(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, const StepScalars* sc,
          AdamHyper hp, cudaStream_t st) {
  adamw_kernel<false><<<kSqnormBlocks, 256, 0, st>>>(p, m, v, g, pb, n / 4, n_decay / 4, sc, hp, nullptr);
  return ok(1);
}

int adamw_with_norm(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, float* partial,
                    StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  adamw_kernel<true><<<kSqnormBlocks, 256, 0, st>>>(p, m, v, g, pb, n / 4, n_decay / 4, sc, hp, partial);
  sqnorm_final_kernel<<<1, 256, 0, st>>>(partial, kSqnormBlocks, sc, hp);
  return ok(2);
}

int adamw_range_with_norm(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, float* partial,
                          const StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  adamw_kernel<true><<<kSqnormBlocks, 256, 0, st>>>(p, m, v, g, pb, n / 4, n_decay / 4, sc, hp, partial);
  return ok(1);
}

int sqnorm_final(const float* partial, int count, StepScalars* sc, AdamHyper hp, cudaStream_t st) {
  sqnorm_final_kernel<<<1, 256, 0, st>>>(partial, count, sc, hp);
  return ok(1);
}

int init_normal(float* p, size_t n, uint64_t seed, int tensor_id, double stddev, int wgu_cols, int f, cudaStream_t st) {
  init_normal_kernel<<<grid_for(n, 256), 256, 0, st>>>(p, n, seed, (unsigned long long)tensor_id, stddev, wgu_cols, f);
  return ok(1);
}

int fill_f32(float* p, size_t n, float v, cudaStream_t st) {
  fill_kernel<<<grid_for(n, 256), 256, 0, st>>>(p, n, v);
  return ok(1);
}

int cast_bf16(const float* src, bf16* dst, size_t n, cudaStream_t st) {
  cast_bf16_kernel<<<grid_for(n, 256), 256, 0, st>>>(src, dst, n);
  return ok(1);
}

}  // namespace fs
