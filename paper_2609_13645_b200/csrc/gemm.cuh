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
  EPI_SWIGLU = 5,      // acc columns alternate 16 gate / 16 up: writes gate|up to gu bf16 [M, 2f] and a = R(silu(G) U) to C [M, f]
  EPI_SWIGLU_BWD = 6   // acc = d_a [M, f] (N = f = d_ffn): reads gate|up from gu [M, 2f] and writes bf16 d_gate, d_up to
                       // C [M, 2f] in the alternating 16 / 16 column layout; d_a = R(alpha acc) is never stored
};

// Weight-gradient GEMMs (EPI_F32 / EPI_F32_ACC) can hand the finished gradient straight to AdamW instead of storing it:
// the epilogue reads the master weight and both moments at the gradient's position, applies the update, and writes
// master, moments and the bf16 copy.  Only valid with gradient clipping off (the update then does not depend on the
// global norm); the squared norm is still summed, one partial per epilogue warp, into sq_slots.
struct AdamFuse {
  float* p = nullptr;   // fp32 master weights, same shape and row stride (ldc) as C
  float* m = nullptr;   // first moment
  float* v = nullptr;   // second moment
  bf16* pb = nullptr;   // bf16 copy of the weights
  const void* scalars = nullptr;  // device StepScalars (bias corrections of the current step)
  float lr = 0, beta1 = 0, beta2 = 0, eps = 0, wd = 0;
  float* sq_slots = nullptr;  // kAdamFuseSlots floats, zeroed by the caller; unused ones stay zero
};
constexpr int kAdamFuseSlots = 1280;

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
  float alpha = 1.0f;  // the accumulator is multiplied by alpha before the epilogue (not for EPI_ROPE / EPI_SWIGLU)
  // EPI_ROPE
  // fp32 tables TRANSPOSED, [head_dim/2][rope_ld] (entry (i, position) at i * rope_ld + position): the 32 rows a warp
  // holds are consecutive positions, so each load of one i is one 128-byte line
  const float* rope_cos = nullptr;
  const float* rope_sin = nullptr;
  int64_t rope_ld = 0;
  int seq = 1, head_dim = 64, rope_cols = 0;
  // EPI_ROPE with per-head QK-Norm (null qk_r: off): every rotated head is first RMS-normalised over its head_dim
  // accumulators and multiplied by a gain (heads below n_q_heads use gain_q, the others gain_k); r = (mean x^2 + eps)^(-1/2)
  // of every (row, head) is written to qk_r [M, rope_cols / head_dim] for the backward pass
  float* qk_r = nullptr;
  const bf16* qk_gain_q = nullptr;
  const bf16* qk_gain_k = nullptr;
  int n_q_heads = 0;
  float qk_eps = 0.f;
  // EPI_SWIGLU (written), EPI_SWIGLU_BWD (read)
  bf16* gu = nullptr;  // [M, 2f] gate | up
  int d_ffn = 0;
  int* err = nullptr;  // device status word
  // Optional device scratch that lets the CTA-pair kernel divide work along K (both deterministic):
  //  - split-K: weight gradients with few output tiles run up to 8 K parts concurrently, a second kernel adds them;
  //  - balanced-K: when the last wave of tiles would keep at most half of the pairs busy, its tiles are divided into K
  //    parts that run first, one per pair; the highest-numbered pair of a tile's group adds the others' fp32 partials.
  // The first 1 KiB holds arrival counters that must be zero at launch; the kernel leaves them zero.  With
  // scratch_reset the launcher clears them itself (one memset node) before a balanced-K launch.
  float* scratch = nullptr;
  size_t scratch_bytes = 0;
  bool scratch_reset = false;
  const AdamFuse* adam = nullptr;
  // Streaming cross-entropy on the logits GEMM (A, B both K-major, CTA-pair kernel; alpha = logit factor).  No logits
  // are stored.  ce_mode 1: every thread reduces its row's 256 accumulator columns to (max, sum of e^(z - max)) and
  // stores the pair at ce_part[row * ce_tiles + column tile]; the tile that holds the row's label column also stores that
  // logit to ce_zy[row].  ce_mode 2: C receives bf16 dz = (e^(z - ce_lse[row]) - [column == label]) * w, with
  // w = inv_count * ce_scale for rows whose label is counted (0 <= label < N) and 0 otherwise.
  int ce_mode = 0;
  float2* ce_part = nullptr;
  int ce_tiles = 0;             // column tiles of 256 per row = (N + 255) / 256
  float* ce_zy = nullptr;
  const float* ce_lse = nullptr;
  const int32_t* ce_labels = nullptr;
  const struct StepScalars* ce_scalars = nullptr;
  float ce_scale = 1.0f;
};

// Enqueues the contraction on `stream`.  Returns cudaErrorInvalidValue for shapes it does not take.  *launches (when
// given) receives the number of kernels the call enqueued (2 for a split-K contraction with its reduction, else 1).
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t stream, int* launches = nullptr);

// Two weight gradients (both operands mn-major, the same contraction length K, the same fp32 / AdamW epilogue kind) as
// ONE launch of the CTA-pair kernel: the tiles of `b` follow the tiles of `a` in the persistent schedule, so the last,
// partly filled wave of `a` and its exposed optimizer epilogue run beside the first tiles of `b`.  Every tile is computed
// exactly as a launch of its own would compute a whole tile; which tiles the balanced schedule divides along K depends on
// the combined tile count.  gemm_group2_ok says whether the pair qualifies (otherwise: two launch_gemm calls).
bool gemm_group2_ok(const GemmArgs& a, const GemmArgs& b);
cudaError_t launch_gemm_group2(const GemmArgs& a, const GemmArgs& b, cudaStream_t stream, int* launches = nullptr);

extern int g_gemm_group;
extern int g_gemm_tma_out;
extern int g_gemm_force_bn;
extern int g_gemm_pairs;
extern int g_gemm_balanced;
extern int g_gemm_swiglu_tma;

}  // namespace fs
