// Host-side interface of the bandwidth-bound kernels: embedding, RMSNorm, SwiGLU backward, cross-entropy,
// deterministic embedding backward, gradient norm, AdamW, initialisation.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace fs {

// Device-resident per-step scalars (nothing here is read by the host inside a step).
struct StepScalars {
  long long step;     // optimizer step counter t
  float bc1, bc2;     // 1 - beta1^t, 1 - beta2^t
  float clip;         // gradient clip coefficient
  float gnorm;        // global gradient norm of the last step
  float loss;         // mean loss of the last step
  float inv_count;    // 1 / number of counted labels
  int count;          // number of labels in [0, vocab)
  int nonfinite;      // 1 if the last loss was not finite
  int err;            // device status word (ERR_*)
  int pad[5];
};

struct AdamHyper {
  float lr, beta1, beta2, eps, wd, max_grad_norm;
};

int elementwise_blocks_for_norm(int T);            // grid of rmsnorm_bwd (also rows of its partial buffer)
constexpr int kSqnormBlocks = 1184;               // partial sums of the gradient norm
size_t sort_pad(size_t n);                         // padded key count of the embedding-backward sort

// each returns the number of kernels it launched, or a negative value after a CUDA launch error
int embed_fwd(const int32_t* tok, const bf16* E, bf16* x, int T, int h, int vocab, float scale, cudaStream_t st);
int rmsnorm_fwd(const bf16* x, const bf16* g, bf16* y, float* r, int T, int h, float eps, cudaStream_t st);
// dx = R(resid + rmsnorm_bwd(dy)) (resid may be null).  The gain gradient is left as one partial row per block in
// `partial` ([elementwise_blocks_for_norm(T)][h] floats, this norm's own slot); colsum_many adds the rows of every slot in
// block order (fp32, fixed order) into the gradient tensors, once, after the backward pass.
int rmsnorm_bwd(const bf16* dy, const bf16* x, const float* r, const bf16* g, const bf16* resid, bf16* dx,
                float* partial, int T, int h, cudaStream_t st);
// out[y][c] = sum over blocks b < elementwise_blocks_for_norm(T) of partial[y * slot_floats + b * h + c] for every slot
// y < nslots; out is a DEVICE array of nslots device pointers.  T as in the rmsnorm_bwd calls that filled the slots.
int colsum_many(const float* partial, float* const* out, int nslots, size_t slot_floats, int T, int h, cudaStream_t st);
// d_gu (physical 16/16 interleave of gate and up columns) from d_a and the saved gate|up activations.
// Per-head QK-Norm backward, in place on dqkv's query and key heads (see the kernel); dgain_q, dgain_k [d] fp32 are
// overwritten; partial: scratch of partial_floats floats (one row of 2 d per block; more room, more blocks, up to 1184).
int qknorm_bwd(bf16* dqkv, const bf16* qkv, const float* r, const bf16* gain_q, const bf16* gain_k, const float* cosT,
               const float* sinT, float* dgain_q, float* dgain_k, float* partial, size_t partial_floats, float inv_mscale2,
               int T, int S, int nh, int nkv, int d, cudaStream_t st);
int swiglu_bwd(const bf16* d_a, const bf16* gu, bf16* d_gu, int T, int f, cudaStream_t st);
// denom_override > 0: the loss mean (and the logit gradient) divide by it instead of by this batch's own label count
// (denom_dev != null: the same number read from device memory when the kernel runs)
// Counted labels are those with 0 <= label < vocab (the predicate of the loss kernels).  tok (may be null) and labels are
// also range-checked: a label >= vocab or an id outside [0, vocab) sets *err to ERR_BAD_INDEX.
int count_labels(const int32_t* labels, const int32_t* tok, int T, int vocab, StepScalars* sc, int* err,
                 long long denom_override, const long long* denom_dev, cudaStream_t st);
// per row: lse, loss contribution, and (if dz != null) dz = R((softmax(z) - onehot) * inv_count), zero for ignored rows
// dz = R(dz_scale * (softmax(z) - onehot) / counted labels)
int cross_entropy_rows(const float* z, const int32_t* labels, float* lse, float* loss_row, bf16* dz, int rows, int V,
                       const StepScalars* sc, float dz_scale, cudaStream_t st);
// streaming cross-entropy: per-tile (max, sum) pairs [rows, tiles] + the label logits -> lse and loss per row
int ce_combine(const float2* part, int tiles, const float* zy, const int32_t* labels, float* lse, float* loss_row, int rows,
               int V, cudaStream_t st);
// MTP head: ids and labels shifted by one inside every sequence of length S; loss <- loss + weight * sc2->loss
int mtp_shift(const int32_t* tok, const int32_t* lab, int32_t* tok2, int32_t* lab2, int T, int S, cudaStream_t st);
int add_loss(StepScalars* sc, const StepScalars* sc2, float weight, cudaStream_t st);
int reduce_loss(const float* loss_row, int T, StepScalars* sc, cudaStream_t st);
// dE[v,:] (+)= scale * sum over positions with token v (fp32, position order); keys: scratch of sort_pad(T) uint64.
// accumulate: dE already holds another gradient of the same table (tied output head) and is not cleared first.
int embed_bwd(const int32_t* tok, const bf16* dx, float* dE, unsigned long long* keys, int T, int h, int vocab,
              float scale, bool accumulate, cudaStream_t st);
int grad_norm_and_clip(const float* g, size_t n, float* partial, StepScalars* sc, AdamHyper hp, cudaStream_t st);
int advance_step(StepScalars* sc, AdamHyper hp, cudaStream_t st);
// *out = sum of squares of g[0, n) (n a multiple of 4), fixed order; partial: kSqnormBlocks floats of scratch
int sqnorm_to(const float* g, size_t n, float* partial, float* out, cudaStream_t st);
// gradient norm and clip coefficient in sc from a sum of squares formed elsewhere
int clip_from_sq(const float* sq_total, StepScalars* sc, AdamHyper hp, cudaStream_t st);
// fused clip + Adam + decoupled decay + bf16 write-back over a flat arena; elements >= n_decay get no decay
int adamw(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, const StepScalars* sc,
          AdamHyper hp, cudaStream_t st);
// clipping off: the same pass also sums the squared gradient norm (reported, not used by the update)
int adamw_with_norm(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, float* partial,
                    StepScalars* sc, AdamHyper hp, cudaStream_t st);
// AdamW over one range of the arenas (clipping off), writing kSqnormBlocks partial sums of g^2 to `partial` and leaving
// the final sum to sqnorm_final, which adds `count` partials in index order and stores the norm in sc.
int adamw_range_with_norm(float* p, float* m, float* v, const float* g, bf16* pb, size_t n, size_t n_decay, float* partial,
                          const StepScalars* sc, AdamHyper hp, cudaStream_t st);
int sqnorm_final(const float* partial, int count, StepScalars* sc, AdamHyper hp, cudaStream_t st);
// wgu_cols > 0: p is the gate|up matrix [2f, wgu_cols] in its interleaved row layout (draws keyed by the logical element)
int init_normal(float* p, size_t n, uint64_t seed, int tensor_id, double std, int wgu_cols, int f, cudaStream_t st);
int fill_f32(float* p, size_t n, float v, cudaStream_t st);
int cast_bf16(const float* src, bf16* dst, size_t n, cudaStream_t st);

}  // namespace fs
