/* forgestep — C ABI of a single-GPU training step (forward, backward, AdamW) of a
 * Llama-style dense decoder for NVIDIA B200 (sm_100a).
 *
 * The operation is the one the ForgeTrain paper optimises: one microbatch through a
 * decoder-only transformer with grouped-query attention, SwiGLU feed-forward blocks,
 * pre-normalisation RMSNorm, RoPE and an untied output head (paper appendix "Model
 * Architectures"), in bf16 with fp32 master weights and fp32 weight gradients, followed
 * by the fused clip + Adam + bf16 write-back update (paper appendix on framework-level
 * optimisation, optimizer-tail listing).
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers, "host" pointers are ordinary host memory.
 *   - The caller owns every buffer it passes, including the workspace; the library owns
 *     only its small host-side handle and allocates no device memory.
 *   - All device work is enqueued on the stream given at ft_init_model.  A call that
 *     returns a value to the host synchronises that stream once, at its end.
 *   - Every function returns an ft_status; ft_last_error gives a message.  Nothing aborts
 *     the process and no kernel traps: device-side problems (a wait that ran out) set a
 *     status word that the next synchronising call reports as FT_ETIMEOUT.
 *   - Parameter tensors are addressed by index (ft_param_info gives name and shape) and
 *     always use the logical row-major [out, in] layout.  Order: "embed", then per layer
 *     "layers.{l}.norm1", ".wqkv" (rows: q heads, k heads, v heads), ".wo", ".norm2",
 *     ".wgu" (rows: gate 0..f-1, then up 0..f-1), ".wd"; then "norm_f", "lm_head".
 */
#ifndef FORGESTEP_H_
#define FORGESTEP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t max_batch, max_seq;     /* ft_train_step requires B <= max_batch, S <= max_seq */
  float rms_eps, rope_theta;
  float lr, beta1, beta2, adam_eps, weight_decay; /* decay applies to matrices, not to RMSNorm gains */
  float max_grad_norm;            /* <= 0: clipping off; else coeff = min(1, max/(norm + 1e-6)) */
  int32_t recompute;              /* 0: keep every layer's activations; 1: keep layer inputs, rerun the layer forward in backward */
  int32_t debug_taps;             /* 1: keep the backward intermediates of every layer for ft_get_tap (needs recompute = 0) */
  /* Variants of the paper's model families (appendix "Model Architectures": rows "Tied input/output embeddings" and
   * "muP (scale_emb, dim_model_base, scale_depth)").  A factor of 0 means 1, so a zero-filled tail is the plain decoder. */
  float emb_scale;                /* x_0 = R(emb_scale * E[token])                         (muP: scale_emb) */
  float resid_scale;              /* x <- R(x + resid_scale * branch), both branches       (muP: scale_depth / sqrt(n_layers)) */
  float logit_scale;              /* z = logit_scale * (h_F W^T)                            (muP: dim_model_base / d_model) */
  int32_t tie_embeddings;         /* 1: no lm_head parameter; the head reads the embedding table and both gradients add */
  int32_t qk_norm;                /* 1: per-head RMSNorm of q and k before the rotation (Qwen3 column of the same appendix);
                                     adds the gains layers.{l}.q_norm and layers.{l}.k_norm [head_dim], eps = rms_eps */
  int32_t mtp;                    /* 1: one-layer multi-token-prediction (Eagle) head (same appendix, row "MTP / Eagle head:
                                     On (1 layer)"; the FLOP appendix of the Ascend models counts it as one more backbone
                                     layer plus one more output head): h' = R(R(hn Wh^T) + en We^T) from the normalised last hidden
                                     state hn and the normalised embedding en of the NEXT token, one more decoder layer, its
                                     own final norm, the backbone's output head, trained on the token after next.
                                     Parameters mtp.norm_h, mtp.norm_e [h], mtp.proj_h, mtp.proj_e [h, h], mtp.layer.*
                                     (a layer's set), mtp.norm_f [h]. */
  float mtp_weight;               /* loss = backbone loss + mtp_weight * (mean cross-entropy of the MTP head); 0 means 1 */
  /* ZeRO-1 sharding of the optimizer state (Section "Sources of the Speedup": "ZeRO-1 optimizer sharding"; appendix
   * "Framework-Level Optimization Trajectory", step "ZeRO-1 sharded optimizer").  dp_world in {2, 4, 8, 16, 32}: the
   * workspace holds fp32 masters and both Adam moments only for this rank's slice of every gradient bucket (slice
   * dp_rank of dp_world equal parts, see ft_dp_bucket), i.e. 12 / dp_world bytes per parameter instead of 12; gradients
   * and the bf16 compute copy stay whole.  Such a model steps through the ft_dp_* calls only (ft_train_step and
   * ft_apply_update return FT_EINVAL); ft_dp_update_range takes ranges inside the rank's own slices; ft_get_param of a
   * master or moment returns the owned elements and 0 elsewhere (the ranks' results add up to the whole tensor),
   * ft_set_param stores the owned elements of the whole tensor it is given (and, for a master, rewrites the bf16 copy of
   * the whole tensor); both use the tensor's span of the gradient arena as staging, so gradients are lost.  Every rank
   * draws the same initial weights from the seed.  0 or 1: unsharded (the default). */
  int32_t dp_world, dp_rank;
} ft_config;

typedef struct ft_model ft_model;

typedef enum {
  FT_OK = 0, FT_EINVAL = 1, FT_ENOMEM = 2, FT_ECUDA = 3, FT_ENONFINITE = 4, FT_ETIMEOUT = 5, FT_ENOTFOUND = 6
} ft_status;

typedef enum { FT_MASTER_F32 = 0, FT_COMPUTE_BF16 = 1, FT_ADAM_M_F32 = 2, FT_ADAM_V_F32 = 3, FT_GRAD_F32 = 4 } ft_kind;

/* Bytes of device workspace a model of this config needs (0 if the config is invalid).  The workspace holds what the
 * paper's forged engine keeps resident for one data-parallel rank (Section "Sources of the Speedup"; appendix
 * "Why the Engine Is Faster, Mechanism by Mechanism"): fp32 masters, both Adam moments, fp32 gradients and the bf16
 * compute copy as five identically laid out flat arenas, every layer's saved activations (or, with recompute, one
 * layer's plus the layer inputs), the backward scratch and one chunk of logits.  Host-only call. */
size_t ft_workspace_bytes(const ft_config* cfg);

/* init_model(config, seed) of the problem statement: creates a model of the architecture tables (appendix "Model
 * Architectures") inside dev_workspace (256-byte aligned, >= ft_workspace_bytes) on the current CUDA device.  The
 * paper prints no initialiser; every matrix is drawn from N(0, 0.02^2) by a counter-based generator keyed by (seed,
 * tensor index, element index) (splitmix64 -> two 24-bit uniforms -> Box-Muller in double), gains are 1, Adam moments
 * 0, step 0, the bf16 copy is the rounded master.  cuda_stream is a cudaStream_t (NULL = default stream); the caller
 * keeps ownership of the workspace and must keep it alive until ft_destroy.  Returns FT_EINVAL for a bad config or a
 * misaligned workspace, FT_ENOMEM when bytes is too small (*out stays NULL), FT_ECUDA on a device that is not sm_100. */
ft_status ft_init_model(const ft_config* cfg, uint64_t seed, void* dev_workspace, size_t bytes,
                        void* cuda_stream, ft_model** out);

/* train_step(tokens, labels) -> loss: forward, loss, backward, global gradient norm, AdamW with fp32 masters and the
 * bf16 write-back (the train step of the forged engine: Section "Sources of the Speedup"; optimizer arithmetic from the fused clip + Adam +
 * cast listing and the device-side clip listing of the appendix "Why the Engine Is Faster, Mechanism by Mechanism").
 * dev_tokens, dev_labels: int32 [B, S] on the device; labels < 0 do not count in the mean loss.
 * host_loss / host_gnorm: optional host floats; if either is non-NULL the call synchronises the stream. */
ft_status ft_train_step(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S,
                        float* host_loss, float* host_gnorm);

/* Optimizer-tail fusion (Section "Sources of the Speedup", vertical integration: clip + Adam + cast as one pass;
 * taken one step further here): with gradient clipping off
 * (max_grad_norm <= 0) the update of a weight matrix does not depend on the global norm, so ft_train_step applies
 * AdamW inside the epilogue of the weight-gradient GEMM (or of its split-K reduction): the finished fp32 gradient
 * never goes to memory, and the separate optimizer pass shrinks to the embedding table and the gains.  The update
 * arithmetic is the same function, so parameters, moments and losses are bit-identical to the unfused step; the
 * reported gradient norm is summed in a different (still fixed) order.  On by default; off automatically when
 * clipping is on or debug_taps is set.  After a fusing ft_train_step, FT_GRAD_F32 of the matrices holds stale
 * values (use ft_forward_backward to materialise gradients).  Changing the setting drops a captured graph. */
ft_status ft_set_fused_update(ft_model* m, int32_t enable);

/* Position tables in the LongRoPE form (appendix "Model Architectures", MiniCPM4 rows): angle(p, i) = p * theta^(-2i/d) /
 * host_factors[i] for i < head_dim / 2 (NULL: all 1), and cos, sin multiplied by mscale (> 0).  Rebuilds both tables on the
 * host in double precision and copies them (synchronises the model's stream).  The factors are model data, like weights. */
ft_status ft_set_rope_scaling(ft_model* m, const float* host_factors, float mscale);

/* Weight-gradient overlap: nothing later in the backward pass depends on a layer's weight gradients (appendix
 * "Optimization Catalog": "Backward-pass fusion" and the auxiliary streams that carry wgrad, turned into concurrency), so the library enqueues those GEMMs on a second stream
 * of its own, ordered by events against the kernels that produce their inputs and against the kernels that later
 * overwrite the buffers they read; they occupy the SMs that the main chain leaves idle in the last wave of each
 * kernel.  Results do not change by a bit (every kernel keeps its own fixed summation order and its own scratch).
 * On by default; switched off internally while profiling or with debug_taps.  Changing it drops a captured graph. */
ft_status ft_set_overlap(ft_model* m, int32_t enable);

/* Stored-dS attention backward (see ft_k_attention_bwd_ws): when max_seq is a multiple of 128 and
 * 2 * max_batch * n_heads * max_seq^2 bytes is at most 24 GiB, the workspace holds one layer's dS^T and the step
 * uses that path for sequences that are multiples of 128; other sequences, and models over the limit, use the
 * recomputing dQ kernel.  On by default; 0 selects the recomputing kernel always.  Changing it drops a captured graph. */
ft_status ft_set_attention_stored_ds(ft_model* m, int32_t enable);

/* Streaming cross-entropy (the appendix' "chunked / streaming cross-entropy" that folds the LM-head GEMM, the loss and
 * the logit gradient into one chunked loop without ever holding logits): the logits GEMM of a row chunk reduces every
 * 256-column tile of a row to (max, sum of exponentials) in its epilogue, a small kernel combines the pairs into the
 * row's log-sum-exp and loss, and the same GEMM runs a second time with an epilogue that writes the bf16 logit
 * gradient directly.  Neither fp32 logits nor a separate cross-entropy pass exist; the price is the second GEMM.  Off
 * by default, as in the paper (slower than the chunked path at the measured shapes).  Results agree with the default
 * path to rounding (the sums are formed per tile, then combined).  Changing it drops a captured graph. */
ft_status ft_set_streaming_ce(ft_model* m, int32_t enable);

/* SwiGLU backward inside the down projection's data-gradient contraction (the appendix' fused elementwise work around
 * the SwiGLU block, applied to the backward pass): the gradient d_a of a = silu(G) U is rounded to bf16 in the
 * epilogue, which reads G and U of the same positions and writes d_G = d_a U s (1 + G (1 - s)) and d_U = d_a G s,
 * s = sigmoid(G); d_a itself is never stored and the separate elementwise pass does not run.  Bit-identical to the
 * unfused path (same arithmetic on the same rounded d_a).  On by default; not used with debug_taps (the tap d_a needs
 * the stored tensor).  Changing it drops a captured graph. */
ft_status ft_set_fused_swiglu_bwd(ft_model* m, int32_t enable);

/* Whole-step CUDA graph (the paper's full-step graph capture): when enabled, the first ft_train_step of a (B, S)
 * runs launch by launch, the second is captured into a graph, later ones replay it (ids are first copied into the
 * model's own buffers).  Needs a capturable stream (not the legacy default stream; otherwise it switches itself
 * off); not used while profiling or with debug_taps.  ft_graph_replays counts the replays so far. */
ft_status ft_set_graph(ft_model* m, int32_t enable);
int64_t ft_graph_replays(const ft_model* m);

/* Same call with HOST token and label arrays: copies them to the device, runs the step, returns the loss. */
ft_status ft_train_step_host(ft_model* m, const int32_t* host_tokens, const int32_t* host_labels, int32_t B,
                             int32_t S, float* host_loss, float* host_gnorm);

/* ---- Data-parallel hooks (Section "Sources of the Speedup" and appendix "Framework-Level Optimization Trajectory":
 * "bucketed reduce-scatter overlapped with backward", "ZeRO-1 sharded optimizer,
 * per-bucket all-gather interleaved with Adam").  The library itself holds no communicator: these calls expose what a
 * data-parallel driver needs, and paper_2609_13645_b200/dp.py drives them with torch.distributed (NCCL).
 *
 * The flat fp32 gradient arena (and the identically laid out master / moment / bf16 arenas, ft_arena_ptr) is cut into
 * buckets in the order in which the backward pass completes them: the untied LM head first, then the layers from the
 * last to the first (each layer's four matrices, contiguous), then the embedding table, then all gains; with the MTP
 * head its six matrices form a bucket between the output head and the last layer.  Every bucket
 * starts on a multiple of 128 elements and has a multiple of 128 elements, so it divides evenly over 2, 4, ... 128
 * ranks.
 *   ft_dp_num_buckets / ft_dp_bucket   number of buckets; arena offset and element count of bucket i.
 *   ft_arena_ptr                       device address and element count of an arena (FT_GRAD_F32, FT_COMPUTE_BF16, ...).
 *   ft_dp_set_label_count              number of labels >= 0 over ALL ranks' batches of the next step: the loss mean and
 *                                      the logit gradients divide by it, so that the SUM of the ranks' gradients is the
 *                                      gradient of the global mean loss (0: this batch's own count, the default).
 *   ft_dp_set_label_count_device       the same number as a device int64 that the step reads when it runs (NULL: off), so
 *                                      that the ranks' counts can be summed on the device with no host round trip; it
 *                                      takes precedence over ft_dp_set_label_count while set.  With the MTP head the
 *                                      pointer addresses TWO int64: the labels' count and the count of the labels
 *                                      shifted by one (labels[:, 1:] >= 0) over all ranks.
 *   ft_dp_backward                     enqueues forward + backward of this rank's batch on the model's stream (gradients
 *                                      materialised, weight gradients in stream order), recording one event per bucket;
 *                                      returns without waiting.
 *   ft_dp_stream_wait_bucket           makes `stream` wait (device side) for bucket i of the last ft_dp_backward.
 *   ft_dp_sqnorm                       *dev_out = sum of squares of the gradient range, fixed summation order, on `stream`.
 *   ft_dp_begin_update                 advances the step counter and bias corrections; with dev_sq_total (the sum of
 *                                      squares over all ranks' shards) it also sets the norm and the clip coefficient,
 *                                      with NULL the coefficient is 1 (only valid when clipping is off).  Once per step,
 *                                      on `stream`, before the first ft_dp_update_range.
 *   ft_dp_update_range                 AdamW (master, moments, bf16 copy) on arena range [offset, offset + count) from
 *                                      the gradient values found there (the reduced shard), on `stream`.
 *   ft_dp_set_norm                     records the norm for reporting when clipping is off (after the update).
 *   ft_dp_collect                      waits for the model's stream; returns this rank's loss share (sum of its label
 *                                      losses / total label count) and the recorded norm, and any device-side status.
 *   ft_dp_scratch                      4 floats of device memory for the driver's scalar reductions.
 * offset and count are multiples of 4.  `stream` may be the model's stream or another one; the driver orders it. */
int32_t ft_dp_num_buckets(ft_model* m);
ft_status ft_dp_bucket(ft_model* m, int32_t i, int64_t* offset, int64_t* count);
ft_status ft_arena_ptr(ft_model* m, ft_kind kind, void** dev_ptr, int64_t* numel);
ft_status ft_dp_scratch(ft_model* m, float** dev_ptr);
ft_status ft_dp_set_label_count(ft_model* m, int64_t total_count);
ft_status ft_dp_set_label_count_device(ft_model* m, const int64_t* dev_total_count);
ft_status ft_dp_backward(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S);
ft_status ft_dp_stream_wait_bucket(ft_model* m, int32_t i, void* stream);
ft_status ft_dp_sqnorm(ft_model* m, int64_t offset, int64_t count, float* dev_out, void* stream);
ft_status ft_dp_begin_update(ft_model* m, const float* dev_sq_total, void* stream);
ft_status ft_dp_update_range(ft_model* m, int64_t offset, int64_t count, void* stream);
ft_status ft_dp_set_norm(ft_model* m, const float* dev_sq_total, void* stream);
ft_status ft_dp_collect(ft_model* m, float* host_loss, float* host_gnorm);

/* Pipelined form of ft_train_step_host for training loops that do not need a step's loss before enqueueing the next
 * step (the paper's rule of keeping host synchronisation out of the hot loop, Section "Sources of the Speedup" (deep customization) / appendix "Optimization
 * Catalog": device-side norm and clipping, no .item() in the step).  ft_submit_step_host enqueues, on the model's
 * stream, the copies of this step's ids, the whole step and a copy of its scalars into a pinned slot owned by the
 * library, and returns without waiting; ft_collect_step waits for the OLDEST submitted step that has not been
 * collected and returns its loss, gradient norm and status.  At most FT_MAX_IN_FLIGHT steps may be outstanding (one
 * more submit returns FT_EINVAL and enqueues nothing); ft_collect_step with nothing outstanding returns FT_ENOTFOUND.
 * host_tokens / host_labels must stay unchanged until that step has been collected; they should be pinned memory
 * (pageable memory works but makes the copy, and so the call, wait for the stream).  Results are bit-identical to
 * ft_train_step_host on the same inputs.  Do not interleave with other step calls while steps are outstanding. */
#define FT_MAX_IN_FLIGHT 2
ft_status ft_submit_step_host(ft_model* m, const int32_t* host_tokens, const int32_t* host_labels, int32_t B, int32_t S);
ft_status ft_collect_step(ft_model* m, float* host_loss, float* host_gnorm);

/* Forward and loss only; no gradients, no update: the per-step loss that the long-run validation of Section "Correctness: The Equivalence Chain and
 * Long-Run Validation" and Section "Training-Trajectory Agreement" compare between engine and reference, available without touching the state.
 * Synchronises the stream; *host_loss is the mean cross-entropy over labels in [0, vocab). */
ft_status ft_forward_loss(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S,
                          float* host_loss);

/* Forward and backward without the update: leaves every fp32 gradient readable through FT_GRAD_F32, which is how the
 * gradient anchors of Section "Correctness: The Equivalence Chain and Long-Run Validation" ("Bit-for-Bit: zero-tolerance adjudication": activations, gradients, optimizer states
 * at per-operator granularity) are read from this engine.  Synchronises the stream. */
ft_status ft_forward_backward(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B,
                              int32_t S, float* host_loss);

/* Gradient norm + clip coefficient + AdamW on whatever the FT_GRAD_F32 buffers hold: the optimizer tail of the appendix
 * listing in isolation (g <- g * clip; m, v updated; update = m_hat / (sqrt(v_hat) + eps) + wd * p; p <- p - lr * update;
 * bf16 copy rewritten), so that the optimizer-state anchors can be checked apart from the gradients.  Synchronises. */
ft_status ft_apply_update(ft_model* m, float* host_gnorm);

/* get / set parameters of the problem statement, extended to the whole training state so that a run can be saved and
 * resumed: Section "Correctness: The Equivalence Chain and Long-Run Validation" lists "checkpoint save-and-restore" and "the first step after resumption" among the edge cases
 * an engine must reproduce exactly; masters, both moments and the step counter are that state (the bf16 copy is derived).
 * ft_num_params / ft_param_info: number of tensors; name (owned by the model, valid until ft_destroy), ndim (1 for a
 * gain vector, 2 for a matrix) and shape of tensor i.
 * ft_get_param / ft_set_param: copy one tensor to / from HOST memory in the logical row-major [out, in] layout, whatever
 * the device layout; bytes must equal the tensor's size in that kind (FT_EINVAL otherwise).  Setting FT_MASTER_F32 also
 * rewrites the bf16 compute copy with the rounded master.  Both synchronise the model's stream.
 * ft_get_step / ft_set_step: the optimizer step counter t (the bias corrections 1 - beta^t of the next update follow
 * from it); restoring masters, moments and t makes the next step bit-identical to the uninterrupted run. */
int32_t ft_num_params(const ft_model* m);
ft_status ft_param_info(const ft_model* m, int32_t i, const char** name, int32_t* ndim, int64_t shape[2]);
ft_status ft_get_param(ft_model* m, int32_t i, ft_kind kind, void* host_dst, size_t bytes);
ft_status ft_set_param(ft_model* m, int32_t i, ft_kind kind, const void* host_src, size_t bytes);
ft_status ft_get_step(const ft_model* m, int64_t* step);
ft_status ft_set_step(ft_model* m, int64_t step);

/* Named intermediate of the last step, copied to the host: this engine's form of the per-operator anchors of Section
 * "Correctness: The Equivalence Chain and Long-Run Validation" ("taken at per-operator granularity, at exact numerical values"): every tensor a kernel hands to the next one can
 * be read back and compared with a reference.  Forward taps of layer l: "x_in", "h1", "qkv"
 * ([T, h_q+2h_kv], q and k already rotated), "attn_lse" (fp32 [B, n_h, S]), "o", "x_mid", "h2", "gu"
 * ([T, 2f]: gate then up), "a", "x_out"; layer -1: "hF", "ce_lse" (fp32 [T]).  Backward taps (debug_taps = 1):
 * "d_x_out", "d_a", "d_gu", "d_h2", "d_x_mid", "d_o", "d_qkv", "d_h1", "d_x_in"; layer -1: "d_hF".
 * *dtype: 0 = bf16, 1 = fp32.  bytes is the capacity of host_dst; *out_bytes the size written. */
ft_status ft_get_tap(ft_model* m, const char* name, int32_t layer, void* host_dst, size_t bytes,
                     size_t* out_bytes, int32_t* dtype);

/* Per-class kernel timing with CUDA events recorded on the model's stream around every launch.  While enabled
 * the step still never synchronises; ft_get_profile synchronises and returns, for one class, the summed device
 * time (ms), the summed algorithmic work (FLOPs for FT_PROF_GEMM and the attention classes, bytes otherwise) and
 * the number of kernels.  Enabling resets the totals. */
typedef enum {
  FT_PROF_GEMM = 0, FT_PROF_ATTN_FWD = 1, FT_PROF_ATTN_BWD = 2, FT_PROF_NORM = 3, FT_PROF_ELEMENTWISE = 4,
  FT_PROF_CE = 5, FT_PROF_OPTIMIZER = 6, FT_PROF_CLASSES = 7
} ft_prof_class;
ft_status ft_set_profiling(ft_model* m, int32_t enable);
ft_status ft_get_profile(ft_model* m, int32_t cls, double* ms, double* work, int64_t* launches);
/* The GEMM class broken down by (M, N, K, a_mn, b_mn, epilogue): entry i of the table built while profiling was on;
 * FT_ENOTFOUND past the end.  shape = {M, N, K, a_mn, b_mn, epilogue kind, M2, N2}: M2 x N2 is the second output of a
 * launch that computed two weight gradients over the same K at once (0, 0 otherwise); its work is 2 K (M N + M2 N2). */
ft_status ft_get_gemm_profile(ft_model* m, int32_t i, int32_t shape[8], double* ms, int64_t* launches);

/* Message of the last call on this model that returned a non-zero status (owned by the model; "null model" for NULL).
 * Error behaviour of the whole boundary: nothing aborts, traps or throws; a device-side wait that ran out, a token id or
 * label outside [0, vocab) and a non-finite loss are recorded in device memory and reported by the next synchronising
 * call as FT_ETIMEOUT, FT_EINVAL and FT_ENONFINITE (the paper's engines keep such checks on the device and out of the
 * hot loop: appendix "Optimization Catalog", device-side norm and clipping). */
const char* ft_last_error(const ft_model* m);
/* Number of kernels the library launched since the model was created (launch accounting for the paper's
 * launch-overhead items: whole-step graph capture and programmatic dependent launch, appendix "Optimization Catalog"). */
int64_t ft_launch_count(const ft_model* m);
/* Destroys the host-side handle, the library's second stream, its events and a captured graph.  The workspace stays
 * the caller's.  The caller must have synchronised the stream (or not care about work in flight). */
void ft_destroy(ft_model* m);

/* ---- single kernels, for unit parity tests and kernel timing (device pointers; stream = cudaStream_t): the operator
 * layer of the paper's two-layer engine (Section "Overview: The Agent Loop and the Golden Reference"; kernel table of Section "Operator-Level Forging").  All
 * buffers are the caller's; the calls enqueue on `stream` and return without waiting. ---- */

/* C[M,N] = sum_k A[m,k] B[n,k] on the tcgen05 tensor cores, fp32 accumulation (the projection, FFN and
 * head contractions of the paper's FLOP table, forward / data-gradient / weight-gradient forms).
 * a_mn = 0: A stored row-major [M, lda>=K];  a_mn = 1: A stored row-major [K, lda>=M] (contraction over rows).
 * b_mn likewise for B ([N, ldb>=K] or [K, ldb>=N]).  out_kind: 0 bf16 store, 1 bf16 store of (resid + acc)
 * with resid bf16 [M, ldc], 2 fp32 store, 3 fp32 accumulate into C.  M, N, K, lda, ldb, ldc multiples of 8. */
ft_status ft_k_gemm(const void* dev_A, int32_t a_mn, int64_t lda, const void* dev_B, int32_t b_mn, int64_t ldb,
                    void* dev_C, int64_t ldc, const void* dev_resid, int32_t out_kind,
                    int32_t M, int32_t N, int32_t K, int32_t* dev_err, void* stream);

/* ft_k_gemm with a device scratch buffer that lets the kernel divide work along K (appendix "Model-FLOPs Utilization": a weight gradient
 * contracts over the token dimension, the long one).  Results stay bit-identical from run to run:
 *  - weight-gradient layout (a_mn = b_mn = 1, fp32 output) with few 256 x 256 output tiles: up to 8 K parts run
 *    concurrently into fp32 partial outputs and a second kernel adds them in index order;
 *  - any layout with a contraction of at least 2560 (40 blocks of 64; below that the division costs more than it saves)
 *    whose last wave of 256 x 256 tiles would keep at most half of the SM pairs busy: the tiles of that wave
 *    are divided into 2 to 8 K parts that run first, one part per pair; all parts but the last leave an fp32 partial
 *    tile in the scratch, and the pair holding the last part (the highest-numbered pair of the group, so that it only
 *    ever waits for pairs that were started before it) adds them in pair order before the usual epilogue.  The other
 *    tiles then run whole, round-robin.
 * dev_scratch: caller-owned device memory, 16-byte aligned, scratch_bytes long; its contents on entry do not matter
 * (the call clears the 1 KiB of counters at its start with a stream-ordered memset) and are unspecified afterwards.
 * 20 MiB covers every case; with less the call degrades to the plain schedule of ft_k_gemm.  Two calls that share a
 * scratch buffer must not overlap on the GPU. */
ft_status ft_k_gemm_ws(const void* dev_A, int32_t a_mn, int64_t lda, const void* dev_B, int32_t b_mn, int64_t ldb,
                       void* dev_C, int64_t ldc, const void* dev_resid, int32_t out_kind,
                       int32_t M, int32_t N, int32_t K, float* dev_scratch, uint64_t scratch_bytes,
                       int32_t* dev_err, void* stream);

/* The single-kernel attention calls below keep their device status word inside the library (ft_k_gemm takes the
 * caller's dev_err instead).  ft_k_status waits for `stream`, then returns FT_ETIMEOUT if a bounded device-side wait ran
 * out in any ft_k_attention_* call on the current device since the last ft_k_status (and clears the word), else FT_OK.
 * (Keeping host synchronisation out of the hot loop, Section "Sources of the Speedup", is why the calls themselves do not check.) */
ft_status ft_k_status(void* stream);

/* Causal attention core forward on a packed qkv buffer bf16 [B*S, (n_h + 2 n_kv) * d] (q heads, k heads,
 * v heads; q, k already rotated): o bf16 [B*S, n_h*d], lse fp32 [B, n_h, S] (natural log). d in {64, 128}. */
ft_status ft_k_attention_fwd(const void* dev_qkv, void* dev_o, float* dev_lse, int32_t B, int32_t S,
                             int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream);

/* Backward of the same: d_qkv bf16 [B*S, (n_h + 2 n_kv) * d] (d_q, d_k NOT rotated back when
 * dev_cos/dev_sin are NULL; with fp32 tables [S, d/2] they are rotated by the negative angle before the
 * single rounding).  dev_delta: fp32 scratch [B, n_h, S]. */
ft_status ft_k_attention_bwd(const void* dev_qkv, const void* dev_o, const void* dev_do, const float* dev_lse,
                             float* dev_delta, void* dev_dqkv, const float* dev_cos, const float* dev_sin,
                             int32_t B, int32_t S, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim,
                             void* stream);

/* The same backward with a second scratch array, dev_ds: B * n_h * S * S bf16 in a chunked order private to the
 * library (ds_bytes >= 2 B n_h S^2, 128-byte aligned, caller-owned device memory; contents on entry do not matter,
 * unspecified afterwards).  The dK/dV kernel
 * writes the rounded dS of the attention backward of appendix "Anatomy of a Forged Kernel" (dS = P o (dP - delta)) there, transposed, and dQ = dS K / sqrt(d)
 * is then one causally truncated batched contraction over the stored tiles: five tile products per (query block, key
 * block) pair instead of seven, the same dS bits feeding dK and dQ.  Needs S % 128 == 0; with dev_ds NULL, ds_bytes too
 * small, a misaligned dev_ds or any other S the call is ft_k_attention_bwd.  Results are deterministic; they agree with
 * ft_k_attention_bwd to rounding, not bit for bit. */
ft_status ft_k_attention_bwd_ws(const void* dev_qkv, const void* dev_o, const void* dev_do, const float* dev_lse,
                                float* dev_delta, void* dev_dqkv, const float* dev_cos, const float* dev_sin,
                                void* dev_ds, uint64_t ds_bytes, int32_t B, int32_t S, int32_t n_heads,
                                int32_t n_kv_heads, int32_t head_dim, void* stream);

/* The same backward for callers that cannot hand over scratch memory they allocated: code running where device
 * allocation is off limits (inside a framework's allocator callback, in a plugin that is given only its input and
 * output tensors, under a memory budget that is already fully committed) has nowhere to get the fp32 "delta"
 * buffer that ft_k_attention_bwd needs.  Here that buffer is a fixed 4 MiB array inside the library image, so the
 * call allocates nothing, on the device or through any library.  (The paper has no counterpart of this call.)
 *   - Limit: B * n_heads * S <= 1,048,576; larger problems return FT_ENOMEM and launch nothing.
 *   - Every GPU that loads the library keeps the 4 MiB until the process exits.
 *   - The first call on each device looks up the array's device address (once, with that device current); make
 *     that first call before starting any stream capture.
 *   - All calls share the one array and it keeps the last call's contents; the pre-pass of each call rewrites
 *     every element it later reads, so no clearing is needed, but two calls whose kernels overlap on the GPU
 *     (different streams, or different threads) race on it: run them one after the other.
 * Inputs, outputs and results are those of ft_k_attention_bwd (same kernels, same bits). */
ft_status ft_k_attention_bwd_noalloc(const void* dev_qkv, const void* dev_o, const void* dev_do, const float* dev_lse,
                                     void* dev_dqkv, const float* dev_cos, const float* dev_sin, int32_t B,
                                     int32_t S, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FORGESTEP_H_ */
