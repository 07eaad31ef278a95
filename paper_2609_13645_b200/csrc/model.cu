// The train-step schedule and the C ABI.  A model is a carve-up of the caller's workspace plus a fixed launch
// order: there is no autograd graph and no host synchronisation inside a step; optimizer scalars live in device
// memory and are advanced by a kernel.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <string>
#include <vector>

#include "../../include/forgestep.h"
#include "forgestep_debug.h"
#include "attention.cuh"
#include "elementwise.cuh"
#include "gemm.cuh"

using namespace fs;

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kAttnDsMaxBytes = 24ull << 30;  // largest dS^T scratch the workspace will carry
// The logit gradient dz of ALL rows is kept (bf16 [T, V]) when it fits in this many bytes: the output head's data and
// weight gradients are then one contraction each over all rows; above it they are formed chunk by chunk, the weight
// gradient accumulating in fp32 memory.  (A variable so that a test can force the chunked form: ft_debug_head_dz_limit.)
size_t g_head_dz_limit = 4ull << 30;
constexpr size_t kSplitKFloats = 6u << 20;  // 24 MiB of split-K partial tiles (74 tiles of 256 x 256 fp32 at most)
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct ParamInfo {
  std::string name;
  int64_t rows, cols;  // cols == 0 for a gain vector of `rows` elements
  size_t offset;       // element offset in every arena
  bool is_wgu;
  size_t numel() const { return (size_t)rows * (size_t)(cols ? cols : 1); }
};

struct Carver {
  uint8_t* base = nullptr;
  size_t off = 0;
  template <typename T>
  T* take(size_t n) {
    off = align_up(off, kAlign);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

struct LayerActs {
  bf16 *h1, *qkv, *o, *x_mid, *h2, *gu, *a;
  float *lse, *r1, *r2;
  float* qk_r;  // per-head QK-Norm: r of every (token, query or key head); null when the variant is off
};

struct LayerTaps {  // debug copies of one layer's backward intermediates
  bf16 *d_x_out, *d_a, *d_gu, *d_h2, *d_x_mid, *d_o, *d_qkv, *d_h1, *d_x_in;
};

}  // namespace

struct ft_model {
  ft_config cfg;
  cudaStream_t stream = nullptr;
  std::string err;
  int64_t launches = 0;
  int h, hq, hkv, nqkv, f, V, L, d, maxT;
  int n_slots;
  int ce_chunk;
  int dz_rows;  // rows of the dz buffer: maxT (gradients of the head in one pass) or ce_chunk (chunk by chunk)

  std::vector<ParamInfo> params;
  size_t arena = 0, n_decay = 0;
  // ZeRO-1 state shard (cfg.dp_world > 1): master and both moments hold only this rank's slice of every gradient bucket,
  // arena / dp_world elements each, bucket after bucket in arena order; gradients and the bf16 copy stay full size
  int dp_world = 1, dp_rank = 0;
  size_t state_elems = 0;  // elements of master / adam_m / adam_v
  bool sharded() const { return dp_world > 1; }
  float *master, *adam_m, *adam_v, *grad;
  bf16* pbf;
  float *rope_cos, *rope_sin;    // [max_seq][d/2]: attention backward, QK-Norm backward
  float *rope_cosT, *rope_sinT;  // the same transposed, [d/2][max_seq]: the QKV GEMM's epilogue
  float rope_mscale = 1.0f;  // magnitude factor folded into both tables (LongRoPE form)
  StepScalars* sc;
  int32_t *tok_dev, *lab_dev;
  std::vector<bf16*> x;  // x[l] = input of layer l, x[L] = output of the last layer
  std::vector<LayerActs> acts;
  std::vector<LayerTaps> taps;
  float *rF, *ce_lse, *loss_row;
  bf16 *hF, *d_hF;
  bf16 *dxA, *dxB, *d_h, *d_a, *d_gu, *d_o, *d_qkv;
  float *delta, *norm_partial, *sq_partial, *z, *splitk;
  // gain gradients of the RMSNorms: every norm's backward leaves block partials in its own slot of norm_partial, and one
  // kernel after the backward pass sums all slots into the gradient tensors (norm_out: device array of their addresses)
  std::vector<int> norm_slot_of;  // parameter index -> slot, -1 for everything that is not a [d_model] gain
  int n_norm_slots = 0;
  float** norm_out = nullptr;
  float* qk_partial = nullptr;    // scratch of the per-head QK-Norm backward (one more slot)
  bf16* dz;
  unsigned long long* keys;
  int lastB = 0, lastS = 0;
  bool have_bwd = false;

  // Weight-gradient GEMMs on a second stream: nothing later in the backward pass depends on them, so they fill the SMs
  // that the main chain's kernels leave idle in their last wave.  ev_d orders a weight gradient after the data
  // gradient of the same layer (which still reads the bf16 weights the fused update overwrites); ev_w[k] lets the main
  // stream wait before it overwrites a buffer the k-th weight gradient of the previous layer still reads.
  bool overlap = true;        // policy switch (ft_set_overlap)
  cudaStream_t side = nullptr;
  cudaEvent_t ev_d = nullptr;
  cudaEvent_t ev_w[4] = {nullptr, nullptr, nullptr, nullptr};
  bool w_pending[4] = {false, false, false, false};
  bool overlapping = false;   // true while a backward pass that uses the second stream is being enqueued
  float* splitk2 = nullptr;   // GEMM scratch of the second stream
  // pipelined host entry: pinned result slots and one event per slot, oldest-first
  StepScalars* ring = nullptr;
  cudaEvent_t ring_ev[FT_MAX_IN_FLIGHT] = {};
  unsigned ring_head = 0, ring_tail = 0;  // submitted, collected (monotonic counters)
  // data-parallel hooks: gradient buckets of the flat arena in the order the backward pass completes them, one event
  // per bucket recorded on the model's stream, and the label count of all ranks for the loss mean
  struct DpBucket { size_t offset, count; };
  std::vector<DpBucket> dp_buckets;
  std::vector<cudaEvent_t> dp_ev;
  bool dp_mode = false;
  long long label_count_override = 0;
  const long long* label_count_dev = nullptr;  // the same, read from device memory at run time (no host round trip)
  float* dp_sq = nullptr;     // 4 floats of device scratch for the callers' norm reduction
  // one-layer MTP head: its layer's activations, inputs, shifted ids and its own loss scalars
  LayerActs acts_mtp{};
  bf16 *mtp_hn = nullptr, *mtp_xe = nullptr, *mtp_en = nullptr, *mtp_u1 = nullptr, *mtp_hF = nullptr, *mtp_d_hF = nullptr,
       *mtp_d_en = nullptr, *mtp_d_hn = nullptr, *mtp_d_xe = nullptr, *mtp_d_xL = nullptr;
  float *mtp_rh = nullptr, *mtp_re = nullptr, *mtp_rF = nullptr, *mtp_lse = nullptr;
  int32_t *mtp_tok = nullptr, *mtp_lab = nullptr;
  StepScalars* sc_mtp = nullptr;
  bool streaming_ce = false;  // policy switch (ft_set_streaming_ce): cross-entropy inside the logits GEMM, recomputed for dz
  float2* ce_part = nullptr;  // [ce_chunk, ceil(V / 256)] per-tile (max, sum) pairs
  float* ce_zy = nullptr;     // [ce_chunk] logit at the label
  bf16* attn_ds = nullptr;    // dS^T scratch of the attention backward (one layer's worth), or null
  size_t attn_ds_bytes = 0;
  bool attn_ds_on = true;

  // AdamW inside the weight-gradient GEMM epilogues (clipping off): the train step then never stores those gradients
  bool fused_update = true;   // policy switch (ft_set_fused_update)
  bool fused_swiglu_bwd = true;  // policy switch (ft_set_fused_swiglu_bwd): SwiGLU backward in the down projection's data-gradient epilogue
  bool fusing = false;        // true while a step that fuses is being enqueued
  int fuse_idx = 0;           // next slot region of fuse_sq
  float* fuse_sq = nullptr;   // partial sums of the squared gradient norm: [4L+1][kAdamFuseSlots] + 2 x [kSqnormBlocks]
  std::vector<AdamFuse> fuse_args;  // kept alive until the launches are enqueued
  // weight-gradient GEMMs that can carry AdamW: four per layer, the untied head, and with the MTP head its layer's four
  // and its two projections
  int n_fused() const { return 4 * L + 1 + (cfg.mtp ? 6 : 0); }
  size_t fuse_sq_count() const { return (size_t)n_fused() * kAdamFuseSlots + 2 * (size_t)kSqnormBlocks; }

  // whole-step CUDA graph: the first step of a (B, S) runs launch by launch, the second is captured, later ones replay
  bool graph_enabled = false;
  int graph_B = 0, graph_S = 0, warm_B = 0, warm_S = 0;
  cudaGraphExec_t graph_exec = nullptr;
  int64_t graph_launches = 0;
  int64_t graph_replays = 0;

  // optional per-class timing with CUDA events on the model's stream
  struct ProfRec { cudaEvent_t a, b; int cls; double work; int shape; };
  struct GemmShape { int M, N, K, a_mn, b_mn, epi, M2, N2; double ms; long long launches; };  // M2, N2: second output of a grouped launch
  std::vector<GemmShape> prof_shapes;
  bool prof = false;
  std::vector<ProfRec> prof_pending;
  std::vector<cudaEvent_t> prof_pool;
  double prof_ms[FT_PROF_CLASSES] = {0};
  double prof_work[FT_PROF_CLASSES] = {0};
  int64_t prof_launches[FT_PROF_CLASSES] = {0};
  cudaEvent_t prof_cur = nullptr;

  const ParamInfo& P(int i) const { return params[i]; }
  int per_layer() const { return cfg.qk_norm ? 8 : 6; }
  // k: 0 norm1, 1 wqkv, 2 wo, 3 norm2, 4 wgu, 5 wd, (QK-Norm: 6 q_norm, 7 k_norm)
  // layer index L + 1 (the slot of the residual stream after the MTP head's input) addresses the MTP head's layer
  int idx_layer(int l, int k) const { return l < L ? 1 + l * per_layer() + k : i_mtp + 4 + k; }
  int i_mtp = -1;  // index of mtp.norm_h: norm_h, norm_e, proj_h, proj_e, then a layer's set, then mtp.norm_f
  bf16* wb(int i) const { return pbf + params[i].offset; }
  float* gr(int i) const { return grad + params[i].offset; }
};

namespace {

// a factor of 0 in the configuration means 1
void normalise(ft_config& c) {
  if (c.emb_scale == 0.f) c.emb_scale = 1.f;
  if (c.resid_scale == 0.f) c.resid_scale = 1.f;
  if (c.logit_scale == 0.f) c.logit_scale = 1.f;
  if (c.mtp_weight == 0.f) c.mtp_weight = 1.f;
}

bool valid_config(const ft_config* c, std::string* why) {
  auto bad = [&](const char* m) { if (why) *why = m; return false; };
  if (!c) return bad("null config");
  if (c->n_layers < 1 || c->d_model < 1 || c->n_heads < 1 || c->n_kv_heads < 1 || c->d_ffn < 1 || c->vocab < 1)
    return bad("non-positive dimension");
  if (c->head_dim != 64 && c->head_dim != 128) return bad("head_dim must be 64 or 128");
  if (c->n_heads % c->n_kv_heads) return bad("n_heads must be a multiple of n_kv_heads");
  if (c->d_model % 256 || c->d_model > 4096) return bad("d_model must be a multiple of 256, at most 4096");
  if (c->d_ffn % 16) return bad("d_ffn must be a multiple of 16");
  if (c->vocab % 8) return bad("vocab must be a multiple of 8");
  if (c->max_batch < 1 || c->max_seq < 1) return bad("max_batch and max_seq must be positive");
  if ((long long)c->max_batch * c->max_seq > (1ll << 24)) return bad("max_batch * max_seq too large");
  if (c->debug_taps && c->recompute) return bad("debug_taps needs recompute = 0");
  if (!(c->rms_eps > 0.f) || !(c->rope_theta > 0.f)) return bad("rms_eps and rope_theta must be positive");
  if (c->emb_scale < 0.f || c->resid_scale < 0.f || c->logit_scale < 0.f) return bad("negative scale factor");
  if (c->tie_embeddings != 0 && c->tie_embeddings != 1) return bad("tie_embeddings must be 0 or 1");
  if (c->qk_norm != 0 && c->qk_norm != 1) return bad("qk_norm must be 0 or 1");
  if (c->mtp != 0 && c->mtp != 1) return bad("mtp must be 0 or 1");
  if (c->mtp_weight < 0.f) return bad("negative mtp_weight");
  if (c->mtp && c->debug_taps) return bad("debug_taps is not available with the MTP head");
  if (c->dp_world < 0 || c->dp_world > 32 || (c->dp_world & (c->dp_world - 1))) return bad("dp_world must be 0, 1, 2, 4, 8, 16 or 32");
  if (c->dp_rank < 0 || c->dp_rank >= (c->dp_world > 1 ? c->dp_world : 1)) return bad("dp_rank must be in [0, dp_world)");
  if (c->dp_world > 1 && c->debug_taps) return bad("debug_taps is not available with a sharded optimizer state");
  return true;
}

int pick_ce_chunk(const ft_config* c) {
  const long long T = (long long)c->max_batch * c->max_seq;
  // larger chunks mean fewer read-modify-write passes over the fp32 head gradient; logits + dlogits scratch <= 2 GiB
  long long rows = 4096;
  while (rows > 128 && rows * (long long)c->vocab * 6 > (2ll << 30)) rows >>= 1;
  if (rows > T) rows = (T + 7) / 8 * 8;
  return (int)rows;
}

void dp_build_buckets(ft_model* m);
long long state_offset(const ft_model* m, size_t off, size_t n);
void owned_part(const ft_model* m, size_t off, size_t n, size_t* lo, size_t* hi);

// Lays the model out in the workspace.  With base == nullptr it only measures.
size_t carve(ft_model* m, uint8_t* base) {
  const ft_config& c = m->cfg;
  m->h = c.d_model; m->d = c.head_dim; m->hq = c.n_heads * c.head_dim; m->hkv = c.n_kv_heads * c.head_dim;
  m->nqkv = m->hq + 2 * m->hkv; m->f = c.d_ffn; m->V = c.vocab; m->L = c.n_layers;
  m->maxT = c.max_batch * c.max_seq;
  m->n_slots = c.recompute ? 1 : c.n_layers;
  m->ce_chunk = pick_ce_chunk(&c);
  m->dz_rows = ((size_t)m->maxT * (size_t)c.vocab * sizeof(bf16) <= g_head_dz_limit && m->maxT > m->ce_chunk) ? m->maxT : m->ce_chunk;
  const size_t T = (size_t)m->maxT, h = m->h, f = m->f, hq = m->hq, nqkv = m->nqkv, V = m->V;

  // parameter table: matrices first (they get weight decay), gains after
  m->params.clear();
  auto add = [&](const std::string& n, int64_t r, int64_t cc, bool wgu) {
    ParamInfo p; p.name = n; p.rows = r; p.cols = cc; p.offset = 0; p.is_wgu = wgu; m->params.push_back(p);
  };
  add("embed", V, h, false);
  for (int l = 0; l < m->L; ++l) {
    const std::string p = "layers." + std::to_string(l) + ".";
    add(p + "norm1", h, 0, false);
    add(p + "wqkv", nqkv, h, false);
    add(p + "wo", h, hq, false);
    add(p + "norm2", h, 0, false);
    add(p + "wgu", 2 * f, h, true);
    add(p + "wd", h, f, false);
    if (c.qk_norm) {
      add(p + "q_norm", c.head_dim, 0, false);
      add(p + "k_norm", c.head_dim, 0, false);
    }
  }
  add("norm_f", h, 0, false);
  if (!c.tie_embeddings) add("lm_head", V, h, false);
  m->i_mtp = -1;
  if (c.mtp) {
    m->i_mtp = (int)m->params.size();
    add("mtp.norm_h", h, 0, false);
    add("mtp.norm_e", h, 0, false);
    add("mtp.proj_h", h, h, false);
    add("mtp.proj_e", h, h, false);
    const std::string p = "mtp.layer.";
    add(p + "norm1", h, 0, false);
    add(p + "wqkv", nqkv, h, false);
    add(p + "wo", h, hq, false);
    add(p + "norm2", h, 0, false);
    add(p + "wgu", 2 * f, h, true);
    add(p + "wd", h, f, false);
    if (c.qk_norm) {
      add(p + "q_norm", c.head_dim, 0, false);
      add(p + "k_norm", c.head_dim, 0, false);
    }
    add("mtp.norm_f", h, 0, false);
  }
  size_t off = 0;
  for (auto& p : m->params) if (p.cols) { p.offset = off; off += align_up(p.numel(), 128); }
  m->n_decay = off;
  for (auto& p : m->params) if (!p.cols) { p.offset = off; off += align_up(p.numel(), 128); }
  m->arena = off;
  m->dp_world = c.dp_world > 1 ? c.dp_world : 1;
  m->dp_rank = c.dp_world > 1 ? c.dp_rank : 0;
  m->dp_buckets.clear();
  dp_build_buckets(m);
  m->state_elems = m->arena / (size_t)m->dp_world;  // every bucket is a multiple of 128 elements, dp_world divides 32

  Carver cv; cv.base = base;
  m->master = cv.take<float>(m->state_elems);
  m->adam_m = cv.take<float>(m->state_elems);
  m->adam_v = cv.take<float>(m->state_elems);
  m->grad = cv.take<float>(m->arena);
  m->pbf = cv.take<bf16>(m->arena);
  m->rope_cosT = cv.take<float>((size_t)c.max_seq * (m->d / 2));
  m->rope_sinT = cv.take<float>((size_t)c.max_seq * (m->d / 2));
  m->rope_cos = cv.take<float>((size_t)c.max_seq * (m->d / 2));
  m->rope_sin = cv.take<float>((size_t)c.max_seq * (m->d / 2));
  m->sc = cv.take<StepScalars>(1);
  m->tok_dev = cv.take<int32_t>(T);
  m->lab_dev = cv.take<int32_t>(T);
  m->x.assign(m->L + 1, nullptr);
  if (c.mtp) m->x.assign(m->L + 3, nullptr);  // x[L+1]: input of the MTP head's layer, x[L+2]: its output
  for (size_t l = 0; l < m->x.size(); ++l) m->x[l] = cv.take<bf16>(T * h);
  m->acts.assign(m->n_slots, LayerActs());
  for (auto& a : m->acts) {
    a.h1 = cv.take<bf16>(T * h); a.qkv = cv.take<bf16>(T * nqkv); a.o = cv.take<bf16>(T * hq);
    a.x_mid = cv.take<bf16>(T * h); a.h2 = cv.take<bf16>(T * h); a.gu = cv.take<bf16>(T * 2 * f);
    a.a = cv.take<bf16>(T * f); a.lse = cv.take<float>(T * c.n_heads); a.r1 = cv.take<float>(T);
    a.r2 = cv.take<float>(T);
    a.qk_r = c.qk_norm ? cv.take<float>(T * (size_t)(c.n_heads + c.n_kv_heads)) : nullptr;
  }
  if (c.mtp) {
    LayerActs& a = m->acts_mtp;
    a.h1 = cv.take<bf16>(T * h); a.qkv = cv.take<bf16>(T * nqkv); a.o = cv.take<bf16>(T * hq);
    a.x_mid = cv.take<bf16>(T * h); a.h2 = cv.take<bf16>(T * h); a.gu = cv.take<bf16>(T * 2 * f);
    a.a = cv.take<bf16>(T * f); a.lse = cv.take<float>(T * c.n_heads); a.r1 = cv.take<float>(T);
    a.r2 = cv.take<float>(T);
    a.qk_r = c.qk_norm ? cv.take<float>(T * (size_t)(c.n_heads + c.n_kv_heads)) : nullptr;
    m->mtp_hn = cv.take<bf16>(T * h); m->mtp_xe = cv.take<bf16>(T * h); m->mtp_en = cv.take<bf16>(T * h);
    m->mtp_u1 = cv.take<bf16>(T * h); m->mtp_hF = cv.take<bf16>(T * h); m->mtp_d_hF = cv.take<bf16>(T * h);
    m->mtp_d_en = cv.take<bf16>(T * h); m->mtp_d_hn = cv.take<bf16>(T * h); m->mtp_d_xe = cv.take<bf16>(T * h);
    m->mtp_d_xL = cv.take<bf16>(T * h);
    m->mtp_rh = cv.take<float>(T); m->mtp_re = cv.take<float>(T); m->mtp_rF = cv.take<float>(T); m->mtp_lse = cv.take<float>(T);
    m->mtp_tok = cv.take<int32_t>(T); m->mtp_lab = cv.take<int32_t>(T);
    m->sc_mtp = cv.take<StepScalars>(1);
  }
  m->rF = cv.take<float>(T); m->ce_lse = cv.take<float>(T); m->loss_row = cv.take<float>(T);
  m->hF = cv.take<bf16>(T * h); m->d_hF = cv.take<bf16>(T * h);
  m->dxA = cv.take<bf16>(T * h); m->dxB = cv.take<bf16>(T * h); m->d_h = cv.take<bf16>(T * h);
  m->d_a = cv.take<bf16>(T * f); m->d_gu = cv.take<bf16>(T * 2 * f); m->d_o = cv.take<bf16>(T * hq);
  m->d_qkv = cv.take<bf16>(T * nqkv);
  m->delta = cv.take<float>(T * c.n_heads);
  // dS^T of one layer's attention backward, when the longest sequence allows the stored-dS path and it stays modest
  m->attn_ds_bytes = attention_bwd_ds_bytes(c.max_batch, c.max_seq, c.n_heads);
  if (m->attn_ds_bytes > kAttnDsMaxBytes) m->attn_ds_bytes = 0;
  m->attn_ds = m->attn_ds_bytes ? cv.take<bf16>(m->attn_ds_bytes / sizeof(bf16)) : nullptr;
  m->norm_slot_of.assign(m->params.size(), -1);
  m->n_norm_slots = 0;
  for (size_t i = 0; i < m->params.size(); ++i)
    if (!m->params[i].cols && m->params[i].rows == (int64_t)h) m->norm_slot_of[i] = m->n_norm_slots++;
  const size_t slot_floats = (size_t)elementwise_blocks_for_norm((int)T) * h;
  m->norm_partial = cv.take<float>((size_t)(m->n_norm_slots + 1) * slot_floats);
  m->qk_partial = m->norm_partial ? m->norm_partial + (size_t)m->n_norm_slots * slot_floats : nullptr;
  m->norm_out = cv.take<float*>((size_t)m->n_norm_slots);
  m->sq_partial = cv.take<float>(kSqnormBlocks);
  m->dp_sq = cv.take<float>(4);
  m->ce_part = cv.take<float2>((size_t)m->ce_chunk * ((V + 255) / 256));
  m->ce_zy = cv.take<float>((size_t)m->ce_chunk);
  m->fuse_sq = cv.take<float>(m->fuse_sq_count());
  m->splitk = cv.take<float>(kSplitKFloats);
  m->splitk2 = cv.take<float>(kSplitKFloats);
  m->z = cv.take<float>((size_t)m->ce_chunk * V);
  m->dz = cv.take<bf16>((size_t)m->dz_rows * V);
  m->keys = cv.take<unsigned long long>(sort_pad(T));
  m->taps.clear();
  if (c.debug_taps) {
    m->taps.assign(m->L, LayerTaps());
    for (auto& t : m->taps) {
      t.d_x_out = cv.take<bf16>(T * h); t.d_a = cv.take<bf16>(T * f); t.d_gu = cv.take<bf16>(T * 2 * f);
      t.d_h2 = cv.take<bf16>(T * h); t.d_x_mid = cv.take<bf16>(T * h); t.d_o = cv.take<bf16>(T * hq);
      t.d_qkv = cv.take<bf16>(T * nqkv); t.d_h1 = cv.take<bf16>(T * h); t.d_x_in = cv.take<bf16>(T * h);
    }
  }
  return align_up(cv.off, kAlign);
}

ft_status fail(ft_model* m, ft_status s, const std::string& msg) {
  if (m) m->err = msg;
  return s;
}
ft_status cuda_fail(ft_model* m, cudaError_t e, const char* where) {
  return fail(m, FT_ECUDA, std::string(where) + ": " + cudaGetErrorString(e));
}

#define FT_CUDA(call)                                              \
  do {                                                             \
    cudaError_t e__ = (call);                                      \
    if (e__ != cudaSuccess) return cuda_fail(m, e__, #call);       \
  } while (0)
// cls: profiling class of the launch, work: its algorithmic bytes (or flops for contractions)
#define FT_LAUNCH(cls, work, call)                                                          \
  do {                                                                                      \
    prof_begin(m);                                                                          \
    int n__ = (call);                                                                       \
    if (n__ < 0) return fail(m, FT_ECUDA, std::string("kernel launch failed: ") + #call);   \
    m->launches += n__;                                                                     \
    prof_end(m, cls, work, n__);                                                            \
  } while (0)
#define FT_GEMM(args) FT_GEMM_ON(args, m->stream)
#define FT_GEMM_ON(args, stream_)                                                           \
  do {                                                                                      \
    prof_begin(m);                                                                          \
    int nl__ = 1;                                                                           \
    cudaError_t e__ = launch_gemm(args, stream_, &nl__);                                    \
    if (e__ != cudaSuccess) return cuda_fail(m, e__, "launch_gemm");                        \
    m->launches += nl__;                                                                    \
    prof_end(m, FT_PROF_GEMM, 2.0 * (double)(args).M * (double)(args).N * (double)(args).K, 1, prof_shape_index(m, args)); \
  } while (0)
// two weight gradients as one launch (gemm_group2_ok(a0, a1) holds)
#define FT_GEMM_GROUP_ON(a0, a1, stream_)                                                   \
  do {                                                                                      \
    prof_begin(m);                                                                          \
    int nl__ = 1;                                                                           \
    cudaError_t e__ = launch_gemm_group2(a0, a1, stream_, &nl__);                           \
    if (e__ != cudaSuccess) return cuda_fail(m, e__, "launch_gemm_group2");                 \
    m->launches += nl__;                                                                    \
    prof_end(m, FT_PROF_GEMM,                                                               \
             2.0 * (double)(a0).K * ((double)(a0).M * (double)(a0).N + (double)(a1).M * (double)(a1).N), 1, \
             prof_shape_index(m, a0, &(a1)));                                               \
  } while (0)

cudaEvent_t prof_event(ft_model* m) {
  if (!m->prof_pool.empty()) { cudaEvent_t e = m->prof_pool.back(); m->prof_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}
inline void prof_begin(ft_model* m) {
  if (!m->prof) return;
  m->prof_cur = prof_event(m);
  cudaEventRecord(m->prof_cur, m->stream);
}
inline void prof_end(ft_model* m, int cls, double work, int launches, int shape = -1) {
  if (!m->prof || !m->prof_cur) return;
  ft_model::ProfRec r;
  r.a = m->prof_cur; r.b = prof_event(m); r.cls = cls; r.work = work; r.shape = shape;
  cudaEventRecord(r.b, m->stream);
  m->prof_pending.push_back(r);
  m->prof_launches[cls] += launches;
  m->prof_cur = nullptr;
}
// turns finished event pairs into per-class totals (the stream must be idle)
void prof_collect(ft_model* m) {
  for (auto& r : m->prof_pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) {
      m->prof_ms[r.cls] += ms;
      m->prof_work[r.cls] += r.work;
      if (r.shape >= 0) { m->prof_shapes[r.shape].ms += ms; m->prof_shapes[r.shape].launches += 1; }
    }
    m->prof_pool.push_back(r.a);
    m->prof_pool.push_back(r.b);
  }
  m->prof_pending.clear();
}

// index of this GEMM's (shape, layout, epilogue) in the per-shape profile table
int prof_shape_index(ft_model* m, const GemmArgs& g, const GemmArgs* second = nullptr) {
  if (!m->prof) return -1;
  const int M2 = second ? second->M : 0, N2 = second ? second->N : 0;
  for (size_t i = 0; i < m->prof_shapes.size(); ++i) {
    const auto& s = m->prof_shapes[i];
    if (s.M == g.M && s.N == g.N && s.K == g.K && s.a_mn == g.a_mn && s.b_mn == g.b_mn && s.epi == g.epi && s.M2 == M2 && s.N2 == N2)
      return (int)i;
  }
  ft_model::GemmShape s = {g.M, g.N, g.K, g.a_mn, g.b_mn, g.epi, M2, N2, 0.0, 0};
  m->prof_shapes.push_back(s);
  return (int)m->prof_shapes.size() - 1;
}

AdamHyper hyper(const ft_model* m) {
  AdamHyper hp;
  hp.lr = m->cfg.lr; hp.beta1 = m->cfg.beta1; hp.beta2 = m->cfg.beta2; hp.eps = m->cfg.adam_eps;
  hp.wd = m->cfg.weight_decay; hp.max_grad_norm = m->cfg.max_grad_norm;
  return hp;
}

GemmArgs gemm_base(ft_model* m) {
  GemmArgs g;
  g.err = &m->sc->err;
  g.scratch = m->splitk;
  g.scratch_bytes = kSplitKFloats * sizeof(float);
  return g;
}

// AdamW arguments for the weight-gradient GEMM of parameter wi (a matrix: decayed), with the next norm-slot region
const AdamFuse* fuse_for(ft_model* m, int wi) {
  const size_t off = m->params[wi].offset;
  AdamFuse a;
  a.p = m->master + off; a.m = m->adam_m + off; a.v = m->adam_v + off; a.pb = m->pbf + off;
  a.scalars = m->sc;
  a.lr = m->cfg.lr; a.beta1 = m->cfg.beta1; a.beta2 = m->cfg.beta2; a.eps = m->cfg.adam_eps; a.wd = m->cfg.weight_decay;
  a.sq_slots = m->fuse_sq + (size_t)m->fuse_idx * kAdamFuseSlots;
  m->fuse_idx += 1;
  m->fuse_args.push_back(a);
  return &m->fuse_args.back();
}

// the slot of norm_partial that receives the block partials of gain parameter i's gradient
float* norm_slot(ft_model* m, int i) {
  return m->norm_partial + (size_t)m->norm_slot_of[i] * (size_t)elementwise_blocks_for_norm(m->maxT) * m->h;
}

// forward of layer l from m->x[l] into activation slot `a`, output to m->x[l+1]
ft_status layer_forward(ft_model* m, int l, LayerActs& a, int B, int S) {
  const int T = B * S, h = m->h, f = m->f, hq = m->hq, nqkv = m->nqkv;
  cudaStream_t st = m->stream;
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(m->x[l], m->wb(m->idx_layer(l, 0)), a.h1, a.r1, T, h, m->cfg.rms_eps, st));
  {
    GemmArgs g = gemm_base(m);
    g.A = a.h1; g.lda = h; g.B = m->wb(m->idx_layer(l, 1)); g.ldb = h; g.C = a.qkv; g.ldc = nqkv;
    g.M = T; g.N = nqkv; g.K = h; g.epi = EPI_ROPE;
    g.rope_cos = m->rope_cosT; g.rope_sin = m->rope_sinT; g.rope_ld = m->cfg.max_seq; g.seq = S; g.head_dim = m->d;
    g.rope_cols = hq + m->hkv;
    if (m->cfg.qk_norm) {
      g.qk_r = a.qk_r; g.qk_gain_q = m->wb(m->idx_layer(l, 6)); g.qk_gain_k = m->wb(m->idx_layer(l, 7));
      g.n_q_heads = m->cfg.n_heads; g.qk_eps = m->cfg.rms_eps;
    }
    FT_GEMM(g);
  }
  prof_begin(m);
  FT_CUDA(attention_fwd(a.qkv, a.o, a.lse, B, S, m->cfg.n_heads, m->cfg.n_kv_heads, m->d, &m->sc->err, st));
  m->launches += 1;
  prof_end(m, FT_PROF_ATTN_FWD, 2.0 * B * m->cfg.n_heads * (double)S * S * m->d, 1);
  {
    GemmArgs g = gemm_base(m);
    g.A = a.o; g.lda = hq; g.B = m->wb(m->idx_layer(l, 2)); g.ldb = hq; g.C = a.x_mid; g.ldc = h; g.resid = m->x[l];
    g.M = T; g.N = h; g.K = hq; g.epi = EPI_BF16_RESID; g.alpha = m->cfg.resid_scale;
    FT_GEMM(g);
  }
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(a.x_mid, m->wb(m->idx_layer(l, 3)), a.h2, a.r2, T, h, m->cfg.rms_eps, st));
  {
    GemmArgs g = gemm_base(m);
    g.A = a.h2; g.lda = h; g.B = m->wb(m->idx_layer(l, 4)); g.ldb = h; g.C = a.a; g.ldc = f; g.gu = a.gu; g.d_ffn = f;
    g.M = T; g.N = 2 * f; g.K = h; g.epi = EPI_SWIGLU;
    FT_GEMM(g);
  }
  {
    GemmArgs g = gemm_base(m);
    g.A = a.a; g.lda = f; g.B = m->wb(m->idx_layer(l, 5)); g.ldb = f; g.C = m->x[l + 1]; g.ldc = h; g.resid = a.x_mid;
    g.M = T; g.N = h; g.K = f; g.epi = EPI_BF16_RESID; g.alpha = m->cfg.resid_scale;
    FT_GEMM(g);
  }
  return FT_OK;
}

ft_status copy_tap(ft_model* m, bf16* dst, const bf16* src, size_t n) {
  FT_CUDA(cudaMemcpyAsync(dst, src, n * sizeof(bf16), cudaMemcpyDeviceToDevice, m->stream));
  return FT_OK;
}

// data gradient  dX[T, n_in] = dY[T, n_out] W[n_out, n_in]  and weight gradient  dW[n_out, n_in] = dY^T X
// Main stream waits until the k-th weight gradient enqueued on the second stream has finished (no-op when none is).
ft_status wait_wgrad(ft_model* m, int k) {
  if (!m->w_pending[k]) return FT_OK;
  FT_CUDA(cudaStreamWaitEvent(m->stream, m->ev_w[k], 0));
  m->w_pending[k] = false;
  return FT_OK;
}

// A weight gradient whose launch is put off until the next one of the layer is ready, so that both run as one launch
struct WgradHold {
  GemmArgs g;
  int k = -1;
  bool valid = false;
};

// Enqueues the weight gradient g (slot k of the layer's four) and, when `held` holds one, that one with it: as ONE grouped
// launch when the two qualify (the partly filled last wave and the exposed optimizer epilogue of the first then run
// beside the second's tiles), else as two launches.  On the second stream when the step overlaps, after every data
// gradient enqueued so far (they still read the bf16 weights the fused update overwrites).
ft_status wgrad_launch(ft_model* m, GemmArgs g, int k, WgradHold* held) {
  const bool have = held != nullptr && held->valid;
  cudaStream_t on = m->stream;
  if (m->overlapping) {
    ft_status s = wait_wgrad(m, k);  // one weight gradient per slot in flight
    if (s) return s;
    if (have && (s = wait_wgrad(m, held->k))) return s;
    FT_CUDA(cudaEventRecord(m->ev_d, m->stream));
    FT_CUDA(cudaStreamWaitEvent(m->side, m->ev_d, 0));
    g.scratch = m->splitk2;
    if (have) held->g.scratch = m->splitk2;
    on = m->side;
  }
  if (have && gemm_group2_ok(held->g, g)) {
    FT_GEMM_GROUP_ON(held->g, g, on);
  } else {
    if (have) FT_GEMM_ON(held->g, on);
    FT_GEMM_ON(g, on);
  }
  if (m->overlapping) {
    FT_CUDA(cudaEventRecord(m->ev_w[k], m->side));
    m->w_pending[k] = true;
    if (have) {
      FT_CUDA(cudaEventRecord(m->ev_w[held->k], m->side));
      m->w_pending[held->k] = true;
    }
  }
  if (held) held->valid = false;
  return FT_OK;
}

// dX = dY W (data gradient) and dW = dY^T X (weight gradient, slot k of the layer's four)
// alpha: factor the branch output carried into the residual stream (its gradient is alpha * dY, never rounded)
// swiglu_gu: when given, X is the SwiGLU output a = silu(G) U of the gate|up tensor swiglu_gu [T, 2 n_in], dX is not
// stored, and the data-gradient epilogue writes d_gate, d_up to swiglu_dgu [T, 2 n_in] (alternating 16 / 16 columns)
// hold: the weight gradient is not enqueued but left there for a later call; join: a held one to enqueue with this one
ft_status linear_backward(ft_model* m, const bf16* dY, const bf16* X, int wi, bf16* dX, int T, int n_out, int n_in, int k,
                          float alpha = 1.0f, const bf16* swiglu_gu = nullptr, bf16* swiglu_dgu = nullptr,
                          WgradHold* hold = nullptr, WgradHold* join = nullptr) {
  {
    GemmArgs g = gemm_base(m);
    g.A = dY; g.lda = n_out; g.B = m->wb(wi); g.b_mn = 1; g.ldb = n_in; g.C = dX; g.ldc = n_in;
    g.M = T; g.N = n_in; g.K = n_out; g.epi = EPI_BF16; g.alpha = alpha;
    if (swiglu_gu != nullptr) {
      g.epi = EPI_SWIGLU_BWD; g.C = swiglu_dgu; g.ldc = 2LL * n_in; g.gu = const_cast<bf16*>(swiglu_gu); g.d_ffn = n_in;
    }
    FT_GEMM(g);
  }
  {
    GemmArgs g = gemm_base(m);
    g.A = dY; g.a_mn = 1; g.lda = n_out; g.B = X; g.b_mn = 1; g.ldb = n_in; g.C = m->gr(wi); g.ldc = n_in;
    g.M = n_out; g.N = n_in; g.K = T; g.epi = EPI_F32; g.alpha = alpha;
    if (m->fusing) g.adam = fuse_for(m, wi);
    if (hold != nullptr) {
      hold->g = g; hold->k = k; hold->valid = true;
      return FT_OK;
    }
    return wgrad_launch(m, g, k, join);
  }
}

ft_status layer_backward(ft_model* m, int l, LayerActs& a, int B, int S) {
  const int T = B * S, h = m->h, f = m->f, hq = m->hq, nqkv = m->nqkv;
  cudaStream_t st = m->stream;
  LayerTaps* tp = m->cfg.debug_taps ? &m->taps[l] : nullptr;
  // m->dxA holds d_x_out
  if (tp) { ft_status s = copy_tap(m, tp->d_x_out, m->dxA, (size_t)T * h); if (s) return s; }
  ft_status s;
  WgradHold held;
  if (m->fused_swiglu_bwd && !tp) {
    // d_a stays in the data-gradient GEMM's accumulators: its epilogue reads gate | up and writes d_gate | d_up
    if ((s = wait_wgrad(m, 1))) return s;  // the previous layer's gate/up weight gradient still reads d_gu
    s = linear_backward(m, m->dxA, a.a, m->idx_layer(l, 5), nullptr, T, h, f, 0, m->cfg.resid_scale, a.gu, m->d_gu, &held);
    if (s) return s;
  } else {
    s = linear_backward(m, m->dxA, a.a, m->idx_layer(l, 5), m->d_a, T, h, f, 0, m->cfg.resid_scale, nullptr, nullptr, &held);
    if (s) return s;
    if ((s = wait_wgrad(m, 1))) return s;  // the previous layer's gate/up weight gradient still reads d_gu
    FT_LAUNCH(FT_PROF_ELEMENTWISE, 10.0 * T * f, swiglu_bwd(m->d_a, a.gu, m->d_gu, T, f, st));
  }
  // the down projection's weight gradient (held) and the gate/up one: one launch
  s = linear_backward(m, m->d_gu, a.h2, m->idx_layer(l, 4), m->d_h, T, 2 * f, h, 1, 1.0f, nullptr, nullptr, nullptr, &held);
  if (s) return s;
  if (tp) {
    if ((s = copy_tap(m, tp->d_a, m->d_a, (size_t)T * f))) return s;
    if ((s = copy_tap(m, tp->d_gu, m->d_gu, (size_t)T * 2 * f))) return s;
    if ((s = copy_tap(m, tp->d_h2, m->d_h, (size_t)T * h))) return s;
  }
  if ((s = wait_wgrad(m, 2))) return s;  // the previous layer's output-projection weight gradient still reads dxB
  FT_LAUNCH(FT_PROF_NORM, 8.0 * T * h, rmsnorm_bwd(m->d_h, a.x_mid, a.r2, m->wb(m->idx_layer(l, 3)), m->dxA, m->dxB,
                                                    norm_slot(m, m->idx_layer(l, 3)), T, h, st));
  s = linear_backward(m, m->dxB, a.o, m->idx_layer(l, 2), m->d_o, T, h, hq, 2, m->cfg.resid_scale, nullptr, nullptr, &held);
  if (s) return s;
  if ((s = wait_wgrad(m, 3))) return s;  // the previous layer's qkv weight gradient still reads d_qkv
  prof_begin(m);
  FT_CUDA(attention_bwd_ws(a.qkv, a.o, m->d_o, a.lse, m->delta, m->d_qkv, m->rope_cos, m->rope_sin,
                           m->attn_ds_on ? m->attn_ds : nullptr, m->attn_ds_bytes, B, S, m->cfg.n_heads, m->cfg.n_kv_heads,
                           m->d, &m->sc->err, st));
  m->launches += 3;
  prof_end(m, FT_PROF_ATTN_BWD, 4.0 * B * m->cfg.n_heads * (double)S * S * m->d, 3);
  if (m->cfg.qk_norm) {
    // d_q, d_k so far are gradients of the normalised heads: through the per-head norm, in place, and the two gain gradients
    FT_LAUNCH(FT_PROF_NORM, 6.0 * T * (hq + m->hkv),
              qknorm_bwd(m->d_qkv, a.qkv, a.qk_r, m->wb(m->idx_layer(l, 6)), m->wb(m->idx_layer(l, 7)), m->rope_cos,
                         m->rope_sin, m->gr(m->idx_layer(l, 6)), m->gr(m->idx_layer(l, 7)), m->qk_partial,
                         (size_t)elementwise_blocks_for_norm(m->maxT) * h, 1.0f / (m->rope_mscale * m->rope_mscale), T, S,
                         m->cfg.n_heads, m->cfg.n_kv_heads, m->d, st));
  }
  // the output projection's weight gradient (held) and the qkv one: one launch
  s = linear_backward(m, m->d_qkv, a.h1, m->idx_layer(l, 1), m->d_h, T, nqkv, h, 3, 1.0f, nullptr, nullptr, nullptr, &held);
  if (s) return s;
  if (tp) {
    if ((s = copy_tap(m, tp->d_x_mid, m->dxB, (size_t)T * h))) return s;
    if ((s = copy_tap(m, tp->d_o, m->d_o, (size_t)T * hq))) return s;
    if ((s = copy_tap(m, tp->d_qkv, m->d_qkv, (size_t)T * nqkv))) return s;
    if ((s = copy_tap(m, tp->d_h1, m->d_h, (size_t)T * h))) return s;
  }
  if ((s = wait_wgrad(m, 0))) return s;  // this layer's down-projection weight gradient still reads dxA
  FT_LAUNCH(FT_PROF_NORM, 8.0 * T * h, rmsnorm_bwd(m->d_h, m->x[l], a.r1, m->wb(m->idx_layer(l, 0)), m->dxB, m->dxA,
                                                    norm_slot(m, m->idx_layer(l, 0)), T, h, st));
  if (tp) { if ((s = copy_tap(m, tp->d_x_in, m->dxA, (size_t)T * h))) return s; }
  return FT_OK;
}

// Output head + cross-entropy (+ both head gradients) of the hidden states hF against `lab`, in chunks of rows: the
// logits of one chunk at a time.  sc holds the label count the mean runs over; dz_scale multiplies the logit gradient
// (logit factor, times the loss weight of this head); accumulate: the head's weight gradient already holds another
// head's contribution; fuse_last: the last chunk completes that gradient and may carry AdamW.
ft_status head_pass(ft_model* m, const bf16* hF, const int32_t* lab, float* lse, bf16* d_hF, StepScalars* sc, float dz_scale,
                    int i_head, int T, bool with_bwd, bool accumulate, bool fuse_last) {
  const int h = m->h, V = m->V;
  cudaStream_t st = m->stream;
  // one_pass: dz of every row is kept and both head gradients are single contractions after the chunk loop
  const bool one_pass = with_bwd && m->dz_rows >= T && T > m->ce_chunk;
  for (int r0 = 0, chunk = 0; r0 < T; r0 += m->ce_chunk, ++chunk) {
    const int rows = (T - r0) < m->ce_chunk ? (T - r0) : m->ce_chunk;
    bf16* dz = one_pass ? m->dz + (size_t)r0 * V : m->dz;
    if (m->streaming_ce) {
      // no logits in memory: the GEMM's epilogue reduces each 256-column tile of a row to (max, sum), a small kernel
      // combines them, and the same GEMM runs again with an epilogue that turns its accumulators into bf16 dz
      GemmArgs g = gemm_base(m);
      g.A = hF + (size_t)r0 * h; g.lda = h; g.B = m->wb(i_head); g.ldb = h; g.C = dz; g.ldc = V;
      g.M = rows; g.N = V; g.K = h; g.epi = EPI_BF16; g.alpha = m->cfg.logit_scale;
      g.ce_mode = 1; g.ce_part = m->ce_part; g.ce_tiles = (V + 255) / 256; g.ce_zy = m->ce_zy; g.ce_labels = lab + r0;
      FT_GEMM(g);
      FT_LAUNCH(FT_PROF_CE, 8.0 * rows * g.ce_tiles,
                ce_combine(m->ce_part, g.ce_tiles, m->ce_zy, lab + r0, lse + r0, m->loss_row + r0, rows, V, st));
      if (with_bwd) {
        g.ce_mode = 2; g.ce_lse = lse + r0; g.ce_scalars = sc; g.ce_scale = dz_scale;
        FT_GEMM(g);
      }
    } else {
      {
        GemmArgs g = gemm_base(m);
        g.A = hF + (size_t)r0 * h; g.lda = h; g.B = m->wb(i_head); g.ldb = h; g.C = m->z; g.ldc = V;
        g.M = rows; g.N = V; g.K = h; g.epi = EPI_F32; g.alpha = m->cfg.logit_scale;
        FT_GEMM(g);
      }
      FT_LAUNCH(FT_PROF_CE, (with_bwd ? 10.0 : 4.0) * rows * V,
                cross_entropy_rows(m->z, lab + r0, lse + r0, m->loss_row + r0, with_bwd ? dz : nullptr, rows, V,
                                   sc, dz_scale, st));
    }
    if (with_bwd && !one_pass) {
      {
        GemmArgs g = gemm_base(m);
        g.A = dz; g.lda = V; g.B = m->wb(i_head); g.b_mn = 1; g.ldb = h; g.C = d_hF + (size_t)r0 * h; g.ldc = h;
        g.M = rows; g.N = h; g.K = V; g.epi = EPI_BF16;
        FT_GEMM(g);
      }
      {
        GemmArgs g = gemm_base(m);
        g.A = dz; g.a_mn = 1; g.lda = V; g.B = hF + (size_t)r0 * h; g.b_mn = 1; g.ldb = h; g.C = m->gr(i_head);
        g.ldc = h; g.M = V; g.N = h; g.K = rows; g.epi = (chunk == 0 && !accumulate) ? EPI_F32 : EPI_F32_ACC;
        // the last chunk completes the gradient (with tied embeddings the table's own part is still to come)
        if (m->fusing && fuse_last && r0 + rows >= T) g.adam = fuse_for(m, i_head);
        FT_GEMM(g);
      }
    }
  }
  if (one_pass) {
    {
      GemmArgs g = gemm_base(m);
      g.A = m->dz; g.lda = V; g.B = m->wb(i_head); g.b_mn = 1; g.ldb = h; g.C = d_hF; g.ldc = h;
      g.M = T; g.N = h; g.K = V; g.epi = EPI_BF16;
      FT_GEMM(g);
    }
    {
      // the weight gradient in one contraction over all rows: no fp32 read-modify-write passes over a [V, h] tensor
      GemmArgs g = gemm_base(m);
      g.A = m->dz; g.a_mn = 1; g.lda = V; g.B = hF; g.b_mn = 1; g.ldb = h; g.C = m->gr(i_head);
      g.ldc = h; g.M = V; g.N = h; g.K = T; g.epi = accumulate ? EPI_F32_ACC : EPI_F32;
      if (m->fusing && fuse_last) g.adam = fuse_for(m, i_head);
      FT_GEMM(g);
    }
  }
  return FT_OK;
}

// One-layer MTP head, forward and its own output-head pass: the normalised last hidden state and the normalised
// embedding of the next token are projected (two h x h matrices, the second GEMM adds the first's rounded output) into
// the input of one more decoder layer; its normalised output goes through the backbone's output head against the
// labels shifted by one; the step's loss becomes loss + mtp_weight * (this head's mean cross-entropy).
ft_status mtp_forward_and_head(ft_model* m, const int32_t* tok, const int32_t* lab, int B, int S, int i_head, bool with_bwd) {
  const int T = B * S, h = m->h, V = m->V, L = m->L, i0 = m->i_mtp, i_nf = i0 + 4 + m->per_layer();
  cudaStream_t st = m->stream;
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 16.0 * T, mtp_shift(tok, lab, m->mtp_tok, m->mtp_lab, T, S, st));
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(m->x[L], m->wb(i0), m->mtp_hn, m->mtp_rh, T, h, m->cfg.rms_eps, st));
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T * h, embed_fwd(m->mtp_tok, m->wb(0), m->mtp_xe, T, h, V, m->cfg.emb_scale, st));
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(m->mtp_xe, m->wb(i0 + 1), m->mtp_en, m->mtp_re, T, h, m->cfg.rms_eps, st));
  {
    GemmArgs g = gemm_base(m);
    g.A = m->mtp_hn; g.lda = h; g.B = m->wb(i0 + 2); g.ldb = h; g.C = m->mtp_u1; g.ldc = h;
    g.M = T; g.N = h; g.K = h; g.epi = EPI_BF16;
    FT_GEMM(g);
  }
  {
    GemmArgs g = gemm_base(m);
    g.A = m->mtp_en; g.lda = h; g.B = m->wb(i0 + 3); g.ldb = h; g.C = m->x[L + 1]; g.ldc = h; g.resid = m->mtp_u1;
    g.M = T; g.N = h; g.K = h; g.epi = EPI_BF16_RESID;
    FT_GEMM(g);
  }
  ft_status s = layer_forward(m, L + 1, m->acts_mtp, B, S);
  if (s) return s;
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(m->x[L + 2], m->wb(i_nf), m->mtp_hF, m->mtp_rF, T, h, m->cfg.rms_eps, st));
  // data parallelism: the second element of the device count array is the shifted labels' count over all ranks
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T,
            count_labels(m->mtp_lab, nullptr, T, V, m->sc_mtp, nullptr, 0, m->label_count_dev ? m->label_count_dev + 1 : nullptr, st));
  // this pass completes the head's weight gradient: its last chunk may carry AdamW (untied head only)
  s = head_pass(m, m->mtp_hF, m->mtp_lab, m->mtp_lse, m->mtp_d_hF, m->sc_mtp, m->cfg.logit_scale * m->cfg.mtp_weight, i_head, T,
                with_bwd, true, m->cfg.tie_embeddings == 0);
  if (s) return s;
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T, reduce_loss(m->loss_row, T, m->sc_mtp, st));
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 0.0, add_loss(m->sc, m->sc_mtp, m->cfg.mtp_weight, st));
  return FT_OK;
}

// Its backward: through the head's final norm, the layer, the two projections and the two input norms.  Leaves the
// gradient with respect to the backbone's last hidden state in mtp_d_xL (bf16; the backbone's final-norm backward adds
// it inside its one rounding) and scatters the next-token embedding gradient into the table's gradient.
ft_status mtp_backward(ft_model* m, int B, int S, bool tied) {
  const int T = B * S, h = m->h, V = m->V, L = m->L, i0 = m->i_mtp, i_nf = i0 + 4 + m->per_layer();
  cudaStream_t st = m->stream;
  FT_LAUNCH(FT_PROF_NORM, 6.0 * T * h, rmsnorm_bwd(m->mtp_d_hF, m->x[L + 2], m->mtp_rF, m->wb(i_nf), nullptr, m->dxA, norm_slot(m, i_nf), T, h, st));
  ft_status s = layer_backward(m, L + 1, m->acts_mtp, B, S);
  if (s) return s;
  // h' = R(u1 + en We^T), u1 = R(hn Wh^T): the add hands the same gradient (dxA) to both projections
  if ((s = linear_backward(m, m->dxA, m->mtp_en, i0 + 3, m->mtp_d_en, T, h, h, 0))) return s;
  if ((s = linear_backward(m, m->dxA, m->mtp_hn, i0 + 2, m->mtp_d_hn, T, h, h, 0))) return s;
  FT_LAUNCH(FT_PROF_NORM, 6.0 * T * h, rmsnorm_bwd(m->mtp_d_en, m->mtp_xe, m->mtp_re, m->wb(i0 + 1), nullptr, m->mtp_d_xe,
                                                    norm_slot(m, i0 + 1), T, h, st));
  // with tied embeddings the head passes have already written the table's gradient; otherwise this is its first part
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 2.0 * T * h + 4.0 * V * h,
            embed_bwd(m->mtp_tok, m->mtp_d_xe, m->gr(0), m->keys, T, h, V, m->cfg.emb_scale, tied, st));
  FT_LAUNCH(FT_PROF_NORM, 6.0 * T * h, rmsnorm_bwd(m->mtp_d_hn, m->x[L], m->mtp_rh, m->wb(i0), nullptr, m->mtp_d_xL, norm_slot(m, i0), T, h, st));
  return FT_OK;
}

// forward (+ backward when with_bwd) of one batch; everything is enqueued, nothing is synchronised
ft_status run_forward_backward(ft_model* m, const int32_t* tok, const int32_t* lab, int B, int S, bool with_bwd,
                               bool fuse = false) {
  if (!m || !tok || !lab) return fail(m, FT_EINVAL, "null argument");
  if (B < 1 || S < 1 || B > m->cfg.max_batch || S > m->cfg.max_seq) return fail(m, FT_EINVAL, "B or S out of range");
  const int T = B * S, h = m->h, V = m->V, L = m->L;
  cudaStream_t st = m->stream;
  m->lastB = B; m->lastS = S; m->have_bwd = false;
  m->fusing = fuse && with_bwd;
  m->overlapping = with_bwd && m->overlap && m->side != nullptr && !m->prof && !m->cfg.debug_taps && !m->dp_mode;
  m->fuse_idx = 0;
  m->fuse_args.clear();
  m->fuse_args.reserve((size_t)m->n_fused());  // pointers into it are handed to the launcher
  if (m->fusing) {
    // the optimizer step counter and bias corrections must be current before the first weight-gradient epilogue
    FT_CUDA(cudaMemsetAsync(m->fuse_sq, 0, m->fuse_sq_count() * sizeof(float), st));
    FT_LAUNCH(FT_PROF_OPTIMIZER, 0.0, advance_step(m->sc, hyper(m), st));
  }

  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T, count_labels(lab, tok, T, V, m->sc, &m->sc->err, m->label_count_override, m->label_count_dev, st));
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T * h, embed_fwd(tok, m->wb(0), m->x[0], T, h, V, m->cfg.emb_scale, st));
  for (int l = 0; l < L; ++l) {
    ft_status s = layer_forward(m, l, m->acts[m->cfg.recompute ? 0 : l], B, S);
    if (s) return s;
  }
  const bool tied = m->cfg.tie_embeddings != 0;
  const int i_normf = 1 + m->per_layer() * L, i_head = tied ? 0 : i_normf + 1;  // tied: the head reads (and adds its gradient to) the table
  FT_LAUNCH(FT_PROF_NORM, 4.0 * T * h, rmsnorm_fwd(m->x[L], m->wb(i_normf), m->hF, m->rF, T, h, m->cfg.rms_eps, st));

  {
    ft_status sh = head_pass(m, m->hF, lab, m->ce_lse, m->d_hF, m->sc, m->cfg.logit_scale, i_head, T, with_bwd, false,
                             !tied && !m->cfg.mtp);
    if (sh) return sh;
  }
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 4.0 * T, reduce_loss(m->loss_row, T, m->sc, st));
  if (m->cfg.mtp) {
    ft_status sm = mtp_forward_and_head(m, tok, lab, B, S, i_head, with_bwd);
    if (sm) return sm;
  }
  if (!with_bwd) return FT_OK;
  // bucket 0 is the untied head, complete here (after the MTP head's pass when there is one); then the MTP head's matrices
  const int dp_base = (tied ? 0 : 1) + (m->cfg.mtp ? 1 : 0);
  if (m->dp_mode && !tied) FT_CUDA(cudaEventRecord(m->dp_ev[0], st));

  if (m->cfg.mtp) {
    ft_status sm = mtp_backward(m, B, S, tied);
    if (sm) return sm;
    if ((sm = wait_wgrad(m, 0))) return sm;  // the projections' weight gradients still read dxA
    if (m->dp_mode) FT_CUDA(cudaEventRecord(m->dp_ev[dp_base - 1], st));
  }
  FT_LAUNCH(FT_PROF_NORM, 6.0 * T * h,
            rmsnorm_bwd(m->d_hF, m->x[L], m->rF, m->wb(i_normf), m->cfg.mtp ? m->mtp_d_xL : nullptr, m->dxA, norm_slot(m, i_normf), T, h, st));
  for (int l = L - 1; l >= 0; --l) {
    LayerActs& a = m->acts[m->cfg.recompute ? 0 : l];
    if (m->cfg.recompute) {
      // the weight gradients of the layer above read the one activation slot that the recomputation overwrites
      for (int k = 0; k < 4; ++k) { ft_status sw = wait_wgrad(m, k); if (sw) return sw; }
      // rerun the layer's forward from its saved input (same kernels, so the same bits as the first time);
      // its output lands in x[l+1], which nothing reads any more
      ft_status s = layer_forward(m, l, a, B, S);
      if (s) return s;
    }
    ft_status s = layer_backward(m, l, a, B, S);
    if (s) return s;
    if (m->dp_mode) FT_CUDA(cudaEventRecord(m->dp_ev[dp_base + (L - 1 - l)], st));
  }
  // every RMSNorm gain's gradient: block partials of all norms summed in one launch
  FT_LAUNCH(FT_PROF_NORM, 4.0 * m->n_norm_slots * (double)elementwise_blocks_for_norm(T) * h,
            colsum_many(m->norm_partial, m->norm_out, m->n_norm_slots, (size_t)elementwise_blocks_for_norm(m->maxT) * h, T, h, st));
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 2.0 * T * h + 4.0 * V * h, embed_bwd(tok, m->dxA, m->gr(0), m->keys, T, h, V, m->cfg.emb_scale, tied || m->cfg.mtp, st));
  for (int k = 0; k < 4; ++k) { ft_status sw = wait_wgrad(m, k); if (sw) return sw; }  // join the second stream
  if (m->dp_mode) {  // the embedding table and the gains (summed over the whole pass) are complete only now
    FT_CUDA(cudaEventRecord(m->dp_ev[dp_base + L], st));
    FT_CUDA(cudaEventRecord(m->dp_ev[dp_base + L + 1], st));
  }
  m->overlapping = false;
  m->have_bwd = !m->fusing;  // a fusing step leaves no gradients of the matrices behind
  return FT_OK;
}

ft_status run_update(ft_model* m) {
  cudaStream_t st = m->stream;
  const AdamHyper hp = hyper(m);
  if (hp.max_grad_norm > 0.f) {
    FT_LAUNCH(FT_PROF_OPTIMIZER, 4.0 * m->arena, grad_norm_and_clip(m->grad, m->arena, m->sq_partial, m->sc, hp, st));
    FT_LAUNCH(FT_PROF_OPTIMIZER, 0.0, advance_step(m->sc, hp, st));
    FT_LAUNCH(FT_PROF_OPTIMIZER, 30.0 * m->arena,
              adamw(m->master, m->adam_m, m->adam_v, m->grad, m->pbf, m->arena, m->n_decay, m->sc, hp, st));
  } else {
    // no clipping: the update does not wait for the norm, which is summed in the same pass over the gradients
    FT_LAUNCH(FT_PROF_OPTIMIZER, 0.0, advance_step(m->sc, hp, st));
    FT_LAUNCH(FT_PROF_OPTIMIZER, 30.0 * m->arena,
              adamw_with_norm(m->master, m->adam_m, m->adam_v, m->grad, m->pbf, m->arena, m->n_decay, m->sq_partial,
                              m->sc, hp, st));
  }
  return FT_OK;
}

// What is left of the update after a fusing backward: the embedding table and the gains (their gradients do not
// come from a GEMM), and the gradient norm from all partial sums in slot order.
ft_status run_update_rest(ft_model* m) {
  cudaStream_t st = m->stream;
  const AdamHyper hp = hyper(m);
  const size_t fused_slots = (size_t)m->n_fused() * kAdamFuseSlots;
  const size_t embed_span = (m->params[0].numel() + 127) / 128 * 128;  // embed is the first tensor of the arenas
  FT_LAUNCH(FT_PROF_OPTIMIZER, 30.0 * embed_span,
            adamw_range_with_norm(m->master, m->adam_m, m->adam_v, m->grad, m->pbf, embed_span, embed_span,
                                  m->fuse_sq + fused_slots, m->sc, hp, st));
  const size_t g0 = m->n_decay, gn = m->arena - m->n_decay;
  FT_LAUNCH(FT_PROF_OPTIMIZER, 30.0 * gn,
            adamw_range_with_norm(m->master + g0, m->adam_m + g0, m->adam_v + g0, m->grad + g0, m->pbf + g0, gn, 0,
                                  m->fuse_sq + fused_slots + kSqnormBlocks, m->sc, hp, st));
  FT_LAUNCH(FT_PROF_OPTIMIZER, 4.0 * m->fuse_sq_count(), sqnorm_final(m->fuse_sq, (int)m->fuse_sq_count(), m->sc, hp, st));
  m->fusing = false;
  return FT_OK;
}

// A wait that nothing ends: one thread waits, with the kernels' own bounded wait, on an mbarrier that gets no arrival.
__global__ void wait_probe_kernel(long long limit_cycles, int* err) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0u, &abort_flag, err, limit_cycles, 0x61);
  __syncthreads();
}

// a non-zero device status word as a status code
ft_status device_status(ft_model* m, int err) {
  if ((err & 0xff) == (int)ERR_BAD_INDEX) return fail(m, FT_EINVAL, "a token id or label is outside [0, vocab) (ids were clamped, such labels ignored)");
  char msg[96];
  snprintf(msg, sizeof(msg), "a device-side wait ran out of time (status word 0x%x: wait site 0x%x)", (unsigned)err, (unsigned)err >> 8);
  return fail(m, FT_ETIMEOUT, msg);
}

// one synchronisation: reads the scalars back and turns device-side flags into a status
ft_status finish(ft_model* m, float* host_loss, float* host_gnorm) {
  StepScalars hs;
  FT_CUDA(cudaMemcpyAsync(&hs, m->sc, sizeof(hs), cudaMemcpyDeviceToHost, m->stream));
  FT_CUDA(cudaStreamSynchronize(m->stream));
  if (host_loss) *host_loss = hs.loss;
  if (host_gnorm) *host_gnorm = hs.gnorm;
  if (hs.err != 0) {
    FT_CUDA(cudaMemsetAsync(&m->sc->err, 0, sizeof(int), m->stream));
    return device_status(m, hs.err);
  }
  if (hs.nonfinite) return fail(m, FT_ENONFINITE, "loss is not finite");
  return FT_OK;
}

// Host <-> device copy ordered on the model's stream and finished on return.  (A plain cudaMemcpy from pageable host
// memory may return while the DMA is still in flight, and is only ordered against the legacy default stream.)
cudaError_t copy_sync(ft_model* m, void* dst, const void* src, size_t bytes, cudaMemcpyKind kind) {
  cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, m->stream);
  if (e != cudaSuccess) return e;
  return cudaStreamSynchronize(m->stream);
}

// wgu rows: logical (gate 0..f-1, up 0..f-1) <-> physical (16 gate rows, 16 up rows, alternating)
inline int64_t wgu_phys_row(int64_t r, int64_t f) {
  const int64_t i = r < f ? r : r - f;
  return (i / 16) * 32 + (r < f ? 0 : 16) + i % 16;
}

size_t kind_elem_size(ft_kind k) { return k == FT_COMPUTE_BF16 ? 2 : 4; }
void* kind_base(ft_model* m, ft_kind k) {
  switch (k) {
    case FT_MASTER_F32: return m->master;
    case FT_COMPUTE_BF16: return m->pbf;
    case FT_ADAM_M_F32: return m->adam_m;
    case FT_ADAM_V_F32: return m->adam_v;
    case FT_GRAD_F32: return m->grad;
  }
  return nullptr;
}

// Arena range [off, off + n) as an offset into the state arrays (master, moments).  Unsharded: the same offset.  Sharded:
// the range must lie inside this rank's slice of ONE bucket; -1 otherwise.
long long state_offset(const ft_model* m, size_t off, size_t n) {
  if (!m->sharded()) return (long long)off;
  for (const auto& b : m->dp_buckets) {
    if (off < b.offset || off >= b.offset + b.count) continue;
    const size_t per = b.count / (size_t)m->dp_world, lo = b.offset + (size_t)m->dp_rank * per;
    if (off < lo || off + n > lo + per) return -1;
    return (long long)(b.offset / (size_t)m->dp_world + (off - lo));
  }
  return -1;
}

// The part of arena range [off, off + n) (inside one bucket) that this rank's state shard holds: [*lo, *hi), may be empty.
void owned_part(const ft_model* m, size_t off, size_t n, size_t* lo, size_t* hi) {
  *lo = off; *hi = off + n;
  if (!m->sharded()) return;
  for (const auto& b : m->dp_buckets) {
    if (off < b.offset || off >= b.offset + b.count) continue;
    const size_t per = b.count / (size_t)m->dp_world, s0 = b.offset + (size_t)m->dp_rank * per, s1 = s0 + per;
    *lo = off > s0 ? off : s0;
    *hi = off + n < s1 ? off + n : s1;
    if (*hi < *lo) *hi = *lo;
    return;
  }
  *hi = *lo;
}

void dp_build_buckets(ft_model* m) {
  if (!m->dp_buckets.empty()) return;
  const int L = m->L, per = m->per_layer();
  auto span = [&](int first, int last) {  // arena range of the matrices first..last (consecutive in the arena)
    ft_model::DpBucket b;
    b.offset = m->params[first].offset;
    b.count = m->params[last].offset + align_up(m->params[last].numel(), 128) - b.offset;
    return b;
  };
  if (!m->cfg.tie_embeddings) { const int ih = 1 + per * L + 1; m->dp_buckets.push_back(span(ih, ih)); }
  // the MTP head's matrices (two projections, then its layer's four: consecutive in the arena) are complete before the
  // backbone's backward pass starts
  if (m->cfg.mtp) m->dp_buckets.push_back(span(m->i_mtp + 2, m->i_mtp + 4 + 5));
  for (int l = L - 1; l >= 0; --l) {
    // a layer's matrices in parameter order: wqkv, wo, wgu, wd (the gains between them live in the gains region)
    m->dp_buckets.push_back(span(m->idx_layer(l, 1), m->idx_layer(l, 5)));
  }
  m->dp_buckets.push_back(span(0, 0));
  ft_model::DpBucket g; g.offset = m->n_decay; g.count = m->arena - m->n_decay;
  m->dp_buckets.push_back(g);
}

}  // namespace

// =============================================================================== C ABI
extern "C" {

size_t ft_workspace_bytes(const ft_config* cfg) {
  if (!valid_config(cfg, nullptr)) return 0;
  ft_model tmp;
  tmp.cfg = *cfg;
  normalise(tmp.cfg);
  return carve(&tmp, nullptr);
}

// RoPE tables: mscale * cos/sin of angle(p, i) = p * theta^(-2i/d) / factors[i], evaluated in double on the host, stored
// as fp32 [max_seq, d/2].  factors == nullptr: all 1.
static ft_status build_rope_tables(ft_model* m, const float* factors, float mscale) {
  const ft_config* cfg = &m->cfg;
  cudaStream_t st = m->stream;
  const int half = m->d / 2;
  std::vector<float> cs((size_t)cfg->max_seq * half), sn((size_t)cfg->max_seq * half);
  for (int i = 0; i < half; ++i) {
    double inv = pow((double)cfg->rope_theta, -2.0 * i / (double)m->d);
    if (factors) inv /= (double)factors[i];
    for (int p = 0; p < cfg->max_seq; ++p) {
      const double ang = (double)p * inv;
      cs[(size_t)p * half + i] = (float)((double)mscale * cos(ang));
      sn[(size_t)p * half + i] = (float)((double)mscale * sin(ang));
    }
  }
  std::vector<float> csT(cs.size()), snT(sn.size());
  for (int i = 0; i < half; ++i)
    for (int p = 0; p < cfg->max_seq; ++p) {
      csT[(size_t)i * cfg->max_seq + p] = cs[(size_t)p * half + i];
      snT[(size_t)i * cfg->max_seq + p] = sn[(size_t)p * half + i];
    }
  FT_CUDA(cudaMemcpyAsync(m->rope_cos, cs.data(), cs.size() * sizeof(float), cudaMemcpyHostToDevice, st));
  FT_CUDA(cudaMemcpyAsync(m->rope_sin, sn.data(), sn.size() * sizeof(float), cudaMemcpyHostToDevice, st));
  FT_CUDA(cudaMemcpyAsync(m->rope_cosT, csT.data(), csT.size() * sizeof(float), cudaMemcpyHostToDevice, st));
  FT_CUDA(cudaMemcpyAsync(m->rope_sinT, snT.data(), snT.size() * sizeof(float), cudaMemcpyHostToDevice, st));
  FT_CUDA(cudaStreamSynchronize(st));
  m->rope_mscale = mscale;
  return FT_OK;
}

ft_status ft_init_model(const ft_config* cfg, uint64_t seed, void* dev_workspace, size_t bytes, void* cuda_stream,
                        ft_model** out) {
  if (!out) return FT_EINVAL;
  *out = nullptr;
  std::string why;
  if (!valid_config(cfg, &why)) return FT_EINVAL;
  if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) & (kAlign - 1))) return FT_EINVAL;
  ft_model* m = new ft_model();
  m->cfg = *cfg;
  normalise(m->cfg);
  m->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t need = carve(m, reinterpret_cast<uint8_t*>(dev_workspace));
  if (bytes < need) { delete m; return FT_ENOMEM; }
  *out = m;  // from here on errors are reported through the handle
  cudaStream_t st = m->stream;
  int dev = 0, major = 0;
  FT_CUDA(cudaGetDevice(&dev));
  FT_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) return fail(m, FT_ECUDA, "this library needs an sm_100 device");
  FT_CUDA(cudaStreamCreateWithFlags(&m->side, cudaStreamNonBlocking));
  FT_CUDA(cudaEventCreateWithFlags(&m->ev_d, cudaEventDisableTiming));
  for (int k = 0; k < 4; ++k) FT_CUDA(cudaEventCreateWithFlags(&m->ev_w[k], cudaEventDisableTiming));

  FT_CUDA(cudaMemsetAsync(m->adam_m, 0, m->state_elems * sizeof(float), st));
  FT_CUDA(cudaMemsetAsync(m->adam_v, 0, m->state_elems * sizeof(float), st));
  FT_CUDA(cudaMemsetAsync(m->grad, 0, m->arena * sizeof(float), st));
  FT_CUDA(cudaMemsetAsync(m->master, 0, m->state_elems * sizeof(float), st));
  // With a sharded state the full set of initial masters exists only for a moment, in the gradient arena (free at this
  // point): the bf16 copy is cast from it and every bucket's owned slice is copied into the master shard.
  float* full = m->sharded() ? m->grad : m->master;
  FT_CUDA(cudaMemsetAsync(m->sc, 0, sizeof(StepScalars), st));
  FT_CUDA(cudaMemsetAsync(m->splitk, 0, 1024, st));  // the GEMM scratch's arrival counters start at zero
  FT_CUDA(cudaMemsetAsync(m->splitk2, 0, 1024, st));
  for (size_t i = 0; i < m->params.size(); ++i) {
    const ParamInfo& p = m->params[i];
    if (p.cols) {
      // element e of the LOGICAL tensor i gets draw (seed, i, e); wgu's rows are written at their physical places
      FT_LAUNCH(FT_PROF_ELEMENTWISE, 0.0,
                init_normal(full + p.offset, p.numel(), seed, (int)i, 0.02, p.is_wgu ? (int)p.cols : 0, m->f, st));
    } else {
      FT_LAUNCH(FT_PROF_ELEMENTWISE, 0.0, fill_f32(full + p.offset, p.numel(), 1.0f, st));
    }
  }
  FT_LAUNCH(FT_PROF_ELEMENTWISE, 0.0, cast_bf16(full, m->pbf, m->arena, st));
  if (m->sharded()) {
    for (const auto& b : m->dp_buckets) {
      size_t lo, hi;
      owned_part(m, b.offset, b.count, &lo, &hi);
      FT_CUDA(cudaMemcpyAsync(m->master + state_offset(m, lo, hi - lo), full + lo, (hi - lo) * sizeof(float),
                              cudaMemcpyDeviceToDevice, st));
    }
    FT_CUDA(cudaMemsetAsync(m->grad, 0, m->arena * sizeof(float), st));
  }

  {
    std::vector<float*> outs((size_t)m->n_norm_slots, nullptr);
    for (size_t i = 0; i < m->params.size(); ++i)
      if (m->norm_slot_of[i] >= 0) outs[(size_t)m->norm_slot_of[i]] = m->gr((int)i);
    FT_CUDA(cudaMemcpyAsync(m->norm_out, outs.data(), outs.size() * sizeof(float*), cudaMemcpyHostToDevice, st));
    FT_CUDA(cudaStreamSynchronize(st));
  }
  {
    ft_status sr = build_rope_tables(m, nullptr, 1.0f);
    if (sr) return sr;
  }
  return FT_OK;
}

// One full step enqueued launch by launch.
static ft_status step_direct(ft_model* m, const int32_t* tok, const int32_t* lab, int32_t B, int32_t S) {
  if (m->sharded()) return fail(m, FT_EINVAL, "a model with a sharded optimizer state (dp_world > 1) steps through the ft_dp_* calls");
  const bool fuse = m->fused_update && m->cfg.max_grad_norm <= 0.f && !m->cfg.debug_taps;
  ft_status s = run_forward_backward(m, tok, lab, B, S, true, fuse);
  if (s) return s;
  return fuse ? run_update_rest(m) : run_update(m);
}

// The same step through a captured graph when that is enabled and possible.  The graph reads the token and label
// ids from the model's own buffers (the caller's pointers may change from step to step), every other address in
// it is fixed, and the optimizer scalars it needs live in device memory, so a replay needs no host value.
static ft_status step_maybe_graphed(ft_model* m, const int32_t* tok, const int32_t* lab, int32_t B, int32_t S) {
  if (!m->graph_enabled || m->prof || m->cfg.debug_taps) return step_direct(m, tok, lab, B, S);
  if (B < 1 || S < 1 || B > m->cfg.max_batch || S > m->cfg.max_seq) return fail(m, FT_EINVAL, "B or S out of range");
  if (!tok || !lab) return fail(m, FT_EINVAL, "null argument");
  if (!(m->graph_exec && m->graph_B == B && m->graph_S == S)) {
    if (!(m->warm_B == B && m->warm_S == S)) {  // first step of this shape: plain launches (one-time kernel set-up)
      m->warm_B = B; m->warm_S = S;
      return step_direct(m, tok, lab, B, S);
    }
    if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }
    if (cudaStreamBeginCapture(m->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();          // e.g. the legacy default stream cannot be captured: keep working without a graph
      m->graph_enabled = false;
      return step_direct(m, tok, lab, B, S);
    }
    const int64_t before = m->launches;
    ft_status s = step_direct(m, m->tok_dev, m->lab_dev, B, S);
    cudaGraph_t graph = nullptr;
    cudaError_t e = cudaStreamEndCapture(m->stream, &graph);
    m->graph_launches = m->launches - before;
    m->launches = before;  // nothing ran yet
    if (s != FT_OK || e != cudaSuccess || !graph) {
      if (graph) cudaGraphDestroy(graph);
      cudaGetLastError();
      m->graph_enabled = false;
      if (s != FT_OK) return s;
      return step_direct(m, tok, lab, B, S);
    }
    e = cudaGraphInstantiate(&m->graph_exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) {
      m->graph_exec = nullptr;
      m->graph_enabled = false;
      return step_direct(m, tok, lab, B, S);
    }
    m->graph_B = B; m->graph_S = S;
  }
  const size_t bytes = (size_t)B * S * sizeof(int32_t);
  if (tok != m->tok_dev) FT_CUDA(cudaMemcpyAsync(m->tok_dev, tok, bytes, cudaMemcpyDeviceToDevice, m->stream));
  if (lab != m->lab_dev) FT_CUDA(cudaMemcpyAsync(m->lab_dev, lab, bytes, cudaMemcpyDeviceToDevice, m->stream));
  FT_CUDA(cudaGraphLaunch(m->graph_exec, m->stream));
  m->launches += m->graph_launches;
  m->graph_replays += 1;
  m->lastB = B; m->lastS = S;
  m->have_bwd = !(m->fused_update && m->cfg.max_grad_norm <= 0.f);  // a fusing step leaves no matrix gradients behind
  return FT_OK;
}

ft_status ft_train_step(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S,
                        float* host_loss, float* host_gnorm) {
  if (!m) return FT_EINVAL;
  ft_status s = step_maybe_graphed(m, dev_tokens, dev_labels, B, S);
  if (s) return s;
  if (host_loss || host_gnorm) return finish(m, host_loss, host_gnorm);
  return FT_OK;
}

ft_status ft_set_rope_scaling(ft_model* m, const float* host_factors, float mscale) {
  if (!m) return FT_EINVAL;
  if (!(mscale > 0.f)) return fail(m, FT_EINVAL, "mscale must be positive");
  if (host_factors)
    for (int i = 0; i < m->d / 2; ++i)
      if (!(host_factors[i] > 0.f)) return fail(m, FT_EINVAL, "rescale factors must be positive");
  return build_rope_tables(m, host_factors, mscale);  // same device addresses: a captured graph stays valid
}

ft_status ft_set_overlap(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->overlap = enable != 0;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // captured with the old setting
  return FT_OK;
}

ft_status ft_set_attention_stored_ds(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->attn_ds_on = enable != 0;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // captured with the old setting
  return FT_OK;
}

ft_status ft_set_streaming_ce(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->streaming_ce = enable != 0;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // captured with the old setting
  return FT_OK;
}

ft_status ft_set_fused_swiglu_bwd(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->fused_swiglu_bwd = enable != 0;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // captured with the old setting
  return FT_OK;
}

ft_status ft_set_fused_update(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->fused_update = enable != 0;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // captured with the old setting
  return FT_OK;
}

ft_status ft_set_graph(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  m->graph_enabled = enable != 0;
  if (!enable && m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }
  return FT_OK;
}

int64_t ft_graph_replays(const ft_model* m) { return m ? m->graph_replays : 0; }

ft_status ft_train_step_host(ft_model* m, const int32_t* host_tokens, const int32_t* host_labels, int32_t B, int32_t S,
                             float* host_loss, float* host_gnorm) {
  if (!m || !host_tokens || !host_labels) return fail(m, FT_EINVAL, "null argument");
  if (B < 1 || S < 1 || B > m->cfg.max_batch || S > m->cfg.max_seq) return fail(m, FT_EINVAL, "B or S out of range");
  const size_t bytes = (size_t)B * S * sizeof(int32_t);
  FT_CUDA(cudaMemcpyAsync(m->tok_dev, host_tokens, bytes, cudaMemcpyHostToDevice, m->stream));
  FT_CUDA(cudaMemcpyAsync(m->lab_dev, host_labels, bytes, cudaMemcpyHostToDevice, m->stream));
  float loss = 0.f;
  ft_status s = ft_train_step(m, m->tok_dev, m->lab_dev, B, S, &loss, host_gnorm);
  if (host_loss) *host_loss = loss;
  return s;
}

ft_status ft_submit_step_host(ft_model* m, const int32_t* host_tokens, const int32_t* host_labels, int32_t B, int32_t S) {
  if (!m || !host_tokens || !host_labels) return fail(m, FT_EINVAL, "null argument");
  if (B < 1 || S < 1 || B > m->cfg.max_batch || S > m->cfg.max_seq) return fail(m, FT_EINVAL, "B or S out of range");
  if (m->ring_head - m->ring_tail >= FT_MAX_IN_FLIGHT) return fail(m, FT_EINVAL, "too many steps in flight: collect one first");
  if (!m->ring) {
    FT_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&m->ring), FT_MAX_IN_FLIGHT * sizeof(StepScalars), cudaHostAllocDefault));
    for (auto& e : m->ring_ev) FT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  }
  const size_t bytes = (size_t)B * S * sizeof(int32_t);
  FT_CUDA(cudaMemcpyAsync(m->tok_dev, host_tokens, bytes, cudaMemcpyHostToDevice, m->stream));
  FT_CUDA(cudaMemcpyAsync(m->lab_dev, host_labels, bytes, cudaMemcpyHostToDevice, m->stream));
  ft_status s = step_maybe_graphed(m, m->tok_dev, m->lab_dev, B, S);
  if (s) return s;
  const unsigned slot = m->ring_head % FT_MAX_IN_FLIGHT;
  FT_CUDA(cudaMemcpyAsync(&m->ring[slot], m->sc, sizeof(StepScalars), cudaMemcpyDeviceToHost, m->stream));
  FT_CUDA(cudaEventRecord(m->ring_ev[slot], m->stream));
  ++m->ring_head;
  return FT_OK;
}

ft_status ft_collect_step(ft_model* m, float* host_loss, float* host_gnorm) {
  if (!m) return FT_EINVAL;
  if (m->ring_head == m->ring_tail) return fail(m, FT_ENOTFOUND, "no step in flight");
  const unsigned slot = m->ring_tail % FT_MAX_IN_FLIGHT;
  FT_CUDA(cudaEventSynchronize(m->ring_ev[slot]));
  ++m->ring_tail;
  const StepScalars hs = m->ring[slot];
  if (host_loss) *host_loss = hs.loss;
  if (host_gnorm) *host_gnorm = hs.gnorm;
  if (hs.err != 0) {
    FT_CUDA(cudaMemsetAsync(&m->sc->err, 0, sizeof(int), m->stream));
    return device_status(m, hs.err);
  }
  if (hs.nonfinite) return fail(m, FT_ENONFINITE, "loss is not finite");
  return FT_OK;
}

// ---------------------------------------------------------------- data-parallel hooks

int32_t ft_dp_num_buckets(ft_model* m) {
  if (!m) return 0;
  dp_build_buckets(m);
  return (int32_t)m->dp_buckets.size();
}

ft_status ft_dp_bucket(ft_model* m, int32_t i, int64_t* offset, int64_t* count) {
  if (!m || !offset || !count) return FT_EINVAL;
  dp_build_buckets(m);
  if (i < 0 || i >= (int32_t)m->dp_buckets.size()) return FT_ENOTFOUND;
  *offset = (int64_t)m->dp_buckets[i].offset;
  *count = (int64_t)m->dp_buckets[i].count;
  return FT_OK;
}

ft_status ft_arena_ptr(ft_model* m, ft_kind kind, void** dev_ptr, int64_t* numel) {
  if (!m || !dev_ptr || !numel) return FT_EINVAL;
  void* b = kind_base(m, kind);
  if (!b) return FT_EINVAL;
  *dev_ptr = b;
  const bool state = kind == FT_MASTER_F32 || kind == FT_ADAM_M_F32 || kind == FT_ADAM_V_F32;
  *numel = (int64_t)(state ? m->state_elems : m->arena);
  return FT_OK;
}

ft_status ft_dp_scratch(ft_model* m, float** dev_ptr) {
  if (!m || !dev_ptr) return FT_EINVAL;
  *dev_ptr = m->dp_sq;
  return FT_OK;
}

ft_status ft_dp_set_label_count(ft_model* m, int64_t total_count) {
  if (!m || total_count < 0) return FT_EINVAL;
  m->label_count_override = total_count;
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // the count is a launch argument
  return FT_OK;
}

ft_status ft_dp_set_label_count_device(ft_model* m, const int64_t* dev_total_count) {
  if (!m) return FT_EINVAL;
  m->label_count_dev = reinterpret_cast<const long long*>(dev_total_count);
  if (m->graph_exec) { cudaGraphExecDestroy(m->graph_exec); m->graph_exec = nullptr; }  // the pointer is a launch argument
  return FT_OK;
}

ft_status ft_dp_backward(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S) {
  if (!m) return FT_EINVAL;
  if (m->cfg.debug_taps) return fail(m, FT_EINVAL, "data-parallel hooks are not available with debug_taps");
  dp_build_buckets(m);
  if (m->dp_ev.empty()) {
    m->dp_ev.assign(m->dp_buckets.size(), nullptr);
    for (auto& e : m->dp_ev) FT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  }
  m->dp_mode = true;
  ft_status s = run_forward_backward(m, dev_tokens, dev_labels, B, S, true, false);
  m->dp_mode = false;
  return s;
}

ft_status ft_dp_stream_wait_bucket(ft_model* m, int32_t i, void* stream) {
  if (!m || i < 0 || i >= (int32_t)m->dp_ev.size() || !m->dp_ev[i]) return FT_EINVAL;
  FT_CUDA(cudaStreamWaitEvent(reinterpret_cast<cudaStream_t>(stream), m->dp_ev[i], 0));
  return FT_OK;
}

namespace {
bool dp_range_ok(const ft_model* m, int64_t offset, int64_t count) {
  return offset >= 0 && count > 0 && (offset & 3) == 0 && (count & 3) == 0 && (size_t)(offset + count) <= m->arena;
}
}  // namespace

ft_status ft_dp_sqnorm(ft_model* m, int64_t offset, int64_t count, float* dev_out, void* stream) {
  if (!m || !dev_out || !dp_range_ok(m, offset, count)) return FT_EINVAL;
  if (sqnorm_to(m->grad + offset, (size_t)count, m->sq_partial, dev_out, reinterpret_cast<cudaStream_t>(stream)) < 0) return FT_ECUDA;
  return FT_OK;
}

ft_status ft_dp_begin_update(ft_model* m, const float* dev_sq_total, void* stream) {
  if (!m) return FT_EINVAL;
  const AdamHyper hp = hyper(m);
  if (!dev_sq_total && hp.max_grad_norm > 0.f) return fail(m, FT_EINVAL, "clipping needs the global sum of squares first");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (advance_step(m->sc, hp, st) < 0) return FT_ECUDA;
  if (!dev_sq_total) {
    FT_CUDA(cudaMemsetAsync(m->dp_sq + 3, 0, sizeof(float), st));
    dev_sq_total = m->dp_sq + 3;  // coefficient 1; the norm is reported later (ft_dp_set_norm)
  }
  if (clip_from_sq(dev_sq_total, m->sc, hp, st) < 0) return FT_ECUDA;
  return FT_OK;
}

ft_status ft_dp_set_norm(ft_model* m, const float* dev_sq_total, void* stream) {
  if (!m || !dev_sq_total) return FT_EINVAL;
  if (clip_from_sq(dev_sq_total, m->sc, hyper(m), reinterpret_cast<cudaStream_t>(stream)) < 0) return FT_ECUDA;
  return FT_OK;
}

ft_status ft_dp_update_range(ft_model* m, int64_t offset, int64_t count, void* stream) {
  if (!m || !dp_range_ok(m, offset, count)) return FT_EINVAL;
  const size_t off = (size_t)offset, n = (size_t)count;
  const size_t n_decay = m->n_decay > off ? (m->n_decay - off < n ? m->n_decay - off : n) : 0;
  const long long so = state_offset(m, off, n);
  if (so < 0) return fail(m, FT_EINVAL, "sharded state: the range must lie inside this rank's slice of one bucket");
  if (adamw(m->master + so, m->adam_m + so, m->adam_v + so, m->grad + off, m->pbf + off, n, n_decay, m->sc, hyper(m),
            reinterpret_cast<cudaStream_t>(stream)) < 0)
    return FT_ECUDA;
  m->have_bwd = false;
  return FT_OK;
}

ft_status ft_dp_collect(ft_model* m, float* host_loss, float* host_gnorm) {
  if (!m) return FT_EINVAL;
  return finish(m, host_loss, host_gnorm);
}

ft_status ft_forward_loss(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S,
                          float* host_loss) {
  if (!m) return FT_EINVAL;
  ft_status s = run_forward_backward(m, dev_tokens, dev_labels, B, S, false);
  if (s) return s;
  return finish(m, host_loss, nullptr);
}

ft_status ft_forward_backward(ft_model* m, const int32_t* dev_tokens, const int32_t* dev_labels, int32_t B, int32_t S,
                              float* host_loss) {
  if (!m) return FT_EINVAL;
  ft_status s = run_forward_backward(m, dev_tokens, dev_labels, B, S, true);
  if (s) return s;
  return finish(m, host_loss, nullptr);
}

ft_status ft_apply_update(ft_model* m, float* host_gnorm) {
  if (!m) return FT_EINVAL;
  if (m->sharded()) return fail(m, FT_EINVAL, "a model with a sharded optimizer state (dp_world > 1) updates through ft_dp_update_range");
  ft_status s = run_update(m);
  if (s) return s;
  return finish(m, nullptr, host_gnorm);
}

int32_t ft_num_params(const ft_model* m) { return m ? (int32_t)m->params.size() : 0; }

ft_status ft_param_info(const ft_model* m, int32_t i, const char** name, int32_t* ndim, int64_t shape[2]) {
  if (!m || i < 0 || i >= (int32_t)m->params.size()) return FT_EINVAL;
  const ParamInfo& p = m->params[i];
  if (name) *name = p.name.c_str();
  if (ndim) *ndim = p.cols ? 2 : 1;
  if (shape) { shape[0] = p.rows; shape[1] = p.cols ? p.cols : 1; }
  return FT_OK;
}

static ft_status param_copy(ft_model* m, int32_t i, ft_kind kind, void* host, size_t bytes, bool to_host) {
  if (!m || !host) return fail(m, FT_EINVAL, "null argument");
  if (i < 0 || i >= (int32_t)m->params.size()) return fail(m, FT_EINVAL, "parameter index out of range");
  if ((int)kind < 0 || (int)kind > (int)FT_GRAD_F32) return fail(m, FT_EINVAL, "unknown kind");
  const ParamInfo& p = m->params[i];
  const size_t es = kind_elem_size(kind);
  if (bytes != p.numel() * es) return fail(m, FT_EINVAL, "byte count does not match the tensor");
  uint8_t* dev = reinterpret_cast<uint8_t*>(kind_base(m, kind)) + p.offset * es;
  uint8_t* hp = reinterpret_cast<uint8_t*>(host);
  FT_CUDA(cudaStreamSynchronize(m->stream));
  // Sharded state: masters and moments exist only for this rank's slices.  The tensor is staged, in its device layout, in
  // its span of the gradient arena (whose contents are lost): reading returns the owned elements and 0 elsewhere (so the
  // ranks' results add up to the whole tensor), writing stores the owned elements (every rank passes the whole tensor).
  const bool staged = m->sharded() && (kind == FT_MASTER_F32 || kind == FT_ADAM_M_F32 || kind == FT_ADAM_V_F32);
  const size_t span = align_up(p.numel(), 128);
  size_t own_lo = 0, own_hi = 0;
  if (staged) {
    float* stage = m->grad + p.offset;
    float* shard = reinterpret_cast<float*>(kind_base(m, kind));
    owned_part(m, p.offset, span, &own_lo, &own_hi);
    m->have_bwd = false;
    dev = reinterpret_cast<uint8_t*>(stage);
    if (to_host) {
      FT_CUDA(cudaMemsetAsync(stage, 0, span * sizeof(float), m->stream));
      if (own_hi > own_lo)
        FT_CUDA(cudaMemcpyAsync(stage + (own_lo - p.offset), shard + state_offset(m, own_lo, own_hi - own_lo),
                                (own_hi - own_lo) * sizeof(float), cudaMemcpyDeviceToDevice, m->stream));
      FT_CUDA(cudaStreamSynchronize(m->stream));
    }
  }
  if (!p.is_wgu) {
    if (to_host) FT_CUDA(copy_sync(m, hp, dev, bytes, cudaMemcpyDeviceToHost));
    else FT_CUDA(copy_sync(m, dev, hp, bytes, cudaMemcpyHostToDevice));
  } else {
    // 16-row blocks of the logical tensor sit at their physical (interleaved) place
    const size_t blk = 16 * (size_t)p.cols * es;
    for (int64_t r0 = 0; r0 < p.rows; r0 += 16) {
      uint8_t* d = dev + (size_t)wgu_phys_row(r0, m->f) * p.cols * es;
      uint8_t* hrow = hp + (size_t)r0 * p.cols * es;
      if (to_host) FT_CUDA(copy_sync(m, hrow, d, blk, cudaMemcpyDeviceToHost));
      else FT_CUDA(copy_sync(m, d, hrow, blk, cudaMemcpyHostToDevice));
    }
  }
  if (!to_host && kind == FT_MASTER_F32) {
    const float* src = staged ? m->grad + p.offset : m->master + p.offset;
    FT_LAUNCH(FT_PROF_ELEMENTWISE, 0.0, cast_bf16(src, m->pbf + p.offset, span, m->stream));
    FT_CUDA(cudaStreamSynchronize(m->stream));
  }
  if (staged && !to_host && own_hi > own_lo) {
    float* shard = reinterpret_cast<float*>(kind_base(m, kind));
    FT_CUDA(cudaMemcpyAsync(shard + state_offset(m, own_lo, own_hi - own_lo), m->grad + own_lo, (own_hi - own_lo) * sizeof(float),
                            cudaMemcpyDeviceToDevice, m->stream));
    FT_CUDA(cudaStreamSynchronize(m->stream));
  }
  return FT_OK;
}

ft_status ft_get_param(ft_model* m, int32_t i, ft_kind kind, void* host_dst, size_t bytes) {
  return param_copy(m, i, kind, host_dst, bytes, true);
}
ft_status ft_set_param(ft_model* m, int32_t i, ft_kind kind, const void* host_src, size_t bytes) {
  return param_copy(m, i, kind, const_cast<void*>(host_src), bytes, false);
}

ft_status ft_get_step(const ft_model* mc, int64_t* step) {
  ft_model* m = const_cast<ft_model*>(mc);
  if (!m || !step) return FT_EINVAL;
  long long s = 0;
  FT_CUDA(cudaStreamSynchronize(m->stream));
  FT_CUDA(copy_sync(m, &s, &m->sc->step, sizeof(s), cudaMemcpyDeviceToHost));
  *step = s;
  return FT_OK;
}

ft_status ft_set_step(ft_model* m, int64_t step) {
  if (!m || step < 0) return FT_EINVAL;
  long long s = step;
  FT_CUDA(cudaStreamSynchronize(m->stream));
  FT_CUDA(copy_sync(m, &m->sc->step, &s, sizeof(s), cudaMemcpyHostToDevice));
  return FT_OK;
}

ft_status ft_get_tap(ft_model* m, const char* name, int32_t layer, void* host_dst, size_t bytes, size_t* out_bytes,
                     int32_t* dtype) {
  if (!m || !name || !host_dst) return fail(m, FT_EINVAL, "null argument");
  if (m->lastB == 0) return fail(m, FT_ENOTFOUND, "no step has run yet");
  const size_t T = (size_t)m->lastB * m->lastS, h = m->h, f = m->f, hq = m->hq, nqkv = m->nqkv;
  const void* src = nullptr;
  size_t n = 0;
  int dt = 0;
  const std::string nm(name);
  if (layer < 0) {
    if (nm == "hF") { src = m->hF; n = T * h; }
    else if (nm == "ce_lse") { src = m->ce_lse; n = T; dt = 1; }
    else if (nm == "d_hF" && m->have_bwd) { src = m->d_hF; n = T * h; }
  } else if (layer < m->L) {
    const bool fwd_ok = !m->cfg.recompute;  // with recomputation only the layer inputs / outputs survive the step
    if (nm == "x_in") { src = m->x[layer]; n = T * h; }
    else if (nm == "x_out" && (!m->cfg.recompute || layer == m->L - 1 || !m->have_bwd)) { src = m->x[layer + 1]; n = T * h; }
    else if (fwd_ok) {
      const LayerActs& a = m->acts[layer];
      if (nm == "h1") { src = a.h1; n = T * h; }
      else if (nm == "qkv") { src = a.qkv; n = T * nqkv; }
      else if (nm == "attn_lse") { src = a.lse; n = T * m->cfg.n_heads; dt = 1; }
      else if (nm == "o") { src = a.o; n = T * hq; }
      else if (nm == "x_mid") { src = a.x_mid; n = T * h; }
      else if (nm == "h2") { src = a.h2; n = T * h; }
      else if (nm == "gu") { src = a.gu; n = T * 2 * f; }
      else if (nm == "a") { src = a.a; n = T * f; }
    }
    if (!src && m->cfg.debug_taps && m->have_bwd) {
      const LayerTaps& t = m->taps[layer];
      if (nm == "d_x_out") { src = t.d_x_out; n = T * h; }
      else if (nm == "d_a") { src = t.d_a; n = T * f; }
      else if (nm == "d_gu") { src = t.d_gu; n = T * 2 * f; }
      else if (nm == "d_h2") { src = t.d_h2; n = T * h; }
      else if (nm == "d_x_mid") { src = t.d_x_mid; n = T * h; }
      else if (nm == "d_o") { src = t.d_o; n = T * hq; }
      else if (nm == "d_qkv") { src = t.d_qkv; n = T * nqkv; }
      else if (nm == "d_h1") { src = t.d_h1; n = T * h; }
      else if (nm == "d_x_in") { src = t.d_x_in; n = T * h; }
    }
  }
  if (!src) return fail(m, FT_ENOTFOUND, "no such tap (or it was not kept in this mode)");
  const size_t nbytes = n * (dt ? 4 : 2);
  if (out_bytes) *out_bytes = nbytes;
  if (dtype) *dtype = dt;
  if (bytes < nbytes) return fail(m, FT_EINVAL, "destination too small");
  FT_CUDA(cudaStreamSynchronize(m->stream));
  FT_CUDA(copy_sync(m, host_dst, src, nbytes, cudaMemcpyDeviceToHost));
  if (nm == "d_gu") {
    // undo the physical interleave: [T, 2f] columns back to gate | up
    std::vector<uint16_t> tmp(2 * f);
    uint16_t* rows = reinterpret_cast<uint16_t*>(host_dst);
    for (size_t t = 0; t < T; ++t) {
      uint16_t* r = rows + t * 2 * f;
      for (size_t c = 0; c < 2 * f; ++c) tmp[c] = r[wgu_phys_row((int64_t)c, (int64_t)f)];
      memcpy(r, tmp.data(), 2 * f * sizeof(uint16_t));
    }
  }
  return FT_OK;
}

ft_status ft_set_profiling(ft_model* m, int32_t enable) {
  if (!m) return FT_EINVAL;
  FT_CUDA(cudaStreamSynchronize(m->stream));
  prof_collect(m);
  m->prof = enable != 0;
  if (enable) {
    for (int c = 0; c < FT_PROF_CLASSES; ++c) { m->prof_ms[c] = 0; m->prof_work[c] = 0; m->prof_launches[c] = 0; }
    m->prof_shapes.clear();
  }
  return FT_OK;
}

ft_status ft_get_profile(ft_model* m, int32_t cls, double* ms, double* work, int64_t* launches) {
  if (!m || cls < 0 || cls >= FT_PROF_CLASSES) return FT_EINVAL;
  FT_CUDA(cudaStreamSynchronize(m->stream));
  prof_collect(m);
  if (ms) *ms = m->prof_ms[cls];
  if (work) *work = m->prof_work[cls];
  if (launches) *launches = m->prof_launches[cls];
  return FT_OK;
}

void ft_debug_gemm_tile(int32_t bn) { g_gemm_force_bn = bn; }
void ft_debug_gemm_balanced(int32_t on) { g_gemm_balanced = on; }
void ft_debug_gemm_group(int32_t on) { g_gemm_group = on; }
void ft_debug_gemm_tma_out(int32_t on) { g_gemm_tma_out = on; }
void ft_debug_gemm_swiglu_tma(int32_t on) { g_gemm_swiglu_tma = on; }
void ft_debug_pdl(int32_t on) { g_pdl = on; }
void ft_debug_gemm_pairs(int32_t on) { g_gemm_pairs = on; }
void ft_debug_head_dz_limit(uint64_t bytes) { g_head_dz_limit = (size_t)bytes; }

ft_status ft_debug_wait_probe(ft_model* m, int64_t limit_cycles) {
  if (!m) return FT_EINVAL;
  if (limit_cycles < 1 || limit_cycles > 20000000) return fail(m, FT_EINVAL, "limit_cycles must be in [1, 20000000]");
  wait_probe_kernel<<<1, 32, 0, m->stream>>>((long long)limit_cycles, &m->sc->err);
  FT_CUDA(cudaGetLastError());
  m->launches += 1;
  return FT_OK;
}

ft_status ft_get_gemm_profile(ft_model* m, int32_t i, int32_t shape[8], double* ms, int64_t* launches) {
  if (!m || !shape) return FT_EINVAL;
  FT_CUDA(cudaStreamSynchronize(m->stream));
  prof_collect(m);
  if (i < 0 || i >= (int32_t)m->prof_shapes.size()) return FT_ENOTFOUND;
  const auto& s = m->prof_shapes[i];
  shape[0] = s.M; shape[1] = s.N; shape[2] = s.K; shape[3] = s.a_mn; shape[4] = s.b_mn; shape[5] = s.epi;
  shape[6] = s.M2; shape[7] = s.N2;
  if (ms) *ms = s.ms;
  if (launches) *launches = s.launches;
  return FT_OK;
}

const char* ft_last_error(const ft_model* m) { return m ? m->err.c_str() : "null model"; }
int64_t ft_launch_count(const ft_model* m) { return m ? m->launches : 0; }
void ft_destroy(ft_model* m) {
  if (!m) return;
  for (auto& r : m->prof_pending) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  for (auto e : m->prof_pool) cudaEventDestroy(e);
  if (m->graph_exec) cudaGraphExecDestroy(m->graph_exec);
  if (m->side) cudaStreamDestroy(m->side);
  if (m->ev_d) cudaEventDestroy(m->ev_d);
  for (auto e : m->ev_w) if (e) cudaEventDestroy(e);
  for (auto e : m->ring_ev) if (e) cudaEventDestroy(e);
  for (auto e : m->dp_ev) if (e) cudaEventDestroy(e);
  if (m->ring) cudaFreeHost(m->ring);
  delete m;
}

// ---------------------------------------------------------------- single kernels
ft_status ft_k_gemm(const void* dev_A, int32_t a_mn, int64_t lda, const void* dev_B, int32_t b_mn, int64_t ldb,
                    void* dev_C, int64_t ldc, const void* dev_resid, int32_t out_kind, int32_t M, int32_t N, int32_t K,
                    int32_t* dev_err, void* stream) {
  if (out_kind < 0 || out_kind > 3) return FT_EINVAL;
  GemmArgs g;
  g.A = reinterpret_cast<const bf16*>(dev_A); g.a_mn = a_mn; g.lda = lda;
  g.B = reinterpret_cast<const bf16*>(dev_B); g.b_mn = b_mn; g.ldb = ldb;
  g.C = dev_C; g.ldc = ldc; g.resid = reinterpret_cast<const bf16*>(dev_resid);
  g.epi = out_kind; g.M = M; g.N = N; g.K = K; g.err = dev_err;
  cudaError_t e = launch_gemm(g, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}

ft_status ft_k_gemm_ws(const void* dev_A, int32_t a_mn, int64_t lda, const void* dev_B, int32_t b_mn, int64_t ldb,
                       void* dev_C, int64_t ldc, const void* dev_resid, int32_t out_kind, int32_t M, int32_t N, int32_t K,
                       float* dev_scratch, uint64_t scratch_bytes, int32_t* dev_err, void* stream) {
  if (out_kind < 0 || out_kind > 3 || !dev_scratch) return FT_EINVAL;
  GemmArgs g;
  g.A = reinterpret_cast<const bf16*>(dev_A); g.a_mn = a_mn; g.lda = lda;
  g.B = reinterpret_cast<const bf16*>(dev_B); g.b_mn = b_mn; g.ldb = ldb;
  g.C = dev_C; g.ldc = ldc; g.resid = reinterpret_cast<const bf16*>(dev_resid);
  g.epi = out_kind; g.M = M; g.N = N; g.K = K; g.err = dev_err;
  g.scratch = dev_scratch; g.scratch_bytes = scratch_bytes; g.scratch_reset = true;
  cudaError_t e = launch_gemm(g, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}

ft_status ft_k_status(void* stream) {
  int* status = attention_status_word();
  if (!status) return FT_ECUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int v = 0;
  if (cudaMemcpyAsync(&v, status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return FT_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FT_ECUDA;
  if (v == 0) return FT_OK;
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return FT_ECUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return FT_ECUDA;
  return FT_ETIMEOUT;
}

ft_status ft_k_attention_fwd(const void* dev_qkv, void* dev_o, float* dev_lse, int32_t B, int32_t S, int32_t n_heads,
                             int32_t n_kv_heads, int32_t head_dim, void* stream) {
  if (!dev_qkv || !dev_o || !dev_lse) return FT_EINVAL;
  int* status = attention_status_word();
  if (!status) return FT_ECUDA;
  cudaError_t e = attention_fwd(reinterpret_cast<const bf16*>(dev_qkv), reinterpret_cast<bf16*>(dev_o), dev_lse, B, S,
                                n_heads, n_kv_heads, head_dim, status, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}

ft_status ft_k_attention_bwd(const void* dev_qkv, const void* dev_o, const void* dev_do, const float* dev_lse,
                             float* dev_delta, void* dev_dqkv, const float* dev_cos, const float* dev_sin, int32_t B,
                             int32_t S, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream) {
  if (!dev_qkv || !dev_o || !dev_do || !dev_lse || !dev_delta || !dev_dqkv) return FT_EINVAL;
  int* status = attention_status_word();
  if (!status) return FT_ECUDA;
  cudaError_t e = attention_bwd(reinterpret_cast<const bf16*>(dev_qkv), reinterpret_cast<const bf16*>(dev_o),
                                reinterpret_cast<const bf16*>(dev_do), dev_lse, dev_delta,
                                reinterpret_cast<bf16*>(dev_dqkv), dev_cos, dev_sin, B, S, n_heads, n_kv_heads, head_dim,
                                status, reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}

ft_status ft_k_attention_bwd_ws(const void* dev_qkv, const void* dev_o, const void* dev_do, const float* dev_lse,
                                float* dev_delta, void* dev_dqkv, const float* dev_cos, const float* dev_sin, void* dev_ds,
                                uint64_t ds_bytes, int32_t B, int32_t S, int32_t n_heads, int32_t n_kv_heads,
                                int32_t head_dim, void* stream) {
  if (!dev_qkv || !dev_o || !dev_do || !dev_lse || !dev_delta || !dev_dqkv) return FT_EINVAL;
  int* status = attention_status_word();
  if (!status) return FT_ECUDA;
  cudaError_t e = attention_bwd_ws(reinterpret_cast<const bf16*>(dev_qkv), reinterpret_cast<const bf16*>(dev_o),
                                   reinterpret_cast<const bf16*>(dev_do), dev_lse, dev_delta,
                                   reinterpret_cast<bf16*>(dev_dqkv), dev_cos, dev_sin, reinterpret_cast<bf16*>(dev_ds),
                                   (size_t)ds_bytes, B, S, n_heads, n_kv_heads, head_dim, status,
                                   reinterpret_cast<cudaStream_t>(stream));
  if (e == cudaErrorInvalidValue) return FT_EINVAL;
  return e == cudaSuccess ? FT_OK : FT_ECUDA;
}

}  // extern "C"
