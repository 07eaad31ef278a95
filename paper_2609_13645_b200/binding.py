"""ctypes binding of libforgestep.so: argument marshalling only.

Every step of the training path runs inside the CUDA library; PyTorch is used here for
device memory and the stream.  Loading fails loudly when the library has not been built:
there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Tuple

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libforgestep.so")
_lib = None

FT_OK, FT_EINVAL, FT_ENOMEM, FT_ECUDA, FT_ENONFINITE, FT_ETIMEOUT, FT_ENOTFOUND = range(7)
STATUS_NAMES = ["FT_OK", "FT_EINVAL", "FT_ENOMEM", "FT_ECUDA", "FT_ENONFINITE", "FT_ETIMEOUT", "FT_ENOTFOUND"]
KIND_MASTER, KIND_BF16, KIND_ADAM_M, KIND_ADAM_V, KIND_GRAD = range(5)
MAX_IN_FLIGHT = 2  # FT_MAX_IN_FLIGHT of the header
PROF_CLASSES = ["gemm", "attn_fwd", "attn_bwd", "norm", "elementwise", "ce", "optimizer"]


class FtConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab",
                                          "max_batch", "max_seq")] + \
               [(n, C.c_float) for n in ("rms_eps", "rope_theta", "lr", "beta1", "beta2", "adam_eps", "weight_decay",
                                         "max_grad_norm")] + \
               [("recompute", C.c_int32), ("debug_taps", C.c_int32)] + \
               [(n, C.c_float) for n in ("emb_scale", "resid_scale", "logit_scale")] + [("tie_embeddings", C.c_int32),
                                                                                         ("qk_norm", C.c_int32)] + \
               [("mtp", C.c_int32), ("mtp_weight", C.c_float), ("dp_world", C.c_int32), ("dp_rank", C.c_int32)]


class ForgeStepError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < 7 else status}: {msg}")
        self.status = status


def lib():
    """The loaded C-ABI library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_13645_b200.build`")
        L = C.CDLL(_LIB_PATH)
        vp, i32, i64, f32p, i32p = C.c_void_p, C.c_int32, C.c_int64, C.POINTER(C.c_float), C.POINTER(C.c_int32)
        cfgp = C.POINTER(FtConfig)
        L.ft_workspace_bytes.restype = C.c_size_t
        L.ft_workspace_bytes.argtypes = [cfgp]
        L.ft_init_model.argtypes = [cfgp, C.c_uint64, vp, C.c_size_t, vp, C.POINTER(vp)]
        L.ft_train_step.argtypes = [vp, vp, vp, i32, i32, f32p, f32p]
        L.ft_train_step_host.argtypes = [vp, vp, vp, i32, i32, f32p, f32p]
        L.ft_forward_loss.argtypes = [vp, vp, vp, i32, i32, f32p]
        L.ft_forward_backward.argtypes = [vp, vp, vp, i32, i32, f32p]
        L.ft_apply_update.argtypes = [vp, f32p]
        L.ft_num_params.restype = i32
        L.ft_num_params.argtypes = [vp]
        L.ft_param_info.argtypes = [vp, i32, C.POINTER(C.c_char_p), i32p, C.POINTER(i64)]
        L.ft_get_param.argtypes = [vp, i32, i32, vp, C.c_size_t]
        L.ft_set_param.argtypes = [vp, i32, i32, vp, C.c_size_t]
        L.ft_get_step.argtypes = [vp, C.POINTER(i64)]
        L.ft_set_step.argtypes = [vp, i64]
        L.ft_get_tap.argtypes = [vp, C.c_char_p, i32, vp, C.c_size_t, C.POINTER(C.c_size_t), i32p]
        L.ft_last_error.restype = C.c_char_p
        L.ft_last_error.argtypes = [vp]
        L.ft_launch_count.restype = i64
        L.ft_launch_count.argtypes = [vp]
        L.ft_set_profiling.argtypes = [vp, i32]
        L.ft_set_profiling.restype = C.c_int
        L.ft_get_profile.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(i64)]
        L.ft_get_profile.restype = C.c_int
        L.ft_debug_gemm_tile.argtypes = [i32]
        L.ft_debug_gemm_tile.restype = None
        L.ft_debug_gemm_pairs.argtypes = [i32]
        L.ft_debug_gemm_pairs.restype = None
        L.ft_debug_gemm_swiglu_tma.argtypes = [i32]
        L.ft_debug_gemm_swiglu_tma.restype = None
        L.ft_debug_gemm_group.argtypes = [i32]
        L.ft_debug_gemm_group.restype = None
        L.ft_debug_gemm_tma_out.argtypes = [i32]
        L.ft_debug_gemm_tma_out.restype = None
        L.ft_get_gemm_profile.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(C.c_double), C.POINTER(i64)]
        L.ft_get_gemm_profile.restype = C.c_int
        L.ft_set_fused_update.argtypes = [vp, i32]
        L.ft_set_fused_update.restype = C.c_int
        L.ft_set_rope_scaling.argtypes = [vp, vp, C.c_float]
        L.ft_set_rope_scaling.restype = C.c_int
        L.ft_set_overlap.argtypes = [vp, i32]
        L.ft_set_overlap.restype = C.c_int
        L.ft_submit_step_host.argtypes = [vp, vp, vp, i32, i32]
        L.ft_submit_step_host.restype = C.c_int
        L.ft_collect_step.argtypes = [vp, vp, vp]
        L.ft_collect_step.restype = C.c_int
        L.ft_set_streaming_ce.argtypes = [vp, i32]
        L.ft_set_streaming_ce.restype = C.c_int
        L.ft_set_attention_stored_ds.argtypes = [vp, i32]
        L.ft_set_attention_stored_ds.restype = C.c_int
        L.ft_set_fused_swiglu_bwd.argtypes = [vp, i32]
        L.ft_set_fused_swiglu_bwd.restype = C.c_int
        L.ft_set_graph.argtypes = [vp, i32]
        L.ft_set_graph.restype = C.c_int
        L.ft_graph_replays.argtypes = [vp]
        L.ft_graph_replays.restype = i64
        L.ft_destroy.restype = None
        L.ft_destroy.argtypes = [vp]
        L.ft_k_gemm.argtypes = [vp, i32, i64, vp, i32, i64, vp, i64, vp, i32, i32, i32, i32, vp, vp]
        L.ft_k_gemm_ws.argtypes = [vp, i32, i64, vp, i32, i64, vp, i64, vp, i32, i32, i32, i32, vp, C.c_uint64, vp, vp]
        L.ft_k_gemm_ws.restype = C.c_int
        L.ft_k_attention_fwd.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.ft_k_attention_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.ft_k_attention_bwd_ws.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_uint64, i32, i32, i32, i32, i32, vp]
        L.ft_k_attention_bwd_ws.restype = C.c_int
        L.ft_k_attention_bwd_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp]
        L.ft_k_attention_bwd_noalloc.restype = C.c_int
        for name in ("ft_init_model", "ft_train_step", "ft_train_step_host", "ft_forward_loss", "ft_forward_backward",
                     "ft_apply_update", "ft_param_info", "ft_get_param", "ft_set_param", "ft_get_step", "ft_set_step",
                     "ft_get_tap", "ft_k_gemm", "ft_k_attention_fwd", "ft_k_attention_bwd"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def make_config(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, max_batch, max_seq, rms_eps=1e-5,
                rope_theta=1e4, lr=1e-3, beta1=0.9, beta2=0.95, adam_eps=1e-8, weight_decay=0.1, max_grad_norm=0.0,
                recompute=0, debug_taps=0, emb_scale=1.0, resid_scale=1.0, logit_scale=1.0, tie_embeddings=0, qk_norm=0,
                mtp=0, mtp_weight=1.0, dp_world=0, dp_rank=0) -> FtConfig:
    return FtConfig(n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, max_batch, max_seq, rms_eps,
                    rope_theta, lr, beta1, beta2, adam_eps, weight_decay, max_grad_norm, recompute, debug_taps,
                    emb_scale, resid_scale, logit_scale, int(tie_embeddings), int(qk_norm), int(mtp), mtp_weight, int(dp_world),
                    int(dp_rank))


def workspace_bytes(cfg: FtConfig) -> int:
    return int(lib().ft_workspace_bytes(C.byref(cfg)))


def _stream_ptr():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32 values (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


class Model:
    """A decoder + optimizer state living in one torch-allocated workspace on the current CUDA device."""

    def __init__(self, cfg: FtConfig, seed: int = 1234):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("forgestep needs a CUDA device (sm_100a); there is no CPU path")
        self.cfg = cfg
        nbytes = workspace_bytes(cfg)
        if nbytes == 0:
            raise ForgeStepError(FT_EINVAL, "invalid config")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self._h = C.c_void_p()
        self._pending = []
        st = lib().ft_init_model(C.byref(cfg), C.c_uint64(seed), C.c_void_p(self.workspace.data_ptr()), nbytes,
                                 _stream_ptr(), C.byref(self._h))
        self._check(st)
        self.params: List[Tuple[str, Tuple[int, ...]]] = []
        for i in range(lib().ft_num_params(self._h)):
            name, nd, shp = C.c_char_p(), C.c_int32(), (C.c_int64 * 2)()
            self._check(lib().ft_param_info(self._h, i, C.byref(name), C.byref(nd), shp))
            self.params.append((name.value.decode(), (int(shp[0]), int(shp[1])) if nd.value == 2 else (int(shp[0]),)))
        self.index: Dict[str, int] = {n: i for i, (n, _) in enumerate(self.params)}

    def _check(self, st: int):
        if st != FT_OK:
            msg = lib().ft_last_error(self._h).decode() if self._h else "no handle"
            raise ForgeStepError(st, msg)

    def close(self):
        if self._h:
            # the library also works on streams of its own (weight gradients): nothing of this model may still be running
            # when its workspace goes back to the allocator
            import torch
            torch.cuda.synchronize()
            lib().ft_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- steps (device tensors: int32 [B, S], contiguous) -------------------------------------------
    def train_step(self, tokens, labels, want_loss: bool = True):
        B, S = tokens.shape
        loss, gn = C.c_float(), C.c_float()
        st = lib().ft_train_step(self._h, C.c_void_p(tokens.data_ptr()), C.c_void_p(labels.data_ptr()), B, S,
                                 C.byref(loss) if want_loss else None, C.byref(gn) if want_loss else None)
        self._check(st)
        return (loss.value, gn.value) if want_loss else None

    def train_step_host(self, tokens: np.ndarray, labels: np.ndarray):
        """tokens, labels: int32 numpy arrays [B, S] in host memory (copied to the device inside the call)."""
        B, S = tokens.shape
        loss, gn = C.c_float(), C.c_float()
        st = lib().ft_train_step_host(self._h, C.c_void_p(tokens.ctypes.data), C.c_void_p(labels.ctypes.data), B, S,
                                      C.byref(loss), C.byref(gn))
        self._check(st)
        return loss.value, gn.value

    def submit_step_host(self, tokens: np.ndarray, labels: np.ndarray):
        """Enqueue one train step on host int32 arrays [B, S] (ideally pinned) without waiting for it; at most
        MAX_IN_FLIGHT steps may be outstanding.  The arrays must stay unchanged until the step is collected."""
        B, S = tokens.shape
        self._pending.append((tokens, labels))  # keep the buffers alive while the copy may still run
        self._check(lib().ft_submit_step_host(self._h, C.c_void_p(tokens.ctypes.data), C.c_void_p(labels.ctypes.data), B, S))

    def collect_step(self):
        """Wait for the oldest submitted step; returns its (loss, gradient norm)."""
        loss, gn = C.c_float(), C.c_float()
        st = lib().ft_collect_step(self._h, C.byref(loss), C.byref(gn))
        if self._pending:
            self._pending.pop(0)
        self._check(st)
        return loss.value, gn.value

    def forward_loss(self, tokens, labels) -> float:
        B, S = tokens.shape
        loss = C.c_float()
        self._check(lib().ft_forward_loss(self._h, C.c_void_p(tokens.data_ptr()), C.c_void_p(labels.data_ptr()), B, S,
                                          C.byref(loss)))
        return loss.value

    def forward_backward(self, tokens, labels) -> float:
        B, S = tokens.shape
        loss = C.c_float()
        self._check(lib().ft_forward_backward(self._h, C.c_void_p(tokens.data_ptr()), C.c_void_p(labels.data_ptr()), B,
                                              S, C.byref(loss)))
        return loss.value

    def apply_update(self) -> float:
        gn = C.c_float()
        self._check(lib().ft_apply_update(self._h, C.byref(gn)))
        return gn.value

    # ---- state ------------------------------------------------------------------------------------------
    def get_param(self, name: str, kind: int = KIND_MASTER) -> np.ndarray:
        i = self.index[name]
        shape = self.params[i][1]
        out = np.empty(shape, dtype=np.uint16 if kind == KIND_BF16 else np.float32)
        self._check(lib().ft_get_param(self._h, i, kind, C.c_void_p(out.ctypes.data), out.nbytes))
        return bf16_bits_to_f32(out) if kind == KIND_BF16 else out

    def set_param(self, name: str, value: np.ndarray, kind: int = KIND_MASTER):
        if kind == KIND_BF16:
            raise ValueError("the bf16 copy is derived from the master; set the master instead")
        i = self.index[name]
        v = np.ascontiguousarray(value, dtype=np.float32).reshape(self.params[i][1])
        self._check(lib().ft_set_param(self._h, i, kind, C.c_void_p(v.ctypes.data), v.nbytes))

    @property
    def step(self) -> int:
        s = C.c_int64()
        self._check(lib().ft_get_step(self._h, C.byref(s)))
        return s.value

    @step.setter
    def step(self, v: int):
        self._check(lib().ft_set_step(self._h, int(v)))

    def get_tap(self, name: str, layer: int = -1) -> np.ndarray:
        """Named intermediate of the last step as a flat float32 array."""
        need, dt = C.c_size_t(), C.c_int32()
        probe = np.empty(1, dtype=np.uint8)
        st = lib().ft_get_tap(self._h, name.encode(), layer, C.c_void_p(probe.ctypes.data), 0, C.byref(need),
                              C.byref(dt))
        if st == FT_ENOTFOUND:
            self._check(st)
        buf = np.empty(need.value, dtype=np.uint8)
        self._check(lib().ft_get_tap(self._h, name.encode(), layer, C.c_void_p(buf.ctypes.data), buf.nbytes,
                                     C.byref(need), C.byref(dt)))
        return buf.view(np.float32).copy() if dt.value == 1 else bf16_bits_to_f32(buf.view(np.uint16))

    def set_fused_update(self, enable: bool):
        """AdamW inside the weight-gradient GEMM epilogues (default on; only takes effect with clipping off)."""
        self._check(lib().ft_set_fused_update(self._h, 1 if enable else 0))

    def set_rope_scaling(self, factors=None, mscale: float = 1.0):
        """LongRoPE-form position tables: per-frequency rescale factors (head_dim / 2 floats, None = 1) and a magnitude
        factor on cos and sin."""
        f = None if factors is None else np.ascontiguousarray(factors, dtype=np.float32)
        self._check(lib().ft_set_rope_scaling(self._h, None if f is None else C.c_void_p(f.ctypes.data), float(mscale)))

    def set_overlap(self, enable: bool):
        """Weight-gradient GEMMs on a second stream, concurrent with the rest of the backward pass (default on)."""
        self._check(lib().ft_set_overlap(self._h, 1 if enable else 0))

    def set_streaming_ce(self, enable: bool):
        """Cross-entropy inside the logits GEMM's epilogues (no logits in memory, the GEMM runs twice); default off."""
        self._check(lib().ft_set_streaming_ce(self._h, 1 if enable else 0))

    def set_attention_stored_ds(self, enable: bool):
        """Attention backward that stores dS^T once and computes dQ as one batched contraction (default on)."""
        self._check(lib().ft_set_attention_stored_ds(self._h, 1 if enable else 0))

    def set_fused_swiglu_bwd(self, enable: bool):
        """SwiGLU backward in the epilogue of the down projection's data-gradient GEMM (default on; bit-identical)."""
        self._check(lib().ft_set_fused_swiglu_bwd(self._h, 1 if enable else 0))

    def set_graph(self, enable: bool):
        """Capture the whole step into a CUDA graph on its second run and replay it afterwards."""
        self._check(lib().ft_set_graph(self._h, 1 if enable else 0))

    @property
    def graph_replays(self) -> int:
        return int(lib().ft_graph_replays(self._h))

    def set_profiling(self, enable: bool):
        self._check(lib().ft_set_profiling(self._h, 1 if enable else 0))

    def get_profile(self) -> Dict[str, Dict[str, float]]:
        """Per kernel class: device milliseconds, algorithmic work (FLOPs or bytes) and kernel count."""
        out = {}
        for cls, name in enumerate(PROF_CLASSES):
            ms, work, n = C.c_double(), C.c_double(), C.c_int64()
            self._check(lib().ft_get_profile(self._h, cls, C.byref(ms), C.byref(work), C.byref(n)))
            out[name] = dict(ms=ms.value, work=work.value, launches=int(n.value))
        return out

    def get_gemm_profile(self):
        """List of dicts (M, N, K, a_mn, b_mn, epi, M2, N2, ms, launches, tflops) for every GEMM shape seen while profiling;
        M2 x N2: the second output of a launch that computed two weight gradients at once (0 otherwise)."""
        out, i = [], 0
        while True:
            shp, ms, n = (C.c_int32 * 8)(), C.c_double(), C.c_int64()
            st = lib().ft_get_gemm_profile(self._h, i, shp, C.byref(ms), C.byref(n))
            if st == FT_ENOTFOUND:
                break
            self._check(st)
            M, N, K, M2, N2 = shp[0], shp[1], shp[2], shp[6], shp[7]
            out.append(dict(M=M, N=N, K=K, a_mn=shp[3], b_mn=shp[4], epi=shp[5], M2=M2, N2=N2, ms=ms.value, launches=int(n.value),
                            tflops=2.0 * (M * N + M2 * N2) * K * n.value / (ms.value * 1e-3) / 1e12 if ms.value > 0 else 0.0))
            i += 1
        return out

    @property
    def launch_count(self) -> int:
        return int(lib().ft_launch_count(self._h))


# ---- single kernels (torch device tensors) ---------------------------------------------------------------
def k_gemm(A, a_mn: int, B, b_mn: int, Cout, out_kind: int, M: int, N: int, K: int, err, resid=None):
    """C[M,N] = sum_k A[m,k] B[n,k] on device tensors; leading dimensions are the tensors' row strides."""
    st = lib().ft_k_gemm(C.c_void_p(A.data_ptr()), a_mn, A.stride(0), C.c_void_p(B.data_ptr()), b_mn, B.stride(0),
                         C.c_void_p(Cout.data_ptr()), Cout.stride(0),
                         C.c_void_p(resid.data_ptr()) if resid is not None else None, out_kind, M, N, K,
                         C.c_void_p(err.data_ptr()), _stream_ptr())
    if st != FT_OK:
        raise ForgeStepError(st, "ft_k_gemm")


def k_gemm_ws(A, a_mn: int, B, b_mn: int, Cout, out_kind: int, M: int, N: int, K: int, scratch, err, resid=None):
    """k_gemm with an fp32 device scratch tensor, which enables the deterministic split-K / balanced-K schedules."""
    st = lib().ft_k_gemm_ws(C.c_void_p(A.data_ptr()), a_mn, A.stride(0), C.c_void_p(B.data_ptr()), b_mn, B.stride(0),
                            C.c_void_p(Cout.data_ptr()), Cout.stride(0),
                            C.c_void_p(resid.data_ptr()) if resid is not None else None, out_kind, M, N, K,
                            C.c_void_p(scratch.data_ptr()), scratch.numel() * 4, C.c_void_p(err.data_ptr()),
                            _stream_ptr())
    if st != FT_OK:
        raise ForgeStepError(st, "ft_k_gemm_ws")


def k_attention_fwd(qkv, o, lse, B, S, n_heads, n_kv, d):
    st = lib().ft_k_attention_fwd(C.c_void_p(qkv.data_ptr()), C.c_void_p(o.data_ptr()), C.c_void_p(lse.data_ptr()), B,
                                  S, n_heads, n_kv, d, _stream_ptr())
    if st != FT_OK:
        raise ForgeStepError(st, "ft_k_attention_fwd")


def k_attention_bwd(qkv, o, d_o, lse, delta, dqkv, B, S, n_heads, n_kv, d, cos=None, sin=None):
    st = lib().ft_k_attention_bwd(C.c_void_p(qkv.data_ptr()), C.c_void_p(o.data_ptr()), C.c_void_p(d_o.data_ptr()),
                                  C.c_void_p(lse.data_ptr()), C.c_void_p(delta.data_ptr()),
                                  C.c_void_p(dqkv.data_ptr()), C.c_void_p(cos.data_ptr()) if cos is not None else None,
                                  C.c_void_p(sin.data_ptr()) if sin is not None else None, B, S, n_heads, n_kv, d,
                                  _stream_ptr())
    if st != FT_OK:
        raise ForgeStepError(st, "ft_k_attention_bwd")


def k_attention_bwd_ws(qkv, o, d_o, lse, delta, dqkv, ds, B, S, n_heads, n_kv, d, cos=None, sin=None):
    """Attention backward with a dS^T scratch tensor `ds` (bf16, at least B * n_heads * S * S elements) or None."""
    st = lib().ft_k_attention_bwd_ws(C.c_void_p(qkv.data_ptr()), C.c_void_p(o.data_ptr()), C.c_void_p(d_o.data_ptr()),
                                     C.c_void_p(lse.data_ptr()), C.c_void_p(delta.data_ptr()),
                                     C.c_void_p(dqkv.data_ptr()), C.c_void_p(cos.data_ptr()) if cos is not None else None,
                                     C.c_void_p(sin.data_ptr()) if sin is not None else None,
                                     C.c_void_p(ds.data_ptr()) if ds is not None else None,
                                     ds.numel() * ds.element_size() if ds is not None else 0, B, S, n_heads, n_kv, d,
                                     _stream_ptr())
    if st != FT_OK:
        raise ForgeStepError(st, "ft_k_attention_bwd_ws")


def k_attention_bwd_noalloc(qkv, o, d_o, lse, dqkv, B, S, n_heads, n_kv, d, cos=None, sin=None):
    """Attention backward whose scratch lives inside the library: for callers that may not allocate device memory.
    Returns the status code instead of raising, so a caller can tell "too large for the built-in scratch" apart."""
    return lib().ft_k_attention_bwd_noalloc(
        C.c_void_p(qkv.data_ptr()), C.c_void_p(o.data_ptr()), C.c_void_p(d_o.data_ptr()), C.c_void_p(lse.data_ptr()),
        C.c_void_p(dqkv.data_ptr()), C.c_void_p(cos.data_ptr()) if cos is not None else None,
        C.c_void_p(sin.data_ptr()) if sin is not None else None, B, S, n_heads, n_kv, d, _stream_ptr())
