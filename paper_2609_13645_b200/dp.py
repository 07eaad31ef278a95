"""Data-parallel train step over the library's C-ABI hooks: the paper's recipe (Section "Sources of the Speedup";
appendix "Framework-Level Optimization Trajectory": gradient bucketing, per-bucket all-gather + optimizer overlap, ZeRO-1
sharded optimizer) of a bucketed gradient reduce-scatter overlapped with the backward pass, a ZeRO-1 sharded AdamW and a
per-bucket all-gather of the bf16 compute copy interleaved with it.

The exchange is `torch.distributed` (NCCL between GPUs); everything else — forward, backward, norm, AdamW — runs in the
library's own kernels through `ft_dp_*`.  One process per GPU.  Per step and rank:

  1. the number of labels >= 0 is summed over the ranks (one 8-byte all-reduce, on the device) and handed to the library
     as a device pointer (no host round trip), so that every rank's loss and gradients are already divided by the GLOBAL
     count and the reduction is a plain sum;
  2. the second (communication) stream is ordered behind what the model's stream holds so far, i.e. the PREVIOUS step,
     BEFORE this step's backward pass is enqueued: from here on it waits only for the per-bucket events;
  3. `ft_dp_backward` enqueues forward + backward on the model's stream and records one event per gradient bucket, in
     the order the backward pass completes them (head, layers last to first, embedding table, gains);
  4. on the second stream, per bucket: wait for its event, reduce-scatter it in place (rank r keeps slice r), and, when
     clipping is off, run AdamW on that slice and all-gather the bucket's bf16 copy right away, while the model's stream
     is still busy with the layers below; with clipping on the updates wait for the global norm (sum of squares of every
     rank's slices, one 4-byte all-reduce);
  5. the model's stream waits for the second stream; the rank's loss share is read back and summed over the ranks.

A bucket's event follows the last kernel that reads that bucket's bf16 weights (its data gradients, and with
recomputation its re-run forward), so the all-gather that rewrites them cannot overtake a reader.

Optimizer state: with `dp_world` / `dp_rank` in the model's config (they must equal the group's size and this rank) the
workspace holds masters and moments only for the rank's own slices, 12 / world bytes per parameter; without them (one
rank, or an unsharded model on several) the arenas are full size and only the owned slices are kept current.
`DataParallel.get_state` / `set_state` assemble or distribute whole tensors for checkpoints.

`DataParallel` talks to a backend object, so the bucket / slice / collective logic is exercised on CPU (gloo) with a
stand-in backend; `LibraryBackend` is the real one.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Tuple


class LibraryBackend:
    """The C-ABI hooks of one `binding.Model` as the backend of `DataParallel` (CUDA tensors, raw stream pointers)."""

    def __init__(self, model):
        import torch
        from . import binding as B
        self.B, self.torch, self.model = B, torch, model
        L = B.lib()
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.ft_dp_num_buckets.argtypes = [vp]; L.ft_dp_num_buckets.restype = i32
        L.ft_dp_bucket.argtypes = [vp, i32, C.POINTER(i64), C.POINTER(i64)]
        L.ft_arena_ptr.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(i64)]
        L.ft_dp_scratch.argtypes = [vp, C.POINTER(vp)]
        L.ft_dp_set_label_count.argtypes = [vp, i64]
        L.ft_dp_set_label_count_device.argtypes = [vp, vp]
        L.ft_dp_backward.argtypes = [vp, vp, vp, i32, i32]
        L.ft_dp_stream_wait_bucket.argtypes = [vp, i32, vp]
        L.ft_dp_sqnorm.argtypes = [vp, i64, i64, vp, vp]
        L.ft_dp_begin_update.argtypes = [vp, vp, vp]
        L.ft_dp_update_range.argtypes = [vp, i64, i64, vp]
        L.ft_dp_set_norm.argtypes = [vp, vp, vp]
        L.ft_dp_collect.argtypes = [vp, vp, vp]
        for n in ("ft_dp_bucket", "ft_arena_ptr", "ft_dp_scratch", "ft_dp_set_label_count", "ft_dp_set_label_count_device",
                  "ft_dp_backward", "ft_dp_stream_wait_bucket", "ft_dp_sqnorm", "ft_dp_begin_update", "ft_dp_update_range", "ft_dp_set_norm",
                  "ft_dp_collect"):
            getattr(L, n).restype = C.c_int
        self.L = L
        self.clipping = float(model.cfg.max_grad_norm) > 0.0
        self.device = model.workspace.device
        self.main_stream = torch.cuda.current_stream()
        self.comm_stream = torch.cuda.Stream()
        self._grad = self._arena(B.KIND_GRAD, torch.float32)
        self._bf16 = self._arena(B.KIND_BF16, torch.bfloat16)

    def _arena(self, kind, dtype):
        ptr, n = C.c_void_p(), C.c_int64()
        self.model._check(self.L.ft_arena_ptr(self.model._h, kind, C.byref(ptr), C.byref(n)))
        ws = self.model.workspace
        off = ptr.value - ws.data_ptr()
        nbytes = n.value * (4 if dtype == self.torch.float32 else 2)
        assert 0 <= off and off + nbytes <= ws.numel()
        return ws[off:off + nbytes].view(dtype)  # aliases the library's memory

    # ---- what DataParallel needs
    def buckets(self) -> List[Tuple[int, int]]:
        out = []
        for i in range(self.L.ft_dp_num_buckets(self.model._h)):
            o, c = C.c_int64(), C.c_int64()
            self.model._check(self.L.ft_dp_bucket(self.model._h, i, C.byref(o), C.byref(c)))
            out.append((o.value, c.value))
        return out

    def grad(self):
        return self._grad

    def compute_copy(self):
        return self._bf16

    def new_scalars(self, n):
        return self.torch.zeros(n, dtype=self.torch.float32, device=self.device)

    def count_labels(self, labels):
        """[labels counted by the backbone's loss, labels counted by the MTP head's loss (shifted by one)] as int64."""
        t = self.torch
        return t.stack([(labels >= 0).sum(), (labels[:, 1:] >= 0).sum()]).to(t.int64)

    def set_label_count(self, total):
        """total: int64 tensor on the device holding the label counts of all ranks (kept alive here)."""
        self._total = total
        self.model._check(self.L.ft_dp_set_label_count_device(self.model._h, C.c_void_p(total.data_ptr())))

    def backward(self, tokens, labels):
        Bsz, S = tokens.shape
        self.model._check(self.L.ft_dp_backward(self.model._h, C.c_void_p(tokens.data_ptr()), C.c_void_p(labels.data_ptr()), Bsz, S))

    def comm(self):
        """Context in which collectives and the calls below are enqueued on the second stream."""
        return self.torch.cuda.stream(self.comm_stream)

    def begin_comm(self):
        # ordered behind the PREVIOUS step only (its readers of what this step's collectives overwrite): called before this
        # step's backward pass is enqueued, so that the per-bucket events are the only thing the collectives wait for
        self.comm_stream.wait_stream(self.main_stream)

    def shard(self):
        """(dp_world, dp_rank) of the model's optimizer-state shard; (1, 0) when the state is whole."""
        w = int(self.model.cfg.dp_world)
        return (w, int(self.model.cfg.dp_rank)) if w > 1 else (1, 0)

    def get_param(self, name, kind):
        return self.torch.from_numpy(self.model.get_param(name, kind)).to(self.device)

    def set_param(self, name, value, kind):
        self.model.set_param(name, value, kind)

    def param_names(self):
        return [n for n, _ in self.model.params]

    def end_comm(self):
        self.main_stream.wait_stream(self.comm_stream)

    def wait_bucket(self, i: int):
        self.model._check(self.L.ft_dp_stream_wait_bucket(self.model._h, i, C.c_void_p(self.comm_stream.cuda_stream)))

    def sqnorm(self, offset: int, count: int, out):
        self.model._check(self.L.ft_dp_sqnorm(self.model._h, offset, count, C.c_void_p(out.data_ptr()),
                                              C.c_void_p(self.comm_stream.cuda_stream)))

    def begin_update(self, sq_total):
        self.model._check(self.L.ft_dp_begin_update(self.model._h, C.c_void_p(sq_total.data_ptr()) if sq_total is not None else None,
                                                    C.c_void_p(self.comm_stream.cuda_stream)))

    def update_range(self, offset: int, count: int):
        self.model._check(self.L.ft_dp_update_range(self.model._h, offset, count, C.c_void_p(self.comm_stream.cuda_stream)))

    def set_norm(self, sq_total):
        self.model._check(self.L.ft_dp_set_norm(self.model._h, C.c_void_p(sq_total.data_ptr()),
                                                C.c_void_p(self.comm_stream.cuda_stream)))

    def collect(self):
        loss, gn = C.c_float(), C.c_float()
        self.model._check(self.L.ft_dp_collect(self.model._h, C.byref(loss), C.byref(gn)))
        return loss.value, gn.value


class DataParallel:
    """One data-parallel train step per call of `step`; see the module text for the sequence."""

    def __init__(self, backend, group=None, dist=None):
        """dist: the module that provides the collectives (default torch.distributed); a stand-in with the same calls
        lets tests run several ranks inside one process."""
        if dist is None:
            import torch.distributed as dist
        self.dist, self.backend, self.group = dist, backend, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.buckets = backend.buckets()
        shard = backend.shard() if hasattr(backend, "shard") else (1, 0)
        if shard != (1, 0) and shard != (self.world, self.rank):
            raise ValueError(f"the model's state shard {shard} is not (world, rank) = ({self.world}, {self.rank}) of the group")
        self.sharded = shard != (1, 0)
        for off, cnt in self.buckets:
            if cnt % (4 * self.world) or off % 4:
                raise ValueError(f"bucket ({off}, {cnt}) does not divide into {self.world} slices of whole 16-byte groups")
        # in-place reduce-scatter / all-gather (output = slice `rank` of the input) is what NCCL supports natively
        self.in_place = dist.get_backend(group) == "nccl"
        self.sq = backend.new_scalars(len(self.buckets) + 1)  # one sum of squares per bucket slice, then their total

    def slice_of(self, bucket: int, rank: Optional[int] = None) -> Tuple[int, int]:
        """Arena (offset, count) of the slice of `bucket` that `rank` (default: this rank) owns."""
        off, cnt = self.buckets[bucket]
        n = cnt // self.world
        r = self.rank if rank is None else rank
        return off + r * n, n

    def _reduce_scatter(self, whole, mine):
        if self.in_place:
            self.dist.reduce_scatter_tensor(mine, whole, op=self.dist.ReduceOp.SUM, group=self.group)
        else:
            tmp = mine.clone()
            self.dist.reduce_scatter_tensor(tmp, whole.clone(), op=self.dist.ReduceOp.SUM, group=self.group)
            mine.copy_(tmp)

    def _all_gather(self, whole, mine):
        if self.in_place:
            self.dist.all_gather_into_tensor(whole, mine, group=self.group)
        else:
            tmp = whole.clone()
            self.dist.all_gather_into_tensor(tmp, mine.clone(), group=self.group)
            whole.copy_(tmp)

    def step(self, tokens, labels):
        """tokens, labels: this rank's batch.  Returns (global mean loss, global gradient norm)."""
        be, dist = self.backend, self.dist
        total = be.count_labels(labels)
        dist.all_reduce(total, op=dist.ReduceOp.SUM, group=self.group)
        be.set_label_count(total)  # stays on the device: no host round trip before the step is enqueued
        be.begin_comm()            # behind the previous step, ahead of this step's backward pass
        be.backward(tokens, labels)
        grad, comp = be.grad(), be.compute_copy()
        with be.comm():
            for i, (off, cnt) in enumerate(self.buckets):
                so, sn = self.slice_of(i)
                be.wait_bucket(i)
                if i == 0 and not be.clipping:
                    be.begin_update(None)  # step counter and bias corrections, once, behind the first finished bucket
                self._reduce_scatter(grad[off:off + cnt], grad[so:so + sn])
                be.sqnorm(so, sn, self.sq[i:i + 1])
                if not be.clipping:
                    be.update_range(so, sn)
                    self._all_gather(comp[off:off + cnt], comp[so:so + sn])
            nb = len(self.buckets)
            self.sq[nb:nb + 1] = self.sq[:nb].sum()
            dist.all_reduce(self.sq[nb:nb + 1], op=dist.ReduceOp.SUM, group=self.group)
            if be.clipping:
                be.begin_update(self.sq[nb:nb + 1])
                for i, (off, cnt) in enumerate(self.buckets):
                    so, sn = self.slice_of(i)
                    be.update_range(so, sn)
                    self._all_gather(comp[off:off + cnt], comp[so:so + sn])
            else:
                be.set_norm(self.sq[nb:nb + 1])
        be.end_comm()
        share, gnorm = be.collect()
        loss = be.new_scalars(1)
        loss[0] = share
        dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=self.group)
        return float(loss.item()), gnorm

    # ---- whole tensors for checkpoints (masters, moments), whatever the sharding
    def get_state(self, name, kind):
        """The whole tensor `name` of `kind` (binding.KIND_MASTER / KIND_ADAM_M / KIND_ADAM_V) on every rank.  With a
        sharded state every rank contributes its owned elements (the library returns 0 elsewhere) and the parts are summed."""
        t = self.backend.get_param(name, kind)
        if self.sharded:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t

    def set_state(self, name, value, kind):
        """Every rank passes the whole tensor; with a sharded state each keeps its own elements."""
        self.backend.set_param(name, value, kind)
