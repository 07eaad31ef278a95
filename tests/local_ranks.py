"""Several data-parallel ranks inside ONE process, for tests on a machine with one GPU: every rank is a host thread with
its own model and streams, and the collectives are done by hand between the threads (host barriers, plain tensor
arithmetic).  No kernel ever waits for another rank's kernel: a collective first drains the caller's stream, then the
threads meet on a host barrier."""
import threading

import torch


class LocalGroup:
    def __init__(self, world: int, timeout: float = 120.0):
        self.world = world
        self.barrier = threading.Barrier(world, timeout=timeout)
        self.slots = [None] * world


class LocalDist:
    """The subset of torch.distributed that paper_2609_13645_b200.dp.DataParallel uses, for one rank of a LocalGroup."""

    class ReduceOp:
        SUM = "sum"

    def __init__(self, group: LocalGroup, rank: int):
        self.g, self.rank = group, rank

    def get_world_size(self, group=None):
        return self.g.world

    def get_rank(self, group=None):
        return self.rank

    def get_backend(self, group=None):
        return "nccl"  # in-place reduce-scatter / all-gather semantics

    def _publish(self, t):
        if t.is_cuda:
            torch.cuda.current_stream().synchronize()
        self.g.slots[self.rank] = t
        self.g.barrier.wait()
        return list(self.g.slots)

    def _finish(self, out, value):
        # every rank has computed its result from the published inputs before any input is overwritten
        if out.is_cuda:
            torch.cuda.current_stream().synchronize()
        self.g.barrier.wait()
        out.copy_(value)
        if out.is_cuda:
            torch.cuda.current_stream().synchronize()
        self.g.barrier.wait()

    def all_reduce(self, t, op=None, group=None):
        parts = self._publish(t)
        total = parts[0].clone()
        for p in parts[1:]:
            total += p
        self._finish(t, total)

    def reduce_scatter_tensor(self, out, inp, op=None, group=None):
        parts = self._publish(inp)
        n = out.numel()
        lo = self.rank * n
        total = parts[0][lo:lo + n].clone()
        for p in parts[1:]:
            total += p[lo:lo + n]
        self._finish(out, total)

    def all_gather_into_tensor(self, out, inp, group=None):
        parts = self._publish(inp)
        whole = torch.cat([p.reshape(-1).clone() for p in parts])
        self._finish(out, whole.view_as(out))

    def barrier(self, group=None):
        self.g.barrier.wait()


def run_ranks(world: int, fn):
    """Runs fn(rank, dist) on `world` threads; returns the list of results, re-raising the first exception."""
    group = LocalGroup(world)
    results, errors = [None] * world, [None] * world

    def work(r):
        try:
            torch.cuda.set_device(0)
            results[r] = fn(r, LocalDist(group, r))
        except BaseException as e:  # noqa: BLE001
            errors[r] = e
            group.barrier.abort()

    threads = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for e in errors:
        if e is not None and not isinstance(e, threading.BrokenBarrierError):
            raise e
    for e in errors:
        if e is not None:
            raise e
    return results
