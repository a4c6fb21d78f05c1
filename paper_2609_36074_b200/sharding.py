"""Host side of a row-sharded run (one process and one handle per GPU; see the sharding section of gem_nlr.h).

The library takes two callbacks: an all-gather of equal-sized records on a CUDA stream and a rank-ordered sum of a
small host vector.  This module provides them over torch.distributed (NCCL on GPUs, gloo on the CPU for the
protocol tests) and, for tests on a single GPU, over Python threads that stand in for the ranks (the ranks'
kernels never wait on one another: only host threads meet at a barrier, with no kernel in flight).

Nothing here does arithmetic of the method except `ordered_sum`, the rank-ordered addition of the setup's
host-side d-vectors; the per-iteration sums are taken by the library's own kernels from the gathered records.
"""
from __future__ import annotations

import ctypes as C
import threading

import numpy as np

GATHER_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p)
HOST_SUM_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.POINTER(C.c_double), C.c_int64)


def row_ranges(n: int, world: int):
    """Contiguous, balanced row blocks: the first n % world ranks hold one row more."""
    base, rem = divmod(int(n), int(world))
    out, lo = [], 0
    for g in range(world):
        hi = lo + base + (1 if g < rem else 0)
        out.append((lo, hi))
        lo = hi
    return out


def ordered_sum(parts) -> np.ndarray:
    """Sum of equally shaped FP64 arrays added in list (= rank) order."""
    acc = np.array(parts[0], dtype=np.float64, copy=True)
    for p in parts[1:]:
        acc += p
    return acc


class _Exchange:
    """Common part: owns the exchange tensor and the ctypes callback objects (kept alive with the object)."""

    def __init__(self, rank: int, world: int):
        self.rank, self.world = int(rank), int(world)
        self.xbuf = None            # torch float64 tensor: [xcount] send area, then [world * xcount] receive area
        self.stream = None
        self.gather_c = GATHER_FN(self._gather_cb)
        self.host_sum_c = HOST_SUM_FN(self._host_sum_cb)

    def bind(self, xbuf, stream=None):
        self.xbuf, self.stream = xbuf, stream
        self.xcount = xbuf.numel() // (self.world + 1)

    def _views(self, send_ptr, recv_ptr, nbytes):
        base = self.xbuf.data_ptr()
        count = nbytes // 8
        if send_ptr != base or recv_ptr != base + 8 * self.xcount or count > self.xcount:
            raise ValueError("gather called with pointers outside the exchange area")
        return self.xbuf[:count], self.xbuf[self.xcount: self.xcount + self.world * count], count

    def _gather_cb(self, ctx, send_ptr, recv_ptr, nbytes, stream_ptr):
        try:
            send, recv, count = self._views(send_ptr, recv_ptr, nbytes)
            self.gather(send, recv, count)
            return 0
        except Exception:        # no exception may cross the C boundary
            import traceback
            traceback.print_exc()
            return 1

    def _host_sum_cb(self, ctx, buf, count):
        try:
            arr = np.ctypeslib.as_array(buf, shape=(int(count),))
            arr[:] = self.host_sum(arr.copy())
            return 0
        except Exception:
            import traceback
            traceback.print_exc()
            return 1


class TorchDistExchange(_Exchange):
    """Ranks are torch.distributed processes (backend nccl with the exchange tensor on the GPU, or gloo with a CPU
    tensor).  The all-gather is enqueued on the handle's stream."""

    def __init__(self, group=None):
        import torch.distributed as dist
        super().__init__(dist.get_rank(group), dist.get_world_size(group))
        self.group = group

    def gather(self, send, recv, count):
        import torch
        import torch.distributed as dist
        if send.is_cuda and self.stream is not None:
            with torch.cuda.stream(self.stream):
                dist.all_gather_into_tensor(recv, send, group=self.group)
        else:
            parts = [torch.empty_like(send) for _ in range(self.world)]
            dist.all_gather(parts, send.contiguous(), group=self.group)
            for g, t in enumerate(parts):
                recv[g * count:(g + 1) * count].copy_(t)

    def host_sum(self, vec: np.ndarray) -> np.ndarray:
        import torch
        import torch.distributed as dist
        mine = torch.from_numpy(np.ascontiguousarray(vec, dtype=np.float64))
        dev = self.xbuf.device if (self.xbuf is not None and dist.get_backend(self.group) == "nccl") else "cpu"
        mine = mine.to(dev)
        parts = [torch.empty_like(mine) for _ in range(self.world)]
        dist.all_gather(parts, mine, group=self.group)
        return ordered_sum([t.cpu().numpy() for t in parts])


class ThreadRanks:
    """Several ranks inside one process, one Python thread each, for tests on a single GPU.  The threads meet at a
    host barrier only after each has synchronized its own stream, so no kernel ever waits for another rank."""

    def __init__(self, world: int):
        self.world = int(world)
        self.barrier = threading.Barrier(self.world)
        self.members = [None] * self.world
        self.host_parts = [None] * self.world

    def member(self, rank: int) -> "_ThreadExchange":
        ex = _ThreadExchange(rank, self)
        self.members[rank] = ex
        return ex


class _ThreadExchange(_Exchange):
    def __init__(self, rank: int, ranks: ThreadRanks):
        super().__init__(rank, ranks.world)
        self.ranks = ranks

    def gather(self, send, recv, count):
        import torch
        R = self.ranks
        if send.is_cuda:
            self.stream.synchronize()            # my record is complete
        R.barrier.wait()
        ctx = torch.cuda.stream(self.stream) if send.is_cuda else _null()
        with ctx:
            for g, other in enumerate(R.members):
                recv[g * count:(g + 1) * count].copy_(other.xbuf[:count])
        if send.is_cuda:
            self.stream.synchronize()            # every copy out of the others' send areas has finished
        R.barrier.wait()

    def host_sum(self, vec: np.ndarray) -> np.ndarray:
        R = self.ranks
        R.host_parts[self.rank] = vec
        R.barrier.wait()
        out = ordered_sum(R.host_parts)
        R.barrier.wait()
        return out


class _null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def attach(solver, exchange: _Exchange, n_global: int):
    """gem_nlr_shard_attach for a GemNlr handle: allocates the exchange area next to the solver's buffers."""
    import torch
    from . import binding
    L = binding.lib()
    nbytes = int(L.gem_nlr_shard_exchange_bytes(C.byref(solver.params), exchange.world))
    xbuf = torch.zeros(nbytes // 8, dtype=torch.float64, device=solver.U.device)
    exchange.bind(xbuf, solver._stream)
    rc = L.gem_nlr_shard_attach(solver._h, exchange.rank, exchange.world, int(n_global),
                                C.cast(exchange.gather_c, C.c_void_p), C.cast(exchange.host_sum_c, C.c_void_p), None,
                                xbuf.data_ptr(), nbytes)
    if rc != 0:
        raise RuntimeError(f"gem_nlr_shard_attach failed: {rc}")
    solver._exchange = exchange          # keeps the callbacks and the exchange area alive
    return exchange
