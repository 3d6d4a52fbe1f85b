"""Exchanges between ranks for data-distributed training (Sec. 7.3 of the paper: rows divided over
the workers, integer histograms summed across them).

The C library asks for every exchange through one callback (``qgbdt_set_distributed``); this module
holds two implementations of it.  ``TorchDistReducer`` is the real one: an all-reduce of
``torch.distributed`` (NCCL over NVLink for GPUs of one node) on the library's own device buffer,
enqueued on the stream the library works on.  ``LocalGroup`` joins several contexts of ONE process
(each driven by a thread of its own, all on one GPU): the ranks meet at a host barrier and one
thread adds the buffers up; no kernel ever waits for another.  Both only move and add integers:
none of the method's arithmetic lives here.
"""
from __future__ import annotations

import ctypes as C
import threading

import torch

REDUCE_SUM_I64, REDUCE_MAX_U32 = 0, 1
ALLREDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p)


class _DeviceWords:
    """CUDA array interface over `count` words of borrowed device memory."""

    def __init__(self, ptr: int, count: int, kind: int):
        # 32-bit words hold float bits of non-negative floats and 0/1 flags: they order alike as int32
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<i8" if kind == REDUCE_SUM_I64 else "<i4",
                                         "data": (ptr, False), "version": 2}


def device_words(ptr: int, count: int, kind: int) -> torch.Tensor:
    return torch.as_tensor(_DeviceWords(ptr, count, kind), device="cuda")


def allreduce_tensor(t: torch.Tensor, kind: int, group=None) -> None:
    """In-place sum (64-bit integers) or maximum (32-bit words) of a tensor over the ranks of a group."""
    import torch.distributed as dist
    dist.all_reduce(t, op=dist.ReduceOp.SUM if kind == REDUCE_SUM_I64 else dist.ReduceOp.MAX, group=group)


class TorchDistReducer:
    """All-reduce over a torch.distributed process group, on the stream the library passes."""

    def __init__(self, group=None):
        self.group = group
        self.calls = 0
        self.words = 0
        self.callback = ALLREDUCE_FN(self._reduce)

    def _reduce(self, user, d_buf, count, kind, stream):
        try:
            with torch.cuda.stream(torch.cuda.ExternalStream(stream or 0)):
                allreduce_tensor(device_words(d_buf, count, kind), kind, self.group)
            self.calls += 1
            self.words += count
            return 0
        except Exception:       # the C caller turns a non-zero return into an error code
            import traceback
            traceback.print_exc()
            return 1


class LocalGroup:
    """World of `world` contexts inside one process; rank r calls ``reducer(r).callback``."""

    def __init__(self, world: int):
        self.world = world
        self.barrier = threading.Barrier(world)
        self.slots = [None] * world
        self.calls = 0
        self.words = 0
        self.error = None

    def reducer(self, rank: int):
        group = self

        def reduce(user, d_buf, count, kind, stream):
            try:
                torch.cuda.ExternalStream(stream or 0).synchronize()       # this rank's work so far
                group.slots[rank] = (d_buf, count, kind)
                group.barrier.wait(timeout=120)
                if rank == 0:
                    assert all(s[1:] == (count, kind) for s in group.slots), "ranks disagree on an exchange"
                    parts = [device_words(s[0], count, kind) for s in group.slots]
                    total = torch.stack(parts).sum(0) if kind == REDUCE_SUM_I64 else torch.stack(parts).max(0).values
                    for t in parts:
                        t.copy_(total)
                    torch.cuda.synchronize()
                    group.calls += 1
                    group.words += count
                group.barrier.wait(timeout=120)
                return 0
            except Exception as e:
                group.error = e
                group.barrier.abort()
                return 1

        cb = ALLREDUCE_FN(reduce)
        return cb
