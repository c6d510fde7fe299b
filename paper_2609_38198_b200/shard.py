"""Row-sharded operation (fd_set_shard): the two exchange callbacks the C library asks for, on torch.distributed.

The library itself links no communication library.  `Shard` owns the exchange buffer and the ctypes callbacks of one
context; a *transport* does the two collectives:

  TorchDistTransport  one process per GPU; rows gathered with all_gather_into_tensor on the device group (NCCL over
                      NVLink), small host sums on a gloo group when one is given, else staged through the device.
                      With CPU tensors and a gloo group the same class runs without a GPU (the world-size-2 CPU test).
  ThreadTransport     several in-process ranks (threads) that share ONE GPU, each with its own context and stream:
                      the exchange happens on the host side between launches, no kernel ever waits for another rank.
                      For tests and debugging of the sharded drivers where only one GPU is available.

Marshalling only: every arithmetic step stays in the library's kernels.
"""
from __future__ import annotations

import ctypes
import threading
from ctypes import CFUNCTYPE, POINTER, Structure, byref, c_double, c_int, c_int32, c_int64, c_size_t, c_void_p

import numpy as np
import torch

from . import binding as B

ALLREDUCE_FN = CFUNCTYPE(c_int, c_void_p, POINTER(c_double), c_int64)
ALLGATHER_FN = CFUNCTYPE(c_int, c_void_p, c_void_p, c_void_p, c_int64)


class fd_shard(Structure):
    _fields_ = [("rank", c_int32), ("world", c_int32), ("allreduce_sum_host", ALLREDUCE_FN),
                ("allgather_dev", ALLGATHER_FN), ("user", c_void_p), ("xchg_dev", c_void_p), ("xchg_bytes", c_size_t)]


B.lib.fd_shard_rows.argtypes = [c_int64, c_int32, c_int32, POINTER(c_int64), POINTER(c_int64)]
B.lib.fd_shard_exchange_bytes.argtypes = [c_int64, c_int32, c_int32]
B.lib.fd_shard_exchange_bytes.restype = c_size_t
B.lib.fd_set_shard.argtypes = [c_void_p, POINTER(fd_shard)]


def fd_shard_rows(N: int, world: int, rank: int):
    b, e = c_int64(), c_int64()
    st = B.lib.fd_shard_rows(N, world, rank, byref(b), byref(e))
    if st != B.FD_OK:
        raise B.FdError(st)
    return b.value, e.value


def fd_shard_exchange_bytes(N: int, b_max: int, world: int) -> int:
    return int(B.lib.fd_shard_exchange_bytes(N, b_max, world))


class TorchDistTransport:
    """Collectives of one rank on torch.distributed process groups."""

    def __init__(self, rank: int, world: int, group=None, host_group=None):
        import torch.distributed as dist
        self.dist, self.rank, self.world = dist, rank, world
        self.group, self.host_group = group, host_group

    def allreduce_sum_host(self, arr: np.ndarray, device, stream):
        t = torch.from_numpy(arr)                               # shares memory with the library's host buffer
        if self.host_group is not None or device.type == "cpu":
            self.dist.all_reduce(t, group=self.host_group if self.host_group is not None else self.group)
        else:
            with torch.cuda.stream(stream):
                td = t.to(device)
                self.dist.all_reduce(td, group=self.group)
                t.copy_(td.cpu())

    def allgather(self, send: torch.Tensor, recv: torch.Tensor, stream):
        if send.is_cuda:
            with torch.cuda.stream(stream):                     # ordered on the context's stream on both sides
                self.dist.all_gather_into_tensor(recv, send, group=self.group)
        else:
            self.dist.all_gather_into_tensor(recv, send, group=self.group)


class ThreadTransport:
    """In-process ranks on one GPU.  Create one ThreadTransport.Hub(world) and give hub.rank(r) to rank r's Shard; every
    rank must run in its own thread and make the same library calls in the same order."""

    class Hub:
        def __init__(self, world: int, timeout: float = 120.0):
            self.world = world
            self.barrier = threading.Barrier(world, timeout=timeout)
            self.host = [None] * world
            self.send = [None] * world

        def rank(self, r: int) -> "ThreadTransport":
            return ThreadTransport(self, r)

    def __init__(self, hub: "ThreadTransport.Hub", rank: int):
        self.hub, self.rank, self.world = hub, rank, hub.world

    def allreduce_sum_host(self, arr: np.ndarray, device, stream):
        h = self.hub
        h.host[self.rank] = arr.copy()
        h.barrier.wait()
        total = h.host[0].copy()
        for r in range(1, self.world):                          # fixed order: bit-identical on every rank
            total += h.host[r]
        h.barrier.wait()
        arr[:] = total

    def allgather(self, send: torch.Tensor, recv: torch.Tensor, stream):
        h = self.hub
        if send.is_cuda:
            stream.synchronize()                                # this rank's contribution is complete
        h.send[self.rank] = send
        h.barrier.wait()
        n = send.numel()
        ctx = torch.cuda.stream(stream) if send.is_cuda else _null()
        with ctx:
            for r in range(self.world):
                recv[r * n:(r + 1) * n].copy_(h.send[r])
        if send.is_cuda:
            stream.synchronize()                                # nobody overwrites a send buffer that is still being read
        h.barrier.wait()


class _null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


class Shard:
    """Exchange buffer + callbacks of one rank for one (N, b_max); attach with Context.set_shard(shard)."""

    def __init__(self, transport, N: int, b_max: int, device, stream=None):
        self.transport = transport
        self.rank, self.world = int(transport.rank), int(transport.world)
        self.N, self.b_max = int(N), int(b_max)
        self.device = torch.device(device)
        self.row_begin, self.row_end = fd_shard_rows(self.N, self.world, self.rank)
        nbytes = fd_shard_exchange_bytes(self.N, self.b_max, self.world)
        if nbytes == 0:
            raise B.FdError(B.FD_ERR_INVALID, "fd_shard_exchange_bytes rejected the shape")
        self.xchg_bytes = nbytes
        self._buf = torch.empty(nbytes // 4 + 64, dtype=torch.float32, device=self.device)
        self._off = ((-self._buf.data_ptr()) % 256) // 4
        self._base = self._buf.data_ptr() + 4 * self._off
        self.stream = stream if stream is not None else (torch.cuda.current_stream(self.device) if self.device.type == "cuda" else None)
        self.error = None                                       # the exception a callback swallowed, for the caller to re-raise
        self._ar = ALLREDUCE_FN(self._allreduce)
        self._ag = ALLGATHER_FN(self._allgather)
        self.struct = fd_shard(self.rank, self.world, self._ar, self._ag, None, c_void_p(self._base), nbytes)

    def _view(self, ptr: int, count: int) -> torch.Tensor:
        o = (ptr - self._base) // 4
        if o < 0 or (o + count) * 4 > self.xchg_bytes:
            raise ValueError("exchange pointer outside the exchange buffer")
        return self._buf[self._off + o: self._off + o + count]

    # ctypes callbacks: never let an exception cross into C
    def _allreduce(self, user, buf, n):
        try:
            arr = np.ctypeslib.as_array(buf, shape=(int(n),))
            self.transport.allreduce_sum_host(arr, self.device, self.stream)
            return 0
        except BaseException as e:                              # noqa: BLE001
            self.error = e
            return 1

    def _allgather(self, user, send_ptr, recv_ptr, count):
        try:
            count = int(count)
            send = self._view(int(send_ptr), count)
            recv = self._view(int(recv_ptr), count * self.world)
            self.transport.allgather(send, recv, self.stream)
            return 0
        except BaseException as e:                              # noqa: BLE001
            self.error = e
            return 1
