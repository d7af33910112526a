"""One communicator on the GPUs of a `torch.distributed` job, one process per GPU.

Argument marshalling around `sparbit_allgather_multi`: every process allocates the receive buffers
of the ranks its device holds, the processes exchange IPC handles of those buffers once, and each
collective is one call into the library, which launches this device's kernel of every step and
calls back for the barrier between steps.  The copies themselves - local ones and the stores into
the other devices' buffers - all happen in the library's kernels.

The barrier is the process group's: with the NCCL backend a one-element all-reduce enqueued on
the collective's stream (stream-ordered, the host does not wait); with any other backend (gloo) a
stream synchronise followed by the group's host barrier.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as sp


class MultiDeviceAllgather:
    """P ranks with blocks of m bytes on the `world_size` devices of `group`.

    `recv` is this device's receive buffers, `[n_local][P][m]` bytes (rank order), allocated here;
    `allgather(send_local)` fills it from every device's send blocks (`[n_local][m]` bytes each).
    Every process of the group must construct the object and make the same calls in the same order.
    """

    def __init__(self, P: int, block_bytes: int, algo: int = sp.ALGO_SPARBIT, mapping: int = sp.MAP_SEQUENTIAL,
                 group=None, device=None):
        self.group = group
        self.G = dist.get_world_size(group)
        self.me = dist.get_rank(group)
        if self.G > sp.MULTI_MAX_DEVICES:
            raise ValueError(f"at most {sp.MULTI_MAX_DEVICES} devices")
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.P, self.m, self.mapping = P, block_bytes, mapping
        self.plan = sp.Plan(P, block_bytes, algo)
        self.n_local = sp.multi_rank_count(P, self.G, mapping, self.me)
        self.ranks = [r for r in range(P) if sp.lib.sparbit_rank_device(P, self.G, mapping, r) == self.me]
        with torch.cuda.device(self.device):
            self.recv = torch.empty(max(self.n_local * P * block_bytes, 1), dtype=torch.uint8, device=self.device)
            self._token = torch.zeros(1, dtype=torch.int32, device=self.device)
            torch.cuda.synchronize()
            handles = [None] * self.G
            dist.all_gather_object(handles, sp.ipc_export(self.recv), group=group)
            self._opened, self.bases = [], []
            for g in range(self.G):
                if g == self.me:
                    self.bases.append(self.recv.data_ptr())
                else:
                    ptr, base = sp.ipc_open(*handles[g])
                    self.bases.append(ptr)
                    self._opened.append(base)
        self._nccl = dist.get_backend(group) == "nccl"
        self.barrier_calls = 0

    def _barrier(self, stream: torch.cuda.Stream):
        self.barrier_calls += 1
        if self._nccl:
            with torch.cuda.stream(stream):
                dist.all_reduce(self._token, group=self.group)
        else:
            stream.synchronize()
            dist.barrier(group=self.group)

    def allgather(self, send_local: torch.Tensor, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Enqueues the collective on `stream` (default: the current one) and returns `recv`, which is
        complete for work enqueued on that stream afterwards."""
        if send_local.numel() * send_local.element_size() != self.n_local * self.m:
            raise ValueError(f"send_local must hold {self.n_local} blocks of {self.m} bytes")
        with torch.cuda.device(self.device):
            st = torch.cuda.current_stream() if stream is None else stream
            self.plan.allgather_multi(self.G, self.mapping, self.me, send_local, self.bases,
                                      lambda _handle: self._barrier(st), st)
        return self.recv

    def close(self) -> None:
        """Unmaps the other devices' buffers; collective (nobody frees a buffer that is still mapped)."""
        if getattr(self, "_opened", None) is None:
            return
        with torch.cuda.device(self.device):
            torch.cuda.synchronize()
            dist.barrier(group=self.group)
            while self._opened:
                sp.ipc_close(self._opened.pop())
            dist.barrier(group=self.group)
        self._opened = None
        self.plan.destroy()
