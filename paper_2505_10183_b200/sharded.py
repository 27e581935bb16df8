"""One rank per device: the multi-process plumbing around the library's sharded calls.

Every rank is a process with a device of its own (paper Section III-A: the devices of a group
run their collective among themselves; groups exchange through host memory).  This module
holds no arithmetic.  It moves handles and names between the processes with
``torch.distributed`` (object collectives on a host-side process group, at set-up only), maps the
group mates' gradient and output tensors into this process (``kt_ipc_open``), maps one block of
host memory that all processes of the node share (POSIX shared memory, page-locked with
``kt_host_register``; it also holds the block of ``kt_host_barrier``, where the ranks meet
during a step), and then runs steps, each one library call (``kt_shard_step``) that does, in order:

    barrier                         every rank's gradients are complete
    kt_hier_reduce(KT_INTRA)        my share of each bucket, read from all members of my group
    kt_stage_to_host(KT_D2H)        my share of my group's partial -> shared host memory
    then bucket by bucket:
      wait for my copy, barrier     every rank's share of the bucket is in host memory
      kt_stage_to_host(KT_H2D)      my element range of the other groups' partials -> device
      kt_unpack_scale               combine, scale, cast; my share written into the output
                                    tensors of every member of my group
    wait for my kernels, barrier    every rank holds the whole reduced gradient

With a single group the middle collapses to one kt_sync_direct call.  Ranks wait for one
another on the host only; no kernel waits for another device.
"""
from __future__ import annotations

import ctypes as C
import mmap
import os
import secrets
from typing import List, Optional, Sequence

import torch
import torch.distributed as dist

from . import binding as kt


class ShardedSync:
    def __init__(self, rank: int, group_of: Sequence[int], shares: Sequence[int], grads: Sequence[torch.Tensor],
                 outs: Optional[Sequence[torch.Tensor]] = None, bucket_cap_bytes: int = 25 << 20,
                 host_group=None, per_bucket: bool = True, wait_ms: int = 60000, narrow_transport: bool = False):
        """grads: this rank's gradient tensors (device, contiguous, one dtype); outs: where this
        rank wants the reduced gradients (None: in place, over `grads`); host_group: a
        torch.distributed group whose collectives run on the host (gloo) and whose ranks are
        numbered like `group_of`; narrow_transport: the library's bf16 transport (an extension:
        half the bytes through host memory, one extra rounding of every group partial; without
        effect when all ranks are one group, where no partial is stored)."""
        self.rank, self.group_of, self.K = rank, list(group_of), len(group_of)
        self.G = max(group_of) + 1
        self.g = group_of[rank]
        self.members = [r for r in range(self.K) if group_of[r] == self.g]
        self.member = self.members.index(rank)
        self.host_group = host_group
        self.wait_ms = wait_ms
        outs = list(grads) if outs is None else list(outs)
        self.grads, self.outs = list(grads), outs
        self.numel = [int(t.numel()) for t in grads]
        T = len(self.numel)
        if any(o.numel() != n or not o.is_contiguous() for o, n in zip(outs, self.numel)) or len(outs) != T:
            raise kt.KtError(kt.KT_ERR_SHAPE, "outs must match grads in count and sizes")
        self.in_dtype = kt._DTYPES[grads[0].dtype]
        self.out_dtype = kt._DTYPES[outs[0].dtype]

        # 1. every rank tells every other how its tensors can be reached
        mine = {"grads": [kt.kt_ipc_export(t.data_ptr()) if t.numel() else (b"", 0) for t in grads],
                "outs": [kt.kt_ipc_export(t.data_ptr()) if t.numel() else (b"", 0) for t in outs],
                "numel": self.numel}
        everyone: List[Optional[dict]] = [None] * self.K
        dist.all_gather_object(everyone, mine, group=host_group)
        self._opened: List[bytes] = []

        def address(r: int, kind: str, t: int) -> int:
            if r == rank:
                return (grads if kind == "grads" else outs)[t].data_ptr()
            handle, offset = everyone[r][kind][t]
            if not handle:
                return 0
            self._opened.append(handle)
            return kt.kt_ipc_open(handle, offset)

        for r in self.members:
            if everyone[r]["numel"] != self.numel:
                raise kt.KtError(kt.KT_ERR_SHAPE, "rank %d holds other tensor sizes than rank %d" % (r, rank))
        grad_ptrs = [address(r, "grads", t) for r in self.members for t in range(T)]
        out_ptrs = [address(r, "outs", t) for r in self.members for t in range(T)]

        # 2. the context of this rank
        self.ctx = kt.kt_groups_init(self.group_of, list(shares), self.G)
        kt.kt_shard_bind(self.ctx, rank, self.group_of)
        if narrow_transport:
            kt.kt_set_transport_dtype(self.ctx, kt.KT_BF16)
        tdt, tsize = (torch.bfloat16, 2) if narrow_transport else (torch.float32, 4)
        kt.kt_bucket_pack_ptrs(self.ctx, kt.PtrArray.from_addresses(grad_ptrs, keep=self.grads), self.numel,
                               self.in_dtype, bucket_cap_bytes)
        self.plan = kt.kt_plan_query(self.ctx)
        self.buckets = list(range(self.plan.n_buckets)) if per_bucket else [-1]
        self.out_ptrs = kt.PtrArray.from_addresses(out_ptrs, keep=self.outs)
        n = self.plan.transport_numel
        # row g: my share of my group's partial; rows h != g: the other groups' partials over my range
        self.partials = torch.zeros(self.G, max(n, 1), dtype=tdt, device=grads[0].device)
        self.partial_rows = kt.kt_ptrs(list(self.partials))
        self.main = torch.cuda.Stream()
        self.side = torch.cuda.Stream()                   # copies down
        self.up = torch.cuda.Stream()                     # copies up

        # 3. host memory that all processes share: a barrier block, then the G partials end to
        #    end, in a file of the node's shared-memory file system that every rank maps and
        #    page-locks
        self._header = 4096
        nbytes = self._header + (self.G * max(n, 1) * tsize if self.G > 1 else 0)
        name = [None]
        if rank == 0:
            name[0] = "/dev/shm/kt_partials_%d_%s" % (os.getpid(), secrets.token_hex(4))
            fd = os.open(name[0], os.O_CREAT | os.O_EXCL | os.O_RDWR, 0o600)
            os.ftruncate(fd, nbytes)                      # new pages read as zero: the barrier starts clean
        dist.broadcast_object_list(name, src=0, group=host_group)
        if rank != 0:
            fd = os.open(name[0], os.O_RDWR)
        self._map = mmap.mmap(fd, nbytes)
        os.close(fd)
        self._view = C.c_char.from_buffer(self._map)
        self._host_address = C.addressof(self._view)
        kt.kt_host_register(self._host_address, nbytes)
        self.host_rows = None
        if self.G > 1:
            first = self._host_address + self._header
            self.host_rows = kt.PtrArray.from_addresses([first + g * max(n, 1) * tsize for g in range(self.G)],
                                                        keep=self._map)
        dist.barrier(group=host_group)
        if rank == 0:
            os.unlink(name[0])                            # every rank has it mapped: the name can go

    def barrier(self) -> None:
        """All ranks of the job meet here, on the host, in the shared block; a rank that does not
        come within `wait_ms` ends the wait of the others with KT_ERR_TIMEOUT."""
        kt.kt_host_barrier(self._host_address, self.K, self.wait_ms)

    def my_range(self, bucket: int = -1):
        return kt.kt_shard_query(self.ctx, bucket)[:2]

    def step(self, scale: float = 1.0) -> None:
        """One synchronisation (kt_shard_step: the whole sequence of the module's header in one
        library call).  On return this rank's `outs` hold the reduced gradients and every other
        rank has finished reading this rank's `grads`."""
        kt.kt_shard_step(self.ctx, self._host_address, self.partial_rows if self.G > 1 else None, self.host_rows,
                         self.out_ptrs, len(self.members), self.out_dtype, scale=scale,
                         per_bucket=self.buckets != [-1], main_stream=self.main, down_stream=self.side,
                         up_stream=self.up, timeout_ms=self.wait_ms)

    def set_shares(self, shares: Sequence[int]) -> None:
        """New batch shares (every rank calls this with the same list, between steps): the weights
        of all later steps follow them (kt_set_shares)."""
        kt.kt_set_shares(self.ctx, list(shares))

    def broadcast(self, root: int) -> None:
        """Model synchronisation: rank `root`'s `grads` tensors (here: parameters) reach the same
        tensors of every other rank, bit for bit (kt_shard_bcast; blocks until all ranks are done)."""
        if getattr(self, "_bcast_flat", None) is None:
            n = max(self.plan.transport_numel, 1)
            self._bcast_flat = torch.empty(n, dtype=self.grads[0].dtype, device=self.grads[0].device)
        flat = self._bcast_flat.data_ptr()
        host = self._host_address + self._header if self.G > 1 else 0
        kt.kt_shard_bcast(self.ctx, root, self._host_address, flat, host, flat, self.buckets != [-1], self.main,
                          self.side, self.up, timeout_ms=self.wait_ms)

    def close(self, meet: bool = True) -> None:
        """Unmaps everything.  meet=False skips the barrier in the shared block: for ranks that
        have seen a barrier time out (the block is then in an undefined state) and have made sure
        by other means that no rank still uses this one's memory."""
        torch.cuda.synchronize()
        if meet:
            self.barrier()                            # nobody still reads what is unmapped next
        kt.kt_destroy(self.ctx)
        for handle in self._opened:
            kt.kt_ipc_close(handle)
        self._opened = []
        kt.kt_host_unregister(self._host_address)
        self.host_rows = None
        del self._view
        self._map.close()
        self._map = None
