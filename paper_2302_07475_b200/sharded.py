"""Workers spread over several GPUs: the deployment shape of Algorithm 1.

Every rank (one process per GPU) holds the gradients of its own ``M_local`` workers and a replica of x.
One step is

1. TopKSign of the local rows                      (``s3gd_topk_sign``, CUDA),
2. all-gather of the message over the ranks         (the uplink of Section 2.2: per worker K uint32
   indices and ceil(K/32) sign words, 4.125 bytes per kept entry; NCCL),
3. majority vote over all ``world * M_local`` workers and the update of x, replicated on every rank
   (``s3gd_majority_vote`` + ``s3gd_apply``), which replaces the server's broadcast of the vote: every
   rank derives the same vote from the same gathered message, so the replicas of x stay bit-identical.

Only the exchange in step 2 crosses GPUs.  This module is host-side ordering and buffer management;
all arithmetic stays in the CUDA library.  ``ops`` exists so that the rank logic (buffer layout,
row order of the gathered message) can be exercised on CPU ranks with other implementations of the
three calls; the default is the CUDA binding and there is no fallback.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import binding


class ShardedStep:
    """Buffers and call order for one (M_local, d, K) on one rank of ``group``."""

    def __init__(self, M_local: int, d: int, K: int, device, group: Optional[dist.ProcessGroup] = None, ops=None):
        if M_local <= 0 or d <= 0 or not 0 <= K <= d:
            raise ValueError("need M_local > 0, d > 0, 0 <= K <= d")
        self.ops = ops if ops is not None else binding
        self.group = group
        self.collective = dist.is_available() and dist.is_initialized()     # a 1-rank group still goes through NCCL
        self.world = dist.get_world_size(group) if self.collective else 1
        self.rank = dist.get_rank(group) if self.collective else 0
        self.M_local, self.d, self.K = M_local, d, K
        self.M = self.world * M_local
        self.words = binding.words(K)
        dev = torch.device(device)
        # every rank must use the same shape, or the gathered rows would not line up
        if self.world > 1:
            shape = torch.tensor([M_local, d, K], dtype=torch.int64, device=dev)
            lo, hi = shape.clone(), shape.clone()
            dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
            dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
            if not (torch.equal(lo, shape) and torch.equal(hi, shape)):
                raise ValueError("all ranks must be created with the same (M_local, d, K)")
        self.ws_local = self.ops.alloc_workspace(M_local, d, K, dev)
        self.ws_all = self.ops.alloc_workspace(self.M, d, K, dev)
        self.idx_local = torch.empty((M_local, K), dtype=torch.int32, device=dev)
        self.sgn_local = torch.empty((M_local, self.words), dtype=torch.int32, device=dev)
        # row r * M_local + m of the gathered message is worker m of rank r
        if self.collective:
            self.idx_all = torch.empty((self.M, K), dtype=torch.int32, device=dev)
            self.sgn_all = torch.empty((self.M, self.words), dtype=torch.int32, device=dev)
        else:
            self.idx_all, self.sgn_all = self.idx_local, self.sgn_local
        self.vote = torch.empty(d, dtype=torch.int8, device=dev)

    def message_bytes_per_rank(self) -> int:
        """Bytes each rank contributes to the all-gather per step."""
        return 4 * self.M_local * (self.K + self.words)

    def step(self, x: torch.Tensor, local_grads: torch.Tensor, lr: float) -> None:
        """x [d] (replica, updated in place) from this rank's local_grads [M_local, d]."""
        if tuple(local_grads.shape) != (self.M_local, self.d) or x.numel() != self.d:
            raise ValueError("shape mismatch with the ShardedStep this was created for")
        self.ops.s3gd_topk_sign(local_grads, self.K, self.idx_local, self.sgn_local, self.ws_local)
        if self.collective and self.K > 0:
            dist.all_gather_into_tensor(self.idx_all, self.idx_local, group=self.group)
            dist.all_gather_into_tensor(self.sgn_all, self.sgn_local, group=self.group)
        self.ops.s3gd_majority_vote(self.idx_all, self.sgn_all, self.M, self.K, self.d, self.vote, self.ws_all)
        self.ops.s3gd_apply(x, self.vote, lr)
