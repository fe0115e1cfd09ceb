"""Workers spread over several GPUs: the deployment shape of Algorithm 1.

Every rank (one process per GPU) holds the gradients of its own ``M_local`` workers and a replica of x.
Three ways through one step, chosen with ``downlink``:

``"replicated"`` -- the uplink of Section 2.2 is the only exchange.
    1. TopKSign of the local rows into this rank's piece of the message: K uint32 indices and
       ceil(K/32) sign words per worker, 4.125 bytes per kept entry (``s3gd_topk_sign``);
    2. ONE all-gather of the pieces (indices and sign words travel in one buffer);
    3. majority vote over all ``world * M_local`` workers fused with the update, on every rank
       (``s3gd_vote_apply``).  Every rank derives the same vote from the same gathered message, which
       replaces the server's broadcast; the replicas of x stay bit-identical because the vote is
       integer arithmetic on identical inputs.
    Bytes received per rank and step: world * M_local * (4K + 4 ceil(K/32)).  Best while M K << d.

``"two_bit"`` -- the server is split over the ranks by coordinate range, and its answer comes back in
    the dense two-bit form.
    1. TopKSign of the local rows;
    2. vote sums of the local workers over all coordinates (``s3gd_vote_counts``: one byte per
       coordinate while world * M_local <= 127, int32 above);
    3. reduce-scatter (sum) of the sums: rank r receives the totals of coordinate range r;
    4. sign of the totals in two bits per coordinate (``s3gd_encode_vote2``);
    5. all-gather of the ranges' words: d / 4 bytes in all -- the downlink of Section 2.2;
    6. update of x from the words (``s3gd_apply_vote2``).
    Bytes received per rank and step: about d (bytes) or 4d (int32) + d / 4, whatever M and K.
    Best once M K reaches a fraction of d.

``"sparse"`` -- as ``"two_bit"`` up to the reduce-scatter; then every rank lists the non-zero votes of its range
    (``s3gd_encode_vote_sparse``: count, ascending coordinates, one sign bit each -- the form Section 2.2's
    downlink count assumes), the fixed-size pieces are all-gathered and applied (``s3gd_apply_vote_sparse``).
    A piece has room for min(range length, world * M_local * K) votes, which is all a range can receive.
    Smaller than the two-bit form when fewer than about one coordinate in 16 is voted on.

This module is host-side ordering and buffer management; all arithmetic stays in the CUDA library.
``ops`` exists so that the rank logic (buffer layout, order of the gathered pieces, padding of the
coordinate ranges) can be exercised on CPU ranks with other implementations of the calls; the
default is the CUDA binding and there is no fallback.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import binding

DOWNLINKS = ("replicated", "two_bit", "sparse")


class ShardedStep:
    """Buffers and call order for one (M_local, d, K) on one rank of ``group``."""

    def __init__(self, M_local: int, d: int, K: int, device, group: Optional[dist.ProcessGroup] = None, ops=None,
                 downlink: str = "replicated"):
        if M_local <= 0 or d <= 0 or not 0 <= K <= d:
            raise ValueError("need M_local > 0, d > 0, 0 <= K <= d")
        if downlink not in DOWNLINKS:
            raise ValueError(f"downlink must be one of {DOWNLINKS}")
        self.ops = ops if ops is not None else binding
        self.group = group
        self.downlink = downlink
        self.collective = dist.is_available() and dist.is_initialized()     # a 1-rank group still goes through NCCL
        self.world = dist.get_world_size(group) if self.collective else 1
        self.rank = dist.get_rank(group) if self.collective else 0
        self.M_local, self.d, self.K = M_local, d, K
        self.M = self.world * M_local
        self.words = binding.words(K)
        dev = torch.device(device)
        # every rank must use the same shape, or the gathered pieces would not line up
        if self.world > 1:
            shape = torch.tensor([M_local, d, K, DOWNLINKS.index(downlink)], dtype=torch.int64, device=dev)
            lo, hi = shape.clone(), shape.clone()
            dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
            dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
            if not (torch.equal(lo, shape) and torch.equal(hi, shape)):
                raise ValueError("all ranks must be created with the same (M_local, d, K, downlink)")
        self.ws_local = self.ops.alloc_workspace(M_local, d, K, dev)
        # this rank's piece of the message: indices [M_local x K], then sign words [M_local x words]
        self.piece_words = M_local * (K + self.words)
        self.msg_all = torch.empty(max(self.world * self.piece_words, 1), dtype=torch.int32, device=dev)
        mine = self.msg_all[self.rank * self.piece_words:(self.rank + 1) * self.piece_words]
        self.msg_local = mine
        self.idx_local = mine[:M_local * K].view(M_local, K)
        self.sgn_local = mine[M_local * K:].view(M_local, self.words)
        if downlink == "replicated":
            self.ws_all = self.ops.alloc_workspace(self.M, d, K, dev)
        else:
            # coordinate ranges of equal length, a multiple of 16 so that every range is whole words
            self.range_len = ((d + self.world - 1) // self.world + 15) // 16 * 16
            self.d_padded = self.range_len * self.world
            self.count_bytes = self.M <= 127
            cdtype = torch.uint8 if self.count_bytes else torch.int32
            self.counts = torch.empty(self.d_padded, dtype=cdtype, device=dev)
            self.counts_mine = torch.empty(self.range_len, dtype=cdtype, device=dev)
            if downlink == "two_bit":
                self.words2_mine = torch.empty(self.range_len // 16, dtype=torch.int32, device=dev)
                self.words2_all = torch.empty(self.d_padded // 16, dtype=torch.int32, device=dev)
            else:
                self.sparse_cap = max(1, min(self.range_len, self.M * K))
                self.piece2_words = binding.sparse_piece_words(self.sparse_cap)
                self.sparse_mine = torch.empty(self.piece2_words, dtype=torch.int32, device=dev)
                self.sparse_all = torch.empty(self.world * self.piece2_words, dtype=torch.int32, device=dev)
                self.sparse_ws = torch.empty(max(self.ops.s3gd_sparse_workspace_bytes(self.range_len), 4),
                                             dtype=torch.uint8, device=dev)

    def describe(self) -> str:
        if self.downlink == "replicated":
            return "s3gd_topk_sign + one all-gather of the message + s3gd_vote_apply"
        if self.downlink == "sparse":
            return ("s3gd_topk_sign + s3gd_vote_counts + reduce-scatter of the sums + s3gd_encode_vote_sparse + "
                    "all-gather of the sparse vote + s3gd_apply_vote_sparse")
        return ("s3gd_topk_sign + s3gd_vote_counts + reduce-scatter of the sums + s3gd_encode_vote2 + "
                "all-gather of the two-bit vote + s3gd_apply_vote2")

    def message_bytes_per_rank(self) -> int:
        """Bytes each rank contributes to the exchange per step."""
        if self.downlink == "replicated":
            return 4 * self.piece_words
        down = self.range_len // 4 if self.downlink == "two_bit" else 4 * self.piece2_words
        return self.d_padded * (1 if self.count_bytes else 4) + down

    # row r * M_local + m of the gathered message is worker m of rank r
    def gathered_indices(self) -> torch.Tensor:
        """[world * M_local, K] view-free copy of the gathered indices (for inspection and tests)."""
        pieces = self.msg_all[: self.world * self.piece_words].view(self.world, self.piece_words)
        return pieces[:, : self.M_local * self.K].reshape(self.M, self.K)

    def gathered_signbits(self) -> torch.Tensor:
        pieces = self.msg_all[: self.world * self.piece_words].view(self.world, self.piece_words)
        return pieces[:, self.M_local * self.K:].reshape(self.M, self.words)

    def _reduce_scatter_sum(self, out: torch.Tensor, full: torch.Tensor) -> None:
        if not self.collective:
            out.copy_(full[: out.numel()])
            return
        try:
            dist.reduce_scatter_tensor(out, full, op=dist.ReduceOp.SUM, group=self.group)
        except (RuntimeError, NotImplementedError):
            # a backend without reduce-scatter (gloo): the same result from an all-reduce
            tmp = full.clone()
            dist.all_reduce(tmp, op=dist.ReduceOp.SUM, group=self.group)
            out.copy_(tmp[self.rank * out.numel():(self.rank + 1) * out.numel()])

    def step(self, x: torch.Tensor, local_grads: torch.Tensor, lr: float) -> None:
        """x [d] (replica, updated in place) from this rank's local_grads [M_local, d]."""
        if tuple(local_grads.shape) != (self.M_local, self.d) or x.numel() != self.d:
            raise ValueError("shape mismatch with the ShardedStep this was created for")
        self.ops.s3gd_topk_sign(local_grads, self.K, self.idx_local, self.sgn_local, self.ws_local)
        if self.downlink == "replicated":
            if self.collective and self.K > 0:
                dist.all_gather_into_tensor(self.msg_all[: self.world * self.piece_words], self.msg_local, group=self.group)
            self.ops.s3gd_vote_apply(x, self.msg_all, self.world, self.piece_words, self.M_local, self.K, lr, self.ws_all)
            return
        self.ops.s3gd_vote_counts(self.idx_local, self.sgn_local, self.M_local, self.K, self.d, self.counts)
        self._reduce_scatter_sum(self.counts_mine, self.counts)
        if self.downlink == "sparse":
            self.ops.s3gd_encode_vote_sparse(self.counts_mine, self.sparse_mine, self.sparse_cap, self.sparse_ws,
                                             index_base=self.rank * self.range_len, n_summed=self.world)
            if self.collective:
                dist.all_gather_into_tensor(self.sparse_all, self.sparse_mine, group=self.group)
            else:
                self.sparse_all.copy_(self.sparse_mine)
            self.ops.s3gd_apply_vote_sparse(x, self.sparse_all, self.world, self.piece2_words, self.sparse_cap, lr)
            return
        self.ops.s3gd_encode_vote2(self.counts_mine, self.words2_mine, n_summed=self.world)
        if self.collective:
            dist.all_gather_into_tensor(self.words2_all, self.words2_mine, group=self.group)
        else:
            self.words2_all.copy_(self.words2_mine)
        self.ops.s3gd_apply_vote2(x, self.words2_all, lr)
