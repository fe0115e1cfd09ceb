"""Workers spread over ranks (ShardedStep): the gathered message must list the workers of rank 0, then
rank 1, ..., and every rank must end with the x of the single-process step over all workers.

CPU: two gloo ranks, with the oracle standing in for the three CUDA calls so that only the rank logic
is under test.  GPU: one NCCL rank with the real library (the collective runs, over one rank)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


class OracleOps:
    """The three calls of the step on CPU tensors, computed by the oracle (tests only)."""

    @staticmethod
    def alloc_workspace(M, d, K, device):
        return torch.empty(1, dtype=torch.uint8)

    @staticmethod
    def s3gd_topk_sign(grads, K, out_idx, out_signbits, ws):
        from oracle import s3gd_oracle as O
        i, s = O.topk_sign(grads.numpy(), K)
        out_idx.copy_(torch.from_numpy(i.view(np.int32).copy()))
        out_signbits.copy_(torch.from_numpy(s.view(np.int32).copy()))

    @staticmethod
    def s3gd_majority_vote(idx, signbits, M, K, d, out_vote, ws):
        from oracle import s3gd_oracle as O
        v, bad = O.majority_vote(idx.numpy().view(np.uint32), signbits.numpy().view(np.uint32), M, K, d)
        assert bad == 0
        out_vote.copy_(torch.from_numpy(v))

    @staticmethod
    def s3gd_apply(x, vote, lr):
        from oracle import s3gd_oracle as O
        x.copy_(torch.from_numpy(O.apply_vote(x.numpy(), vote.numpy(), lr)))

    @staticmethod
    def s3gd_vote_apply(x, msg, n_groups, group_stride, M_group, K, lr, ws, opt_vote=None):
        from oracle import s3gd_oracle as O
        W = (K + 31) // 32
        m = msg.numpy().view(np.uint32)
        idx = np.concatenate([m[g * group_stride: g * group_stride + M_group * K].reshape(M_group, K) for g in range(n_groups)])
        sgn = np.concatenate([m[g * group_stride + M_group * K: g * group_stride + M_group * (K + W)].reshape(M_group, W)
                              for g in range(n_groups)])
        v, bad = O.majority_vote(idx, sgn, n_groups * M_group, K, x.numel())
        assert bad == 0
        x.copy_(torch.from_numpy(O.apply_vote(x.numpy(), v, lr)))

    @staticmethod
    def s3gd_vote_counts(idx, signbits, M, K, d, out_counts, opt_bad_count=None):
        from oracle import s3gd_oracle as O
        c = O.vote_counts(idx.numpy().view(np.uint32), signbits.numpy().view(np.uint32), M, K, d)
        full = np.zeros(out_counts.numel(), dtype=np.int64)
        full[:d] = c
        if out_counts.dtype == torch.uint8:
            out_counts.copy_(torch.from_numpy((full + 128).astype(np.uint8)))
        else:
            out_counts.copy_(torch.from_numpy(full.astype(np.int32)))

    @staticmethod
    def s3gd_encode_vote2(src, out_words, n_summed=1):
        from oracle import s3gd_oracle as O
        a = src.numpy()
        if src.dtype == torch.uint8:                 # bytes summed modulo 256, each sender added 128
            a = ((a.astype(np.int64) - 128 * n_summed) % 256).astype(np.uint8).view(np.int8)
        vote = np.sign(a.astype(np.int64)).astype(np.int8)
        out_words.copy_(torch.from_numpy(O.encode_vote_2bit(vote).view(np.int32).copy()))

    @staticmethod
    def s3gd_sparse_workspace_bytes(n):
        return 4

    @staticmethod
    def s3gd_encode_vote_sparse(src, out_piece, cap, ws, index_base=0, n_summed=1):
        from oracle import s3gd_oracle as O
        a = src.numpy()
        if src.dtype == torch.uint8:
            a = ((a.astype(np.int64) - 128 * n_summed) % 256).astype(np.uint8).view(np.int8)
        idx, sgn = O.encode_vote_sparse(np.sign(a.astype(np.int64)).astype(np.int8))
        piece = np.zeros(out_piece.numel(), dtype=np.uint32)
        piece[0] = idx.shape[0]
        assert idx.shape[0] <= cap
        piece[1:1 + idx.shape[0]] = idx + np.uint32(index_base)
        piece[1 + cap:1 + cap + sgn.shape[0]] = sgn
        out_piece.copy_(torch.from_numpy(piece.view(np.int32).copy()))

    @staticmethod
    def s3gd_apply_vote_sparse(x, pieces, n_pieces, piece_stride, cap, lr, opt_bad_count=None):
        from oracle import s3gd_oracle as O
        m = pieces.numpy().view(np.uint32)
        vote = np.zeros(x.numel(), dtype=np.int8)
        for p in range(n_pieces):
            piece = m[p * piece_stride:(p + 1) * piece_stride]
            n = int(piece[0])
            part = O.decode_vote_sparse(piece[1:1 + n], piece[1 + cap:1 + cap + (n + 31) // 32], x.numel())
            assert not np.any((vote != 0) & (part != 0))            # the ranges do not overlap
            vote += part
        x.copy_(torch.from_numpy(O.apply_vote(x.numpy(), vote, lr)))

    @staticmethod
    def s3gd_apply_vote2(x, words2, lr, opt_vote=None):
        from oracle import s3gd_oracle as O
        v = O.decode_vote_2bit(words2.numpy().view(np.uint32), x.numel())
        x.copy_(torch.from_numpy(O.apply_vote(x.numpy(), v, lr)))


def _global_problem(world, M_local, d, seed):
    g = torch.Generator().manual_seed(seed)
    grads = torch.randn((world * M_local, d), generator=g)
    grads[:, ::5] = grads[:, 1::5][:, : grads[:, ::5].shape[1]].abs()      # some exact magnitude ties across columns
    x = torch.randn(d, generator=g)
    return grads, x


def _cpu_rank(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200.sharded import ShardedStep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    M_local, d, K, lr = 3, 1003, 37, 0.125
    grads, x = _global_problem(world, M_local, d, 99)
    mine = grads[rank * M_local:(rank + 1) * M_local].contiguous()
    x_ref = x.numpy()
    for _ in range(3):
        x_ref, idx_ref, sgn_ref, _ = O.step(x_ref, grads.numpy(), K, lr)
    ok, ok_rows = True, True
    for downlink in ("replicated", "two_bit", "sparse"):
        st = ShardedStep(M_local, d, K, "cpu", ops=OracleOps, downlink=downlink)
        assert st.M == world * M_local
        if downlink == "replicated":
            assert st.message_bytes_per_rank() == 4 * M_local * (K + 2)
        elif downlink == "two_bit":                 # d = 1003 over 2 ranks: ranges of 512 coordinates (a multiple of 16)
            assert st.range_len == 512 and st.d_padded == 1024 and st.message_bytes_per_rank() == 1024 + 128
        else:                                       # room for min(512, 6 workers x 37) = 222 votes per range
            assert st.sparse_cap == 222 and st.message_bytes_per_rank() == 1024 + 4 * (1 + 222 + 7)
        x_rank = x.clone()
        for _ in range(3):
            st.step(x_rank, mine, lr)
        ok = ok and np.array_equal(x_rank.numpy().view(np.uint32), x_ref.view(np.uint32))
        if downlink == "replicated":                # the gathered message lists rank 0's workers, then rank 1's
            ok_rows = np.array_equal(st.gathered_indices().numpy().view(np.uint32), idx_ref) and \
                np.array_equal(st.gathered_signbits().numpy().view(np.uint32), sgn_ref)
    # ranks that disagree on the shape are refused on every rank
    refused = False
    try:
        ShardedStep(M_local + rank, d, K, "cpu", ops=OracleOps)
    except ValueError:
        refused = True
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{int(ok)} {int(ok_rows)} {int(refused)}")
    dist.destroy_process_group()


def test_two_cpu_ranks_match_the_single_process_step(tmp_path):
    port = 31500 + os.getpid() % 2000
    mp.spawn(_cpu_rank, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert open(tmp_path / f"r{r}.txt").read() == "1 1 1"


@pytest.mark.parametrize("downlink", ["replicated", "two_bit", "sparse"])
def test_without_a_process_group_it_is_the_plain_step(downlink):
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200.sharded import ShardedStep
    grads, x = _global_problem(1, 4, 500, 5)
    st = ShardedStep(4, 500, 20, "cpu", ops=OracleOps, downlink=downlink)
    xr = x.clone()
    st.step(xr, grads, 0.5)
    x_ref, _, _, _ = O.step(x.numpy(), grads.numpy(), 20, 0.5)
    assert np.array_equal(xr.numpy().view(np.uint32), x_ref.view(np.uint32))
    with pytest.raises(ValueError):
        st.step(xr, grads[:2], 0.5)
    with pytest.raises(ValueError):
        ShardedStep(4, 500, 20, "cpu", ops=OracleOps, downlink="carrier pigeon")


def _cpu_rank_many_workers(rank, world, port, out_dir):
    """More than 127 workers in all: the sums travel as int32, not bytes."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200.sharded import ShardedStep
    dist.init_process_group("gloo", rank=rank, world_size=world)
    M_local, d, K, lr = 70, 200, 9, 0.5
    grads, x = _global_problem(world, M_local, d, 7)
    grads[:, 3] = 50.0                               # every one of the 140 workers votes +1 here: beyond a byte
    st = ShardedStep(M_local, d, K, "cpu", ops=OracleOps, downlink="two_bit")
    x_rank = x.clone()
    st.step(x_rank, grads[rank * M_local:(rank + 1) * M_local].contiguous(), lr)
    x_ref, _, _, _ = O.step(x.numpy(), grads.numpy(), K, lr)
    ok = (not st.count_bytes) and np.array_equal(x_rank.numpy().view(np.uint32), x_ref.view(np.uint32))
    dist.barrier()
    with open(os.path.join(out_dir, f"m{rank}.txt"), "w") as f:
        f.write(str(int(ok)))
    dist.destroy_process_group()


def test_two_cpu_ranks_with_more_workers_than_a_byte_counts(tmp_path):
    port = 32500 + os.getpid() % 2000
    mp.spawn(_cpu_rank_many_workers, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert open(tmp_path / f"m{r}.txt").read() == "1"


def _gpu_rank(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200 import workloads as W
    from paper_2302_07475_b200.sharded import ShardedStep
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    s = W.spec("resnet18", d=300_007, M=6)
    grads, x = W.make_grads(s, dev), W.make_x(s, dev)
    K = 3000
    ok = True
    for downlink in ("replicated", "two_bit", "sparse"):
        st = ShardedStep(s.M, s.d, K, dev, downlink=downlink)
        xr = x.clone()
        x_ref = x.cpu().numpy()
        for _ in range(2):
            st.step(xr, grads, s.lr)
            x_ref, idx_ref, sgn_ref, _ = O.step(x_ref, grads.cpu().numpy(), K, s.lr)
        torch.cuda.synchronize()
        ok = ok and np.array_equal(xr.cpu().numpy().view(np.uint32), x_ref.view(np.uint32))
        if downlink == "replicated":
            ok = ok and np.array_equal(st.gathered_indices().cpu().numpy().view(np.uint32), idx_ref) and \
                np.array_equal(st.gathered_signbits().cpu().numpy().view(np.uint32), sgn_ref)
    with open(os.path.join(out_dir, f"g{rank}.txt"), "w") as f:
        f.write(str(int(ok)))
    dist.destroy_process_group()


@pytest.mark.gpu
def test_one_nccl_rank_with_the_cuda_library(tmp_path):
    port = 33500 + os.getpid() % 2000
    mp.spawn(_gpu_rank, args=(1, port, str(tmp_path)), nprocs=1, join=True)
    assert open(tmp_path / "g0.txt").read() == "1"
