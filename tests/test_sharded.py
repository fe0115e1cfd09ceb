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
    M_local, d, K, lr = 3, 1000, 37, 0.125
    grads, x = _global_problem(world, M_local, d, 99)
    mine = grads[rank * M_local:(rank + 1) * M_local].contiguous()
    st = ShardedStep(M_local, d, K, "cpu", ops=OracleOps)
    assert st.M == world * M_local and st.message_bytes_per_rank() == 4 * M_local * (K + 2)
    x_rank = x.clone()
    for _ in range(3):
        st.step(x_rank, mine, lr)
    x_ref = x.numpy()
    for _ in range(3):
        x_ref, idx_ref, sgn_ref, _ = O.step(x_ref, grads.numpy(), K, lr)
    ok = np.array_equal(x_rank.numpy().view(np.uint32), x_ref.view(np.uint32))
    ok_rows = np.array_equal(st.idx_all.numpy().view(np.uint32), idx_ref) and \
        np.array_equal(st.sgn_all.numpy().view(np.uint32), sgn_ref)
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


def test_without_a_process_group_it_is_the_plain_unfused_step():
    from oracle import s3gd_oracle as O
    from paper_2302_07475_b200.sharded import ShardedStep
    grads, x = _global_problem(1, 4, 500, 5)
    st = ShardedStep(4, 500, 20, "cpu", ops=OracleOps)
    xr = x.clone()
    st.step(xr, grads, 0.5)
    x_ref, _, _, _ = O.step(x.numpy(), grads.numpy(), 20, 0.5)
    assert np.array_equal(xr.numpy().view(np.uint32), x_ref.view(np.uint32))
    with pytest.raises(ValueError):
        st.step(xr, grads[:2], 0.5)


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
    st = ShardedStep(s.M, s.d, K, dev)
    x_ref = x.cpu().numpy()
    for _ in range(2):
        st.step(x, grads, s.lr)
        x_ref, idx_ref, sgn_ref, _ = O.step(x_ref, grads.cpu().numpy(), K, s.lr)
    torch.cuda.synchronize()
    ok = np.array_equal(x.cpu().numpy().view(np.uint32), x_ref.view(np.uint32)) and \
        np.array_equal(st.idx_all.cpu().numpy().view(np.uint32), idx_ref) and \
        np.array_equal(st.sgn_all.cpu().numpy().view(np.uint32), sgn_ref)
    with open(os.path.join(out_dir, f"g{rank}.txt"), "w") as f:
        f.write(str(int(ok)))
    dist.destroy_process_group()


@pytest.mark.gpu
def test_one_nccl_rank_with_the_cuda_library(tmp_path):
    port = 33500 + os.getpid() % 2000
    mp.spawn(_gpu_rank, args=(1, port, str(tmp_path)), nprocs=1, join=True)
    assert open(tmp_path / "g0.txt").read() == "1"
