"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job value,
and the reference arm's rule that only rank 0 works."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slow one: both ranks must see its time
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 100.0 - rank], dist, torch.device("cpu"))
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "e2e": e2e, "value": bench.whole_job_value(world, 4, 1000, 10, ms)}, f)
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(2)]
    for r in res:
        assert r["ms"] == 15.0 and r["e2e"] == 100.0
        # 2 replicas x 4 x 1000 elements x 10 steps in 15 ms
        assert abs(r["value"] - 2 * 4 * 1000 * 10 / 0.015) < 1e-6


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks([3.5, 0.0], None, torch.device("cpu")) == [3.5, 0.0]
    assert bench.whole_job_value(1, 100, 11_173_962, 1, 1.0) == 100 * 11_173_962 / 1e-3


def test_byte_models():
    import bench
    b = bench.byte_models(100, 11_173_962, 11_174)
    g = b["grad"]
    msg = 2 * 100 * (4 * 11_174 + 4 * 350)
    assert g == 4 * 100 * 11_173_962
    assert b["dense"] == g + msg + 10 * 11_173_962      # byte counters: 2d + x: 8d
    assert b["json"] == g + msg + 16 * 11_173_962       # int32 counters: 8d + x: 8d
    assert b["moved"] == g + 10 * 11_173_962            # no message in the fused step
    assert bench.byte_models(128, 1000, 10)["dense"] == 4 * 128 * 1000 + 2 * 128 * (40 + 4) + 16 * 1000
    assert b["min"] == g + 8 * 100 * 11_174
    # the published table's figures for the headline shape (GB, three decimals)
    assert round(b["json"] / 1e9, 3) == 4.658 and round(b["min"] / 1e9, 3) == 4.479
    f = bench.fractions(b, 1.0, 6457.4)
    assert abs(f["json"]["GBps"] - b["json"] / 1e6) < 1e-6 and abs(f["json"]["of_8TBps"] - f["json"]["GBps"] / 8000) < 1e-12


def test_repeats_cover_about_a_second():
    import bench
    assert bench.pick_repeats(7, 20, 0.76) == 7                 # asked for
    assert bench.pick_repeats(0, 20, 0.76) == 50                # 20 x 0.76 ms regions: capped
    assert bench.pick_repeats(0, 300, 0.76) == 5                # long regions: the floor
    assert bench.pick_repeats(0, 5, 12.0) == 17


def test_make_rows_matches_make_grads():
    from paper_2302_07475_b200 import workloads as W
    s = W.spec("resnet18", d=5_003, M=6)
    full = W.make_grads(s, "cpu")
    assert torch.equal(W.make_rows(s, [4, 1], "cpu"), full[[4, 1]])


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
