"""Host-side logic of the N > 1 benchmark path, on CPU with the gloo backend (world size 2).

The GEMM shards by rows with no data-path collective; what ranks exchange is timing only:
a barrier, a max over ranks, and the aggregation of the whole-job figure on rank 0.
"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2511_16041_b200 import inputs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # per-rank operands: different rows of A, the same B everywhere
        a = inputs.make_A("normal", 8, 64, bench.rank_seed(inputs.BASE_SEED, rank))
        b = inputs.make_B_bits(64, 8)
        mine = [10.0 + rank, 2.0 - rank, 5.0, 1.0 + 3 * rank]
        dist.barrier()
        got = bench.max_over_ranks(mine, torch.device("cpu"), world)
        res = {"rank": rank, "max": got, "a_sum": float(a.astype("float64").sum()), "b_sum": int(b.astype("int64").sum()),
               "value": bench.aggregate_tflops(1e12, world, got[0])}
        with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
            json.dump(res, f)
    finally:
        dist.destroy_process_group()


def test_two_rank_timing_reduction(tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r = [json.load(open(tmp_path / f"r{i}.json")) for i in range(world)]
    assert r[0]["max"] == r[1]["max"] == [11.0, 2.0, 5.0, 4.0]
    assert r[0]["a_sum"] != r[1]["a_sum"]             # different rows per rank
    assert r[0]["b_sum"] == r[1]["b_sum"]             # B replicated
    # whole-job figure: both ranks' work in the slowest rank's time
    assert abs(r[0]["value"] - 2 * 1e12 / 11e-3 / 1e12) < 1e-9


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_single_rank_helpers():
    import bench
    assert bench.max_over_ranks([3.0, 1.0], torch.device("cpu"), 1) == [3.0, 1.0]
    assert bench.rank_seed(7, 0) == 7 and bench.rank_seed(7, 3) == 10
    assert bench.aggregate_tflops(2.0 * 8192 ** 3, 1, 1.0) == 2.0 * 8192 ** 3 / 1e-3 / 1e12


def test_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself; with the stub step
    (gloo, no GPU work) the line rank 0 prints carries the world size and the slowest rank's time."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--stub-step"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                 # rank 0 alone prints
    assert lines[0]["stub"] is True and lines[0]["n_gpus"] == 2
    assert lines[0]["ms_per_step"] == 2.0                  # max over ranks of (1 + rank)
    assert abs(lines[0]["value"] - 2 * 1e9 / 2e-3 / 1e12) < 1e-12
