"""The N > 1 path of the benchmark on CPU: two `gloo` ranks go through the same barrier /
max-over-ranks / rank-0-prints protocol that `bench.py --gpus N` runs over NCCL, and the reference
arm under a two-rank launcher prints exactly one line."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2601_19278_b200 import replicas
    w, r, local = replicas.env()
    assert (w, r, local) == (world, rank, rank)
    replicas.init(w, "gloo")
    synced = []
    replicas.barrier(w, lambda: synced.append(True))
    assert synced == [True]
    # each rank "measured" a different time for the two timed regions; everyone must end up with the slowest
    mine = [100.0 + 10.0 * rank, 250.0 - 20.0 * rank]
    total_ms, e2e_ms = replicas.max_over_ranks(mine, w)
    value = replicas.job_steps_per_second(w, 50, total_ms)
    replicas.barrier(w)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"total_ms": total_ms, "e2e_ms": e2e_ms, "value": value, "prints": rank == 0}, f)
    replicas.finish(w)


def test_two_gloo_ranks_agree_on_the_slowest_time(tmp_path):
    world, port = 2, 29541
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for g in got:
        assert g["total_ms"] == 110.0 and g["e2e_ms"] == 250.0           # max over ranks of each entry
        assert abs(g["value"] - 2 * 50 / 0.110) < 1e-9                     # whole-job aggregate: both replicas' steps
    assert [g["prints"] for g in got] == [True, False]


def test_single_rank_needs_no_process_group():
    from paper_2601_19278_b200 import replicas
    assert replicas.max_over_ranks([3.0, 4.0], 1) == [3.0, 4.0]
    replicas.barrier(1)
    assert replicas.job_steps_per_second(1, 10, 5.0) == 2000.0
    assert not torch.distributed.is_initialized()


def test_reference_arm_under_a_two_rank_launch_prints_one_line():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", "29543", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1", "--gpus", "2",
           "--steps", "1", "--warmup", "3"]
    out = subprocess.run(cmd, cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, timeout=300)
    assert out.returncode == 0
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                                  # rank 0 alone runs and prints
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["metric"] == "draft_steps_per_second"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
