"""The N > 1 path of the benchmark on CPU: the drafter's hot path does not shard (no data-path collective), so
N GPUs run N replicas and the only cross-rank step is the measurement's max-over-ranks. Two gloo ranks check
that aggregation, and that the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms, value = bench.replica_aggregate(local_ms, units_per_rank=6.0)
    dist.barrier()
    out.put((rank, ms, value))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_sum_of_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in got:
        assert ms == 15.0                               # max over ranks
        assert abs(value - 2 * 6.0 / 15e-3) < 1e-6      # both replicas' units over the slowest time


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    ms, value = bench.replica_aggregate(4.0, 6.0)
    assert ms == 4.0 and abs(value - 1500.0) < 1e-9


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line_on_the_small_workload():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "draft_tree_steps_per_sec" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
