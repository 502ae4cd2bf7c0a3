"""Multi-process host logic of the benchmark on CPU (gloo, world size 2).

The draft head does not shard: `bench.py --gpus N` runs N independent replicas, one process per
GPU, with no collective on the data path.  What the ranks do share is the timing protocol
(barrier on both sides, MAX over ranks of the device time, rank 0 prints) and the reference arm's
rule that only rank 0 works.  Both are exercised here without a GPU.
"""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_info() == (rank, world, rank)
        mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        dist.barrier()
        slowest = bench.max_over_ranks(mine, world, backend_is_gloo=True)
        dist.barrier()
        # whole-job throughput: every rank drafts batch * gamma * steps tokens in the slowest rank's time
        w = bench.WL.WORKLOADS[bench.HEADLINE]
        value = bench.serve_result(None, w, slowest, 7, world)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump({"slowest": slowest, "value": value}, f)
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value_world_size_2(tmp_path):
    world, port = 2, free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    sys.path.insert(0, ROOT)
    import bench
    w = bench.WL.WORKLOADS[bench.HEADLINE]
    for r in res:
        assert r["slowest"] == 15.0                    # MAX over ranks, seen by every rank
        assert r["value"] == pytest.approx(world * w.batch * w.gamma * 7 / 15.0e-3)
    assert bench.max_over_ranks(3.5, 1) == 3.5         # one rank: identity, no process group needed


def test_reference_arm_runs_on_rank_0_only():
    """Under a 2-rank launch the reference arm's rank 1 prints nothing and exits 0."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()))
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line_on_a_small_workload():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1_tiny_fp32", "--steps", "2",
                        "--warmup", "1"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "draft_tokens_per_s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "c1_tiny_fp32" and line["higher_is_better"] is True
    # `config` holds the workload only (what depends on the run sits elsewhere in the line), so the library's arm prints the same object
    sys.path.insert(0, ROOT)
    import bench
    from paper_2505_24544_b200 import workloads as WL
    assert line["config"] == bench.workload_config(WL.WORKLOADS["c1_tiny_fp32"], "single")
    assert set(line["config"]) == {"workload", "batch", "gamma", "ctx", "hidden", "heads", "mlp", "vocab", "step", "l2", "parallelism"}
