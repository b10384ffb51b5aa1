"""Host-side logic of bench.py that needs no GPU: the multi-rank aggregation (two gloo ranks on CPU), the
reference arm's JSON contract on a cut-down shape, and the algorithmic byte count."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    # rank r measured (10 + r) ms for 100 * (r + 1) tokens with 7 launches
    times, counts = bench.aggregate_over_ranks(dist, [10.0 + rank, 20.0 - rank], [100 * (rank + 1), 5, 7], "cpu")
    dist.barrier()
    q.put((rank, times, counts))
    dist.destroy_process_group()


def test_replica_aggregation_takes_slowest_time_and_total_work():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, times, counts in got:
        assert times == [11.0, 20.0]          # max over ranks
        assert counts == [300, 10, 14]        # sum over ranks


def test_algorithmic_bytes_of_the_llama_shape():
    w, kv = bench.algorithmic_bytes(synth.LLAMA3_8B, 1024, 68)
    assert w == 15_009_316_864                # every layer matrix + LM head once, bf16
    assert kv == (1024 + 68) * 32 * 2 * 8 * 128 * 2


def test_reference_arm_prints_the_contract_line():
    """`--impl reference` on rank != 0 prints nothing and exits 0; on rank 0 it prints one JSON line."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_runs_whole_steps_and_reports_what_it_ran():
    """Rank 0 of `--impl reference` on a one-layer cut of the shape: the line carries the contract's keys, the
    `config` object has exactly the keys and values the GPU arm prints for the same workload, and steps x
    ms_per_step is the time the steps really took (nothing extrapolated)."""
    import time
    t0 = time.time()
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--layers", "1",
                          "--steps", "2", "--warmup", "0"], env=dict(os.environ, RANK="0", WORLD_SIZE="1"),
                         capture_output=True, text=True, timeout=600)
    wall = time.time() - t0
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["steps"] == 2 and line["warmup"] == 0 and line["higher_is_better"] is True
    assert line["config"] == bench.workload_config("llama3-8b", 1024, 1, 0.0, 4, 10, 64, 68, 1)
    assert line["steps"] * line["ms_per_step"] * 1e-3 < wall
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
