"""Host-side logic of the multi-GPU benchmark path, on CPU ranks (gloo, world size 2).

With N GPUs every rank serves its own pool and there is no data-path collective; what the
ranks share is the timing protocol: barrier, device-timed region, MAX over ranks of the
time, SUM over ranks of the units.  That protocol is exercised here without a GPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    # rank r pretends to have needed (10 + 5r) ms for 100 queries
    max_ms, value = bench.aggregate(10.0 + 5.0 * rank, 100.0, world, "cpu")
    out.put((rank, max_ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_aggregate_takes_max_time_and_sums_units_over_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, max_ms, value in res:
        assert max_ms == 15.0                       # the slowest rank
        assert abs(value - 200.0 / 0.015) < 1e-6    # all ranks' queries over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    max_ms, value = bench.aggregate(4.0, 8.0, 1, "cpu")
    assert max_ms == 4.0 and value == 2000.0


def test_reference_arm_on_other_ranks_does_nothing(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        config, nq, steps, warmup, cpu_budget = "C1", 0, 1, 1, 1.0
    bench.run_reference(A)
    assert capsys.readouterr().out == ""


@pytest.mark.parametrize("keys", ["bf16", "e4m3"])
def test_reference_arm_prints_one_contract_line(keys):
    # the reference arm is the CPU oracle timed on the host cores; it needs no GPU
    import json
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference",
                        "--config", "C1", "--steps", "2", "--warmup", "1", "--keys", keys],
                       capture_output=True, text=True, timeout=300, cwd=root)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == "semantic_pool_queries_per_sec"
    assert j["unit"] == "queries/s" and j["higher_is_better"] is True and j["value"] > 0
    assert j["n_gpus"] == 1 and j["steps"] == 2 and j["warmup"] == 1
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1
    assert j["e2e"] == {"value": j["value"], "unit": j["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert "workload" in j["config"] and "model" not in j["config"]
