"""bench.py pieces that need no GPU: the CPU-oracle arm, and the multi-rank plumbing over gloo."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT


def _run(cmd, **kw):
    return subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600, **kw)


def test_reference_arm_prints_one_contract_line():
    r = _run([sys.executable, "bench.py", "--impl", "reference", "--workload", "tiny", "--steps", "50", "--warmup", "3"])
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "transitions/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 50 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["config"]["workload"] == "tiny"


def test_reference_arm_under_torchrun_two_ranks():
    # launched the way a multi-GPU run is: rank 0 alone works and prints, rank 1 exits 0 silently
    r = _run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
              "127.0.0.1", "--master-port", "29541", "bench.py", "--impl", "reference", "--gpus", "2", "--workload", "tiny",
              "--steps", "20", "--warmup", "2"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2


def test_gpus_flag_launches_the_ranks_itself():
    # `python bench.py --gpus 2` outside any launcher starts two ranks itself; the one line says n_gpus 2
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = _run([sys.executable, "bench.py", "--gpus", "2", "--impl", "reference", "--workload", "tiny", "--steps", "20",
              "--warmup", "2"], env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    got = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))       # each rank's own "time"
    out.put((rank, got))
    dist.barrier()
    dist.destroy_process_group()


def test_time_is_max_over_ranks_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, 29543, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 15.0, 1: 15.0}


def test_sweep_grid_is_the_stated_one():
    # capacity x fanout x batch, batches above half the capacity left out: 140 cells
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    cells = [(n, k, b) for n in bench.SWEEP_CAPACITIES for k in bench.SWEEP_FANOUTS for b in bench.SWEEP_BATCHES if b <= n // 2]
    assert len(cells) == 140
    assert bench.SWEEP_CAPACITIES[0] == 1 << 16 and bench.SWEEP_CAPACITIES[-1] == 1 << 26
    assert bench.SWEEP_FANOUTS == [2, 4, 16, 32] and max(bench.SWEEP_BATCHES) == 65536
