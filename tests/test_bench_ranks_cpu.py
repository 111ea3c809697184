"""Host-side multi-rank logic of bench.py on CPU: the max over ranks and the whole-job aggregate with two gloo
ranks, and the reference arm under a two-rank launch (rank 0 alone prints its line, the other rank exits 0)."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, str(ROOT))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow replica
    slowest = bench.max_over_ranks(local_ms, "cpu")
    q.put((rank, slowest, bench.whole_job_gbs(1e9, world, slowest)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    for rank, slowest, gbs in got:
        assert slowest == 15.0                        # every rank sees the slowest rank's time
        assert abs(gbs - 2 * 1e9 / 15e-3 / 1e9) < 1e-9   # two replicas' bytes over that time


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    units = bench.step_units_bytes()
    assert units["compress"] == units["decompress"] == units["fused"] == 4 * bench.N_ELEMS
    per_rank = 4 * bench.N_ELEMS // bench.RANKS
    chunk = per_rank // bench.RANKS
    assert units["allreduce"] == bench.RANKS * chunk * (1 + 2 * (bench.RANKS - 1))


def test_reference_arm_prints_one_line_under_two_ranks():
    port = 29600 + os.getpid() % 300
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "1"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
