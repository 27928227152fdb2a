"""Host-side parts of bench.py that need no GPU: the reference arm (the oracle timed on the host cores), the rank
handling of that arm under a multi-rank launch, and the cross-rank reductions used by the replica runs (gloo, 2 ranks)."""
import json
import os
import subprocess
import sys

import pytest

from tests.conftest import ROOT


def _run(args, env_extra=None):
    env = dict(os.environ, **(env_extra or {}))
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=env, cwd=ROOT, capture_output=True,
                          text=True, timeout=600)


def test_reference_arm_prints_one_json_line():
    r = _run(["--impl", "reference", "--workload", "small-gqa-bs1-4k-cpu50", "--steps", "2", "--warmup", "1"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "KV-tokens/s" and d["value"] > 0 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "KV-tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "small-gqa-bs1-4k-cpu50" and d["vs_baseline"] is None
    # both arms describe the workload with the same object, made from the workload's table entry alone
    sys.path.insert(0, ROOT)
    import bench
    assert d["config"] == bench.workload_config("small-gqa-bs1-4k-cpu50", bench.WORKLOADS["small-gqa-bs1-4k-cpu50"])
    assert d["config"]["layers"] >= 1 and "l2" in d["config"]


def test_reference_arm_other_ranks_exit_quietly():
    r = _run(["--impl", "reference", "--workload", "small-gqa-bs1-4k-cpu50", "--steps", "1", "--warmup", "0", "--gpus", "2"],
             {"RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "2"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    mx = bench.reduce_over_ranks(10.0 + rank, "max", "cpu")          # slowest replica's time
    sm = bench.reduce_over_ranks(1000.0 * (rank + 1), "sum", "cpu")  # every replica's work
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, mx, sm))


def test_replica_reductions_two_ranks_gloo():
    import socket
    import torch.multiprocessing as mp
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 11.0, 3000.0), (1, 11.0, 3000.0)]


def test_single_rank_reduction_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5, "max", "cpu") == 3.5 and bench.reduce_over_ranks(7, "sum", "cpu") == 7.0


def test_gpus_flag_without_a_launcher_starts_one_replica_per_gpu():
    """`bench.py --gpus N` with no WORLD_SIZE in the environment spawns the N replicas itself: every rank gets its own
    RANK / LOCAL_RANK, the common WORLD_SIZE and a loopback rendezvous; checked here on the environments and, end to
    end, on the reference arm (rank 0 prints the line, rank 1 stays quiet), which needs no GPU."""
    sys.path.insert(0, ROOT)
    import bench
    envs = bench.replica_envs(3, 29999, base_env={"PATH": "/bin"})
    assert [e["RANK"] for e in envs] == ["0", "1", "2"] and [e["LOCAL_RANK"] for e in envs] == ["0", "1", "2"]
    assert all(e["WORLD_SIZE"] == "3" and e["MASTER_ADDR"] == "127.0.0.1" and e["MASTER_PORT"] == "29999" and e["PATH"] == "/bin" for e in envs)
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "small-gqa-bs1-4k-cpu50",
                        "--steps", "1", "--warmup", "0", "--gpus", "2"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
