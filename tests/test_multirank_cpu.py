"""The N > 1 logic of bench.py on CPU: two gloo ranks.  The data path has no collective
(every rank runs its own replica); what is shared is the timing rule -- barrier, slowest rank's
time, whole-job bytes -- and the rule that only rank 0 reports."""
import io
import json
import os
import socket
from contextlib import redirect_stdout

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        local_ms = 1.0 + rank                       # rank 1 is the slow one
        ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
        out.put((rank, ms, bench.whole_job_gbs(world, ms)))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_gloo():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, gbs in res:
        assert ms == 2.0                            # every rank sees the slowest rank's time
        assert gbs == pytest.approx(2 * bench.step_bytes() / 2.0e-3 / 1e9)


def test_single_rank_passthrough_and_step_bytes():
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.step_bytes() == 29 * 8192 * 8192 * 2            # (8+5+5+5+2+2+2) |T|
    assert bench.whole_job_gbs(1, 1.0) == pytest.approx(bench.step_bytes() / 1e6)


def test_reference_arm_only_rank0_reports(monkeypatch):
    args = type("A", (), {"steps": 1, "warmup": 0, "gpus": 2})()
    monkeypatch.setattr(bench, "oracle_sweep_sample", lambda rows: (1000, 0.5, 1))
    buf = io.StringIO()
    monkeypatch.setenv("RANK", "1")
    with redirect_stdout(buf):
        assert bench.reference_arm(args) == 0
    assert buf.getvalue() == ""
    monkeypatch.setenv("RANK", "0")
    with redirect_stdout(buf):
        assert bench.reference_arm(args) == 0
    line = json.loads(buf.getvalue())
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] == pytest.approx(1000 / 0.5 / 1e9)


def _run_bench(argv, env_extra=None, timeout=300):
    import subprocess
    import sys
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env.update(env_extra or {})
    return subprocess.run([sys.executable, os.path.join(os.path.dirname(bench.__file__), "bench.py")] + argv,
                          capture_output=True, text=True, timeout=timeout, env=env)


def test_gpus_flag_starts_the_ranks_itself_dry_run():
    """`python bench.py --gpus 2` with no launcher around it: the process starts two ranks through
    torch.distributed.run, and rank 0 alone prints one line that claims two ranks."""
    r = _run_bench(["--gpus", "2", "--steps", "3", "--warmup", "1", "--dry-run-cpu"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["world_size"] == 2 and d["dry_run"] is True
    assert d["ms_per_step"] == 2.0                                # the slow rank's stand-in time
    assert d["value"] == pytest.approx(2 * bench.step_bytes() / 2.0e-3 / 1e9)


def test_world_size_that_contradicts_gpus_is_refused():
    r = _run_bench(["--gpus", "4", "--dry-run-cpu"], {"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0",
                                                      "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(_free_port())})
    assert r.returncode == 2
    assert "WORLD_SIZE=2" in r.stderr and r.stdout.strip() == ""
    # the reference arm checks the same thing, and prints n_gpus from the same flag
    r = _run_bench(["--gpus", "4", "--impl", "reference"], {"WORLD_SIZE": "2", "RANK": "0"})
    assert r.returncode == 2


def test_single_process_dry_run_is_one_rank():
    r = _run_bench(["--dry-run-cpu"])
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["n_gpus"] == 1 and d["world_size"] == 1 and d["ms_per_step"] == 1.0
