"""bench.py --gpus N starts N ranks by itself (torchrun on 127.0.0.1) when it is not already inside one.
Covered here without a GPU: the stub arm runs the timing protocol's barrier and max/sum reductions on two
gloo ranks, and the real arm, started the same way on a box without a CUDA device, ends every rank with
the "needs a CUDA device" message instead of computing anything on the CPU."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BENCH = os.path.join(ROOT, "bench.py")


def _env():
    env = dict(os.environ)
    for name in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(name, None)
    return env


def test_gpus_2_spawns_two_ranks_and_reduces_over_them():
    out = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--impl", "stub"], capture_output=True, text=True,
                         env=_env(), timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # rank 0 alone prints
    assert lines[0]["impl"] == "stub" and lines[0]["n_gpus"] == 2
    assert lines[0]["ranks_seen"] == 2.0 and lines[0]["max_over_ranks"] == 2.0


def test_real_arm_has_no_cpu_fallback_when_spawned():
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    out = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--steps", "1"], capture_output=True, text=True,
                         env=_env(), timeout=300)
    assert out.returncode != 0
    assert "needs a CUDA device" in out.stderr
    assert not any(l.startswith("{") for l in out.stdout.splitlines())


def test_inside_torchrun_no_second_spawn():
    # with WORLD_SIZE already set (the driver's torchrun launch) main() must not start ranks again
    sys.path.insert(0, ROOT)
    import bench
    calls = []
    old_spawn, old_stub = bench.spawn_ranks, bench.run_stub
    bench.spawn_ranks = lambda n, argv: calls.append(("spawn", n)) or 0
    bench.run_stub = lambda args: calls.append(("stub", args.gpus)) or 0
    old = os.environ.get("WORLD_SIZE")
    try:
        os.environ["WORLD_SIZE"] = "2"
        assert bench.main(["--gpus", "2", "--impl", "stub"]) == 0
        os.environ.pop("WORLD_SIZE")
        assert bench.main(["--gpus", "2", "--impl", "stub"]) == 0
    finally:
        bench.spawn_ranks, bench.run_stub = old_spawn, old_stub
        if old is None:
            os.environ.pop("WORLD_SIZE", None)
        else:
            os.environ["WORLD_SIZE"] = old
    assert calls == [("stub", 2), ("spawn", 2)]
