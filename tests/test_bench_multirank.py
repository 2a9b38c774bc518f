"""The N>1 path of the benchmark on CPU: two gloo ranks go through the same rendezvous,
barrier, max-over-ranks and whole-job aggregation code as the NCCL run (replicas only: the
path has no exchange step, so there is nothing else to distribute)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run(nproc):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()),
           os.path.join(ROOT, "bench.py"), "--gpus", str(nproc), "--steps", "4", "--warmup", "3", "--dry-run"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=240, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout            # rank 0 alone prints the JSON line
    return json.loads(lines[0])


def test_two_gloo_ranks_aggregate_as_replicas():
    j = _run(2)
    assert j["n_gpus"] == 2 and j["scaling"] == "weak"
    # ranks took 100 and 150 ms per step; the job is as slow as the slowest rank and moved 2x the bytes
    assert abs(j["ms_per_step"] - 150.0) < 1e-9
    assert abs(j["value"] - 2 * 1e9 / 0.150 / 1e9) < 1e-9


def test_single_process_dry_run():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--dry-run", "--steps", "2"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    j = json.loads(out.stdout.strip().splitlines()[-1])
    assert j["n_gpus"] == 1 and abs(j["value"] - 1e9 / 0.100 / 1e9) < 1e-9


def test_plain_invocation_with_gpus_2_starts_its_own_two_ranks():
    """`python bench.py --gpus 2` as the driver calls it, without a launcher around it."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "4", "--warmup", "3"],
                         capture_output=True, text=True, timeout=240, cwd=ROOT,
                         env={k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")})
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout
    j = json.loads(lines[0])
    assert j["n_gpus"] == 2 and abs(j["ms_per_step"] - 150.0) < 1e-9


def test_a_failing_extra_is_reported_and_the_rest_skipped(monkeypatch):
    """bench.py's secondary workloads run after the headline numbers are taken: one that raises
    must leave a record beside the others' results instead of losing the line."""
    import argparse
    import importlib
    import types
    sys.path.insert(0, ROOT)
    bench = importlib.import_module("bench")

    def ok(args, tc, torch, stream, out):
        out["first"] = 1

    def boom(args, tc, torch, stream, out):
        raise RuntimeError("an illegal memory access was encountered")

    def never(args, tc, torch, stream, out):
        out["third"] = 3

    monkeypatch.setattr(bench, "EXTRAS", [("a", ok), ("b", boom), ("c", never)])
    fake_torch = types.SimpleNamespace(cuda=types.SimpleNamespace(empty_cache=lambda: None))
    args = argparse.Namespace(extras="all", only_kv_shapes=False, only_misaligned=False)
    out = bench.run_extras(args, None, fake_torch, None)
    assert out["first"] == 1 and "third" not in out
    assert out["FAILED"]["extra"] == "b" and out["FAILED"]["skipped_after_it"] == ["c"] and "illegal memory access" in out["FAILED"]["error"]
