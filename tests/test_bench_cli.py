"""Command-line behaviour of bench.py that needs no GPU: asking for more GPUs than the node has
must fail loudly instead of quietly running fewer ranks, and a torchrun environment that
contradicts --gpus is refused."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env=None):
    e = dict(os.environ)
    e.pop("WORLD_SIZE", None)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], env=e,
                          capture_output=True, text=True, timeout=300)


def test_more_gpus_than_the_node_has_is_an_error():
    import torch
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    r = _run(["--gpus", str(have + 2), "--steps", "1", "--warmup", "1"])
    assert r.returncode != 0
    assert "refusing to run fewer ranks" in (r.stderr + r.stdout)
    assert "\"metric\"" not in r.stdout


def test_world_size_must_match_gpus():
    r = _run(["--gpus", "1"], env={"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    assert r.returncode != 0 and "contradicts WORLD_SIZE" in (r.stderr + r.stdout)
