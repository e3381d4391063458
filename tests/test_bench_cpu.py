"""What of bench.py and of the binding can be checked without a GPU: the reference arm (the CPU oracle on a
bounded sample) under a two-rank launch, and that the product path refuses to run without CUDA instead of
falling back to anything."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(args, rank=None, world=None):
    env = dict(os.environ)
    if rank is not None:
        env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29533")
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=env, capture_output=True,
                          text=True, timeout=600)


def test_reference_arm_two_ranks():
    """Rank 0 alone runs the oracle and prints the line; the other rank exits 0 without work."""
    args = ["--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "3", "--warmup", "1"]
    r0, r1 = run_bench(args, 0, 2), run_bench(args, 1, 2)
    assert r0.returncode == 0 and r1.returncode == 0
    assert r1.stdout.strip() == ""
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 3 and line["warmup"] == 1
    assert line["value"] > 0 and line["unit"] == "steps/s" and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
    assert line["config"]["workload"] == "tiny"


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour on a machine without a GPU")
def test_product_path_fails_loudly_without_cuda():
    r = run_bench(["--steps", "1", "--warmup", "0"])
    assert r.returncode != 0 and "CUDA" in (r.stderr + r.stdout)
    from paper_2412_00099_b200 import binding as mb
    with pytest.raises(mb.McceError, match="no CUDA device"):
        mb.Engine(L=1, E=8, K=2, J=1, n_shared=0, d=64, I=64, C_cap=4, S=4, lam=0.5)
