"""Host logic of bench.py: byte model, whole-job aggregation over ranks (gloo, world size 2)."""
import json
import os
import subprocess
import sys

import synth_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_algorithmic_bytes_match_the_shape_tables():
    import bench
    s7, s13, st = si.SHAPES["7b"], si.SHAPES["13b"], si.SHAPES["tiny"]
    assert bench.verify_weight_bytes(s7) == 2 * 6607077376
    assert bench.verify_weight_bytes(s13) == 2 * 12851609600
    assert bench.verify_weight_bytes(st) == 2 * 2629632
    assert bench.draft_step_bytes(s7) == 2 * 367001600
    assert bench.draft_step_bytes(s13) == 2 * 533463040
    assert bench.kv_bytes_per_token(s7) == 512 * 1024 and bench.kv_bytes_per_token(s13) == 800 * 1024


_WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group(backend="gloo")
r = dist.get_rank()
ms, units = bench.aggregate(dist, 10.0 + 5.0 * r, 100.0 * (r + 1))
if r == 0:
    print(json.dumps({"ms": ms, "units": units}))
dist.barrier()
dist.destroy_process_group()
"""


def test_whole_job_aggregation_over_two_ranks(tmp_path):
    script = tmp_path / "w.py"
    script.write_text(_WORKER % ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res == {"ms": 15.0, "units": 300.0}      # max of the times, sum of the units


def test_reference_arm_prints_its_line_on_tiny():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "8", "--warmup", "1"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    res = json.loads(out.stdout.strip().splitlines()[-1])
    assert res["impl"] == "reference" and res["value"] > 0 and res["cpu_baseline"]["kind"] == "oracle"
    assert res["e2e"]["h2d_bytes_per_step"] == 0
