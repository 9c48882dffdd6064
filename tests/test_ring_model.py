"""The weight ring of the pass kernel, modelled on the host: the header the kernel's producer threads run
(csrc/ada_ring.h) is compiled with g++ and driven over stage-size sequences of the shapes in use and of
awkward ones (sizes that fill the ring exactly, leave a tail, change from phase to phase)."""
import os
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2412_18910_b200", "csrc")


@pytest.fixture(scope="module")
def model(tmp_path_factory):
    exe = str(tmp_path_factory.mktemp("ring") / "ring_model")
    subprocess.check_call(["g++", "-O2", "-std=c++17", "-I", CSRC, "-o", exe, os.path.join(ROOT, "tests", "ring_model.cpp")])
    return exe


def _stage(rows, boxes_per_stage):
    return ((rows + 7) // 8) * 8 * 128 * boxes_per_stage


SEQUENCES = {
    # per layer: QKV, O, gate/up, down (stage bytes : stages per CTA)
    "7b pairs": [(_stage(84, 2), 32), (_stage(56, 4), 8), (_stage(75, 2), 64), (_stage(56, 4), 22)],
    "13b pairs": [(_stage(105, 2), 40), (_stage(70, 2), 20), (_stage(94, 2), 80), (_stage(70, 2), 54)],
    "7b no K split": [(_stage(84, 2), 32), (_stage(28, 4), 16), (_stage(75, 2), 64), (_stage(28, 4), 43)],
    "7b groups of 4": [(_stage(84, 2), 32), (_stage(111, 2), 8), (_stage(75, 2), 64), (_stage(111, 2), 22)],
    "fills the ring exactly": [(16384, 8), (32768, 5), (16384, 3)],
    "tail of 1 KB": [(1024 * 127 // 4 // 1024 * 1024, 9), (31744, 3), (1024, 40)],
    "small then large": [(1024, 33), (32768, 3), (2048, 17), (9216, 11), (4096, 7), (18432, 13)],
}


@pytest.mark.parametrize("name", sorted(SEQUENCES))
def test_no_stage_is_written_over_an_unread_one(model, name):
    spec = ",".join("%d:%d" % sc for sc in SEQUENCES[name])
    r = subprocess.run([model, spec, "40"], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert r.stdout.startswith("ok")
