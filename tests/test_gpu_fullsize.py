"""Full-size GPU parity (7B / 13B shapes, through the C ABI, in the configuration bench.py times) against
stored oracle trajectories.  The goldens are written by tests/golden/make_goldens.py from the CPU oracle only;
each holds the first token and a bounded number of lock-step iterations with every margin needed to decide
which positions are exempt.  Weights and prompts are regenerated from the seed."""
import json
import os

import numpy as np
import pytest
import torch

import synth_inputs as si
from tests import lockstep

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    path = os.path.join(GOLDEN, name + ".json")
    if not os.path.exists(path):
        pytest.skip("golden %s.json not generated yet" % name)
    return json.load(open(path))


@pytest.fixture(scope="module")
def w7b():
    return si.make_weights(si.SHAPES["7b"])


def _run(sh, weights, golden, batch, **kw):
    from paper_2412_18910_b200 import Engine
    prompts = si.make_prompts(sh)
    assert [len(p) for p in prompts] == golden["prompt_lens"]
    e = Engine(sh, weights, max_batch=batch, kv_capacity=sh.kv_capacity)
    try:
        for b, p in enumerate(prompts):
            first = e.prefill(b, p)
            assert first == golden["seqs"][b]["first"], "first token of sequence %d differs from the oracle's" % b
        streams = [s.get("greedy") for s in golden["seqs"]] if kw.pop("teacher", False) else None
        res = lockstep.run_golden(e, golden, prompts, greedy_streams=streams, **kw)
        c = e.ada_get_counters()
    finally:
        e.close()
    assert c["status"] == 0
    assert not res["failures"], res["failures"]
    assert res["exempt"] <= max(1, res["iterations"] // 3)
    print("iterations %d exempt %d max top-1 logit diff %.4f" % (res["iterations"], res["exempt"], res["max_top1_diff"]))
    return res


def test_7b_predictor_lengths(w7b):
    _run(si.SHAPES["7b"], w7b, _golden("7b"), 1)


def test_7b_teacher_forced_every_length(w7b):
    g = _golden("7b_tf")
    sh = si.SHAPES["7b_tf"]
    sched = [n for n in range(1, sh.n_max + 1) for _ in range(2)]
    res = _run(sh, w7b, g, 1, forced_n_schedule=sched, teacher=True)
    assert all(it["k"] == it["n"] for it in g["seqs"][0]["iters"])   # the oracle accepted every forced draft
    assert res["exempt"] <= 2


def test_13b_predictor_lengths():
    g = _golden("13b")
    sh = si.SHAPES["13b"]
    _run(sh, si.make_weights(sh), g, 1)


def test_7b_batch8_ragged(w7b):
    g = _golden("7b_b8")
    _run(si.SHAPES["7b_b8"], w7b, g, 8)


@pytest.mark.parametrize("name", ["7b", "13b"])
def test_full_width_two_layers_against_the_live_oracle(name):
    """Full matrix widths (slab heights, K-split pairs, ring stage sizes of the real shapes) with two layers, so that
    the oracle runs live: prefill with a ragged last chunk, lock-step iterations, and the same pass twice in two
    engines must give bit-identical features (no schedule-dependent result)."""
    import oracle
    from paper_2412_18910_b200 import Engine
    sh = si.scaled(si.SHAPES[name], n_layers=2)
    w = si.make_weights(sh)
    prompt = si.make_prompts(sh)[0][:40]
    m = oracle.Model(sh, w)
    feats = []
    for rep in range(2):
        e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity)
        try:
            seq = m.new_seq(512)
            t_o = seq.prefill(prompt)
            t_g = e.prefill(0, prompt)
            f = e.ada_debug_buffer(0, torch.float32, (1, sh.kv_capacity, sh.d_model))[0, :len(prompt)].cpu().numpy()
            assert np.abs(f - seq.features(0, len(prompt))).max() < 2e-2
            assert t_o == t_g
            feats.append(f)
            res = lockstep.run_lockstep(e, [seq], 8)
            assert e.ada_get_counters()["status"] == 0
        finally:
            e.close()
        assert not res["failures"], res["failures"]
        assert res["exempt"] <= 2
    assert np.array_equal(feats[0], feats[1])


def test_full_width_ddd_stopping_rule_against_the_live_oracle():
    """Section 4 (AdaEAGLE-DDD) at the 7B widths and vocabulary (two layers): the log-probabilities come from the
    LM-head phase of the draft pass, the length from the device-side rule."""
    import oracle
    from paper_2412_18910_b200 import Engine
    sh = si.scaled(si.SHAPES["7b"], n_layers=2)
    w = si.make_weights(sh)
    prompt = si.make_prompts(sh)[0][:40]
    thr = -22.0
    m = oracle.Model(sh, w, ddd_threshold=thr)
    e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity, ddd_threshold=thr)
    try:
        seq = m.new_seq(512)
        assert seq.prefill(prompt) == e.prefill(0, prompt)
        e.ada_force_n([1])
        res = lockstep.run_lockstep(e, [seq], 8, n_forced=1, ddd=thr)
        assert e.ada_get_counters()["status"] == 0
        c = e.ada_get_counters()
    finally:
        e.close()
    assert not res["failures"], res["failures"]
    assert res["exempt"] <= 2
    assert c["n_draft"] > c["n_target"]          # drafts did grow past n = 1
