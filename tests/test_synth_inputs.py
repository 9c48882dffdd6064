import numpy as np

import synth_inputs as si


def test_weights_are_reproducible_and_have_the_stated_distribution():
    a = si.normal_bf16(si.DEFAULT_SEED, "x", (512, 512))
    b = si.normal_bf16(si.DEFAULT_SEED, "x", (512, 512))
    c = si.normal_bf16(si.DEFAULT_SEED, "y", (512, 512))
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    f = si.bf16_bits_to_f32(a)
    assert abs(f.mean()) < 2e-4 and abs(f.std() - 0.02) < 2e-4
    # counter based: a prefix of a longer tensor is the shorter tensor
    assert np.array_equal(si.normal_bf16(1, "z", (100,)), si.normal_bf16(1, "z", (1000,))[:100])


def test_prompts_and_ragged_lengths():
    sh = si.SHAPES["7b_b8"]
    p = si.make_prompts(sh)
    assert len(p) == 8 and all(128 <= len(x) <= 2048 for x in p)
    assert all(x.min() >= 0 and x.max() < sh.vocab for x in p)
    t = si.make_prompts(si.SHAPES["tiny"])
    assert len(t) == 1 and len(t[0]) == 64


def test_tiny_weight_shapes():
    sh = si.SHAPES["tiny"]
    w = si.make_weights(sh)
    assert w["eagle_fc"].shape == (256, 512) and w["ldlp_w1"].shape == (128, 512) and w["ldlp_w2"].shape == (8, 128)
    assert len(w["wq"]) == 2 and w["w_down"][0].shape == (256, 688)
    assert np.all(si.bf16_bits_to_f32(w["final_norm"]) == 1.0)
