"""Pins for the CPU oracle: each test ties one part of it to something that is not the oracle."""
import os

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import torch_ref as tr

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- target forward

def test_target_matches_stock_op_restatement(tiny):
    sh, w, prompt, m = tiny
    logits, feat = m.forward_nocache(prompt, want_features=True)
    ref_f = tr.target_features(w, sh, prompt)
    ref_l = ref_f[-1] @ tr.t64(w["lm_head"]).T
    assert np.abs(feat - ref_f.numpy()).max() < 2e-5
    assert np.abs(logits - ref_l.numpy()).max() < 2e-5


def test_target_matches_library_llama(tiny):
    tf = pytest.importorskip("transformers")
    sh, w, prompt, m = tiny
    cfg = tf.LlamaConfig(vocab_size=sh.vocab, hidden_size=sh.d_model, intermediate_size=sh.d_ffn,
                         num_hidden_layers=sh.n_layers, num_attention_heads=sh.n_heads,
                         num_key_value_heads=sh.n_heads, head_dim=sh.head_dim, rms_norm_eps=sh.rms_eps,
                         rope_theta=sh.rope_theta, attention_bias=False, mlp_bias=False,
                         tie_word_embeddings=False, max_position_embeddings=4096)
    hf = tf.LlamaForCausalLM(cfg).float().eval()
    f32 = lambda a: torch.from_numpy(si.bf16_bits_to_f32(a).copy())
    sd = {"model.embed_tokens.weight": f32(w["embed"]), "lm_head.weight": f32(w["lm_head"]),
          "model.norm.weight": f32(w["final_norm"])}
    names = dict(wq="self_attn.q_proj", wk="self_attn.k_proj", wv="self_attn.v_proj", wo="self_attn.o_proj",
                 w_gate="mlp.gate_proj", w_up="mlp.up_proj", w_down="mlp.down_proj",
                 norm_attn="input_layernorm", norm_mlp="post_attention_layernorm")
    for l in range(sh.n_layers):
        for k, v in names.items():
            sd["model.layers.%d.%s.weight" % (l, v)] = f32(w[k][l])
    res = hf.load_state_dict(sd, strict=False)
    assert not [k for k in res.missing_keys if "rotary" not in k]
    ids = torch.from_numpy(prompt.astype(np.int64))[None]
    with torch.no_grad():
        ref_logits = hf(ids).logits[0, -1].numpy()
        ref_feat = hf.model(ids).last_hidden_state[0].numpy()
    logits, feat = m.forward_nocache(prompt, want_features=True)
    assert np.abs(logits - ref_logits).max() < 1e-4
    assert np.abs(feat - ref_feat).max() < 1e-4


def test_cached_path_equals_cache_free_recompute(tiny):
    """Prefill + multi-row verifies through the caches == one pass over the whole sequence."""
    sh, w, prompt, m = tiny
    seq = m.new_seq(256)
    seq.prefill(prompt[:40])
    for n in (3, 0, 8, 1):
        forced = si.uniform_ids(7, "junk%d" % n, max(n, 1), sh.vocab)[:n]
        tt, _, _, _ = seq.verify(forced)
        seq.accept(forced, np.concatenate([forced, tt[-1:]]))  # accept everything: rows all stay
    toks = seq.tokens()
    n_cached = seq.len - 1
    _, feat = m.forward_nocache(toks[:n_cached], want_features=True)
    got = seq.features(0, n_cached)
    assert np.array_equal(got, feat), np.abs(got - feat).max()


# ----------------------------------------------------------------- lossless property

@pytest.mark.parametrize("policy", [-1, 1, 2, 3, 5, 8])
def test_speculative_tokens_equal_greedy_decoding(tiny, policy):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, sh.max_new, n_policy=0)
    sd = oracle.decode(m, prompt, sh.max_new, n_policy=policy)
    assert np.array_equal(ar["tokens"], sd["tokens"])
    assert all(1 <= it["n"] <= sh.n_max for it in sd["iters"])


def test_greedy_decoding_is_argmax_of_cache_free_logits(tiny):
    """Brute force: every emitted token is the argmax of a from-scratch pass over its prefix."""
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 6, n_policy=0)
    toks = list(prompt)
    for t in ar["tokens"]:
        logits, _ = m.forward_nocache(np.array(toks, dtype=np.int32))
        assert int(np.argmax(logits)) == int(t)
        toks.append(int(t))


def test_teacher_forced_drafts_are_all_accepted(tiny):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 48, n_policy=0)
    for n in (1, 4, 8):
        tf = oracle.decode(m, prompt, 40, n_policy=n, forced_stream=ar["tokens"])
        assert np.array_equal(tf["tokens"], ar["tokens"][:40])
        assert all(it["k"] == it["n"] for it in tf["iters"])
        c = tf["counters"]
        assert c["n_waste"] == 0 and c["n_tokens"] == c["n_target"] * (n + 1)


# ----------------------------------------------------------------- acceptance (footnote of Section 3.1, Eq. 1)

def test_accept_length_is_longest_correct_prefix(tiny):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 16, n_policy=0)["tokens"]
    n = 6
    for c in range(0, n + 1):  # c = index of the first corrupted draft (n = none corrupted)
        seq = m.new_seq(256)
        first = seq.prefill(prompt)
        assert first == ar[0]
        draft = ar[1: 1 + n].copy()
        if c < n:
            draft[c] = (draft[c] + 1) % sh.vocab
        tt, _, _, _ = seq.verify(draft)
        k, emitted = seq.accept(draft, tt)
        assert k == c
        assert np.array_equal(emitted, ar[1: 2 + c])  # accepted drafts + bonus = greedy continuation
        assert seq.len == len(prompt) + 1 + c + 1


def test_state_after_accept_equals_fresh_prefill(tiny):
    """Compaction: continuing from the kept cache rows == continuing from a prefill of the committed tokens."""
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 24, n_policy=0)["tokens"]
    seq = m.new_seq(256)
    seq.prefill(prompt)
    draft = ar[1:6].copy()
    draft[2] = (draft[2] + 5) % sh.vocab           # rows after the 2nd draft become garbage
    tt, _, _, _ = seq.verify(draft)
    k, _ = seq.accept(draft, tt)
    assert k == 2
    committed = seq.tokens()
    fresh = m.new_seq(256)
    fresh.prefill(committed[:-1])
    assert fresh.tokens()[-1] == committed[-1]
    a = [seq.step(-1) for _ in range(4)]
    b = [fresh.step(-1) for _ in range(4)]
    for x, y in zip(a, b):
        assert x["n"] == y["n"] and x["k"] == y["k"]
        assert np.array_equal(x["emitted"], y["emitted"]) and np.array_equal(x["draft"], y["draft"])
        assert np.array_equal(x["v_top1"], y["v_top1"])


def test_rewound_sequence_continues_like_a_fresh_prefill(tiny):
    """orc_rewind: a sequence rolled back to its prefilled state (with or without the draft head's prompt rows)
    repeats, bit for bit, what a freshly prefilled sequence does; counters restart."""
    sh, w, prompt, m = tiny
    fresh = m.new_seq(256)
    fresh.prefill(prompt)
    a = [fresh.step(n) for n in (-1, 3, 8, -1)]
    for keep_draft_rows in (True, False):
        seq = m.new_seq(256)
        seq.prefill(prompt)
        for n in (5, -1, 2):
            seq.step(n)
        seq.rewind(len(prompt) + 1, len(prompt) - 1 if keep_draft_rows else 0)
        assert seq.len == len(prompt) + 1 and seq.counters()["n_target"] == 0
        b = [seq.step(n) for n in (-1, 3, 8, -1)]
        for x, y in zip(a, b):
            assert x["n"] == y["n"] and x["k"] == y["k"]
            assert np.array_equal(x["emitted"], y["emitted"]) and np.array_equal(x["draft"], y["draft"])
            assert np.array_equal(x["v_top1"], y["v_top1"]) and np.array_equal(x["d_top1"], y["d_top1"])
        assert seq.counters() == fresh.counters()
    with pytest.raises(AssertionError):
        seq.rewind(seq.len + 1, 0)


def test_golden_writer_step_equals_the_oracle_step(tiny):
    """tests/golden/make_goldens.py keeps complete logit rows by composing predict, draft, verify and accept
    itself: that composition must be the iteration Seq.step runs, and its logits must carry the stored top-2."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("make_goldens", os.path.join(GOLDEN, "make_goldens.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    sh, w, prompt, m = tiny
    a, b = m.new_seq(256), m.new_seq(256)
    assert a.prefill(prompt) == b.prefill(prompt)
    ar = oracle.decode(m, prompt, 40, n_policy=0)["tokens"]
    for n, teacher in ((-1, False), (0, False), (4, False), (-1, False), (3, True)):
        forced = np.asarray(ar[a.len - len(prompt): a.len - len(prompt) + sh.n_max], dtype=np.int32) if teacher else None
        x = a.step(n, forced)
        y, lg = mg.step_with_logits(b, n, forced)
        assert x["n"] == y["n"] and x["k"] == y["k"] and x["j"] == y["j"]
        for key in ("emitted", "draft", "target", "v_top1", "v_top2", "d_top1", "d_top2"):
            assert np.array_equal(x[key], y[key]), key
        if n < 0:
            assert np.array_equal(x["ldlp_z"][: sh.n_max], y["ldlp_z"][: sh.n_max])
        assert lg.shape == (x["n"] + 1, sh.vocab)
        assert np.array_equal(lg.argmax(axis=1), x["target"]) and np.array_equal(lg.max(axis=1), x["v_top1"])
        if teacher:
            assert x["k"] == 3
    assert a.counters() == b.counters()


# ----------------------------------------------------------------- draft head

def test_draft_head_block_matches_stock_op_restatement(tiny):
    sh, w, prompt, m = tiny
    seq = m.new_seq(256)
    seq.prefill(prompt)
    T = len(prompt)
    feat = seq.features(0, T)
    nxt = seq.tokens()[1: T + 1]
    dk = np.zeros((T, sh.d_model), dtype=np.float32)
    dv = np.zeros_like(dk)
    got = m.draft_rows(nxt, feat, 0, dk, dv)
    e = tr.t64(w["embed"])[torch.as_tensor(nxt, dtype=torch.long)]
    x = torch.cat([e, torch.from_numpy(feat.astype(np.float64))], -1) @ tr.t64(w["eagle_fc"]).T
    ref = tr.block(x, tr.eagle_layer_weights(w), sh)
    assert np.abs(got - ref.numpy()).max() < 2e-5


def test_draft_steps_equal_cache_free_recompute(tiny):
    """Catch-up rows + single-row steps through the head's cache == the head run over all rows at once."""
    sh, w, prompt, m = tiny
    seq = m.new_seq(256)
    seq.prefill(prompt)
    n = 5
    draft, _, _ = seq.draft(n)
    own = seq.draft_features(n)                      # estimates of f_j .. f_{j+n-1}
    j = len(prompt)
    feats = np.concatenate([seq.features(0, j), own[: n - 1]])
    nxt = np.concatenate([seq.tokens()[1: j + 1], draft[: n - 1]])
    dk = np.zeros((j + n, sh.d_model), dtype=np.float32)
    dv = np.zeros_like(dk)
    allrows = m.draft_rows(nxt, feats, 0, dk, dv)
    assert np.array_equal(allrows[j - 1:], own)
    lm = si.bf16_bits_to_f32(w["lm_head"]).astype(np.float64)
    for s in range(n):                               # token s+1 = argmax of the shared LM head on the estimate
        assert int(np.argmax(lm @ own[s].astype(np.float64))) == int(draft[s])


# ----------------------------------------------------------------- length predictor (Eq. 3)

def _ldlp_model(sh, w, **over):
    w2 = dict(w)
    w2.update(over)
    return w2


def _bf16(a):
    t = torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def test_ldlp_closed_forms(tiny):
    sh, w, prompt, _ = tiny
    d, hid, nmax = sh.d_model, sh.ldlp_hidden, sh.n_max
    zeros = lambda *s: np.zeros(s, dtype=np.uint16)
    # (a) W1 = 0, W2 = 0: z = b2, so n = argmax(b2) + 1, ties to the lowest index
    b2 = np.zeros(nmax, dtype=np.float32)
    b2[[3, 5]] = 1.5
    m = oracle.Model(sh, _ldlp_model(sh, w, ldlp_w1=zeros(hid, 2 * d), ldlp_w2=zeros(nmax, hid), ldlp_b2=_bf16(b2)))
    seq = m.new_seq(128)
    seq.prefill(prompt)
    n, z = seq.ldlp()
    assert n == 4 and np.array_equal(z, b2)
    # (b) W1 = 0: h = ReLU(b1); z = W2 ReLU(b1) + b2 with hand-picked numbers
    b1 = np.zeros(hid, dtype=np.float32)
    b1[0], b1[1] = 2.0, -3.0                         # ReLU -> (2, 0)
    W2 = np.zeros((nmax, hid), dtype=np.float32)
    W2[6, 0], W2[2, 1], W2[1, 0] = 0.5, 100.0, 0.25  # z6 = 1, z2 = 0 (killed by ReLU), z1 = 0.5
    m = oracle.Model(sh, _ldlp_model(sh, w, ldlp_w1=zeros(hid, 2 * d), ldlp_b1=_bf16(b1), ldlp_w2=_bf16(W2),
                                     ldlp_b2=zeros(nmax)))
    seq = m.new_seq(128)
    seq.prefill(prompt)
    n, z = seq.ldlp()
    assert n == 7 and z[6] == 1.0 and z[1] == 0.5 and z[2] == 0.0
    # (c) W1 picks single coordinates of x = [e ; f]: unit 0 reads x[0] (embedding part), unit 1 reads
    # x[d] (feature part); the inputs are those of position len-2 (token before the pending one)
    W1 = np.zeros((hid, 2 * d), dtype=np.float32)
    W1[0, 0], W1[1, d], W1[2, 0], W1[3, d] = 1.0, 1.0, -1.0, -1.0
    W2 = np.zeros((nmax, hid), dtype=np.float32)
    W2[0, 0], W2[1, 1], W2[2, 2], W2[3, 3] = 1.0, 1.0, 1.0, 1.0
    m = oracle.Model(sh, _ldlp_model(sh, w, ldlp_w1=_bf16(W1), ldlp_b1=zeros(hid), ldlp_w2=_bf16(W2), ldlp_b2=zeros(nmax)))
    seq = m.new_seq(128)
    seq.prefill(prompt)
    n, z = seq.ldlp()
    e0 = si.bf16_bits_to_f32(w["embed"])[prompt[-1], 0]
    f0 = seq.features(len(prompt) - 1, len(prompt))[0, 0]
    expect = np.array([max(e0, 0), max(f0, 0), max(-e0, 0), max(-f0, 0)], dtype=np.float32)
    assert np.array_equal(z[:4], expect)
    assert n == int(np.argmax(expect)) + 1
    # the other reading (embedding of the pending token) is a switch and gives that token's embedding
    m2 = oracle.Model(sh, m.weights, ldlp_embed_shift=1)
    seq2 = m2.new_seq(128)
    first = seq2.prefill(prompt)
    _, z2 = seq2.ldlp()
    e1 = si.bf16_bits_to_f32(w["embed"])[first, 0]
    assert z2[0] == max(e1, 0) and z2[2] == max(-e1, 0) and z2[1] == expect[1]


def test_ldlp_range(tiny):
    sh, w, prompt, m = tiny
    sd = oracle.decode(m, prompt, 32, n_policy=-1)
    assert all(1 <= it["n"] <= sh.n_max for it in sd["iters"])


@pytest.mark.parametrize("scalar,expect", [(2.5, 2), (3.5, 4), (0.5, 1), (-3.0, 1), (100.0, 8), (7.25, 7), (6.5, 6), (1.0, 1)])
def test_ldlp_scalar_form_rounds_half_to_even_and_clamps(tiny, scalar, expect):
    sh, w, prompt, _ = tiny
    d, hid = sh.d_model, sh.ldlp_hidden
    zeros = lambda *s: np.zeros(s, dtype=np.uint16)
    b2 = np.zeros(sh.n_max, dtype=np.float32)
    b2[0] = scalar
    m = oracle.Model(sh, _ldlp_model(sh, w, ldlp_w1=zeros(hid, 2 * d), ldlp_b1=zeros(hid), ldlp_w2=zeros(sh.n_max, hid),
                                     ldlp_b2=_bf16(b2), ldlp_wr=zeros(2, hid, hid), ldlp_br=zeros(2, hid)),
                     ldlp_mode=1)
    seq = m.new_seq(128)
    seq.prefill(prompt)
    n, z = seq.ldlp()
    assert n == expect


def test_ldlp_scalar_form_residual_blocks(tiny):
    """h0 = ReLU(b1); h1 = h0 + ReLU(Wr0 h0 + br0); h2 = h1 + ReLU(Wr1 h1 + br1); z = w2 . h2 + b2."""
    sh, w, prompt, _ = tiny
    d, hid = sh.d_model, sh.ldlp_hidden
    zeros = lambda *s: np.zeros(s, dtype=np.uint16)
    b1 = np.zeros(hid, dtype=np.float32); b1[0] = 1.0               # h0 = (1, 0, ...)
    wr = np.zeros((2, hid, hid), dtype=np.float32)
    wr[0, 1, 0] = 2.0                                               # block 0 adds 2 to unit 1 -> h1 = (1, 2)
    wr[1, 0, 1] = -1.0                                              # block 1: unit 0 gets ReLU(-2) = 0
    br = np.zeros((2, hid), dtype=np.float32); br[1, 2] = 0.5       # block 1 adds 0.5 to unit 2 -> h2 = (1, 2, .5)
    w2 = np.zeros((sh.n_max, hid), dtype=np.float32); w2[0, :3] = (1.0, 1.0, 2.0)   # z = 1 + 2 + 1 = 4
    m = oracle.Model(sh, _ldlp_model(sh, w, ldlp_w1=zeros(hid, 2 * d), ldlp_b1=_bf16(b1), ldlp_w2=_bf16(w2),
                                     ldlp_b2=zeros(sh.n_max), ldlp_wr=_bf16(wr), ldlp_br=_bf16(br)), ldlp_mode=1)
    seq = m.new_seq(128)
    seq.prefill(prompt)
    n, z = seq.ldlp()
    assert z[0] == 4.0 and n == 4


# ----------------------------------------------------------------- counters (Table 2)

def _table2():
    rows = []
    for line in open(os.path.join(GOLDEN, "table2_counts.txt")):
        if line.strip() and not line.startswith("#"):
            lab, dl, tau, nd, nt, nw = line.split()
            rows.append((lab, dl, float(tau), int(nd), int(nt), int(nw)))
    return rows


def test_tau_formula_reproduces_table2():
    for lab, dl, tau, nd, nt, nw in _table2():
        # the paper averages tau over samples, so the pooled counts match it to the printed digits
        # except on the EAGLE-Oracle row (3.39 pooled vs 3.41 printed)
        tol = 0.03 if lab == "eagle_oracle" else 0.0051
        assert abs(oracle.tau(nd, nt, nw) - tau) < tol, (lab, dl)
        if dl != "dyn":
            assert nd == int(dl) * nt            # N_draft = sum of the draft lengths


def test_counter_identities(tiny):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 40, n_policy=0)["tokens"]
    # drafts forced to the greedy continuation but corrupted at every 4th emitted position
    bad = ar.copy()
    bad[3::4] = (bad[3::4] + 1) % sh.vocab
    run = oracle.decode(m, prompt, 32, n_policy=5, forced_stream=bad)
    assert np.array_equal(run["tokens"], ar[:32])
    c, its = run["counters"], run["iters"]
    assert c["n_target"] == len(its)
    assert c["n_draft"] == sum(it["n"] for it in its)
    assert c["n_waste"] == sum(it["n"] - it["k"] for it in its)
    assert c["n_tokens"] == sum(it["k"] + 1 for it in its)
    assert abs(oracle.tau(c["n_draft"], c["n_target"], c["n_waste"]) - c["n_tokens"] / c["n_target"]) < 1e-12
    assert any(it["k"] > 0 for it in its) and any(it["k"] < it["n"] for it in its)


def test_drafting_exactly_the_accept_length_wastes_nothing(tiny):
    """Section 2.3 / Lemma 1 setting: told the acceptance length in advance, N_waste = 0 and the output is unchanged."""
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 40, n_policy=0)["tokens"]
    bad = ar.copy()
    bad[3::4] = (bad[3::4] + 1) % sh.vocab
    probe = oracle.decode(m, prompt, 32, n_policy=5, forced_stream=bad)
    # acceptance length available at emitted-token offset o: distance to the next corrupted position
    def policy(r, seq):
        o = seq.len - 1 - len(prompt)            # tokens emitted so far minus one... offset of pending token
        k = 0
        while k < sh.n_max and (o + 1 + k) % 4 != 3:
            k += 1
        return k
    run = oracle.decode(m, prompt, 32, n_policy=policy, forced_stream=bad)
    assert np.array_equal(run["tokens"], ar[:32])
    assert run["counters"]["n_waste"] == 0
    assert run["counters"]["n_target"] <= probe["counters"]["n_target"]


# ----------------------------------------------------------------- AdaEAGLE-DDD stopping rule (Section 4)

def _ddd_seq(sh, w, prompt, thr, cap=512):
    m = oracle.Model(sh, w, ddd_threshold=thr)
    seq = m.new_seq(cap)
    seq.prefill(prompt)
    return m, seq


def test_ddd_off_drafts_exactly_n(tiny):
    sh, w, prompt, m0 = tiny
    _, seq = _ddd_seq(sh, w, prompt, 0.0)
    ref = m0.new_seq(512)
    ref.prefill(prompt)
    for n in (1, 3, sh.n_max):
        a = seq.step(n_forced=n)
        b = ref.step(n_forced=n)
        assert a["n"] == n and list(a["draft"]) == list(b["draft"]) and list(a["emitted"]) == list(b["emitted"])


def test_ddd_log_probability_is_log_softmax_of_the_draft_logits(tiny):
    """The running log-probability against float64 log-softmax of (draft feature x LM head), built from stock ops."""
    sh, w, prompt, _ = tiny
    _, seq = _ddd_seq(sh, w, prompt, -1e30)                 # never stops early: n_max tokens
    toks, _, _, lp = seq.draft_dyn(1)
    assert len(toks) == sh.n_max
    feats = seq.draft_features(sh.n_max).astype(np.float64)
    W = si.bf16_bits_to_f32(w["lm_head"]).astype(np.float64)
    logits = feats @ W.T
    ls = logits - logits.max(1, keepdims=True)
    logsm = ls - np.log(np.exp(ls).sum(1, keepdims=True))
    assert list(toks) == list(logits.argmax(1))
    expect = np.cumsum(logsm[np.arange(sh.n_max), toks])
    assert np.abs(lp - expect).max() < 1e-3
    assert np.all(np.diff(lp) < 0)                           # a product of probabilities only shrinks


@pytest.mark.parametrize("n", [1, 2, 5])
@pytest.mark.parametrize("thr", [-4.0, -12.5, -17.0, -26.0, -41.0, -1e30])
def test_ddd_length_is_first_step_past_n_below_the_threshold(tiny, n, thr):
    """Brute force on the log-probabilities of a full-length draft: stop at the first s >= n with S_s < thr."""
    sh, w, prompt, _ = tiny
    _, full = _ddd_seq(sh, w, prompt, -1e30)
    _, _, _, lp = full.draft_dyn(1)
    expect = next((s for s in range(n, sh.n_max + 1) if lp[s - 1] < thr), sh.n_max)
    _, seq = _ddd_seq(sh, w, prompt, thr)
    toks, _, _, lp2 = seq.draft_dyn(n)
    assert len(toks) == expect
    assert np.array_equal(lp2, lp[:expect])


def test_ddd_respects_the_cache_capacity(tiny):
    sh, w, prompt, _ = tiny
    cap = len(prompt) + 4                                     # j = len(prompt): room for j + n + 2 <= cap -> n <= 2
    _, seq = _ddd_seq(sh, w, prompt, -1e30, cap=cap)
    o = seq.step(n_forced=1)
    assert o["n"] == 2


def test_ddd_output_is_still_greedy_decoding(tiny):
    sh, w, prompt, m0 = tiny
    ar = oracle.decode(m0, prompt, 24, n_policy=0)["tokens"]
    m = oracle.Model(sh, w, ddd_threshold=-17.0)
    sd = oracle.decode(m, prompt, 24, n_policy=1)
    assert list(sd["tokens"]) == list(ar)
    assert sd["counters"]["n_draft"] > sd["counters"]["n_target"]   # the rule did extend drafts past n = 1


# ----------------------------------------------------------------- draft-length labels / EAGLE-Oracle (Sections 2.3, 3.3)

def test_label_is_the_accept_length_of_a_full_draft_and_leaves_the_state_alone(tiny):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 40, n_policy=0)["tokens"]
    a, b = m.new_seq(512), m.new_seq(512)
    a.prefill(prompt)
    b.prefill(prompt)
    bad = ar.copy()
    bad[2::3] = (bad[2::3] + 1) % sh.vocab
    for it in range(6):
        k = a.label()
        o = b.step(n_forced=sh.n_max)                   # same state: a full-length draft, verified and accepted
        assert k == o["k"]
        o2 = a.step(n_forced=sh.n_max)                  # the labelled sequence continues exactly like the other
        assert list(o2["emitted"]) == list(o["emitted"]) and list(o2["draft"]) == list(o["draft"])
    # with teacher-forced drafts corrupted at known places the label is the distance to the next corruption
    c = m.new_seq(512)
    c.prefill(prompt)
    # (label() drafts with the head's own tokens, so here the corrupted stream is checked through step())
    o = c.step(n_forced=sh.n_max, forced_draft=bad[1:1 + sh.n_max])
    assert o["k"] == 1                                   # bad[2] is the first corrupted token: drafts 0..0 confirmed


def test_told_the_label_no_draft_is_wasted(tiny):
    """EAGLE-Oracle of Section 2.3: N_waste = 0, output unchanged, no more target passes than any fixed length."""
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 32, n_policy=0)["tokens"]
    run = oracle.decode(m, prompt, 32, n_policy=lambda r, seq: seq.label())
    assert np.array_equal(run["tokens"], ar)
    assert run["counters"]["n_waste"] == 0
    for n in (1, 4, sh.n_max):
        assert run["counters"]["n_target"] <= oracle.decode(m, prompt, 32, n_policy=n)["counters"]["n_target"]


def test_labels_over_start_positions_equal_labels_after_fresh_prefills(tiny):
    """Section 3.3, data collection: Seq.label_positions (roll back to each start position, last first) gives, for
    every position of a generated sequence, the label, drafts and target choices that a sequence freshly prefilled up
    to that position gives."""
    sh, w, prompt, m = tiny
    dec = oracle.decode(m, prompt, 14, n_policy=-1)
    seq = dec["seq"]
    toks = seq.tokens()
    j0, count = len(prompt) + 1, len(toks) - 1 - len(prompt) - 1
    assert count >= 8
    got = seq.label_positions(j0, count)
    for j in range(j0, j0 + count):
        fresh = m.new_seq(256)
        assert fresh.prefill(toks[:j]) == toks[j]          # the sequence is the model's own greedy output
        k, dr, tg = fresh.label_tokens()
        assert got[j][0] == k and np.array_equal(got[j][1], dr) and np.array_equal(got[j][2], tg), j
        assert len(dr) == sh.n_max and tg[0] == toks[j + 1]   # row 0 is the committed token j: the target repeats its choice
