"""GPU parity of the CUDA library against the CPU oracle on the tiny configuration (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import lockstep

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def eng(tiny):
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, m = tiny
    e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity)
    yield e
    e.close()


def _prefill_both(e, m, prompt, cap=512):
    seq = m.new_seq(cap)
    t_o = seq.prefill(prompt)
    t_g = e.prefill(0, prompt)
    return seq, t_o, t_g


def test_stage_by_stage_parity_with_logits(tiny, eng):
    sh, w, prompt, m = tiny
    seq, t_o, t_g = _prefill_both(eng, m, prompt)
    assert t_o == t_g
    feat = eng.ada_debug_buffer(0, torch.float32, (1, sh.kv_capacity, sh.d_model))
    T = len(prompt)
    assert np.abs(feat[0, :T].cpu().numpy() - seq.features(0, T)).max() < 2e-2
    logits = torch.zeros(1, sh.n_max + 1, sh.vocab, dtype=torch.float32, device=eng.dev)
    zbuf = eng.ada_debug_buffer(1, torch.float32, (1, 16))
    dfeat = eng.ada_debug_buffer(4, torch.float32, (1, sh.n_max, sh.d_model))
    worst = 0.0
    for it in range(12):
        n_o, z_o = seq.ldlp()
        eng.ada_ldlp_predict(eng.d_n)
        assert int(eng.d_n.cpu()[0]) == n_o
        assert np.abs(zbuf[0, : sh.n_max].cpu().numpy() - z_o[: sh.n_max]).max() < 2e-3
        if it % 3 == 2:            # other lengths than the predictor's
            n_o = 1 + (it * 5) % sh.n_max
            eng.d_n.fill_(n_o)
        d_o, d1, d2 = seq.draft(n_o)
        eng.ada_draft(eng.d_n, eng.d_draft)
        d_g = eng.d_draft.cpu().numpy()[0, :n_o]
        assert np.abs(dfeat[0, :n_o].cpu().numpy() - seq.draft_features(n_o)).max() < 2e-2
        for i in range(n_o):
            if d_g[i] != d_o[i]:
                assert d1[i] - d2[i] <= lockstep.TOKEN_MARGIN
                break
        # verify the oracle's drafts on both sides so that every row is comparable
        eng.d_draft[0, :n_o] = torch.from_numpy(d_o).to(eng.dev)
        tt_o, v1, v2, lg_o = seq.verify(d_o, want_logits=True)
        eng.ada_verify(eng.d_draft, eng.d_n, eng.d_target, logits)
        lg_g = logits[0, : n_o + 1].cpu().numpy()
        worst = max(worst, float(np.abs(lg_g - lg_o).max()))
        assert worst < 2e-2
        tt_g = eng.d_target.cpu().numpy()[0, : n_o + 1]
        for i in range(n_o + 1):
            assert tt_g[i] == tt_o[i] or v1[i] - v2[i] <= lockstep.TOKEN_MARGIN
        k_o, em_o = seq.accept(d_o, tt_o)
        eng.ada_accept(eng.d_accept, eng.d_emitted, eng.d_nemit)
        k_g = int(eng.d_accept.cpu()[0])
        em_g = eng.d_emitted.cpu().numpy()[0, : int(eng.d_nemit.cpu()[0])]
        if k_g != k_o or list(em_g) != list(em_o):
            assert min(v1[: k_o + 1] - v2[: k_o + 1]) <= lockstep.TOKEN_MARGIN
            eng.ada_force_commit(0, torch.from_numpy(em_o).to(eng.dev), len(em_o))
    print("max |logit diff| =", worst)
    assert eng.ada_get_counters()["status"] == 0


@pytest.mark.parametrize("n_forced", [-1, 1, 3, 8])
def test_step_lockstep(tiny, eng, n_forced):
    sh, w, prompt, m = tiny
    seq, t_o, t_g = _prefill_both(eng, m, prompt)
    assert t_o == t_g
    eng.ada_force_draft(None)
    eng.ada_force_n(None if n_forced < 0 else [n_forced])
    res = lockstep.run_lockstep(eng, [seq], 24, n_forced=n_forced)
    eng.ada_force_n(None)
    print(lockstep.format_stats(res["stats"]))
    assert not res["failures"], res["failures"]
    assert res["exempt"] <= res["iterations"] // 2


def test_scalar_form_predictor_lockstep(tiny):
    """Eq. 3 in its scalar form: residual blocks, one output, round (ties to even) and clip to [k_min, n_max].
    The predictor's weights are rescaled so that the scalar really moves over the whole range."""
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, _ = tiny
    hid = sh.ldlp_hidden
    w2 = dict(w)
    w2["ldlp_w1"] = si.normal_bf16(7, "t.ldlp.w1", (hid, 2 * sh.d_model), std=0.08)
    w2["ldlp_wr"] = si.normal_bf16(7, "t.ldlp.wr", (2, hid, hid), std=0.08)
    w2["ldlp_w2"] = si.normal_bf16(7, "t.ldlp.w2", (sh.n_max, hid), std=0.1)
    b2 = si.normal_bf16(7, "t.ldlp.b2", (sh.n_max,))
    b2[0] = np.frombuffer(np.float32(9.0).tobytes(), dtype=np.uint16)[1]   # bf16 bits of 9.0
    w2["ldlp_b2"] = b2
    seen = set()
    for k_min in (1, 6):
        m = oracle.Model(sh, w2, ldlp_mode=1, ldlp_blocks=2, k_min=k_min)
        e = Engine(sh, w2, max_batch=1, kv_capacity=sh.kv_capacity, ldlp_mode=1, ldlp_blocks=2, k_min=k_min)
        try:
            seq, t_o, t_g = _prefill_both(e, m, prompt)
            assert t_o == t_g
            zbuf = e.ada_debug_buffer(1, torch.float32, (1, 16))
            for it in range(10):   # the scalar itself, before any decision
                o = lockstep.with_draft_scale(seq.step(), seq)
                g = e.step()
                assert abs(float(zbuf[0, 0]) - float(o["ldlp_z"][0])) < 2e-2
                ok, ex, resync, msg = lockstep.compare_iteration(o, g["n"][0], *_bufs(e), g["k"][0], g["emitted"][0],
                                                                 sh.n_max, ldlp_scalar=True)
                assert ok, msg
                assert k_min <= g["n"][0] <= sh.n_max
                seen.add(int(g["n"][0]))
                if resync:
                    em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(e.dev)
                    e.ada_force_commit(0, em, len(o["emitted"]))
        finally:
            e.close()
    assert len(seen) >= 3, "the test's predictor should produce several different lengths, saw %s" % sorted(seen)


def _bufs(e):
    d = e.ada_debug_buffer(7, torch.int32, (e.B, e.nmax)).cpu().numpy()[0]
    t = e.ada_debug_buffer(8, torch.int32, (e.B, e.nmax + 1)).cpu().numpy()[0]
    return d, t


def test_teacher_forced_drafts_accept_everything(tiny, eng):
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 120, n_policy=0)["tokens"]
    for n in (2, 8):
        seq, t_o, t_g = _prefill_both(eng, m, prompt)
        eng.ada_force_n([n])
        res = lockstep.run_lockstep(eng, [seq], 8, n_forced=n, forced_stream=[ar], prompts=[prompt])
        eng.ada_force_n(None)
        eng.ada_force_draft(None)
        assert not res["failures"], res["failures"]
        assert seq.counters()["n_waste"] == 0


def test_library_speculative_output_equals_its_own_greedy_output(tiny, eng):
    """Lossless property on the GPU itself, bit for bit: no row's result depends on the rows beside it."""
    sh, w, prompt, m = tiny

    def run(n):
        first = eng.prefill(0, prompt)
        eng.ada_force_n(None if n < 0 else [n])
        out = [first]
        while len(out) < 40:
            out.extend(eng.step()["emitted"][0])
        eng.ada_force_n(None)
        return out[:40]

    ar = run(0)
    for n in (-1, 1, 4, 8):
        assert run(n) == ar


def test_counters_and_launch_count(tiny, eng):
    sh, w, prompt, m = tiny
    eng.prefill(0, prompt)
    c0 = eng.ada_get_counters()
    tot = dict(n=0, k=0, e=0)
    for _ in range(5):
        g = eng.step()
        tot["n"] += g["n"][0]; tot["k"] += g["k"][0]; tot["e"] += g["n_emitted"][0]
    c1 = eng.ada_get_counters()
    assert c1["n_target"] - c0["n_target"] == 5
    assert c1["n_draft"] - c0["n_draft"] == tot["n"]
    assert c1["n_waste"] - c0["n_waste"] == tot["n"] - tot["k"]
    assert c1["n_tokens"] - c0["n_tokens"] == tot["e"]
    assert c1["launches"] > c0["launches"] + 5 * 20
    assert c1["status"] == 0


def test_ragged_batch_matches_per_sequence_oracle(tiny):
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, m = tiny
    B = 3
    prompts = [si.uniform_ids(11, "rag%d" % b, L, sh.vocab) for b, L in enumerate((17, 64, 41))]
    e = Engine(sh, w, max_batch=B, kv_capacity=256)
    try:
        seqs = []
        for b in range(B):
            s = m.new_seq(256)
            assert s.prefill(prompts[b]) == e.prefill(b, prompts[b])
            seqs.append(s)
        res = lockstep.run_lockstep(e, seqs, 10)
        assert not res["failures"], res["failures"]
        # per-sequence forced lengths: the verify block is ragged (2, 6 and 9 rows); every sequence's drafts, target
        # choices, accepted length and emitted tokens against its own batch-1 oracle run
        e.ada_force_n([1, 5, 8])
        draft_buf = e.ada_debug_buffer(7, torch.int32, (B, sh.n_max))
        target_buf = e.ada_debug_buffer(8, torch.int32, (B, sh.n_max + 1))
        stats = lockstep.new_stats(sh.n_max)
        for it in range(3):
            olist = [lockstep.with_draft_scale(s.step(n), s) for s, n in zip(seqs, (1, 5, 8))]
            g = e.step()
            assert g["n"] == [1, 5, 8]
            gd, gt = draft_buf.cpu().numpy(), target_buf.cpu().numpy()
            for b, o in enumerate(olist):
                ok, ex, resync, msg = lockstep.compare_iteration(o, g["n"][b], gd[b], gt[b], g["k"][b], g["emitted"][b],
                                                                 sh.n_max, forced_n=True, stats=stats)
                assert ok, (it, b, msg)
                if resync:
                    em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(e.dev)
                    e.ada_force_commit(b, em, len(o["emitted"]))
        print(lockstep.format_stats(stats))
        assert sum(stats["draft_compared"]) >= 3 * 10 and stats["target_compared"] >= 9
        assert e.ada_get_counters()["status"] == 0
    finally:
        e.close()


def test_batch_of_two_with_sixteen_rows_matches_per_sequence_oracle():
    """max_batch = 2 with n_max = 7: a decode pass has at most 16 rows, as at batch 1, but two sequences: it must take
    the multi-kernel path (the persistent pass kernel's attention reads one sequence's cache)."""
    from paper_2412_18910_b200 import Engine
    sh = si.scaled(si.SHAPES["tiny"], n_max=7)
    w = si.make_weights(sh)
    m = oracle.Model(sh, w)
    prompts = [si.uniform_ids(13, "two%d" % b, L, sh.vocab) for b, L in enumerate((23, 70))]
    e = Engine(sh, w, max_batch=2, kv_capacity=256)
    try:
        seqs = []
        for b in range(2):
            s = m.new_seq(256)
            assert s.prefill(prompts[b]) == e.prefill(b, prompts[b])
            seqs.append(s)
        res = lockstep.run_lockstep(e, seqs, 6)
        assert not res["failures"], res["failures"]
        e.ada_force_n([7, 7])             # both sequences at full length: 16 rows
        res = lockstep.run_lockstep(e, seqs, 4, n_forced=7)
        assert not res["failures"], res["failures"]
        assert res["stats"]["draft_compared"][6] > 0
        assert e.ada_get_counters()["status"] == 0
    finally:
        e.close()


def test_launch_chain_equals_plain_stream_order_bit_for_bit(monkeypatch):
    """The multi-kernel path launches a layer's kernels with programmatic dependent launch (each may start while the
    one before it runs and waits inside before it touches that kernel's data).  With ADA_NO_PDL set at ada_init the
    same kernels run in plain stream order: prompt features, draft features, tokens and all verify logits of a ragged
    batch must be the same bits, through the separate calls and through the step graph."""
    from paper_2412_18910_b200 import Engine
    sh = si.SHAPES["tiny"]
    w = si.make_weights(sh)
    prompts = [si.uniform_ids(17, "pdl%d" % b, L, sh.vocab) for b, L in enumerate((150, 33, 64))]
    runs = []
    for no_pdl in (False, True):
        if no_pdl:
            monkeypatch.setenv("ADA_NO_PDL", "1")
        else:
            monkeypatch.delenv("ADA_NO_PDL", raising=False)
        e = Engine(sh, w, max_batch=3, kv_capacity=256)
        try:
            rec = []
            for b in range(3):
                rec.append(e.prefill(b, prompts[b]))
            feat = e.ada_debug_buffer(0, torch.float32, (3, 256, sh.d_model))
            rec.append(feat[0, :150].cpu().numpy().copy())
            e.ada_force_n([3, 8, 5])
            logits = torch.zeros(3 * (sh.n_max + 1), sh.vocab, dtype=torch.float32, device=e.dev)
            for it in range(3):                     # separate calls, with the logits of every verify row
                e.ada_ldlp_predict(e.d_n)
                e.ada_draft(e.d_n, e.d_draft)
                e.ada_verify(e.d_draft, e.d_n, e.d_target, logits)
                e.ada_accept()
                torch.cuda.synchronize()
                rec.append(e.d_draft.cpu().numpy().copy())
                rec.append(e.d_target.cpu().numpy().copy())
                rec.append(logits.cpu().numpy().copy())
            dfeat = e.ada_debug_buffer(4, torch.float32, (3, sh.n_max, sh.d_model))
            for b, n in enumerate((3, 8, 5)):       # (rows past a sequence's draft length are never written)
                rec.append(dfeat[b, :n].cpu().numpy().copy())
            for it in range(4):                     # the step graph
                g = e.step()
                rec.append(np.asarray(g["k"])); rec.append(np.asarray([t for em in g["emitted"] for t in em]))
            assert e.ada_get_counters()["status"] == 0
            runs.append(rec)
        finally:
            e.close()
    assert len(runs[0]) == len(runs[1])
    for i, (a, b) in enumerate(zip(runs[0], runs[1])):
        assert np.array_equal(np.asarray(a), np.asarray(b)), "record %d differs between launch modes" % i


def test_argument_errors_are_reported_not_launched(tiny, eng):
    import ctypes as C
    from paper_2412_18910_b200 import AdaError, Config, lib
    sh, w, prompt, m = tiny
    L = lib()
    bad = Config(2, 256, 4, 64, 688, 4096, 1e4, 1e-6, 128, 8, 0, 1, 500, 64)   # capacity not a page multiple
    assert L.ada_workspace_bytes(C.byref(bad)) == 0
    bad = Config(2, 256, 4, 60, 688, 4096, 1e4, 1e-6, 128, 8, 0, 1, 512, 64)
    assert L.ada_workspace_bytes(C.byref(bad)) == 0
    with pytest.raises(AdaError):
        eng.prefill(0, np.zeros(sh.kv_capacity, dtype=np.int32))     # does not fit
    with pytest.raises(AdaError):
        eng.prefill(1, prompt)                                       # no such sequence
    with pytest.raises(AdaError):
        eng.ada_force_n([sh.n_max + 1])
    assert L.ada_step(None, None, None, None, None) == -2


def test_cache_full_clips_the_draft_length(tiny):
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, m = tiny
    e = Engine(sh, w, max_batch=1, kv_capacity=128)
    try:
        e.prefill(0, si.uniform_ids(3, "long", 118, sh.vocab))       # 118 + n_max + 2 = 128
        e.ada_force_n([8])
        lens = e.ada_debug_buffer(3, torch.int32, (1, 8))
        for _ in range(12):
            g = e.step()
            assert int(lens[0, 0].cpu()) <= 128
        assert e.ada_get_counters()["status"] & 1                   # clipped at least once
    finally:
        e.close()


@pytest.mark.parametrize("plen", [88, 128, 129, 200, 333, 420, 451, 1500])
def test_long_context_attention_spans_blocks_and_rounds(tiny, plen):
    """Contexts of several hundred positions: every KV split holds more than one 32-key block.  The prompt pass
    takes 128 rows at a time through the multi-row tensor-core GEMM (88: a partial chunk; 128: one full chunk; 129: a
    one-row tail; the others: several chunks and a ragged tail) and writes the caches that the 16-row decode passes then read."""
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, m = tiny
    long_prompt = si.uniform_ids(5, "long%d" % plen, plen, sh.vocab)
    cap = sh.kv_capacity if plen + 64 < sh.kv_capacity else 2048   # 1500: splits of more than four blocks (two rounds)
    e = Engine(sh, w, max_batch=1, kv_capacity=cap)
    try:
        seq = m.new_seq(cap)
        t_o = seq.prefill(long_prompt)
        t_g = e.prefill(0, long_prompt)
        feat = e.ada_debug_buffer(0, torch.float32, (1, cap, sh.d_model))
        err = np.abs(feat[0, :plen].cpu().numpy() - seq.features(0, plen)).max(axis=1)
        assert err.max() < 2e-2, (int(err.argmax()), float(err.max()))
        if t_o != t_g:      # only inside the oracle's own margin; the two states then differ, stop here
            lg, _ = m.forward_nocache(long_prompt)
            top = np.sort(lg)
            assert top[-1] - top[-2] <= lockstep.TOKEN_MARGIN
            return
        logits = torch.zeros(1, sh.n_max + 1, sh.vocab, dtype=torch.float32, device=e.dev)
        dfeat = e.ada_debug_buffer(4, torch.float32, (1, sh.n_max, sh.d_model))
        for it in range(4):
            n = sh.n_max
            e.d_n.fill_(n)
            d_o, d1, d2 = seq.draft(n)
            e.ada_draft(e.d_n, e.d_draft)
            derr = np.abs(dfeat[0, :n].cpu().numpy() - seq.draft_features(n)).max(axis=1)
            assert derr.max() < 2e-2, (it, derr)
            e.d_draft[0, :n] = torch.from_numpy(d_o).to(e.dev)
            tt_o, v1, v2, lg_o = seq.verify(d_o, want_logits=True)
            e.ada_verify(e.d_draft, e.d_n, e.d_target, logits)
            lerr = np.abs(logits[0, : n + 1].cpu().numpy() - lg_o).max(axis=1)
            assert lerr.max() < 2e-2, (it, lerr)
            k_o, em_o = seq.accept(d_o, tt_o)
            e.ada_accept(e.d_accept, e.d_emitted, e.d_nemit)
            em_g = e.d_emitted.cpu().numpy()[0, : int(e.d_nemit.cpu()[0])]
            if list(em_g) != list(em_o):
                e.ada_force_commit(0, torch.from_numpy(em_o).to(e.dev), len(em_o))
        assert e.ada_get_counters()["status"] == 0
    finally:
        e.close()


@pytest.mark.parametrize("thr,n_forced", [(-17.0, 1), (-26.0, 2), (-12.5, 1), (-1e30, 3), (-4.0, 2)])
def test_ddd_stopping_rule_lockstep(tiny, thr, n_forced):
    """Section 4 (AdaEAGLE-DDD): drafts grow past the predicted length while the sequence log-probability holds."""
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, _ = tiny
    m = oracle.Model(sh, w, ddd_threshold=thr)
    e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity, ddd_threshold=thr)
    try:
        seq, t_o, t_g = _prefill_both(e, m, prompt)
        assert t_o == t_g
        e.ada_force_n([n_forced])
        lens = set()
        lpbuf = e.ada_debug_buffer(10, torch.float32, (1, sh.n_max))
        for it in range(10):
            o = lockstep.with_draft_scale(seq.step(n_forced=n_forced), seq)
            g = e.step()
            ok, ex, resync, msg = lockstep.compare_iteration(o, g["n"][0], *_bufs(e), g["k"][0], g["emitted"][0],
                                                             sh.n_max, ddd=thr)
            assert ok, msg
            if g["n"][0] == o["n"]:   # per-token log-probabilities: differences of the running sums
                glp = np.cumsum(lpbuf[0, : o["n"]].cpu().numpy().astype(np.float64))
                assert np.abs(glp - o["d_logp"]).max() < 0.1
            lens.add(int(g["n"][0]))
            if resync:
                em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(e.dev)
                e.ada_force_commit(0, em, len(o["emitted"]))
        assert e.ada_get_counters()["status"] == 0
    finally:
        e.close()
    if thr == -1e30:
        assert lens == {sh.n_max}
    if thr == -4.0:
        assert lens == {n_forced}


def test_label_pass_and_told_the_label_nothing_is_wasted(tiny, eng):
    """Sections 2.3 / 3.3: ada_label = accept length of a full-length draft, state untouched; forcing n = label
    gives N_waste = 0 (EAGLE-Oracle).  Teacher-forced drafts with planted mistakes make the labels non-trivial."""
    sh, w, prompt, m = tiny
    ar = oracle.decode(m, prompt, 48, n_policy=0)["tokens"]
    bad = ar.copy()
    bad[3::4] = (bad[3::4] + 1) % sh.vocab
    seq, t_o, t_g = _prefill_both(eng, m, prompt)
    assert t_o == t_g
    d_k = torch.zeros(1, dtype=torch.int32, device=eng.dev)
    before = eng.ada_get_counters()
    labels = []
    for it in range(8):
        off = seq.len - len(prompt)
        forced = np.asarray(bad[off: off + sh.n_max], dtype=np.int32)
        ft = torch.zeros(1, sh.n_max, dtype=torch.int32)
        ft[0, : len(forced)] = torch.from_numpy(forced)
        eng.ada_force_draft(ft.to(eng.dev))
        eng.ada_label(d_k)
        k = int(d_k.cpu()[0])
        # the label against the planted pattern; that the state is untouched shows in the step below
        expect = 0
        while expect < sh.n_max and (off + expect) % 4 != 3:
            expect += 1
        assert k == expect, (it, off, k, expect)
        labels.append(k)
        eng.ada_force_n([k])
        o = seq.step(n_forced=k, forced_draft=forced)
        g = eng.step()
        assert g["n"][0] == k and g["k"][0] == o["k"] == k and list(g["emitted"][0]) == list(o["emitted"])
    eng.ada_force_n(None)
    eng.ada_force_draft(None)
    after = eng.ada_get_counters()
    assert after["n_waste"] == before["n_waste"]
    assert max(labels) >= 3
    assert after["status"] == 0


def test_label_pass_matches_the_oracle_label_on_own_drafts(tiny, eng):
    """Without forced drafts: the head's own full-length draft (random weights: labels are almost always 0)."""
    sh, w, prompt, m = tiny
    seq, t_o, t_g = _prefill_both(eng, m, prompt)
    assert t_o == t_g
    eng.ada_force_draft(None)
    d_k = torch.zeros(1, dtype=torch.int32, device=eng.dev)
    for it in range(4):
        eng.ada_label(d_k)
        assert int(d_k.cpu()[0]) == seq.label()
        res = lockstep.run_lockstep(eng, [seq], 1)
        assert not res["failures"], res["failures"]


@pytest.mark.parametrize("mode", [0, 1])
def test_bounded_waits_give_up_and_the_context_stays_usable(tiny, eng, mode):
    """Failure detection: the pass kernel's wait routines (mode 0: mbarrier wait, mode 1: grid barrier) on a barrier
    that nothing completes, with a limit of 1000 polls.  The wait returns, the status word gets the time-out bit, and
    after ada_reset_status the same context decodes in lock step with the oracle again."""
    sh, w, prompt, m = tiny
    with pytest.raises(Exception):
        eng.ada_selftest_bounded_wait(2, 1000, torch.zeros(2, dtype=torch.int32, device=eng.dev))   # no such mode
    res = torch.zeros(2, dtype=torch.int32, device=eng.dev)
    eng.ada_reset_status()
    assert eng.ada_get_counters()["status"] == 0
    eng.ada_selftest_bounded_wait(mode, 1000, res)
    c = eng.ada_get_counters()
    assert c["status"] & 4, c
    assert int(res.cpu()[mode]) == 1
    eng.ada_reset_status()
    assert eng.ada_get_counters()["status"] == 0
    seq, t_o, t_g = _prefill_both(eng, m, prompt)
    assert t_o == t_g
    eng.ada_force_n(None)
    eng.ada_force_draft(None)
    out = lockstep.run_lockstep(eng, [seq], 4)
    assert not out["failures"], out["failures"]
    assert eng.ada_get_counters()["status"] == 0


def test_labels_over_start_positions_match_the_oracle_and_leave_the_state_alone(tiny):
    """Section 3.3, data collection: ada_label_positions over the generated part of a decoded sequence against the
    oracle's Seq.label_positions (label, drafts and target choices of every start position), then the sequence goes on
    decoding in lock step as if nothing had happened."""
    from paper_2412_18910_b200 import Engine
    sh, w, prompt, m = tiny
    e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity)
    try:
        seq, t_o, t_g = _prefill_both(e, m, prompt)
        assert t_o == t_g
        res = lockstep.run_lockstep(e, [seq], 12)          # a decoded sequence, the two sides on the same tokens
        assert not res["failures"], res["failures"]
        toks = seq.tokens()
        j0, count = len(prompt) + 1, len(toks) - 1 - len(prompt)     # up to and including the pending token
        shadow = m.new_seq(512)                                        # the oracle's copy for the roll-backs
        shadow.prefill(prompt)
        while shadow.len < seq.len:
            shadow.step(-1)
        assert np.array_equal(shadow.tokens(), toks)
        want = shadow.label_positions(j0, count)
        d_k = torch.full((count,), -9, dtype=torch.int32, device=e.dev)
        d_dr = torch.zeros(count, sh.n_max, dtype=torch.int32, device=e.dev)
        d_tg = torch.zeros(count, sh.n_max + 1, dtype=torch.int32, device=e.dev)
        e.ada_label_positions(0, j0, count, d_k, d_dr, d_tg)
        k_g, dr_g, tg_g = d_k.cpu().numpy(), d_dr.cpu().numpy(), d_tg.cpu().numpy()
        same = 0
        for i in range(count):
            k_o, dr_o, tg_o = want[j0 + i]
            n = len(dr_o)
            # drafts may flip only inside the oracle's margins, which this call does not return: count the positions
            # that agree token for token and demand that nearly all do; where the drafts agree, so must the rest
            if np.array_equal(dr_g[i, :n], dr_o):
                same += 1
                assert k_g[i] == k_o
                assert tg_g[i, 0] == tg_o[0]
                if j0 + i + 1 < len(toks):
                    assert tg_o[0] == toks[j0 + i + 1]       # row 0 is committed token j: the target repeats its choice
            assert np.all(dr_g[i, n:] == -1) and np.all(tg_g[i, n + 1:] == -1)
        assert same >= count - 3, (same, count)
        # out-of-range requests are refused on the host
        from paper_2412_18910_b200 import AdaError
        with pytest.raises(AdaError):
            e.ada_label_positions(0, 0, 1, d_k)
        with pytest.raises(AdaError):
            e.ada_label_positions(0, len(toks) - 1, 2, d_k)
        # the state is as before: the next iterations match the oracle's
        res = lockstep.run_lockstep(e, [seq], 6)
        assert not res["failures"], res["failures"]
        assert e.ada_get_counters()["status"] == 0
    finally:
        e.close()
