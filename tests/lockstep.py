"""Lock-step comparison of the CUDA library with the CPU oracle.

Both sides start every iteration from the same committed tokens.  The library's draft length,
drafts, target choices, accepted length and emitted tokens are compared with the oracle's; a
difference is tolerated only where the oracle's own top-1/top-2 margin at the deciding row is at
most the margin of that row, in which case the library is put back on the oracle's trajectory with
ada_force_commit.

Margins.  Verify rows: 0.05 (their logits come from features of unit root mean square, after the
final norm).  Draft step i: 0.05 x max(1, r_i), r_i the root mean square of the oracle's draft-head
feature at that step.  The head feeds on its own output, which has no norm after it, so r_i grows
along the chain (7B shape: 2.6 at step 1, x1.33 per step, 35 at step 10) and the draft logits, their
top-1/top-2 gaps and the deviation between the two implementations all grow with it; the margin is the
same 0.05 relative to the scale of the logits it applies to.
"""
import numpy as np
import torch

TOKEN_MARGIN = 0.05   # logits of unit-scale features: positions with a smaller oracle margin may flip (16-bit cache vs fp32)
DDD_MARGIN = 0.1      # log-probabilities inherit the logits' 2e-2 bound, summed over up to n_max draft tokens
LDLP_MARGIN = 2e-3    # predictor logits are fp32 on both sides; only features differ
LOGIT_TOL = 2e-2      # max-abs bound on verify logits


def new_stats(n_max):
    """Counts kept over a run: per draft step and for verify rows, how many positions were compared and how many
    of those differed inside the margin (exempt)."""
    return dict(draft_compared=[0] * n_max, draft_exempt=[0] * n_max, target_compared=0, target_exempt=0,
                length_exempt=0, logit_rows=0, max_logit_diff=0.0, max_top1_diff=0.0)


def format_stats(st):
    return ("draft steps compared %s exempt %s; verify rows compared %d exempt %d; lengths exempt %d; complete logit rows %d "
            "(max |diff| %.4f); max top-1 logit diff %.4f" % (st["draft_compared"], st["draft_exempt"], st["target_compared"],
                                                            st["target_exempt"], st["length_exempt"], st["logit_rows"],
                                                            st["max_logit_diff"], st["max_top1_diff"]))


def _top2_gap(z):
    s = np.sort(np.asarray(z, dtype=np.float64))
    return float(s[-1] - s[-2]) if len(s) > 1 else float("inf")


def _round_gap(z):
    """Distance of a scalar from the nearest point where rounding to an integer changes."""
    return abs((float(z) - np.floor(float(z))) - 0.5)


def draft_margin(o, i):
    """Margin of draft step i (0-based): TOKEN_MARGIN times the scale of the oracle's draft feature at that step."""
    return TOKEN_MARGIN * max(1.0, float(o["d_rms"][i]))


def with_draft_scale(o, oseq):
    """Adds d_rms (root mean square of the oracle's draft-head feature per step) to a dict from Seq.step()."""
    n = int(o["n"])
    if n > 0 and "d_rms" not in o:
        f = oseq.draft_features(n).astype(np.float64)
        o = dict(o, d_rms=np.sqrt((f * f).mean(axis=1)))
    return o


def compare_iteration(o, g_n, g_draft, g_target, g_k, g_emitted, n_max, forced_n=False, ldlp_scalar=False, ddd=None,
                      stats=None, drafts_forced=False):
    """o: dict from oracle Seq.step() with d_rms (see with_draft_scale).  Returns (ok, exempt, needs_resync, message).

    ldlp_scalar: the predictor is the scalar form (Eq. 3): its decision flips where z crosses k + 1/2.
    drafts_forced: the library's drafts were forced to the oracle's (not a comparison)."""
    st = stats if stats is not None else new_stats(n_max)
    n = o["n"]
    if g_n != n and ddd is not None:
        # Section 4 rule: the length is decided by comparing the running log-probability of the draft sequence with
        # the threshold; the two sides may differ only where the oracle's value at a deciding step is that close
        lp = np.asarray(o["d_logp"], dtype=np.float64)
        close = any(abs(lp[s - 1] - ddd) < DDD_MARGIN for s in range(1, len(lp) + 1))
        if not close:
            return False, 0, True, "draft length %d != oracle %d (log-probabilities %s, threshold %g)" % (g_n, n, lp, ddd)
        st["length_exempt"] += 1
        return True, 1, True, "draft length flipped inside the threshold margin"
    if g_n != n:
        gap = _round_gap(o["ldlp_z"][0]) if ldlp_scalar else _top2_gap(o["ldlp_z"][:n_max])
        if forced_n or gap > LDLP_MARGIN:
            return False, 0, True, "draft length %d != oracle %d" % (g_n, n)
        st["length_exempt"] += 1
        return True, 1, list(g_emitted) != list(o["emitted"]), "n flipped inside the predictor margin"
    if not drafts_forced:
        for i in range(n):
            st["draft_compared"][i] += 1
            if g_draft[i] != o["draft"][i]:
                gap = o["d_top1"][i] - o["d_top2"][i]
                if gap > draft_margin(o, i):
                    return False, 0, True, "draft %d: %d != %d (margin %.3f, allowed %.3f)" % (
                        i, g_draft[i], o["draft"][i], gap, draft_margin(o, i))
                # a flipped draft changes the rows after it: compare only what the oracle decided
                st["draft_exempt"][i] += 1
                return True, 1, list(g_emitted) != list(o["emitted"]), "draft flipped inside the margin"
    for i in range(o["k"] + 1):   # rows whose inputs are committed tokens on both sides
        st["target_compared"] += 1
        if g_target[i] != o["target"][i]:
            if o["v_top1"][i] - o["v_top2"][i] > TOKEN_MARGIN:
                return False, 0, True, "target row %d: %d != %d (margin %.3f)" % (
                    i, g_target[i], o["target"][i], o["v_top1"][i] - o["v_top2"][i])
            st["target_exempt"] += 1
            return True, 1, True, "target flipped inside the margin"
    if g_k != o["k"] or list(g_emitted) != list(o["emitted"]):
        return False, 0, True, "accept %d / emitted %s != oracle %d / %s" % (g_k, list(g_emitted), o["k"], list(o["emitted"]))
    return True, 0, False, ""


def run_lockstep(engine, oseqs, iters, n_forced=-1, forced_stream=None, prompts=None, ldlp_scalar=False, ddd=None):
    """Runs `iters` ada_step iterations against oracle sequences (one per batch slot).

    Returns dict(iterations, exempt, failures[list of str], stats).
    """
    B, nmax = engine.B, engine.nmax
    dev = engine.dev
    draft_buf = engine.ada_debug_buffer(7, torch.int32, (B, nmax))
    target_buf = engine.ada_debug_buffer(8, torch.int32, (B, nmax + 1))
    failures, exempt, compared = [], 0, 0
    stats = new_stats(nmax)
    for r in range(iters):
        forced = None
        olist = []
        if forced_stream is not None:
            ft = torch.zeros(B, nmax, dtype=torch.int32)
            for b, os_ in enumerate(oseqs):
                off = os_.len - len(prompts[b])       # tokens emitted so far = index of the next one in the stream
                chunk = np.asarray(forced_stream[b][off: off + nmax], dtype=np.int32)
                ft[b, : len(chunk)] = torch.from_numpy(chunk)
            forced = ft
            engine.ada_force_draft(ft.to(dev))
        for b, os_ in enumerate(oseqs):
            olist.append(with_draft_scale(os_.step(n_forced, None if forced is None else forced[b].numpy()), os_))
        g = engine.step()
        gd, gt = draft_buf.cpu().numpy(), target_buf.cpu().numpy()
        for b, o in enumerate(olist):
            ok, ex, resync, msg = compare_iteration(o, g["n"][b], gd[b], gt[b], g["k"][b], g["emitted"][b], nmax,
                                                    forced_n=n_forced >= 0 and ddd is None, ldlp_scalar=ldlp_scalar, ddd=ddd,
                                                    stats=stats, drafts_forced=forced_stream is not None)
            compared += 1
            exempt += ex
            if not ok:
                failures.append("iter %d seq %d: %s" % (r, b, msg))
            if resync:
                em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(dev)
                engine.ada_force_commit(b, em, len(o["emitted"]))
    return dict(iterations=compared, exempt=exempt, failures=failures, stats=stats)


def split_step(engine, d_logits=None):
    """One iteration through the four separate calls (predict, draft, verify, accept), which give what ada_step gives;
    the verify call can return all logits.  Same result dict as Engine.step()."""
    engine.ada_ldlp_predict(engine.d_n)
    engine.ada_draft(engine.d_n, engine.d_draft)
    engine.ada_draft_lengths(engine.d_nused)
    engine.ada_verify(engine.d_draft, engine.d_nused, engine.d_target, d_logits)
    engine.ada_accept(engine.d_accept, engine.d_emitted, engine.d_nemit)
    ne = engine.d_nemit.cpu().tolist()
    em = engine.d_emitted.cpu().tolist()
    return dict(n=engine.d_nused.cpu().tolist(), k=engine.d_accept.cpu().tolist(), n_emitted=ne,
                emitted=[em[b][: ne[b]] for b in range(engine.B)])


def _np_iter(o):
    return dict(o, ldlp_z=np.asarray(o["ldlp_z"]), d_top1=np.asarray(o["d_top1"]), d_top2=np.asarray(o["d_top2"]),
                v_top1=np.asarray(o["v_top1"]), v_top2=np.asarray(o["v_top2"]), d_rms=np.asarray(o.get("d_rms", [])))


def run_golden(engine, golden, prompts, logit_rows=None, row_tol=LOGIT_TOL):
    """Replays stored oracle iterations (tests/golden/*.json, written by make_goldens.py) in lock step.

    golden: the parsed file; prompts: the same seeded prompts (already prefilled into the engine unless the file holds
    teacher-forced sweeps, each of which starts from a fresh prefill made here).  logit_rows: the opened
    <config>_logits.npz; at the iterations it names the library runs the four separate calls, with the oracle's drafts
    forced so that every row sees the same inputs, and the complete logit row must agree within row_tol (LOGIT_TOL
    unless the caller states a measured deviation); the top-1 logit of every comparable row within LOGIT_TOL.
    Returns dict(iterations, exempt, failures, stats).
    """
    B, nmax, V = engine.B, engine.nmax, engine.shape.vocab
    dev = engine.dev
    draft_buf = engine.ada_debug_buffer(7, torch.int32, (B, nmax))
    target_buf = engine.ada_debug_buffer(8, torch.int32, (B, nmax + 1))
    vtop = engine.ada_debug_buffer(5, torch.float32, (B, nmax + 1, 2))
    failures, exempt, compared = [], 0, 0
    stats = new_stats(nmax)
    d_logits = torch.zeros(B, nmax + 1, V, dtype=torch.float32, device=dev) if logit_rows is not None else None
    wanted = {}
    for key in (golden.get("logit_rows") or []) if logit_rows is not None else []:
        parts = key.split("_")        # seq<b>_[n<n>_]it<r>_row<i>
        b = int(parts[0][3:])
        n_sweep = int(parts[1][1:]) if parts[1].startswith("n") else None
        r = int(parts[-2][2:])
        wanted.setdefault((n_sweep, r), []).append((b, int(parts[-1][3:]), key))

    teacher = "sweeps" in golden["seqs"][0]
    if teacher:
        episodes = [(sw["n"], [s["sweeps"][i]["iters"] for s in golden["seqs"]]) for i, sw in
                    enumerate(golden["seqs"][0]["sweeps"])]
    else:
        episodes = [(None, [s["iters"] for s in golden["seqs"]])]
    for n_forced, per_seq in episodes:
        emitted_so_far = [1] * B
        if teacher:      # every sweep from the same prefilled state
            for b in range(B):
                assert engine.prefill(b, prompts[b]) == golden["seqs"][b]["first"]
            engine.ada_force_n([n_forced] * B)
        n_iters = min(len(it) for it in per_seq)
        for r in range(n_iters):
            want = wanted.get((n_forced if teacher else None, r), [])
            drafts_forced = teacher or bool(want)
            if teacher:
                ft = torch.zeros(B, nmax, dtype=torch.int32)
                for b in range(B):
                    stream = golden["seqs"][b]["greedy"]
                    chunk = np.asarray(stream[emitted_so_far[b]: emitted_so_far[b] + nmax], dtype=np.int32)
                    ft[b, : len(chunk)] = torch.from_numpy(chunk)
                engine.ada_force_draft(ft.to(dev))
            elif want:       # the oracle's own drafts of this iteration, so that every verify row is comparable
                ft = torch.zeros(B, nmax, dtype=torch.int32)
                for b in range(B):
                    d = np.asarray(per_seq[b][r]["draft"], dtype=np.int32)
                    ft[b, : len(d)] = torch.from_numpy(d)
                engine.ada_force_draft(ft.to(dev))
            g = split_step(engine, d_logits) if want else engine.step()
            if want and not teacher:
                engine.ada_force_draft(None)
            gd, gt, gv = draft_buf.cpu().numpy(), target_buf.cpu().numpy(), vtop.cpu().numpy()
            for b in range(B):
                o = _np_iter(per_seq[b][r])
                ok, ex, resync, msg = compare_iteration(o, g["n"][b], gd[b], gt[b], g["k"][b], g["emitted"][b], nmax,
                                                        forced_n=teacher, stats=stats, drafts_forced=drafts_forced)
                compared += 1
                exempt += ex
                if not ok:
                    failures.append("sweep %s iter %d seq %d: %s" % (n_forced, r, b, msg))
                same_rows = g["n"][b] == o["n"] and (drafts_forced or list(gd[b][: o["n"]]) == list(o["draft"]))
                if same_rows:
                    # same rows on both sides: the top logit of every verify row must agree within the logit bound
                    diff = float(np.abs(gv[b, : o["n"] + 1, 0] - o["v_top1"]).max())
                    stats["max_top1_diff"] = max(stats["max_top1_diff"], diff)
                    if diff > LOGIT_TOL:
                        failures.append("sweep %s iter %d seq %d: top-1 logit differs by %.4f" % (n_forced, r, b, diff))
                for wb, row, key in want:
                    if wb != b:
                        continue
                    if not same_rows:
                        failures.append("%s: rows not comparable (draft length %d vs %d)" % (key, g["n"][b], o["n"]))
                        continue
                    diff = float(np.abs(d_logits[b, row].cpu().numpy() - logit_rows[key]).max())
                    stats["logit_rows"] += 1
                    stats["max_logit_diff"] = max(stats["max_logit_diff"], diff)
                    if diff > row_tol:
                        failures.append("%s: complete logit row differs by %.4f" % (key, diff))
                if resync:
                    em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(dev)
                    engine.ada_force_commit(b, em, len(o["emitted"]))
                emitted_so_far[b] += len(o["emitted"])
    if teacher:
        engine.ada_force_n(None)
        engine.ada_force_draft(None)
    return dict(iterations=compared, exempt=exempt, failures=failures, stats=stats)
