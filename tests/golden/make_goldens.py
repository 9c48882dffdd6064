"""Writes the full-size golden trajectories from the CPU oracle (and from nothing else).

    python tests/golden/make_goldens.py 7b 7b_tf 13b 7b_b8

For each configuration the oracle prefills the seeded prompt(s) and runs lock-step iterations; per iteration
the file keeps the draft length, the drafts, the target's choices, the accepted length, the emitted tokens,
the top-1/top-2 logits of every draft step and verify row (the margins decide which positions are exempt), the
root mean square of the draft head's feature at every step, and the predictor's outputs.  Lengths:

    7b      the configuration's 256 new tokens
    13b     64 iterations
    7b_b8   16 iterations of each of the 8 sequences
    7b_tf   for every forced length n = 1..n_max, 8 iterations with teacher-forced drafts (the oracle's own greedy
            continuation), every sweep from the same prefilled state

Beside <config>.json (small text) it writes <config>_logits.npz: the complete logit rows (vocab floats each) of a
few sampled verify rows, named seq<b>_it<r>_row<i> (7b_tf: seq0_n<n>_it<r>_row<i>), for the max-abs logit bound.
Takes from twenty minutes to over an hour per configuration on 8 cores.
"""
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import oracle  # noqa: E402
import synth_inputs as si  # noqa: E402

ITERS = {"13b": 64, "7b_b8": 16}
TF_REPEATS = 8   # teacher-forced configuration: iterations per forced length
# sampled verify rows whose complete logits are kept: (sequence, iteration, row; -1 = the block's last row)
LOGIT_ROWS = {"7b": [(0, 2, -1), (0, 200, 0)], "13b": [(0, 1, -1), (0, 60, 0)],
              "7b_b8": [(1, 3, -1), (6, 12, 0)]}
TF_LOGIT_ROWS = [(10, 0, -1), (5, 7, 0)]   # (forced length, iteration of that sweep, row)


def it_json(it, seq=None):
    extra = {}
    if seq is not None and it["n"] > 0:
        # root mean square of the draft head's output at every step: the head feeds on its own unnormalised output,
        # so the scale of its features, and with it of the draft logits, grows along the chain
        f = seq.draft_features(int(it["n"])).astype(np.float64)
        extra["d_rms"] = [float(x) for x in np.sqrt((f * f).mean(axis=1))]
    return dict(extra, j=int(it["j"]), n=int(it["n"]), k=int(it["k"]), emitted=[int(t) for t in it["emitted"]],
                draft=[int(t) for t in it["draft"]], target=[int(t) for t in it["target"]],
                v_top1=[float(x) for x in it["v_top1"]], v_top2=[float(x) for x in it["v_top2"]],
                d_top1=[float(x) for x in it["d_top1"]], d_top2=[float(x) for x in it["d_top2"]],
                ldlp_z=[float(x) for x in it["ldlp_z"]])


def step_with_logits(seq, n_forced=-1, forced=None):
    """One iteration composed from the oracle's separate calls, in the order of Seq.step (predict, draft,
    verify, accept), keeping all logits of the verify rows.  Returns (the dict Seq.step returns, logits)."""
    nm = seq.m.shape.n_max
    j = seq.len - 1
    z = np.zeros(nm, dtype=np.float32)
    n = n_forced
    if n < 0:
        n, z = seq.ldlp()
    assert j + n + 2 <= seq.cap
    if n >= 1:
        draft, d1, d2 = seq.draft(n, None if forced is None else np.asarray(forced[:n], dtype=np.int32))
    else:
        draft, d1, d2 = np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.float32)
    tt, v1, v2, lg = seq.verify(draft, want_logits=True)
    k, em = seq.accept(draft, tt)
    return dict(j=j, n=n, k=k, emitted=em, draft=draft, target=tt, v_top1=v1, v_top2=v2, d_top1=d1, d_top2=d2,
                ldlp_z=z), lg


def main(names):
    for name in names:
        t0 = time.time()
        sh = si.SHAPES[name]
        w = si.make_weights(sh)
        m = oracle.Model(sh, w)
        prompts = si.make_prompts(sh)
        out = dict(config=name, seed=si.DEFAULT_SEED, prompt_lens=[int(len(p)) for p in prompts], seqs=[],
                   logit_rows=[])
        rows = {}

        def keep(key, it, lg, row):
            i = it["n"] if row < 0 else row
            rows[key + "_row%d" % i] = lg[i].astype(np.float32)
            out["logit_rows"].append(key + "_row%d" % i)

        for b, prompt in enumerate(prompts):
            rec = dict(first=None, iters=[])
            if name == "7b_tf":
                need = TF_REPEATS * (sh.n_max + 1) + 2
                seq = m.new_seq(len(prompt) + need + 2 * sh.n_max + 8)
                rec["first"] = int(seq.prefill(prompt))
                # the oracle's own greedy continuation, then teacher-forced sweeps from the prefilled state
                ar = [rec["first"]]
                while len(ar) < need + sh.n_max:
                    ar.extend(int(t) for t in seq.step(0)["emitted"])
                rec["greedy"] = ar
                rec["sweeps"] = []
                print(name, "greedy stream done at %.0f s" % (time.time() - t0), flush=True)
                dlen = 0
                for n in range(1, sh.n_max + 1):
                    seq.rewind(len(prompt) + 1, dlen)
                    sweep = dict(n=n, iters=[])
                    for r in range(TF_REPEATS):
                        off = seq.len - len(prompt)
                        forced = np.array(ar[off: off + sh.n_max], dtype=np.int32)
                        want = [x for x in TF_LOGIT_ROWS if x[0] == n and x[1] == r]
                        if want:
                            it, lg = step_with_logits(seq, n, forced)
                            keep("seq0_n%d_it%d" % (n, r), it, lg, want[0][2])
                        else:
                            it = seq.step(n, forced)
                        assert it["k"] == n
                        sweep["iters"].append(it_json(it, seq))
                    rec["sweeps"].append(sweep)
                    dlen = len(prompt) - 1   # the draft head's prompt rows stay valid for the later sweeps
                    print(name, "n", n, "done at %.0f s" % (time.time() - t0), flush=True)
            else:
                budget = sh.max_new if name == "7b" else None
                iters = ITERS.get(name, 10 ** 9)
                seq = m.new_seq(len(prompt) + (sh.max_new if budget else iters * (sh.n_max + 1)) + 2 * sh.n_max + 8)
                rec["first"] = int(seq.prefill(prompt))
                emitted = 1
                r = 0
                while r < iters and (budget is None or emitted < budget):
                    want = [x for x in LOGIT_ROWS[name] if x[0] == b and x[1] == r]
                    if want:
                        it, lg = step_with_logits(seq)
                        keep("seq%d_it%d" % (b, r), it, lg, want[0][2])
                    else:
                        it = seq.step(-1)
                    rec["iters"].append(it_json(it, seq))
                    emitted += len(it["emitted"])
                    r += 1
                    if r % 16 == 0:
                        print(name, "seq", b, "iteration", r, "at %.0f s" % (time.time() - t0), flush=True)
            out["seqs"].append(rec)
            print(name, "seq", b, "done at %.0f s" % (time.time() - t0), flush=True)
        out["oracle_seconds"] = round(time.time() - t0, 1)
        out["oracle_threads"] = oracle.num_threads()
        with open(os.path.join(ROOT, "tests", "golden", name + ".json"), "w") as f:
            json.dump(out, f)
        np.savez(os.path.join(ROOT, "tests", "golden", name + "_logits.npz"), **rows)
        print("wrote", name, flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["7b", "7b_tf", "13b", "7b_b8"])
