"""Writes the full-size golden trajectories from the CPU oracle (and from nothing else).

    python tests/golden/make_goldens.py 7b 7b_tf 13b 7b_b8

For each configuration the oracle prefills the seeded prompt(s) and runs a bounded number of
lock-step iterations; per iteration the file keeps the draft length, the drafts, the target's
choices, the accepted length, the emitted tokens, the top-1/top-2 logits of every draft step and
verify row (the margins decide which positions are exempt) and the predictor's outputs.
Output: tests/golden/<config>.json (small text).  Takes minutes to an hour per configuration.
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

ITERS = {"7b": 12, "13b": 8, "7b_b8": 4}
TF_REPEATS = 2   # teacher-forced configuration: iterations per forced length 1..n_max, one after another


def it_json(it):
    return dict(j=int(it["j"]), n=int(it["n"]), k=int(it["k"]), emitted=[int(t) for t in it["emitted"]],
                draft=[int(t) for t in it["draft"]], target=[int(t) for t in it["target"]],
                v_top1=[float(x) for x in it["v_top1"]], v_top2=[float(x) for x in it["v_top2"]],
                d_top1=[float(x) for x in it["d_top1"]], d_top2=[float(x) for x in it["d_top2"]],
                ldlp_z=[float(x) for x in it["ldlp_z"]])


def main(names):
    for name in names:
        t0 = time.time()
        sh = si.SHAPES[name]
        w = si.make_weights(sh)
        m = oracle.Model(sh, w)
        prompts = si.make_prompts(sh)
        out = dict(config=name, seed=si.DEFAULT_SEED, prompt_lens=[int(len(p)) for p in prompts], seqs=[])
        for b, prompt in enumerate(prompts):
            rec = dict(first=None, iters=[])
            if name == "7b_tf":
                need = sum(TF_REPEATS * (n + 1) for n in range(1, sh.n_max + 1)) + 2
                seq = m.new_seq(len(prompt) + 2 * need + 32)
                rec["first"] = int(seq.prefill(prompt))
                # the oracle's own greedy continuation, then teacher-forced iterations on a second sequence
                ar = [rec["first"]]
                while len(ar) < need:
                    ar.extend(int(t) for t in seq.step(0)["emitted"])
                rec["greedy"] = ar
                seq2 = m.new_seq(len(prompt) + need + 32)
                assert seq2.prefill(prompt) == rec["first"]
                for n in range(1, sh.n_max + 1):
                    for _ in range(TF_REPEATS):
                        off = seq2.len - len(prompt)
                        forced = np.array(ar[off: off + sh.n_max] + [0] * sh.n_max, dtype=np.int32)[: sh.n_max]
                        it = seq2.step(n, forced)
                        assert it["k"] == n
                        rec["iters"].append(it_json(it))
            else:
                seq = m.new_seq(len(prompt) + (ITERS[name] + 2) * (sh.n_max + 1) + 8)
                rec["first"] = int(seq.prefill(prompt))
                for _ in range(ITERS[name]):
                    rec["iters"].append(it_json(seq.step(-1)))
            out["seqs"].append(rec)
            print(name, "seq", b, "done at %.0f s" % (time.time() - t0), flush=True)
        out["oracle_seconds"] = round(time.time() - t0, 1)
        out["oracle_threads"] = oracle.num_threads()
        with open(os.path.join(ROOT, "tests", "golden", name + ".json"), "w") as f:
            json.dump(out, f)
        print("wrote", name, flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["7b", "7b_tf", "13b", "7b_b8"])
