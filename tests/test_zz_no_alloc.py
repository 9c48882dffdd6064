"""ada_ldlp_eval_static: the length predictor for callers that cannot allocate device memory.

Such callers (a plugin inside an application that owns all device memory, code running while
another allocator holds the GPU) cannot give the library a workspace, so this entry point keeps
its scratch in a fixed array inside the library.  The test calls it through the C ABI twice in a
row, on different inputs, and checks each result against ada_ldlp_predict of a context fed the same
inputs and against the CPU oracle's predictor on the same decoding state.  This file sorts last so that
a run stopping at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

Z_TOL = 2e-3   # the tolerance the other tests use for predictor logits


def test_static_predictor_matches_the_context_predictor_twice(tiny):
    from paper_2412_18910_b200 import Engine, ada_ldlp_eval_static
    sh, w, prompt, m = tiny
    e = Engine(sh, w, max_batch=1, kv_capacity=sh.kv_capacity)
    try:
        seq = m.new_seq(sh.kv_capacity)
        assert seq.prefill(prompt) == e.prefill(0, prompt)
        feat = e.ada_debug_buffer(0, torch.float32, (1, sh.kv_capacity, sh.d_model))
        toks = e.ada_debug_buffer(2, torch.int32, (1, sh.kv_capacity))
        lens = e.ada_debug_buffer(3, torch.int32, (1, 8))
        zbuf = e.ada_debug_buffer(1, torch.float32, (1, 16))
        n_out = torch.zeros(1, dtype=torch.int32, device=e.dev)
        z_out = torch.zeros(sh.n_max, dtype=torch.float32, device=e.dev)
        seen = []
        for call in range(2):
            e.ada_ldlp_predict(e.d_n)
            torch.cuda.synchronize()
            p = int(lens[0, 0].cpu()) - 2                       # last token of the validated prefix
            tok = int(toks[0, p].cpu())
            rc = ada_ldlp_eval_static(e.w["ldlp_w1"], e.w["ldlp_b1"], e.w["ldlp_w2"], e.w["ldlp_b2"],
                                      e.w["embed"][tok], feat[0, p], n_out, z_out, stream=e.stream)
            assert rc == 0
            torch.cuda.synchronize()
            assert int(n_out.cpu()[0]) == int(e.d_n.cpu()[0])
            assert np.abs(z_out.cpu().numpy() - zbuf[0, : sh.n_max].cpu().numpy()).max() <= Z_TOL
            n_o, z_o = seq.ldlp()                               # the oracle's predictor on the same state
            assert int(n_out.cpu()[0]) == n_o
            assert np.abs(z_out.cpu().numpy() - z_o[: sh.n_max]).max() <= Z_TOL
            seen.append(z_out.cpu().numpy().copy())
            o = seq.step()                                      # move on: the second call sees other inputs
            g = e.step()
            if list(g["emitted"][0]) != [int(t) for t in o["emitted"]]:   # a flip inside the oracle's margin: follow the oracle
                em = torch.as_tensor(np.asarray(o["emitted"], dtype=np.int32)).to(e.dev)
                e.ada_force_commit(0, em, len(o["emitted"]))
        assert not np.array_equal(seen[0], seen[1])
    finally:
        e.close()


def test_static_predictor_rejects_a_hidden_width_beyond_its_array(tiny):
    from paper_2412_18910_b200 import ada_ldlp_eval_static
    dev = torch.device("cuda:0")
    hid, d, nmax = 4097, 8, 4                                  # one more than ADA_STATIC_MAX_HIDDEN
    bf = dict(dtype=torch.bfloat16, device=dev)
    n_out = torch.full((1,), -7, dtype=torch.int32, device=dev)
    rc = ada_ldlp_eval_static(torch.zeros(hid, 2 * d, **bf), torch.zeros(hid, **bf), torch.zeros(nmax, hid, **bf),
                              torch.zeros(nmax, **bf), torch.zeros(d, **bf),
                              torch.zeros(d, dtype=torch.float32, device=dev), n_out)
    assert rc == -8                                            # ADA_ERR_TOO_LARGE, nothing launched
    torch.cuda.synchronize()
    assert int(n_out.cpu()[0]) == -7
