"""ctypes binding of include/ada.h: same names, argument marshalling only.

`lib()` loads libada.so (building it with nvcc when missing or stale) and raises if that is not
possible: there is no fallback path.  `Engine` owns the torch tensors the context borrows
(weights, workspace, I/O buffers) and forwards every call to the library.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

ADA_ERRORS = {0: "ADA_OK", -1: "ADA_ERR_BAD_CONFIG", -2: "ADA_ERR_NULL", -3: "ADA_ERR_RANGE", -4: "ADA_ERR_KV_FULL",
              -5: "ADA_ERR_CUDA", -6: "ADA_ERR_WORKSPACE", -7: "ADA_ERR_STATE",
              -8: "ADA_ERR_TOO_LARGE (a size exceeds a fixed maximum of the library)"}

exported_symbols = ("ada_workspace_bytes", "ada_init", "ada_prefill", "ada_ldlp_predict", "ada_draft", "ada_draft_lengths", "ada_label", "ada_label_positions",
                    "ada_verify",
                    "ada_accept", "ada_step", "ada_force_n", "ada_force_draft", "ada_force_commit",
                    "ada_get_counters", "ada_debug_buffer", "ada_profile", "ada_get_profile", "ada_last_error",
                    "ada_destroy", "ada_ldlp_eval_static", "ada_reset_status", "ada_selftest_bounded_wait")


class AdaError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("ldlp_hidden", "n_max", "ldlp_mode", "max_batch", "kv_capacity", "page_size",
                                         "ldlp_blocks", "k_min")] + [("ddd_threshold", C.c_float)]


_PER_LAYER = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_mlp")
_SINGLE_A = ("embed", "lm_head", "final_norm")
_SINGLE_B = ("eagle_fc", "e_wq", "e_wk", "e_wv", "e_wo", "e_gate", "e_up", "e_down", "e_norm_attn", "e_norm_mlp",
             "ldlp_w1", "ldlp_b1", "ldlp_w2", "ldlp_b2")
_OPTIONAL = ("ldlp_wr", "ldlp_br")   # scalar-form predictor only
_ALIAS = {"e_gate": "e_w_gate", "e_up": "e_w_up", "e_down": "e_w_down"}


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _SINGLE_A] + [(n, C.POINTER(C.c_void_p)) for n in _PER_LAYER] + \
               [(n, C.c_void_p) for n in _SINGLE_B + _OPTIONAL]


_lib = None


def lib():
    """The loaded CUDA library; built in-tree on first use.  Raises if it cannot be built or loaded."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int32
    L.ada_workspace_bytes.restype = C.c_size_t
    L.ada_workspace_bytes.argtypes = [C.POINTER(Config)]
    L.ada_init.argtypes = [C.POINTER(vp), C.POINTER(Config), C.POINTER(Weights), vp, C.c_size_t, vp]
    L.ada_prefill.argtypes = [vp, C.c_int, vp, i32, vp]
    L.ada_ldlp_predict.argtypes = [vp, vp]
    L.ada_draft.argtypes = [vp, vp, vp]
    L.ada_draft_lengths.argtypes = [vp, vp]
    L.ada_label.argtypes = [vp, vp]
    L.ada_label_positions.argtypes = [vp, C.c_int, i32, i32, vp, vp, vp]
    L.ada_verify.argtypes = [vp, vp, vp, vp, vp]
    L.ada_accept.argtypes = [vp, vp, vp, vp]
    L.ada_step.argtypes = [vp, vp, vp, vp, vp]
    L.ada_force_n.argtypes = [vp, C.POINTER(i32)]
    L.ada_force_draft.argtypes = [vp, vp]
    L.ada_force_commit.argtypes = [vp, C.c_int, vp, i32]
    L.ada_get_counters.argtypes = [vp, C.POINTER(C.c_int64)]
    L.ada_debug_buffer.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(C.c_size_t)]
    L.ada_reset_status.argtypes = [vp]
    L.ada_selftest_bounded_wait.argtypes = [vp, i32, C.c_uint32, vp]
    L.ada_profile.argtypes = [vp, C.c_int]
    L.ada_get_profile.argtypes = [vp, C.POINTER(C.c_double)]
    L.ada_ldlp_eval_static.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp]
    L.ada_last_error.restype = C.c_char_p
    L.ada_last_error.argtypes = [vp]
    L.ada_destroy.argtypes = [vp]
    for name in exported_symbols:
        if name not in ("ada_workspace_bytes", "ada_last_error"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _dp(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def ada_ldlp_eval_static(w1, b1, w2, b2, embed_row, feature, n_out, z_out=None, stream=None) -> int:
    """Length predictor without a context or workspace, for callers that cannot allocate device memory
    (its scratch is a fixed 16 KiB array inside the library).  All arguments are torch device tensors:
    bf16 w1 [hid][2d], b1 [hid], w2 [n_max][hid], b2 [n_max], embed_row [d]; fp32 feature [d];
    int32 n_out [1]; optional fp32 z_out [n_max].  Returns the library's status code (0 = enqueued)."""
    hid, d2 = w1.shape
    return lib().ada_ldlp_eval_static(_dp(w1), _dp(b1), _dp(w2), _dp(b2), _dp(embed_row), _dp(feature), d2 // 2, hid,
                                      w2.shape[0], _dp(n_out), _dp(z_out),
                                      C.c_void_p(stream.cuda_stream if stream is not None else 0))


class Engine:
    """One library context plus the device tensors it borrows.

    shape: an object with the model fields (n_layers, d_model, n_heads, head_dim, d_ffn, vocab, rope_theta,
    rms_eps, ldlp_hidden, n_max).  weights: dict of uint16 numpy arrays holding bf16 bit patterns
    (per-layer entries are lists); they are uploaded as they are.
    """

    def __init__(self, shape, weights: dict, max_batch: int = 1, kv_capacity: int = 4096, device: str = "cuda:0",
                 stream=None, ldlp_mode: int = 0, ldlp_blocks: int = 2, k_min: int = 1, ddd_threshold: float = 0.0):
        import numpy as np
        import torch

        if not torch.cuda.is_available():
            raise AdaError("a CUDA device is required: this library has no CPU path")
        self.torch = torch
        self.L = lib()
        self.shape = shape
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.B, self.nmax, self.cap = max_batch, shape.n_max, kv_capacity
        self.cfg = Config(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                          shape.rope_theta, shape.rms_eps, shape.ldlp_hidden, shape.n_max, ldlp_mode, max_batch,
                          kv_capacity, 64, ldlp_blocks, k_min, ddd_threshold)
        need = self.L.ada_workspace_bytes(C.byref(self.cfg))
        if need == 0:
            raise AdaError("invalid configuration")

        def up(a):
            assert a.dtype == np.uint16
            return torch.from_numpy(a.view(np.int16)).to(self.dev).view(torch.bfloat16)

        self.w = {}
        cw = Weights()
        self._keep = []
        for n in _SINGLE_A + _SINGLE_B:
            t = up(weights[_ALIAS.get(n, n)])
            self.w[n] = t
            setattr(cw, n, t.data_ptr())
        for n in _OPTIONAL:
            if ldlp_mode == 1 and ldlp_blocks > 0:
                t = up(weights[n][:ldlp_blocks])
                self.w[n] = t
                setattr(cw, n, t.data_ptr())
        for n in _PER_LAYER:
            ts = [up(a) for a in weights[n]]
            self.w[n] = ts
            arr = (C.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
            self._keep.append(arr)
            setattr(cw, n, arr)
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.dev)
        off = (-self.workspace.data_ptr()) % 256
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.dev)
        h = C.c_void_p()
        rc = self.L.ada_init(C.byref(h), C.byref(self.cfg), C.byref(cw), C.c_void_p(self.workspace.data_ptr() + off),
                             need, C.c_void_p(self.stream.cuda_stream))
        if rc != 0:
            raise AdaError("ada_init failed: %s" % ADA_ERRORS.get(rc, rc))
        self.h = h
        self.workspace_bytes = need
        i32 = dict(dtype=torch.int32, device=self.dev)
        self.d_n = torch.zeros(self.B, **i32)
        self.d_draft = torch.zeros(self.B, self.nmax, **i32)
        self.d_target = torch.zeros(self.B, self.nmax + 1, **i32)
        self.d_accept = torch.zeros(self.B, **i32)
        self.d_emitted = torch.zeros(self.B, self.nmax + 1, **i32)
        self.d_nemit = torch.zeros(self.B, **i32)
        self.d_nused = torch.zeros(self.B, **i32)
        self.d_first = torch.zeros(1, **i32)

    def _check(self, rc, what):
        if rc != 0:
            raise AdaError("%s: %s (%s)" % (what, ADA_ERRORS.get(rc, rc), self.L.ada_last_error(self.h).decode()))

    def close(self):
        if getattr(self, "h", None):
            self.L.ada_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- the calls of include/ada.h -------------------------------------------------------------
    def ada_prefill(self, seq: int, d_prompt, d_first=None):
        self._check(self.L.ada_prefill(self.h, seq, _dp(d_prompt), d_prompt.numel(), _dp(d_first)), "ada_prefill")

    def ada_ldlp_predict(self, d_n):
        self._check(self.L.ada_ldlp_predict(self.h, _dp(d_n)), "ada_ldlp_predict")

    def ada_draft(self, d_n, d_draft):
        self._check(self.L.ada_draft(self.h, _dp(d_n), _dp(d_draft)), "ada_draft")

    def ada_label(self, d_k):
        self._check(self.L.ada_label(self.h, _dp(d_k)), "ada_label")

    def ada_label_positions(self, seq: int, j0: int, count: int, d_k, d_drafts=None, d_targets=None):
        self._check(self.L.ada_label_positions(self.h, seq, j0, count, _dp(d_k), _dp(d_drafts), _dp(d_targets)),
                    "ada_label_positions")

    def ada_draft_lengths(self, d_n):
        self._check(self.L.ada_draft_lengths(self.h, _dp(d_n)), "ada_draft_lengths")

    def ada_verify(self, d_draft, d_n, d_target, d_logits=None):
        self._check(self.L.ada_verify(self.h, _dp(d_draft), _dp(d_n), _dp(d_target), _dp(d_logits)), "ada_verify")

    def ada_accept(self, d_accept=None, d_emitted=None, d_nemit=None):
        self._check(self.L.ada_accept(self.h, _dp(d_accept), _dp(d_emitted), _dp(d_nemit)), "ada_accept")

    def ada_step(self, d_emitted=None, d_nemit=None, d_nused=None, d_accept=None):
        self._check(self.L.ada_step(self.h, _dp(d_emitted), _dp(d_nemit), _dp(d_nused), _dp(d_accept)), "ada_step")

    def ada_force_n(self, n):
        if n is None:
            self._check(self.L.ada_force_n(self.h, None), "ada_force_n")
        else:
            arr = (C.c_int32 * self.B)(*[int(v) for v in n])
            self._check(self.L.ada_force_n(self.h, arr), "ada_force_n")

    def ada_force_draft(self, d_tokens):
        self._forced = d_tokens  # keep alive
        self._check(self.L.ada_force_draft(self.h, _dp(d_tokens)), "ada_force_draft")

    def ada_force_commit(self, seq: int, d_tokens, count: int):
        self._check(self.L.ada_force_commit(self.h, seq, _dp(d_tokens), count), "ada_force_commit")

    def ada_get_counters(self) -> dict:
        out = (C.c_int64 * 8)()
        self._check(self.L.ada_get_counters(self.h, out), "ada_get_counters")
        return dict(n_target=out[0], n_draft=out[1], n_waste=out[2], n_tokens=out[3], status=out[4], launches=out[5])

    def ada_reset_status(self):
        self._check(self.L.ada_reset_status(self.h), "ada_reset_status")

    def ada_selftest_bounded_wait(self, mode: int, spin_limit: int, d_result):
        self._check(self.L.ada_selftest_bounded_wait(self.h, mode, spin_limit, _dp(d_result)), "ada_selftest_bounded_wait")

    def ada_profile(self, enable: bool):
        self._check(self.L.ada_profile(self.h, 1 if enable else 0), "ada_profile")

    def ada_get_profile(self) -> dict:
        out = (C.c_double * 8)()
        self._check(self.L.ada_get_profile(self.h, out), "ada_get_profile")
        return dict(gemm_launches=int(out[0]), gemm_ms=out[1], gemm_bytes=out[2], attn_launches=int(out[3]),
                    attn_ms=out[4])

    def ada_debug_buffer(self, which: int, dtype, shape):
        """A torch view (no copy) of an internal buffer."""
        p, nbytes = C.c_void_p(), C.c_size_t()
        self._check(self.L.ada_debug_buffer(self.h, which, C.byref(p), C.byref(nbytes)), "ada_debug_buffer")
        torch = self.torch
        off = p.value - self.workspace.data_ptr()
        return self.workspace[off: off + nbytes.value].view(dtype).view(*shape)

    # --- conveniences built from the calls above ---------------------------------------------------
    def prefill(self, seq: int, prompt) -> int:
        """Host token list / array -> first generated token (synchronises)."""
        torch = self.torch
        d_prompt = torch.as_tensor(prompt, dtype=torch.int32).to(self.dev)
        self.ada_prefill(seq, d_prompt, self.d_first)
        return int(self.d_first.cpu()[0])

    def step(self) -> dict:
        """One ada_step; returns host copies of what it emitted (synchronises)."""
        self.ada_step(self.d_emitted, self.d_nemit, self.d_nused, self.d_accept)
        ne = self.d_nemit.cpu().tolist()
        em = self.d_emitted.cpu().tolist()
        return dict(n=self.d_nused.cpu().tolist(), k=self.d_accept.cpu().tolist(), n_emitted=ne,
                    emitted=[em[b][: ne[b]] for b in range(self.B)])
