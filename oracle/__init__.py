"""CPU oracle of the adaptive speculative-decoding iteration: TEST INFRASTRUCTURE ONLY.

`ada_oracle.c` restates the decode iteration from the paper in plain fp32 C; this
module compiles it with gcc and marshals arguments through ctypes.  Only tests,
the smoke check and the benchmark's CPU-baseline leg may import it; the CUDA
library and its Python binding never do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ada_oracle.c")
_LIB = os.path.join(_HERE, "libada_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc when the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O3", "-march=native", "-ffp-contract=off", "-fopenmp", "-shared",
                               "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("ldlp_hidden", "n_max", "ldlp_mode", "ldlp_embed_shift",
                                         "ldlp_blocks", "k_min")] + [("ddd_threshold", C.c_float)]


_PER_LAYER = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm_attn", "norm_mlp")
_SINGLE_A = ("embed", "lm_head", "final_norm")
_SINGLE_B = ("eagle_fc", "e_wq", "e_wk", "e_wv", "e_wo", "e_gate", "e_up", "e_down", "e_norm_attn",
             "e_norm_mlp", "ldlp_w1", "ldlp_b1", "ldlp_w2", "ldlp_b2", "ldlp_wr", "ldlp_br")
# names in the synthetic weight dictionary that differ from the struct's
_ALIAS = {"e_gate": "e_w_gate", "e_up": "e_w_up", "e_down": "e_w_down"}


class _Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _SINGLE_A] + \
               [(n, C.POINTER(C.c_void_p)) for n in _PER_LAYER] + \
               [(n, C.c_void_p) for n in _SINGLE_B]


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(build())
    vp, i32p, f32p = C.c_void_p, C.c_void_p, C.c_void_p
    L.orc_num_threads.restype = C.c_int
    L.orc_model_create.restype = vp
    L.orc_model_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights)]
    L.orc_model_destroy.argtypes = [vp]
    L.orc_seq_create.restype = vp
    L.orc_seq_create.argtypes = [vp, C.c_int]
    L.orc_seq_destroy.argtypes = [vp]
    L.orc_prefill.argtypes = [vp, vp, i32p, C.c_int]
    L.orc_ldlp.argtypes = [vp, vp, f32p]
    L.orc_draft.argtypes = [vp, vp, C.c_int, i32p, i32p, f32p, f32p]
    L.orc_verify.argtypes = [vp, vp, i32p, C.c_int, i32p, f32p, f32p, f32p]
    L.orc_accept.argtypes = [vp, vp, i32p, i32p, C.c_int, i32p, i32p]
    L.orc_step.argtypes = [vp, vp, C.c_int, i32p, i32p, i32p, i32p, i32p, i32p, f32p, f32p, f32p, f32p, f32p, f32p]
    L.orc_draft_dyn.argtypes = [vp, vp, C.c_int, i32p, i32p, f32p, f32p, f32p, i32p]
    L.orc_label.argtypes = [vp, vp, i32p, i32p, i32p]
    L.orc_rewind.argtypes = [vp, C.c_int, C.c_int]
    L.orc_forward_nocache.argtypes = [vp, i32p, C.c_int, f32p, f32p]
    L.orc_draft_rows.argtypes = [vp, i32p, f32p, C.c_int, C.c_int, f32p, f32p, f32p]
    L.orc_seq_len.argtypes = [vp]
    L.orc_seq_dlen.argtypes = [vp]
    for name in ("orc_seq_tokens", "orc_seq_features", "orc_seq_draft_features", "orc_seq_target_k",
                 "orc_seq_target_v"):
        getattr(L, name).restype = vp
        getattr(L, name).argtypes = [vp]
    L.orc_seq_counters.argtypes = [vp, vp]
    L.orc_tau.restype = C.c_double
    L.orc_tau.argtypes = [C.c_int64, C.c_int64, C.c_int64]
    _lib = L
    return L


def num_threads() -> int:
    return _load().orc_num_threads()


def tau(n_draft: int, n_target: int, n_waste: int) -> float:
    return _load().orc_tau(n_draft, n_target, n_waste)


def _ptr(a):
    return None if a is None else a.ctypes.data


class Model:
    """The oracle's view of one set of weights (bf16 bit patterns as uint16 numpy arrays)."""

    def __init__(self, shape, weights: dict, ldlp_mode: int = 0, ldlp_embed_shift: int = 0,
                 ldlp_blocks: int = 2, k_min: int = 1, ddd_threshold: float = 0.0):
        self.lib = _load()
        self.shape = shape
        self.weights = weights  # keeps the arrays alive
        c = _Config(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                    shape.rope_theta, shape.rms_eps, shape.ldlp_hidden, shape.n_max, ldlp_mode,
                    ldlp_embed_shift, ldlp_blocks, k_min, ddd_threshold)
        w = _Weights()
        self._arrays = []
        for n in _SINGLE_A + _SINGLE_B:
            a = weights.get(_ALIAS.get(n, n))
            if a is not None:
                assert a.dtype == np.uint16 and a.flags.c_contiguous
                setattr(w, n, a.ctypes.data)
        for n in _PER_LAYER:
            arr = (C.c_void_p * shape.n_layers)(*[a.ctypes.data for a in weights[n]])
            self._arrays.append(arr)
            setattr(w, n, arr)
        self.cfg, self.w = c, w
        self.h = self.lib.orc_model_create(C.byref(c), C.byref(w))

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.orc_model_destroy(self.h)
            self.h = None

    def new_seq(self, capacity: int) -> "Seq":
        return Seq(self, capacity)

    def forward_nocache(self, tokens, want_features: bool = False):
        """Cache-free target pass; returns (logits of the last row, features or None)."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        logits = np.empty(self.shape.vocab, dtype=np.float32)
        feat = np.empty((len(t), self.shape.d_model), dtype=np.float32) if want_features else None
        rc = self.lib.orc_forward_nocache(self.h, t.ctypes.data, len(t), _ptr(feat), logits.ctypes.data)
        assert rc == 0
        return logits, feat

    def draft_rows(self, next_tok, feat, pos0: int, dk, dv):
        """Draft head alone over len(next_tok) rows starting at pos0, on caller-held caches."""
        t = np.ascontiguousarray(next_tok, dtype=np.int32)
        f = np.ascontiguousarray(feat, dtype=np.float32)
        out = np.empty((len(t), self.shape.d_model), dtype=np.float32)
        rc = self.lib.orc_draft_rows(self.h, t.ctypes.data, f.ctypes.data, len(t), pos0, dk.ctypes.data,
                                     dv.ctypes.data, out.ctypes.data)
        assert rc == 0
        return out


class Seq:
    """One sequence's state in the oracle (tokens, features, target and draft caches, counters)."""

    def __init__(self, model: Model, capacity: int):
        self.m, self.lib, self.cap = model, model.lib, capacity
        self.h = self.lib.orc_seq_create(model.h, capacity)

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.orc_seq_destroy(self.h)
            self.h = None

    @property
    def len(self):
        return self.lib.orc_seq_len(self.h)

    @property
    def dlen(self):
        return self.lib.orc_seq_dlen(self.h)

    def tokens(self) -> np.ndarray:
        p = self.lib.orc_seq_tokens(self.h)
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_int32)), shape=(self.len,)).copy()

    def features(self, lo: int, hi: int) -> np.ndarray:
        d = self.m.shape.d_model
        p = self.lib.orc_seq_features(self.h)
        a = np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_float)), shape=(self.cap, d))
        return a[lo:hi].copy()

    def draft_features(self, n: int) -> np.ndarray:
        d = self.m.shape.d_model
        p = self.lib.orc_seq_draft_features(self.h)
        return np.ctypeslib.as_array(C.cast(p, C.POINTER(C.c_float)), shape=(max(self.m.shape.n_max, 1), d))[:n].copy()

    def target_kv(self):
        s = self.m.shape
        shp = (s.n_layers, self.cap, s.d_model)
        k = np.ctypeslib.as_array(C.cast(self.lib.orc_seq_target_k(self.h), C.POINTER(C.c_float)), shape=shp)
        v = np.ctypeslib.as_array(C.cast(self.lib.orc_seq_target_v(self.h), C.POINTER(C.c_float)), shape=shp)
        return k, v

    def counters(self) -> dict:
        out = np.zeros(4, dtype=np.int64)
        self.lib.orc_seq_counters(self.h, out.ctypes.data)
        return dict(n_target=int(out[0]), n_draft=int(out[1]), n_waste=int(out[2]), n_tokens=int(out[3]))

    def prefill(self, prompt) -> int:
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        t = self.lib.orc_prefill(self.m.h, self.h, p.ctypes.data, len(p))
        assert t >= 0, "prefill failed"
        return t

    def ldlp(self):
        """Returns (n, z): the predicted draft length and the predictor's raw outputs."""
        z = np.zeros(max(self.m.shape.n_max, 1), dtype=np.float32)
        n = self.lib.orc_ldlp(self.m.h, self.h, z.ctypes.data)
        assert n >= 0
        return n, z

    def draft(self, n: int, forced=None):
        """Returns (draft tokens, top1, top2) for n draft steps."""
        out = np.zeros(n, dtype=np.int32)
        t1 = np.zeros(n, dtype=np.float32)
        t2 = np.zeros(n, dtype=np.float32)
        f = None if forced is None else np.ascontiguousarray(forced, dtype=np.int32)
        rc = self.lib.orc_draft(self.m.h, self.h, n, _ptr(f), out.ctypes.data, t1.ctypes.data, t2.ctypes.data)
        assert rc == 0, "draft failed rc=%d" % rc
        return out, t1, t2

    def draft_dyn(self, n: int, forced=None):
        """Draft with the model's stopping rule (AdaEAGLE-DDD when its threshold is negative).
        Returns (draft tokens [n_used], top1, top2, running log-probability of the draft sequence)."""
        nm = self.m.shape.n_max
        out = np.zeros(nm, dtype=np.int32)
        t1, t2, lp = (np.zeros(nm, dtype=np.float32) for _ in range(3))
        nu = C.c_int32(0)
        f = None if forced is None else np.ascontiguousarray(forced, dtype=np.int32)
        rc = self.lib.orc_draft_dyn(self.m.h, self.h, n, _ptr(f), out.ctypes.data, t1.ctypes.data, t2.ctypes.data,
                                    lp.ctypes.data, C.addressof(nu))
        assert rc == 0, "draft failed rc=%d" % rc
        k = nu.value
        return out[:k].copy(), t1[:k].copy(), t2[:k].copy(), lp[:k].copy()

    def verify(self, draft, want_logits: bool = False):
        """Returns (target tokens [n+1], top1, top2, logits or None)."""
        d = np.ascontiguousarray(draft, dtype=np.int32)
        n = len(d)
        tt = np.zeros(n + 1, dtype=np.int32)
        t1 = np.zeros(n + 1, dtype=np.float32)
        t2 = np.zeros(n + 1, dtype=np.float32)
        lg = np.empty((n + 1, self.m.shape.vocab), dtype=np.float32) if want_logits else None
        rc = self.lib.orc_verify(self.m.h, self.h, d.ctypes.data if n else None, n, tt.ctypes.data, _ptr(lg),
                                 t1.ctypes.data, t2.ctypes.data)
        assert rc == 0, "verify failed rc=%d" % rc
        return tt, t1, t2, lg

    def accept(self, draft, target_tok):
        """Returns (k_accept, emitted tokens)."""
        d = np.ascontiguousarray(draft, dtype=np.int32)
        t = np.ascontiguousarray(target_tok, dtype=np.int32)
        em = np.zeros(len(d) + 1, dtype=np.int32)
        ne = C.c_int32(0)
        k = self.lib.orc_accept(self.m.h, self.h, d.ctypes.data if len(d) else None, t.ctypes.data, len(d),
                                em.ctypes.data, C.addressof(ne))
        return k, em[: ne.value].copy()

    def step(self, n_forced: int = -1, forced_draft=None) -> dict:
        """One iteration (predict -> draft -> verify -> accept); returns everything observed."""
        nm = max(self.m.shape.n_max, 1)
        em = np.zeros(nm + 1, dtype=np.int32)
        ne, nu = C.c_int32(0), C.c_int32(0)
        dr = np.zeros(nm, dtype=np.int32)
        tg = np.zeros(nm + 1, dtype=np.int32)
        v1, v2 = np.zeros(nm + 1, dtype=np.float32), np.zeros(nm + 1, dtype=np.float32)
        d1, d2 = np.zeros(nm, dtype=np.float32), np.zeros(nm, dtype=np.float32)
        z = np.zeros(nm, dtype=np.float32)
        lp = np.zeros(nm, dtype=np.float32)
        f = None if forced_draft is None else np.ascontiguousarray(forced_draft, dtype=np.int32)
        j = self.len - 1
        k = self.lib.orc_step(self.m.h, self.h, n_forced, _ptr(f), em.ctypes.data, C.addressof(ne),
                              C.addressof(nu), dr.ctypes.data, tg.ctypes.data, v1.ctypes.data, v2.ctypes.data,
                              d1.ctypes.data, d2.ctypes.data, z.ctypes.data, lp.ctypes.data)
        assert k >= 0, "step failed rc=%d" % k
        n = nu.value
        return dict(j=j, n=n, k=k, emitted=em[: ne.value].copy(), draft=dr[:n].copy(), target=tg[: n + 1].copy(),
                    v_top1=v1[: n + 1].copy(), v_top2=v2[: n + 1].copy(), d_top1=d1[:n].copy(),
                    d_top2=d2[:n].copy(), ldlp_z=z.copy(), d_logp=lp[:n].copy())

    def label(self) -> int:
        """The optimal draft length for the current state (longest confirmed prefix of a full-length draft);
        the sequence is left unchanged."""
        k = self.lib.orc_label(self.m.h, self.h, None, None, None)
        assert k >= 0, "label failed rc=%d" % k
        return k

    def label_tokens(self):
        """As label(), also returning what it was decided on: (k, drafted tokens [n], target choices [n + 1])."""
        nm = max(self.m.shape.n_max, 1)
        dr, tg = np.zeros(nm, dtype=np.int32), np.zeros(nm + 1, dtype=np.int32)
        n = C.c_int32(0)
        k = self.lib.orc_label(self.m.h, self.h, dr.ctypes.data, tg.ctypes.data, C.addressof(n))
        assert k >= 0, "label failed rc=%d" % k
        return k, dr[: n.value].copy(), tg[: n.value + 1].copy()

    def label_positions(self, j0: int, count: int) -> dict:
        """Labels of Section 3.3 for start positions j0 .. j0 + count - 1 of this sequence's committed tokens: for each
        j the sequence is rolled back to the state in which token j was pending and labelled (Seq.label_tokens: the
        label, the drafts, the target's choices).  Positions
        run from the last to the first, so that a label never reads a cache row a later position's passes wrote.
        The sequence is left rolled back to j0: use a sequence kept for this purpose."""
        out = {}
        for j in range(j0 + count - 1, j0 - 1, -1):
            self.rewind(j + 1, min(self.dlen, j - 1))
            out[j] = self.label_tokens()
        return out

    def rewind(self, length: int, dlen: int) -> None:
        """Back to an earlier state of this sequence: `length` committed tokens (the last one pending), `dlen`
        draft-head rows of true features; counters restart."""
        rc = self.lib.orc_rewind(self.h, length, dlen)
        assert rc == 0, "rewind out of range"


def decode(model: Model, prompt, max_new: int, n_policy=-1, capacity=None, forced_stream=None) -> dict:
    """Algorithm 1 until max_new tokens are emitted (overshoot trimmed).

    n_policy: -1 = length predictor, 0 = plain autoregressive, k > 0 = fixed length,
    or a callable (iteration index, Seq) -> n.  forced_stream: optional token array;
    the drafts of an iteration starting at pending index j are forced to
    forced_stream[j+1-len(prompt)-1 ...] (teacher forcing).
    """
    s = model.shape
    cap = capacity or (len(prompt) + max_new + s.n_max + 2)
    seq = model.new_seq(cap)
    first = seq.prefill(prompt)
    out = [first]
    iters = []
    r = 0
    while len(out) < max_new:
        n = n_policy(r, seq) if callable(n_policy) else n_policy
        forced = None
        if forced_stream is not None:
            forced = np.asarray(forced_stream[len(out): len(out) + max(s.n_max, 1)], dtype=np.int32)
            if len(forced) < max(s.n_max, 1):
                forced = np.concatenate([forced, np.zeros(max(s.n_max, 1) - len(forced), dtype=np.int32)])
        it = seq.step(n, forced)
        iters.append(it)
        out.extend(int(t) for t in it["emitted"])
        r += 1
    return dict(tokens=np.array(out[:max_new], dtype=np.int32), iters=iters, seq=seq, counters=seq.counters())
