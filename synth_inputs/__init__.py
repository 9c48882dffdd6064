"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

Only reproducible random data lives here (weights as bf16 bit patterns, prompt
token ids, ragged prompt lengths) plus the shape tables of the five workloads.
None of the decoding method's arithmetic is in this module.

The model's weights ARE the bf16-rounded values: both consumers read the same
uint16 bit patterns, one widens them to fp32 on the CPU, the other uploads them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libsynth.so")

DEFAULT_SEED = 20241218


def build(force: bool = False) -> str:
    """Compile gen.c into libsynth.so with gcc when missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.synth_normal_bf16.argtypes = [ctypes.c_uint64, ctypes.c_double, ctypes.c_int64, ctypes.c_void_p]
        lib.synth_const_bf16.argtypes = [ctypes.c_double, ctypes.c_int64, ctypes.c_void_p]
        lib.synth_uniform_i32.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p]
        for f in (lib.synth_normal_bf16, lib.synth_const_bf16, lib.synth_uniform_i32):
            f.restype = None
        _lib = lib
    return _lib


def _fnv1a64(name: str) -> int:
    h = 0xCBF29CE484222325
    for b in name.encode():
        h = ((h ^ b) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _key(seed: int, name: str) -> int:
    return (seed * 0x9E3779B97F4A7C15 ^ _fnv1a64(name)) & 0xFFFFFFFFFFFFFFFF


def normal_bf16(seed: int, name: str, shape, std: float = 0.02) -> np.ndarray:
    """uint16 array of bf16 bit patterns of std*N(0,1), keyed by (seed, name)."""
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(_key(seed, name), float(std), out.size, out.ctypes.data)
    return out


def const_bf16(value: float, shape) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_const_bf16(float(value), out.size, out.ctypes.data)
    return out


def uniform_ids(seed: int, name: str, count: int, modulus: int) -> np.ndarray:
    out = np.empty(count, dtype=np.int32)
    _load().synth_uniform_i32(_key(seed, name), int(modulus), out.size, out.ctypes.data)
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


@dataclass(frozen=True)
class Shape:
    """Model and workload shape of one configuration."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    ldlp_hidden: int
    n_max: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-6
    kv_capacity: int = 4096
    batch: int = 1
    prompt_len: int = 64          # batch 1; ragged batches draw lengths from prompt_range
    prompt_range: tuple = ()
    max_new: int = 32


SHAPES = {
    "tiny": Shape("tiny", 2, 256, 4, 64, 688, 4096, 128, 8, kv_capacity=512, prompt_len=64, max_new=32),
    "7b": Shape("7b", 32, 4096, 32, 128, 11008, 32000, 512, 10, prompt_len=512, max_new=256),
    "7b_tf": Shape("7b_tf", 32, 4096, 32, 128, 11008, 32000, 512, 10, prompt_len=1024, max_new=64 * 11),
    "13b": Shape("13b", 40, 5120, 40, 128, 13824, 32000, 512, 10, prompt_len=1024, max_new=256),
    "7b_b8": Shape("7b_b8", 32, 4096, 32, 128, 11008, 32000, 512, 10, batch=8, prompt_range=(128, 2048), max_new=128),
}


def scaled(shape: Shape, **kw) -> Shape:
    """A copy of `shape` with some fields changed (e.g. fewer layers for a quick case)."""
    return replace(shape, **kw)


TARGET_LAYER_TENSORS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


LDLP_BLOCKS = 2   # residual blocks generated for the scalar-form predictor


def make_weights(shape: Shape, seed: int = DEFAULT_SEED) -> dict:
    """All model tensors as uint16 bf16 bit patterns, row-major [out][in].

    Linear and embedding weights and the predictor's biases are 0.02*N(0,1);
    RMSNorm gains are 1.0.  Per-layer tensors are lists of arrays.
    """
    d, f, v, hid, nmax = shape.d_model, shape.d_ffn, shape.vocab, shape.ldlp_hidden, shape.n_max
    dims = {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
            "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    w = {"embed": normal_bf16(seed, "embed", (v, d)),
         "lm_head": normal_bf16(seed, "lm_head", (v, d)),
         "final_norm": const_bf16(1.0, (d,))}
    for t in TARGET_LAYER_TENSORS:
        w[t] = [normal_bf16(seed, "layer%d.%s" % (l, t), dims[t]) for l in range(shape.n_layers)]
    w["norm_attn"] = [const_bf16(1.0, (d,)) for _ in range(shape.n_layers)]
    w["norm_mlp"] = [const_bf16(1.0, (d,)) for _ in range(shape.n_layers)]
    w["eagle_fc"] = normal_bf16(seed, "eagle.fc", (d, 2 * d))
    for t in TARGET_LAYER_TENSORS:
        w["e_" + t] = normal_bf16(seed, "eagle.%s" % t, dims[t])
    w["e_norm_attn"] = const_bf16(1.0, (d,))
    w["e_norm_mlp"] = const_bf16(1.0, (d,))
    w["ldlp_w1"] = normal_bf16(seed, "ldlp.w1", (hid, 2 * d))
    w["ldlp_b1"] = normal_bf16(seed, "ldlp.b1", (hid,))
    w["ldlp_w2"] = normal_bf16(seed, "ldlp.w2", (nmax, hid))
    w["ldlp_b2"] = normal_bf16(seed, "ldlp.b2", (nmax,))
    # scalar-form predictor (Eq. 3): residual blocks between the two linear maps
    w["ldlp_wr"] = normal_bf16(seed, "ldlp.wr", (LDLP_BLOCKS, hid, hid))
    w["ldlp_br"] = normal_bf16(seed, "ldlp.br", (LDLP_BLOCKS, hid))
    return w


def make_prompts(shape: Shape, seed: int = DEFAULT_SEED) -> list:
    """One int32 array of uniform-random token ids per sequence of the batch."""
    if shape.batch == 1 and not shape.prompt_range:
        lens = [shape.prompt_len]
    else:
        lo, hi = shape.prompt_range
        lens = (uniform_ids(seed, "prompt_lens", shape.batch, hi - lo + 1) + lo).tolist()
    return [uniform_ids(seed, "prompt%d" % b, int(m), shape.vocab) for b, m in enumerate(lens)]
