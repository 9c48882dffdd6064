"""Stock-op (PyTorch CPU, fp64) restatement of the Llama-style block, used only to pin the oracle.

Written independently of the oracle's C code: whole-matrix matmuls, torch.softmax, complex-free
rotate-half rotary embedding built from torch.cat.
"""
import numpy as np
import torch

import synth_inputs as si


def t64(bits):
    return torch.from_numpy(si.bf16_bits_to_f32(np.asarray(bits)).astype(np.float64))


def rms(x, g, eps):
    return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + eps) * g


def rotate_half(x):
    h = x.shape[-1] // 2
    return torch.cat([-x[..., h:], x[..., :h]], dim=-1)


def rotary(x, pos, theta):
    # x: [T, H, hd]; pos: [T]
    hd = x.shape[-1]
    inv = theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]
    cos = torch.cat([ang.cos(), ang.cos()], -1)[:, None, :]
    sin = torch.cat([ang.sin(), ang.sin()], -1)[:, None, :]
    return x * cos + rotate_half(x) * sin


def block(h, lw, shape, pos0=0):
    """h: [T, d] rows at positions pos0..; full causal attention among the T rows (pos0 must be 0
    unless the caller passes the whole history)."""
    T, d = h.shape
    H, hd = shape.n_heads, shape.head_dim
    pos = torch.arange(pos0, pos0 + T)
    u = rms(h, lw["na"], shape.rms_eps)
    q = rotary((u @ lw["wq"].T).view(T, H, hd), pos, shape.rope_theta)
    k = rotary((u @ lw["wk"].T).view(T, H, hd), pos, shape.rope_theta)
    v = (u @ lw["wv"].T).view(T, H, hd)
    s = torch.einsum("qhd,khd->hqk", q, k) / np.sqrt(hd)
    mask = torch.ones(T, T, dtype=torch.bool).tril()
    s = s.masked_fill(~mask, float("-inf"))
    a = torch.einsum("hqk,khd->qhd", torch.softmax(s, -1), v).reshape(T, d)
    h = h + a @ lw["wo"].T
    u = rms(h, lw["nm"], shape.rms_eps)
    return h + (torch.nn.functional.silu(u @ lw["wg"].T) * (u @ lw["wu"].T)) @ lw["wd"].T


def target_layer_weights(w, l):
    return dict(wq=t64(w["wq"][l]), wk=t64(w["wk"][l]), wv=t64(w["wv"][l]), wo=t64(w["wo"][l]),
                wg=t64(w["w_gate"][l]), wu=t64(w["w_up"][l]), wd=t64(w["w_down"][l]),
                na=t64(w["norm_attn"][l]), nm=t64(w["norm_mlp"][l]))


def eagle_layer_weights(w):
    return dict(wq=t64(w["e_wq"]), wk=t64(w["e_wk"]), wv=t64(w["e_wv"]), wo=t64(w["e_wo"]),
                wg=t64(w["e_w_gate"]), wu=t64(w["e_w_up"]), wd=t64(w["e_w_down"]),
                na=t64(w["e_norm_attn"]), nm=t64(w["e_norm_mlp"]))


def target_features(w, shape, tokens):
    h = t64(w["embed"])[torch.as_tensor(np.asarray(tokens), dtype=torch.long)]
    for l in range(shape.n_layers):
        h = block(h, target_layer_weights(w, l), shape)
    return rms(h, t64(w["final_norm"]), shape.rms_eps)


def target_logits(w, shape, tokens):
    return target_features(w, shape, tokens) @ t64(w["lm_head"]).T
