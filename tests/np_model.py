"""Independent float64 numpy decoder used only to pin the oracle.

It recomputes every position of a whole token sequence from scratch (no KV cache, whole-matrix
products, rotary embedding as a complex multiplication, masked softmax), i.e. a different formulation
from the oracle's cached row-by-row C code.
"""
from __future__ import annotations

import numpy as np

import synth


def _f64(a):
    return synth.bf16_to_f32(a).astype(np.float64)


def rmsnorm(x, gain, eps):
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * gain


def rope_complex(x, positions, hd, theta):
    """x: [T, n_heads, hd]; pairs (j, j + hd/2) form complex numbers rotated by pos * theta^(-2j/hd)."""
    half = hd // 2
    freqs = theta ** (-2.0 * np.arange(half) / hd)
    ang = positions[:, None] * freqs[None, :]
    z = x[..., :half] + 1j * x[..., half:]
    z = z * np.exp(1j * ang)[:, None, :]
    return np.concatenate([z.real, z.imag], axis=-1)


def forward_all(cfg, w: synth.Weights, tokens, n_layers=None):
    """Hidden states of every layer for every position: list of [T, d] arrays, index 0 = embedding."""
    tokens = np.asarray(tokens)
    T = len(tokens)
    L = cfg.n_layers if n_layers is None else n_layers
    nh, nkv, hd = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    pos = np.arange(T, dtype=np.float64)
    h = _f64(w.tok_emb)[tokens]
    out = [h]
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)
    for l in range(L):
        lw = w.layers[l]
        a = rmsnorm(h, _f64(lw["attn_norm"]), cfg.rms_eps)
        q = (a @ _f64(lw["wq"]).T).reshape(T, nh, hd)
        k = (a @ _f64(lw["wk"]).T).reshape(T, nkv, hd)
        v = (a @ _f64(lw["wv"]).T).reshape(T, nkv, hd)
        q = rope_complex(q, pos, hd, cfg.rope_theta)
        k = rope_complex(k, pos, hd, cfg.rope_theta)
        k = np.repeat(k, nh // nkv, axis=1)
        v = np.repeat(v, nh // nkv, axis=1)
        sc = np.einsum("thd,shd->hts", q, k) / np.sqrt(hd)
        sc = np.where(mask[None], -np.inf, sc)
        sc = sc - sc.max(axis=-1, keepdims=True)
        p = np.exp(sc)
        p = p / p.sum(axis=-1, keepdims=True)
        o = np.einsum("hts,shd->thd", p, v).reshape(T, nh * hd)
        h = h + o @ _f64(lw["wo"]).T
        b = rmsnorm(h, _f64(lw["ffn_norm"]), cfg.rms_eps)
        g = b @ _f64(lw["w_gate"]).T
        u = b @ _f64(lw["w_up"]).T
        h = h + ((g / (1.0 + np.exp(-g))) * u) @ _f64(lw["w_down"]).T
        out.append(h)
    return out


def kv_rows(cfg, w: synth.Weights, h_in, layer: int):
    """Keys (rotated) and values (not rotated) that 1-based `layer` caches for every position, from the hidden
    states entering it: two [T, n_kv_heads * hd] arrays."""
    lw = w.layers[layer - 1]
    T = h_in.shape[0]
    a = rmsnorm(h_in, _f64(lw["attn_norm"]), cfg.rms_eps)
    k = (a @ _f64(lw["wk"]).T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
    v = a @ _f64(lw["wv"]).T
    k = rope_complex(k, np.arange(T, dtype=np.float64), cfg.head_dim, cfg.rope_theta)
    return k.reshape(T, -1), v


def exit_logits(cfg, w: synth.Weights, h):
    """Shared final RMSNorm + LM head on hidden rows [.., d] -> logits [.., V]."""
    a = rmsnorm(h, _f64(w.final_norm), cfg.rms_eps)
    return a @ _f64(w.lm_head).T
