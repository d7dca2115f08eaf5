"""Seeded synthetic inputs: model shapes, weights (bf16 bit patterns) and prompts.

This package only produces INPUTS.  It is the one module that both the CPU
oracle's tests and the CUDA path's tests / bench import; it holds none of the
decoding method's arithmetic.  The numeric kernel is ``gen.c`` (a counter-based
hash feeding a 65536-entry normal-quantile table), compiled on first use.

The five named configurations reproduce the shapes of the benchmark contract:
a tiny 4-layer decoder, and Llama-2-7B / Llama-3.2-1B / Llama-2-13B /
Llama-3-8B shaped decoders with random weights whose residual-branch output
projections decay with depth so that early-exit predictions agree with the
final layer more often the deeper the exit.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field, replace
from typing import Dict, List

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libsynth.so")
_SRC = os.path.join(_HERE, "gen.c")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libsynth.so (gcc, OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        lib.synth_normal_bf16.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64,
                                          ctypes.c_float, ctypes.c_float, ctypes.c_void_p]
        lib.synth_gain_bf16.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64,
                                        ctypes.c_float, ctypes.c_void_p]
        lib.synth_tokens.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64,
                                     ctypes.c_int32, ctypes.c_void_p]
        lib.synth_uniform_int.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64,
                                          ctypes.c_int32]
        lib.synth_uniform_int.restype = ctypes.c_int32
        _lib = lib
    return _lib


@dataclass(frozen=True)
class Config:
    """Model shape + workload of one benchmark configuration."""
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 1e4
    batch: int = 1
    prompt_len: int = 32
    gen_len: int = 64
    e_min: int = 1
    e_max: int = 3
    g_min: int = 1
    g_max: int = 4
    page_size: int = 16
    init_window: int = 32
    omega: float = 0.95
    seed: int = 20250405
    weight_std: float = 0.02
    # residual-branch scaling: "tiny" = layers >= 3 scaled by 0.1; "decay" = 0.5 ** (l / 8), l 1-based
    residual_scaling: str = "decay"
    gain_spread: float = 0.0          # 0 -> all norm gains exactly 1.0
    # the token-embedding table is drawn with std weight_std * emb_scale = 1.0: with std 0.02 the
    # residual stream forgets the current token after layer 1 and greedy decoding emits one constant token
    emb_scale: float = 50.0
    prompt_kind: str = "uniform"      # or "spans64"

    @property
    def max_seq(self) -> int:
        ps = self.page_size
        need = self.prompt_len + self.gen_len + self.g_max + 1
        return (need + ps - 1) // ps * ps

    def layer_bytes(self) -> int:
        d, hd = self.d_model, self.head_dim
        return 2 * (d * (self.n_heads + 2 * self.n_kv_heads) * hd + self.n_heads * hd * d
                    + 3 * d * self.d_ffn) + 4 * d

    def lm_head_bytes(self) -> int:
        return 2 * self.vocab * self.d_model

    def kv_bytes_per_pos_layer(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * 2


CONFIGS: Dict[str, Config] = {
    "tiny": Config("tiny", 4, 256, 4, 4, 64, 688, 1024, prompt_len=32, gen_len=64,
                   e_min=1, e_max=3, g_min=1, g_max=4, seed=20250405 + 1, residual_scaling="tiny"),
    "llama2_7b": Config("llama2_7b", 32, 4096, 32, 32, 128, 11008, 32000, prompt_len=512, gen_len=256,
                        e_min=4, e_max=28, g_min=1, g_max=12, seed=20250405 + 2),
    "llama32_1b": Config("llama32_1b", 16, 2048, 32, 8, 64, 8192, 128256, rope_theta=5e5,
                         prompt_len=1024, gen_len=256, e_min=2, e_max=14, g_min=1, g_max=10,
                         seed=20250405 + 3),
    "llama2_13b": Config("llama2_13b", 40, 5120, 40, 40, 128, 13824, 32000, prompt_len=3072, gen_len=128,
                         e_min=4, e_max=36, g_min=1, g_max=12, seed=20250405 + 4, prompt_kind="spans64"),
    "llama3_8b_b4": Config("llama3_8b_b4", 32, 4096, 32, 8, 128, 14336, 128256, rope_theta=5e5, batch=4,
                           prompt_len=1024, gen_len=512, e_min=4, e_max=28, g_min=1, g_max=12,
                           seed=20250405 + 5),
}


def small_variant(cfg: Config, **kw) -> Config:
    """A reshaped copy (tests use it for ragged / GQA / non-unit-gain cases)."""
    return replace(cfg, **kw)


# tensor ids: fixed enumeration
TID_TOK_EMB, TID_LM_HEAD, TID_FINAL_NORM = 1, 2, 3
_LAYER_FIELDS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def _tid(layer1: int, field_index: int) -> int:
    return 16 * layer1 + field_index


def residual_scale(cfg: Config, layer1: int) -> float:
    """Factor applied to o_proj / down_proj of 1-based layer ``layer1``."""
    if cfg.residual_scaling == "tiny":
        return 0.1 if layer1 >= 3 else 1.0
    if cfg.residual_scaling == "decay":
        return float(0.5 ** (layer1 / 8.0))
    return 1.0


def _normal(cfg: Config, tid: int, shape, scale: float = 1.0) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(cfg.seed, tid, out.size, cfg.weight_std, scale, out.ctypes.data)
    return out


def _gain(cfg: Config, tid: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.uint16)
    _load().synth_gain_bf16(cfg.seed, tid, n, cfg.gain_spread, out.ctypes.data)
    return out


@dataclass
class Weights:
    """All tensors as numpy uint16 arrays holding bf16 bit patterns; matrices are [out, in] row-major."""
    tok_emb: np.ndarray
    lm_head: np.ndarray
    final_norm: np.ndarray
    layers: List[Dict[str, np.ndarray]] = field(default_factory=list)

    def nbytes(self) -> int:
        n = self.tok_emb.nbytes + self.lm_head.nbytes + self.final_norm.nbytes
        for lw in self.layers:
            n += sum(a.nbytes for a in lw.values())
        return n


def make_layer(cfg: Config, layer1: int) -> Dict[str, np.ndarray]:
    d, hd, F = cfg.d_model, cfg.head_dim, cfg.d_ffn
    nq, nk = cfg.n_heads * hd, cfg.n_kv_heads * hd
    rs = residual_scale(cfg, layer1)
    return {
        "attn_norm": _gain(cfg, _tid(layer1, 0), d),
        "wq": _normal(cfg, _tid(layer1, 1), (nq, d)),
        "wk": _normal(cfg, _tid(layer1, 2), (nk, d)),
        "wv": _normal(cfg, _tid(layer1, 3), (nk, d)),
        "wo": _normal(cfg, _tid(layer1, 4), (d, nq), rs),
        "ffn_norm": _gain(cfg, _tid(layer1, 5), d),
        "w_gate": _normal(cfg, _tid(layer1, 6), (F, d)),
        "w_up": _normal(cfg, _tid(layer1, 7), (F, d)),
        "w_down": _normal(cfg, _tid(layer1, 8), (d, F), rs),
    }


def make_weights(cfg: Config) -> Weights:
    w = Weights(
        tok_emb=_normal(cfg, TID_TOK_EMB, (cfg.vocab, cfg.d_model), cfg.emb_scale),
        lm_head=_normal(cfg, TID_LM_HEAD, (cfg.vocab, cfg.d_model)),
        final_norm=_gain(cfg, TID_FINAL_NORM, cfg.d_model),
    )
    for l1 in range(1, cfg.n_layers + 1):
        w.layers.append(make_layer(cfg, l1))
    return w


def make_prompt(cfg: Config, seq: int = 0) -> np.ndarray:
    """Prompt token ids (int32) of sequence ``seq`` of the batch."""
    lib = _load()
    P = cfg.prompt_len
    out = np.empty(P, dtype=np.int32)
    stream = 1000 + seq
    if cfg.prompt_kind == "uniform":
        lib.synth_tokens(cfg.seed, stream, P, cfg.vocab, out.ctypes.data)
        return out
    if cfg.prompt_kind == "spans64":
        # slots of 64 tokens, each a copy of one of 12 seeded random spans
        span, pool = 64, 12
        spans = np.empty((pool, span), dtype=np.int32)
        for j in range(pool):
            lib.synth_tokens(cfg.seed, 2000 + 16 * seq + j, span, cfg.vocab, spans[j].ctypes.data)
        n_slots = (P + span - 1) // span
        buf = np.empty(n_slots * span, dtype=np.int32)
        for s in range(n_slots):
            j = lib.synth_uniform_int(cfg.seed, 3000 + seq, s, pool)
            buf[s * span:(s + 1) * span] = spans[j]
        return buf[:P].copy()
    raise ValueError(cfg.prompt_kind)


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Expand bf16 bit patterns to float32 (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32)
