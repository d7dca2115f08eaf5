"""ctypes access to the CPU oracle (``del_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``; the product package never imports it
and it imports nothing from the product.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libdel_oracle.so")
_SRCS = [os.path.join(_HERE, "del_oracle.c"), os.path.join(_HERE, "del_oracle.h")]
_lib = None
MAX_GAMMA = 32


def build(force: bool = False) -> str:
    newest = max(os.path.getmtime(p) for p in _SRCS)
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < newest:
        subprocess.check_call(["gcc", "-O3", "-march=native", "-mprefer-vector-width=512", "-ffp-contract=off", "-fopenmp", "-shared",
                               "-fPIC", "-o", _SO, _SRCS[0], "-lm"])
    return _SO


class Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn",
                                         "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("max_seq", C.c_int32)] + \
               [(n, C.c_int32) for n in ("e_min", "e_max", "g_min", "g_max", "init_window")] + \
               [("omega", C.c_double)]


_P16 = C.POINTER(C.c_uint16)
_PP16 = C.POINTER(_P16)


class WeightsC(C.Structure):
    _fields_ = [("tok_emb", _P16), ("final_norm", _P16), ("lm_head", _P16)] + \
               [(n, _PP16) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class RoundInfo(C.Structure):
    _fields_ = [("E", C.c_int32), ("gamma", C.c_int32), ("g", C.c_int32), ("n_accept", C.c_int32),
                ("n_emitted", C.c_int32), ("drafts", C.c_int32 * MAX_GAMMA),
                ("emitted", C.c_int32 * (MAX_GAMMA + 1)), ("next_E", C.c_int32), ("next_gamma", C.c_int32),
                ("loaded_layers", C.c_int32), ("Sn", C.c_double),
                ("stopped", C.c_int32), ("pad_", C.c_int32), ("tau", C.c_double), ("next_tau", C.c_double),
                ("draft_conf", C.c_double * (MAX_GAMMA + 1))]


class SampleInfo(C.Structure):
    _fields_ = [("n_tests", C.c_int32), ("from_residual", C.c_int32), ("u_draft", C.c_double * MAX_GAMMA),
                ("u_accept", C.c_double * MAX_GAMMA), ("u_final", C.c_double), ("q_x", C.c_double * MAX_GAMMA),
                ("p_x", C.c_double * MAX_GAMMA)]


def lib():
    global _lib
    if _lib is not None:
        return _lib
    build()
    L = C.CDLL(_SO)
    vp, i32, f32, f64 = C.c_void_p, C.c_int32, C.c_float, C.c_double
    L.ora_seq_create.restype = vp
    L.ora_seq_create.argtypes = [C.POINTER(Shape), C.POINTER(WeightsC)]
    L.ora_seq_destroy.argtypes = [vp]
    L.ora_set_policy.argtypes = [vp, i32, i32]
    L.ora_prefill.restype = i32
    L.ora_prefill.argtypes = [vp, vp, i32, vp, vp, C.POINTER(RoundInfo)]
    L.ora_round.restype = C.c_int
    L.ora_round.argtypes = [vp, i32, C.POINTER(RoundInfo), vp, vp, vp]
    L.ora_committed_len.restype = i32
    L.ora_committed_len.argtypes = [vp]
    L.ora_get_stats.argtypes = [vp, vp, C.POINTER(f64), C.POINTER(i32), C.POINTER(i32)]
    L.ora_set_stats.argtypes = [vp, vp, f64, i32, i32]
    for fn in ("ora_hidden", "ora_k_row", "ora_v_row"):
        getattr(L, fn).restype = C.POINTER(f32)
        getattr(L, fn).argtypes = [vp, i32, i32]
    L.ora_embed.argtypes = [vp, i32, vp]
    L.ora_rmsnorm.argtypes = [vp, vp, i32, f32, vp]
    L.ora_rope.argtypes = [vp, i32, i32, i32, f32]
    L.ora_softmax.argtypes = [vp, i32, vp]
    L.ora_silu.restype = f32
    L.ora_silu.argtypes = [f32]
    L.ora_layer_rows.argtypes = [vp, i32, vp, i32, i32, vp]
    L.ora_exit_head.argtypes = [vp, vp, C.POINTER(i32), C.POINTER(f32), vp]
    L.ora_accept_len.restype = i32
    L.ora_accept_len.argtypes = [vp, vp, i32]
    L.ora_decay_step.restype = f64
    L.ora_decay_step.argtypes = [f64, f64, f64]
    L.ora_tpl.restype = f64
    L.ora_tpl.argtypes = [f64, i32, i32, i32]
    L.ora_select.argtypes = [vp, f64, i32, i32, i32, i32, i32, C.POINTER(i32), C.POINTER(i32)]
    L.ora_num_threads.restype = C.c_int
    L.ora_set_policy_fs.argtypes = [vp, i32, i32]
    L.ora_fs_next_gamma.restype = i32
    L.ora_fs_next_gamma.argtypes = [i32, i32, i32, i32, i32]
    L.ora_set_exit_mode.argtypes = [vp, i32]
    L.ora_get_conf_stats.argtypes = [vp, vp, vp, vp]
    L.ora_set_conf_stats.argtypes = [vp, vp, vp]
    L.ora_get_conf.argtypes = [vp, vp, i32]
    L.ora_confidence.restype = f64
    L.ora_confidence.argtypes = [vp, i32]
    L.ora_threshold.restype = f64
    L.ora_threshold.argtypes = [f64, f64, f64, f64]
    L.ora_uniform.restype = f64
    L.ora_uniform.argtypes = [C.c_uint64, C.c_int64, i32]
    L.ora_nucleus.argtypes = [vp, i32, f64, f64, vp]
    L.ora_sample_cdf.restype = i32
    L.ora_sample_cdf.argtypes = [vp, i32, f64]
    L.ora_residual.restype = f64
    L.ora_residual.argtypes = [vp, vp, i32, vp]
    L.ora_set_sampling.argtypes = [vp, f64, f64, C.c_uint64]
    L.ora_get_sample_info.argtypes = [vp, C.POINTER(SampleInfo)]
    L.ora_round_logits.restype = C.POINTER(f32)
    L.ora_round_logits.argtypes = [vp, i32, i32]
    _lib = L
    return L


def _p16(a: np.ndarray):
    assert a.dtype == np.uint16 and a.flags.c_contiguous
    return a.ctypes.data_as(_P16)


class Round:
    """Plain-Python copy of one round's record."""
    __slots__ = ("E", "gamma", "g", "n_accept", "emitted", "drafts", "next_E", "next_gamma", "loaded_layers",
                 "shadow", "margin", "counts", "Sn", "stopped", "tau", "next_tau", "draft_conf", "conf")

    def __init__(self, info: RoundInfo, shadow, margin, counts):
        self.E, self.gamma, self.g, self.n_accept = info.E, info.gamma, info.g, info.n_accept
        self.emitted = [int(info.emitted[i]) for i in range(info.n_emitted)]
        self.drafts = [int(info.drafts[i]) for i in range(info.g)]
        self.next_E, self.next_gamma = info.next_E, info.next_gamma
        self.loaded_layers, self.Sn = info.loaded_layers, info.Sn
        self.shadow, self.margin, self.counts = shadow, margin, counts
        self.stopped, self.tau, self.next_tau = bool(info.stopped), info.tau, info.next_tau
        self.draft_conf = [float(info.draft_conf[i]) for i in range(info.g + info.stopped)]
        self.conf = None            # [L][columns] confidence of the shadow tokens, filled by OracleSeq


class OracleSeq:
    """One sequence decoded by the oracle: KV cache, statistics and the (E, gamma) policy.

    ``cfg`` needs the attributes of ``synth.Config``; ``weights`` those of ``synth.Weights``
    (numpy uint16 arrays of bf16 bit patterns).
    """

    def __init__(self, cfg, weights, max_seq: Optional[int] = None):
        self.cfg, self.weights = cfg, weights
        L = cfg.n_layers
        self.shape = Shape(L, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab,
                           cfg.rms_eps, cfg.rope_theta, max_seq or cfg.max_seq, cfg.e_min, cfg.e_max,
                           cfg.g_min, cfg.g_max, cfg.init_window, cfg.omega)
        self._keep = []
        wc = WeightsC()
        wc.tok_emb, wc.final_norm, wc.lm_head = _p16(weights.tok_emb), _p16(weights.final_norm), _p16(weights.lm_head)
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
            arr = (_P16 * L)(*[_p16(weights.layers[l][name]) for l in range(L)])
            self._keep.append(arr)
            setattr(wc, name, C.cast(arr, _PP16))
        self._wc = wc
        self._h = lib().ora_seq_create(C.byref(self.shape), C.byref(wc))
        self.stride = cfg.g_max + 1

    def close(self):
        if self._h:
            lib().ora_seq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- policy / state
    def set_policy(self, E: int, gamma: int):
        lib().ora_set_policy(self._h, E, gamma)

    def set_policy_fs(self, E: int, gamma0: int):
        """Baseline FS(E-gamma): fixed exit layer, speculation length moved by +-1 per round."""
        lib().ora_set_policy_fs(self._h, E, gamma0)

    @property
    def T(self) -> int:
        return lib().ora_committed_len(self._h)

    def get_stats(self):
        L = self.cfg.n_layers
        Sc = np.zeros(L, dtype=np.float64)
        Sn, E, g = C.c_double(), C.c_int32(), C.c_int32()
        lib().ora_get_stats(self._h, Sc.ctypes.data, C.byref(Sn), C.byref(E), C.byref(g))
        return Sc, Sn.value, E.value, g.value

    def set_stats(self, Sc, Sn, E, gamma):
        Sc = np.ascontiguousarray(Sc, dtype=np.float64)
        lib().ora_set_stats(self._h, Sc.ctypes.data, float(Sn), int(E), int(gamma))

    def set_exit_mode(self, on: bool):
        """Dynamic draft-exiting (Sec. 4.4): draft up to g_max tokens, stop at the first low-confidence one."""
        lib().ora_set_exit_mode(self._h, 1 if on else 0)

    def set_sampling(self, temperature: float, top_p: float, seed: int):
        """Speculative sampling (Sec. 2) with temperature and nucleus filtering; temperature <= 0: greedy."""
        lib().ora_set_sampling(self._h, float(temperature), float(top_p), int(seed))

    def sample_info(self) -> SampleInfo:
        out = SampleInfo()
        lib().ora_get_sample_info(self._h, C.byref(out))
        return out

    def round_logits(self, which: int, row: int) -> np.ndarray:
        """Logits of the last round: which = 0 the exit head's row of draft `row`, 1 the target's row."""
        p = lib().ora_round_logits(self._h, which, row)
        return np.ctypeslib.as_array(p, shape=(self.cfg.vocab,)).copy()

    def get_conf_stats(self):
        L = self.cfg.n_layers
        Stcs, Sfcs, tau = (np.zeros(L, dtype=np.float64) for _ in range(3))
        lib().ora_get_conf_stats(self._h, Stcs.ctypes.data, Sfcs.ctypes.data, tau.ctypes.data)
        return Stcs, Sfcs, tau

    def set_conf_stats(self, Stcs, Sfcs):
        Stcs = np.ascontiguousarray(Stcs, dtype=np.float64)
        Sfcs = np.ascontiguousarray(Sfcs, dtype=np.float64)
        lib().ora_set_conf_stats(self._h, Stcs.ctypes.data, Sfcs.ctypes.data)

    def get_conf(self, n_cols: int) -> np.ndarray:
        out = np.zeros((self.cfg.n_layers, n_cols), dtype=np.float64)
        lib().ora_get_conf(self._h, out.ctypes.data, n_cols)
        return out

    def hidden(self, layer: int, row: int) -> np.ndarray:
        p = lib().ora_hidden(self._h, layer, row)
        return np.ctypeslib.as_array(p, shape=(self.cfg.d_model,)).copy()

    def k_row(self, layer: int, pos: int) -> np.ndarray:
        p = lib().ora_k_row(self._h, layer, pos)
        return np.ctypeslib.as_array(p, shape=(self.cfg.n_kv_heads * self.cfg.head_dim,)).copy()

    def v_row(self, layer: int, pos: int) -> np.ndarray:
        p = lib().ora_v_row(self._h, layer, pos)
        return np.ctypeslib.as_array(p, shape=(self.cfg.n_kv_heads * self.cfg.head_dim,)).copy()

    # ---- the method
    def prefill(self, prompt: np.ndarray):
        prompt = np.ascontiguousarray(prompt, dtype=np.int32)
        L, W = self.cfg.n_layers, self.cfg.init_window
        shadow = np.full((L, W), -1, dtype=np.int32)
        margin = np.zeros((L, W), dtype=np.float32)
        info = RoundInfo()
        tok = lib().ora_prefill(self._h, prompt.ctypes.data, len(prompt), shadow.ctypes.data, margin.ctypes.data,
                                C.byref(info))
        w = min(W, len(prompt))
        r = Round(info, shadow[:, :w], margin[:, :w], None)
        r.conf = self.get_conf(w)
        return tok, r

    def round(self, remaining: int) -> Round:
        L = self.cfg.n_layers
        shadow = np.full((L, self.stride), -1, dtype=np.int32)
        margin = np.zeros((L, self.stride), dtype=np.float32)
        counts = np.zeros(L, dtype=np.int32)
        info = RoundInfo()
        rc = lib().ora_round(self._h, remaining, C.byref(info), shadow.ctypes.data, margin.ctypes.data,
                             counts.ctypes.data)
        if rc != 0:
            raise RuntimeError(f"ora_round failed: {rc}")
        r = Round(info, shadow[:, :info.g + 1], margin[:, :info.g + 1], counts)
        r.conf = self.get_conf(info.g + 1)
        return r

    def generate(self, prompt: np.ndarray, n_tokens: int):
        """Prefill then rounds until n_tokens tokens exist (the prefill's token included)."""
        tok, init = self.prefill(prompt)
        out: List[int] = [tok]
        rounds: List[Round] = []
        while len(out) < n_tokens:
            r = self.round(n_tokens - len(out))
            rounds.append(r)
            out.extend(r.emitted)
        return out, init, rounds

    # ---- building blocks
    def embed(self, token: int) -> np.ndarray:
        h = np.zeros(self.cfg.d_model, dtype=np.float32)
        lib().ora_embed(self._h, token, h.ctypes.data)
        return h

    def layer_rows(self, layer: int, h_in: np.ndarray, pos0: int) -> np.ndarray:
        h_in = np.ascontiguousarray(h_in, dtype=np.float32).reshape(-1, self.cfg.d_model)
        out = np.zeros_like(h_in)
        lib().ora_layer_rows(self._h, layer, h_in.ctypes.data, pos0, h_in.shape[0], out.ctypes.data)
        return out

    def exit_head(self, h: np.ndarray, want_logits: bool = False):
        h = np.ascontiguousarray(h, dtype=np.float32)
        tok, mg = C.c_int32(), C.c_float()
        lg = np.zeros(self.cfg.vocab, dtype=np.float32) if want_logits else None
        lib().ora_exit_head(self._h, h.ctypes.data, C.byref(tok), C.byref(mg), lg.ctypes.data if want_logits else None)
        return tok.value, mg.value, lg


# thin functional wrappers over the stateless building blocks
def rmsnorm(x: np.ndarray, gain_bf16: np.ndarray, eps: float) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.zeros_like(x)
    lib().ora_rmsnorm(x.ctypes.data, gain_bf16.ctypes.data, x.size, eps, out.ctypes.data)
    return out


def rope(x: np.ndarray, n_heads: int, head_dim: int, pos: int, theta: float) -> np.ndarray:
    y = np.ascontiguousarray(x, dtype=np.float32).copy()
    lib().ora_rope(y.ctypes.data, n_heads, head_dim, pos, theta)
    return y


def softmax(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    p = np.zeros(x.size, dtype=np.float64)
    lib().ora_softmax(x.ctypes.data, x.size, p.ctypes.data)
    return p


def confidence(logits: np.ndarray) -> float:
    x = np.ascontiguousarray(logits, dtype=np.float32)
    return lib().ora_confidence(x.ctypes.data, x.size)


def uniform(seed: int, pos: int, purpose: int) -> float:
    return lib().ora_uniform(int(seed), int(pos), int(purpose))


def nucleus(logits: np.ndarray, temperature: float, top_p: float) -> np.ndarray:
    x = np.ascontiguousarray(logits, dtype=np.float32)
    p = np.zeros(x.size, dtype=np.float64)
    lib().ora_nucleus(x.ctypes.data, x.size, float(temperature), float(top_p), p.ctypes.data)
    return p


def sample_cdf(probs: np.ndarray, u: float) -> int:
    p = np.ascontiguousarray(probs, dtype=np.float64)
    return lib().ora_sample_cdf(p.ctypes.data, p.size, float(u))


def residual(p: np.ndarray, q: np.ndarray):
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    r = np.zeros_like(p)
    R = lib().ora_residual(p.ctypes.data, q.ctypes.data, p.size, r.ctypes.data)
    return r, R


def threshold(Stcs: float, Sc: float, Sfcs: float, Smis: float) -> float:
    return lib().ora_threshold(Stcs, Sc, Sfcs, Smis)


def fs_next_gamma(gamma: int, g: int, n: int, g_min: int, g_max: int) -> int:
    return lib().ora_fs_next_gamma(gamma, g, n, g_min, g_max)


def silu(x: float) -> float:
    return lib().ora_silu(x)


def accept_len(drafts, verified) -> int:
    d = np.ascontiguousarray(drafts, dtype=np.int32)
    v = np.ascontiguousarray(verified, dtype=np.int32)
    return lib().ora_accept_len(d.ctypes.data, v.ctypes.data, len(d))


def decay_step(S: float, omega: float, a: float) -> float:
    return lib().ora_decay_step(S, omega, a)


def tpl(alpha: float, l: int, d: int, L: int) -> float:
    return lib().ora_tpl(alpha, l, d, L)


def select(Sc, Sn: float, L: int, e_min: int, e_max: int, g_min: int, g_max: int):
    Sc = np.ascontiguousarray(Sc, dtype=np.float64)
    E, g = C.c_int32(), C.c_int32()
    lib().ora_select(Sc.ctypes.data, Sn, L, e_min, e_max, g_min, g_max, C.byref(E), C.byref(g))
    return E.value, g.value


def num_threads() -> int:
    return lib().ora_num_threads()
