"""Python binding of libdel: the greedy self-speculative decode round with dynamic exit-layer
selection (DEL) as hand-written sm_100a CUDA kernels behind a C ABI (see include/del.h).

This module only marshals arguments: torch provides device memory and the CUDA stream, every step of
the method runs inside the library's kernels.  There is no CPU fallback: importing works anywhere
(so that the exported symbols can be checked), creating a context needs the built library and a GPU.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdel.so")
MAX_GAMMA = 31
MAX_ROWS = 64

OK, EINVAL, ENOSPC, ESTATE, ETIMEOUT, ECUDA = 0, -1, -2, -3, -4, -5
FLAG_PDL, FLAG_GRAPH, FLAG_TC, FLAG_TIMING, FLAG_ONECTA, FLAG_NO_BULK_PREFILL, FLAG_DECODE_ATTN_PREFILL, FLAG_TRIM_ROWS = 1, 2, 4, 8, 16, 32, 64, 128
FLAG_MMA_SYNC_PREFILL_ATTN, FLAG_NO_WEIGHT_PREFETCH = 256, 512
KERNEL_CLASSES = ["qkv_rope", "attention", "o_proj", "gate_up", "down", "lm_head_draft", "lm_head_stacked", "other"]

EXPORTS = ["del_workspace_bytes", "del_init", "del_prefill", "del_draft", "del_verify", "del_layer_accept",
           "del_select", "del_round", "del_set_policy", "del_get_stats", "del_set_stats", "del_get_shadow",
           "del_get_drafts", "del_force_token", "del_get_hidden", "del_debug_logits", "del_get_kv", "del_committed_len", "del_release",
           "del_launch_count", "del_get_traffic", "del_set_flags", "del_get_kernel_times", "del_head_argmax_static",
           "del_set_policy_fs", "del_set_exit_mode", "del_get_window", "del_set_sampling", "del_get_sample_info", "del_get_round_logits", "del_sample_probe", "del_get_conf_stats", "del_set_conf_stats", "del_get_conf", "del_debug_inject_error", "del_strerror", "del_last_cuda_error", "del_destroy"]


class Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_batch", "max_seq", "page_size", "n_pages", "e_min", "e_max", "g_min",
                                         "g_max", "init_window")] + \
               [("omega", C.c_double)]


class WeightsC(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up",
                                                     "w_down")] + \
               [("rope_cos", C.c_void_p), ("rope_sin", C.c_void_p)]


class KvC(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("page_table", C.c_void_p)]


class RoundOut(C.Structure):
    _fields_ = [("E", C.c_int32), ("gamma", C.c_int32), ("g", C.c_int32), ("n_accept", C.c_int32),
                ("n_emitted", C.c_int32), ("tokens", C.c_int32 * (MAX_GAMMA + 1)), ("next_E", C.c_int32),
                ("next_gamma", C.c_int32), ("status", C.c_int32), ("stopped", C.c_int32),
                ("tau", C.c_double), ("next_tau", C.c_double)]

    def emitted(self) -> List[int]:
        return [int(self.tokens[i]) for i in range(self.n_emitted)]


_lib = None


def load_library(build_if_missing: bool = True):
    """dlopen libdel.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        _build.build()
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2504_05598_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, i32, ci = C.c_void_p, C.c_int32, C.c_int
    L.del_workspace_bytes.restype = C.c_size_t
    L.del_workspace_bytes.argtypes = [C.POINTER(Shape)]
    L.del_init.restype = ci
    L.del_init.argtypes = [C.POINTER(vp), C.POINTER(Shape), C.POINTER(WeightsC), C.POINTER(KvC), vp, C.c_size_t, vp]
    L.del_prefill.restype = ci
    L.del_prefill.argtypes = [vp, ci, vp, ci, ci, C.POINTER(RoundOut)]
    L.del_draft.restype = ci
    L.del_draft.argtypes = [vp, ci, ci, ci]
    L.del_verify.restype = ci
    L.del_verify.argtypes = [vp, ci]
    L.del_layer_accept.restype = ci
    L.del_layer_accept.argtypes = [vp, ci, C.POINTER(RoundOut)]
    L.del_select.restype = ci
    L.del_select.argtypes = [vp, ci, C.POINTER(i32), C.POINTER(i32)]
    L.del_round.restype = ci
    L.del_round.argtypes = [vp, C.POINTER(RoundOut)]
    L.del_set_policy.restype = ci
    L.del_set_policy.argtypes = [vp, ci, ci, ci]
    L.del_get_stats.restype = ci
    L.del_get_stats.argtypes = [vp, ci, vp, C.POINTER(C.c_double), C.POINTER(i32), C.POINTER(i32)]
    L.del_set_stats.restype = ci
    L.del_set_stats.argtypes = [vp, ci, vp, C.c_double, i32, i32]
    L.del_set_policy_fs.restype = ci
    L.del_set_policy_fs.argtypes = [vp, ci, ci, ci]
    L.del_set_exit_mode.restype = ci
    L.del_set_exit_mode.argtypes = [vp, ci, ci]
    L.del_get_window.restype = ci
    L.del_get_window.argtypes = [vp, ci, ci, vp, vp]
    L.del_set_sampling.restype = ci
    L.del_set_sampling.argtypes = [vp, ci, C.c_double, C.c_double, C.c_uint64]
    L.del_get_sample_info.restype = ci
    L.del_get_sample_info.argtypes = [vp, ci, vp, vp, vp, vp]
    L.del_get_round_logits.restype = ci
    L.del_get_round_logits.argtypes = [vp, ci, ci, ci, vp]
    L.del_sample_probe.restype = ci
    L.del_sample_probe.argtypes = [vp, vp, vp, ci, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, vp, vp, vp]
    L.del_get_conf_stats.restype = ci
    L.del_get_conf_stats.argtypes = [vp, ci, vp, vp, vp]
    L.del_set_conf_stats.restype = ci
    L.del_set_conf_stats.argtypes = [vp, ci, vp, vp]
    L.del_get_conf.restype = ci
    L.del_get_conf.argtypes = [vp, ci, vp, vp]
    L.del_get_shadow.restype = ci
    L.del_get_shadow.argtypes = [vp, ci, vp, vp]
    L.del_get_drafts.restype = ci
    L.del_get_drafts.argtypes = [vp, ci, vp]
    L.del_force_token.restype = ci
    L.del_force_token.argtypes = [vp, ci, i32]
    L.del_get_hidden.restype = ci
    L.del_get_hidden.argtypes = [vp, ci, ci, ci, vp]
    L.del_debug_logits.restype = ci
    L.del_debug_logits.argtypes = [vp, ci, ci, ci, vp]
    L.del_get_kv.restype = ci
    L.del_get_kv.argtypes = [vp, ci, ci, ci, vp, vp]
    L.del_debug_inject_error.restype = ci
    L.del_debug_inject_error.argtypes = [vp, ci]
    L.del_committed_len.restype = ci
    L.del_committed_len.argtypes = [vp, ci]
    L.del_release.restype = ci
    L.del_release.argtypes = [vp, ci]
    L.del_launch_count.restype = C.c_int64
    L.del_launch_count.argtypes = [vp]
    L.del_get_traffic.restype = ci
    L.del_get_traffic.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.del_set_flags.restype = ci
    L.del_set_flags.argtypes = [vp, ci]
    L.del_get_kernel_times.restype = ci
    L.del_get_kernel_times.argtypes = [vp, vp, vp, vp, ci]
    L.del_head_argmax_static.restype = ci
    L.del_head_argmax_static.argtypes = [vp, vp, ci, ci, ci, vp, vp]
    L.del_strerror.restype = C.c_char_p
    L.del_strerror.argtypes = [ci]
    L.del_last_cuda_error.restype = C.c_char_p
    L.del_last_cuda_error.argtypes = [vp]
    L.del_destroy.argtypes = [vp]
    _lib = L
    return L


class DelError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        super().__init__(f"{what}: {load_library().del_strerror(code).decode()} ({code}) {detail}")
        self.code = code


def rope_tables(max_seq: int, head_dim: int, theta: float):
    """cos / sin of pos * theta^(-2j/head_dim), fp32 [max_seq, head_dim/2] (computed in float64)."""
    j = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = np.power(float(theta), -2.0 * j / head_dim)
    ang = np.arange(max_seq, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def make_shape(cfg, max_batch: Optional[int] = None, max_seq: Optional[int] = None, n_pages: Optional[int] = None) -> Shape:
    """Shape struct from an object with the attributes of synth.Config."""
    B = max_batch or cfg.batch
    ms = max_seq or cfg.max_seq
    ms = (ms + 15) // 16 * 16
    return Shape(cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab,
                 cfg.rms_eps, cfg.rope_theta, B, ms, 16, n_pages or B * (ms // 16), cfg.e_min, cfg.e_max, cfg.g_min,
                 cfg.g_max, cfg.init_window, cfg.omega)


class DelContext:
    """A libdel context plus the torch tensors that back it.

    ``weights``: dict with bf16 CUDA tensors ``tok_emb``, ``final_norm``, ``lm_head`` and a list ``layers`` of
    dicts with ``attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down`` (matrices [out, in]).
    """

    def __init__(self, shape: Shape, weights: Dict, device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("libdel needs a CUDA device; there is no CPU fallback")
        self.lib = load_library()
        self.torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.weights = weights
        L = shape.n_layers
        with torch.cuda.device(self.device):
            self.stream = stream or torch.cuda.Stream(device=self.device)
            cos, sin = rope_tables(shape.max_seq, shape.head_dim, shape.rope_theta)
            self.rope_cos = torch.from_numpy(cos).to(self.device)
            self.rope_sin = torch.from_numpy(sin).to(self.device)
            page_elems = L * shape.n_kv_heads * 16 * shape.head_dim
            # zeros: page slots that are not written yet take part in the products with probability 0
            self.k_pages = torch.zeros(shape.n_pages * page_elems, dtype=torch.bfloat16, device=self.device)
            self.v_pages = torch.zeros(shape.n_pages * page_elems, dtype=torch.bfloat16, device=self.device)
            self.page_table = torch.zeros(shape.max_batch * (shape.max_seq // 16), dtype=torch.int32, device=self.device)
            ws = self.lib.del_workspace_bytes(C.byref(shape))
            if ws == 0:
                raise DelError(EINVAL, "del_workspace_bytes")
            self.workspace = torch.empty(ws + 256, dtype=torch.uint8, device=self.device)
            ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
            wc = WeightsC()
            wc.tok_emb, wc.final_norm, wc.lm_head = (weights[k].data_ptr() for k in ("tok_emb", "final_norm", "lm_head"))
            self._arrays = []
            for name in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down"):
                arr = (C.c_void_p * L)(*[weights["layers"][l][name].data_ptr() for l in range(L)])
                self._arrays.append(arr)
                setattr(wc, name, C.cast(arr, C.POINTER(C.c_void_p)))
            wc.rope_cos, wc.rope_sin = self.rope_cos.data_ptr(), self.rope_sin.data_ptr()
            kv = KvC(self.k_pages.data_ptr(), self.v_pages.data_ptr(), self.page_table.data_ptr())
            torch.cuda.synchronize(self.device)
            h = C.c_void_p()
            rc = self.lib.del_init(C.byref(h), C.byref(shape), C.byref(wc), C.byref(kv), ws_ptr, ws,
                                   C.c_void_p(self.stream.cuda_stream))
            if rc != OK:
                raise DelError(rc, "del_init")
            self._h = h
        self.workspace_bytes = ws

    # ---- plumbing
    def _ck(self, rc: int, what: str):
        if rc != OK:
            raise DelError(rc, what, self.lib.del_last_cuda_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self.lib.del_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the calls of include/del.h, same names
    def prefill(self, seq: int, prompt: Sequence[int], max_new_tokens: int) -> RoundOut:
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        out = RoundOut()
        self._ck(self.lib.del_prefill(self._h, seq, p.ctypes.data, len(p), max_new_tokens, C.byref(out)), "del_prefill")
        return out

    def draft(self, seq: int, E: int, gamma: int):
        self._ck(self.lib.del_draft(self._h, seq, E, gamma), "del_draft")

    def verify(self, seq: int):
        self._ck(self.lib.del_verify(self._h, seq), "del_verify")

    def layer_accept(self, seq: int) -> RoundOut:
        out = RoundOut()
        self._ck(self.lib.del_layer_accept(self._h, seq, C.byref(out)), "del_layer_accept")
        return out

    def select(self, seq: int):
        E, g = C.c_int32(), C.c_int32()
        self._ck(self.lib.del_select(self._h, seq, C.byref(E), C.byref(g)), "del_select")
        return E.value, g.value

    def round(self) -> List[RoundOut]:
        outs = (RoundOut * self.shape.max_batch)()
        self._ck(self.lib.del_round(self._h, outs), "del_round")
        return list(outs)

    def try_round(self):
        outs = (RoundOut * self.shape.max_batch)()
        return self.lib.del_round(self._h, outs), list(outs)

    def set_policy(self, seq: int, E: int, gamma: int):
        self._ck(self.lib.del_set_policy(self._h, seq, E, gamma), "del_set_policy")

    def get_stats(self, seq: int):
        Sc = np.zeros(self.shape.n_layers, dtype=np.float64)
        Sn, E, g = C.c_double(), C.c_int32(), C.c_int32()
        self._ck(self.lib.del_get_stats(self._h, seq, Sc.ctypes.data, C.byref(Sn), C.byref(E), C.byref(g)), "del_get_stats")
        return Sc, Sn.value, E.value, g.value

    def set_stats(self, seq: int, Sc, Sn: float, E: int, gamma: int):
        Sc = np.ascontiguousarray(Sc, dtype=np.float64)
        self._ck(self.lib.del_set_stats(self._h, seq, Sc.ctypes.data, float(Sn), int(E), int(gamma)), "del_set_stats")

    def set_policy_fs(self, seq: int, E: int, gamma0: int):
        """Baseline FS(E-gamma): fixed exit layer, speculation length moved by +-1 per round."""
        self._ck(self.lib.del_set_policy_fs(self._h, seq, E, gamma0), "del_set_policy_fs")

    def set_exit_mode(self, seq: int, on: bool):
        """Dynamic draft-exiting: the draft loop stops at the first token whose confidence is below the threshold."""
        self._ck(self.lib.del_set_exit_mode(self._h, seq, 1 if on else 0), "del_set_exit_mode")

    def set_sampling(self, seq: int, temperature: float, top_p: float = 1.0, seed: int = 0):
        """Speculative sampling with temperature and nucleus filtering for this slot; temperature <= 0: greedy."""
        self._ck(self.lib.del_set_sampling(self._h, seq, float(temperature), float(top_p), int(seed)), "del_set_sampling")

    def get_sample_info(self, seq: int):
        """(acceptance tests made, last token from the residual?, q(x) per draft, p(x) per tested draft)."""
        n, r = C.c_int32(), C.c_int32()
        qx, px = np.zeros(32, dtype=np.float32), np.zeros(32, dtype=np.float32)
        self._ck(self.lib.del_get_sample_info(self._h, seq, C.byref(n), C.byref(r), qx.ctypes.data, px.ctypes.data),
                 "del_get_sample_info")
        return n.value, bool(r.value), qx, px

    def get_round_logits(self, seq: int, which: int, row: int) -> np.ndarray:
        out = np.zeros(self.shape.vocab, dtype=np.float32)
        self._ck(self.lib.del_get_round_logits(self._h, seq, which, row, out.ctypes.data), "del_get_round_logits")
        return out

    def sample_probe(self, p_logits, q_logits, temperature, top_p, u_draft, u_accept, u_final):
        """Test hook: the sampling kernels on one pair of logit rows."""
        p = np.ascontiguousarray(p_logits, dtype=np.float32)
        q = np.ascontiguousarray(q_logits, dtype=np.float32)
        out, prob, stat = np.zeros(4, dtype=np.int32), np.zeros(2, dtype=np.float64), np.zeros(8, dtype=np.int32)
        self._ck(self.lib.del_sample_probe(self._h, p.ctypes.data, q.ctypes.data, p.size, float(temperature), float(top_p),
                                           float(u_draft), float(u_accept), float(u_final), out.ctypes.data,
                                           prob.ctypes.data, stat.ctypes.data), "del_sample_probe")
        return out, prob, stat

    def get_conf_stats(self, seq: int):
        L = self.shape.n_layers
        Stcs, Sfcs, tau = (np.zeros(L, dtype=np.float64) for _ in range(3))
        self._ck(self.lib.del_get_conf_stats(self._h, seq, Stcs.ctypes.data, Sfcs.ctypes.data, tau.ctypes.data),
                 "del_get_conf_stats")
        return Stcs, Sfcs, tau

    def set_conf_stats(self, seq: int, Stcs, Sfcs):
        Stcs = np.ascontiguousarray(Stcs, dtype=np.float64)
        Sfcs = np.ascontiguousarray(Sfcs, dtype=np.float64)
        self._ck(self.lib.del_set_conf_stats(self._h, seq, Stcs.ctypes.data, Sfcs.ctypes.data), "del_set_conf_stats")

    def get_conf(self, seq: int):
        """(shadow confidences [n_layers][g_max + 1], draft confidences [g_max + 1]) of the last round."""
        L, G = self.shape.n_layers, self.shape.g_max + 1
        sc = np.zeros((L, G), dtype=np.float32)
        dc = np.zeros(G, dtype=np.float32)
        self._ck(self.lib.del_get_conf(self._h, seq, sc.ctypes.data, dc.ctypes.data), "del_get_conf")
        return sc, dc

    def get_window(self, seq: int, n_cols: int):
        """(shadow tokens, confidences) of the first n_cols slots of every layer: the prefill's whole window."""
        L = self.shape.n_layers
        sh = np.zeros((L, n_cols), dtype=np.int32)
        cf = np.zeros((L, n_cols), dtype=np.float32)
        self._ck(self.lib.del_get_window(self._h, seq, n_cols, sh.ctypes.data, cf.ctypes.data), "del_get_window")
        return sh, cf

    def get_shadow(self, seq: int):
        L, G = self.shape.n_layers, self.shape.g_max + 1
        sh = np.zeros((L, G), dtype=np.int32)
        cn = np.zeros(L, dtype=np.int32)
        self._ck(self.lib.del_get_shadow(self._h, seq, sh.ctypes.data, cn.ctypes.data), "del_get_shadow")
        return sh, cn

    def get_drafts(self, seq: int) -> np.ndarray:
        d = np.zeros(max(1, self.shape.g_max), dtype=np.int32)
        self._ck(self.lib.del_get_drafts(self._h, seq, d.ctypes.data), "del_get_drafts")
        return d

    def force_token(self, seq: int, token: int):
        self._ck(self.lib.del_force_token(self._h, seq, int(token)), "del_force_token")

    def get_hidden(self, seq: int, layer: int, row: int) -> np.ndarray:
        out = np.zeros(self.shape.d_model, dtype=np.float32)
        self._ck(self.lib.del_get_hidden(self._h, seq, layer, row, out.ctypes.data), "del_get_hidden")
        return out

    def debug_logits(self, seq: int, layer: int, row: int) -> np.ndarray:
        out = np.zeros(self.shape.vocab, dtype=np.float32)
        self._ck(self.lib.del_debug_logits(self._h, seq, layer, row, out.ctypes.data), "del_debug_logits")
        return out

    def get_kv(self, seq: int, layer: int, pos: int):
        n = self.shape.n_kv_heads * self.shape.head_dim
        k, v = np.zeros(n, dtype=np.float32), np.zeros(n, dtype=np.float32)
        self._ck(self.lib.del_get_kv(self._h, seq, layer, pos, k.ctypes.data, v.ctypes.data), "del_get_kv")
        return k, v

    def debug_inject_error(self, code: int):
        self._ck(self.lib.del_debug_inject_error(self._h, int(code)), "del_debug_inject_error")

    def committed_len(self, seq: int) -> int:
        return self.lib.del_committed_len(self._h, seq)

    def release(self, seq: int):
        self._ck(self.lib.del_release(self._h, seq), "del_release")

    def launch_count(self) -> int:
        return int(self.lib.del_launch_count(self._h))

    def traffic(self):
        a, b = C.c_int64(), C.c_int64()
        self._ck(self.lib.del_get_traffic(self._h, C.byref(a), C.byref(b)), "del_get_traffic")
        return a.value, b.value

    def kernel_times(self, reset: bool = True):
        ms = np.zeros(8, dtype=np.float64)
        n = np.zeros(8, dtype=np.int64)
        by = np.zeros(8, dtype=np.float64)
        self._ck(self.lib.del_get_kernel_times(self._h, ms.ctypes.data, n.ctypes.data, by.ctypes.data, int(reset)),
                 "del_get_kernel_times")
        return {k: {"ms": float(ms[i]), "launches": int(n[i]), "bytes": float(by[i])} for i, k in enumerate(KERNEL_CLASSES)}

    def set_flags(self, flags: int) -> int:
        return self.lib.del_set_flags(self._h, flags)


def upload_weights(w, device="cuda:0") -> Dict:
    """numpy uint16 (bf16 bit patterns) weight set -> dict of bf16 CUDA tensors (plain copies)."""
    import torch

    def up(a: np.ndarray):
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)

    return {"tok_emb": up(w.tok_emb), "final_norm": up(w.final_norm), "lm_head": up(w.lm_head),
            "layers": [{k: up(v) for k, v in lw.items()} for lw in w.layers]}


def head_argmax_static(x, lm_head, tokens_out, stream=None) -> int:
    """del_head_argmax_static on torch CUDA tensors: x bf16 [rows, d], lm_head bf16 [vocab, d],
    tokens_out int32 [rows].  Allocates nothing (the kernel's scratch is a fixed array in the library);
    returns the library's status code."""
    import torch
    st = stream or torch.cuda.current_stream(x.device)
    return load_library().del_head_argmax_static(x.data_ptr(), lm_head.data_ptr(), x.shape[0], lm_head.shape[0], x.shape[1],
                                                 tokens_out.data_ptr(), C.c_void_p(st.cuda_stream))
