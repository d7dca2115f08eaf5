"""Writes the oracle's decode traces used as expected values by the GPU parity tests.

Calls only ``synth`` (seeded inputs) and ``oracle`` (the CPU oracle); nothing from the CUDA path.

    python tests/golden/make_traces.py tiny
    python tests/golden/make_traces.py llama2_7b [--gen-len N] [--seqs K]
    python tests/golden/make_traces.py llama2_7b --exit-mode --gen-len 128     (-> trace_llama2_7b_exit.json)
    python tests/golden/make_traces.py llama3_8b_b4 --resume-dir DIR   (hours of CPU: every finished sequence is
                                                                        kept in DIR and reused by a restarted run)

Output: tests/golden/trace_<config>.json.  Per sequence: the prompt recipe's identifiers, the token
emitted by the prefill, the initial window's shadow tokens / margins / statistics, and for every round
E, gamma, g (drafts made), the drafts, every layer's shadow tokens with the top-1 minus top-2 logit
margin (in 1/1000, capped at 9999), the accepted count, per-layer match counts and the next (E, gamma).
With --exit-mode (dynamic draft-exiting) also: every shadow token's confidence (in 1e-7), the drafted
tokens' confidences and the thresholds as full doubles, the stop flag and the decayed confidence sums.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import synth  # noqa: E402


def _q(m: np.ndarray):
    return np.minimum(np.floor(m.astype(np.float64) * 1000.0), 9999).astype(int).tolist()


def _c(conf: np.ndarray):
    return np.rint(conf * 1e7).astype(np.int64).tolist()


def trace_sequence(cfg, weights, seq: int, gen_len: int, exit_mode: bool = False):
    o = oracle.OracleSeq(cfg, weights)
    o.set_exit_mode(exit_mode)
    prompt = synth.make_prompt(cfg, seq)
    t0 = time.time()
    tok, init = o.prefill(prompt)
    t_prefill = time.time() - t0
    Sc, Sn, E, g = o.get_stats()
    rec = {
        "seq": seq, "first_token": int(tok),
        "init": {"shadow": init.shadow.tolist(), "margin_milli": _q(init.margin), "Sc": Sc.tolist(), "Sn": Sn,
                 "E": E, "gamma": g},
        "rounds": [],
    }
    if exit_mode:
        Stcs, Sfcs, _ = o.get_conf_stats()
        rec["init"].update({"conf_e7": _c(init.conf), "Stcs": Stcs.tolist(), "Sfcs": Sfcs.tolist(), "tau": init.next_tau})
    out = [int(tok)]
    t0 = time.time()
    while len(out) < gen_len:
        r = o.round(gen_len - len(out))
        Sc, Sn, _, _ = o.get_stats()
        rec["rounds"].append({
            "E": r.E, "gamma": r.gamma, "g": r.g, "n": r.n_accept, "drafts": r.drafts, "emitted": r.emitted,
            "shadow": r.shadow.tolist(), "margin_milli": _q(r.margin), "counts": r.counts.tolist(),
            "next_E": r.next_E, "next_gamma": r.next_gamma, "Sc": Sc.tolist(), "Sn": Sn,
        })
        if exit_mode:
            Stcs, Sfcs, _ = o.get_conf_stats()
            rec["rounds"][-1].update({"conf_e7": _c(r.conf), "draft_conf": r.draft_conf, "stopped": int(r.stopped),
                                      "tau": r.tau, "next_tau": r.next_tau, "Stcs": Stcs.tolist(), "Sfcs": Sfcs.tolist()})
        out.extend(r.emitted)
        print(f"  seq {seq} round {len(rec['rounds'])}: E={r.E} g={r.g} n={r.n_accept} -> {len(out)}/{gen_len} "
              f"({time.time() - t0:.1f}s)", flush=True)
    rec["tokens"] = out
    rec["oracle_seconds"] = {"prefill": t_prefill, "rounds": time.time() - t0}
    o.close()
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("config")
    ap.add_argument("--gen-len", type=int, default=None)
    ap.add_argument("--seqs", type=int, default=None)
    ap.add_argument("--out", default=None)
    ap.add_argument("--exit-mode", action="store_true")
    ap.add_argument("--resume-dir", default=None)
    a = ap.parse_args()
    cfg = synth.CONFIGS[a.config]
    gen_len = a.gen_len or cfg.gen_len
    n_seq = a.seqs or cfg.batch
    t0 = time.time()
    weights = synth.make_weights(cfg)
    print(f"weights: {weights.nbytes() / 1e9:.2f} GB in {time.time() - t0:.1f}s; threads {oracle.num_threads()}",
          flush=True)
    def one(s):
        if not a.resume_dir:
            return trace_sequence(cfg, weights, s, gen_len, a.exit_mode)
        os.makedirs(a.resume_dir, exist_ok=True)
        part = os.path.join(a.resume_dir, f"{cfg.name}{'_exit' if a.exit_mode else ''}_g{gen_len}_seq{s}.json")
        if os.path.exists(part):
            with open(part) as f:
                return json.load(f)
        rec = trace_sequence(cfg, weights, s, gen_len, a.exit_mode)
        with open(part + ".tmp", "w") as f:
            json.dump(rec, f, separators=(",", ":"))
        os.replace(part + ".tmp", part)
        return rec

    doc = {"config": cfg.name, "seed": cfg.seed, "prompt_len": cfg.prompt_len, "gen_len": gen_len,
           "e_range": [cfg.e_min, cfg.e_max], "g_range": [cfg.g_min, cfg.g_max], "omega": cfg.omega,
           "oracle_threads": oracle.num_threads(),
           "exit_mode": bool(a.exit_mode),
           "sequences": [one(s) for s in range(n_seq)]}
    out = a.out or os.path.join(os.path.dirname(os.path.abspath(__file__)),
                                f"trace_{cfg.name}{'_exit' if a.exit_mode else ''}.json")
    with open(out, "w") as f:
        json.dump(doc, f, separators=(",", ":"))
    print("wrote", out, os.path.getsize(out), "bytes")


if __name__ == "__main__":
    main()
