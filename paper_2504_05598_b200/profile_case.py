"""Small driver for profiling and kernel tuning: a model with the layer shape of a named configuration
but few layers (so that it fits the size limits of a profiler capture), a short prompt, a few rounds.

    python -m paper_2504_05598_b200.profile_case --config llama2_7b --layers 4 --rounds 8 [--policy E,G] [--sampling T,top_p]

Prints per-kernel-class device times (CUDA events around every launch) as JSON.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import torch

    import paper_2504_05598_b200 as dl
    import synth
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="llama2_7b")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--rounds", type=int, default=8)
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--policy", default="")          # "E,G" fixes the setting; default dynamic
    ap.add_argument("--no-timing", action="store_true")
    ap.add_argument("--no-pdl", action="store_true")
    ap.add_argument("--one-cta", action="store_true")
    ap.add_argument("--no-tc", action="store_true")
    ap.add_argument("--trim", action="store_true")   # stacked LM head over the candidate layers only
    ap.add_argument("--sampling", default="")        # "T,top_p": speculative sampling instead of greedy verification
    a = ap.parse_args()
    base = synth.CONFIGS[a.config]
    L = a.layers
    cfg = synth.small_variant(base, n_layers=L, e_min=min(base.e_min, L - 1), e_max=min(base.e_max, L - 1),
                              prompt_len=a.prompt, gen_len=a.rounds * (base.g_max + 1) + 8)
    w = synth.make_weights(cfg)
    ctx = dl.DelContext(dl.make_shape(cfg), dl.upload_weights(w))
    for s in range(cfg.batch):
        if a.sampling:
            T, top_p = (float(v) for v in a.sampling.split(","))
            ctx.set_sampling(s, T, top_p, 1234 + s)
        ctx.prefill(s, synth.make_prompt(cfg, s), cfg.gen_len)
        if a.policy:
            E, G = (int(v) for v in a.policy.split(","))
            ctx.set_policy(s, E, G)
    flags = (0 if a.no_pdl else dl.FLAG_PDL) | (16 if a.one_cta else 0) | (0 if a.no_tc else dl.FLAG_TC) | \
        (dl.FLAG_TRIM_ROWS if a.trim else 0)
    ctx.set_flags(flags)
    ctx.round()
    ctx.round()
    if not a.no_timing:
        ctx.set_flags(flags | dl.FLAG_TIMING)
    ctx.kernel_times(reset=True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(ctx.stream)
    hist = []
    for _ in range(a.rounds):
        o = ctx.round()[0]
        hist.append((o.E, o.g, o.n_accept))
    ev1.record(ctx.stream)
    torch.cuda.synchronize()
    kt = ctx.kernel_times(reset=True)
    rep = {"ms_per_round": ev0.elapsed_time(ev1) / a.rounds, "rounds": hist, "kernels": {}}
    for k, v in kt.items():
        if v["launches"]:
            rep["kernels"][k] = {"launches": v["launches"], "avg_us": round(1000 * v["ms"] / v["launches"], 2),
                                 "gbs": round(v["bytes"] / 1e9 / (v["ms"] / 1e3), 1) if v["bytes"] else None}
    print(json.dumps(rep))
    ctx.close()


if __name__ == "__main__":
    main()
