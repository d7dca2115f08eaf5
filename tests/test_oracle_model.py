"""Pins for the oracle's decoder and for the whole round: an independent non-cached numpy forward,
greedy speculative == greedy auto-regressive, brute-force shadow tokens and counts.  CPU only."""
import numpy as np
import pytest

import oracle
import synth
from cases import TINY, TINY_GQA, TINY_SHORT
from np_model import exit_logits, forward_all, kv_rows, rmsnorm

CASES = [TINY, TINY_GQA, TINY_SHORT]


@pytest.fixture(scope="module", params=CASES, ids=lambda c: c.name)
def case(request):
    cfg = request.param
    return cfg, synth.make_weights(cfg), synth.make_prompt(cfg)


def test_cached_forward_equals_full_recompute(case):
    cfg, w, prompt = case
    o = oracle.OracleSeq(cfg, w)
    tok, init = o.prefill(prompt)
    ref = forward_all(cfg, w, prompt)
    W = min(cfg.init_window, len(prompt))
    for l in range(cfg.n_layers + 1):
        for j in (0, W // 2, W - 1):
            got = o.hidden(l, j).astype(np.float64)
            want = ref[l][len(prompt) - W + j]
            assert np.allclose(got, want, rtol=2e-5, atol=2e-5 * np.abs(want).max()), (l, j)
    # keys/values in the cache, first and last position of layer 1 and L: K is rotated, V is not
    for l in (1, cfg.n_layers):
        k_ref, v_ref = kv_rows(cfg, w, ref[l - 1], l)
        for pos in (0, len(prompt) - 1):
            assert np.allclose(o.k_row(l, pos), k_ref[pos], rtol=2e-5, atol=2e-5 * np.abs(k_ref).max()), (l, pos)
            assert np.allclose(o.v_row(l, pos), v_ref[pos], rtol=2e-5, atol=2e-5 * np.abs(v_ref).max()), (l, pos)
        # the rotation is real: at the last position the cached key differs from the unrotated projection
        a = rmsnorm(ref[l - 1][-1], synth.bf16_to_f32(w.layers[l - 1]["attn_norm"]).astype(np.float64), cfg.rms_eps)
        k_plain = a @ synth.bf16_to_f32(w.layers[l - 1]["wk"]).astype(np.float64).T
        assert np.abs(o.k_row(l, len(prompt) - 1) - k_plain).max() > 1e-2 * np.abs(k_plain).max()
    lg = exit_logits(cfg, w, ref[-1][-1])
    assert int(np.argmax(lg)) == tok
    _, mg, logits = o.exit_head(o.hidden(cfg.n_layers, W - 1), want_logits=True)
    assert np.allclose(logits, lg, atol=1e-4)
    top2 = np.sort(lg)[-2:]
    assert abs(mg - (top2[1] - top2[0])) < 1e-4


def test_rows_together_equal_rows_one_by_one(case):
    cfg, w, prompt = case
    a, b = oracle.OracleSeq(cfg, w), oracle.OracleSeq(cfg, w)
    h0 = np.stack([a.embed(int(t)) for t in prompt[:9]])
    ya = a.layer_rows(1, h0, 0)
    yb = np.concatenate([b.layer_rows(1, h0[i:i + 1], i) for i in range(9)])
    assert np.array_equal(ya, yb)                       # bit-exact: same reduction order for any m
    for pos in (0, 8):
        assert np.array_equal(a.k_row(1, pos), b.k_row(1, pos)) and np.array_equal(a.v_row(1, pos), b.v_row(1, pos))


def test_gqa_with_duplicated_kv_heads_equals_mha():
    gqa = TINY_GQA                                   # 4 query heads, 2 kv heads
    wg = synth.make_weights(gqa)
    mha = synth.small_variant(gqa, n_kv_heads=gqa.n_heads)
    wm = synth.make_weights(gqa)
    hd, rep = gqa.head_dim, gqa.n_heads // gqa.n_kv_heads
    for lw in wm.layers:                               # duplicate each kv head `rep` times
        for name in ("wk", "wv"):
            m = lw[name].reshape(gqa.n_kv_heads, hd, gqa.d_model)
            lw[name] = np.ascontiguousarray(np.repeat(m, rep, axis=0).reshape(-1, gqa.d_model))
    prompt = synth.make_prompt(gqa)[:12]
    a, b = oracle.OracleSeq(gqa, wg), oracle.OracleSeq(mha, wm)
    ta, _ = a.prefill(prompt)
    tb, _ = b.prefill(prompt)
    assert ta == tb
    W = len(prompt)
    assert np.array_equal(a.hidden(gqa.n_layers, W - 1), b.hidden(gqa.n_layers, W - 1))


def run(cfg, w, prompt, policy=None, n=None):
    o = oracle.OracleSeq(cfg, w)
    if policy:
        o.set_policy(*policy)
    out, init, rounds = o.generate(prompt, n or cfg.gen_len)
    return o, out, init, rounds


def test_speculative_stream_equals_autoregressive_stream(case):
    """Greedy verification keeps exactly the target model's greedy tokens, for every (E, gamma)."""
    cfg, w, prompt = case
    _, vanilla, _, vr = run(cfg, w, prompt, policy=(1, 0))
    assert len(vanilla) == cfg.gen_len
    # vanilla is also what a from-scratch greedy loop gives (first 6 tokens, full recompute each step)
    seq = list(prompt)
    for t in range(6):
        lg = exit_logits(cfg, w, forward_all(cfg, w, seq)[-1][-1])
        assert int(np.argmax(lg)) == vanilla[t]
        seq.append(vanilla[t])
    # tokens per loaded layer of plain decoding is 1/L (prefill token not counted)
    assert sum(r.loaded_layers for r in vr) == cfg.n_layers * (cfg.gen_len - 1)
    for E in range(cfg.e_min, cfg.e_max + 1):
        for gamma in range(cfg.g_min, cfg.g_max + 1):
            _, out, _, rounds = run(cfg, w, prompt, policy=(E, gamma))
            assert out == vanilla, (E, gamma)
            for r in rounds:
                assert 1 <= len(r.emitted) <= r.g + 1 <= gamma + 1
                assert r.loaded_layers == r.g * E + cfg.n_layers
    _, out, _, _ = run(cfg, w, prompt)                   # dynamic (E, gamma)
    assert out == vanilla


def test_round_invariants_and_bruteforce_shadow_tokens(case):
    cfg, w, prompt = case
    L = cfg.n_layers
    o, out, init, rounds = run(cfg, w, prompt)
    assert len(out) == cfg.gen_len
    n_rejecting = 0
    committed = list(prompt) + [out[0]]
    Sc_hist = [np.array([(init.shadow[l] == init.shadow[L - 1]).sum() for l in range(L)], dtype=np.float64)]
    n_hist = [float(init.shadow.shape[1])]
    E, gamma = init.next_E, init.next_gamma
    for r in rounds:
        assert (r.E, r.gamma) == (E, gamma)
        g, n = r.g, r.n_accept
        n_rejecting += n < g
        verified = r.shadow[L - 1]
        # the draft layer's shadow tokens are the drafts; layer L always matches itself
        assert list(r.shadow[r.E - 1][:g]) == r.drafts
        assert n == oracle.accept_len(r.drafts, verified) and r.emitted == list(verified[:n + 1])
        assert r.counts[L - 1] == n + 1 and (r.counts <= n + 1).all() and (r.counts >= 0).all()
        # brute force: shadow token of layer l at a valid row = greedy exit of the l-layer truncated
        # model on the committed sequence, recomputed from scratch
        ctx = committed + r.emitted[:-1]                 # inputs of rows 0..n
        hs = forward_all(cfg, w, ctx)
        for l in range(1, L + 1):
            lg = exit_logits(cfg, w, hs[l][len(committed) - 1:])
            for i in range(n + 1):
                if r.margin[l - 1][i] > 1e-3:
                    assert int(np.argmax(lg[i])) == r.shadow[l - 1][i], (l, i)
            c = sum(int(r.shadow[l - 1][i] == verified[i]) for i in range(n + 1))
            assert c == r.counts[l - 1]
        committed += r.emitted
        # statistics: decayed sums straight from the definition over the whole history
        Sc_hist.append(r.counts.astype(np.float64))
        n_hist.append(float(n + 1))
        R = len(n_hist)
        Sn = sum(cfg.omega ** (R - i - 1) * n_hist[i] for i in range(R))
        Sc = sum(cfg.omega ** (R - i - 1) * Sc_hist[i] for i in range(R))
        assert abs(r.Sn - Sn) < 1e-9 * Sn
        alpha = Sc / Sn
        assert abs(alpha[L - 1] - 1.0) < 1e-12 and (alpha <= 1 + 1e-12).all()
        # selection = exhaustive argmax of the printed formula over the allowed grid
        best, arg = -1.0, None
        for l in range(cfg.e_min, cfg.e_max + 1):
            for d in range(cfg.g_min, cfg.g_max + 1):
                a = alpha[l - 1]
                t = (d + 1) / (d * l + L) if abs(a - 1) < 1e-12 else (1 - a ** (d + 1)) / ((1 - a) * (d * l + L))
                if t > best * (1 + 1e-12):
                    best, arg = t, (l, d)
        E, gamma = r.next_E, r.next_gamma
        a = alpha[E - 1]
        got = (gamma + 1) / (gamma * E + L) if abs(a - 1) < 1e-12 else (1 - a ** (gamma + 1)) / ((1 - a) * (gamma * E + L))
        assert abs(got - best) <= 1e-10 * best, ((E, gamma), arg)
    if cfg.name == "tiny_gqa":
        assert n_rejecting >= 3                          # the case really exercises rejection
    Sc_o, Sn_o, _, _ = o.get_stats()
    assert abs(Sc_o[L - 1] - Sn_o) < 1e-12 * Sn_o


def test_resume_from_stats_reproduces_the_trace(case):
    """Re-prefilling on prompt + emitted tokens and restoring the statistics continues identically."""
    cfg, w, prompt = case
    o, out, init, rounds = run(cfg, w, prompt)
    k = len(rounds) // 2
    emitted = [out[0]] + [t for r in rounds[:k] for t in r.emitted]
    a = oracle.OracleSeq(cfg, w)
    a.generate(prompt, len(emitted))
    st = a.get_stats()
    b = oracle.OracleSeq(cfg, w, max_seq=cfg.max_seq)
    tok, _ = b.prefill(np.array(list(prompt) + emitted[:-1], dtype=np.int32))
    assert tok == emitted[-1]
    b.set_stats(*st)
    tail = []
    while len(emitted) + len(tail) < cfg.gen_len:
        r = b.round(cfg.gen_len - len(emitted) - len(tail))
        tail += r.emitted
    assert emitted + tail == out


def test_stored_tiny_trace_is_what_the_oracle_writes_today():
    """tests/golden/trace_tiny.json was written by make_traces.py from the oracle; the oracle as it stands must write
    the same trace (tokens, shadow tokens, margins, counts, statistics, choices): the stored full-size traces, which
    take hours to regenerate, come from the same code path."""
    import importlib.util
    import json
    import os
    golden = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_traces", os.path.join(golden, "make_traces.py"))
    mt = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mt)
    doc = json.load(open(os.path.join(golden, "trace_tiny.json")))
    cfg = synth.CONFIGS["tiny"]
    assert doc["seed"] == cfg.seed and doc["prompt_len"] == cfg.prompt_len
    rec = mt.trace_sequence(cfg, synth.make_weights(cfg), 0, doc["gen_len"])
    want = doc["sequences"][0]
    rec.pop("oracle_seconds"), want.pop("oracle_seconds")
    assert json.loads(json.dumps(rec)) == want
