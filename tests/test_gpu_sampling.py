"""Speculative sampling (Sec. 2) of the CUDA library against the CPU oracle.  Needs a B200."""
import json
import os

import numpy as np
import pytest

import synth
from cases import TINY, TINY_GQA
from parity import ref_from_golden, run_sequence
from sampling_parity import run_sequence_sampling

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_ctx(cfg, weights, **kw):
    import paper_2504_05598_b200 as dl
    dev = dl.upload_weights(weights)
    return dl.DelContext(dl.make_shape(cfg, **kw), dev)


# ---------------------------------------------------------------- the sampling kernels on given rows
def _rows(rng, V, kind):
    """Seeded pairs of logit rows (target, draft) with the structure the method meets."""
    if kind == "random_model":           # near-uniform: what the synthetic random-weight models produce
        p = rng.standard_normal(V) * 0.35
        q = p + rng.standard_normal(V) * 0.05
    elif kind == "peaked":               # a trained model: a few likely tokens, a long tail
        p = rng.standard_normal(V) * 2.5
        p[rng.integers(0, V, 3)] += 9.0
        q = p + rng.standard_normal(V) * 0.8
    elif kind == "disagree":             # draft and target prefer different tokens: rejections, residual draws
        p = rng.standard_normal(V) * 2.0
        q = rng.standard_normal(V) * 2.0
    elif kind == "quantised":            # many equal logits: ties inside and at the edge of the nucleus
        p = np.round(rng.standard_normal(V) * 2.0) * 0.5
        q = np.round(rng.standard_normal(V) * 2.0) * 0.5
    elif kind == "plateau":              # three levels: the nucleus ends inside a run of equal weights (id order decides)
        p = np.zeros(V); p[::7] = 1.0; p[3::13] = -1.0
        q = np.zeros(V); q[2::5] = 1.0; q[1::11] = -1.0
    else:
        raise ValueError(kind)
    return p.astype(np.float32), q.astype(np.float32)


def _margin(probs, x, u):
    c = np.cumsum(probs)
    return min(abs(u - (c[x] - probs[x])), abs(u - c[x]))


def _nucleus_slack(logits, T, top_p):
    """Distance of the nucleus decision from its threshold, in probability mass."""
    import oracle
    full = oracle.nucleus(logits, T, 1.0)
    order = np.argsort(-full, kind="stable")
    before = np.concatenate([[0.0], np.cumsum(full[order])[:-1]])
    return float(np.abs(before - top_p).min())


@pytest.mark.parametrize("V", [1024, 32000, 128256])
def test_sampling_kernels_against_oracle(V):
    """Same rows, same uniform numbers on both sides: the drafted token, the acceptance decision, the residual draw
    and the draw from the target row must be identical, the filtered probabilities equal to 1e-6.  Only a
    decision that the oracle itself takes within 1e-7 of its boundary may differ."""
    import oracle
    cfg = synth.small_variant(TINY, name=f"tiny_v{V}", vocab=V, seed=900 + V % 97)
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    rng = np.random.default_rng(V)
    n_cases = 60 if V <= 32000 else 24
    kinds = ["random_model", "peaked", "disagree", "quantised", "plateau"]
    settings = [(0.6, 0.95), (1.0, 0.9), (0.3, 0.5), (1.3, 1.0), (0.6, 0.999)]
    compared = near = 0
    for k in range(n_cases):
        kind = kinds[k % len(kinds)]
        T, top_p = settings[(k // len(kinds)) % len(settings)]
        p, q = _rows(rng, V, kind)
        ud, ua, uf = (oracle.uniform(V, k, j) for j in range(3))
        out, prob, stat = ctx.sample_probe(p, q, T, top_p, ud, ua, uf)
        qq, pp = oracle.nucleus(q, T, top_p), oracle.nucleus(p, T, top_p)
        x = oracle.sample_cdf(qq, ud)
        slack = min(_nucleus_slack(p, T, top_p), _nucleus_slack(q, T, top_p)) if top_p < 1.0 else 1.0
        tag = f"case {k} ({kind}, T={T}, top_p={top_p})"
        if slack < 1e-7:
            near += 1
            continue                    # the nucleus itself is a coin flip in the last bits
        compared += 1
        if out[0] != x:
            assert _margin(qq, x, ud) < 1e-7, f"{tag}: draft {out[0]} oracle {x}"
            near += 1
            continue
        # (the library's weights are 40-bit fixed point: a filtered probability carries an absolute error below 2e-12)
        assert prob[0] == pytest.approx(qq[x], rel=1e-6, abs=2e-12), tag
        assert prob[1] == pytest.approx(pp[x], rel=1e-6, abs=2e-12), tag
        ratio = min(1.0, pp[x] / qq[x])
        if bool(out[1]) != (ua < ratio):
            assert abs(ua - ratio) < 1e-7, f"{tag}: acceptance {out[1]} oracle u {ua} ratio {ratio}"
            near += 1
        r, R = oracle.residual(pp, qq)
        xr = oracle.sample_cdf(r, uf)
        if out[2] != xr:
            assert R < 1e-6 or _margin(r, xr, uf) < 1e-7 / max(R, 1e-12), f"{tag}: residual draw {out[2]} oracle {xr} (R={R})"
            near += 1
        xb = oracle.sample_cdf(pp, uf)
        if out[3] != xb:
            assert _margin(pp, xb, uf) < 1e-7, f"{tag}: target draw {out[3]} oracle {xb}"
            near += 1
    print(f"V={V}: {compared} pairs compared, {near} decisions at a boundary")
    assert compared >= n_cases * 0.8 and near <= max(3, n_cases // 6)
    ctx.close()


def test_sampling_kernel_ties_and_limits():
    import oracle
    cfg = TINY
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    V = 64
    flat = np.zeros(V, dtype=np.float32)
    # 64 equal logits, top_p = 0.5: the 32 lowest ids stay; u walks through them in id order
    for u in (0.0, 0.26, 0.5, 0.999):
        out, prob, stat = ctx.sample_probe(flat, flat, 1.0, 0.5, u, 0.5, u)
        assert out[0] == int(u * 32) and prob[0] == pytest.approx(1 / 32)
        assert stat[1] == 32 and stat[2] == 64           # ties kept / present
        assert out[1] == 1                               # p == q: always accepted
        assert out[3] == int(u * 32)
    # temperature -> 0: the arg-max, whatever u is
    rng = np.random.default_rng(1)
    z = rng.standard_normal(1000).astype(np.float32)
    for u in (0.0, 0.5, 0.999999):
        out, prob, _ = ctx.sample_probe(z, z, 1e-4, 0.95, u, 0.5, u)
        assert out[0] == int(np.argmax(z)) and out[3] == int(np.argmax(z)) and prob[0] == pytest.approx(1.0)
    # one-hot target against one-hot draft on another token: certain rejection, the residual is the target's token
    p = np.full(100, -50.0, dtype=np.float32); p[7] = 0.0
    q = np.full(100, -50.0, dtype=np.float32); q[9] = 0.0
    out, prob, _ = ctx.sample_probe(p, q, 1.0, 1.0, 0.3, 1e-12, 0.8)
    assert out[0] == 9 and out[1] == 0 and out[2] == 7
    # top_p = 1 keeps everything: the draw follows the plain softmax CDF
    z = rng.standard_normal(500).astype(np.float32)
    cdf = np.cumsum(oracle.nucleus(z, 0.8, 1.0))
    for u in (0.1, 0.5, 0.9):
        out, _, _ = ctx.sample_probe(z, z, 0.8, 1.0, u, 0.5, u)
        assert out[0] == int(np.searchsorted(cdf, u, side="right"))
    ctx.close()


# ---------------------------------------------------------------- whole rounds
@pytest.mark.parametrize("cfg", [TINY, TINY_GQA], ids=lambda c: c.name)
@pytest.mark.parametrize("exit_mode", [False, True], ids=["fixed_gamma", "draft_exiting"])
def test_speculative_sampling_against_oracle(cfg, exit_mode):
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    prompt = synth.make_prompt(cfg)
    total = SReportTotal()
    for seed in (11, 12, 13):
        policy = None if exit_mode else (cfg.e_min, min(3, cfg.g_max))
        rep = run_sequence_sampling(ctx, 0, cfg, w, prompt, 0.6, 0.95, seed, exit_mode=exit_mode, policy=policy)
        print(f"{cfg.name} seed {seed} exit {exit_mode}: rounds {rep.rounds} drafts {rep.drafts} tests {rep.tests} rejections "
              f"{rep.rejections} flips {rep.flips} resyncs {rep.resyncs} max logit diff {rep.eps_max:.4f} max prob rel diff "
              f"{rep.prob_max_rel:.2e}")
        assert rep.ok(), rep.failures[:5]
        total.add(rep)
    assert total.rounds >= 10 and total.drafts > 0
    assert total.flips <= total.rounds // 2          # most rounds agree decision by decision
    ctx.close()


class SReportTotal:
    def __init__(self):
        self.rounds = self.drafts = self.flips = 0

    def add(self, rep):
        self.rounds += rep.rounds
        self.drafts += rep.drafts
        self.flips += rep.flips


def test_dynamic_selection_with_sampling():
    """Sampling with the dynamic (E, gamma) selection on the deeper small model."""
    cfg = TINY_GQA
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    rep = run_sequence_sampling(ctx, 0, cfg, w, synth.make_prompt(cfg), 1.0, 0.9, 5)
    print(f"dynamic selection: rounds {rep.rounds} flips {rep.flips} rejections {rep.rejections}")
    assert rep.ok(), rep.failures[:5]
    ctx.close()


def test_batch_with_sampled_and_greedy_sequences():
    """Three sequences share every round: one greedy, one sampling with a fixed policy, one sampling with dynamic
    draft-exiting; each is compared with its own oracle."""
    from parity import Report, _resync, compare_init, compare_round, ref_from_oracle
    from sampling_parity import SeqSampler
    cfg = synth.small_variant(TINY_GQA, name="tiny_gqa_b3", batch=3, gen_len=32)
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    prompts = [synth.make_prompt(cfg, s) for s in range(3)]
    ref0 = ref_from_oracle(cfg, w, prompts[0])
    rep0 = Report()
    compare_init(ctx, 0, ref0, cfg.gen_len, rep0)
    s1 = SeqSampler(ctx, 1, cfg, w, prompts[1], 0.6, 0.95, 31, policy=(cfg.e_min, 2))
    s2 = SeqSampler(ctx, 2, cfg, w, prompts[2], 0.8, 0.9, 32, exit_mode=True)
    s1.begin()
    s2.begin()
    k0, done0 = 0, 1
    while k0 < len(ref0.rounds) or not s1.done or not s2.done:
        outs = ctx.round()
        if k0 < len(ref0.rounds):
            r = ref0.rounds[k0]
            need = compare_round(ctx, 0, outs[0], r, rep0)
            done0 += r.n + 1
            k0 += 1
            if need and k0 < len(ref0.rounds):
                rep0.resyncs += 1
                _resync(ctx, 0, ref0, done0, r.Sc, r.Sn, r.next_E, r.next_gamma, cfg.gen_len, r.Stcs, r.Sfcs)
        for s in (s1, s2):
            if not s.done:
                s.after_round(outs[s.seq])
        assert len(rep0.failures) + len(s1.rep.failures) + len(s2.rep.failures) == 0, \
            (rep0.failures[:3], s1.rep.failures[:3], s2.rep.failures[:3])
    print(f"greedy: rounds {rep0.rounds} flips {rep0.flips}; sampled: rounds {s1.rep.rounds} flips {s1.rep.flips}; "
          f"sampled + draft-exiting: rounds {s2.rep.rounds} flips {s2.rep.flips}")
    assert rep0.rounds == len(ref0.rounds) and s1.rep.rounds >= 5 and s2.rep.rounds >= 5
    s1.close(); s2.close(); ctx.close()


@pytest.mark.parametrize("exit_mode", [False, True], ids=["fixed_gamma", "draft_exiting"])
def test_sampling_step_calls_equal_round_call(exit_mode):
    """del_draft / del_verify / del_layer_accept / del_select with sampling on give the stream of del_round, and
    three runs with one seed give one stream (no order-dependent arithmetic anywhere on the path)."""
    cfg = TINY_GQA
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    prompt = synth.make_prompt(cfg)
    ctx.set_sampling(0, 0.7, 0.9, 99)

    def by_steps():
        first = ctx.prefill(0, prompt, 30)
        ctx.set_exit_mode(0, exit_mode)
        toks, E, g, trace = [first.tokens[0]], first.next_E, first.next_gamma, []
        while len(toks) < 30:
            ctx.draft(0, E, cfg.g_max if exit_mode else g)
            ctx.verify(0)
            out = ctx.layer_accept(0)
            E, g = ctx.select(0)
            toks += out.emitted()
            trace.append((out.E, out.g, bool(out.stopped), out.n_accept, E, g))
        return toks, trace

    def by_rounds():
        first = ctx.prefill(0, prompt, 30)
        ctx.set_exit_mode(0, exit_mode)
        toks, trace = [first.tokens[0]], []
        while len(toks) < 30:
            out = ctx.round()[0]
            toks += out.emitted()
            trace.append((out.E, out.g, bool(out.stopped), out.n_accept, out.next_E, out.next_gamma))
        return toks, trace

    streams, rejected = [], False
    for seed in (99, 100, 101):                                  # which rounds reject depends on the seed
        ctx.set_sampling(0, 0.7, 0.9, seed)
        a, b, c = by_steps(), by_rounds(), by_rounds()
        assert a == b == c and len(a[0]) == 30, seed
        rejected = rejected or any(t[3] < t[1] for t in a[1])
        streams.append(tuple(a[0]))
    assert rejected or exit_mode                                 # a rejection happened
    assert len(set(streams)) == len(streams)                     # another seed: another stream
    ctx.close()


@pytest.mark.parametrize("name", ["llama2_7b", "llama32_1b", "llama2_13b", "llama3_8b_b4"])
def test_cold_sampling_reproduces_greedy_trace_full_size(name):
    """Temperature -> 0 puts all filtered mass on the arg-max: the sampling path (logit rows of exit head and target,
    nucleus, draws, acceptance ratio, residual) must then reproduce the stored greedy oracle traces of the full-size
    shapes, decision by decision (the four sequences of the 8B shape share their rounds)."""
    from parity import run_batch
    path = os.path.join(GOLDEN, f"trace_{name}.json")
    if not os.path.exists(path):
        pytest.skip("no stored trace")
    doc = json.load(open(path))
    cfg = synth.CONFIGS[name]
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    for s in range(cfg.batch):
        ctx.set_sampling(s, 1e-4, 0.95, 77 + s)
    refs = [ref_from_golden(doc, s, synth.make_prompt(cfg, s)) for s in range(cfg.batch)]
    if cfg.batch > 1:
        reps = run_batch(ctx, refs, doc["gen_len"])
    else:
        reps = [run_sequence(ctx, 0, refs[0], doc["gen_len"], max_rounds=40)]
    for s, rep in enumerate(reps):
        print(f"{name} seq {s} (cold sampling): rounds {rep.rounds} compared {rep.compared} flips {rep.flips} resyncs {rep.resyncs}")
        assert rep.ok(), rep.failures[:8]
        assert rep.rounds >= 20
    ctx.close()


@pytest.mark.parametrize("name", ["llama2_7b", "llama3_8b_b4"])
def test_sampling_full_size_consistency(name):
    """Full-size shapes (Llama-2-7B; Llama-3-8B with four sequences, grouped-query attention and a 128 256-token
    vocabulary) at temperature 0.6 / 1.0, top-p 0.95, one sequence of the batch with draft-exiting: the reported
    decisions are consistent with the reported probabilities and the uniform numbers of (seed, position, purpose);
    tokens are valid ids; a second run with the same seeds gives the same streams."""
    import oracle
    cfg = synth.CONFIGS[name]
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    B, n_tok = cfg.batch, 40
    streams = []
    for attempt in range(2):
        T, toks = [], [[] for _ in range(B)]
        for s in range(B):
            prompt = synth.make_prompt(cfg, s)
            ctx.set_sampling(s, 0.6 if s % 2 == 0 else 1.0, 0.95, 2024 + s)
            first = ctx.prefill(s, prompt, n_tok)
            if B == 1:
                ctx.set_policy(s, 8, 3)
            elif s == B - 1:
                ctx.set_exit_mode(s, True)
            toks[s].append(first.tokens[0])
            T.append(len(prompt))
        tests = 0
        while any(len(t) < n_tok for t in toks):
            outs = ctx.round()
            for s in range(B):
                out = outs[s]
                if out.n_emitted == 0:
                    continue
                n_tests, from_res, qx, px = ctx.get_sample_info(s)
                assert 0 <= out.n_accept <= out.g and out.n_emitted == out.n_accept + 1
                assert n_tests == min(out.n_accept + 1, out.g) and from_res == (out.n_accept < out.g)
                for i in range(n_tests):
                    u = oracle.uniform(2024 + s, T[s] + 1 + i, 1)
                    ratio = min(1.0, float(px[i]) / float(qx[i]))
                    if abs(u - ratio) > 1e-5:
                        assert (u < ratio) == (i < out.n_accept), (s, i, u, ratio)
                    tests += 1
                assert all(0 <= t < cfg.vocab for t in out.emitted())
                toks[s] += out.emitted()
                T[s] += out.n_emitted
        assert tests > 0
        streams.append(toks)
    assert streams[0] == streams[1]
    ctx.close()


def test_sampling_error_codes():
    import paper_2504_05598_b200 as dl
    cfg = TINY
    ctx = make_ctx(cfg, synth.make_weights(cfg))
    assert ctx.lib.del_set_sampling(ctx._h, -1, 0.6, 0.9, 1) == dl.EINVAL
    assert ctx.lib.del_set_sampling(ctx._h, 0, 0.6, 0.0, 1) == dl.EINVAL
    assert ctx.lib.del_set_sampling(ctx._h, 0, 0.0, 0.0, 1) == 0          # off: top_p is not looked at
    buf = np.zeros(cfg.vocab, dtype=np.float32)
    assert ctx.lib.del_get_round_logits(ctx._h, 0, 0, 99, buf.ctypes.data) == dl.EINVAL
    assert ctx.lib.del_sample_probe(ctx._h, buf.ctypes.data, buf.ctypes.data, cfg.vocab + 1, 1.0, 1.0, 0.1, 0.1, 0.1,
                                    buf.ctypes.data, buf.ctypes.data, None) == dl.EINVAL
    ctx.close()
