"""Pins for the oracle's speculative sampling (Sec. 2; temperature and top-p of the inference setup).  CPU only.

What fixes the implementation from outside:
  * the uniform numbers: range, determinism, a Kolmogorov-Smirnov test against the uniform law, no
    correlation between purposes or neighbouring positions;
  * the filtered distribution: scipy's softmax + numpy's stable sort and cumulative sum on the same row; the
    two limits (top_p = 1: plain tempered softmax; top_p -> 0: one-hot on the arg-max); minimality of the
    nucleus; equal probabilities enter in token-id order;
  * the inverse CDF: numpy's searchsorted on the cumulative sum; empirical frequencies (chi-square);
  * acceptance + residual: the identity that makes speculative sampling exact,
    q(t) min(1, p(t)/q(t)) + (1 - sum_x q(x) min(1, p(x)/q(x))) r(t) = p(t), evaluated with the oracle's arrays,
    and a Monte-Carlo run of the whole step whose output frequencies must follow p and not q;
  * the round: every decision it reports is recomputed here from the logits it exposes, with numpy, and the
    uniform numbers keyed by (seed, absolute position, purpose); the statistics count the rows 0..n of the
    tokens that were really emitted; temperature -> 0 reproduces the greedy stream.
"""
import numpy as np
import pytest
from scipy import stats
from scipy.special import softmax as sp_softmax

import oracle
import synth
from cases import TINY, TINY_GQA

CASES = [TINY, TINY_GQA]


@pytest.fixture(scope="module", params=CASES, ids=lambda c: c.name)
def case(request):
    cfg = request.param
    return cfg, synth.make_weights(cfg), synth.make_prompt(cfg)


# ---------------------------------------------------------------- uniform numbers
def test_uniform_numbers():
    u = np.array([oracle.uniform(7, pos, pur) for pos in range(4000) for pur in range(3)]).reshape(4000, 3)
    assert u.min() >= 0.0 and u.max() < 1.0
    assert oracle.uniform(7, 123, 1) == u[123, 1]                        # a pure function of its arguments
    assert oracle.uniform(8, 123, 1) != u[123, 1]
    assert len(np.unique(u)) == u.size
    assert stats.kstest(u.ravel(), "uniform").pvalue > 1e-3
    for a in range(3):
        for b in range(a + 1, 3):
            assert abs(np.corrcoef(u[:, a], u[:, b])[0, 1]) < 0.06       # purposes are independent streams
        assert abs(np.corrcoef(u[:-1, a], u[1:, a])[0, 1]) < 0.06        # so are neighbouring positions
    # 53-bit resolution: the numbers are multiples of 2^-53
    assert all(float(x * 2.0 ** 53).is_integer() for x in u[:50, 0])


# ---------------------------------------------------------------- filtered distribution
def _nucleus_numpy(x, T, top_p):
    p = sp_softmax(x.astype(np.float64) / T)
    if top_p >= 1.0:
        return p
    order = np.argsort(-p, kind="stable")                                # ties: lower id first
    before = np.concatenate([[0.0], np.cumsum(p[order])[:-1]])
    keep = order[before < top_p]
    out = np.zeros_like(p)
    out[keep] = p[keep]
    return out / out.sum()


@pytest.mark.parametrize("V,scale", [(17, 1.0), (1000, 0.3), (1000, 4.0), (32000, 1.0)])
@pytest.mark.parametrize("T,top_p", [(0.6, 0.95), (1.0, 0.5), (0.3, 0.9), (1.5, 0.999)])
def test_nucleus_against_numpy(V, scale, T, top_p):
    rng = np.random.default_rng(V + int(100 * T))
    x = (rng.standard_normal(V) * scale).astype(np.float32)
    got, want = oracle.nucleus(x, T, top_p), _nucleus_numpy(x, T, top_p)
    assert np.array_equal(got > 0, want > 0)
    assert np.allclose(got, want, rtol=1e-12, atol=0)
    assert abs(got.sum() - 1.0) < 1e-12
    # minimal: the kept tokens reach top_p, and no longer without the smallest of them
    full = sp_softmax(x.astype(np.float64) / T)
    kept = full[got > 0]
    assert kept.sum() >= top_p - 1e-12 and kept.sum() - kept.min() < top_p
    assert kept.min() >= full[got == 0].max() if (got == 0).any() else True


def test_nucleus_limits_and_ties():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(300).astype(np.float32)
    assert np.allclose(oracle.nucleus(x, 0.7, 1.0), sp_softmax(x.astype(np.float64) / 0.7), rtol=1e-12)
    one = oracle.nucleus(x, 0.7, 1e-9)
    assert one[np.argmax(x)] == 1.0 and one.sum() == 1.0
    cold = oracle.nucleus(x, 1e-3, 0.95)                                 # temperature -> 0: the arg-max
    assert cold[np.argmax(x)] > 1.0 - 1e-9
    # eight equal logits, top_p = 0.5: the four lowest ids stay (mass before the 5th is exactly 0.5)
    flat = oracle.nucleus(np.zeros(8, dtype=np.float32), 1.0, 0.5)
    assert np.array_equal(flat, [0.25] * 4 + [0.0] * 4)
    # two tied leaders and a tail: 0.4, 0.4, 0.1, 0.1 with top_p = 0.85 keeps ids 0, 1, 2
    t = np.log(np.array([0.4, 0.4, 0.1, 0.1])).astype(np.float32)
    assert np.array_equal(oracle.nucleus(t, 1.0, 0.85) > 0, [True, True, True, False])
    # large logits do not overflow
    big = oracle.nucleus(np.array([3000.0, 2999.0, -3000.0], dtype=np.float32), 1.0, 1.0)
    assert np.allclose(big, sp_softmax([0.0, -1.0, -6000.0]), rtol=1e-12)


# ---------------------------------------------------------------- inverse CDF
def test_sample_cdf_against_searchsorted_and_frequencies():
    rng = np.random.default_rng(11)
    p = oracle.nucleus(rng.standard_normal(40).astype(np.float32) * 2, 1.0, 0.9)
    cdf = np.cumsum(p)
    us = rng.random(5000)
    got = np.array([oracle.sample_cdf(p, u) for u in us])
    want = np.searchsorted(cdf, us, side="right")
    assert np.array_equal(got, want)
    assert (p[got] > 0).all()                                            # never a filtered token
    assert oracle.sample_cdf(p, 0.0) == int(np.flatnonzero(p > 0)[0])
    assert oracle.sample_cdf(p, 1.0 - 2.0 ** -53) == int(np.flatnonzero(p > 0)[-1])
    # frequencies with the oracle's own uniform numbers
    draws = np.array([oracle.sample_cdf(p, oracle.uniform(5, k, 0)) for k in range(20000)])
    keep = p > 0
    obs = np.bincount(draws, minlength=p.size)[keep]
    assert stats.chisquare(obs, p[keep] * len(draws)).pvalue > 1e-3


# ---------------------------------------------------------------- acceptance and residual
def test_residual_and_the_exactness_identity():
    rng = np.random.default_rng(21)
    for V, T, top_p in [(6, 1.0, 1.0), (50, 0.6, 0.95), (400, 0.6, 0.8)]:
        p = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 2, T, top_p)
        q = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 2, T, top_p)
        r, R = oracle.residual(p, q)
        assert abs(r.sum() - 1.0) < 1e-12 and (r[q >= p] == 0).all() and (r >= 0).all()
        assert R == pytest.approx(np.maximum(p - q, 0).sum(), rel=1e-12)
        acc = np.where(q > 0, q * np.minimum(1.0, p / np.where(q > 0, q, 1.0)), 0.0)   # drafted and accepted
        out = acc + (1.0 - acc.sum()) * r                                              # or rejected and resampled
        assert np.allclose(out, p, atol=1e-12)
    same, R = oracle.residual(p, p)          # nothing can be rejected: defined as p itself
    assert R == 0.0 and np.array_equal(same, p)


def test_monte_carlo_step_follows_the_target():
    rng = np.random.default_rng(31)
    V, N = 8, 40000
    p = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 1.5, 1.0, 1.0)
    q = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 1.5, 1.0, 1.0)
    r, _ = oracle.residual(p, q)
    out = np.zeros(V)
    for k in range(N):
        x = oracle.sample_cdf(q, oracle.uniform(9, k, 0))
        if oracle.uniform(9, k, 1) < min(1.0, p[x] / q[x]):
            out[x] += 1
        else:
            out[oracle.sample_cdf(r, oracle.uniform(9, k, 2))] += 1
    assert stats.chisquare(out, p * N).pvalue > 1e-3
    assert stats.chisquare(out, q * N).pvalue < 1e-6                     # and clearly not the draft distribution


# ---------------------------------------------------------------- the round
T_S, P_S = 0.6, 0.95


def _replay_round(cfg, o, r, T0, seed):
    """Recomputes every decision of round r from the logits the oracle exposes, with numpy."""
    si = o.sample_info()
    drafts = []
    for i in range(r.g):
        q = _nucleus_numpy(o.round_logits(0, i), T_S, P_S)
        u = oracle.uniform(seed, T0 + 1 + i, 0)
        assert u == si.u_draft[i]
        x = int(np.searchsorted(np.cumsum(q), u, side="right"))
        drafts.append(x)
        assert si.q_x[i] == pytest.approx(q[x], rel=1e-12)
    assert drafts == r.drafts
    n, rejected = 0, False
    while n < r.g:
        p = _nucleus_numpy(o.round_logits(1, n), T_S, P_S)
        q = _nucleus_numpy(o.round_logits(0, n), T_S, P_S)
        u = oracle.uniform(seed, T0 + 1 + n, 1)
        assert u == si.u_accept[n] and si.p_x[n] == pytest.approx(p[drafts[n]], rel=1e-12, abs=1e-300)
        if u < min(1.0, p[drafts[n]] / q[drafts[n]]):
            n += 1
        else:
            rejected = True
            break
    assert n == r.n_accept and rejected == bool(si.from_residual)
    u = oracle.uniform(seed, T0 + 1 + n, 2)
    assert u == si.u_final
    if rejected:
        res = np.maximum(p - q, 0.0)
        last = int(np.searchsorted(np.cumsum(res / res.sum()), u, side="right"))
    else:
        last = int(np.searchsorted(np.cumsum(_nucleus_numpy(o.round_logits(1, r.g), T_S, P_S)), u, side="right"))
    assert r.emitted == drafts[:n] + [last]


@pytest.mark.parametrize("exit_mode", [False, True])
def test_round_decisions_replayed_from_its_logits(case, exit_mode):
    cfg, w, prompt = case
    seed = 4242
    o = oracle.OracleSeq(cfg, w)
    o.set_sampling(T_S, P_S, seed)
    o.set_exit_mode(exit_mode)
    tok, init = o.prefill(prompt)
    # the first token: drawn from the target's filtered distribution at the last prompt position
    first = _nucleus_numpy(o.round_logits(1, 0), T_S, P_S)
    assert tok == int(np.searchsorted(np.cumsum(first), oracle.uniform(seed, len(prompt), 2), side="right"))
    if not exit_mode:
        o.set_policy(cfg.e_min, min(3, cfg.g_max))       # a weak draft model: rejections happen
    n_tok, rejections, L = 1, 0, cfg.n_layers
    while n_tok < cfg.gen_len:
        T0 = o.T
        Sc0, Sn0, _, _ = o.get_stats()
        r = o.round(cfg.gen_len - n_tok)
        _replay_round(cfg, o, r, T0, seed)
        rejections += r.n_accept < r.g
        # statistics: rows 0..n of the emitted tokens, shadow tokens compared with the target's greedy ones
        Sc1, Sn1, _, _ = o.get_stats()
        assert Sn1 == oracle.decay_step(Sn0, cfg.omega, r.n_accept + 1)
        for l in range(L):
            c = int((r.shadow[l][:r.n_accept + 1] == r.shadow[L - 1][:r.n_accept + 1]).sum())
            assert r.counts[l] == c and Sc1[l] == oracle.decay_step(Sc0[l], cfg.omega, c)
        assert o.T == T0 + r.n_accept + 1
        n_tok += len(r.emitted)
    if not exit_mode and cfg is TINY_GQA:
        assert rejections >= 1           # (the 4-layer case's exit layer agrees with its target almost everywhere)
    o.close()


def test_cold_sampling_is_greedy(case):
    """Temperature -> 0 puts all mass on the arg-max: the sampled stream is the greedy one (wherever the
    top-1 margin is not tiny) and every draft that equals the target's token is accepted."""
    cfg, w, prompt = case
    g = oracle.OracleSeq(cfg, w)
    g.set_policy(cfg.e_min, 2)
    want, _, grounds = g.generate(prompt, 24)
    o = oracle.OracleSeq(cfg, w)
    o.set_sampling(1e-4, 0.95, 1)
    o.set_policy(cfg.e_min, 2)
    got, _, rounds = o.generate(prompt, 24)
    assert got == want
    assert [(r.g, r.n_accept) for r in rounds] == [(r.g, r.n_accept) for r in grounds]
    g.close(); o.close()


def test_sampled_first_tokens_follow_the_target(case):
    """Over many seeds the token that ends round 1 (gamma = 1: accepted draft's successor or the resampled one)
    is distributed like plain sampling from the target would be at the same position: checked on the round's
    first emitted token, whose context is the same for every seed."""
    cfg, w, prompt = case
    prompt = prompt[:8]
    N, bins = 1500, 8
    counts, expect = np.zeros(bins), None
    for seed in range(N):
        o = oracle.OracleSeq(cfg, w)
        o.prefill(prompt)                        # greedy first token: one context for all seeds
        o.set_sampling(1.0, 1.0, seed)
        o.set_policy(cfg.e_min, 1)
        r = o.round(8)
        if expect is None:
            p = _nucleus_numpy(o.round_logits(1, 0), 1.0, 1.0)
            expect = np.array([p[b::bins].sum() for b in range(bins)])
        counts[r.emitted[0] % bins] += 1
        o.close()
    assert stats.chisquare(counts, expect * N).pvalue > 1e-3


# ---------------------------------------------------------------- properties on arbitrary rows
from hypothesis import given, settings, strategies as st


@settings(max_examples=60, deadline=None)
@given(st.integers(2, 400), st.floats(0.05, 3.0), st.floats(0.05, 1.0), st.floats(0.05, 8.0), st.integers(0, 2 ** 31))
def test_nucleus_properties(V, T, top_p, scale, seed):
    rng = np.random.default_rng(seed)
    x = (np.round(rng.standard_normal(V) * scale * 4) / 4).astype(np.float32)      # quantised: ties are common
    p = oracle.nucleus(x, T, top_p)
    full = sp_softmax(x.astype(np.float64) / T)
    kept = p > 0
    assert abs(p.sum() - 1.0) < 1e-12 and kept[np.argmax(x)]
    assert np.allclose(p[kept] / p[kept].sum(), full[kept] / full[kept].sum(), rtol=1e-12)    # renormalised, not reshaped
    if (~kept).any():
        assert full[kept].min() >= full[~kept].max() - 1e-18                        # a top set
        assert full[kept].sum() >= top_p - 1e-12                                    # that reaches top_p
        # among equal probabilities at the edge the lower ids stay
        edge = full[kept].min()
        tied = np.flatnonzero(np.abs(full - edge) <= 1e-18)
        flags = kept[tied]
        assert not (np.diff(flags.astype(int)) > 0).any()


@settings(max_examples=40, deadline=None)
@given(st.integers(2, 200), st.integers(0, 2 ** 31))
def test_inverse_cdf_is_monotone_and_residual_is_a_distribution(V, seed):
    rng = np.random.default_rng(seed)
    p = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 2, 0.8, 0.9)
    q = oracle.nucleus(rng.standard_normal(V).astype(np.float32) * 2, 0.8, 0.9)
    us = np.sort(rng.random(50))
    toks = [oracle.sample_cdf(p, u) for u in us]
    assert toks == sorted(toks) and all(p[t] > 0 for t in toks)
    r, R = oracle.residual(p, q)
    assert abs(r.sum() - 1.0) < 1e-12 and (r >= 0).all() and 0.0 <= R <= 1.0 + 1e-12
    if R > 0:
        assert ((r > 0) <= (p > q)).all()
    else:
        assert np.array_equal(r, p)         # nothing can be rejected: defined as p itself
