"""Pins for the oracle's dynamic draft-exiting (Sec. 4.4, Eq. 3, Algorithm 1).  CPU only.

What fixes the implementation from outside:
  * the confidence is the top-1 softmax probability: checked against scipy's softmax and against an
    independent numpy forward pass of the truncated model;
  * Eq. 3 and the decayed sums: recomputed from the explicit per-round history with the paper's
    S(a) = sum_i omega^(r-i-1) a[i];
  * Algorithm 1's loop: a threshold above 1 stops every round before its first draft (the stream is then
    plain auto-regressive decoding, one token per round), a threshold of 0 never stops (g_max drafts);
    in every mode the emitted stream equals greedy auto-regressive decoding;
  * the break rule itself: every kept draft has confidence >= tau, the dropped one < tau.
"""
import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

import oracle
import synth
from cases import TINY, TINY_GQA
from np_model import exit_logits, forward_all

CASES = [TINY, TINY_GQA]


@pytest.fixture(scope="module", params=CASES, ids=lambda c: c.name)
def case(request):
    cfg = request.param
    return cfg, synth.make_weights(cfg), synth.make_prompt(cfg)


def test_confidence_is_top1_softmax_probability():
    rng = np.random.default_rng(5)
    for scale in (0.1, 1.0, 30.0, 300.0):            # large logits: the max must be subtracted first
        x = (rng.standard_normal(997) * scale).astype(np.float32)
        want = sp_softmax(x.astype(np.float64)).max()
        got = oracle.confidence(x)
        assert abs(got - want) <= 1e-12 * max(1.0, want)
        assert abs(got - oracle.softmax(x).max()) <= 1e-15
    assert oracle.confidence(np.zeros(8, dtype=np.float32)) == pytest.approx(1 / 8)
    assert oracle.confidence(np.array([50.0, -50.0], dtype=np.float32)) == pytest.approx(1.0)


def test_threshold_formula_and_empty_means():
    # Eq. 3: midpoint of mean matched confidence and mean mismatched confidence
    assert oracle.threshold(1.8, 2.0, 0.3, 1.0) == 0.5 * (1.8 / 2.0 + 0.3 / 1.0)
    # no matched token so far: that mean counts as 1; no mismatched token so far: that mean counts as 0
    assert oracle.threshold(0.0, 0.0, 0.3, 1.0) == 0.5 * (1.0 + 0.3)
    assert oracle.threshold(1.8, 2.0, 0.0, 0.0) == 0.5 * (0.9 + 0.0)
    assert oracle.threshold(0.0, 0.0, 0.0, 0.0) == 0.5


def test_shadow_confidences_against_independent_forward(case):
    cfg, w, prompt = case
    o = oracle.OracleSeq(cfg, w)
    tok, init = o.prefill(prompt)
    ref = forward_all(cfg, w, prompt)
    W = min(cfg.init_window, len(prompt))
    assert init.conf.shape == (cfg.n_layers, W)
    for l in range(1, cfg.n_layers + 1):
        for j in (0, W // 2, W - 1):
            lg = exit_logits(cfg, w, ref[l][len(prompt) - W + j])
            want = sp_softmax(lg).max()
            assert abs(init.conf[l - 1, j] - want) < 2e-4 * want + 1e-6, (l, j)


def _decayed(values, omega):
    """S(a) of Sec. 4.2 written out: sum_i omega^(r-i-1) a[i]."""
    r = len(values)
    return sum(omega ** (r - i - 1) * values[i] for i in range(r))


@pytest.mark.parametrize("exit_mode", [False, True])
def test_statistics_and_thresholds_from_explicit_history(case, exit_mode):
    cfg, w, prompt = case
    o = oracle.OracleSeq(cfg, w)
    o.set_exit_mode(exit_mode)
    tok, init = o.prefill(prompt)
    L = cfg.n_layers
    target = init.shadow[L - 1]
    hist_c = [[float((init.shadow[l] == target).sum())] for l in range(L)]
    hist_t = [[float(init.conf[l][init.shadow[l] == target].sum())] for l in range(L)]
    hist_f = [[float(init.conf[l][init.shadow[l] != target].sum())] for l in range(L)]
    hist_u = [float(init.shadow.shape[1])]
    n_tok, rounds = 1, 0
    while n_tok < cfg.gen_len and rounds < 12:
        r = o.round(cfg.gen_len - n_tok)
        n_tok += len(r.emitted)
        rounds += 1
        n = r.n_accept
        verified = r.shadow[L - 1]
        hist_u.append(float(n + 1))
        for l in range(L):
            m = r.shadow[l][:n + 1] == verified[:n + 1]
            hist_c[l].append(float(m.sum()))
            hist_t[l].append(float(r.conf[l][:n + 1][m].sum()))
            hist_f[l].append(float(r.conf[l][:n + 1][~m].sum()))
        Stcs, Sfcs, tau = o.get_conf_stats()
        Sc, Sn, E, g = o.get_stats()
        Su = _decayed(hist_u, cfg.omega)
        assert Sn == pytest.approx(Su, rel=1e-12)
        for l in range(L):
            St, Sf, Scl = _decayed(hist_t[l], cfg.omega), _decayed(hist_f[l], cfg.omega), _decayed(hist_c[l], cfg.omega)
            assert Stcs[l] == pytest.approx(St, rel=1e-11, abs=1e-13)
            assert Sfcs[l] == pytest.approx(Sf, rel=1e-11, abs=1e-13)
            mean_t = St / Scl if Scl > 0 else 1.0
            mean_f = Sf / (Su - Scl) if Su - Scl > 1e-12 else 0.0
            assert tau[l] == pytest.approx(0.5 * (mean_t + mean_f), rel=1e-9)
        assert r.next_tau == tau[E - 1]
    assert rounds >= 3
    o.close()


def _greedy_stream(cfg, w, prompt, n):
    o = oracle.OracleSeq(cfg, w)
    o.set_policy(cfg.e_min, 0)
    out, _, _ = o.generate(prompt, n)
    o.close()
    return out


def test_stream_equals_autoregressive_and_break_rule(case):
    cfg, w, prompt = case
    want = _greedy_stream(cfg, w, prompt, cfg.gen_len)
    o = oracle.OracleSeq(cfg, w)
    o.set_exit_mode(True)
    out, init, rounds = o.generate(prompt, cfg.gen_len)
    assert out == want
    stops = 0
    for r in rounds:
        kept, stopped = r.draft_conf[:r.g], r.stopped
        assert all(c >= r.tau for c in kept)
        if stopped:
            assert r.draft_conf[r.g] < r.tau and len(r.draft_conf) == r.g + 1
            stops += 1
        else:
            assert len(r.draft_conf) == r.g
        assert r.n_accept <= r.g <= cfg.g_max
    print(f"{cfg.name}: {len(rounds)} rounds, {stops} ended on a low confidence, mean g "
          f"{np.mean([r.g for r in rounds]):.2f}")
    o.close()


def test_threshold_limits(case):
    cfg, w, prompt = case
    L = cfg.n_layers
    # thresholds far above 1: every round stops before its first draft -> one token per round
    o = oracle.OracleSeq(cfg, w)
    o.set_exit_mode(True)
    tok, _ = o.prefill(prompt)
    o.set_conf_stats(np.full(L, 1e9), np.full(L, 1e9))
    want = _greedy_stream(cfg, w, prompt, 9)
    got = [tok]
    for _ in range(8):
        r = o.round(cfg.gen_len - len(got))
        assert (r.g, r.stopped, r.n_accept, len(r.emitted)) == (0, True, 0, 1)
        assert r.tau > 1.0
        got.extend(r.emitted)
    assert got == want
    o.close()
    # thresholds of 0: never stop, g_max drafts in the first round
    o = oracle.OracleSeq(cfg, w)
    o.set_exit_mode(True)
    o.prefill(prompt)
    o.set_conf_stats(np.zeros(L), np.zeros(L))
    Sc, Sn, E, g = o.get_stats()
    o.set_stats(np.maximum(Sc, 1e-3), Sn, E, g)        # every layer has matched tokens: tau = 0 exactly
    r = o.round(cfg.gen_len - 1)
    assert r.tau == 0.0 and not r.stopped and r.g == min(cfg.g_max, cfg.gen_len - 2)
    o.close()


def test_exit_mode_off_is_the_fixed_gamma_round(case):
    """Mode 0 drafts exactly gamma tokens whatever the confidences are."""
    cfg, w, prompt = case
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    o.set_conf_stats(np.full(cfg.n_layers, 1e9), np.full(cfg.n_layers, 1e9))
    Sc, Sn, E, g = o.get_stats()
    r = o.round(cfg.gen_len - 1)
    assert r.g == g and not r.stopped
    o.close()


# ---------------------------------------------------------------- baseline policies on the same round (Sec. 5.1)
def test_fs_controller_rule():
    # +1 after a round whose drafts were all accepted, -1 after a rejection, inside [max(1, g_min), g_max]
    assert oracle.fs_next_gamma(4, 4, 4, 1, 12) == 5
    assert oracle.fs_next_gamma(4, 4, 3, 1, 12) == 3
    assert oracle.fs_next_gamma(4, 4, 0, 1, 12) == 3
    assert oracle.fs_next_gamma(12, 12, 12, 1, 12) == 12
    assert oracle.fs_next_gamma(1, 1, 0, 0, 12) == 1          # never down to 0: nothing could be accepted again
    assert oracle.fs_next_gamma(2, 2, 1, 2, 12) == 2
    assert oracle.fs_next_gamma(6, 3, 3, 1, 12) == 7          # clipped round (g < gamma), all accepted
    assert oracle.fs_next_gamma(6, 0, 0, 1, 12) == 6          # no drafts: unchanged


def test_fs_policy_stream_and_trajectory(case):
    cfg, w, prompt = case
    want = _greedy_stream(cfg, w, prompt, cfg.gen_len)
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    E, g0 = cfg.e_min, 3
    o.set_policy_fs(E, g0)
    out, gamma = want[:1], g0
    while len(out) < cfg.gen_len:
        r = o.round(cfg.gen_len - len(out))
        assert (r.E, r.gamma) == (E, gamma)
        gamma = oracle.fs_next_gamma(gamma, r.g, r.n_accept, cfg.g_min, cfg.g_max)
        assert (r.next_E, r.next_gamma) == (E, gamma)
        out.extend(r.emitted)
    assert out == want
    o.close()
