"""Pins for the oracle's stateless building blocks: closed forms, the paper's printed values,
brute force.  CPU only."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_pins.txt")


def paper_pins():
    pins = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split("=")
            pins[k.strip()] = float(v)
    return pins


def bf16(x):
    """float -> bf16 bit pattern (round to nearest even), independent of the generator."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def test_rmsnorm_hand_values():
    # x = (3, 4): mean square 12.5
    one = bf16([1.0, 1.0])
    out = oracle.rmsnorm(np.array([3.0, 4.0], np.float32), one, 0.0)
    assert np.allclose(out, np.array([3.0, 4.0]) / math.sqrt(12.5), rtol=1e-7)
    # eps enters under the root; gains multiply element-wise
    out = oracle.rmsnorm(np.array([3.0, 4.0], np.float32), bf16([2.0, 0.5]), 3.5)
    assert np.allclose(out, np.array([6.0, 2.0]) / 4.0, rtol=1e-7)
    # scale invariance when eps = 0
    x = np.linspace(-2, 3, 64).astype(np.float32)
    g = bf16(np.ones(64))
    assert np.allclose(oracle.rmsnorm(x, g, 0.0), oracle.rmsnorm(8 * x, g, 0.0), rtol=1e-6)
    assert abs(np.mean(oracle.rmsnorm(x, g, 0.0).astype(np.float64) ** 2) - 1.0) < 1e-6


def test_softmax_closed_form():
    p = oracle.softmax(np.log(np.array([1.0, 2.0, 3.0])).astype(np.float32))
    assert np.allclose(p, [1 / 6, 2 / 6, 3 / 6], atol=1e-7)
    # shift invariance and no overflow
    q = oracle.softmax((np.log(np.array([1.0, 2.0, 3.0])) + 1000.0).astype(np.float32))
    assert np.allclose(q, p, atol=1e-4) and abs(q.sum() - 1) < 1e-12


def test_silu_identities():
    assert oracle.silu(0.0) == 0.0
    for x in (0.3, 1.7, 5.0):
        assert abs(oracle.silu(x) - oracle.silu(-x) - x) < 1e-6          # x*s(x) + x*s(-x) = x
        assert abs(oracle.silu(x) - x / (1 + math.exp(-x))) < 1e-6
    assert abs(oracle.silu(30.0) - 30.0) < 1e-5 and abs(oracle.silu(-30.0)) < 1e-5


def test_rope_rotation():
    # head_dim 2: one pair, frequency 1 -> rotation by `pos` radians
    for pos in (0, 1, 5):
        y = oracle.rope(np.array([1.0, 0.0], np.float32), 1, 2, pos, 10000.0)
        assert np.allclose(y, [math.cos(pos), math.sin(pos)], atol=1e-6)
    # head_dim 4, theta 1e4: pair j=1 turns at 1e4^(-1/2) = 0.01 rad per position; pairs are (0,2),(1,3)
    y = oracle.rope(np.array([0.0, 1.0, 0.0, 0.0], np.float32), 1, 4, 50, 10000.0)
    assert np.allclose(y, [0.0, math.cos(0.5), 0.0, math.sin(0.5)], atol=1e-6)
    rng = np.random.default_rng(0)
    q, k = rng.standard_normal(64).astype(np.float32), rng.standard_normal(64).astype(np.float32)
    # norm preserved per head; the score depends on the position difference only
    assert np.allclose(np.linalg.norm(oracle.rope(q, 1, 64, 9, 1e4)), np.linalg.norm(q), rtol=1e-6)
    s1 = oracle.rope(q, 1, 64, 9, 1e4) @ oracle.rope(k, 1, 64, 4, 1e4)
    s2 = oracle.rope(q, 1, 64, 25, 1e4) @ oracle.rope(k, 1, 64, 20, 1e4)
    assert abs(s1 - s2) < 1e-4
    # heads are rotated independently
    two = oracle.rope(np.concatenate([q, k]), 2, 64, 7, 1e4)
    assert np.array_equal(two[:64], oracle.rope(q, 1, 64, 7, 1e4))
    assert np.array_equal(two[64:], oracle.rope(k, 1, 64, 7, 1e4))


def test_accept_worked_example_from_paper():
    pins = paper_pins()
    drafted, accepted = int(pins["fig2.drafted"]), int(pins["fig2.accepted"])
    drafts = [11, 12, 13, 99]                 # 4 drafts, the 4th differs from the target's token
    verified = [11, 12, 13, 14, 15]           # target's greedy tokens at the 5 positions
    n = oracle.accept_len(drafts, verified)
    assert len(drafts) == drafted and n == accepted
    emitted = verified[:n + 1]
    assert len(emitted) == int(pins["fig2.emitted"]) and emitted[-1] == 14   # bonus token replaces the reject


def test_accept_edge_cases():
    assert oracle.accept_len([], [5]) == 0                       # gamma = 0: plain auto-regressive step
    assert oracle.accept_len([1, 2, 3], [1, 2, 3, 4]) == 3       # all accepted -> gamma + 1 tokens
    assert oracle.accept_len([9, 2, 3], [1, 2, 3, 4]) == 0       # first rejected -> 1 token
    assert oracle.accept_len([1, 9, 3], [1, 2, 3, 4]) == 1       # later matches after a mismatch do not count


def test_decayed_sum_definition_and_half_life():
    pins = paper_pins()
    omega = pins["decay.omega"]
    rng = np.random.default_rng(1)
    a = rng.integers(0, 14, size=40).astype(np.float64)
    S = 0.0
    for r, x in enumerate(a, start=1):
        S = oracle.decay_step(S, omega, x)
        direct = sum(omega ** (r - i - 1) * a[i] for i in range(r))      # S(a) as defined in Sec. 4.2
        assert abs(S - direct) <= 1e-12 * max(1.0, abs(direct))
    # newest entry has weight 1; an entry 13 rounds back weighs about one half
    S = oracle.decay_step(0.0, omega, 1.0)
    for _ in range(int(pins["decay.half_life_rounds"])):
        S = oracle.decay_step(S, omega, 0.0)
    assert abs(S - omega ** 13) < 1e-15 and abs(S - pins["decay.half_life_weight"]) < 0.02
    # omega = 1: plain sums (alpha is a plain ratio); omega = 0: last round only
    S1 = S0 = 0.0
    for x in a:
        S1, S0 = oracle.decay_step(S1, 1.0, x), oracle.decay_step(S0, 0.0, x)
    assert S1 == a.sum() and S0 == a[-1]


def closed_form_tpl(alpha, l, d, L):
    return (1 - alpha ** (d + 1)) / ((1 - alpha) * (d * l + L))        # Eq. 1 as printed


def test_tpl_sum_form_equals_eq1():
    for alpha, l, d, L in itertools.product((0.05, 0.3, 0.77, 0.999), (1, 4, 17), (0, 1, 6, 18), (16, 32)):
        assert abs(oracle.tpl(alpha, l, d, L) - closed_form_tpl(alpha, l, d, L)) <= 1e-12
    for L in (16, 32, 40):
        for l in (1, 7):
            assert oracle.tpl(0.6, l, 0, L) == 1.0 / L             # no drafts: one token per L layers
    assert oracle.tpl(1.0, 3, 5, 32) == 6.0 / (15 + 32)            # alpha = 1: the sum form has no 0/0
    assert oracle.tpl(0.0, 3, 5, 32) == 1.0 / (15 + 32)


def brute_select(alpha, L, e_min, e_max, g_min, g_max):
    best, arg = -1.0, None
    for l in range(e_min, e_max + 1):
        for d in range(g_min, g_max + 1):
            a = alpha[l - 1]
            t = (d + 1) / (d * l + L) if a == 1.0 else closed_form_tpl(a, l, d, L)
            if t > best * (1 + 1e-13):
                best, arg = t, (l, d)
    return arg, best


def test_select_matches_exhaustive_search():
    rng = np.random.default_rng(2)
    for trial in range(200):
        L = int(rng.choice([4, 16, 32, 40]))
        e_min, e_max = 1, L - 1
        g_min, g_max = (0, 18) if trial % 2 else (1, 12)
        alpha = np.sort(rng.uniform(0.05, 0.98, size=L))
        Sn = float(rng.uniform(5, 60))
        E, g = oracle.select(alpha * Sn, Sn, L, e_min, e_max, g_min, g_max)
        (bE, bg), best = brute_select(alpha * Sn / Sn, L, e_min, e_max, g_min, g_max)
        got = closed_form_tpl(alpha[E - 1] * Sn / Sn, E, g, L)
        assert abs(got - best) <= 1e-12 * best, (trial, (E, g), (bE, bg))


def test_select_special_cases():
    L = 32
    Sn = 10.0
    # nothing ever matches: drafting is pure cost -> cheapest allowed setting
    assert oracle.select(np.zeros(L), Sn, L, 4, 28, 1, 12) == (4, 1)
    # everything always matches: shallowest exit, longest speculation
    assert oracle.select(np.full(L, Sn), Sn, L, 4, 28, 1, 12) == (4, 12)
    # ties resolve to the lowest layer, then the lowest length (gamma = 0 allowed: TPL = 1/L for all l)
    assert oracle.select(np.zeros(L), Sn, L, 1, 31, 0, 0) == (1, 0)
    # a layer that agrees much more often wins although it is deeper
    Sc = np.full(L, 0.2 * Sn)
    Sc[9:] = 0.95 * Sn
    E, g = oracle.select(Sc, Sn, L, 4, 28, 1, 12)
    assert E == 10 and g > 3


def test_vanilla_etpl_values_from_paper_tables():
    pins = paper_pins()
    for L in (16, 32, 40, 80, 48):
        assert round(oracle.tpl(0.5, 1, 0, L) + 1e-12, 3) == pins[f"etpl.vanilla.L{L}"]


def test_generator_reproducible_and_distribution():
    cfg = synth.CONFIGS["tiny"]
    a = synth.make_layer(cfg, 1)["wq"]
    b = synth.make_layer(cfg, 1)["wq"]
    assert np.array_equal(a, b)
    x = synth.bf16_to_f32(a).astype(np.float64)
    assert abs(x.std() - 0.02) < 5e-4 and abs(x.mean()) < 5e-4
    assert abs(np.mean(x ** 4) / x.var() ** 2 - 3.0) < 0.1          # normal kurtosis
    wo3 = synth.bf16_to_f32(synth.make_layer(cfg, 3)["wo"]).std()
    assert abs(wo3 - 0.002) < 1e-4                                   # layers 3-4 residual branches x0.1
    p = synth.make_prompt(cfg)
    assert p.min() >= 0 and p.max() < cfg.vocab and len(p) == cfg.prompt_len
    big = synth.CONFIGS["llama2_13b"]
    q = synth.make_prompt(synth.small_variant(big, prompt_len=640))
    spans = {tuple(q[i:i + 64]) for i in range(0, 640, 64)}
    assert len(spans) < 10                                           # repeated 64-token spans
