"""Round-by-round comparison of the CUDA library with the oracle under speculative sampling (Sec. 2).

Both sides run freely from the same state with the same counter-based uniform numbers.  What is compared:

  * the logits rows the sampling decisions are taken from (exit head per draft, target per row): element-wise
    within EPS_LOGIT; the largest difference seen in a round, eps, sets that round's decision bands;
  * every decision (drafted token, accept / reject, last token): identical, or inside the band that logits eps
    apart allow: each filtered probability then differs by at most a factor exp(4 eps / T) (numerator,
    normaliser and nucleus mass), so a cumulative probability moves by at most delta = exp(4 eps / T) - 1 and
    an acceptance ratio by twice that (relative); tokens at the very end of a nucleus may be kept on one side only,
    which moves the cumulative probabilities behind them by their filtered mass on top of delta.  A decision inside its band is a tolerated flip: it is
    counted and the library is put back into the oracle's state (re-prefill on the oracle's tokens);
  * the filtered probabilities q(x), p(x) the library reports: relative tolerance delta; a token at the very end
    of a nucleus (mass ahead of it within delta of top_p) may be inside on one side and outside on the other: its
    probability and the decisions that depend on it are then a tolerated flip as well;
  * shadow tokens (margin rule), match counts, decayed statistics, the next (E, gamma): as in the greedy
    comparison, bit for bit once the integers agree.

The exact behaviour of the sampling kernels on given rows is pinned separately (same rows on both sides).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np

from parity import CONF_RTOL, EPS_LOGIT, MARGIN


@dataclass
class SReport:
    rounds: int = 0
    drafts: int = 0
    tests: int = 0
    rejections: int = 0
    flips: int = 0
    resyncs: int = 0
    eps_max: float = 0.0
    prob_max_rel: float = 0.0
    failures: List[str] = field(default_factory=list)

    def ok(self) -> bool:
        return not self.failures


def _cdf_interval(probs, x):
    c = np.cumsum(probs)
    return c[x] - probs[x], c[x]


def _edge_mass(logits, T, top_p, delta) -> float:
    """Filtered mass of the tokens that may be inside the nucleus on one side and outside on the other (mass
    ahead of them within delta of top_p): a cumulative probability behind them can move by that much on top of delta."""
    import oracle
    if top_p >= 1.0:
        return 0.0
    full = oracle.nucleus(logits, T, 1.0)
    order = np.argsort(-full, kind="stable")
    ahead = np.concatenate([[0.0], np.cumsum(full[order])[:-1]])
    unsure = np.abs(ahead - top_p) <= delta + full[order]
    return float(full[order][unsure].sum() / top_p)


def _at_nucleus_edge(logits, x, T, top_p, delta) -> bool:
    """True when token x sits where the nucleus ends: the mass ahead of it in the descending order is within delta
    of top_p, so that logits inside their tolerance put it inside on one side and outside on the other (its
    filtered probability then jumps between 0 and a positive value)."""
    import oracle
    if top_p >= 1.0:
        return False
    full = oracle.nucleus(logits, T, 1.0)
    ahead = float(full[(full > full[x]) | ((full == full[x]) & (np.arange(full.size) < x))].sum())
    return abs(ahead - top_p) <= delta + float(full[x])


class SeqSampler:
    """One sequence of a context followed round by round: the oracle runs beside the library, every round is
    compared, and after a tolerated difference the library is put back into the oracle's state.  Several of
    these (and greedy sequences) can share the context's rounds."""

    def __init__(self, ctx, seq, cfg, weights, prompt, temperature, top_p, seed, exit_mode=False, policy=None, layers=None):
        import oracle
        self.layers = list(range(cfg.n_layers)) if layers is None else list(layers)
        self.ctx, self.seq, self.cfg, self.prompt = ctx, seq, cfg, prompt
        self.T, self.top_p, self.seed, self.exit_mode, self.policy = temperature, top_p, seed, exit_mode, policy
        self.total = cfg.gen_len
        self.rep = SReport()
        self.o = oracle.OracleSeq(cfg, weights)
        self.o.set_sampling(temperature, top_p, seed)
        self.o.set_exit_mode(exit_mode)
        tok, _ = self.o.prefill(prompt)
        if policy:
            self.o.set_policy(*policy)
        self.tokens = [tok]

    def sync_library(self):
        """Library into the oracle's present state."""
        ctx, seq, o = self.ctx, self.seq, self.o
        ctx.set_sampling(seq, self.T, self.top_p, self.seed)
        ctx.prefill(seq, list(self.prompt) + self.tokens[:-1], self.total - len(self.tokens) + 1)
        ctx.force_token(seq, self.tokens[-1])
        Sc, Sn, E, g = o.get_stats()
        Stcs, Sfcs, _ = o.get_conf_stats()
        ctx.set_conf_stats(seq, Stcs, Sfcs)
        ctx.set_stats(seq, Sc, Sn, E, g)
        if self.policy:
            ctx.set_policy(seq, *self.policy)
        ctx.set_exit_mode(seq, self.exit_mode)

    def begin(self):
        """Prefill: the first token is drawn from the target's row of the last prompt position."""
        import oracle
        ctx, seq, o, rep = self.ctx, self.seq, self.o, self.rep
        ctx.set_sampling(seq, self.T, self.top_p, self.seed)
        first = ctx.prefill(seq, self.prompt, self.total)
        lg_lib, lg_or = ctx.get_round_logits(seq, 1, 0), o.round_logits(1, 0)
        eps = float(np.abs(lg_lib - lg_or).max())
        rep.eps_max = max(rep.eps_max, eps)
        if eps > EPS_LOGIT:
            rep.failures.append(f"prefill: target logits differ by {eps:.4f}")
        if first.tokens[0] != self.tokens[0]:
            delta = float(np.exp(4 * eps / self.T) - 1.0) + 1e-6
            delta += _edge_mass(lg_or, self.T, self.top_p, delta)
            lo, hi = _cdf_interval(oracle.nucleus(lg_or, self.T, self.top_p), first.tokens[0])
            u = oracle.uniform(self.seed, len(self.prompt), 2)
            if not (lo - delta <= u <= hi + delta):
                rep.failures.append(f"prefill: first token {first.tokens[0]} vs {self.tokens[0]}, u {u:.6f} outside "
                                    f"[{lo:.6f}, {hi:.6f}]")
            rep.flips += 1
        # (the statistics of the window do not depend on the drawn token; put the library on the oracle's state anyway)
        self.sync_library()

    @property
    def done(self) -> bool:
        return len(self.tokens) >= self.total or len(self.rep.failures) > 10

    def after_round(self, out):
        """`out`: this sequence's result of the context's latest round."""
        o, rep = self.o, self.rep
        T0 = o.T
        r = o.round(self.total - len(self.tokens))
        si = o.sample_info()
        rep.rounds += 1
        self.tokens.extend(r.emitted)
        flip = _compare(self.ctx, self.seq, o, r, si, out, T0, self.T, self.top_p, self.seed, self.layers, rep)
        if flip:
            rep.flips += 1
        if (flip or rep.failures) and len(self.tokens) < self.total:
            rep.resyncs += 1
            self.sync_library()

    def close(self):
        self.o.close()


def run_sequence_sampling(ctx, seq, cfg, weights, prompt, temperature, top_p, seed, exit_mode=False, policy=None,
                          max_rounds=None, layers=None) -> SReport:
    s = SeqSampler(ctx, seq, cfg, weights, prompt, temperature, top_p, seed, exit_mode, policy, layers)
    s.begin()
    while not s.done:
        if max_rounds is not None and s.rep.rounds >= max_rounds:
            break
        s.after_round(ctx.round()[seq])
    s.close()
    return s.rep


def _compare(ctx, seq, o, r, si, out, T0, T, top_p, seed, layers, rep: SReport) -> bool:
    """Returns True when a tolerated difference makes the rest of the round incomparable."""
    import oracle
    what = f"round {rep.rounds}"
    if (out.E, out.gamma) != (r.E, r.gamma):
        rep.failures.append(f"{what}: ran with (E,gamma) {(out.E, out.gamma)}, oracle {(r.E, r.gamma)}")
        return True
    drafts = ctx.get_drafts(seq)
    n_tests_lib, from_res_lib, qx_lib, px_lib = ctx.get_sample_info(seq)
    eps = 0.0
    rows = min(out.g + int(out.stopped), r.g + int(r.stopped))
    for i in range(rows):
        d = float(np.abs(ctx.get_round_logits(seq, 0, i) - o.round_logits(0, i)).max())
        eps = max(eps, d)
        if d > EPS_LOGIT:
            rep.failures.append(f"{what}: exit-head logits of draft {i} differ by {d:.4f}")
            return True
        if i >= min(out.g, r.g):
            break                   # the dropped token of a stopped loop: its row exists, no token was drawn
        delta = float(np.exp(4 * eps / T) - 1.0) + 1e-6
        rep.drafts += 1
        if drafts[i] != r.drafts[i]:
            qq = oracle.nucleus(o.round_logits(0, i), T, top_p)
            lo, hi = _cdf_interval(qq, drafts[i])
            band = delta + _edge_mass(o.round_logits(0, i), T, top_p, delta)
            if not (lo - band <= si.u_draft[i] <= hi + band):
                rep.failures.append(f"{what}: draft {i} gpu {drafts[i]} oracle {r.drafts[i]}, u {si.u_draft[i]:.6f} "
                                    f"outside [{lo:.6f}, {hi:.6f}] +- {delta:.2e}")
            return True
        rel = abs(float(qx_lib[i]) - si.q_x[i]) / si.q_x[i]
        rep.prob_max_rel = max(rep.prob_max_rel, rel)
        if rel > delta:
            rep.failures.append(f"{what}: q(x) of draft {i} gpu {qx_lib[i]:.6e} oracle {si.q_x[i]:.6e}")
    rep.eps_max = max(rep.eps_max, eps)
    if (out.g, bool(out.stopped)) != (r.g, bool(r.stopped)):
        # the confidence break fell the other way: allowed only inside the confidence band
        k = min(out.g, r.g)
        dc = r.draft_conf[k] if k < len(r.draft_conf) else None
        if dc is None or abs(dc - r.tau) > CONF_RTOL * (dc + r.tau):
            rep.failures.append(f"{what}: loop ended at g={out.g} stopped={bool(out.stopped)}, oracle g={r.g} "
                                f"stopped={r.stopped}")
        return True
    for i in range(r.g + 1):
        d = float(np.abs(ctx.get_round_logits(seq, 1, i) - o.round_logits(1, i)).max())
        eps = max(eps, d)
        if d > EPS_LOGIT:
            rep.failures.append(f"{what}: target logits of row {i} differ by {d:.4f}")
            return True
    rep.eps_max = max(rep.eps_max, eps)
    delta = float(np.exp(4 * eps / T) - 1.0) + 1e-6
    # acceptance tests in order
    for i in range(min(n_tests_lib, si.n_tests)):
        rep.tests += 1
        if (float(px_lib[i]) > 0) != (si.p_x[i] > 0) and _at_nucleus_edge(o.round_logits(1, i), r.drafts[i], T, top_p, delta):
            return True                 # the draft sits at the end of the target's nucleus: inside on one side only
        if si.p_x[i] > 0:
            rel = abs(float(px_lib[i]) - si.p_x[i]) / si.p_x[i]
            rep.prob_max_rel = max(rep.prob_max_rel, rel)
            if rel > delta:
                rep.failures.append(f"{what}: p(x) of draft {i} gpu {px_lib[i]:.6e} oracle {si.p_x[i]:.6e}")
        elif float(px_lib[i]) > 0:
            rep.failures.append(f"{what}: p(x) of draft {i} gpu {px_lib[i]:.6e}, outside the oracle's nucleus")
        acc_or, acc_lib = i < r.n_accept, i < out.n_accept
        if acc_or != acc_lib:
            ratio = min(1.0, si.p_x[i] / si.q_x[i])
            if abs(si.u_accept[i] - ratio) > 2 * delta * ratio + 1e-6:
                rep.failures.append(f"{what}: test {i} gpu {'accept' if acc_lib else 'reject'}, oracle u "
                                    f"{si.u_accept[i]:.6f} vs ratio {ratio:.6f}")
            return True
    rep.rejections += int(si.from_residual)
    if out.n_accept != r.n_accept or from_res_lib != bool(si.from_residual):
        rep.failures.append(f"{what}: accepted {out.n_accept} (residual {from_res_lib}), oracle {r.n_accept} "
                            f"({bool(si.from_residual)})")
        return True
    n = r.n_accept
    if out.emitted()[:n] != r.emitted[:n]:
        rep.failures.append(f"{what}: emitted {out.emitted()} oracle {r.emitted}")
        return True
    if out.emitted()[n] != r.emitted[n]:
        x = out.emitted()[n]
        pp = oracle.nucleus(o.round_logits(1, n), T, top_p)
        if si.from_residual:
            # a difference of two nearly equal probabilities: its support is all that the bands still fix
            qq = oracle.nucleus(o.round_logits(0, n), T, top_p)
            edge = _at_nucleus_edge(o.round_logits(1, n), x, T, top_p, delta) or \
                _at_nucleus_edge(o.round_logits(0, n), x, T, top_p, delta)
            if not edge and not pp[x] * (1 + delta) > qq[x] * (1 - delta):
                rep.failures.append(f"{what}: last token {x} has no residual mass within the band")
        else:
            lo, hi = _cdf_interval(pp, x)
            band = delta + _edge_mass(o.round_logits(1, n), T, top_p, delta)
            if not (lo - band <= si.u_final <= hi + band):
                rep.failures.append(f"{what}: last token {x} oracle {r.emitted[n]}, u {si.u_final:.6f} outside "
                                    f"[{lo:.6f}, {hi:.6f}]")
        return True
    # integers agree: shadow tokens by the margin rule, then counts and statistics bit for bit
    sh, counts = ctx.get_shadow(seq)
    low = False
    for l in layers:
        for i in range(r.g + 1):
            if sh[l, i] != r.shadow[l, i]:
                if r.margin[l, i] > MARGIN:
                    rep.failures.append(f"{what}: shadow l={l + 1} i={i} gpu {sh[l, i]} oracle {r.shadow[l, i]} margin "
                                        f"{r.margin[l, i]:.3f}")
                low = True
    if low:
        return True
    Sc, Sn, E, g = ctx.get_stats(seq)
    Sc_or, Sn_or, _, _ = o.get_stats()
    if not np.array_equal(counts[layers], r.counts[layers]):
        rep.failures.append(f"{what}: counts {counts.tolist()} oracle {r.counts.tolist()}")
    if not (np.array_equal(Sc[layers], Sc_or[layers]) and Sn == Sn_or):
        rep.failures.append(f"{what}: statistics differ (Sn {Sn!r} vs {Sn_or!r})")
    if (out.next_E, out.next_gamma) != (r.next_E, r.next_gamma):
        rep.failures.append(f"{what}: next (E,gamma) {(out.next_E, out.next_gamma)} oracle {(r.next_E, r.next_gamma)}")
    return False
