"""Round-by-round comparison of the CUDA library with the oracle's trace.

Integer results (draft tokens, shadow tokens, accept lengths, match counts, the chosen (E, gamma)) must
be identical wherever the oracle's top-1 minus top-2 logit margin of the deciding arg-max exceeds
MARGIN.  A difference at a smaller margin is a tolerated flip: it is counted, and the library is
re-synchronised to the oracle (re-prefill on the oracle's tokens, forced next token, statistics
restored) so that later rounds stay comparable.  The acceptance statistics are doubles computed with the
same operation order on both sides, so after identical integer inputs they must agree bit for bit.

Confidence scores (top-1 softmax probabilities) are floating point on both sides: fp32 from bf16
activations in the library, fp64 in the oracle.  With logits within EPS_LOGIT of each other the sum of
exponentials changes by at most a factor exp(2 * EPS_LOGIT), so confidences, their decayed sums and the
thresholds are compared with the relative tolerance CONF_RTOL = exp(2 * EPS_LOGIT) - 1.  The draft
loop's decision "confidence < threshold" must be the same wherever the oracle's two numbers are further
apart than that tolerance allows; a decision inside the band is a tolerated flip (counted, re-synchronised).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

MARGIN = 0.05
EPS_LOGIT = 3e-2
CONF_RTOL = float(np.exp(2 * EPS_LOGIT) - 1.0)


@dataclass
class RoundRef:
    E: int
    gamma: int
    g: int
    n: int
    drafts: List[int]
    emitted: List[int]
    shadow: np.ndarray          # [L][g+1]
    margin: np.ndarray          # [L][g+1] float
    counts: np.ndarray          # [L]
    next_E: int
    next_gamma: int
    Sc: np.ndarray
    Sn: float
    # dynamic draft-exiting (None / defaults when the reference trace does not carry them)
    conf: Optional[np.ndarray] = None       # [L][g+1] confidence of the shadow tokens
    draft_conf: Optional[List[float]] = None  # confidence of each drafted token, the dropped one included
    stopped: bool = False
    tau: float = 0.0
    next_tau: float = 0.0
    Stcs: Optional[np.ndarray] = None
    Sfcs: Optional[np.ndarray] = None


@dataclass
class SeqRef:
    prompt: np.ndarray
    first_token: int
    init_shadow: np.ndarray     # [L][W]
    init_margin: np.ndarray
    init_Sc: np.ndarray
    init_Sn: float
    init_E: int
    init_gamma: int
    rounds: List[RoundRef]
    tokens: List[int]
    init_conf: Optional[np.ndarray] = None
    init_Stcs: Optional[np.ndarray] = None
    init_Sfcs: Optional[np.ndarray] = None
    init_tau: float = 0.0
    exit_mode: bool = False


@dataclass
class Report:
    rounds: int = 0
    flips: int = 0
    resyncs: int = 0
    compared: int = 0
    conf_compared: int = 0
    conf_max_rel: float = 0.0
    decisions: int = 0
    decision_flips: int = 0
    max_flip_margin: float = 0.0            # largest oracle margin among the arg-max results that differ
    failures: List[str] = field(default_factory=list)

    def ok(self) -> bool:
        return not self.failures


def ref_from_oracle(cfg, weights, prompt, gen_len=None, policy=None, exit_mode=False, policy_fs=None) -> SeqRef:
    """Runs the oracle now (small models)."""
    import oracle
    o = oracle.OracleSeq(cfg, weights)
    if policy:
        o.set_policy(*policy)
    o.set_exit_mode(exit_mode)
    n_tok = gen_len or cfg.gen_len
    tok, init = o.prefill(prompt)
    if policy_fs:
        o.set_policy_fs(*policy_fs)
    Sc, Sn, E, g = o.get_stats()
    Stcs, Sfcs, _ = o.get_conf_stats()
    ref = SeqRef(np.asarray(prompt, dtype=np.int32), tok, init.shadow, init.margin, Sc, Sn, E, g, [], [tok],
                 init_conf=init.conf, init_Stcs=Stcs, init_Sfcs=Sfcs, init_tau=init.next_tau, exit_mode=exit_mode)
    while len(ref.tokens) < n_tok:
        r = o.round(n_tok - len(ref.tokens))
        Sc, Sn, _, _ = o.get_stats()
        Stcs, Sfcs, _ = o.get_conf_stats()
        ref.rounds.append(RoundRef(r.E, r.gamma, r.g, r.n_accept, r.drafts, r.emitted, r.shadow, r.margin, r.counts,
                                   r.next_E, r.next_gamma, Sc, Sn, conf=r.conf, draft_conf=r.draft_conf,
                                   stopped=r.stopped, tau=r.tau, next_tau=r.next_tau, Stcs=Stcs, Sfcs=Sfcs))
        ref.tokens.extend(r.emitted)
    o.close()
    return ref


def ref_from_golden(doc, seq_index, prompt) -> SeqRef:
    """Builds the reference from a stored trace (tests/golden/trace_*.json, written by make_traces.py)."""
    s = doc["sequences"][seq_index]
    init = s["init"]
    ref = SeqRef(np.asarray(prompt, dtype=np.int32), s["first_token"], np.array(init["shadow"], dtype=np.int32),
                 np.array(init["margin_milli"], dtype=np.float64) / 1000.0, np.array(init["Sc"]), init["Sn"], init["E"],
                 init["gamma"], [], list(s["tokens"]))
    exit_mode = bool(doc.get("exit_mode", False))
    if exit_mode:
        ref.exit_mode = True
        ref.init_conf = np.array(init["conf_e7"], dtype=np.float64) / 1e7
        ref.init_Stcs, ref.init_Sfcs, ref.init_tau = np.array(init["Stcs"]), np.array(init["Sfcs"]), init["tau"]
    for r in s["rounds"]:
        rr = RoundRef(r["E"], r["gamma"], r["g"], r["n"], r["drafts"], r["emitted"],
                      np.array(r["shadow"], dtype=np.int32).reshape(len(r["shadow"]), -1),
                      np.array(r["margin_milli"], dtype=np.float64).reshape(len(r["shadow"]), -1) / 1000.0,
                      np.array(r["counts"], dtype=np.int32), r["next_E"], r["next_gamma"], np.array(r["Sc"]), r["Sn"])
        if exit_mode:
            rr.conf = np.array(r["conf_e7"], dtype=np.float64).reshape(len(r["shadow"]), -1) / 1e7
            rr.draft_conf, rr.stopped, rr.tau, rr.next_tau = list(r["draft_conf"]), bool(r["stopped"]), r["tau"], r["next_tau"]
            rr.Stcs, rr.Sfcs = np.array(r["Stcs"]), np.array(r["Sfcs"])
        ref.rounds.append(rr)
    return ref


def _resync(ctx, seq, ref: SeqRef, n_done_tokens: int, Sc, Sn, E, gamma, total_tokens: int, Stcs=None, Sfcs=None):
    """Puts the library into the oracle's state after `n_done_tokens` emitted tokens."""
    ctx_tokens = list(ref.prompt) + ref.tokens[:n_done_tokens - 1]
    ctx.prefill(seq, ctx_tokens, total_tokens - n_done_tokens + 1)
    ctx.force_token(seq, ref.tokens[n_done_tokens - 1])
    if Stcs is not None:
        ctx.set_conf_stats(seq, Stcs, Sfcs)
    ctx.set_stats(seq, Sc, Sn, E, gamma)
    if ref.exit_mode:
        ctx.set_exit_mode(seq, True)


def _compare_conf(rep: Report, what: str, got, want):
    """Element-wise relative comparison of confidence-like numbers."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    rel = np.abs(got - want) / np.maximum(np.abs(want), 1e-6)
    rel = np.where(np.abs(got - want) < 1e-6, 0.0, rel)
    rep.conf_compared += rel.size
    if rel.size:
        rep.conf_max_rel = max(rep.conf_max_rel, float(rel.max()))
        if rel.max() > CONF_RTOL:
            k = int(np.argmax(rel))
            rep.failures.append(f"{what}: element {k} gpu {got.flat[k]:.6f} oracle {want.flat[k]:.6f}")


def compare_init(ctx, seq, ref: SeqRef, total_tokens: int, rep: Report, policy=None, layers=None, check_choice=True) -> None:
    """layers: 0-based layers to compare (default all; with trimmed stacked-head rows only those are maintained)."""
    out = ctx.prefill(seq, ref.prompt, total_tokens)
    if policy:
        ctx.set_policy(seq, *policy)
    L, W = ref.init_shadow.shape
    layers = list(range(L)) if layers is None else list(layers)
    # after the prefill the shadow buffer holds the window's tokens and confidences in its first W columns
    sh, win_conf = ctx.get_window(seq, W)
    ncol = W
    flips = 0
    for l in layers:
        for j in range(ncol):
            rep.compared += 1
            if sh[l, j] != ref.init_shadow[l, j]:
                rep.max_flip_margin = max(rep.max_flip_margin, float(ref.init_margin[l, j]))
                if ref.init_margin[l, j] > MARGIN:
                    rep.failures.append(f"init shadow l={l + 1} j={j}: gpu {sh[l, j]} oracle {ref.init_shadow[l, j]} "
                                        f"margin {ref.init_margin[l, j]:.3f}")
                flips += 1
    Sc, Sn, E, g = ctx.get_stats(seq)
    if flips == 0 and ref.init_conf is not None:
        _compare_conf(rep, "init confidences", win_conf[layers, :ncol], ref.init_conf[layers, :ncol])
        Stcs, Sfcs, tau = ctx.get_conf_stats(seq)
        if ncol == W:       # the sums run over the whole window
            _compare_conf(rep, "init Stcs", Stcs[layers], ref.init_Stcs[layers])
            _compare_conf(rep, "init Sfcs", Sfcs[layers], ref.init_Sfcs[layers])
    same = (out.tokens[0] == ref.first_token and np.array_equal(Sc[layers], ref.init_Sc[layers]) and Sn == ref.init_Sn
            and (policy or not check_choice or (E, g) == (ref.init_E, ref.init_gamma)))
    if not same:
        # the statistics sum over the whole window; any difference must come from a low-margin position
        low = (ref.init_margin[layers] <= MARGIN).any()
        if not low:
            rep.failures.append(f"init state differs without a low-margin position: token {out.tokens[0]} vs "
                                f"{ref.first_token}, (E,g) {(E, g)} vs {(ref.init_E, ref.init_gamma)}")
        flips += 1
    if flips:
        rep.flips += flips
        rep.resyncs += 1
        ctx.force_token(seq, ref.first_token)
        if ref.init_Stcs is not None:
            ctx.set_conf_stats(seq, ref.init_Stcs, ref.init_Sfcs)
        ctx.set_stats(seq, ref.init_Sc, ref.init_Sn, ref.init_E, ref.init_gamma)
    if ref.exit_mode:
        ctx.set_exit_mode(seq, True)


def compare_round(ctx, seq, out, r: RoundRef, rep: Report, check_choice=True, layers=None) -> bool:
    """Compares one finished round; returns True if the library must be re-synchronised."""
    L = r.shadow.shape[0]
    layers = list(range(L)) if layers is None else list(layers)
    rep.rounds += 1
    if r.draft_conf is not None and r.tau > 0.0 and out.tau > 0.0:
        # dynamic draft-exiting: the loop's decisions, wherever the oracle's numbers are clearly apart
        _, dc = ctx.get_conf(seq)
        got_drafts = ctx.get_drafts(seq)
        n_dec = min(len(r.draft_conf), out.g + int(out.stopped))
        rep.decisions += n_dec
        _compare_conf(rep, f"round {rep.rounds}: tau", [out.tau], [r.tau])
        for i in range(n_dec):
            if i > 0 and got_drafts[i - 1] != r.drafts[i - 1]:
                # the previous draft differs (allowed at a low margin): this token saw another input, its
                # confidence is not comparable any more
                if r.margin[r.E - 1, i - 1] > MARGIN:
                    rep.failures.append(f"round {rep.rounds}: draft {i - 1} gpu {got_drafts[i - 1]} oracle {r.drafts[i - 1]} "
                                        f"margin {r.margin[r.E - 1, i - 1]:.3f}")
                rep.flips += 1
                return True
            want_stop, got_stop = r.draft_conf[i] < r.tau, float(dc[i]) < out.tau
            if want_stop != got_stop:
                band = CONF_RTOL * (r.draft_conf[i] + r.tau)
                if abs(r.draft_conf[i] - r.tau) > band:
                    rep.failures.append(f"round {rep.rounds}: draft {i} confidence {dc[i]:.5f} vs tau {out.tau:.5f}, oracle "
                                        f"{r.draft_conf[i]:.5f} vs {r.tau:.5f}")
                rep.decision_flips += 1
                rep.flips += 1
                return True
            if want_stop:
                break
    if (out.E, out.gamma, out.g) != (r.E, r.gamma, r.g) or bool(out.stopped) != bool(r.stopped):
        # a draft token that differs at a low margin changes the confidences that follow
        drafts = ctx.get_drafts(seq)
        k = next((i for i in range(min(out.g, r.g)) if drafts[i] != r.drafts[i]), None)
        if k is not None and r.margin[r.E - 1, k] <= MARGIN:
            rep.flips += 1
            return True
        rep.failures.append(f"round {rep.rounds}: ran with (E,gamma,g,stopped)={(out.E, out.gamma, out.g, bool(out.stopped))}, "
                            f"oracle {(r.E, r.gamma, r.g, bool(r.stopped))}")
        return True
    sh, counts = ctx.get_shadow(seq)
    drafts = ctx.get_drafts(seq)[:r.g]
    flips = 0
    # rows are comparable up to the first differing draft (later rows saw different inputs)
    last_row = r.g
    for i in range(r.g):
        if drafts[i] != r.drafts[i]:
            rep.max_flip_margin = max(rep.max_flip_margin, float(r.margin[r.E - 1, i]))
            if r.margin[r.E - 1, i] > MARGIN:
                rep.failures.append(f"round {rep.rounds}: draft {i} gpu {drafts[i]} oracle {r.drafts[i]} margin "
                                    f"{r.margin[r.E - 1, i]:.3f}")
            flips += 1
            last_row = i
            break
    for l in layers:
        for i in range(last_row + 1):
            rep.compared += 1
            if sh[l, i] != r.shadow[l, i]:
                rep.max_flip_margin = max(rep.max_flip_margin, float(r.margin[l, i]))
                if r.margin[l, i] > MARGIN:
                    rep.failures.append(f"round {rep.rounds}: shadow l={l + 1} i={i} gpu {sh[l, i]} oracle {r.shadow[l, i]} "
                                        f"margin {r.margin[l, i]:.3f}")
                flips += 1
    if flips == 0 and r.conf is not None:
        sc, dc = ctx.get_conf(seq)
        _compare_conf(rep, f"round {rep.rounds}: shadow confidences", sc[layers, :r.g + 1], r.conf[layers])
        if r.draft_conf:
            _compare_conf(rep, f"round {rep.rounds}: draft confidences", dc[:len(r.draft_conf)], r.draft_conf)
        Stcs, Sfcs, tau = ctx.get_conf_stats(seq)
        _compare_conf(rep, f"round {rep.rounds}: Stcs", Stcs[layers], r.Stcs[layers])
        _compare_conf(rep, f"round {rep.rounds}: Sfcs", Sfcs[layers], r.Sfcs[layers])
        _compare_conf(rep, f"round {rep.rounds}: next tau", [out.next_tau], [r.next_tau])
    if flips == 0:
        Sc, Sn, E, g = ctx.get_stats(seq)
        if out.n_accept != r.n or out.emitted() != list(r.emitted):
            rep.failures.append(f"round {rep.rounds}: accept {out.n_accept}/{out.emitted()} oracle {r.n}/{r.emitted}")
        if not np.array_equal(counts[layers], r.counts[layers]):
            rep.failures.append(f"round {rep.rounds}: counts {counts.tolist()} oracle {r.counts.tolist()}")
        if not (np.array_equal(Sc[layers], r.Sc[layers]) and Sn == r.Sn):
            rep.failures.append(f"round {rep.rounds}: statistics differ (Sn {Sn!r} vs {r.Sn!r})")
        if check_choice and (out.next_E, out.next_gamma) != (r.next_E, r.next_gamma):
            rep.failures.append(f"round {rep.rounds}: next (E,gamma) {(out.next_E, out.next_gamma)} oracle "
                                f"{(r.next_E, r.next_gamma)}")
        return False
    rep.flips += flips
    return True


def run_sequence(ctx, seq, ref: SeqRef, total_tokens: int, policy=None, max_rounds=None, policy_fs=None, layers=None) -> Report:
    """Prefill + rounds of one sequence through del_round, compared with the oracle's trace.
    policy = (E, gamma) fixes both; policy_fs = (E, gamma0) fixes E and lets the +-1 controller move gamma."""
    rep = Report()
    # (with the FS baseline the reference's first (E, gamma) is the policy's, set after the prefill: nothing to compare)
    compare_init(ctx, seq, ref, total_tokens, rep, policy, layers=layers, check_choice=policy_fs is None)
    if policy_fs:
        ctx.set_policy_fs(seq, *policy_fs)
    done = 1
    for k, r in enumerate(ref.rounds):
        if max_rounds is not None and k >= max_rounds:
            break
        outs = ctx.round()
        need = compare_round(ctx, seq, outs[seq], r, rep, check_choice=policy is None, layers=layers)
        done += r.n + 1
        if need and k + 1 < len(ref.rounds):
            rep.resyncs += 1
            _resync(ctx, seq, ref, done, r.Sc, r.Sn, r.next_E, r.next_gamma, total_tokens, r.Stcs, r.Sfcs)
            if policy:
                ctx.set_policy(seq, *policy)
            if policy_fs:
                ctx.set_policy_fs(seq, policy_fs[0], r.next_gamma)
        if len(rep.failures) > 20:
            break
    return rep


def run_batch(ctx, refs: List[SeqRef], total_tokens: int, max_rounds=None) -> List[Report]:
    """All sequences of a batch through shared del_round calls, each compared with its own oracle trace."""
    n = len(refs)
    reps = [Report() for _ in refs]
    for s in range(n):
        compare_init(ctx, s, refs[s], total_tokens, reps[s])
    done, k = [1] * n, [0] * n
    calls = 0
    while any(k[s] < len(refs[s].rounds) for s in range(n)):
        if max_rounds is not None and calls >= max_rounds:
            break
        outs = ctx.round()
        calls += 1
        for s in range(n):
            if k[s] >= len(refs[s].rounds):
                continue
            r = refs[s].rounds[k[s]]
            need = compare_round(ctx, s, outs[s], r, reps[s])
            done[s] += r.n + 1
            k[s] += 1
            if need and k[s] < len(refs[s].rounds):
                reps[s].resyncs += 1
                _resync(ctx, s, refs[s], done[s], r.Sc, r.Sn, r.next_E, r.next_gamma, total_tokens, r.Stcs, r.Sfcs)
        if sum(len(rp.failures) for rp in reps) > 20:
            break
    return reps
