"""Round-by-round comparison of the CUDA library with the oracle's trace.

Integer results (draft tokens, shadow tokens, accept lengths, match counts, the chosen (E, gamma)) must
be identical wherever the oracle's top-1 minus top-2 logit margin of the deciding arg-max exceeds
MARGIN.  A difference at a smaller margin is a tolerated flip: it is counted, and the library is
re-synchronised to the oracle (re-prefill on the oracle's tokens, forced next token, statistics
restored) so that later rounds stay comparable.  The acceptance statistics are doubles computed with the
same operation order on both sides, so after identical integer inputs they must agree bit for bit.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np

MARGIN = 0.05


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


@dataclass
class Report:
    rounds: int = 0
    flips: int = 0
    resyncs: int = 0
    compared: int = 0
    failures: List[str] = field(default_factory=list)

    def ok(self) -> bool:
        return not self.failures


def ref_from_oracle(cfg, weights, prompt, gen_len=None, policy=None) -> SeqRef:
    """Runs the oracle now (small models)."""
    import oracle
    o = oracle.OracleSeq(cfg, weights)
    if policy:
        o.set_policy(*policy)
    n_tok = gen_len or cfg.gen_len
    tok, init = o.prefill(prompt)
    Sc, Sn, E, g = o.get_stats()
    ref = SeqRef(np.asarray(prompt, dtype=np.int32), tok, init.shadow, init.margin, Sc, Sn, E, g, [], [tok])
    while len(ref.tokens) < n_tok:
        r = o.round(n_tok - len(ref.tokens))
        Sc, Sn, _, _ = o.get_stats()
        ref.rounds.append(RoundRef(r.E, r.gamma, r.g, r.n_accept, r.drafts, r.emitted, r.shadow, r.margin, r.counts,
                                   r.next_E, r.next_gamma, Sc, Sn))
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
    for r in s["rounds"]:
        ref.rounds.append(RoundRef(r["E"], r["gamma"], r["g"], r["n"], r["drafts"], r["emitted"],
                                   np.array(r["shadow"], dtype=np.int32).reshape(len(r["shadow"]), -1),
                                   np.array(r["margin_milli"], dtype=np.float64).reshape(len(r["shadow"]), -1) / 1000.0,
                                   np.array(r["counts"], dtype=np.int32), r["next_E"], r["next_gamma"], np.array(r["Sc"]),
                                   r["Sn"]))
    return ref


def _resync(ctx, seq, ref: SeqRef, n_done_tokens: int, Sc, Sn, E, gamma, total_tokens: int):
    """Puts the library into the oracle's state after `n_done_tokens` emitted tokens."""
    ctx_tokens = list(ref.prompt) + ref.tokens[:n_done_tokens - 1]
    ctx.prefill(seq, ctx_tokens, total_tokens - n_done_tokens + 1)
    ctx.force_token(seq, ref.tokens[n_done_tokens - 1])
    ctx.set_stats(seq, Sc, Sn, E, gamma)


def compare_init(ctx, seq, ref: SeqRef, total_tokens: int, rep: Report, policy=None) -> None:
    out = ctx.prefill(seq, ref.prompt, total_tokens)
    if policy:
        ctx.set_policy(seq, *policy)
    L, W = ref.init_shadow.shape
    # after the prefill the shadow buffer holds the window's tokens in its first W columns; only g_max+1
    # of them are exported, which is enough to pin the head of the window
    sh, _ = ctx.get_shadow(seq)
    ncol = min(W, sh.shape[1])
    flips = 0
    for l in range(L):
        for j in range(ncol):
            rep.compared += 1
            if sh[l, j] != ref.init_shadow[l, j]:
                if ref.init_margin[l, j] > MARGIN:
                    rep.failures.append(f"init shadow l={l + 1} j={j}: gpu {sh[l, j]} oracle {ref.init_shadow[l, j]} "
                                        f"margin {ref.init_margin[l, j]:.3f}")
                flips += 1
    Sc, Sn, E, g = ctx.get_stats(seq)
    same = (out.tokens[0] == ref.first_token and np.array_equal(Sc, ref.init_Sc) and Sn == ref.init_Sn
            and (policy or (E, g) == (ref.init_E, ref.init_gamma)))
    if not same:
        # the statistics sum over the whole window; any difference must come from a low-margin position
        low = (ref.init_margin <= MARGIN).any()
        if not low:
            rep.failures.append(f"init state differs without a low-margin position: token {out.tokens[0]} vs "
                                f"{ref.first_token}, (E,g) {(E, g)} vs {(ref.init_E, ref.init_gamma)}")
        flips += 1
    if flips:
        rep.flips += flips
        rep.resyncs += 1
        ctx.force_token(seq, ref.first_token)
        ctx.set_stats(seq, ref.init_Sc, ref.init_Sn, ref.init_E, ref.init_gamma)


def compare_round(ctx, seq, out, r: RoundRef, rep: Report, check_choice=True) -> bool:
    """Compares one finished round; returns True if the library must be re-synchronised."""
    L = r.shadow.shape[0]
    rep.rounds += 1
    if (out.E, out.gamma, out.g) != (r.E, r.gamma, r.g):
        rep.failures.append(f"round {rep.rounds}: ran with (E,gamma,g)={(out.E, out.gamma, out.g)}, oracle {(r.E, r.gamma, r.g)}")
        return True
    sh, counts = ctx.get_shadow(seq)
    drafts = ctx.get_drafts(seq)[:r.g]
    flips = 0
    # rows are comparable up to the first differing draft (later rows saw different inputs)
    last_row = r.g
    for i in range(r.g):
        if drafts[i] != r.drafts[i]:
            if r.margin[r.E - 1, i] > MARGIN:
                rep.failures.append(f"round {rep.rounds}: draft {i} gpu {drafts[i]} oracle {r.drafts[i]} margin "
                                    f"{r.margin[r.E - 1, i]:.3f}")
            flips += 1
            last_row = i
            break
    for l in range(L):
        for i in range(last_row + 1):
            rep.compared += 1
            if sh[l, i] != r.shadow[l, i]:
                if r.margin[l, i] > MARGIN:
                    rep.failures.append(f"round {rep.rounds}: shadow l={l + 1} i={i} gpu {sh[l, i]} oracle {r.shadow[l, i]} "
                                        f"margin {r.margin[l, i]:.3f}")
                flips += 1
    if flips == 0:
        Sc, Sn, E, g = ctx.get_stats(seq)
        if out.n_accept != r.n or out.emitted() != list(r.emitted):
            rep.failures.append(f"round {rep.rounds}: accept {out.n_accept}/{out.emitted()} oracle {r.n}/{r.emitted}")
        if not np.array_equal(counts, r.counts):
            rep.failures.append(f"round {rep.rounds}: counts {counts.tolist()} oracle {r.counts.tolist()}")
        if not (np.array_equal(Sc, r.Sc) and Sn == r.Sn):
            rep.failures.append(f"round {rep.rounds}: statistics differ (Sn {Sn!r} vs {r.Sn!r})")
        if check_choice and (out.next_E, out.next_gamma) != (r.next_E, r.next_gamma):
            rep.failures.append(f"round {rep.rounds}: next (E,gamma) {(out.next_E, out.next_gamma)} oracle "
                                f"{(r.next_E, r.next_gamma)}")
        return False
    rep.flips += flips
    return True


def run_sequence(ctx, seq, ref: SeqRef, total_tokens: int, policy=None, max_rounds=None) -> Report:
    """Prefill + rounds of one sequence through del_round, compared with the oracle's trace."""
    rep = Report()
    compare_init(ctx, seq, ref, total_tokens, rep, policy)
    done = 1
    for k, r in enumerate(ref.rounds):
        if max_rounds is not None and k >= max_rounds:
            break
        outs = ctx.round()
        need = compare_round(ctx, seq, outs[seq], r, rep, check_choice=policy is None)
        done += r.n + 1
        if need and k + 1 < len(ref.rounds):
            rep.resyncs += 1
            _resync(ctx, seq, ref, done, r.Sc, r.Sn, r.next_E, r.next_gamma, total_tokens)
            if policy:
                ctx.set_policy(seq, *policy)
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
                _resync(ctx, s, refs[s], done[s], r.Sc, r.Sn, r.next_E, r.next_gamma, total_tokens)
        if sum(len(rp.failures) for rp in reps) > 20:
            break
    return reps
