"""Parity of the CUDA library (through its C ABI) with the CPU oracle.  Needs a B200."""
import json
import os

import numpy as np
import pytest

import synth
from cases import TINY, TINY_GQA, TINY_GQA_LONG, TINY_HD128, TINY_HD128_GQA, TINY_LONG, TINY_LONG2, TINY_LONG3, TINY_SHORT
from parity import MARGIN, Report, _resync, compare_init, compare_round, ref_from_golden, ref_from_oracle, run_batch, run_sequence

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_ctx(cfg, weights, **kw):
    import paper_2504_05598_b200 as dl
    dev = dl.upload_weights(weights)
    return dl.DelContext(dl.make_shape(cfg, **kw), dev)


@pytest.fixture(scope="module", params=[TINY, TINY_GQA, TINY_SHORT], ids=lambda c: c.name)
def small(request):
    cfg = request.param
    w = synth.make_weights(cfg)
    return cfg, w, make_ctx(cfg, w)


def test_prefill_hidden_kv_and_logits(small):
    """Element-wise: hidden states of every layer, cached K/V rows and exit-head logits after a prefill."""
    import oracle
    cfg, w, ctx = small
    prompt = synth.make_prompt(cfg)
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    ctx.prefill(0, prompt, cfg.gen_len)
    W = min(cfg.init_window, len(prompt))
    P = len(prompt)
    for l in range(cfg.n_layers + 1):
        for j in (0, W - 1):
            ref = o.hidden(l, j)
            got = ctx.get_hidden(0, l, j)
            scale = np.abs(ref).max()
            assert np.abs(got - ref).max() <= 2e-2 * scale + 1e-6, (l, j, np.abs(got - ref).max(), scale)
    for l in (1, cfg.n_layers):
        for pos in (0, P // 2, P - 1):
            k, v = ctx.get_kv(0, l, pos)
            kr, vr = o.k_row(l, pos), o.v_row(l, pos)
            assert np.abs(k - kr).max() <= 2e-2 * np.abs(kr).max() + 1e-6, ("k", l, pos)
            assert np.abs(v - vr).max() <= 2e-2 * np.abs(vr).max() + 1e-6, ("v", l, pos)
    # per-layer logits of the exit head: max-abs 3e-2 after bf16
    for l in (1, cfg.n_layers // 2, cfg.n_layers):
        _, _, ref = o.exit_head(o.hidden(l, W - 1), want_logits=True)
        got = ctx.debug_logits(0, l, W - 1)
        assert np.abs(got - ref).max() <= 3e-2, (l, np.abs(got - ref).max())
        if np.sort(ref)[-1] - np.sort(ref)[-2] > MARGIN:
            assert int(np.argmax(got)) == int(np.argmax(ref))


@pytest.mark.parametrize("cfg", [TINY_LONG, TINY_GQA_LONG, TINY_LONG2, TINY_LONG3, TINY_HD128, TINY_HD128_GQA], ids=lambda c: c.name)
def test_tensor_core_prefill_against_oracle(cfg):
    """Prompts longer than the initialisation window: their bulk is prefilled by the tcgen05 GEMMs (only the KV
    cache comes out of it).  Cached K/V of bulk positions in every layer, the window's hidden states (which
    attend to those keys), and the rounds that follow must match the oracle; the same through the decode kernels."""
    import oracle
    import paper_2504_05598_b200 as dl
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    prompt = synth.make_prompt(cfg)
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    P, W = len(prompt), min(cfg.init_window, len(prompt))
    ref = ref_from_oracle(cfg, w, prompt)
    # attention of the bulk prefill: tcgen05 (head dimension 128) or mma.sync flash-style; the mma.sync one where the
    # other is the default; the decode attention kernel in passes of 64 rows; everything through the decode kernels
    for flags in (dl.FLAG_PDL | dl.FLAG_TC, dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_MMA_SYNC_PREFILL_ATTN,
                  dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_DECODE_ATTN_PREFILL, dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_NO_BULK_PREFILL):
        ctx.set_flags(flags)
        launches0 = ctx.launch_count()
        ctx.prefill(0, prompt, cfg.gen_len)
        n_launch = ctx.launch_count() - launches0
        for l in range(1, cfg.n_layers + 1):
            for pos in sorted({0, 1, 15, 16, 127, 128, min(511, P - 1), min(512, P - 1), P - W - 1, P - W, P - 1}):
                k, v = ctx.get_kv(0, l, pos)
                kr, vr = o.k_row(l, pos), o.v_row(l, pos)
                assert np.abs(k - kr).max() <= 2e-2 * np.abs(kr).max() + 1e-6, ("k", flags, l, pos)
                assert np.abs(v - vr).max() <= 2e-2 * np.abs(vr).max() + 1e-6, ("v", flags, l, pos)
        for l in range(cfg.n_layers + 1):
            for j in (0, W - 1):
                r, got = o.hidden(l, j), ctx.get_hidden(0, l, j)
                assert np.abs(got - r).max() <= 2e-2 * np.abs(r).max() + 1e-6, ("h", flags, l, j)
        rep = run_sequence(ctx, 0, ref, cfg.gen_len)
        print(f"{cfg.name} flags {flags}: prefill launches {n_launch}, rounds {rep.rounds} flips {rep.flips}")
        assert rep.ok(), rep.failures[:5]
    o.close()


@pytest.mark.parametrize("prompt_len", [1, 2, 95, 96, 97])
def test_prompt_length_edges(prompt_len):
    """One-token prompt (window of one position), and the lengths around the switch to the tensor-core
    prefill (64 positions before the 32-position window)."""
    import oracle
    cfg = synth.small_variant(TINY, name=f"tiny_p{prompt_len}", prompt_len=prompt_len, gen_len=12, emb_scale=10.0,
                              seed=300 + prompt_len)
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    prompt = synth.make_prompt(cfg)
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    ctx.prefill(0, prompt, cfg.gen_len)
    for l in (1, cfg.n_layers):
        for pos in sorted({0, prompt_len // 2, prompt_len - 1}):
            k, v = ctx.get_kv(0, l, pos)
            kr, vr = o.k_row(l, pos), o.v_row(l, pos)
            assert np.abs(k - kr).max() <= 2e-2 * np.abs(kr).max() + 1e-6, ("k", l, pos)
            assert np.abs(v - vr).max() <= 2e-2 * np.abs(vr).max() + 1e-6, ("v", l, pos)
    o.close()
    ref = ref_from_oracle(cfg, w, prompt)
    rep = run_sequence(ctx, 0, ref, cfg.gen_len)
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)
    ctx.close()


def test_largest_speculation_length():
    """g_max = 31 (the largest the library accepts): 32-row verify passes and a 32-row draft/verify history."""
    cfg = synth.small_variant(TINY_GQA, name="tiny_gqa_g31", g_max=31, gen_len=80, seed=91)
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    prompt = synth.make_prompt(cfg)
    for policy in ((2, 31), None):
        ref = ref_from_oracle(cfg, w, prompt, policy=policy)
        rep = run_sequence(ctx, 0, ref, cfg.gen_len, policy=policy)
        print(f"{cfg.name} policy {policy}: rounds {rep.rounds} compared {rep.compared} flips {rep.flips}")
        assert rep.ok(), rep.failures[:5]
        assert rep.rounds == len(ref.rounds)
    assert max(r.g for r in ref_from_oracle(cfg, w, prompt, policy=(2, 31)).rounds) == 31
    ctx.close()


def test_dynamic_rounds_match_oracle(small):
    cfg, w, ctx = small
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg))
    rep = run_sequence(ctx, 0, ref, cfg.gen_len)
    print(f"{cfg.name}: rounds {rep.rounds} compared {rep.compared} flips {rep.flips} resyncs {rep.resyncs}")
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)
    assert rep.flips <= max(3, rep.compared // 50)          # flips are rare, not the rule


def test_every_fixed_setting_reproduces_the_greedy_stream(small):
    """Speculative greedy output equals plain greedy output for every (E, gamma), gamma = 0 included."""
    cfg, w, ctx = small
    prompt = synth.make_prompt(cfg)
    settings = [(1, 0)] + [(E, g) for E in range(cfg.e_min, cfg.e_max + 1) for g in range(max(1, cfg.g_min), cfg.g_max + 1)]
    for E, g in settings:
        ref = ref_from_oracle(cfg, w, prompt, policy=(E, g))
        rep = run_sequence(ctx, 0, ref, cfg.gen_len, policy=(E, g))
        assert rep.ok(), ((E, g), rep.failures[:5])
        assert rep.rounds == len(ref.rounds)


def test_step_calls_equal_round_call(small):
    cfg, w, ctx = small
    prompt = synth.make_prompt(cfg)
    first = ctx.prefill(0, prompt, 24)
    a_tokens, E, g = [first.tokens[0]], first.next_E, first.next_gamma
    a_trace = []
    while len(a_tokens) < 24:
        ctx.draft(0, E, g)
        ctx.verify(0)
        out = ctx.layer_accept(0)
        sh, cn = ctx.get_shadow(0)
        E, g = ctx.select(0)
        a_tokens += out.emitted()
        a_trace.append((out.E, out.g, out.n_accept, sh.copy(), cn.copy(), E, g))
    first = ctx.prefill(0, prompt, 24)
    b_tokens = [first.tokens[0]]
    k = 0
    while len(b_tokens) < 24:
        out = ctx.round()[0]
        sh, cn = ctx.get_shadow(0)
        b_tokens += out.emitted()
        t = a_trace[k]
        assert (out.E, out.g, out.n_accept, out.next_E, out.next_gamma) == (t[0], t[1], t[2], t[5], t[6])
        assert np.array_equal(sh[:, :out.g + 1], t[3][:, :out.g + 1]) and np.array_equal(cn, t[4])
        k += 1
    assert a_tokens == b_tokens and len(a_tokens) == 24
    # run-to-run determinism: a third pass gives the same tokens
    first = ctx.prefill(0, prompt, 24)
    c_tokens = [first.tokens[0]]
    while len(c_tokens) < 24:
        c_tokens += ctx.round()[0].emitted()
    assert c_tokens == b_tokens


def test_error_codes(small):
    import paper_2504_05598_b200 as dl
    cfg, w, ctx = small
    lib, h = ctx.lib, ctx._h
    prompt = synth.make_prompt(cfg)
    p = np.ascontiguousarray(prompt, dtype=np.int32)
    assert lib.del_prefill(h, 99, p.ctypes.data, len(p), 8, None) == dl.EINVAL
    assert lib.del_prefill(h, 0, p.ctypes.data, 0, 8, None) == dl.EINVAL
    assert lib.del_prefill(h, 0, p.ctypes.data, len(p), 10 ** 6, None) == dl.ENOSPC
    bad = p.copy()
    bad[3] = cfg.vocab
    assert lib.del_prefill(h, 0, bad.ctypes.data, len(bad), 8, None) == dl.EINVAL
    ctx.release(0)
    assert lib.del_draft(h, 0, 1, 1) == dl.ESTATE                      # no prefill yet
    ctx.prefill(0, prompt, 8)
    assert lib.del_verify(h, 0) == dl.ESTATE                           # verify before draft
    assert lib.del_draft(h, 0, cfg.n_layers, 1) == dl.EINVAL           # E must leave layers to verify with
    assert lib.del_draft(h, 0, 1, cfg.g_max + 1) == dl.EINVAL
    assert lib.del_layer_accept(h, 0, None) == dl.ESTATE
    ctx.draft(0, 1, 1)
    assert lib.del_draft(h, 0, 1, 1) == dl.ESTATE                      # round in progress
    ctx.verify(0)
    ctx.layer_accept(0)
    # policy / mode calls
    L = cfg.n_layers
    assert lib.del_set_policy(h, 0, L, 1) == dl.EINVAL                 # E must be < n_layers
    assert lib.del_set_policy_fs(h, 0, 1, 0) == dl.EINVAL              # the controller needs gamma0 >= 1
    assert lib.del_set_policy_fs(h, 0, 0, 2) == dl.EINVAL              # ... and a fixed exit layer
    assert lib.del_set_policy_fs(h, 0, 1, cfg.g_max + 1) == dl.EINVAL
    assert lib.del_set_exit_mode(h, 99, 1) == dl.EINVAL
    assert lib.del_get_conf_stats(h, 99, None, None, None) == dl.EINVAL
    assert lib.del_set_conf_stats(h, 0, None, None) == dl.EINVAL
    assert lib.del_get_conf(h, 99, None, None) == dl.EINVAL
    assert lib.del_get_conf(h, 0, None, None) == dl.OK                 # both outputs are optional
    # the context is still healthy
    assert ctx.round()[0].n_emitted >= 1


def test_expired_device_wait_is_reported_cleared_and_survivable(small):
    """The path a bounded device-side wait takes when it gives up: a non-zero error word -> DEL_ETIMEOUT from the next
    call that reads results, the word cleared, the context usable.  The word is written from the host (test hook), so
    no kernel waits and nothing on the GPU misbehaves."""
    import paper_2504_05598_b200 as dl
    cfg, w, ctx = small
    lib, h = ctx.lib, ctx._h
    prompt = synth.make_prompt(cfg)
    ref = ref_from_oracle(cfg, w, prompt)
    assert lib.del_debug_inject_error(h, 0) == dl.EINVAL
    # through del_round (results come back by the mailbox, whose status word carries the error)
    ctx.prefill(0, prompt, cfg.gen_len)
    ctx.round()
    ctx.debug_inject_error(3)
    outs = (dl.RoundOut * ctx.shape.max_batch)()
    assert lib.del_round(h, outs) == dl.ETIMEOUT
    assert b"wait" in lib.del_strerror(dl.ETIMEOUT)
    # through the step calls (results come back by copy)
    ctx.prefill(0, prompt, cfg.gen_len)
    ctx.draft(0, cfg.e_min, 1)
    ctx.verify(0)
    ctx.debug_inject_error(4)
    assert lib.del_layer_accept(h, 0, None) == dl.ETIMEOUT
    # and through a prefill
    ctx.debug_inject_error(1)
    p = np.ascontiguousarray(prompt, dtype=np.int32)
    assert lib.del_prefill(h, 0, p.ctypes.data, len(p), cfg.gen_len, None) == dl.ETIMEOUT
    # the word was cleared each time: a fresh run of the sequence matches the oracle from start to end
    rep = run_sequence(ctx, 0, ref, cfg.gen_len)
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)


def test_early_reads_and_l2_requests_change_no_result(small):
    """The decode attention reads committed cache pages and asks for the O-projection's weights before it waits for the
    QKV launch: scheduling only.  With the weight requests switched off, and through the step calls (whose launches
    meet other timing), the stream and the last hidden states are bit-identical."""
    import paper_2504_05598_b200 as dl
    cfg, w, ctx = small
    prompt = synth.make_prompt(cfg)

    def run(flags):
        old = ctx.set_flags(flags)
        try:
            toks = [ctx.prefill(0, prompt, cfg.gen_len).tokens[0]]
            while len(toks) < cfg.gen_len:
                toks += ctx.round()[0].emitted()
            return toks, ctx.get_hidden(0, cfg.n_layers, 0).copy()
        finally:
            ctx.set_flags(old)

    a = run(dl.FLAG_PDL | dl.FLAG_TC)
    b = run(dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_NO_WEIGHT_PREFETCH)
    c = run(dl.FLAG_TC | dl.FLAG_NO_WEIGHT_PREFETCH)                  # no programmatic dependent launch either
    assert a[0] == b[0] == c[0] and len(a[0]) == cfg.gen_len
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[1], c[1])


def test_kv_pages_run_out_and_come_back():
    """Two sequences share a page pool that holds one and a half of them: the second prefill is refused with
    DEL_ENOSPC, the first sequence keeps decoding correctly, and after its release the second one fits."""
    import paper_2504_05598_b200 as dl
    cfg = synth.small_variant(TINY, batch=2, gen_len=16)
    w = synth.make_weights(cfg)
    # pages are handed out as positions are reached: sequence 0 holds 3 of the 7 pages after two rounds, the
    # long prompt below needs 5 for its prefill
    ctx = dl.DelContext(dl.make_shape(cfg, max_seq=160, n_pages=7), dl.upload_weights(w))
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg, 0))
    p1 = np.ascontiguousarray(synth.make_prompt(cfg, 1), dtype=np.int32)
    ctx.prefill(0, ref.prompt, cfg.gen_len)
    ctx.round()
    ctx.round()                                                                # sequence 0 now holds most of its pages
    big = np.ascontiguousarray(np.tile(p1, 3)[:cfg.prompt_len * 2 + 8], dtype=np.int32)
    rc = ctx.lib.del_prefill(ctx._h, 1, big.ctypes.data, len(big), 8, None)
    assert rc == dl.ENOSPC
    rep = run_sequence(ctx, 0, ref, cfg.gen_len)                               # sequence 0 is unharmed
    assert rep.ok(), rep.failures[:5]
    ctx.release(0)
    assert ctx.lib.del_prefill(ctx._h, 1, big.ctypes.data, len(big), 8, None) == dl.OK
    assert ctx.round()[1].n_emitted >= 1
    ctx.close()


def test_generation_stops_at_budget(small):
    cfg, w, ctx = small
    import paper_2504_05598_b200 as dl
    first = ctx.prefill(0, synth.make_prompt(cfg), 9)
    n = 1
    while True:
        rc, outs = ctx.try_round()
        if rc != dl.OK:
            assert rc == dl.ESTATE
            break
        assert 1 <= outs[0].n_emitted <= outs[0].g + 1
        n += outs[0].n_emitted
    assert n == 9


def test_batch_of_independent_sequences():
    """Three sequences with their own prompts, (E, gamma), statistics and generation lengths share the layer passes;
    a sequence that has emitted all its tokens drops out of the later rounds."""
    import paper_2504_05598_b200 as dl
    cfg = synth.small_variant(TINY_GQA, batch=3)
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    totals = [20 + 7 * s for s in range(3)]
    refs = [ref_from_oracle(cfg, w, synth.make_prompt(cfg, s), gen_len=totals[s]) for s in range(3)]
    reps = [Report() for _ in refs]
    for s in range(3):
        compare_init(ctx, s, refs[s], totals[s], reps[s])
    k, done = [0, 0, 0], [1, 1, 1]
    while True:
        rc, outs = ctx.try_round()
        if rc != dl.OK:
            assert rc == dl.ESTATE                      # no live sequence is left
            break
        for s in range(3):
            if k[s] >= len(refs[s].rounds):
                assert outs[s].n_emitted == 0           # finished: takes no part in the round
                continue
            r = refs[s].rounds[k[s]]
            need = compare_round(ctx, s, outs[s], r, reps[s])
            done[s] += r.n + 1
            k[s] += 1
            if need and k[s] < len(refs[s].rounds):
                reps[s].resyncs += 1
                _resync(ctx, s, refs[s], done[s], r.Sc, r.Sn, r.next_E, r.next_gamma, totals[s], r.Stcs, r.Sfcs)
    for s in range(3):
        print(f"seq {s}: rounds {reps[s].rounds} compared {reps[s].compared} flips {reps[s].flips}")
        assert reps[s].ok(), (s, reps[s].failures[:5])
        assert k[s] == len(refs[s].rounds) and done[s] == totals[s]


@pytest.mark.parametrize("name,max_rounds", [("llama2_7b", None), ("llama32_1b", None), ("llama2_13b", None)])
def test_full_size_config_against_stored_trace(name, max_rounds):
    """The benchmark shapes, in the configuration bench.py times, against the oracle's stored trace."""
    path = os.path.join(GOLDEN, f"trace_{name}.json")
    if not os.path.exists(path):
        pytest.skip("no stored trace")
    doc = json.load(open(path))
    cfg = synth.CONFIGS[name]
    assert doc["seed"] == cfg.seed and doc["prompt_len"] == cfg.prompt_len
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    ref = ref_from_golden(doc, 0, synth.make_prompt(cfg, 0))
    rep = run_sequence(ctx, 0, ref, doc["gen_len"], max_rounds=max_rounds)
    print(f"{name}: rounds {rep.rounds} compared {rep.compared} flips {rep.flips} resyncs {rep.resyncs} "
          f"largest differing margin {rep.max_flip_margin:.3f}")
    # the bar is 0.05 (a failure above it); what actually differs sits well inside
    assert rep.max_flip_margin <= 0.03
    assert rep.ok(), rep.failures[:8]
    assert rep.flips <= rep.compared // 20


def test_streaming_lm_head_against_oracle(small):
    """The stacked LM head also exists as a streaming (mma.sync) kernel; it must match the oracle too."""
    import paper_2504_05598_b200 as dl
    cfg, w, ctx = small
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg))
    old = ctx.set_flags(dl.FLAG_PDL)
    try:
        rep = run_sequence(ctx, 0, ref, cfg.gen_len)
    finally:
        ctx.set_flags(old)
    print(f"{cfg.name} (streaming head): rounds {rep.rounds} compared {rep.compared} flips {rep.flips}")
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)


def test_dynamic_draft_exiting_against_oracle(small):
    """Sec. 4.4 / Algorithm 1 with the confidence break: the draft loop runs up to g_max tokens and stops at
    the first token whose confidence is below the exit layer's threshold; same streams, same g, same
    stop decisions (outside the tolerance band), confidences and thresholds within tolerance."""
    cfg, w, ctx = small
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg), exit_mode=True)
    rep = run_sequence(ctx, 0, ref, cfg.gen_len)
    ctx.set_exit_mode(0, False)
    stops = sum(r.stopped for r in ref.rounds)
    print(f"{cfg.name} (draft-exiting): rounds {rep.rounds} stops {stops} decisions {rep.decisions} decision flips "
          f"{rep.decision_flips} conf compared {rep.conf_compared} max rel err {rep.conf_max_rel:.2e} flips {rep.flips}")
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)
    assert rep.decisions > 0 and rep.decision_flips <= max(1, rep.decisions // 10)


def test_draft_exiting_step_calls_equal_round_call(small):
    """del_draft in exit mode runs the same confidence-checked loop as del_round."""
    cfg, w, ctx = small
    prompt = synth.make_prompt(cfg)
    first = ctx.prefill(0, prompt, 24)
    ctx.set_exit_mode(0, True)
    a_tokens, E, trace = [first.tokens[0]], first.next_E, []
    while len(a_tokens) < 24:
        ctx.draft(0, E, cfg.g_max)
        ctx.verify(0)
        out = ctx.layer_accept(0)
        E, _ = ctx.select(0)
        a_tokens += out.emitted()
        trace.append((out.E, out.g, out.stopped, out.n_accept, E))
    first = ctx.prefill(0, prompt, 24)
    ctx.set_exit_mode(0, True)
    b_tokens, k = [first.tokens[0]], 0
    while len(b_tokens) < 24:
        out = ctx.round()[0]
        b_tokens += out.emitted()
        assert (out.E, out.g, out.stopped, out.n_accept, out.next_E) == trace[k], k
        k += 1
    assert a_tokens == b_tokens and len(a_tokens) == 24
    assert any(t[2] for t in trace)                     # the break did fire
    ctx.set_exit_mode(0, False)


def test_batch_with_mixed_exit_modes():
    """Three sequences share the layer passes; two of them draft with the confidence break, one does not."""
    cfg = synth.small_variant(TINY_GQA, batch=3)
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    refs = [ref_from_oracle(cfg, w, synth.make_prompt(cfg, s), gen_len=24, exit_mode=(s != 1)) for s in range(3)]
    reps = run_batch(ctx, refs, 24)
    for s, rep in enumerate(reps):
        print(f"seq {s} exit {refs[s].exit_mode}: rounds {rep.rounds} decisions {rep.decisions} flips {rep.flips} "
              f"resyncs {rep.resyncs}")
        assert rep.ok(), (s, rep.failures[:5])
        assert rep.rounds == len(refs[s].rounds)


@pytest.mark.parametrize("exit_mode", [False, True], ids=["fixed_gamma", "draft_exiting"])
def test_stacked_head_rows_trimmed_to_candidate_layers(exit_mode):
    """With the rows of the stacked LM head restricted to the layers the selection can pick (e_min..e_max) plus
    the last one, everything the method uses is unchanged: the stream, the accept lengths, the statistics of the
    candidate layers, the thresholds and the (E, gamma) trajectory; fewer rows go through the head."""
    import paper_2504_05598_b200 as dl
    cfg = synth.small_variant(TINY_GQA, name="tiny_gqa_trim", e_min=2, e_max=4, gen_len=40)      # L = 6
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg), exit_mode=exit_mode)
    layers = list(range(cfg.e_min - 1, cfg.e_max)) + [cfg.n_layers - 1]
    ctx.set_flags(dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_TRIM_ROWS)
    rep = run_sequence(ctx, 0, ref, cfg.gen_len, layers=layers)
    print(f"trimmed rows (exit mode {exit_mode}): rounds {rep.rounds} compared {rep.compared} flips {rep.flips}")
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds)
    # the same through the streaming head, and with speculative sampling on top
    ctx.set_flags(dl.FLAG_PDL | dl.FLAG_TRIM_ROWS)
    rep = run_sequence(ctx, 0, ref, cfg.gen_len, layers=layers)
    assert rep.ok(), rep.failures[:5]
    ctx.set_flags(dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_TRIM_ROWS)
    from sampling_parity import run_sequence_sampling
    srep = run_sequence_sampling(ctx, 0, cfg, w, synth.make_prompt(cfg), 0.6, 0.95, 3, exit_mode=exit_mode, layers=layers)
    assert srep.ok() and srep.rounds >= 5, srep.failures[:5]
    ctx.close()


def test_random_shapes_against_oracle():
    """Seeded random small models: depth, head dimension 64 / 128, candidate-layer and speculation-length ranges (g_min = 0 included),
    prompt lengths on both sides of the window and of the tensor-core prefill's chunk, batch sizes 1 to 3, greedy
    and draft-exiting sequences mixed; every one compared with the oracle round by round."""
    rng = np.random.default_rng(20250405)
    rounds = compared = 0
    for k in range(24):
        base = TINY_GQA if k % 2 else TINY
        if k % 4 >= 2:                                   # head dimension 128, two query heads on two or one kv head
            base = synth.small_variant(base, head_dim=128, n_heads=2, n_kv_heads=2 if k % 8 < 4 else 1)
        L = int(rng.integers(3, 9))
        e_min = int(rng.integers(1, L - 1))
        e_max = min(int(rng.integers(e_min, L)), L - 1)
        g_max = int(rng.integers(1, 9))
        g_min = int(rng.integers(0, min(2, g_max) + 1))
        cfg = synth.small_variant(base, name=f"random{k}", n_layers=L, e_min=e_min, e_max=e_max, g_min=g_min, g_max=g_max,
                                  prompt_len=int(rng.choice([1, 5, 31, 32, 33, 70, 96, 130, 300, 520, 700])),
                                  gen_len=int(rng.integers(4, 40)), seed=int(rng.integers(1, 10 ** 6)), emb_scale=10.0,
                                  batch=int(rng.choice([1, 1, 2, 3])))
        w = synth.make_weights(cfg)
        ctx = make_ctx(cfg, w)
        exit_mode = k % 3 == 0
        refs = [ref_from_oracle(cfg, w, synth.make_prompt(cfg, s), exit_mode=exit_mode and s % 2 == 0) for s in range(cfg.batch)]
        reps = run_batch(ctx, refs, cfg.gen_len) if cfg.batch > 1 else [run_sequence(ctx, 0, refs[0], cfg.gen_len)]
        for ref, rep in zip(refs, reps):
            assert rep.ok() and rep.rounds == len(ref.rounds), (k, cfg, rep.failures[:3])
            rounds += rep.rounds
            compared += rep.compared
        ctx.close()
    print(f"24 random shapes: {rounds} rounds, {compared} arg-max results compared")


def test_interleaved_sequence_lifetimes_with_few_pages():
    """Four slots, 22 KV pages: sequences of random prompt and generation lengths start, run, finish and are released
    at random times (some with draft-exiting), so that pages change hands and some prefills or rounds are refused for
    lack of pages (DEL_ENOSPC, after which the context goes on).  Every sequence is compared with its own oracle."""
    import paper_2504_05598_b200 as dl
    from parity import Report, _resync, compare_init, compare_round
    rng = np.random.default_rng(1)
    B = 4
    base = synth.small_variant(TINY_GQA, name="lifetimes", batch=B, prompt_len=64, gen_len=40, g_max=4)
    w = synth.make_weights(base)
    ctx = dl.DelContext(dl.make_shape(base, max_seq=256, n_pages=22), dl.upload_weights(w))
    slots = [None] * B
    n = dict(starts=0, refused=0, rounds=0, released=0, finished=0)
    for step in range(300):
        act = rng.random()
        free = [s for s in range(B) if slots[s] is None]
        live = [s for s in range(B) if slots[s] is not None]
        if free and (act < 0.3 or not live):
            s = int(rng.choice(free))
            G = int(rng.integers(3, 40))
            cfg = synth.small_variant(base, prompt_len=int(rng.choice([1, 7, 33, 64, 100, 130])), gen_len=G,
                                      seed=int(rng.integers(1, 10 ** 6)))
            ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg, s), exit_mode=bool(rng.random() < 0.3))
            rep = Report()
            try:
                compare_init(ctx, s, ref, G, rep)
            except dl.DelError as e:
                assert e.code == dl.ENOSPC
                n["refused"] += 1
                continue
            slots[s] = dict(ref=ref, k=0, done=1, rep=rep, G=G)
            n["starts"] += 1
        elif live and act < 0.4:
            s = int(rng.choice(live))
            ctx.release(s)
            slots[s] = None
            n["released"] += 1
        elif live:
            try:
                outs = ctx.round()
            except dl.DelError as e:                      # no page for some sequence's round: give up the longest one
                assert e.code == dl.ENOSPC
                s = max(live, key=lambda q: len(slots[q]["ref"].prompt) + slots[q]["done"])
                ctx.release(s)
                slots[s] = None
                n["refused"] += 1
                continue
            n["rounds"] += 1
            for s in live:
                st = slots[s]
                ref = st["ref"]
                r = ref.rounds[st["k"]]
                need = compare_round(ctx, s, outs[s], r, st["rep"])
                assert st["rep"].ok(), (step, s, st["rep"].failures[:3])
                st["done"] += r.n + 1
                st["k"] += 1
                if st["k"] >= len(ref.rounds):
                    n["finished"] += 1
                    ctx.release(s)
                    slots[s] = None
                elif need:
                    try:
                        _resync(ctx, s, ref, st["done"], r.Sc, r.Sn, r.next_E, r.next_gamma, st["G"], r.Stcs, r.Sfcs)
                    except dl.DelError as e:
                        assert e.code == dl.ENOSPC
                        slots[s] = None
                        n["refused"] += 1
    print(n)
    assert n["finished"] >= 15 and n["refused"] >= 3 and n["released"] >= 10
    ctx.close()


@pytest.mark.parametrize("n_layers,layers", [(6, (1, 2, 3, 4, 5, 6)), (32, (8, 16, 24, 32))])
def test_logit_error_at_full_width(n_layers, layers):
    """The 7B layer shape (d = 4096, F = 11008, V = 32000), six layers and the full 32, a 100-token prompt, oracle run
    live: exit-head logits over the whole vocabulary must stay within max-abs 3e-2 of the oracle's at every layer
    compared, through the tensor-core prefill and through the decode kernels.  (Every GEMM input is a bf16 high + low
    pair; with single bf16 inputs the largest difference was 0.042 at layer 6.)"""
    import oracle
    import paper_2504_05598_b200 as dl
    base = synth.CONFIGS["llama2_7b"]
    cfg = synth.small_variant(base, name=f"llama2_7b_L{n_layers}", n_layers=n_layers, e_min=1, e_max=n_layers - 1, g_max=5,
                              prompt_len=100, gen_len=20, seed=11)
    w = synth.make_weights(cfg)
    prompt = synth.make_prompt(cfg)
    o = oracle.OracleSeq(cfg, w)
    o.prefill(prompt)
    j = cfg.init_window - 1
    want = {}
    for l in layers:
        ho = o.hidden(l, j)
        want[l] = (ho, o.exit_head(ho, want_logits=True)[2])
    o.close()
    dev = dl.upload_weights(w)
    for path, flags in (("tensor-core prefill", dl.FLAG_PDL | dl.FLAG_TC), ("decode kernels", dl.FLAG_PDL | dl.FLAG_TC | dl.FLAG_NO_BULK_PREFILL)):
        ctx = dl.DelContext(dl.make_shape(cfg), dev)
        ctx.set_flags(flags)
        ctx.prefill(0, prompt, cfg.gen_len)
        for l in layers:
            ho, lo = want[l]
            hl = ctx.get_hidden(0, l, j)
            h_rel = float(np.sqrt(((hl - ho) ** 2).mean()) / np.sqrt((ho ** 2).mean()))
            ll = ctx.debug_logits(0, l, j)
            rms, mx = float(np.sqrt(((ll - lo) ** 2).mean())), float(np.abs(ll - lo).max())
            print(f"{path}, layer {l}: hidden rel rms {h_rel:.2e}, logits rms {rms:.4f} max {mx:.4f} (logit std {lo.std():.2f})")
            assert mx <= 3e-2, (path, l, mx)
            assert h_rel <= 6e-3 and rms <= 8e-3, (path, l, h_rel, rms)
        ctx.close()


def test_fs_baseline_policy_against_oracle(small):
    """Baseline FS(E-gamma) of Sec. 5.1 on the same kernels: fixed exit layer, gamma moved by +-1 on the device."""
    cfg, w, ctx = small
    fs = (cfg.e_min, 3)
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg), policy_fs=fs)
    rep = run_sequence(ctx, 0, ref, cfg.gen_len, policy_fs=fs)
    gammas = [r.gamma for r in ref.rounds]
    print(f"{cfg.name} (FS): rounds {rep.rounds} gamma trajectory {gammas[:12]} flips {rep.flips}")
    assert rep.ok(), rep.failures[:5]
    assert rep.rounds == len(ref.rounds) and len(set(gammas)) > 1


def test_confidences_in_fixed_gamma_rounds(small):
    """The confidence statistics are maintained in every mode; here with the streaming LM head as well."""
    import paper_2504_05598_b200 as dl
    cfg, w, ctx = small
    ref = ref_from_oracle(cfg, w, synth.make_prompt(cfg))
    for flags in (dl.FLAG_PDL | dl.FLAG_TC, dl.FLAG_PDL):
        old = ctx.set_flags(flags)
        try:
            rep = run_sequence(ctx, 0, ref, cfg.gen_len)
        finally:
            ctx.set_flags(old)
        print(f"{cfg.name} flags {flags}: conf compared {rep.conf_compared} max rel err {rep.conf_max_rel:.2e}")
        assert rep.ok(), rep.failures[:5]
        assert rep.conf_compared > 0 and rep.conf_max_rel <= 0.02     # far inside the derived bound in practice


@pytest.mark.parametrize("name", ["llama2_7b", "llama32_1b", "llama2_13b"])
def test_dynamic_draft_exiting_full_size(name):
    """Full-size shapes with the confidence break, against the stored oracle traces."""
    path = os.path.join(GOLDEN, f"trace_{name}_exit.json")
    if not os.path.exists(path):
        pytest.skip("no stored trace")
    doc = json.load(open(path))
    cfg = synth.CONFIGS[name]
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    ref = ref_from_golden(doc, 0, synth.make_prompt(cfg, 0))
    assert ref.exit_mode
    rep = run_sequence(ctx, 0, ref, doc["gen_len"])
    stops = sum(r.stopped for r in ref.rounds)
    print(f"{name} (draft-exiting): rounds {rep.rounds} stops {stops} decisions {rep.decisions} decision flips "
          f"{rep.decision_flips} conf compared {rep.conf_compared} max rel err {rep.conf_max_rel:.2e} flips {rep.flips} "
          f"resyncs {rep.resyncs}")
    assert rep.ok(), rep.failures[:8]
    assert rep.decisions > 0 and rep.decision_flips <= max(2, rep.decisions // 10)


def test_streaming_lm_head_full_size():
    import paper_2504_05598_b200 as dl
    name = "llama2_7b"
    doc = json.load(open(os.path.join(GOLDEN, f"trace_{name}.json")))
    cfg = synth.CONFIGS[name]
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    ctx.set_flags(dl.FLAG_PDL)
    ref = ref_from_golden(doc, 0, synth.make_prompt(cfg, 0))
    rep = run_sequence(ctx, 0, ref, doc["gen_len"], max_rounds=40)
    print(f"{name} (streaming head): rounds {rep.rounds} compared {rep.compared} flips {rep.flips} resyncs {rep.resyncs}")
    assert rep.ok(), rep.failures[:8]


def test_full_size_batch_of_four_against_stored_trace():
    """Llama-3-8B shape, four sequences with their own (E, gamma) state and paged KV, lock-step rounds."""
    name = "llama3_8b_b4"
    path = os.path.join(GOLDEN, f"trace_{name}.json")
    if not os.path.exists(path):
        pytest.skip("no stored trace")
    doc = json.load(open(path))
    cfg = synth.CONFIGS[name]
    assert doc["seed"] == cfg.seed and len(doc["sequences"]) == cfg.batch
    assert doc["gen_len"] == cfg.gen_len == 512                  # the whole generation of every sequence, not a prefix
    w = synth.make_weights(cfg)
    ctx = make_ctx(cfg, w)
    refs = [ref_from_golden(doc, s, synth.make_prompt(cfg, s)) for s in range(cfg.batch)]
    reps = run_batch(ctx, refs, doc["gen_len"])
    for s, rep in enumerate(reps):
        print(f"{name} seq {s}: rounds {rep.rounds} compared {rep.compared} flips {rep.flips} resyncs {rep.resyncs}")
        assert rep.ok(), (s, rep.failures[:8])
        assert rep.rounds == len(refs[s].rounds) >= 300
