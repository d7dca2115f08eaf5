"""The allocation-free exit-head entry point, for callers that cannot call cudaMalloc (frozen memory
pools, plug-ins without an allocator): its tokens must equal those of the regular path, whose scratch
sits in the caller's workspace.  Collected last on purpose; passes alone and after the other tests."""
import numpy as np
import pytest

import synth
from cases import TINY_GQA

pytestmark = pytest.mark.gpu


def bf16_bits(x):
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) & 0xFFFF).astype(np.uint16)


def test_static_scratch_head_equals_workspace_head():
    import torch
    import paper_2504_05598_b200 as dl
    cfg = TINY_GQA                                           # non-unit norm gains, ragged row counts
    w = synth.make_weights(cfg)
    dev = dl.upload_weights(w)
    ctx = dl.DelContext(dl.make_shape(cfg), dev)
    ctx.set_flags(dl.FLAG_PDL)                               # regular path on the same streaming kernel
    ctx.prefill(0, synth.make_prompt(cfg), cfg.gen_len)
    gain = synth.bf16_to_f32(w.final_norm)
    tokens = torch.empty(dl.MAX_ROWS, dtype=torch.int32, device="cuda")
    checked = 0
    for call in range(2):                                    # two calls in a row share the static array
        out = ctx.round()[0]
        shadow, _ = ctx.get_shadow(0)                        # regular entry points' result
        rows, want = [], []
        for layer in range(1, cfg.n_layers + 1):
            for i in range(out.g + 1):
                rows.append(ctx.get_hidden(0, layer, i) * gain)
                want.append(int(shadow[layer - 1, i]))
        x = torch.from_numpy(bf16_bits(np.stack(rows)).view(np.int16)).cuda().view(torch.bfloat16)
        tokens.fill_(-1)
        free_before = torch.cuda.mem_get_info()[0]
        rc = dl.head_argmax_static(x, dev["lm_head"], tokens)
        torch.cuda.synchronize()
        assert rc == dl.OK
        if call == 1:                                        # (the first call may load kernel code lazily)
            assert torch.cuda.mem_get_info()[0] == free_before   # nothing was allocated on the device
        got = tokens[:len(want)].cpu().tolist()
        assert got == want, (call, got, want)
        checked += len(want)
        # and against the oracle's exit head on the same hidden rows, wherever its decision is clear
        if call == 0:
            import oracle
            o = oracle.OracleSeq(cfg, w)
            k = 0
            for layer in range(1, cfg.n_layers + 1):
                for i in range(out.g + 1):
                    tok, margin = o.exit_head(ctx.get_hidden(0, layer, i))[:2]
                    assert margin <= 0.05 or got[k] == tok, (layer, i, got[k], tok, margin)
                    k += 1
            o.close()
    assert checked >= 2 * cfg.n_layers
    # sizes beyond the fixed array are refused, not truncated
    big = torch.zeros(dl.MAX_ROWS + 1, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    assert dl.head_argmax_static(big, dev["lm_head"], tokens) == dl.EINVAL
    ctx.close()


def test_static_scratch_head_at_full_size():
    """64 rows against a 32 000-token vocabulary: the launch then uses one CTA per SM (the widest row tiling) and the
    reduction walks as many partials as there are SMs.  Compared with an fp32 arg-max of the same bf16 inputs
    computed by numpy; rows whose two best logits are closer than the 0.05 bar are skipped."""
    import torch
    import paper_2504_05598_b200 as dl
    rng = np.random.default_rng(5)
    rows, vocab, d = dl.MAX_ROWS, 32000, 512
    xb = bf16_bits(rng.standard_normal((rows, d)).astype(np.float32))
    wb = bf16_bits((rng.standard_normal((vocab, d)) * 0.05).astype(np.float32))
    xf, wf = synth.bf16_to_f32(xb), synth.bf16_to_f32(wb)
    logits = xf @ wf.T
    best = np.argmax(logits, axis=1)
    top2 = np.partition(logits, -2, axis=1)[:, -2:]
    clear = (top2[:, 1] - top2[:, 0]) > 0.05
    x = torch.from_numpy(xb.view(np.int16)).cuda().view(torch.bfloat16)
    wt = torch.from_numpy(wb.view(np.int16)).cuda().view(torch.bfloat16)
    tokens = torch.empty(rows, dtype=torch.int32, device="cuda")
    for call in range(2):
        tokens.fill_(-1)
        assert dl.head_argmax_static(x, wt, tokens) == dl.OK
        torch.cuda.synchronize()
        got = tokens.cpu().numpy()
        assert clear.sum() >= rows // 2
        assert np.array_equal(got[clear], best[clear]), (call, np.nonzero(got != best)[0][:8])
        assert ((got >= 0) & (got < vocab)).all()
