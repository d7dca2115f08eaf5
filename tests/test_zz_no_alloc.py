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
    assert checked >= 2 * cfg.n_layers
    # sizes beyond the fixed array are refused, not truncated
    big = torch.zeros(dl.MAX_ROWS + 1, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    assert dl.head_argmax_static(big, dev["lm_head"], tokens) == dl.EINVAL
    ctx.close()
