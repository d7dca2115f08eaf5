"""CPU-only checks of the C-ABI library: it builds, loads, exports every declared symbol, and its pure
host-side entry points behave (no compute call is made here)."""
import ctypes as C
import os
import re

import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "del.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(del_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    import paper_2504_05598_b200 as dl
    lib = dl.load_library()
    names = declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(dl.EXPORTS) == names


def test_workspace_size_and_shape_validation():
    import paper_2504_05598_b200 as dl
    lib = dl.load_library()
    for name, cfg in synth.CONFIGS.items():
        shape = dl.make_shape(cfg)
        ws = lib.del_workspace_bytes(C.byref(shape))
        assert ws > 0 and ws % 256 == 0, name
        assert ws < 4 << 30, (name, ws)                         # modest next to 180 GB of HBM
    bad = dl.make_shape(synth.CONFIGS["tiny"])
    bad.head_dim = 96
    assert lib.del_workspace_bytes(C.byref(bad)) == 0
    bad = dl.make_shape(synth.CONFIGS["tiny"])
    bad.e_max = bad.n_layers                                    # the exit layer must leave layers to verify with
    assert lib.del_workspace_bytes(C.byref(bad)) == 0
    bad = dl.make_shape(synth.CONFIGS["tiny"])
    bad.max_batch = 16                                          # 16 * (g_max + 1) rows exceed one pass
    assert lib.del_workspace_bytes(C.byref(bad)) == 0
    bad = dl.make_shape(synth.CONFIGS["tiny"])
    bad.vocab = 1000
    assert lib.del_workspace_bytes(C.byref(bad)) == 0


def test_error_strings_and_null_handling():
    import paper_2504_05598_b200 as dl
    lib = dl.load_library()
    for code in (dl.OK, dl.EINVAL, dl.ENOSPC, dl.ESTATE, dl.ETIMEOUT, dl.ECUDA):
        assert len(lib.del_strerror(code)) > 0
    assert lib.del_strerror(-99) == b"unknown error"
    assert lib.del_round(None, None) == dl.EINVAL
    assert lib.del_draft(None, 0, 1, 1) == dl.EINVAL
    assert lib.del_launch_count(None) == 0
    h = C.c_void_p()
    shape = dl.make_shape(synth.CONFIGS["tiny"])
    assert lib.del_init(C.byref(h), C.byref(shape), None, None, None, 0, None) == dl.EINVAL
    lib.del_destroy(None)


def test_rope_tables_follow_the_definition():
    import numpy as np
    import paper_2504_05598_b200 as dl
    cos, sin = dl.rope_tables(64, 8, 1e4)
    assert cos.shape == (64, 4) and cos.dtype == np.float32
    assert np.allclose(cos[0], 1) and np.allclose(sin[0], 0)
    assert abs(sin[3, 0] - np.sin(3.0)) < 1e-6 and abs(cos[10, 2] - np.cos(10 * 1e4 ** (-0.5))) < 1e-6
