"""CPU-side checks of the C ABI: the library loads, exports every symbol the header declares,
and its host-only entry points (slice strategy, model layout) agree with the paper's numbers."""
import os
import re

import numpy as np
import pytest

from conftest import GOLDEN, ROOT


def _binding():
    from paper_2408_11500_b200 import build
    build.build()
    from paper_2408_11500_b200 import binding
    return binding


def test_library_exports_every_declared_symbol():
    B = _binding()
    header = open(os.path.join(ROOT, "include", "slicegcn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)          # declarations only, not prose
    declared = set(re.findall(r"(?:slicegcn_status_t|const char\*)\s+(slicegcn_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    import ctypes
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in include/slicegcn.h but not exported"
    assert declared == set(B.EXPORTS)


def test_slice_strategy_golden_through_abi():
    B = _binding()
    for line in open(os.path.join(GOLDEN, "alg1_slices.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        a, b, c = [t.strip() for t in line.split("|")]
        in_d, p, scale = a.split()
        want = [tuple(int(v) for v in t.split(":")) for t in c.split()]
        got, size = B.slicegcn_slice_strategy(int(in_d), int(p), float(scale))
        assert got == want and size == int(b)


def test_slice_strategy_errors():
    B = _binding()
    for args in [(8, 0, 1.0), (0, 2, 1.0), (8, 2, 0.1), (8, 2, 3.0), (8, 65, 1.0)]:
        with pytest.raises(B.SliceGCNError) as e:
            B.slicegcn_slice_strategy(*args)
        assert e.value.status == B.ERR_INVALID_ARG
    with pytest.raises(B.SliceGCNError):
        B.slicegcn_slice_strategy(8, 2, 1.0, 7)
    assert B.slicegcn_slice_strategy(300, 3, 1.0, B.RULE_FLOOR_PLUS_1)[1] == 101


def _fmt(n):
    return f"{n / 1e6:.2f}M" if n >= 1e6 else f"{n / 1e3:.2f}K"


def test_table3_parameter_counts_through_abi():
    B = _binding()
    ds, rows = [], []
    for line in open(os.path.join(GOLDEN, "table3_param_counts.txt")):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "dataset":
            ds.append((t[1], int(t[2]), int(t[3]), int(t[4])))
        elif t[0] == "row":
            rows.append((int(t[1]), int(t[2]), int(t[3]), t[5:]))
    checked = 0
    for p, ff, se, vals in rows:
        for (name, in_d, classes, L), want in zip(ds, vals):
            if p == 0:
                m = B.slicegcn_model_create(in_d, 512, L, classes, 1, use_self=True, use_b_self=True)
            else:
                m = B.slicegcn_model_create(in_d, 512, L, classes, p, slice_rule=B.RULE_FLOOR_PLUS_1, use_ff=bool(ff),
                                            use_se=bool(se), use_self=True, use_b_self=True)
            assert _fmt(B.slicegcn_model_param_count(m)) == want, (name, p, ff, se)
            B.slicegcn_model_destroy(m)
            checked += 1
    assert checked == 54


def test_model_layout_and_pack_roundtrip():
    B = _binding()
    from oracle import slicegcn_oracle as orc
    from paper_2408_11500_b200 import synth
    m = B.slicegcn_model_create(100, 256, 3, 47, 8, use_ff=True, use_se=True, dtype=B.BF16)
    od = orc.ModelDesc(100, 256, 3, 47, p=8, use_ff=True, use_se=True)
    assert B.slicegcn_model_param_count(m) == orc.param_count(od)
    slices, size, hs = B.slicegcn_model_slices(m, 8)
    assert slices == od.slices and size == od.slice_size == 13 and hs == od.h_s == 32
    assert [B.slicegcn_model_layer_order(m, l) for l in range(3)] == [B.AGG_FIRST] * 3
    named = synth.init_params(orc.param_shapes(od), seed=1, bias_scale=0.1, se_scale=0.1)
    flat = B.pack_params(m, named)
    assert flat.size == B.slicegcn_model_param_elems(m) >= B.slicegcn_model_param_count(m)
    back = B.unpack_params(m, flat)
    assert set(back) == set(named)
    for k in named:
        np.testing.assert_array_equal(back[k], named[k])
    offs = [off for _, off, _ in B.tensor_table(m)]
    assert all(o % 4 == 0 for o in offs)          # 16-byte aligned tensors
    B.slicegcn_model_destroy(m)
    m1 = B.slicegcn_model_create(1433, 16, 2, 7, 4)
    assert [B.slicegcn_model_layer_order(m1, l) for l in range(2)] == [B.XFORM_FIRST, B.AGG_FIRST]
    B.slicegcn_model_destroy(m1)
    with pytest.raises(B.SliceGCNError):
        B.slicegcn_model_create(16, 8, 0, 3, 2)
    with pytest.raises(B.SliceGCNError):
        B.slicegcn_model_create(16, 8, 2, 3, 65)
