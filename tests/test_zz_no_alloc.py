"""The allocation-free aggregation entry point (slicegcn_spmm_static_scratch).

Who needs it: code that runs where device allocation is off limits -- inside a stream capture, on a host
whose device memory is planned once at start-up, or in a plugin that may not touch its host's allocator.
It must give exactly what slicegcn_spmm gives, call after call, with the hub-row scratch coming from the
buffer compiled into the library, and it must refuse (not overrun) a problem that needs more than that buffer.
Collected last on purpose: a failure here must not hide the results of the other GPU tests.
"""
import numpy as np
import pytest

from paper_2408_11500_b200 import synth

pytestmark = pytest.mark.gpu


def _graph_with_hubs(B, n=6000, m=40000, max_degree=2500, seed=7):
    src, dst = synth.chung_lu_powerlaw(n, m, 2.2, max_degree, seed=seed)
    g = B.slicegcn_graph_create(n, src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    assert B.slicegcn_graph_info(g)["n_segments"] > 0        # the path that needs scratch is exercised
    return g, n


@pytest.mark.parametrize("dtype,width", [("f32", 128), ("f32", 72), ("bf16", 256)])
def test_static_scratch_matches_workspace_entry_point_twice(dtype, width):
    import torch
    from paper_2408_11500_b200 import binding as B
    g, n = _graph_with_hubs(B)
    try:
        tdt, bdt = (torch.float32, B.F32) if dtype == "f32" else (torch.bfloat16, B.BF16)
        st = torch.cuda.current_stream().cuda_stream
        wsb = B.slicegcn_spmm_workspace_bytes(g, width)
        assert 0 < wsb <= 8 << 20
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        for call in range(2):                                  # two calls in a row share the built-in buffer
            X = torch.from_numpy(synth.gaussian_features(n, width, seed=call)).cuda().to(tdt)
            want = torch.full_like(X, float("nan"))
            got = torch.full_like(X, float("nan"))
            B.slicegcn_spmm(g, 0, bdt, bdt, X, width, want, width, width, ws, wsb, st)
            B.slicegcn_spmm_static_scratch(g, 0, bdt, bdt, X, width, got, width, width, st)
            torch.cuda.synchronize()
            assert not torch.isnan(got.float()).any()
            a, b = got.float().cpu().numpy(), want.float().cpu().numpy()
            assert np.abs(a - b).max() <= 2e-6 * np.abs(b).max()   # same kernels, same order: in practice identical
        assert B.slicegcn_graph_device_status(g) == 0
    finally:
        B.slicegcn_graph_destroy(g)


def test_static_scratch_refuses_what_does_not_fit():
    import torch
    from paper_2408_11500_b200 import binding as B
    # every row is long (degree ~600): ~3 segments per row, far more partial rows than 8 MiB holds at width 256
    rng = np.random.default_rng(1)
    n = 4096
    src = np.repeat(np.arange(n, dtype=np.int32), 300)
    dst = rng.integers(0, n, src.size).astype(np.int32)
    g = B.slicegcn_graph_create(n, src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    try:
        assert B.slicegcn_spmm_workspace_bytes(g, 256) > 8 << 20
        X = torch.zeros((n, 256), device="cuda"); Y = torch.zeros_like(X)
        with pytest.raises(B.SliceGCNError) as e:
            B.slicegcn_spmm_static_scratch(g, 0, B.F32, B.F32, X, 256, Y, 256, 256, None)
        assert e.value.status == B.ERR_UNSUPPORTED and "8388608" in str(e.value)
        # a width that fits still works on the same graph
        assert B.slicegcn_spmm_workspace_bytes(g, 16) <= 8 << 20
        X = torch.ones((n, 16), device="cuda"); Y = torch.empty_like(X); W = torch.empty_like(X)
        wsb = B.slicegcn_spmm_workspace_bytes(g, 16); ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        B.slicegcn_spmm(g, 0, B.F32, B.F32, X, 16, W, 16, 16, ws, wsb, None)
        B.slicegcn_spmm_static_scratch(g, 0, B.F32, B.F32, X, 16, Y, 16, 16, None)
        torch.cuda.synchronize()
        assert torch.equal(Y, W)
    finally:
        B.slicegcn_graph_destroy(g)
