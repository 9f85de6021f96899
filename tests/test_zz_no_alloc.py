"""The allocation-free aggregation entry point (slicegcn_spmm_static_scratch).

Who needs it: code that runs where device allocation is off limits -- inside a stream capture, on a host
whose device memory is planned once at start-up, or in a plugin that may not touch its host's allocator.
It must give exactly what slicegcn_spmm gives, call after call, with the hub-row scratch coming from the
buffer compiled into the library, and it must refuse (not overrun) a problem that needs more than that buffer.
Collected last on purpose: a failure here must not hide the results of the other GPU tests.
"""
import numpy as np
import pytest

from oracle import slicegcn_oracle as orc
from paper_2408_11500_b200 import synth

pytestmark = pytest.mark.gpu


def _graph_with_hubs(B, n=6000, m=40000, max_degree=2500, seed=7):
    src, dst = synth.chung_lu_powerlaw(n, m, 2.2, max_degree, seed=seed)
    g = B.slicegcn_graph_create(n, src, dst, B.SYMMETRIZE | B.ADD_SELF_LOOPS)
    assert B.slicegcn_graph_info(g)["n_segments"] > 0        # the path that needs scratch is exercised
    return g, n, orc.build_graph(n, src, dst, True, True)


@pytest.mark.parametrize("dtype,width", [("f32", 128), ("f32", 72), ("bf16", 256)])
def test_static_scratch_matches_workspace_entry_point_twice(dtype, width):
    import torch
    from paper_2408_11500_b200 import binding as B
    g, n, og = _graph_with_hubs(B)
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
            # and against the definition itself (the CPU oracle), not only against the sibling entry point
            ref = orc.spmm(og, X.float().cpu().numpy().astype(np.float64))
            if dtype == "f32":
                assert np.abs(a - ref).max() <= 2e-6 * np.abs(ref).max()
            else:
                assert np.all(np.abs(a - ref) <= 2 ** -8 * np.abs(ref) + 1e-5 * np.abs(ref).max())
        assert B.slicegcn_graph_device_status(g) == 0
    finally:
        B.slicegcn_graph_destroy(g)


def test_static_scratch_transposed_directed_graph_and_no_allocation():
    """A directed graph (its transpose has its own hub rows): the transposed aggregation through the built-in buffer
    matches the oracle, and the calls leave the device's free memory and torch's allocator exactly as they were."""
    import torch
    from paper_2408_11500_b200 import binding as B
    rng = np.random.default_rng(3)
    n = 4000
    src = rng.integers(0, n, 40000).astype(np.int32); dst = rng.integers(0, n, 40000).astype(np.int32)
    dst[:900] = 11                                           # a long column -> a long row of the transpose
    og = orc.build_graph(n, src, dst, False, False)
    g = B.slicegcn_graph_create(n, src, dst, 0)
    try:
        assert not B.slicegcn_graph_info(g)["symmetric"]
        X = torch.from_numpy(synth.gaussian_features(n, 64, seed=9)).cuda()
        Y = torch.empty_like(X)
        B.slicegcn_spmm_static_scratch(g, 1, B.F32, B.F32, X, 64, Y, 64, 64, None)   # the first call looks the buffer up
        torch.cuda.synchronize()
        import gc
        gc.collect()                # tensors of earlier tests that only a reference cycle keeps alive go now, not mid-measurement
        free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        for transpose in (1, 0, 1):
            B.slicegcn_spmm_static_scratch(g, transpose, B.F32, B.F32, X, 64, Y, 64, 64, None)
            torch.cuda.synchronize()
            ref = orc.spmm(og, X.cpu().numpy().astype(np.float64), transpose=bool(transpose))
            assert np.abs(Y.cpu().numpy() - ref).max() <= 2e-6 * np.abs(ref).max()
        assert torch.cuda.mem_get_info()[0] == free0
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
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
