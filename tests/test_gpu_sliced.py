"""The paper's own placement (Section IV-A, Eq. 8): each process computes a range of the slices and the slice
outputs meet once.  `slicegcn_train_epoch_sliced` on ONE GPU: the processes are emulated one after the other, and
because the epoch is deterministic an exchange step can be answered from what the other emulated processes produced
in an earlier, aborted replay of the same epoch -- no kernel here ever waits for another process.  The result must be
the single-process epoch (which the other tests hold against the oracle)."""
import numpy as np
import pytest

from helpers import GpuProblem, small_problem, rel_inf
from paper_2408_11500_b200 import slice_exchange as sx

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2408_11500_b200 import binding
    return binding


def _run_emulated(B, gps, ranges, opt_of):
    """All replays of one epoch for the emulated processes `gps` (one GpuProblem each, identical state).  Returns
    nothing: every GpuProblem ends with its updated parameters, gradients, logits and loss."""
    import torch
    world = len(gps)
    stages = [B.EXCHANGE_GATHER_H, B.EXCHANGE_SUM_DXFF, B.EXCHANGE_SUM_GRADS]
    saved = {}                                   # (stage, rank) -> this process's contribution
    use_ff = bool(gps[0].kw.get("use_ff", False))
    plan = [s for s in stages if s != B.EXCHANGE_SUM_DXFF or use_ff]
    init = [(gp.params.clone(), gp.m1.clone(), gp.m2.clone()) for gp in gps]
    for depth in range(len(plan) + 1):           # replay `depth` answers its first `depth` exchanges, aborts at the next
        for r, gp in enumerate(gps):
            gp.params.copy_(init[r][0]); gp.m1.copy_(init[r][1]); gp.m2.copy_(init[r][2])
            seen = []

            def exchange(what, buf, rows, ld, col0, cols, dtype, stream, r=r, seen=seen):
                k = plan.index(what)
                seen.append(what)
                n_el = rows if what == B.EXCHANGE_SUM_GRADS else rows * ld
                t = sx.view_buffer(buf, n_el, dtype, "cuda")
                if what != B.EXCHANGE_SUM_GRADS:
                    t = t.view(rows, ld)
                if k == depth:                   # contribute and stop this replay
                    saved[(what, r)] = (t[:, col0:col0 + cols].clone() if what != B.EXCHANGE_SUM_GRADS else t.clone(), col0, cols)
                    return B.ERR_UNSUPPORTED
                if what == B.EXCHANGE_GATHER_H:
                    for q in range(world):
                        blk, c0, cw = saved[(what, q)]
                        t[:, c0:c0 + cw].copy_(blk)
                elif what == B.EXCHANGE_SUM_DXFF:
                    acc = saved[(what, 0)][0].clone()
                    for q in range(1, world):
                        acc += saved[(what, q)][0]       # fixed order: the sum every process would get from the collective
                    t[:, col0:col0 + cols].copy_(acc)
                else:
                    acc = saved[(what, 0)][0].clone()
                    for q in range(1, world):
                        acc += saved[(what, q)][0]
                    t.copy_(acc)
                return B.OK

            s0, s1 = ranges[r]
            try:
                B.slicegcn_train_epoch_sliced(gp.m, gp.g, gp.X, gp.X.shape[1], gp.y, gp.train_idx,
                                              0 if gp.train_idx is None else gp.train_idx.numel(), gp.params, gp.grads,
                                              gp.m1, gp.m2, opt_of(), s0, s1, exchange, gp.logits, gp.loss, gp.ws, gp.ws_bytes,
                                              torch.cuda.current_stream().cuda_stream)
                finished = True
            except B.SliceGCNError as e:
                assert e.status == B.ERR_UNSUPPORTED, e
                finished = False
            torch.cuda.synchronize()
            assert finished == (depth == len(plan)), (depth, r, seen)
            assert seen == plan[:depth + 1] if depth < len(plan) else seen == plan


CASES = [
    (dict(p=4, in_d=64, hidden=64, C=8, n=1111), 2),                                            # direct slicing, two processes
    (dict(p=4, in_d=64, hidden=64, C=8, n=1111, use_se=True, use_b_self=True), 4),              # one slice per process
    (dict(p=4, in_d=37, hidden=64, C=5, n=900, L=3), 2),                                        # repacked input slices
    (dict(p=8, in_d=100, hidden=256, C=47, L=3, n=1400, use_ff=True, use_se=True), 2),          # fused input shared by all slices
    (dict(p=8, in_d=100, hidden=256, C=47, L=2, n=900, use_ff=True), 8),
    (dict(p=4, in_d=64, hidden=64, C=8, n=1111, order=2), 2),                                   # transform-first layers
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("kw,world", CASES)
def test_sliced_epoch_equals_single_process_epoch(B, kw, world, dtype):
    kw = dict(kw)
    order = kw.pop("order", 0)
    src, dst, X, y, mk, od, params = small_problem(**kw)
    mk["order"] = order
    if dtype == "bf16":
        mk["dtype"] = B.BF16
    train_idx = np.arange(0, len(X), 3).astype(np.int32)
    opt_of = lambda: B.OptDesc(1e-3, 0.9, 0.999, 1e-8, 0.0, 2, 10)
    ref = GpuProblem(len(X), src, dst, X, y, params, train_idx=train_idx, **mk)
    gps = [GpuProblem(len(X), src, dst, X, y, params, train_idx=train_idx, **mk) for _ in range(world)]
    try:
        loss_ref = ref.epoch(opt_of())
        _run_emulated(B, gps, sx.slice_ranges(mk["num_slices"], world), opt_of)
        # fp32: the same kernels on the same values; only sums that now form in two steps (the fused input's gradient,
        # weight gradients whose row chunks depend on the number of groups) may differ in rounding order
        tol = 2e-5 if dtype == "f32" else 2e-2
        g_ref, p_ref = ref.named_grads(), ref.named_params()
        for gp in gps:
            assert abs(float(gp.loss.item()) - loss_ref) <= 1e-6 * max(1.0, abs(loss_ref))
            assert rel_inf(gp.logits.cpu().numpy(), ref.logits.cpu().numpy()) <= 1e-6
            g, pr = gp.named_grads(), gp.named_params()
            for k in g_ref:
                assert rel_inf(g[k], g_ref[k]) <= tol, (k, rel_inf(g[k], g_ref[k]))
                assert np.abs(pr[k] - p_ref[k]).max() <= 2.5e-3, k   # one Adam step of 1e-3
        # every process ends with the same parameters as every other: replicas without having been sent
        for gp in gps[1:]:
            assert np.array_equal(gp.params.cpu().numpy(), gps[0].params.cpu().numpy())
    finally:
        ref.close()
        for gp in gps:
            gp.close()


def test_sliced_epoch_argument_errors(B):
    import torch
    src, dst, X, y, mk, od, params = small_problem(p=4, in_d=64, hidden=64, C=8, n=700)
    gp = GpuProblem(len(X), src, dst, X, y, params, **mk)
    try:
        def call(s0, s1, ex):
            B.slicegcn_train_epoch_sliced(gp.m, gp.g, gp.X, gp.X.shape[1], gp.y, None, 0, gp.params, gp.grads, gp.m1, gp.m2,
                                          None, s0, s1, ex, gp.logits, gp.loss, gp.ws, gp.ws_bytes,
                                          torch.cuda.current_stream().cuda_stream)
        for bad in ((0, 5), (-1, 2), (2, 2), (3, 1)):
            with pytest.raises(B.SliceGCNError) as e:
                call(bad[0], bad[1], lambda *a: 0)
            assert e.value.status == B.ERR_INVALID_ARG
        with pytest.raises(B.SliceGCNError) as e:
            call(0, 2, None)                     # a partial range without an exchange function
        assert e.value.status == B.ERR_INVALID_ARG
        call(0, 4, None)                         # the whole range is the ordinary epoch
        torch.cuda.synchronize()
        whole = gp.grads.clone()
        gp.epoch(None)
        assert torch.equal(whole, gp.grads)
    finally:
        gp.close()
    # per-slice widths that need the padded internal layout are refused (p = 3 of hidden 100 -> 34 columns)
    src, dst, X, y, mk, od, params = small_problem(p=3, in_d=48, hidden=100, C=6, n=700)
    gp = GpuProblem(len(X), src, dst, X, y, params, **mk)
    try:
        with pytest.raises(B.SliceGCNError) as e:
            B.slicegcn_train_epoch_sliced(gp.m, gp.g, gp.X, gp.X.shape[1], gp.y, None, 0, gp.params, gp.grads, gp.m1, gp.m2,
                                          None, 0, 1, lambda *a: 0, gp.logits, gp.loss, gp.ws, gp.ws_bytes,
                                          torch.cuda.current_stream().cuda_stream)
        assert e.value.status == B.ERR_UNSUPPORTED
    finally:
        gp.close()


def test_exchange_on_device_buffers_single_process_group(B):
    """`slice_exchange.make_exchange` on device memory: the address views (fp32 and bf16), the stream hand-over and the
    NCCL calls, in a process group of one (the only size one GPU allows): every step must leave the data as it is."""
    import socket
    import torch
    import torch.distributed as dist
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        ex = sx.make_exchange(None, device="cuda")
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            H = torch.randn(300, 40, device="cuda")
            Hb = torch.randn(300, 40, device="cuda").to(torch.bfloat16)
            d = torch.randn(300, 16, device="cuda")
            gvec = torch.randn(5000, device="cuda")
            keep = [t.clone() for t in (H, Hb, d, gvec)]
            assert ex(B.EXCHANGE_GATHER_H, H.data_ptr(), 300, 40, 0, 32, B.F32, st.cuda_stream) == B.OK
            assert ex(B.EXCHANGE_GATHER_H, Hb.data_ptr(), 300, 40, 0, 32, B.BF16, st.cuda_stream) == B.OK
            assert ex(B.EXCHANGE_SUM_DXFF, d.data_ptr(), 300, 16, 0, 13, B.F32, st.cuda_stream) == B.OK
            assert ex(B.EXCHANGE_SUM_GRADS, gvec.data_ptr(), 5000, 1, 0, 1, B.F32, st.cuda_stream) == B.OK
        st.synchronize()
        for a, b in zip((H, Hb, d, gvec), keep):
            assert torch.equal(a, b)
    finally:
        dist.destroy_process_group()
