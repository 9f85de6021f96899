"""The exchange steps of the slices-on-separate-processes epoch (Section IV-A, Eq. 8), two gloo processes on CPU.

The library hands its exchange function raw addresses; here the addresses are those of host arrays laid out as the
library's buffers are (the slice outputs with a leading dimension, the fused-input gradient, the flat gradient
vector), so the packing, the collectives and the write-back of `slice_exchange.make_exchange` run exactly as they
would between GPUs, without one."""
import json
import os
import socket
import subprocess
import sys
import textwrap

import pytest

from conftest import ROOT


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_slice_ranges():
    from paper_2408_11500_b200 import slice_exchange as sx
    assert sx.slice_ranges(8, 2) == [(0, 4), (4, 8)]
    assert sx.slice_ranges(3, 3) == [(0, 1), (1, 2), (2, 3)]
    assert sx.slice_ranges(4, 1) == [(0, 4)]
    with pytest.raises(ValueError):
        sx.slice_ranges(8, 3)


def test_exchange_steps_two_gloo_processes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(textwrap.dedent("""
        import os, sys, json
        import numpy as np
        import torch, torch.distributed as dist
        sys.path.insert(0, os.getcwd())
        from paper_2408_11500_b200 import binding as B, slice_exchange as sx
        rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
        dist.init_process_group("gloo", rank=rank, world_size=world)
        ex = sx.make_exchange(None, device="cpu")
        rows, p, h_s, ld = 37, 4, 6, 32                      # 4 slices of 6 columns, rows padded to 32 columns
        (s0, s1), = [sx.slice_ranges(p, world)[rank]]
        truth = np.arange(rows * p * h_s, dtype=np.float32).reshape(rows, p * h_s) * 0.5 - 100.0
        out = {}
        # Eq. 8: every process holds its own column block, garbage elsewhere; afterwards all columns everywhere
        for name, dt in (("f32", B.F32), ("bf16", B.BF16)):
            if dt == B.F32:
                H = np.full((rows, ld), -7.0, np.float32)
                H[:, s0 * h_s:s1 * h_s] = truth[:, s0 * h_s:s1 * h_s]
                want = truth
            else:   # bf16 bit patterns travel as 16-bit words
                words = (truth.view(np.uint32) >> 16).astype(np.uint16)
                H = np.full((rows, ld), 0x7fc0, np.uint16)
                H[:, s0 * h_s:s1 * h_s] = words[:, s0 * h_s:s1 * h_s]
                want = words
            rc = ex(B.EXCHANGE_GATHER_H, H.ctypes.data, rows, ld, s0 * h_s, (s1 - s0) * h_s, dt, None)
            out["gather_" + name] = bool(rc == 0 and np.array_equal(H[:, :p * h_s], want))
            out["gather_pad_" + name] = bool(np.array_equal(H[:, p * h_s:], np.full((rows, ld - p * h_s), H[0, -1])))
        # the fused input's gradient: partial sums over each process's slices, 13 columns in rows of 16
        part = np.zeros((rows, 16), np.float32)
        part[:, :13] = (rank + 1) * np.arange(rows * 13, dtype=np.float32).reshape(rows, 13)
        part[:, 13:] = -7.0                                   # padding is not touched
        rc = ex(B.EXCHANGE_SUM_DXFF, part.ctypes.data, rows, 16, 0, 13, B.F32, None)
        tot = sum(r + 1 for r in range(world))
        out["dxff"] = bool(rc == 0 and np.array_equal(part[:, :13], tot * np.arange(rows * 13, dtype=np.float32).reshape(rows, 13))
                           and (part[:, 13:] == -7.0).all())
        # the flat gradient vector: per-slice blocks on their owners, replicated tensors on the first process only
        grads = np.zeros(1000, np.float32)
        grads[100 * rank:100 * rank + 100] = rank + 1.0      # a per-slice tensor's block
        if rank == 0:
            grads[900:] = 3.0                                # a replicated tensor
        rc = ex(B.EXCHANGE_SUM_GRADS, grads.ctypes.data, 1000, 1, 0, 1, B.F32, None)
        want_g = np.zeros(1000, np.float32)
        for r in range(world):
            want_g[100 * r:100 * r + 100] = r + 1.0
        want_g[900:] = 3.0
        out["grads"] = bool(rc == 0 and np.array_equal(grads, want_g))
        out["bad"] = ex(99, grads.ctypes.data, 1, 1, 0, 1, B.F32, None) != 0
        print(json.dumps(out))
        dist.destroy_process_group()
    """))
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                                      text=True, cwd=ROOT))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    for o in outs:
        res = json.loads(o[0].strip().splitlines()[-1])
        assert all(res.values()), res
