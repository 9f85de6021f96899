"""The exchange steps of `slicegcn_train_epoch_sliced` over torch.distributed (Section IV-A / Eq. 8 of the paper:
each process computes a range of the feature slices and the slice outputs meet once, for the concatenation).

The library calls back with raw addresses; this module views them as tensors (no copy), runs one collective per
call -- an all-gather of column blocks for the slice outputs, a sum for the two gradient exchanges -- and returns.
NCCL for device buffers, gloo for host buffers (the CPU tests drive the callbacks with host arrays).  No kernel of
the library waits on another process: the collectives are ordinary stream-ordered library calls between launches.
"""
from __future__ import annotations

import contextlib
import ctypes
from typing import Callable, Optional

import numpy as np
import torch
import torch.distributed as dist

from . import binding as B

_NP = {B.F32: np.float32, B.BF16: np.uint16}           # bf16 travels as 16-bit words and is re-viewed
_TORCH = {B.F32: torch.float32, B.BF16: torch.bfloat16}


class _CudaView:
    """A device range as an object torch.as_tensor can wrap without copying."""

    def __init__(self, address: int, n_elems: int, typestr: str):
        self.__cuda_array_interface__ = {"shape": (n_elems,), "typestr": typestr, "data": (address, False), "version": 3}


def view_buffer(address: int, n_elems: int, dtype: int, device: str) -> torch.Tensor:
    """1-D tensor over `n_elems` elements of the library's `dtype` at `address` (host or device memory)."""
    if device == "cpu":
        npdt = _NP[dtype]
        raw = (ctypes.c_char * (n_elems * np.dtype(npdt).itemsize)).from_address(address)
        t = torch.from_numpy(np.frombuffer(raw, dtype=npdt))
    else:
        t = torch.as_tensor(_CudaView(address, n_elems, "<f4" if dtype == B.F32 else "<i2"), device=device)
    return t.view(_TORCH[dtype]) if dtype == B.BF16 else t


def slice_ranges(p: int, world: int):
    """Equal ranges of the p slices, one per process (p must be a multiple of the number of processes)."""
    if p % world:
        raise ValueError(f"{p} slices do not divide among {world} processes")
    k = p // world
    return [(r * k, (r + 1) * k) for r in range(world)]


def make_exchange(group=None, device: str = "cuda") -> Callable:
    """The callable `binding.slicegcn_train_epoch_sliced` takes as `exchange`, for the processes of `group`.

    Every process must hold an equal share of the columns in the gather step (see `slice_ranges`)."""
    world = dist.get_world_size(group)

    def on_stream(stream_address: Optional[int]):
        if device == "cpu":
            return contextlib.nullcontext()
        s = torch.cuda.ExternalStream(stream_address) if stream_address else torch.cuda.default_stream()
        return torch.cuda.stream(s)   # the collective is ordered after the kernels the library queued on its stream

    def exchange(what: int, buf: int, rows: int, ld: int, col0: int, cols: int, dtype: int, stream) -> int:
        with on_stream(stream):
            if what == B.EXCHANGE_SUM_GRADS:
                flat = view_buffer(buf, rows, dtype, device)
                dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
                return B.OK
            full = view_buffer(buf, rows * ld, dtype, device).view(rows, ld)
            if what == B.EXCHANGE_SUM_DXFF:
                part = full[:, col0:col0 + cols].contiguous()
                dist.all_reduce(part, op=dist.ReduceOp.SUM, group=group)
                full[:, col0:col0 + cols].copy_(part)
                return B.OK
            if what == B.EXCHANGE_GATHER_H:
                mine = full[:, col0:col0 + cols].contiguous()
                blocks = [torch.empty_like(mine) for _ in range(world)]
                dist.all_gather(blocks, mine, group=group)   # process r owns columns [r * cols, (r + 1) * cols)
                for r, blk in enumerate(blocks):
                    full[:, r * cols:(r + 1) * cols].copy_(blk)
                return B.OK
        return B.ERR_INVALID_ARG

    return exchange
