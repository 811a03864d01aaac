"""Host-buffer entry points: the calls a user with gradients in (pinned) host memory makes.

Each call stages its inputs to the device on a copy stream, runs the CUDA compression through the
C ABI on torch's current stream, and returns the compressed rows in host memory.  Copies of the next
chunk overlap the kernels of the current one (two device staging slots).  Only marshalling and copies
happen here; every step of the compression runs in the kernels.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B


def _pinned_like(shape, dtype) -> torch.Tensor:
    return torch.empty(shape, dtype=dtype, pin_memory=True)


def grass_compress_host(g_chunks: Sequence[torch.Tensor], idx: np.ndarray, k: int, s: int, seed: int,
                        out_host: Optional[torch.Tensor] = None, device="cuda") -> torch.Tensor:
    """GraSS over host-resident gradients given as a sequence of (rows_i, p) host tensors (pinned for
    asynchronous copies; the same tensor may appear several times).  Returns the (sum rows_i, k) fp32
    result in pinned host memory.  H2D bytes = all chunks, D2H bytes = the result."""
    n = sum(int(c.shape[0]) for c in g_chunks)
    if out_host is None:
        out_host = _pinned_like((n, k), torch.float32)
    didx = None if idx is None else B.mask_to_device(idx, device)
    cur = torch.cuda.current_stream()
    copy = torch.cuda.Stream()
    max_rows = max(int(c.shape[0]) for c in g_chunks)
    p = int(g_chunks[0].shape[1])
    slots = [torch.empty((max_rows, p), dtype=g_chunks[0].dtype, device=device) for _ in range(2)]
    outs = [torch.empty((max_rows, k), dtype=torch.float32, device=device) for _ in range(2)]
    ready = [torch.cuda.Event() for _ in range(2)]
    freed = [torch.cuda.Event() for _ in range(2)]
    copy.wait_stream(cur)

    def stage(i):
        sl = i % 2
        with torch.cuda.stream(copy):
            if i >= 2:
                copy.wait_event(freed[sl])
            slots[sl][: g_chunks[i].shape[0]].copy_(g_chunks[i], non_blocking=True)
            ready[sl].record(copy)

    stage(0)
    row = 0
    for i, c in enumerate(g_chunks):
        sl = i % 2
        if i + 1 < len(g_chunks):
            stage(i + 1)
        rows = int(c.shape[0])
        cur.wait_event(ready[sl])
        B.grass_compress(slots[sl][:rows], didx, k, s, seed, out=outs[sl][:rows])
        out_host[row:row + rows].copy_(outs[sl][:rows], non_blocking=True)
        freed[sl].record(cur)
        row += rows
    cur.synchronize()
    return out_host


def factgrass_compress_host(groups: Sequence[Sequence[dict]], Bsz: int, T: int, out_dim: int,
                            out_host: Optional[torch.Tensor] = None, device="cuda") -> torch.Tensor:
    """FactGraSS over host-resident layer tensors.  ``groups`` is a sequence of layer groups (for
    instance one transformer block each); a layer is a dict with A, G (host tensors, B x T x d, pinned
    for asynchronous copies), mask_in, mask_out (uint32 numpy), k, s, seed, out_offset.  Every group is
    copied to the device and compressed with one grouped launch; the (B, out_dim) fp32 result is
    returned in pinned host memory."""
    if out_host is None:
        out_host = _pinned_like((Bsz, out_dim), torch.float32)
    cur = torch.cuda.current_stream()
    copy = torch.cuda.Stream()
    out_dev = torch.empty((Bsz, out_dim), dtype=torch.float32, device=device)
    max_layers = max(len(g) for g in groups)
    ws = [torch.empty(B.factgrass_grouped_workspace_bytes(max_layers), dtype=torch.uint8, device=device)
          for _ in range(2)]

    # device staging slots sized for the largest group
    def group_elems(g):
        return sum(l["A"].numel() + l["G"].numel() for l in g)

    cap = max(group_elems(g) for g in groups)
    dt = groups[0][0]["A"].dtype
    slots = [torch.empty(cap, dtype=dt, device=device) for _ in range(2)]
    masks = {}

    def dev_mask(m):
        key = (m.ctypes.data, m.size)
        if key not in masks:
            masks[key] = B.mask_to_device(m, device)
        return masks[key]

    ready = [torch.cuda.Event() for _ in range(2)]
    freed = [torch.cuda.Event() for _ in range(2)]
    copy.wait_stream(cur)
    staged: List[Optional[list]] = [None, None]

    def stage(i):
        sl = i % 2
        descs, off = [], 0
        with torch.cuda.stream(copy):
            if i >= 2:
                copy.wait_event(freed[sl])
            for l in groups[i]:
                a = slots[sl][off:off + l["A"].numel()].view(l["A"].shape)
                off += l["A"].numel()
                g = slots[sl][off:off + l["G"].numel()].view(l["G"].shape)
                off += l["G"].numel()
                a.copy_(l["A"], non_blocking=True)
                g.copy_(l["G"], non_blocking=True)
                descs.append(dict(A=a, G=g, mask_in=dev_mask(l["mask_in"]), mask_out=dev_mask(l["mask_out"]),
                                  k=l["k"], s=l["s"], seed=l["seed"], out_offset=l["out_offset"]))
            ready[sl].record(copy)
        staged[sl] = descs

    stage(0)
    for i in range(len(groups)):
        sl = i % 2
        if i + 1 < len(groups):
            stage(i + 1)
        cur.wait_event(ready[sl])
        B.factgrass_compress_grouped(B.GroupedLayers(staged[sl]), out_dev, ws[sl])
        freed[sl].record(cur)
    out_host.copy_(out_dev, non_blocking=True)
    cur.synchronize()
    return out_host


def grass_score_host(train_host: torch.Tensor, test_host: torch.Tensor, device="cuda") -> torch.Tensor:
    """Scores of host-resident compressed vectors; returns the (N, M) result in pinned host memory."""
    tr = train_host.to(device, non_blocking=True)
    te = test_host.to(device, non_blocking=True)
    sc = B.grass_score(tr, te)
    out = _pinned_like(tuple(sc.shape), torch.float32)
    out.copy_(sc, non_blocking=True)
    torch.cuda.current_stream().synchronize()
    return out
