"""Host-buffer entry points: the calls a user with gradients in (pinned) host memory makes.

Two ways in, both through the C ABI on torch's current stream, both returning the compressed rows in host
memory.  Staged: the inputs are copied to the device on a copy stream, the copy of the next chunk overlapping
the kernels of the current one (two device staging slots).  In place (``zero_copy``): the kernels gather the
masked elements straight from the page-locked host buffers, so only the 64-byte pieces the masks touch cross the
bus instead of every byte of the inputs.  Left to choose (``zero_copy=None``), the FactGraSS call decides tensor by
tensor: a factor whose mask touches less than 70 % of its bytes is read in place, a denser one is copied to the
device first, and one grouped launch takes both kinds of pointers.  Only marshalling and copies happen here;
every step of the compression runs in the kernels.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B


def _pinned_like(shape, dtype) -> torch.Tensor:
    return torch.empty(shape, dtype=dtype, pin_memory=True)


# Gathering in place moves 64-byte pieces across the bus at about 0.7 of the rate of a bulk copy (measured: 38
# against 55 GB/s), so it pays when the masks touch less than about this fraction of the input bytes.
IN_PLACE_MAX_FRACTION = 0.7


def touched_fraction(idx: np.ndarray, row_elems: int, elem_bytes: int) -> float:
    """Fraction of a row's bytes that a gather of ``idx`` moves at 64-byte granularity."""
    per = 64 // elem_bytes
    pieces = np.unique(np.asarray(idx, dtype=np.int64) // per).size
    return min(1.0, pieces * 64.0 / (row_elems * elem_bytes))


def grass_in_place(g_chunks: Sequence[torch.Tensor], idx: Optional[np.ndarray]) -> bool:
    """Whether grass_compress_host, left to choose, gathers from the host buffers in place."""
    return (idx is not None and all(c.is_pinned() for c in g_chunks) and
            touched_fraction(idx, int(g_chunks[0].shape[1]), g_chunks[0].element_size()) <= IN_PLACE_MAX_FRACTION)


def factgrass_host_plan(groups: Sequence[Sequence[dict]]):
    """What factgrass_compress_host does when left to choose: per layer (A in place?, G in place?), and the bytes
    that cross the bus (whole tensors that are copied + the 64-byte pieces the masks touch of the others; a host
    count, not a bus counter)."""
    plan, moved = [], 0.0
    for g in groups:
        for l in g:
            dec = []
            for t, m in ((l["A"], l["mask_in"]), (l["G"], l["mask_out"])):
                nbytes = t.numel() * t.element_size()
                frac = touched_fraction(m, int(t.shape[-1]), t.element_size())
                in_place = bool(t.is_pinned() and frac <= IN_PLACE_MAX_FRACTION)
                moved += nbytes * (frac if in_place else 1.0)
                dec.append(in_place)
            plan.append(tuple(dec))
    return plan, int(moved)


def factgrass_in_place(groups: Sequence[Sequence[dict]]) -> bool:
    """Whether factgrass_compress_host, left to choose, reads at least one tensor in place."""
    plan, _ = factgrass_host_plan(groups)
    return any(a or g for a, g in plan)


def grass_compress_host(g_chunks: Sequence[torch.Tensor], idx: np.ndarray, k: int, s: int, seed: int,
                        out_host: Optional[torch.Tensor] = None, device="cuda",
                        zero_copy: Optional[bool] = None) -> torch.Tensor:
    """GraSS over host-resident gradients given as a sequence of (rows_i, p) host tensors (pinned for
    asynchronous copies; the same tensor may appear several times).  Returns the (sum rows_i, k) fp32
    result in pinned host memory.  Staged: H2D bytes = all chunks; in place: the pieces the mask touches.
    D2H bytes = the result.  The identity mask (idx None) reads everything and is always staged."""
    n = sum(int(c.shape[0]) for c in g_chunks)
    if out_host is None:
        out_host = _pinned_like((n, k), torch.float32)
    didx = None if idx is None else B.mask_to_device(idx, device)
    cur = torch.cuda.current_stream()
    if zero_copy is None:
        zero_copy = grass_in_place(g_chunks, idx)
    if zero_copy:
        out_dev = torch.empty((n, k), dtype=torch.float32, device=device)
        row = 0
        for c in g_chunks:
            rows = int(c.shape[0])
            B.grass_compress(c, didx, k, s, seed, out=out_dev[row:row + rows])
            row += rows
        out_host.copy_(out_dev, non_blocking=True)
        cur.synchronize()
        return out_host
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
                            out_host: Optional[torch.Tensor] = None, device="cuda",
                            zero_copy: Optional[bool] = None) -> torch.Tensor:
    """FactGraSS over host-resident layer tensors.  ``groups`` is a sequence of layer groups (for
    instance one transformer block each); a layer is a dict with A, G (host tensors, B x T x d, pinned
    for asynchronous copies), mask_in, mask_out (uint32 numpy), k, s, seed, out_offset.  Staged: every
    group is copied to the device and compressed with one grouped launch.  In place: all layers go into
    grouped launches that gather from the pinned host tensors directly.  The (B, out_dim) fp32 result is
    returned in pinned host memory."""
    if out_host is None:
        out_host = _pinned_like((Bsz, out_dim), torch.float32)
    cur = torch.cuda.current_stream()
    out_dev = torch.empty((Bsz, out_dim), dtype=torch.float32, device=device)
    masks = {}

    def dev_mask(m):
        key = (m.ctypes.data, m.size)
        if key not in masks:
            masks[key] = B.mask_to_device(m, device)
        return masks[key]

    if zero_copy is None:
        plan, _ = factgrass_host_plan(groups)
        zero_copy = any(a or g for a, g in plan)
    elif zero_copy:
        plan = [(True, True) for g in groups for l in g]
    if zero_copy:
        # tensors that are not read in place are copied to the device first (same stream: the kernels that gather
        # across the bus would compete with the copies for it anyway)
        def operand(t, in_place):
            return t if in_place else t.to(device, non_blocking=True)
        layers = [l for g in groups for l in g]
        flat = [dict(A=operand(l["A"], pa), G=operand(l["G"], pg), mask_in=dev_mask(l["mask_in"]),
                     mask_out=dev_mask(l["mask_out"]), k=l["k"], s=l["s"], seed=l["seed"], out_offset=l["out_offset"])
                for l, (pa, pg) in zip(layers, plan)]
        per_call = 256
        wsz = torch.empty(B.factgrass_grouped_workspace_bytes(min(per_call, len(flat))), dtype=torch.uint8,
                          device=device)
        for i in range(0, len(flat), per_call):
            B.factgrass_compress_grouped(B.GroupedLayers(flat[i:i + per_call]), out_dev, wsz)
        out_host.copy_(out_dev, non_blocking=True)
        cur.synchronize()
        return out_host
    copy = torch.cuda.Stream()
    max_layers = max(len(g) for g in groups)
    ws = [torch.empty(B.factgrass_grouped_workspace_bytes(max_layers), dtype=torch.uint8, device=device)
          for _ in range(2)]

    # device staging slots sized for the largest group
    def group_elems(g):
        return sum(l["A"].numel() + l["G"].numel() for l in g)

    cap = max(group_elems(g) for g in groups)
    dt = groups[0][0]["A"].dtype
    slots = [torch.empty(cap, dtype=dt, device=device) for _ in range(2)]

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
