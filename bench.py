#!/usr/bin/env python
"""Benchmark of the GraSS / FactGraSS compression hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config {1..5}] [--impl ours|reference]

Prints ONE JSON line.  The default workload is config 5: FactGraSS over the 224 linear layers of a
Llama-3-8B-shaped model (B=4 x T=2048 bf16, k'=64x64, k=4096 per layer) followed by grass_score of
16,384 x 256 compressed vectors -- the configuration the paper's headline throughput (Table 2) is
shaped like.  A step is one pass of the whole path over one batch.  Inputs are seeded and synthetic.

--impl reference times the CPU oracle (plain C, fp64), as it stands, on a bounded sample.
With N > 1 (torchrun) every rank runs an independent replica of the workload: the path does not shard.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "per-sample gradients compressed/sec"
UNIT = "samples/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 1024 * 1024
L2_FLUSHED = "L2 flushed between steps (252 MB written)"


# ----------------------------------------------------------------------------- plumbing

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            # the tool needs a moment to start: wait for its first line so that a short timed region is covered
            t_end = time.time() + 3.0
            while time.time() < t_end and os.path.getsize(self.path) == 0 and self.proc.poll() is None:
                time.sleep(0.01)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for ln in open(self.path):
                f = [x.strip() for x in ln.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    mx.append(float(f[1]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend)
    return world, rank, local


def max_over_ranks(value: float, world: int, device) -> float:
    """Largest `value` over all ranks (a rank's timing counts only as the slowest one)."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


class L2Flush:
    """Evicts the inputs from L2 between timed steps by writing a buffer of twice the L2 size.  That leaves L2
    full of modified lines, which the next step has to write back; `clean=True` reads another buffer of the same
    size afterwards, so that L2 holds only unmodified lines (reported beside the default: on B200 the two differ
    by a few microseconds in either direction)."""

    def __init__(self, device):
        self.w = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
        self.r = torch.zeros(2 * L2_BYTES // 8, dtype=torch.int64, device=device)
        self.sink = None

    def __call__(self, clean=False):
        self.w.zero_()
        if clean:
            self.sink = self.r.sum()


# ----------------------------------------------------------------------------- workloads (GPU arm)

def sector_bytes_per_row(idx: np.ndarray, elem_bytes: int, gran: int = 32) -> int:
    """Bytes of one row that a gather of `idx` must move at `gran`-byte granularity (32 = L2 sector, the
    algorithmic figure; 64 = the smallest piece a B200 load can make DRAM deliver, with the L2::64B
    prefetch-size hint the gather kernels use; without the hint it is the whole 128-byte line)."""
    per = gran // elem_bytes
    return int(np.unique(idx.astype(np.int64) // per).size) * gran


class GrassJob:
    """configs 1-2: n samples in batches through grass_compress."""

    def __init__(self, cfg, device, G, W):
        self.cfg, self.G, self.device = cfg, G, device
        self.idx = G.grass_random_mask_host(cfg.p, cfg.kprime, cfg.mask_seed)
        self.didx = G.mask_to_device(self.idx, device)
        self.nbatch = cfg.n // cfg.batch
        batch_bytes = cfg.batch * cfg.p * 4
        # distinct resident batches: enough that a batch is out of L2 when it is read again
        self.ncopies = 1 if batch_bytes > 4 * L2_BYTES else min(8, max(2, (4 * L2_BYTES) // batch_bytes + 1))
        self.g = [W.dense_gradients(cfg.batch, cfg.p, cfg.zero_prob, cfg.dist, cfg.scale, cfg.data_seed + c,
                                    device=device) for c in range(self.ncopies)]
        self.out = torch.empty((cfg.batch, cfg.k), dtype=torch.float32, device=device)
        self.samples_per_step = cfg.n
        self.alg_bytes_per_launch = cfg.batch * sector_bytes_per_row(self.idx, 4) + cfg.batch * cfg.k * 4
        self.fetch_bytes_per_launch = cfg.batch * sector_bytes_per_row(self.idx, 4, 64) + cfg.batch * cfg.k * 4
        self.dense_bytes_per_launch = batch_bytes
        self.launches_per_step = self.nbatch
        # one kernel per call: with these shapes the position splits of a row are reduced inside a cluster (config 2)
        # or a thread block owns a whole row (config 1), so there is no zero-fill before the compress kernel
        self.kernels_per_step = self.nbatch
        self.dominant = "grass_compress_kernel"
        self.l2 = (f"{self.ncopies} resident batch(es) of {batch_bytes / 1e6:.0f} MB rotated; "
                   + ("input >> L2" if self.ncopies == 1 else L2_FLUSHED))
        self.need_flush = self.ncopies > 1
        self._i = 0

    def step(self, ev=None):
        c = self.cfg
        for b in range(self.nbatch):
            g = self.g[self._i % self.ncopies]
            self._i += 1
            self.G.grass_compress(g, self.didx, c.k, c.s, c.hash_seed, out=self.out)

    def dominant_ms(self, step_ms):
        return step_ms / self.nbatch

    def desc(self):
        c = self.cfg
        return {"workload": c.name, "n": c.n, "batch": c.batch, "p": c.p, "kprime": c.kprime, "k": c.k, "s": c.s,
                "l2": self.l2}


class FactJob:
    """configs 3-5: all layers through one factgrass_compress_grouped launch (+ score for config 5)."""

    def __init__(self, cfg, device, G, W, seq_len_aware=False, fp32_inputs=False, precondition=False, out_bf16=False):
        self.cfg, self.G, self.device = cfg, G, device
        self.out_bf16 = out_bf16
        self.fp32 = fp32_inputs
        eb = 4 if fp32_inputs else 2
        layers, alg, line = [], 0, 0
        self.tok_count = None
        tokens = cfg.B * cfg.T
        self.dense = 0
        self.host_masks = []
        for l, lay in enumerate(cfg.layers):
            A, Gt = W.layer_io(cfg, l, device=device, dtype=torch.float32 if fp32_inputs else torch.bfloat16)
            s_in, s_out = W.layer_mask_seeds(cfg, l)
            mi = G.grass_random_mask_host(lay.d_in, cfg.kin, s_in)
            mo = G.grass_random_mask_host(lay.d_out, cfg.kout, s_out)
            self.host_masks.append((mi, mo))
            if seq_len_aware and self.tok_count is None:
                # per-sample lengths = tokens before the trailing padding (rows of G that are all zero)
                self.tok_count = (Gt.abs().amax(dim=2) > 0).int().sum(dim=1).int().contiguous()
                tokens = int(self.tok_count.sum().item())
            layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi, device), mask_out=G.mask_to_device(mo, device),
                               k=cfg.k, s=cfg.s, seed=W.layer_hash_seed(cfg, l), out_offset=l * cfg.k))
            alg += tokens * (sector_bytes_per_row(mi, eb) + sector_bytes_per_row(mo, eb)) + cfg.B * cfg.k * 4
            line += tokens * (sector_bytes_per_row(mi, eb, 64) + sector_bytes_per_row(mo, eb, 64)) + cfg.B * cfg.k * 4
            self.dense += cfg.B * cfg.T * (lay.d_in + lay.d_out) * eb
        self.layers = layers
        self.group = G.GroupedLayers(layers)
        self.out = torch.empty((cfg.B, cfg.out_dim), dtype=torch.bfloat16 if out_bf16 else torch.float32, device=device)
        self.ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(layers)), dtype=torch.uint8, device=device)
        self.score = None
        if cfg.score_n_train:
            self.score = W.score_vectors(cfg.score_n_train, cfg.score_n_test, cfg.k, cfg.data_seed + 7, device=device)
            self.score_out = torch.empty((cfg.score_n_train, cfg.score_n_test), dtype=torch.float32, device=device)
        # --precondition: the attribute stage with the damped inverse of the projected FIM of the train vectors
        # (one layer block): F = train^T train / n, Cholesky of F + lambda I, solve for the test rows, then scores
        self.precondition = bool(precondition and self.score)
        if self.precondition:
            self.fim = torch.empty((cfg.k, cfg.k), dtype=torch.float32, device=device)
            self.test_pre = torch.empty_like(self.score[1])
        self.samples_per_step = cfg.B
        self.alg_bytes_per_launch = alg
        self.fetch_bytes_per_launch = line
        self.dense_bytes_per_launch = self.dense
        self.launches_per_step = 1
        nb = (cfg.k + 63) // 64
        # the grouped call is one kernel when it takes the cluster kernel (few (layer, sample) items: config 3), else a
        # zero-fill kernel and the streaming kernel (the library's rule: items <= thread-block slots of one wave)
        items, slots = len(cfg.layers) * cfg.B, 148 * (1 if max(cfg.kin, cfg.kout) > 64 else 2)
        fact_kernels = 1 if (items <= slots and not fp32_inputs and max(cfg.kin, cfg.kout) <= 128) else 2
        self.kernels_per_step = fact_kernels + (1 if self.score else 0) + ((2 + 3 * nb + 4 * nb) if self.precondition else 0)
        self.dominant = "factgrass_kernel"
        self.need_flush = self.dense < 4 * L2_BYTES
        self.l2 = L2_FLUSHED if self.need_flush else "inputs >> L2"
        self.ev = []

    def dominant_ms(self, step_ms):
        return step_ms

    def step(self, ev=None):
        # a step that is nothing but the grouped call is timed as a whole: an extra pair of events inside the timed
        # region costs several microseconds, as much as a tenth of a small configuration's step
        if not (self.score or self.precondition):
            ev = None
        if ev is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        if self.tok_count is not None:
            self.G.factgrass_compress_grouped_varlen(self.group, self.out, self.ws, self.cfg.B, self.cfg.T,
                                                     tok_count=self.tok_count)
        else:
            self.G.factgrass_compress_grouped(self.group, self.out, self.ws)
        if ev is not None:
            e1.record()
            ev.append((e0, e1))
        if self.precondition:
            self.G.grass_fim(self.score[0], out=self.fim)
            self.G.grass_fim_factor(self.fim, 0.1)
            self.test_pre.copy_(self.score[1])
            self.G.grass_fim_apply(self.fim, self.test_pre)
            self.G.grass_score(self.score[0], self.test_pre, out=self.score_out)
        elif self.score:
            self.G.grass_score(self.score[0], self.score[1], out=self.score_out)

    def desc(self):
        c = self.cfg
        d = {"workload": c.name, "layers": len(c.layers), "B": c.B, "T": c.T, "kin": c.kin, "kout": c.kout,
             "k_per_layer": c.k, "l2": self.l2}
        if self.score:
            d["score"] = f"{c.score_n_train}x{c.score_n_test}x{c.k} fp32"
        if self.fp32:
            d["inputs"] = "fp32"
        if self.out_bf16:
            d["compressed_rows"] = "bf16 (rounded at the final store)"
        if self.precondition:
            d["score"] += ", preconditioned by the damped projected FIM (lambda 0.1)"
        if self.tok_count is not None:
            d["seq_len_aware"] = True
            d["tokens"] = int(self.tok_count.sum().item())
        return d


def small_config(cfg_id, W):
    """A reduced case of the same kernels (inputs still larger than L2, a few GB at most) for profiler
    captures."""
    import dataclasses
    cfg = W.CONFIGS[cfg_id]
    if cfg_id == 2:
        return dataclasses.replace(cfg, n=64, batch=64)
    if cfg_id == 4:
        return dataclasses.replace(cfg, layers=cfg.layers[:16])
    if cfg_id == 5:
        return dataclasses.replace(cfg, layers=cfg.layers[:14], score_n_train=2048)
    return cfg


def make_job(cfg_id, device, G, W, small=False, seq_len_aware=False, fp32_inputs=False, precondition=False,
             out_bf16=False):
    cfg = small_config(cfg_id, W) if small else W.CONFIGS[cfg_id]
    if cfg_id in (1, 2):
        return GrassJob(cfg, device, G, W)
    return FactJob(cfg, device, G, W, seq_len_aware, fp32_inputs, precondition, out_bf16)


def time_job(job, steps, warmup, world, device):
    """K timed steps.  Big inputs: one event pair around all K steps.  Inputs that fit in L2: one event
    pair per step with an L2 flush in between (not timed)."""
    flush = L2Flush(device) if job.need_flush else None
    for _ in range(warmup):
        if flush:
            flush()
        job.step()
    torch.cuda.synchronize()
    barrier(world)
    torch.cuda.synchronize()
    dom_events = []
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            job.step(ev=dom_events)
        e1.record()
        torch.cuda.synchronize()
        total_ms = e0.elapsed_time(e1)
    else:
        pairs = []
        for _ in range(steps):
            flush()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            job.step(ev=dom_events)
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        total_ms = sum(a.elapsed_time(b) for a, b in pairs)
    barrier(world)
    torch.cuda.synchronize()
    ms_per_step = max_over_ranks(total_ms / steps, world, device)
    if dom_events:
        dom_ms = sum(a.elapsed_time(b) for a, b in dom_events) / len(dom_events)
    else:
        dom_ms = job.dominant_ms(total_ms / steps)
    warm_ms = dirty_ms = None
    if flush is not None:
        # the same steps back to back with the inputs left in L2 (reported beside the cold figure, never as `value`)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            job.step()
        e1.record()
        torch.cuda.synchronize()
        warm_ms = max_over_ranks(e0.elapsed_time(e1) / steps, world, device)
        # and cold after a write pass followed by a read pass: L2 full of unmodified lines, nothing to write back
        pairs = []
        for _ in range(steps):
            flush(clean=True)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            job.step()
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        dirty_ms = max_over_ranks(sum(a.elapsed_time(b) for a, b in pairs) / steps, world, device)
    return ms_per_step, dom_ms, warm_ms, dirty_ms


# ----------------------------------------------------------------------------- end-to-end (host buffers)

def e2e_job(cfg_id, job, steps, warmup, world, device, G, W):
    """The same metric through the host-buffer API with the inputs in pinned host memory, the result read back
    every step.  Two legs: "in place" (the API's default for pinned inputs: the kernels gather the masked elements
    from host memory across the bus, so only the 64-byte pieces the masks touch are moved) and "staged" (every
    input byte is copied to the device first).  The line's `e2e` is the call left to choose between them (by the
    masks' density); both legs ride along."""
    from paper_2505_18976_b200 import host_api
    cfg = job.cfg
    if cfg_id in (1, 2):
        rows = min(cfg.batch, max(1, (1 << 30) // (cfg.p * 4)))           # <= 1 GiB pinned staging
        pinned = torch.empty((rows, cfg.p), dtype=torch.float32, pin_memory=True)
        pinned.copy_(job.g[0][:rows])
        chunks = [pinned] * (cfg.n // rows)
        out_host = torch.empty((cfg.n, cfg.k), dtype=torch.float32, pin_memory=True)
        h2d = cfg.n * cfg.p * 4
        d2h = cfg.n * cfg.k * 4
        note = f"{cfg.n // rows} chunk copies of {rows} rows from one pinned staging buffer"

        pieces = (job.fetch_bytes_per_launch - cfg.batch * cfg.k * 4) * job.launches_per_step
        in_place = host_api.grass_in_place(chunks, job.idx)

        def run(zero_copy):
            host_api.grass_compress_host(chunks, job.idx, cfg.k, cfg.s, cfg.hash_seed, out_host=out_host, device=device,
                                         zero_copy=zero_copy)
    else:
        # pinned copies of the first block's layers; later blocks of the same shape reuse those host
        # tensors (the bytes copied per step are those of the whole model)
        per_block = 7 if cfg_id == 5 else (4 if cfg_id == 4 else 1)
        pinned = []
        for l in range(per_block):
            A, Gt = job.layers[l]["A"], job.layers[l]["G"]
            pinned.append((torch.empty(A.shape, dtype=A.dtype, pin_memory=True).copy_(A),
                           torch.empty(Gt.shape, dtype=Gt.dtype, pin_memory=True).copy_(Gt)))
        groups, h2d = [], 0
        for b0 in range(0, len(cfg.layers), per_block):
            grp = []
            for j in range(per_block):
                l = b0 + j
                mi, mo = job.host_masks[l]
                grp.append(dict(A=pinned[j][0], G=pinned[j][1], mask_in=mi, mask_out=mo, k=cfg.k, s=cfg.s,
                                seed=W.layer_hash_seed(cfg, l), out_offset=l * cfg.k))
                h2d += pinned[j][0].numel() * 2 + pinned[j][1].numel() * 2
            groups.append(grp)
        out_host = torch.empty((cfg.B, cfg.out_dim), dtype=torch.float32, pin_memory=True)
        d2h = cfg.B * cfg.out_dim * 4
        note = f"{len(groups)} block copies from one block's pinned tensors"
        score_host = None
        if job.score:
            score_host = (torch.empty(job.score[0].shape, pin_memory=True).copy_(job.score[0]),
                          torch.empty(job.score[1].shape, pin_memory=True).copy_(job.score[1]))
            h2d += (score_host[0].numel() + score_host[1].numel()) * 4
            d2h += cfg.score_n_train * cfg.score_n_test * 4

        score_bytes = (score_host[0].numel() + score_host[1].numel()) * 4 if score_host else 0
        pieces = job.fetch_bytes_per_launch - cfg.B * cfg.out_dim * 4 + score_bytes
        in_place = host_api.factgrass_in_place(groups)
        plan, mixed_bytes = host_api.factgrass_host_plan(groups)
        mixed = {"tensors_in_place": sum(int(a) + int(g) for a, g in plan), "tensors_copied":
                 sum(2 - int(a) - int(g) for a, g in plan), "h2d_bytes_per_step": int(mixed_bytes + score_bytes)}

        def run(zero_copy):
            host_api.factgrass_compress_host(groups, cfg.B, cfg.T, cfg.out_dim, out_host=out_host, device=device,
                                             zero_copy=zero_copy)
            if score_host:
                host_api.grass_score_host(score_host[0], score_host[1], device=device)

    def leg(zero_copy):
        for _ in range(max(1, min(warmup, 2))):
            run(zero_copy)
        torch.cuda.synchronize()
        barrier(world)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            run(zero_copy)
        e1.record()
        torch.cuda.synchronize()
        return max_over_ranks(e0.elapsed_time(e1) / steps, world, device)

    ms_staged = leg(False)
    ms_in_place = leg(True)
    ms_default = leg(None)                 # what the call does when left to choose
    per_s = world * job.samples_per_step
    h2d_default = pieces if in_place else h2d
    if cfg_id >= 3:
        h2d_default = mixed["h2d_bytes_per_step"]
    out = {"value": per_s / (ms_default * 1e-3), "unit": UNIT, "ms_per_step": ms_default,
            "h2d_bytes_per_step": int(h2d_default), "d2h_bytes_per_step": int(d2h), "steps": steps,
            "path": ("in place: the kernels gather from the pinned host inputs; h2d = 64-byte pieces the masks touch "
                     "(host count)" + (" + the score operands, which are copied" if cfg_id == 5 else ""))
                    if in_place else "staged: every input byte is copied to the device (" + note + ")",
            "host_input_bytes_per_step": int(h2d),
            "staged": {"value": per_s / (ms_staged * 1e-3), "ms_per_step": ms_staged, "h2d_bytes_per_step": int(h2d)},
            "in_place": {"value": per_s / (ms_in_place * 1e-3), "ms_per_step": ms_in_place,
                         "h2d_bytes_per_step": int(pieces)}}
    if cfg_id >= 3:
        out["chosen_per_tensor"] = mixed       # the default leg decides tensor by tensor (host_api.factgrass_host_plan)
        out["path"] = ("per tensor: a factor whose mask touches at most 70 % of its bytes is gathered in place from the "
                       "pinned host input, a denser one is copied first; h2d = copied tensors + touched 64-byte pieces "
                       "(host count)" + (" + the score operands, which are copied" if cfg_id == 5 else ""))
    return out


# ----------------------------------------------------------------------------- CPU oracle arm

def oracle_sample(cfg_id, W, budget="baseline"):
    """A bounded sample of the workload for the CPU oracle, as host numpy arrays, and the fraction of
    one step (in sample-equivalents) that it covers."""
    import oracle
    cfg = W.CONFIGS[cfg_id]
    if cfg_id in (1, 2):
        rows = 256 if cfg_id == 1 else 64
        g = W.dense_gradients(rows, cfg.p, cfg.zero_prob, cfg.dist, cfg.scale, cfg.data_seed, device="cpu")
        idx = oracle.random_mask(cfg.p, cfg.kprime, cfg.mask_seed)
        gh = W.bits_of(g)

        def run():
            oracle.grass(gh, idx, cfg.k, cfg.s, cfg.hash_seed, want_absum=False)
        return run, float(rows), f"{rows} of {cfg.n} samples, full p and k'"
    nl = {3: 1, 4: 8, 5: 7}[cfg_id]
    items = []
    for l in range(nl):
        lay = cfg.layers[l]
        A, Gt = W.layer_io(cfg, l, device="cpu")
        s_in, s_out = W.layer_mask_seeds(cfg, l)
        items.append((W.bits_of(A), W.bits_of(Gt), oracle.random_mask(lay.d_in, cfg.kin, s_in),
                      oracle.random_mask(lay.d_out, cfg.kout, s_out), W.layer_hash_seed(cfg, l)))

    def run():
        for (A, Gt, mi, mo, seed) in items:
            oracle.factgrass(A, Gt, mi, mo, cfg.k, cfg.s, seed, want_absum=False)
    frac = nl / len(cfg.layers)
    return run, cfg.B * frac, f"first {nl} of {len(cfg.layers)} layers, all {cfg.B} samples x {cfg.T} tokens"


def cpu_baseline(cfg_id, W, min_seconds=10.0, max_repeats=20000):
    """The oracle on the bounded sample, repeated until about `min_seconds` of wall time."""
    import oracle
    oracle.build()
    run, sample_equiv, what = oracle_sample(cfg_id, W)
    t0 = time.perf_counter()
    repeats = 0
    while repeats < max_repeats and (repeats == 0 or time.perf_counter() - t0 < min_seconds):
        run()
        repeats += 1
    dt = (time.perf_counter() - t0) / repeats
    what = f"{what}; {repeats} repeat(s)"
    return {"value": sample_equiv / dt, "unit": UNIT, "cores": min(oracle.num_threads(), len(os.sched_getaffinity(0))),
            "kind": "oracle", "sample": what, "seconds": dt}


def fig4_microbench(device, G, W, steps=20):
    """Plain SJLT (identity mask) at p = 131,072 for several input sparsities and output sizes: the shape of
    the paper's projection benchmark figure (its data are not available; this reports our kernel only).
    Per case: time per batch of 1,024 samples and the mean relative error of pairwise distances."""
    p, n, out = 131_072, 1_024, []
    flush = L2Flush(device)
    for zero_prob in (0.0, 0.9, 0.99, 0.999):
        g = W.dense_gradients(n, p, zero_prob, "normal", 1.0, 4242, device=device)
        sub = g[:128].double()
        d_true = torch.cdist(sub, sub)
        iu = torch.triu_indices(128, 128, offset=1, device=device)
        for k in (512, 4_096, 32_768):
            res = torch.empty((n, k), dtype=torch.float32, device=device)
            for _ in range(3):
                G.grass_compress(g, None, k, 1, 0xF164, out=res)
            pairs = []
            for _ in range(steps):
                flush()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                G.grass_compress(g, None, k, 1, 0xF164, out=res)
                e1.record()
                pairs.append((e0, e1))
            torch.cuda.synchronize()
            ms = sorted(a.elapsed_time(b) for a, b in pairs)[len(pairs) // 2]
            d_proj = torch.cdist(res[:128].double(), res[:128].double())
            rel = ((d_proj - d_true).abs() / d_true)[iu[0], iu[1]].mean().item()
            out.append({"zero_prob": zero_prob, "k": k, "ms_per_batch": ms, "samples_per_s": n / (ms * 1e-3),
                        "dense_gbs": n * p * 4 / (ms * 1e-3) / 1e9, "pairwise_distance_rel_err": rel})
    return {"fig4": {"p": p, "n": n, "s": 1, "l2": "flushed before every call", "cases": out}}


def score_full_concatenation(device, G, W, steps=5):
    """grass_score over config 5's whole compressed vector: train 16,384 x 917,504 fp32 (60 GB, far beyond L2),
    test 256 x 917,504.  Reported beside the per-layer-block shape the default step times; not a bench line."""
    c = W.CONFIG5
    N, M, D = c.score_n_train, c.score_n_test, c.out_dim
    gen = torch.Generator(device=device)
    gen.manual_seed(c.data_seed + 9)
    tr = torch.empty((N, D), dtype=torch.float32, device=device)
    for i in range(0, N, 1_024):
        tr[i:i + 1_024].normal_(generator=gen)
    te = torch.randn((M, D), generator=gen, device=device)
    out = torch.empty((N, M), dtype=torch.float32, device=device)
    for _ in range(2):
        G.grass_score(tr, te, out=out)
    pairs = []
    for _ in range(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        G.grass_score(tr, te, out=out)
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    ms = sorted(a.elapsed_time(b) for a, b in pairs)[len(pairs) // 2]
    peaks, src = load_peaks()
    tf = 2.0 * N * M * D / (ms * 1e-3) / 1e12
    # the same scores from a bf16 cache of the same vectors (grass_to_bf16 + grass_score_bf16)
    tr16 = torch.empty((N, D), dtype=torch.bfloat16, device=device)
    for i in range(0, N, 1_024):
        G.grass_to_bf16(tr[i:i + 1_024], out=tr16[i:i + 1_024])
    te16 = G.grass_to_bf16(te)
    del tr
    torch.cuda.empty_cache()
    for _ in range(2):
        G.grass_score_bf16(tr16, te16, out=out)
    pairs = []
    for _ in range(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        G.grass_score_bf16(tr16, te16, out=out)
        e1.record()
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    ms16 = sorted(a.elapsed_time(b) for a, b in pairs)[len(pairs) // 2]
    tf16 = 2.0 * N * M * D / (ms16 * 1e-3) / 1e12
    return {"score_full": {"N": N, "M": M, "D": D, "ms": ms, "fp32_equivalent_tflops": tf,
                           "bf16_product_tflops": 6 * tf, "frac_of_bf16_peak": 6 * tf / peaks["bf16_tflops"],
                           "peak_source": src, "train_gbs": N * D * 4 / (ms * 1e-3) / 1e9,
                           "bf16_cache": {"ms": ms16, "tflops": tf16, "frac_of_bf16_peak": tf16 / peaks["bf16_tflops"],
                                          "train_gbs": N * D * 2 / (ms16 * 1e-3) / 1e9,
                                          "frac_of_hbm_peak": N * D * 2 / (ms16 * 1e-3) / 1e9 / peaks["hbm_gbs"]}}}


def compare_compressors(cfg_id, device, G, W, steps=5):
    """On-box ordering of the compressors of the paper's Tables 1d / 2 on one configuration's shapes:
    FactGraSS and factorised Mask (this library) next to LoGra, the Gaussian factorised projection, written here
    with torch matmuls (cuBLAS) as the paper's own baseline is: a comparison arm, not part of the library."""
    job = FactJob(W.CONFIGS[cfg_id], device, G, W)
    cfg = job.cfg
    kin = kout = int(round(cfg.k ** 0.5))                  # LoGra projects each factor to sqrt(k_l)
    gen = torch.Generator(device=device)
    gen.manual_seed(99)
    proj = {}
    for lay in cfg.layers:
        for d, kk in ((lay.d_in, kin), (lay.d_out, kout)):
            if (d, kk) not in proj:
                proj[(d, kk)] = torch.randn((d, kk), generator=gen, device=device).to(torch.bfloat16)
    mask_out = torch.empty((cfg.B, len(cfg.layers) * cfg.kin * cfg.kout), dtype=torch.float32, device=device)
    mask_layers = [dict(l, out_offset=i * cfg.kin * cfg.kout) for i, l in enumerate(job.layers)]
    mask_group = G.GroupedLayers(mask_layers)
    logra_out = torch.empty((cfg.B, len(cfg.layers), kin * kout), dtype=torch.float32, device=device)

    def logra():
        for i, (l, lay) in enumerate(zip(job.layers, cfg.layers)):
            a = torch.matmul(l["A"], proj[(lay.d_in, kin)])             # B x T x kin
            g = torch.matmul(l["G"], proj[(lay.d_out, kout)])           # B x T x kout
            logra_out[:, i] = torch.bmm(a.transpose(1, 2), g).float().reshape(cfg.B, -1)

    # factorised SJLT without reconstruction (the paper's SJLT_{k_in (x) k_out} row): every token row of A and G is
    # projected on its own, then the k_in x k_out block is the token sum of the projected factors; composed of three
    # calls of this library per layer, the projected factors (a few MB) going through HBM
    fa = torch.empty((cfg.B * cfg.T, kin), dtype=torch.float32, device=device)
    fg = torch.empty((cfg.B * cfg.T, kout), dtype=torch.float32, device=device)
    fs_out = torch.empty((cfg.B, len(cfg.layers), kin * kout), dtype=torch.float32, device=device)

    def fact_sjlt():
        for i, (l, lay) in enumerate(zip(job.layers, cfg.layers)):
            G.grass_compress(l["A"].view(cfg.B * cfg.T, lay.d_in), None, kin, 1, 1000 + i, out=fa)
            G.grass_compress(l["G"].view(cfg.B * cfg.T, lay.d_out), None, kout, 1, 2000 + i, out=fg)
            G.factmask_compress(fa.view(cfg.B, cfg.T, kin), fg.view(cfg.B, cfg.T, kout), None, None, out=fs_out[:, i])

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    res = {"FactGraSS (SJLT o Mask, this library)": timed(lambda: G.factgrass_compress_grouped(job.group, job.out, job.ws)),
           "factorised Mask alone (this library)": timed(lambda: G.factmask_compress_grouped(mask_group, mask_out, job.ws)),
           "factorised SJLT without reconstruction (this library, three calls per layer)": timed(fact_sjlt),
           "LoGra (Gaussian factorised projection, torch/cuBLAS)": timed(logra)}
    tokens = cfg.B * cfg.T
    return {"compare": {"workload": cfg.name, "k_per_layer": cfg.k, "mask": f"{cfg.kin}x{cfg.kout}",
                        "logra_factors": f"{kin}x{kout}",
                        "ms_per_batch": res, "tokens_per_s": {n: tokens / (ms * 1e-3) for n, ms in res.items()}}}


def reference_full(args, W):
    """--impl reference --full: the oracle over the WHOLE FactGraSS configuration, one step, layer by layer (the inputs
    of a layer are drawn, untimed, just before its call, so the host never holds more than one layer)."""
    import oracle
    oracle.build()
    cfg = W.CONFIGS[args.config]
    total = 0.0
    for l, lay in enumerate(cfg.layers):
        A, Gt = W.layer_io(cfg, l, device="cpu")
        s_in, s_out = W.layer_mask_seeds(cfg, l)
        mi, mo = oracle.random_mask(lay.d_in, cfg.kin, s_in), oracle.random_mask(lay.d_out, cfg.kout, s_out)
        a, g = W.bits_of(A), W.bits_of(Gt)
        t0 = time.perf_counter()
        oracle.factgrass(a, g, mi, mo, cfg.k, cfg.s, W.layer_hash_seed(cfg, l), want_absum=False)
        total += time.perf_counter() - t0
    cores = min(oracle.num_threads(), len(os.sched_getaffinity(0)))
    what = f"all {len(cfg.layers)} layers, all {cfg.B} samples x {cfg.T} tokens, one step (the score step is not included)"
    val = cfg.B / total
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": 1,
                      "warmup": 0, "ms_per_step": total * 1e3, "higher_is_better": True, "scaling": "weak",
                      "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                      "config": {"workload": cfg.name, "sample": what},
                      "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
                      "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                      "gpu_launches": 0}))


def reference_arm(args, W):
    """--impl reference: the CPU oracle, as it stands, timed on the host cores."""
    world, rank, _ = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), 0
    if rank != 0:
        return
    if args.full and args.config >= 3:
        return reference_full(args, W)
    import oracle
    oracle.build()
    run, sample_equiv, what = oracle_sample(args.config, W)
    for _ in range(min(args.warmup, 1)):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    ms = (time.perf_counter() - t0) / args.steps * 1e3
    val = sample_equiv / (ms * 1e-3)
    cores = min(oracle.num_threads(), len(os.sched_getaffinity(0)))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": W.CONFIGS[args.config].name, "sample": what},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--full", action="store_true",
                    help="with --impl reference, configs 3-5: the oracle over the whole configuration, one step "
                         "(minutes; the default is a bounded sample)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="default workload only: skip the per_config object (configs 1-4 timed in the same run)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--small", action="store_true", help="reduced case for profiler captures (not a bench value)")
    ap.add_argument("--compare", action="store_true",
                    help="configs 3-5: FactGraSS / factorised Mask (this library) next to a torch LoGra arm (not a bench line)")
    ap.add_argument("--fig4", action="store_true",
                    help="plain SJLT at p = 131,072 over input sparsity and k (not a bench line)")
    ap.add_argument("--score-full", action="store_true",
                    help="grass_score over config 5's full concatenation, D = 917,504 (60 GB; not a bench line)")
    ap.add_argument("--fp32-inputs", action="store_true", help="configs 3-5: fp32 A and G instead of bf16")
    ap.add_argument("--precondition", action="store_true",
                    help="config 5: projected FIM of the train vectors, damped solve for the test vectors, then scores")
    ap.add_argument("--tune", action="append", default=[], metavar="KEY=VALUE",
                    help="force a launch-shape choice of the library (grass_set_tuning), e.g. factgrass_path=0; "
                         "for profiler captures and sweeps")
    ap.add_argument("--out-bf16", action="store_true",
                    help="configs 3-5: compressed rows written as bf16 by the compress call (not a bench line)")
    ap.add_argument("--seq-len-aware", action="store_true",
                    help="configs 3-5: pass per-sample token counts so that padding tokens are not read")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    from paper_2505_18976_b200 import workloads as W
    if args.impl == "reference":
        reference_arm(args, W)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    world, rank, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    import paper_2505_18976_b200 as G
    G.lib()
    for kv in args.tune:
        key, val = kv.split("=")
        G.grass_set_tuning(key, int(val))
    warmup = args.warmup if args.small else max(args.warmup, 3)
    if args.fig4:
        if rank == 0:
            print(json.dumps(fig4_microbench(device, G, W)))
        return
    if args.score_full:
        if rank == 0:
            print(json.dumps(score_full_concatenation(device, G, W)))
        return
    if args.compare:
        if rank == 0:
            print(json.dumps(compare_compressors(args.config if args.config >= 3 else 5, device, G, W)))
        return

    peaks, peak_src = load_peaks()

    def measure(cfg_id, steps, **kw):
        """One configuration, device-resident inputs: (job, ms per step, clocks, roofline object, extra config keys)."""
        job = make_job(cfg_id, device, G, W, **kw)
        sampler = ClockSampler(local)
        sampler.start()
        ms_per_step, dom_ms, warm_ms, dirty_ms = time_job(job, steps, warmup, world, device)
        clocks = sampler.stop()
        achieved = job.alg_bytes_per_launch / (dom_ms * 1e-3) / 1e9
        plain = not (kw.get("fp32_inputs") or kw.get("seq_len_aware") or kw.get("small") or kw.get("out_bf16"))
        roofline = {"bound": "hbm", "kernel": job.dominant, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "peak_source": peak_src,
                    "algorithmic_bytes_per_launch": int(job.alg_bytes_per_launch),
                    "dense_bytes_per_launch": int(job.dense_bytes_per_launch), "ms_per_launch": dom_ms,
                    "fetch64_bytes_per_launch": int(job.fetch_bytes_per_launch),
                    "fetch64_achieved": job.fetch_bytes_per_launch / (dom_ms * 1e-3) / 1e9,
                    "fetch64_frac": job.fetch_bytes_per_launch / (dom_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "traffic": TRAFFIC.get(cfg_id) if plain else None}
        extra = {}
        if warm_ms is not None:
            extra["ms_per_step_l2_warm"] = warm_ms     # `ms_per_step` is the cold figure (L2 flushed before each step)
            extra["ms_per_step_l2_unmodified"] = dirty_ms  # cold, flush = write pass then read pass (no write-backs left)
        return job, ms_per_step, clocks, roofline, extra

    job, ms_per_step, clocks, roofline, extra = measure(args.config, args.steps, small=args.small,
                                                        seq_len_aware=args.seq_len_aware, fp32_inputs=args.fp32_inputs,
                                                        precondition=args.precondition, out_bf16=args.out_bf16)
    if args.fp32_inputs or args.precondition or args.out_bf16:
        args.no_e2e = True      # the host-buffer leg covers the default path only
    value = world * job.samples_per_step / (ms_per_step * 1e-3)

    e2e = None
    if not args.no_e2e:
        e2e = e2e_job(args.config, job, max(1, args.e2e_steps), warmup, world, device, G, W)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_baseline(args.config, W)

    # The default run also times the other four configurations (device-resident inputs, same cold-L2 protocol,
    # fewer steps), so that one line carries all five; `value` stays the default workload's.
    per_config = None
    default_run = (args.config == 5 and not (args.small or args.fp32_inputs or args.precondition or args.seq_len_aware
                                             or args.no_per_config or args.out_bf16 or args.tune))
    if default_run:
        main_desc = job.desc()
        kernels_main = job.kernels_per_step * args.steps
        del job
        torch.cuda.empty_cache()
        per_config = {}
        for cid in (1, 2, 3, 4):
            steps_c = max(3, min(args.steps, 20))
            j, ms_c, clocks_c, roof_c, extra_c = measure(cid, steps_c)
            d = j.desc()
            d.update(extra_c)
            v = world * j.samples_per_step / (ms_c * 1e-3)
            per_config[f"c{cid}"] = {"value": v, "unit": UNIT, "ms_per_step": ms_c, "steps": steps_c,
                                     "tokens_per_s": (v * j.cfg.T if cid >= 3 else None), "config": d,
                                     "roofline": roof_c, "clocks": clocks_c,
                                     "gpu_launches": j.kernels_per_step * steps_c}
            del j
            torch.cuda.empty_cache()
    else:
        main_desc = job.desc()
        kernels_main = job.kernels_per_step * args.steps

    if rank == 0:
        cfgd = main_desc
        cfgd["replicas"] = world
        cfgd.update(extra)
        if args.small:
            cfgd["small"] = True
        if args.tune:
            cfgd["tuning"] = args.tune
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if (args.config >= 3 and not args.fp32_inputs) else "f32", "data": "synthetic", "config": cfgd,
                "tokens_per_s": (value * W.CONFIGS[args.config].T if args.config >= 3 else None),
                "clocks": clocks, "e2e": e2e, "gpu_launches": kernels_main,
                "roofline": roofline, "cpu_baseline": cpu}
        if per_config is not None:
            line["per_config"] = per_config
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel per launch, from ncu captures
# summarised under profiles/ (bytes; None until captured)
TRAFFIC = {1: 58_796_800 + 536_832, 2: 8 * (239_980_032 + 3_712_256), 3: 100_758_016 + 3_166_464,
           4: 3 * (1_044_538_368 + 3_582_976), 5: 16 * (729_330_944 + 4_280_320)}

if __name__ == "__main__":
    main()
