#!/usr/bin/env python
"""Benchmark of the whole hot path: one step = B, R, H, H*, fused conv forward / adjoint and
affine forward / adjoint, each on its full-size configuration, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the algorithmic bytes of one step divided by the
device time of one step (CUDA events, max over ranks); every rank of a multi-GPU run works on its
own replica of the workload (the path has no exchange between GPUs).
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fwd+adjoint GB/s and % of B200 HBM peak for halo/broadcast/sum-reduce"
UNIT = "GB/s"
WORKLOAD = ("one pass over B+R (fp32 4096x4096, k=8), H+H* (fp32 512^3, 4x4x4 workers, halo 4), "
            "fused depthwise 5x5 conv fwd+adj (fp32 16x16x1024x1024, 4x4 workers) and "
            "affine fwd+adj (bf16 256x8192x8192, 4x4 workers)")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------
# Workload on the device
# ----------------------------------------------------------------------------------------------

def conv_algorithmic_bytes(part):
    """Bulk read once + halo cells inside the tensor read once from the neighbours + output written once."""
    gs = part.global_shape
    total = 0
    for w in range(part.num_workers):
        st, bulk, _, lo, hi = part.shard_extents(w)
        planes = bulk[0] * bulk[1]
        r0, r1 = max(st[2] - lo[2], 0), min(st[2] + bulk[2] + hi[2], gs[2])
        c0, c1 = max(st[3] - lo[3], 0), min(st[3] + bulk[3] + hi[3], gs[3])
        total += planes * 4 * (2 * bulk[2] * bulk[3] + (r1 - r0) * (c1 - c0) - bulk[2] * bulk[3])
    return total


class Workload:
    """All buffers of one step, resident on `dev`, and the eight operator calls."""

    def __init__(self, dev, small=False):
        import torch
        import paper_2006_03108_b200 as distdl
        self.torch, self.d, self.dev = torch, distdl, dev
        g = torch.Generator(device=dev)
        g.manual_seed(2006_03108)
        u = lambda *s: torch.rand(*s, device=dev, generator=g) * 2 - 1
        n = lambda *s: torch.randn(*s, device=dev, generator=g)
        # broadcast / sum-reduce: fp32 [4096, 4096], 8 workers
        self.k = 8
        rows = 1024 if small else 4096   # small: the reduced case for profiler captures
        self.b_src = u(rows, 4096)
        self.b_dst = [torch.empty(rows, 4096, device=dev) for _ in range(self.k)]
        self.r_src = [u(rows, 4096) for _ in range(self.k)]
        self.r_dst = torch.empty(rows, 4096, device=dev)
        # 3-D halo: 512^3 over 4x4x4 workers, halo 4
        side, pw = 512, 4
        self.hpart = distdl.Partition((side,) * 3, (pw,) * 3, (4,) * 3, (4,) * 3)
        self.h_x = [u(*self.hpart.padded_shape(w)) for w in range(self.hpart.num_workers)]
        self.h_y = [u(*self.hpart.padded_shape(w)) for w in range(self.hpart.num_workers)]
        # conv: NCHW [16,16,1024,1024] over 1x1x4x4 workers, depthwise 5x5
        nc = 4 if small else 16
        self.cpart = distdl.Partition((nc, 16, 1024, 1024), (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2))
        P = self.cpart.num_workers
        self.c_x = [n(*self.cpart.padded_shape(w)) for w in range(P)]
        self.c_y = [torch.empty(*self.cpart.bulk_shape(w), device=dev) for w in range(P)]
        self.c_dy = [n(*self.cpart.bulk_shape(w)) for w in range(P)]
        self.c_dx = [torch.empty(*self.cpart.padded_shape(w), device=dev) for w in range(P)]
        self.c_w = n(16, 5, 5) * 0.1
        # affine: x bf16 [256, 8192], W bf16 [8192, 8192] on a 4x4 grid
        self.nb, self.nf, self.pf = 256, 8192, 4
        blk = self.nf // self.pf
        self.a_x = [n(self.nb, blk).bfloat16() for _ in range(self.pf)]
        self.a_w = [(n(blk, blk) * self.nf ** -0.5).bfloat16() for _ in range(self.pf * self.pf)]
        self.a_dy = [n(self.nb, blk).bfloat16() for _ in range(self.pf)]
        self.a_y = [torch.empty(self.nb, blk, device=dev) for _ in range(self.pf)]
        self.a_dx = [torch.empty(self.nb, blk, device=dev) for _ in range(self.pf)]

        d = distdl
        el = self.b_src.numel() * 4
        conv_bytes = conv_algorithmic_bytes(self.cpart)
        # the adjoint also clears the ghost cells of the padded dx shards (as H* does): one more write per ghost cell
        conv_ghost_bytes = 4 * sum(a.numel() - b.numel() for a, b in zip(self.c_dx, self.c_dy))
        aff_flops = 2 * self.nb * self.nf * self.nf
        aff_bytes = self.nf * self.nf * 2 + self.nb * self.nf * 2 + self.nb * self.nf * 4
        # name, call, algorithmic bytes, flops, kernel launches, bound
        self.ops = [
            ("broadcast_fwd", lambda: d.broadcast_fwd(self.b_src, self.b_dst), el * (1 + self.k), 0, 1, "hbm"),
            ("sumreduce_fwd", lambda: d.sumreduce_fwd(self.r_src, self.r_dst), el * (1 + self.k), 0, 1, "hbm"),
            ("halo_fwd", lambda: d.halo_fwd(self.hpart, self.h_x), self.hpart.halo_stats(False)[2], 0, 1, "hbm"),
            ("halo_adj", lambda: d.halo_adj(self.hpart, self.h_y), self.hpart.halo_stats(True)[2], 0, 1, "hbm"),
            ("conv_fwd", lambda: d.conv_fwd(self.cpart, self.c_x, self.c_w, None, self.c_y), conv_bytes,
             2 * 25 * self._conv_outputs(), 1, "hbm"),
            ("conv_adj", lambda: d.conv_adj(self.cpart, self.c_dy, self.c_w, self.c_dx), conv_bytes + conv_ghost_bytes,
             2 * 25 * self._conv_outputs(), 1, "hbm"),
            ("affine_fwd", lambda: d.affine_fwd(self.nb, self.nf, self.nf, self.pf, self.pf, self.a_x, self.a_w,
                                                None, self.a_y), aff_bytes, aff_flops, 1, "tensor"),
            ("affine_adj", lambda: d.affine_adj(self.nb, self.nf, self.nf, self.pf, self.pf, self.a_dy, self.a_w,
                                                self.a_dx), aff_bytes, aff_flops, 1, "tensor"),
        ]
        self.bytes_per_step = sum(o[2] for o in self.ops)
        self.launches_per_step = sum(o[4] for o in self.ops)

        # Distributed pooling layer (3 x 3 max pooling, stride 2, padding 1: ghost widths (1, 0) per worker):
        # timed on its own after the step, reported under "extra_ops", not part of `value`.
        k, st, pad = (3, 3), (2, 2), ((1, 1), (1, 1))
        gsp = (nc, 16, 1024, 1024)
        hl, hh = [0, 0], [0, 0]
        for dim in (2, 3):
            lo, hi, _, _ = d.halo_widths_1d(gsp[dim], 4, k[dim - 2], st[dim - 2], 1, pad[dim - 2][0], pad[dim - 2][1])
            hl.append(lo)
            hh.append(hi)
        self.ppart = d.Partition(gsp, (1, 1, 4, 4), hl, hh)
        oh = ((gsp[2] + 2 - 3) // 2 + 1) // 4
        P = self.ppart.num_workers
        self.p_x = [n(*self.ppart.padded_shape(w)) for w in range(P)]
        self.p_y = [torch.empty(nc, 16, oh, oh, device=dev) for _ in range(P)]
        self.p_arg = [torch.zeros(nc, 16, oh, oh, dtype=torch.int32, device=dev) for _ in range(P)]
        self.p_dy = [n(nc, 16, oh, oh) for _ in range(P)]
        self.p_dx = [torch.empty(*self.ppart.padded_shape(w), device=dev) for w in range(P)]
        out_b = sum(t.numel() for t in self.p_y) * 4
        need_b = P * nc * 16 * ((oh - 1) * 2 + 3) ** 2 * 4
        pad_b = sum(t.numel() for t in self.p_dx) * 4
        self.extra_ops = [
            ("pool_fwd", lambda: d.pool_fwd(self.ppart, self.p_x, k, st, pad, d.POOL_MAX, self.p_y, self.p_arg),
             self.ppart.halo_stats(False)[2] + need_b + 2 * out_b, 0, 2, "hbm"),
            ("pool_adj", lambda: d.pool_adj(self.ppart, self.p_dy, self.p_arg, k, st, pad, d.POOL_MAX, self.p_dx),
             2 * out_b + pad_b + self.ppart.halo_stats(True)[2], 0, 2, "hbm"),
        ]

        # Parameter gradients of the two layers (dw, db of the convolution; dW, db of the affine layer) on the
        # step's own buffers, and the generalized all-to-all between a row and a column partition of a
        # fp32 8192 x 8192 tensor (8 -> 8 workers); timed on their own like the pooling layer.
        self.c_dw = torch.empty(16, 5, 5, device=dev)
        self.c_db = torch.empty(16, device=dev)
        self.c_ws = torch.empty(d.conv_adj_params_workspace(self.cpart, 5, 5), dtype=torch.uint8, device=dev)
        self.a_dw = [torch.empty(blk, blk, device=dev) for _ in range(self.pf * self.pf)]
        self.a_db = [torch.empty(blk, device=dev) for _ in range(self.pf)]
        side2 = 8192
        self.rep = d.Repartition((side2, side2), (8, 1), (1, 8))
        self.t_src = [u(side2 // 8, side2) for _ in range(8)]
        self.t_dst = [torch.empty(side2, side2 // 8, device=dev) for _ in range(8)]
        # fused halo exchange + 25-point star (radius 4) on the step's 512^3 volume (4 x 4 x 4 workers)
        self.s_w = [[0.05 * (1 + abs(k - 4)) * (-1) ** k for k in range(9)] for _ in range(3)]
        nw = self.hpart.num_workers
        if small:
            self.spart = d.Partition((256, 512, 512), (2, 4, 4), (4,) * 3, (4,) * 3)
            nw = self.spart.num_workers
            self.s_x = self.h_x[:nw]
        else:
            self.spart, self.s_x = self.hpart, self.h_x
        self.s_y = [torch.empty(*self.spart.bulk_shape(w), device=dev) for w in range(nw)]
        self.s_dx = [torch.empty(*self.spart.padded_shape(w), device=dev) for w in range(nw)]
        cells = 1
        for v in self.spart.global_shape:
            cells *= v
        halo_read = (self.spart.halo_stats(False)[2] - sum(t.numel() - y.numel() for t, y in zip(self.s_dx, self.s_y)) * 4)
        st_bytes = 8 * cells + halo_read
        ghost_b = sum(t.numel() - y.numel() for t, y in zip(self.s_dx, self.s_y)) * 4
        self.extra_ops += [
            ("stencil3d_fwd", lambda: d.stencil3d_fwd(self.spart, self.s_x, self.s_w, self.s_y), st_bytes, 2 * 27 * cells, 1,
             "hbm"),
            ("stencil3d_adj", lambda: d.stencil3d_adj(self.spart, self.s_y, self.s_w, self.s_dx), st_bytes + ghost_b,
             2 * 27 * cells, 1, "hbm"),
        ]
        # generalized convolution: 16 -> 16 channels, 5 x 5, channel partitions 2 x 2, feature space 2 x 2
        gN = 1 if small else 4
        self.gpart = d.Partition((gN, 16, 1024, 1024), (1, 2, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
        self.g_x = [n(*self.gpart.padded_shape(w)) for w in range(8)]
        self.g_y = [torch.empty(gN, 8, 512, 512, device=dev) for _ in range(8)]
        self.g_dx = [torch.empty(*self.gpart.padded_shape(w), device=dev) for w in range(8)]
        self.g_w = [n(8, 8, 5, 5) * 0.05 for _ in range(4)]
        self.g_dw = [torch.empty(8, 8, 5, 5, device=dev) for _ in range(4)]
        self.g_ws = torch.empty(d.convg_adj_params_workspace(self.gpart, 16, 2, 5, 5), dtype=torch.uint8, device=dev)
        g_flops = 2 * 25 * 16 * 16 * gN * 1024 * 1024
        g_bytes = 2 * gN * 16 * 1024 * 1024 * 4
        self.extra_ops += [
            ("convg_fwd", lambda: d.convg_fwd(self.gpart, 16, 2, self.g_x, self.g_w, None, self.g_y), g_bytes, g_flops, 1, "alu"),
            ("convg_adj", lambda: d.convg_adj(self.gpart, 16, 2, self.g_y, self.g_w, self.g_dx), g_bytes, g_flops, 2, "alu"),
            ("convg_adj_params", lambda: d.convg_adj_params(self.gpart, 16, 2, self.g_x, self.g_y, (5, 5), self.g_dw, None,
                                                            self.g_ws), g_bytes, g_flops, 2, "alu"),
        ]
        self.extra_ops += [
            ("conv_adj_params", lambda: d.conv_adj_params(self.cpart, self.c_x, self.c_dy, (5, 5), self.c_dw, self.c_db,
                                                          self.c_ws), conv_bytes, 2 * 25 * self._conv_outputs(), 2, "hbm"),
            ("affine_adj_params", lambda: d.affine_adj_params(self.nb, self.nf, self.nf, self.pf, self.pf, self.a_dy,
                                                              self.a_x, self.a_dw, self.a_db),
             self.nf * self.nf * 4 + 2 * self.nb * self.nf * 2 + self.nf * 4, aff_flops, 2, "hbm"),
            ("repartition_fwd", lambda: d.repartition_fwd(self.rep, self.t_src, self.t_dst), 2 * side2 * side2 * 4, 0, 1,
             "hbm"),
            ("repartition_adj", lambda: d.repartition_adj(self.rep, self.t_dst, self.t_src), 2 * side2 * side2 * 4, 0, 1,
             "hbm"),
        ]

    def _conv_outputs(self):
        gs = self.cpart.global_shape
        return gs[0] * gs[1] * gs[2] * gs[3]

    def step(self, events=None):
        """Enqueues the eight operators; with `events`, records one CUDA event before each and one after."""
        torch = self.torch
        for i, op in enumerate(self.ops):
            if events is not None:
                events[i].record()
            op[1]()
        if events is not None:
            events[len(self.ops)].record()

    # ---- end-to-end variant: inputs come from pinned host memory, results go back to it ----
    def e2e_setup(self):
        """Pinned host copies of every input and output, per operator, and the three streams of the pipeline."""
        torch = self.torch
        per_op = [
            ([self.b_src], self.b_dst),
            (self.r_src, [self.r_dst]),
            (self.h_x, self.h_x),
            (self.h_y, self.h_y),
            (self.c_x + [self.c_w], self.c_y),
            (self.c_dy, self.c_dx),
            (self.a_x + self.a_w, self.a_y),
            (self.a_dy, self.a_dx),
        ]
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        self.e2e_ops = [([(t, pin(t)) for t in ins], [(t, pin(t)) for t in outs]) for ins, outs in per_op]
        for ins, _ in self.e2e_ops:
            for t, h in ins:
                h.copy_(t)
        torch.cuda.synchronize()
        self.h2d_bytes = sum(t.numel() * t.element_size() for ins, _ in self.e2e_ops for t, _ in ins)
        self.d2h_bytes = sum(t.numel() * t.element_size() for _, outs in self.e2e_ops for t, _ in outs)
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.e2e_done = None

    def e2e_step(self):
        """One step through the public calls with host buffers on both ends: the inputs of every operator come
        from pinned host memory and its results go back to it.  Three streams: uploads, the operators, downloads;
        the upload of the next operator's inputs and the download of the previous one's results run while an
        operator computes, so both directions of the host link are busy.  A step starts its uploads only when
        the previous step's downloads are done (some buffers are input and output at once)."""
        torch = self.torch
        main = torch.cuda.current_stream()
        if self.e2e_done is not None:
            self.s_in.wait_event(self.e2e_done)
        else:
            self.s_in.wait_stream(main)
        for (ins, outs), op in zip(self.e2e_ops, self.ops):
            with torch.cuda.stream(self.s_in):
                for t, h in ins:
                    t.copy_(h, non_blocking=True)
                up = torch.cuda.Event()
                up.record()
            main.wait_event(up)
            op[1]()
            ran = torch.cuda.Event()
            ran.record(main)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(ran)
                for t, h in outs:
                    h.copy_(t, non_blocking=True)
        self.e2e_done = torch.cuda.Event()
        self.e2e_done.record(self.s_out)
        main.wait_event(self.e2e_done)      # the step is over when its last result has reached the host


# ----------------------------------------------------------------------------------------------
# Clock sampling during the timed region
# ----------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        cmd = ["nvidia-smi", "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits", "-lms", "50"]
        if uuid:
            cmd += ["-i", uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for nme, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on a bounded sample of the same workload
# ----------------------------------------------------------------------------------------------

# Sample sizes of the oracle leg: (rows of the B/R tensor, halo shard edge, conv planes, affine features,
# rough oracle seconds per step).  The level is chosen so that the whole run stays within minutes.
ORACLE_LEVELS = [
    dict(rows=4096, edge=128, planes=16, feats=8192, secs=10.0),
    dict(rows=512, edge=128, planes=4, feats=2048, secs=1.9),
    dict(rows=128, edge=64, planes=1, feats=1024, secs=0.4),
]


def oracle_level(total_steps):
    for lv in ORACLE_LEVELS:
        if lv["secs"] * total_steps <= 150.0:
            return lv
    return ORACLE_LEVELS[-1]


def oracle_sample_text(lv):
    return ("per op: B,R on fp32 [%d,4096] k=8; H,H* on 2x2x2 workers of %d^3 shards, halo 4; conv on %d of the 256 "
            "planes (1024x1024, 4x4 workers); affine 256x%dx%d on the 4x4 grid; GB/s = algorithmic bytes of the "
            "sample / oracle seconds, numpy limited to one thread"
            % (lv["rows"], lv["edge"], lv["planes"], lv["feats"], lv["feats"]))


def oracle_sample_step(lv):
    """One pass of the oracle over a bounded sample of the workload; returns (bytes, seconds, per-op GB/s)."""
    import numpy as np
    from threadpoolctl import threadpool_limits
    import oracle
    import paper_2006_03108_b200 as distdl
    from paper_2006_03108_b200 import inputs
    res = {}
    clock = time.perf_counter
    with threadpool_limits(limits=1):
        src = inputs.uniform_pm1((lv["rows"], 4096), 1)
        parts = [inputs.uniform_pm1((lv["rows"], 4096), 10 + i) for i in range(8)]
        t = clock(); oracle.broadcast_fwd(src, 8); res["broadcast_fwd"] = (src.nbytes * 9, clock() - t)
        t = clock(); oracle.sumreduce_fwd(parts); res["sumreduce_fwd"] = (src.nbytes * 9, clock() - t)
        e = lv["edge"]
        part = oracle.Partition((2 * e,) * 3, (2,) * 3, 4, 4)
        x = [inputs.uniform_pm1(part.padded_shape(w), 100 + w) for w in range(8)]
        hstat = distdl.Partition((2 * e,) * 3, (2,) * 3, (4,) * 3, (4,) * 3)       # byte counts only (host)
        t = clock(); oracle.halo_fwd_sequence(part, x); res["halo_fwd"] = (hstat.halo_stats(False)[2], clock() - t)
        t = clock(); oracle.halo_adj_sequence(part, x); res["halo_adj"] = (hstat.halo_stats(True)[2], clock() - t)
        pl = lv["planes"]
        cshape = (1, pl, 1024, 1024)
        cpart = oracle.Partition(cshape, (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2))
        xg = inputs.normal(cshape, 200)
        w = inputs.normal((pl, 5, 5), 201, 0.1)
        xs = oracle.scatter_global(cpart, xg)
        dys = oracle.scatter_global(oracle.Partition(cshape, (1, 1, 4, 4)), xg)
        cbytes = conv_algorithmic_bytes(distdl.Partition(cshape, (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2)))
        t = clock(); oracle.conv_fwd(cpart, xs, w); res["conv_fwd"] = (cbytes, clock() - t)
        t = clock(); oracle.conv_adj(cpart, dys, w); res["conv_adj"] = (cbytes, clock() - t)
        nb, nf, pf = 256, lv["feats"], 4
        xa = [inputs.normal((nb, nf // pf), 300 + j).astype(np.float64) for j in range(pf)]
        wa = [inputs.normal((nf // pf, nf // pf), 310 + i, nf ** -0.5).astype(np.float64) for i in range(pf * pf)]
        abytes = nf * nf * 2 + nb * nf * 2 + nb * nf * 4
        t = clock(); oracle.affine_fwd(xa, wa, pf, pf); res["affine_fwd"] = (abytes, clock() - t)
        t = clock(); oracle.affine_adj(xa, wa, pf, pf); res["affine_adj"] = (abytes, clock() - t)
    nbytes = sum(v[0] for v in res.values())
    secs = sum(v[1] for v in res.values())
    return nbytes, secs, {k: round(v[0] / v[1] / 1e9, 3) for k, v in res.items()}


def run_reference(args, rank):
    """The oracle arm: K steps (after W warm-up steps) of the oracle on a bounded sample, rank 0 only."""
    if rank != 0:
        return
    lv = oracle_level(args.steps + args.warmup)
    sample = oracle_sample_text(lv)
    for _ in range(args.warmup):
        oracle_sample_step(lv)
    tot_b, tot_s, per = 0, 0.0, None
    for _ in range(args.steps):
        b, s, per = oracle_sample_step(lv)
        tot_b += b
        tot_s += s
    value = tot_b / tot_s / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_s / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64/f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "per_op_gbs": per},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# Main
# ----------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-op", default=None,
                    help="run only this operator, three times, on a reduced case (for profiler captures) and exit")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    warmup = max(args.warmup, 3)
    peaks = measured_peaks()

    if args.profile_op:
        wl = Workload(dev, small=True)
        op = [o for o in wl.ops + wl.extra_ops if o[0] == args.profile_op]
        if not op:
            raise SystemExit("unknown operator %r" % args.profile_op)
        for _ in range(3):
            op[0][1]()
        torch.cuda.synchronize()
        import paper_2006_03108_b200 as distdl
        distdl.device_status()
        print(json.dumps({"profile_op": args.profile_op, "algorithmic_bytes": op[0][2], "flops": op[0][3]}))
        return

    wl = Workload(dev)
    nops = len(wl.ops)
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K steps, per-op events inside every step ----
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(nops + 1)] for _ in range(args.steps)]
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid) if rank == 0 else None
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for s in range(args.steps):
        wl.step(ev[s])
    t_stop.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    elapsed_ms = t_start.elapsed_time(t_stop)
    per_op_ms = [statistics.fmean(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(args.steps)) for i in range(nops)]
    if world > 1:
        t = torch.tensor([elapsed_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    ms_per_step = elapsed_ms / args.steps
    value = world * wl.bytes_per_step / (ms_per_step * 1e-3) / 1e9

    # ---- the operators outside the step, each timed on its own (not part of `value`) ----
    extra_ms = []
    for name, call, _, _, _, _ in wl.extra_ops:
        for _ in range(3):
            call()
        reps = 20
        xe = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        for r in range(reps):
            xe[r].record()
            call()
            wl.ops[0][1]()          # 0.6 GB of other traffic between two launches (the inputs alone exceed L2 anyway)
        xe[reps].record()
        torch.cuda.synchronize()
        b0 = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        for r in range(reps):
            b0[r].record()
            wl.ops[0][1]()
        b0[reps].record()
        torch.cuda.synchronize()
        extra_ms.append((xe[0].elapsed_time(xe[reps]) - b0[0].elapsed_time(b0[reps])) / reps)

    # ---- the small 2-D configuration (256 x 256 on 2 x 2 workers, halo 1): launch-bound, so H + H* are timed as
    # separate calls and as replays of a CUDA graph that holds 50 such pairs ----
    small_cfg = None
    if True:
        import paper_2006_03108_b200 as distdl
        p1 = distdl.Partition((256, 256), (2, 2), (1, 1), (1, 1))
        sx = [torch.rand(*p1.padded_shape(w), device=dev) for w in range(4)]
        pairs = 50

        def run_pairs():
            for _ in range(pairs):
                distdl.halo_fwd(p1, sx)
                distdl.halo_adj(p1, sx)

        run_pairs()
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        run_pairs()
        c1.record()
        torch.cuda.synchronize()
        eager_us = c0.elapsed_time(c1) * 1e3 / pairs
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            run_pairs()
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                run_pairs()
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        c0.record()
        for _ in range(5):
            graph.replay()
        c1.record()
        torch.cuda.synchronize()
        graph_us = c0.elapsed_time(c1) * 1e3 / (5 * pairs)
        nb = p1.halo_stats(False)[2] + p1.halo_stats(True)[2]
        small_cfg = {"workload": "H + H* on fp32 256x256, 2x2 workers, halo 1 (32,896 algorithmic bytes per pair)",
                     "us_per_pair_separate_calls": round(eager_us, 2), "us_per_pair_cuda_graph": round(graph_us, 2),
                     "gbs_cuda_graph": round(nb / graph_us / 1e3, 2), "bound": "launch latency"}

    # ---- end to end: inputs from pinned host memory, results back to the host, every step ----
    wl.e2e_setup()
    wl.e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        wl.e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = world * wl.bytes_per_step / (e2e_ms / args.e2e_steps * 1e-3) / 1e9

    if rank == 0:
        ops = {}
        for (name, _, nbytes, flops, _, bound), ms in zip(wl.ops, per_op_ms):
            entry = {"ms": round(ms, 5), "gbs": round(nbytes / ms / 1e6, 1), "bound": bound,
                     "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm"], 4)}
            if flops:
                entry["tflops"] = round(flops / ms / 1e9, 2)
            if bound == "tensor":
                entry["frac_tensor"] = round(flops / ms / 1e9 / peaks["bf16_sustained"], 4)
            ops[name] = entry
        extra = {}
        for (name, _, nbytes, flops, _, bound), ms in zip(wl.extra_ops, extra_ms):
            extra[name] = {"ms": round(ms, 5), "gbs": round(nbytes / ms / 1e6, 1), "bound": bound,
                           "frac_hbm": round(nbytes / ms / 1e6 / peaks["hbm"], 4)}
            if bound == "alu":
                # fp32 FMA peak: 148 SMs x 128 lanes x 2 flop x max SM clock (packed pairs issue at half rate)
                extra[name]["tflops"] = round(flops / ms / 1e9, 2)
                extra[name]["frac_alu"] = round(flops / ms / 1e9 / FP32_PEAK_TFLOPS, 4)
        # dominant kernel = the launch with the largest share of the step
        top = max(range(nops), key=lambda i: per_op_ms[i])
        tname, _, tbytes, _, _, tbound = wl.ops[top]
        achieved = tbytes / per_op_ms[top] / 1e6
        roofline = {"kernel": tname, "bound": tbound, "achieved": round(achieved, 1), "peak": peaks["hbm"],
                    "unit": "GB/s", "frac": round(achieved / peaks["hbm"], 4), "traffic": NCU_TRAFFIC.get(tname),
                    "peak_source": "of " + peaks["source"], "share_of_step": round(per_op_ms[top] / sum(per_op_ms), 3)}
        dm = [o for o in ("broadcast_fwd", "sumreduce_fwd", "halo_fwd", "halo_adj")]
        dm_bytes = sum(w[2] for w in wl.ops if w[0] in dm)
        dm_ms = sum(ms for w, ms in zip(wl.ops, per_op_ms) if w[0] in dm)
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 (bf16 inputs, f32 accumulation in the affine layer)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "l2": "inputs larger than L2: the 6.9 GB working set of a step cycles through between "
                             "two launches of the same operator",
                       "bytes_per_step": wl.bytes_per_step},
            "frac_of_hbm_peak": round(value / world / peaks["hbm"], 4),
            "halo_bcast_reduce": {"gbs": round(dm_bytes / dm_ms / 1e6, 1),
                                  "frac_of_hbm_peak": round(dm_bytes / dm_ms / 1e6 / peaks["hbm"], 4)},
            "ops": ops,
            "extra_ops": {"note": "timed separately, not part of value: 3x3 max pooling, stride 2, padding 1 on fp32 "
                                  "16x16x1024x1024 over 4x4 workers (H + local kernel, local adjoint + H*); parameter "
                                  "gradients of the step's convolution (dw, db) and affine layer (dW, db); fused halo + radius-4 star stencil "
                                  "on the step's 512^3 volume (4x4x4 workers); generalized convolution 16 -> 16 channels, 5x5, fp32 "
                                  "4x16x1024x1024 on channel partitions 2x2 and 2x2 feature-space workers; generalized "
                                  "all-to-all of fp32 8192x8192 between 8 row blocks and 8 column blocks",
                          **extra},
            "small_config": small_cfg,
            "roofline": roofline,
            "clocks": clocks,
            "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": wl.h2d_bytes,
                    "d2h_bytes_per_step": wl.d2h_bytes, "steps": args.e2e_steps},
            "gpu_launches": wl.launches_per_step * args.steps,
        }
        if world == 1 and not args.no_cpu_baseline:
            lv = ORACLE_LEVELS[0]
            b, s, per = oracle_sample_step(lv)
            line["cpu_baseline"] = {"value": round(b / s / 1e9, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": oracle_sample_text(lv), "per_op_gbs": per}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) per launch from the committed ncu summaries under profiles/ (captures of
# the quarter-size case are scaled by 4: traffic grows with the number of planes / rows); None for a
# kernel whose counters were not meaningful (the broadcast's output was still in L2 when the short
# capture ended) or that changed since its counters were taken.
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 74.4

NCU_TRAFFIC = {
    "broadcast_fwd": None,
    "sumreduce_fwd": 4 * (134225152 + 5290496),
    "halo_fwd": 203393024 + 116994304,
    "halo_adj": 261256448 + 164833792,
    "conv_fwd": 4 * (278041088 + 221260288),
    "conv_adj": 4 * (269701888 + 228404480),
    "affine_fwd": 138435072 + 3728128,
    "affine_adj": 138447104 + 3240448,
}

if __name__ == "__main__":
    main()
