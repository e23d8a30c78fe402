#!/usr/bin/env python
"""Benchmark of the whole hot path: one step = B, R, H, H*, fused conv forward / adjoint and
affine forward / adjoint, each on its full-size configuration, through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is the algorithmic bytes of one step divided by the
device time of one step (CUDA events, max over ranks); every rank of a multi-GPU run works on its
own replica of the workload (the path has no exchange between GPUs).

Per-operator figures (`ops`, `extra_ops`) are timed directly: a CUDA graph that holds 24 launches of
the operator, cycling over three disjoint buffer sets so that every launch finds its data cold in
L2, replayed between one pair of events.  Inside the timed steps only the launch with the largest
share of the step carries its own event pair (the `roofline` entry).
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
# Order of the operators inside a step: the two affine launches read the same 134 MB of weights, which
# would otherwise still sit in the 126 MB L2 when the second one starts; 2.7 GB (after the forward) and
# 2.8 GB (after the adjoint, into the next step) of other operators' traffic separate them.
STEP_ORDER = ["broadcast_fwd", "affine_fwd", "sumreduce_fwd", "halo_fwd", "halo_adj", "conv_fwd", "affine_adj",
              "conv_adj"]
STEP_OPS = ["broadcast_fwd", "sumreduce_fwd", "halo_fwd", "halo_adj", "conv_fwd", "conv_adj", "affine_fwd",
            "affine_adj"]
EXTRA_GROUPS = [["pool_fwd", "pool_adj"], ["stencil3d_fwd", "stencil3d_adj"],
                ["convg_fwd", "convg_adj", "convg_adj_params"], ["conv_adj_params"], ["affine_adj_params"],
                ["repartition_fwd", "repartition_adj"], ["partition_broadcast_fwd", "partition_broadcast_adj"]]
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12      # 74.4: 148 SMs x 128 lanes x 2 flop x max SM clock
GRAPH_LAUNCHES = 24                                    # launches per replayed graph (eight per buffer set)
# The 512^3 halo exchange and its parts: the same tensor split (and exchanged) along one dimension only, which
# leaves one class of ghost cells each -- planes of whole rows (z), runs of four whole rows (y), 16 bytes at both
# ends of every row (x) -- against the full case, which adds the edges and corners.  (workers, ghost widths)
HALO_CASES = {
    "full": ((4, 4, 4), (4, 4, 4)),
    "z": ((4, 1, 1), (4, 0, 0)),
    "y": ((1, 4, 1), (0, 4, 0)),
    "x": ((1, 1, 4), (0, 0, 4)),
    "zy": ((4, 4, 1), (4, 4, 0)),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------
# Algorithmic bytes of H, H* and the fused convolution, counted from partition geometry alone (any
# object with num_workers, rank, global_shape, bulk_start(w), bulk_shape(w), widths(w), coords(w),
# pshape, hlo, hhi, size: the oracle's Partition).  The CPU tests check these counts against the
# byte counts of the library's own planner.
# ----------------------------------------------------------------------------------------------

def _prod(vals):
    out = 1
    for v in vals:
        out *= int(v)
    return out


def halo_algorithmic_bytes(part, elem=4):
    """(H bytes, H* bytes) of a non-periodic partition: H writes every ghost cell and reads the ones that lie
    inside the tensor; H* reads and rewrites every bulk cell that a neighbour holds a copy of, reads every ghost
    cell inside the tensor once and clears every ghost cell."""
    ghosts = inside = receiving = 0
    for w in range(part.num_workers):
        c = part.coords(w)
        st, b = part.bulk_start(w), part.bulk_shape(w)
        lo, hi = part.widths(w)
        padded = _prod(b[k] + lo[k] + hi[k] for k in range(part.rank))
        clipped = _prod(min(st[k] + b[k] + hi[k], part.global_shape[k]) - max(st[k] - lo[k], 0)
                        for k in range(part.rank))
        bulk = _prod(b)
        ghosts += padded - bulk
        inside += clipped - bulk
        # cells of the bulk out of every neighbour's reach, per dimension
        untouched = []
        for k in range(part.rank):
            reach_lo = part.hhi[k][c[k] - 1] if c[k] > 0 else 0                      # low neighbour's high ghost
            reach_hi = part.hlo[k][c[k] + 1] if c[k] + 1 < part.pshape[k] else 0    # high neighbour's low ghost
            untouched.append(max(b[k] - reach_lo - reach_hi, 0))
        receiving += bulk - _prod(untouched)
    return elem * (ghosts + inside), elem * (2 * receiving + inside + ghosts)


def conv_algorithmic_bytes(part, elem=4):
    """Bulk read once + halo cells inside the tensor read once from the neighbours + output written once."""
    total = 0
    for w in range(part.num_workers):
        st, b = part.bulk_start(w), part.bulk_shape(w)
        lo, hi = part.widths(w)
        planes = b[0] * b[1]
        r0, r1 = max(st[2] - lo[2], 0), min(st[2] + b[2] + hi[2], part.global_shape[2])
        c0, c1 = max(st[3] - lo[3], 0), min(st[3] + b[3] + hi[3], part.global_shape[3])
        total += planes * elem * (2 * b[2] * b[3] + (r1 - r0) * (c1 - c0) - b[2] * b[3])
    return total


class _Geometry:
    """Extents of an evenly split tensor with uniform ghost widths, for the byte counts above (no arithmetic of
    the operators: sizes only)."""

    def __init__(self, global_shape, pshape, lo, hi):
        self.global_shape, self.pshape, self.rank = tuple(global_shape), tuple(pshape), len(global_shape)
        self.num_workers = _prod(pshape)
        self.size, self.start = [], []
        for n, p in zip(global_shape, pshape):
            q, r = divmod(n, p)
            sizes = [q + 1 if c < r else q for c in range(p)]
            self.size.append(sizes)
            self.start.append([sum(sizes[:c]) for c in range(p)])
        self.hlo = [[lo[k]] * pshape[k] for k in range(self.rank)]
        self.hhi = [[hi[k]] * pshape[k] for k in range(self.rank)]

    def coords(self, w):
        c = []
        for k in reversed(range(self.rank)):
            c.append(w % self.pshape[k])
            w //= self.pshape[k]
        return tuple(reversed(c))

    def bulk_start(self, w):
        return tuple(self.start[k][c] for k, c in enumerate(self.coords(w)))

    def bulk_shape(self, w):
        return tuple(self.size[k][c] for k, c in enumerate(self.coords(w)))

    def widths(self, w):
        c = self.coords(w)
        return (tuple(self.hlo[k][c[k]] for k in range(self.rank)), tuple(self.hhi[k][c[k]] for k in range(self.rank)))


# ----------------------------------------------------------------------------------------------
# Workload on the device
# ----------------------------------------------------------------------------------------------

class Op:
    def __init__(self, name, calls, nbytes, flops, launches, bound):
        self.name, self.calls, self.bytes, self.flops, self.launches, self.bound = name, calls, nbytes, flops, launches, bound


class Workload:
    """Buffers and calls of the named operators on `dev`.  Every operator owns `nsets` disjoint buffer sets
    (calls[i] works on set i); a step runs set 0 of the eight operators of the hot path."""

    def __init__(self, dev, names, small=False, nsets=1, halo_case="full"):
        import torch
        import paper_2006_03108_b200 as distdl
        self.torch, self.d, self.dev, self.small, self.nsets = torch, distdl, dev, small, nsets
        self.halo_case = halo_case
        g = torch.Generator(device=dev)
        g.manual_seed(2006_03108)
        self.u = lambda *s: torch.rand(*s, device=dev, generator=g) * 2 - 1
        self.n = lambda *s: torch.randn(*s, device=dev, generator=g)
        self.ops = {}
        self._shared = {}
        for name in names:
            if name not in self.ops:
                getattr(self, "_build_bcast" if name in ("broadcast_fwd", "sumreduce_fwd") else "_build_" + name)()
        self.step_ops = [self.ops[nm] for nm in STEP_ORDER if nm in self.ops]
        self.bytes_per_step = sum(o.bytes for o in self.step_ops)
        self.launches_per_step = sum(o.launches for o in self.step_ops)

    def _sets(self, make):
        return [make() for _ in range(self.nsets)]

    # ---- B and R: fp32 [4096, 4096], 8 workers ----
    def _build_bcast(self):
        if "broadcast_fwd" in self.ops:
            return
        torch, d, dev, k = self.torch, self.d, self.dev, 8
        rows = 1024 if self.small else 4096   # small: the reduced case for profiler captures
        el = rows * 4096 * 4
        bs = self._sets(lambda: (self.u(rows, 4096), [torch.empty(rows, 4096, device=dev) for _ in range(k)]))
        rs = self._sets(lambda: ([self.u(rows, 4096) for _ in range(k)], torch.empty(rows, 4096, device=dev)))
        self.b_sets, self.r_sets = bs, rs
        self.ops["broadcast_fwd"] = Op("broadcast_fwd", [(lambda s=s: d.broadcast_fwd(s[0], s[1])) for s in bs],
                                       el * (1 + k), 0, 1, "hbm")
        self.ops["sumreduce_fwd"] = Op("sumreduce_fwd", [(lambda s=s: d.sumreduce_fwd(s[0], s[1])) for s in rs],
                                       el * (1 + k), 0, 1, "hbm")

    # ---- 3-D halo: 512^3 over 4x4x4 workers, halo 4 ----
    def _halo_part(self):
        if "hpart" not in self._shared:
            ps, h = HALO_CASES[self.halo_case]
            self._shared["hpart"] = self.d.Partition((512,) * 3, ps, h, h)
            self._shared["hbytes"] = halo_algorithmic_bytes(_Geometry((512,) * 3, ps, h, h))
        return self._shared["hpart"]

    def _build_halo_fwd(self):
        d, part = self.d, self._halo_part()
        self.h_x = self._sets(lambda: [self.u(*part.padded_shape(w)) for w in range(part.num_workers)])
        self.ops["halo_fwd"] = Op("halo_fwd", [(lambda s=s: d.halo_fwd(part, s)) for s in self.h_x],
                                  self._shared["hbytes"][0], 0, 1, "hbm")

    def _build_halo_adj(self):
        d, part = self.d, self._halo_part()
        self.h_y = self._sets(lambda: [self.u(*part.padded_shape(w)) for w in range(part.num_workers)])
        self.ops["halo_adj"] = Op("halo_adj", [(lambda s=s: d.halo_adj(part, s)) for s in self.h_y],
                                  self._shared["hbytes"][1], 0, 1, "hbm")

    # ---- conv: NCHW [16,16,1024,1024] over 1x1x4x4 workers, depthwise 5x5 ----
    def _conv_part(self):
        if "cpart" not in self._shared:
            nc = 4 if self.small else 16
            gs = (nc, 16, 1024, 1024)
            self._shared["cpart"] = self.d.Partition(gs, (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2))
            self._shared["cbytes"] = conv_algorithmic_bytes(_Geometry(gs, (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2)))
            self._shared["cout"] = _prod(gs)
            self._shared["cw"] = self.n(16, 5, 5) * 0.1
        return self._shared["cpart"]

    def _build_conv_fwd(self):
        torch, d, dev, part = self.torch, self.d, self.dev, self._conv_part()
        P, w = part.num_workers, self._shared["cw"]
        self.c_fwd = self._sets(lambda: ([self.n(*part.padded_shape(i)) for i in range(P)],
                                         [torch.empty(*part.bulk_shape(i), device=dev) for i in range(P)]))
        self.ops["conv_fwd"] = Op("conv_fwd", [(lambda s=s: d.conv_fwd(part, s[0], w, None, s[1])) for s in self.c_fwd],
                                  self._shared["cbytes"], 2 * 25 * self._shared["cout"], 1, "hbm")

    def _build_conv_adj(self):
        torch, d, dev, part = self.torch, self.d, self.dev, self._conv_part()
        P, w = part.num_workers, self._shared["cw"]
        self.c_adj = self._sets(lambda: ([self.n(*part.bulk_shape(i)) for i in range(P)],
                                         [torch.empty(*part.padded_shape(i), device=dev) for i in range(P)]))
        # the adjoint also clears the ghost cells of the padded dx shards (as H* does): one more write per ghost cell
        ghost = 4 * sum(a.numel() - b.numel() for b, a in zip(*self.c_adj[0]))
        self.ops["conv_adj"] = Op("conv_adj", [(lambda s=s: d.conv_adj(part, s[0], w, s[1])) for s in self.c_adj],
                                  self._shared["cbytes"] + ghost, 2 * 25 * self._shared["cout"], 1, "hbm")

    # ---- affine: x bf16 [256, 8192], W bf16 [8192, 8192] on a 4x4 grid ----
    def _affine(self):
        if "aff" not in self._shared:
            torch, dev = self.torch, self.dev
            nb, nf, pf = 256, 8192, 4
            blk = nf // pf
            sets = self._sets(lambda: dict(
                x=[self.n(nb, blk).bfloat16() for _ in range(pf)],
                w=[(self.n(blk, blk) * nf ** -0.5).bfloat16() for _ in range(pf * pf)],
                dy=[self.n(nb, blk).bfloat16() for _ in range(pf)],
                y=[torch.empty(nb, blk, device=dev) for _ in range(pf)],
                dx=[torch.empty(nb, blk, device=dev) for _ in range(pf)]))
            self._shared["aff"] = (nb, nf, pf, sets)
        return self._shared["aff"]

    def _build_affine_fwd(self):
        d = self.d
        nb, nf, pf, sets = self._affine()
        self.ops["affine_fwd"] = Op("affine_fwd",
                                    [(lambda s=s: d.affine_fwd(nb, nf, nf, pf, pf, s["x"], s["w"], None, s["y"])) for s in sets],
                                    nf * nf * 2 + nb * nf * 2 + nb * nf * 4, 2 * nb * nf * nf, 1, "tensor")

    def _build_affine_adj(self):
        d = self.d
        nb, nf, pf, sets = self._affine()
        self.ops["affine_adj"] = Op("affine_adj",
                                    [(lambda s=s: d.affine_adj(nb, nf, nf, pf, pf, s["dy"], s["w"], s["dx"])) for s in sets],
                                    nf * nf * 2 + nb * nf * 2 + nb * nf * 4, 2 * nb * nf * nf, 1, "tensor")

    def _build_affine_adj_params(self):
        torch, d, dev = self.torch, self.d, self.dev
        nb, nf, pf, sets = self._affine()
        blk = nf // pf
        outs = self._sets(lambda: ([torch.empty(blk, blk, device=dev) for _ in range(pf * pf)],
                                   [torch.empty(blk, device=dev) for _ in range(pf)]))
        self.ops["affine_adj_params"] = Op(
            "affine_adj_params",
            [(lambda s=s, o=o: d.affine_adj_params(nb, nf, nf, pf, pf, s["dy"], s["x"], o[0], o[1])) for s, o in zip(sets, outs)],
            nf * nf * 4 + 2 * nb * nf * 2 + nf * 4, 2 * nb * nf * nf, 2, "hbm")

    # ---- operators beyond the step ----
    def _build_pool_fwd(self):
        # 3 x 3 max pooling, stride 2, padding 1 on fp32 16x16x1024x1024 over 4x4 workers: ghost widths (1, 0)
        if "pool_fwd" in self.ops:
            return
        torch, d, dev = self.torch, self.d, self.dev
        nc = 4 if self.small else 16
        k, st, pad = (3, 3), (2, 2), ((1, 1), (1, 1))
        gsp = (nc, 16, 1024, 1024)
        hl, hh = [0, 0], [0, 0]
        for dim in (2, 3):
            lo, hi, _, _ = d.halo_widths_1d(gsp[dim], 4, k[dim - 2], st[dim - 2], 1, pad[dim - 2][0], pad[dim - 2][1])
            hl.append(lo)
            hh.append(hi)
        part = d.Partition(gsp, (1, 1, 4, 4), hl, hh)
        self._shared["ppart"] = part
        oh = ((gsp[2] + 2 - 3) // 2 + 1) // 4
        P = part.num_workers
        sets = self._sets(lambda: dict(
            x=[self.n(*part.padded_shape(w)) for w in range(P)],
            y=[torch.empty(nc, 16, oh, oh, device=dev) for _ in range(P)],
            arg=[torch.zeros(nc, 16, oh, oh, dtype=torch.int32, device=dev) for _ in range(P)],
            dy=[self.n(nc, 16, oh, oh) for _ in range(P)],
            dx=[torch.empty(*part.padded_shape(w), device=dev) for w in range(P)]))
        out_b = P * nc * 16 * oh * oh * 4
        need_b = P * nc * 16 * ((oh - 1) * 2 + 3) ** 2 * 4
        pad_b = sum(t.numel() for t in sets[0]["dx"]) * 4
        for s in sets:      # the adjoint reads the positions the forward recorded
            d.pool_fwd(part, s["x"], k, st, pad, d.POOL_MAX, s["y"], s["arg"])
        self.ops["pool_fwd"] = Op("pool_fwd", [(lambda s=s: d.pool_fwd(part, s["x"], k, st, pad, d.POOL_MAX, s["y"], s["arg"]))
                                               for s in sets], part.halo_stats(False)[2] + need_b + 2 * out_b, 0, 2, "hbm")
        self.ops["pool_adj"] = Op("pool_adj", [(lambda s=s: d.pool_adj(part, s["dy"], s["arg"], k, st, pad, d.POOL_MAX, s["dx"]))
                                               for s in sets], 2 * out_b + pad_b + part.halo_stats(True)[2], 0, 2, "hbm")

    _build_pool_adj = _build_pool_fwd

    def _build_stencil3d_fwd(self):
        # fused halo exchange + 25-point star (radius 4) on a 512^3 volume (4 x 4 x 4 workers)
        if "stencil3d_fwd" in self.ops:
            return
        torch, d, dev = self.torch, self.d, self.dev
        taps = [[0.05 * (1 + abs(k - 4)) * (-1) ** k for k in range(9)] for _ in range(3)]
        part = d.Partition((256, 512, 512), (2, 4, 4), (4,) * 3, (4,) * 3) if self.small else self._halo_part()
        nw = part.num_workers
        sets = self._sets(lambda: dict(
            x=[self.u(*part.padded_shape(w)) for w in range(nw)],
            y=[torch.empty(*part.bulk_shape(w), device=dev) for w in range(nw)],
            dx=[torch.empty(*part.padded_shape(w), device=dev) for w in range(nw)]))
        cells = _prod(part.global_shape)
        ghost_b = sum(t.numel() - y.numel() for t, y in zip(sets[0]["dx"], sets[0]["y"])) * 4
        st_bytes = 8 * cells + part.halo_stats(False)[2] - ghost_b
        for s in sets:
            d.stencil3d_fwd(part, s["x"], taps, s["y"])
        self.ops["stencil3d_fwd"] = Op("stencil3d_fwd", [(lambda s=s: d.stencil3d_fwd(part, s["x"], taps, s["y"])) for s in sets],
                                       st_bytes, 2 * 27 * cells, 1, "hbm")
        self.ops["stencil3d_adj"] = Op("stencil3d_adj", [(lambda s=s: d.stencil3d_adj(part, s["y"], taps, s["dx"])) for s in sets],
                                       st_bytes + ghost_b, 2 * 27 * cells, 1, "hbm")

    _build_stencil3d_adj = _build_stencil3d_fwd

    def _build_convg_fwd(self):
        # generalized convolution: 16 -> 16 channels, 5 x 5, channel partitions 2 x 2, feature space 2 x 2
        if "convg_fwd" in self.ops:
            return
        torch, d, dev = self.torch, self.d, self.dev
        gN = 1 if self.small else 4
        part = d.Partition((gN, 16, 1024, 1024), (1, 2, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
        self._shared["gpart"] = part
        ws = torch.empty(d.convg_adj_params_workspace(part, 16, 2, 5, 5), dtype=torch.uint8, device=dev)
        sets = self._sets(lambda: dict(
            x=[self.n(*part.padded_shape(w)) for w in range(8)],
            y=[self.n(gN, 8, 512, 512) for _ in range(8)],
            dx=[torch.empty(*part.padded_shape(w), device=dev) for w in range(8)],
            w=[self.n(8, 8, 5, 5) * 0.05 for _ in range(4)],
            dw=[torch.empty(8, 8, 5, 5, device=dev) for _ in range(4)]))
        g_flops = 2 * 25 * 16 * 16 * gN * 1024 * 1024
        g_bytes = 2 * gN * 16 * 1024 * 1024 * 4
        self.ops["convg_fwd"] = Op("convg_fwd", [(lambda s=s: d.convg_fwd(part, 16, 2, s["x"], s["w"], None, s["y"])) for s in sets],
                                   g_bytes, g_flops, 1, "alu")
        self.ops["convg_adj"] = Op("convg_adj", [(lambda s=s: d.convg_adj(part, 16, 2, s["y"], s["w"], s["dx"])) for s in sets],
                                   g_bytes, g_flops, 2, "alu")
        self.ops["convg_adj_params"] = Op(
            "convg_adj_params",
            [(lambda s=s: d.convg_adj_params(part, 16, 2, s["x"], s["y"], (5, 5), s["dw"], None, ws)) for s in sets],
            g_bytes, g_flops, 2, "alu")

    _build_convg_adj = _build_convg_fwd
    _build_convg_adj_params = _build_convg_fwd

    def _build_conv_adj_params(self):
        torch, d, dev, part = self.torch, self.d, self.dev, self._conv_part()
        P = part.num_workers
        ws = torch.empty(d.conv_adj_params_workspace(part, 5, 5), dtype=torch.uint8, device=dev)
        sets = self._sets(lambda: dict(x=[self.n(*part.padded_shape(i)) for i in range(P)],
                                       dy=[self.n(*part.bulk_shape(i)) for i in range(P)],
                                       dw=torch.empty(16, 5, 5, device=dev), db=torch.empty(16, device=dev)))
        self.ops["conv_adj_params"] = Op(
            "conv_adj_params",
            [(lambda s=s: d.conv_adj_params(part, s["x"], s["dy"], (5, 5), s["dw"], s["db"], ws)) for s in sets],
            self._shared["cbytes"], 2 * 25 * self._shared["cout"], 2, "hbm")

    def _build_repartition_fwd(self):
        # generalized all-to-all between a row and a column partition of a fp32 8192 x 8192 tensor (8 -> 8 workers)
        if "repartition_fwd" in self.ops:
            return
        torch, d, dev = self.torch, self.d, self.dev
        side = 8192
        rep = d.Repartition((side, side), (8, 1), (1, 8))
        self._shared["rep"] = rep
        sets = self._sets(lambda: ([self.u(side // 8, side) for _ in range(8)],
                                   [torch.empty(side, side // 8, device=dev) for _ in range(8)]))
        self.ops["repartition_fwd"] = Op("repartition_fwd", [(lambda s=s: d.repartition_fwd(rep, s[0], s[1])) for s in sets],
                                         2 * side * side * 4, 0, 1, "hbm")
        self.ops["repartition_adj"] = Op("repartition_adj", [(lambda s=s: d.repartition_adj(rep, s[1], s[0])) for s in sets],
                                         2 * side * side * 4, 0, 1, "hbm")

    _build_repartition_adj = _build_repartition_fwd

    def _build_partition_broadcast_fwd(self):
        # partition broadcast of the affine layer's x (1 x 4 workers -> 4 x 4 workers) at sixteen times its batch, so
        # that the operator moves more than L2 holds: fp32 [4096, 8192] as 4 column blocks, each copied to the 4 grid rows
        if "partition_broadcast_fwd" in self.ops:
            return
        torch, d, dev = self.torch, self.d, self.dev
        rows, blk, src_p, dst_p = (1024 if self.small else 4096), 2048, (1, 4), (4, 4)
        sets = self._sets(lambda: ([self.u(rows, blk) for _ in range(4)], [self.u(rows, blk) for _ in range(16)]))
        nb = 4 * rows * blk * 4
        self.ops["partition_broadcast_fwd"] = Op("partition_broadcast_fwd",
                                                 [(lambda s=s: d.partition_broadcast_fwd(src_p, dst_p, s[0], s[1])) for s in sets],
                                                 nb * (1 + 4), 0, 4, "hbm")
        self.ops["partition_broadcast_adj"] = Op("partition_broadcast_adj",
                                                 [(lambda s=s: d.partition_broadcast_adj(src_p, dst_p, s[1], s[0])) for s in sets],
                                                 nb * (1 + 4), 0, 4, "hbm")

    _build_partition_broadcast_adj = _build_partition_broadcast_fwd

    def step(self, bracket=None, events=None):
        """Enqueues the eight operators (buffer set 0); the operator named `bracket` gets an event before and after."""
        for op in self.step_ops:
            if op.name == bracket:
                events[0].record()
                op.calls[0]()
                events[1].record()
            else:
                op.calls[0]()

    # ---- end-to-end variant: inputs come from pinned host memory, results go back to it ----
    def e2e_setup(self):
        """Pinned host copies of every input and output, per operator, and the three streams of the pipeline."""
        torch = self.torch
        aff = self._shared["aff"][3][0]
        per_op = {
            "broadcast_fwd": ([self.b_sets[0][0]], self.b_sets[0][1]),
            "sumreduce_fwd": (self.r_sets[0][0], [self.r_sets[0][1]]),
            "halo_fwd": (self.h_x[0], self.h_x[0]),
            "halo_adj": (self.h_y[0], self.h_y[0]),
            "conv_fwd": (self.c_fwd[0][0] + [self._shared["cw"]], self.c_fwd[0][1]),
            "conv_adj": (self.c_adj[0][0], self.c_adj[0][1]),
            "affine_fwd": (aff["x"] + aff["w"], aff["y"]),
            "affine_adj": (aff["dy"], aff["dx"]),
        }
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        self.e2e_ops = [([(t, pin(t)) for t in per_op[o.name][0]], [(t, pin(t)) for t in per_op[o.name][1]], o)
                        for o in self.step_ops]
        for ins, _, _ in self.e2e_ops:
            for t, h in ins:
                h.copy_(t)
        torch.cuda.synchronize()
        self.h2d_bytes = sum(t.numel() * t.element_size() for ins, _, _ in self.e2e_ops for t, _ in ins)
        self.d2h_bytes = sum(t.numel() * t.element_size() for _, outs, _ in self.e2e_ops for t, _ in outs)
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        self.e2e_done = None

    def e2e_step(self):
        """One step through the public calls with host buffers on both ends: the inputs of every operator come
        from pinned host memory and its results go back to it.  Three streams: uploads, the operators, downloads;
        the upload of the next operator's inputs and the download of the previous one's results run while an
        operator computes, so both directions of the host link are busy.  The upload of an operator's inputs waits
        for the previous step's download of the same operator's results (some buffers are input and output at
        once) and for the previous step's last operator (the convolution weights are read by two of them), not for
        the whole previous step, so the uploads of a step overlap the downloads of the one before."""
        torch = self.torch
        main = torch.cuda.current_stream()
        if self.e2e_done is None:
            self.s_in.wait_stream(main)
            self.e2e_down = [None] * len(self.e2e_ops)
        else:
            self.s_in.wait_event(self.e2e_ran)
        for k, (ins, outs, op) in enumerate(self.e2e_ops):
            with torch.cuda.stream(self.s_in):
                if self.e2e_down[k] is not None:
                    self.s_in.wait_event(self.e2e_down[k])
                for t, h in ins:
                    t.copy_(h, non_blocking=True)
                up = torch.cuda.Event()
                up.record()
            main.wait_event(up)
            op.calls[0]()
            ran = torch.cuda.Event()
            ran.record(main)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(ran)
                for t, h in outs:
                    h.copy_(t, non_blocking=True)
                down = torch.cuda.Event()
                down.record()
            self.e2e_down[k] = down
        self.e2e_ran = ran
        self.e2e_done = down
        main.wait_event(self.e2e_done)      # the step is over when its last result has reached the host


def time_direct(torch, op, replays=3):
    """Milliseconds per launch of `op`: GRAPH_LAUNCHES launches cycling over the operator's buffer sets, captured
    once in a CUDA graph (no host work between launches) and replayed between one pair of events."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    n = GRAPH_LAUNCHES

    def body():
        for r in range(n):
            op.calls[r % len(op.calls)]()

    with torch.cuda.stream(side):
        body()                                  # warm-up, and every one-time set-up happens outside the capture
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            body()
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * n)


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
# CPU baseline: the oracle, as it stands, on a bounded sample of the same workload.  Nothing here
# touches the CUDA library: byte counts come from the oracle's own partition geometry.
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
            "sample / oracle seconds"
            % (lv["rows"], lv["edge"], lv["planes"], lv["feats"], lv["feats"]))


def oracle_sample_step(lv, seed=0):
    """One pass of the oracle over a bounded sample of the workload; returns (bytes, seconds, per-op GB/s)."""
    import numpy as np
    from threadpoolctl import threadpool_limits
    import oracle
    from paper_2006_03108_b200 import inputs      # seeded input generators only: no operator arithmetic, no CUDA
    res = {}
    clock = time.perf_counter
    with threadpool_limits(limits=1):
        src = inputs.uniform_pm1((lv["rows"], 4096), seed + 1)
        parts = [inputs.uniform_pm1((lv["rows"], 4096), seed + 10 + i) for i in range(8)]
        t = clock(); oracle.broadcast_fwd(src, 8); res["broadcast_fwd"] = (src.nbytes * 9, clock() - t)
        t = clock(); oracle.sumreduce_fwd(parts); res["sumreduce_fwd"] = (src.nbytes * 9, clock() - t)
        e = lv["edge"]
        part = oracle.Partition((2 * e,) * 3, (2,) * 3, 4, 4)
        x = [inputs.uniform_pm1(part.padded_shape(w), seed + 100 + w) for w in range(8)]
        hb = halo_algorithmic_bytes(part)
        t = clock(); oracle.halo_fwd_sequence(part, x); res["halo_fwd"] = (hb[0], clock() - t)
        t = clock(); oracle.halo_adj_sequence(part, x); res["halo_adj"] = (hb[1], clock() - t)
        pl = lv["planes"]
        cshape = (1, pl, 1024, 1024)
        cpart = oracle.Partition(cshape, (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2))
        xg = inputs.normal(cshape, seed + 200)
        w = inputs.normal((pl, 5, 5), seed + 201, 0.1)
        xs = oracle.scatter_global(cpart, xg)
        dys = oracle.scatter_global(oracle.Partition(cshape, (1, 1, 4, 4)), xg)
        cbytes = conv_algorithmic_bytes(cpart)
        t = clock(); oracle.conv_fwd(cpart, xs, w); res["conv_fwd"] = (cbytes, clock() - t)
        t = clock(); oracle.conv_adj(cpart, dys, w); res["conv_adj"] = (cbytes, clock() - t)
        nb, nf, pf = 256, lv["feats"], 4
        xa = [inputs.normal((nb, nf // pf), seed + 300 + j).astype(np.float64) for j in range(pf)]
        wa = [inputs.normal((nf // pf, nf // pf), seed + 310 + i, nf ** -0.5).astype(np.float64) for i in range(pf * pf)]
        abytes = nf * nf * 2 + nb * nf * 2 + nb * nf * 4
        t = clock(); oracle.affine_fwd(xa, wa, pf, pf); res["affine_fwd"] = (abytes, clock() - t)
        t = clock(); oracle.affine_adj(xa, wa, pf, pf); res["affine_adj"] = (abytes, clock() - t)
    nbytes = sum(v[0] for v in res.values())
    secs = sum(v[1] for v in res.values())
    return nbytes, secs, {k: round(v[0] / v[1] / 1e9, 3) for k, v in res.items()}


def _oracle_worker(args):
    lv, seed = args
    t0 = time.time()
    b, s, _ = oracle_sample_step(lv, seed)
    return b, s, t0, time.time()


class OraclePool:
    """The oracle on every host core: one process per core, each running the one-thread sample on inputs of its
    own.  The pool is started with `spawn` before the first GPU call of the parent."""

    MAX_PROCS = 32

    def __init__(self):
        import multiprocessing as mp
        self.cores = max(1, min(len(os.sched_getaffinity(0)), self.MAX_PROCS))
        self.pool = mp.get_context("spawn").Pool(self.cores)

    def run(self, lv):
        jobs = [(lv, 1000 * (i + 1)) for i in range(self.cores)]
        out = self.pool.map(_oracle_worker, jobs)
        self.pool.close()
        self.pool.join()
        nbytes = sum(o[0] for o in out)
        wall = max(o[3] for o in out) - min(o[2] for o in out)
        return {"value": round(nbytes / wall / 1e9, 3), "unit": UNIT, "cores": self.cores, "kind": "oracle",
                "sample": "%d processes at once, one thread each; each: %s" % (self.cores, oracle_sample_text(lv))}


def run_reference(args, rank):
    """The oracle arm: K steps (after W warm-up steps) of the oracle on a bounded sample, rank 0 only."""
    if rank != 0:
        return
    lv = oracle_level(args.steps + args.warmup)
    sample = oracle_sample_text(lv) + "; numpy limited to one thread"
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


def reduce_max_ms(ms, world, dist=None, torch=None, dev=None):
    """Max over ranks of a device time (the figure a multi-GPU run reports)."""
    if world <= 1:
        return float(ms)
    t = torch.tensor([ms], device=dev, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_step, world, ms_per_step):
    """Whole-job GB/s: every rank moves `bytes_per_step` on its own replica in the slowest rank's step time."""
    return world * bytes_per_step / (ms_per_step * 1e-3) / 1e9


# ----------------------------------------------------------------------------------------------
# Main
# ----------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-ops", action="store_true")
    ap.add_argument("--profile-op", default=None,
                    help="run only this operator, three times, on a reduced case (for profiler captures) and exit")
    ap.add_argument("--profile-full", action="store_true",
                    help="with --profile-op: the operator's full-size case (only its own buffers are allocated)")
    ap.add_argument("--halo-case", default="full", choices=sorted(HALO_CASES),
                    help="with --profile-op halo_fwd / halo_adj: exchange along one dimension only (see HALO_CASES)")
    ap.add_argument("--halo-classes", action="store_true",
                    help="time H and H* of the 512^3 tensor for every entry of HALO_CASES and print one JSON object")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    # the all-cores oracle leg runs in processes of its own, started before this process touches the GPU
    pool = None
    if world == 1 and not args.no_cpu_baseline and not args.profile_op:
        pool = OraclePool()

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
    import paper_2006_03108_b200 as distdl

    if args.halo_classes:
        table = {}
        for case in ("z", "y", "x", "zy", "full"):
            wl = Workload(dev, ["halo_fwd", "halo_adj"], nsets=3, halo_case=case)
            row = {}
            for name in ("halo_fwd", "halo_adj"):
                op = wl.ops[name]
                ms = time_direct(torch, op)
                row[name] = {"bytes": op.bytes, "us": round(ms * 1e3, 2), "gbs": round(op.bytes / ms / 1e6, 1),
                             "frac_hbm": round(op.bytes / ms / 1e6 / peaks["hbm"], 4)}
            table[case] = {"workers": HALO_CASES[case][0], "halo": HALO_CASES[case][1], **row}
            del wl
            torch.cuda.empty_cache()
        print(json.dumps({"halo_classes": table, "peak_gbs": peaks["hbm"], "peak_source": peaks["source"]}))
        return

    if args.profile_op:
        wl = Workload(dev, [args.profile_op], small=not args.profile_full, nsets=1, halo_case=args.halo_case)
        op = wl.ops[args.profile_op]
        for _ in range(3):
            op.calls[0]()
        torch.cuda.synchronize()
        distdl.device_status()
        print(json.dumps({"profile_op": args.profile_op, "algorithmic_bytes": op.bytes, "flops": op.flops,
                          "full_size": bool(args.profile_full)}))
        return

    wl = Workload(dev, STEP_OPS, nsets=3)
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- every operator of the step timed directly (cold buffers, no host work between launches) ----
    direct_ms = {o.name: time_direct(torch, o) for o in wl.step_ops}
    top = max(direct_ms, key=direct_ms.get)

    # ---- timed region: K steps; the launch with the largest share carries an event pair in every step ----
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid) if rank == 0 else None
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for s in range(args.steps):
        wl.step(top, ev[s])
    t_stop.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    elapsed_ms = reduce_max_ms(t_start.elapsed_time(t_stop), world, dist, torch, dev)
    top_ms = statistics.fmean(ev[s][0].elapsed_time(ev[s][1]) for s in range(args.steps))
    ms_per_step = elapsed_ms / args.steps
    value = aggregate_value(wl.bytes_per_step, world, ms_per_step)
    distdl.device_status()

    # ---- the small 2-D configuration (256 x 256 on 2 x 2 workers, halo 1): launch-bound, so H + H* are timed as
    # separate calls and as replays of a CUDA graph that holds 50 such pairs ----
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
    nb = sum(halo_algorithmic_bytes(_Geometry((256, 256), (2, 2), (1, 1), (1, 1))))
    small_cfg = {"workload": "H + H* on fp32 256x256, 2x2 workers, halo 1 (%d algorithmic bytes per pair)" % nb,
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
    e2e_ms = reduce_max_ms(e0.elapsed_time(e1), world, dist, torch, dev)
    e2e_value = aggregate_value(wl.bytes_per_step, world, e2e_ms / args.e2e_steps)
    h2d, d2h = wl.h2d_bytes, wl.d2h_bytes
    step_ops, bytes_per_step, launches_per_step = wl.step_ops, wl.bytes_per_step, wl.launches_per_step
    del wl
    torch.cuda.empty_cache()

    # ---- the operators outside the step, each timed on its own (not part of `value`) ----
    extra = {}
    if rank == 0 and not args.no_extra_ops:
        for group in EXTRA_GROUPS:
            xw = Workload(dev, group[:1], nsets=3)
            for name in group:
                if name in xw.ops:
                    op = xw.ops[name]
                    extra[name] = (Op(name, None, op.bytes, op.flops, op.launches, op.bound), time_direct(torch, op))
            del xw
            torch.cuda.empty_cache()
        distdl.device_status()

    def entry(op, ms):
        e = {"ms": round(ms, 5), "gbs": round(op.bytes / ms / 1e6, 1), "bound": op.bound,
             "frac_hbm": round(op.bytes / ms / 1e6 / peaks["hbm"], 4)}
        if op.flops:
            e["tflops"] = round(op.flops / ms / 1e9, 2)
        if op.bound == "tensor":
            e["frac_tensor"] = round(op.flops / ms / 1e9 / peaks["bf16"], 4)                      # of the burst figure
            e["frac_tensor_sustained"] = round(op.flops / ms / 1e9 / peaks["bf16_sustained"], 4)
        if op.bound == "alu":
            e["frac_alu"] = round(op.flops / ms / 1e9 / FP32_PEAK_TFLOPS, 4)
        return e

    if rank == 0:
        ops = {o.name: entry(o, direct_ms[o.name]) for o in step_ops}
        topop = [o for o in step_ops if o.name == top][0]
        achieved = topop.bytes / top_ms / 1e6
        roofline = {"kernel": top, "bound": topop.bound, "achieved": round(achieved, 1), "peak": peaks["hbm"],
                    "unit": "GB/s", "frac": round(achieved / peaks["hbm"], 4), "traffic": NCU_TRAFFIC.get(top),
                    "peak_source": "of " + peaks["source"], "ms_in_step": round(top_ms, 5),
                    "share_of_step": round(top_ms / ms_per_step, 3)}
        dm = ("broadcast_fwd", "sumreduce_fwd", "halo_fwd", "halo_adj")
        dm_bytes = sum(o.bytes for o in step_ops if o.name in dm)
        dm_ms = sum(direct_ms[o.name] for o in step_ops if o.name in dm)
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 (bf16 inputs, f32 accumulation in the affine layer)",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "l2": "inputs larger than L2: the 6.9 GB working set of a step cycles through between two "
                             "launches of the same operator; the affine forward and adjoint, which read the same "
                             "134 MB of weights, are kept 2.7 GB of other operators' traffic apart (order: %s); "
                             "per-operator figures: %d launches from a CUDA graph cycling over 3 disjoint buffer "
                             "sets between one pair of events" % (", ".join(STEP_ORDER), GRAPH_LAUNCHES),
                       "bytes_per_step": bytes_per_step},
            "frac_of_hbm_peak": round(value / world / peaks["hbm"], 4),
            "halo_bcast_reduce": {"gbs": round(dm_bytes / dm_ms / 1e6, 1),
                                  "frac_of_hbm_peak": round(dm_bytes / dm_ms / 1e6 / peaks["hbm"], 4)},
            "ops": ops,
            "extra_ops": {"note": "timed like `ops`, not part of value: 3x3 max pooling, stride 2, padding 1 on fp32 "
                                  "16x16x1024x1024 over 4x4 workers (H + local kernel, local adjoint + H*); parameter "
                                  "gradients of the step's convolution (dw, db) and affine layer (dW, db); fused halo + radius-4 star stencil "
                                  "on a 512^3 volume (4x4x4 workers); generalized convolution 16 -> 16 channels, 5x5, fp32 "
                                  "4x16x1024x1024 on channel partitions 2x2 and 2x2 feature-space workers; generalized "
                                  "all-to-all of fp32 8192x8192 between 8 row blocks and 8 column blocks; partition "
                                  "broadcast / sum-reduce of fp32 4096x8192 from 1x4 to 4x4 workers",
                          **{k: entry(v[0], v[1]) for k, v in extra.items()}},
            "small_config": small_cfg,
            "roofline": roofline,
            "clocks": clocks,
            "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": args.e2e_steps},
            "gpu_launches": launches_per_step * args.steps,
        }
        if world == 1 and not args.no_cpu_baseline:
            lv = ORACLE_LEVELS[0]
            b, s, per = oracle_sample_step(lv)
            line["cpu_baseline"] = {"value": round(b / s / 1e9, 3), "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": oracle_sample_text(lv) + "; numpy limited to one thread", "per_op_gbs": per}
            if pool is not None:
                line["cpu_baseline_all_cores"] = pool.run(ORACLE_LEVELS[1])
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) per launch from the committed ncu summaries under profiles/ (one launch of
# `bench.py --profile-op <op>`: full size for H, H*, the affine layer and -- with --profile-full and the two DRAM
# byte counters alone -- the convolution; the quarter-size case scaled by 4 for R, whose traffic grows with the
# number of rows); None for a kernel whose counters were not meaningful (the broadcast's output was still in L2
# when the short capture ended) or that changed since its counters were taken.
NCU_TRAFFIC = {
    "broadcast_fwd": None,
    "sumreduce_fwd": 4 * (134225152 + 5290496),
    "halo_fwd": 194266368 + 124569856,
    "halo_adj": (107870464 + 72062976) + (139435264 + 39406592),      # box kernel + row-end kernel
    "conv_fwd": 1137867008 + 1029683968,
    "conv_adj": 1099090944 + 1063217152,
    "affine_fwd": 138435072 + 3728128,
    "affine_adj": 138447104 + 3240448,
}

if __name__ == "__main__":
    main()
