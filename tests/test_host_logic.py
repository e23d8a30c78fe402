"""CPU tests of the host side of the library: the shared object loads and exports every symbol the
header declares, the planner's geometry and byte counts, and the error codes of the validation paths.
No kernel is launched here."""

import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2006_03108_b200 as distdl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(inc, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(distdl_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(distdl.LIB_PATH)
    names = _declared_symbols()
    assert len(names) >= 19
    for n in names:
        assert hasattr(lib, n), "libdistdl.so does not export %s" % n


APPENDIX_B = [
    # n, p, kernel, stride, pad -> halo_lo, halo_hi, unused_lo, unused_hi   (Figs. B1-B4)
    ((11, 3, 5, 1, 2), ([2, 2, 2], [2, 2, 2], [0, 0, 0], [0, 0, 0])),
    ((11, 3, 5, 1, 0), ([0, 1, 3], [3, 1, 0], [0, 0, 0], [0, 0, 0])),
    ((10, 3, 2, 2, 0), ([0, 0, 0], [0, 1, 0], [0, 0, 1], [0, 0, 0])),
    ((20, 6, 2, 2, 0), ([0] * 6, [0, 0, 1, 2, 1, 0], [0, 0, 0, 1, 2, 1], [0] * 6)),
]


@pytest.mark.parametrize("args,expect", APPENDIX_B)
def test_halo_widths_match_appendix_b_and_the_oracle(args, expect):
    n, p, k, s, pad = args
    got = distdl.halo_widths_1d(n, p, k, stride=s, pad_lo=pad, pad_hi=pad)
    assert tuple(got) == expect
    ref = oracle.halo_widths_1d(n, p, k, s, 1, pad, pad)
    assert list(got[0]) == [r["halo_lo"] for r in ref] and list(got[1]) == [r["halo_hi"] for r in ref]
    assert list(got[2]) == [r["unused_lo"] for r in ref] and list(got[3]) == [r["unused_hi"] for r in ref]


@pytest.mark.parametrize("n,p,k,s,d,pl,ph", [(37, 5, 3, 2, 2, 1, 0), (64, 7, 4, 3, 1, 2, 2), (9, 9, 3, 1, 1, 1, 1), (50, 4, 7, 1, 3, 0, 5)])
def test_halo_widths_random_cases_against_the_oracle(n, p, k, s, d, pl, ph):
    got = distdl.halo_widths_1d(n, p, k, stride=s, dilation=d, pad_lo=pl, pad_hi=ph)
    ref = oracle.halo_widths_1d(n, p, k, s, d, pl, ph)
    for i, key in enumerate(["halo_lo", "halo_hi", "unused_lo", "unused_hi"]):
        assert list(got[i]) == [r[key] for r in ref]


def test_shard_extents_match_the_oracle_partition():
    cases = [((11,), (3,), [2], [2]), ((67, 61, 68), (3, 2, 2), [2, 4, 4], [3, 4, 4]),
             ((9, 8), (2, 2), [[0, 4], [0, 3]], [[2, 0], [0, 0]])]
    for gs, ps, lo, hi in cases:
        g = distdl.Partition(gs, ps, lo, hi)
        o = oracle.Partition(gs, ps, lo, hi)
        assert g.num_workers == o.num_workers
        for w in range(o.num_workers):
            st, bulk, padded, hl, hh = g.shard_extents(w)
            assert st == o.bulk_start(w) and bulk == o.bulk_shape(w) and padded == o.padded_shape(w)
            assert (hl, hh) == o.widths(w)


def test_plan_bytes_of_the_baseline_configurations():
    # 2-D: 4 shards of 130^2, width 1.  3-D: 64 shards of 136^3, width 4.
    p1 = distdl.Partition((256, 256), (2, 2), (1, 1), (1, 1))
    assert p1.halo_stats(False) == (32, 32, 12368)
    assert p1.halo_stats(True)[2] == 20528
    p3 = distdl.Partition((512,) * 3, (4,) * 3, (4,) * 3, (4,) * 3)
    boxes, tiles, nbytes = p3.halo_stats(False)
    assert boxes == 64 * 26 and nbytes == 186177536
    assert p3.halo_stats(True)[2] == 330205184
    # independent count: ghost cells written + interior ghost cells read (fp32)
    ghost = 64 * (136 ** 3 - 128 ** 3)
    interior = sum(np.prod([min(s + 132, 512) - max(s - 4, 0) for s in (a, b, c)]) - 128 ** 3
                   for a in range(0, 512, 128) for b in range(0, 512, 128) for c in range(0, 512, 128))
    assert nbytes == 4 * (ghost + int(interior))


def _status(fn, *a, **k):
    with pytest.raises(distdl.DistdlError) as e:
        fn(*a, **k)
    return e.value.status


def test_partition_validation_errors():
    assert _status(distdl.Partition, (4, 4), (8, 1)) == 2                       # fewer cells than workers
    assert _status(distdl.Partition, (8, 8), (4, 1), (3, 0), (0, 0)) == 2        # ghost wider than the neighbour
    assert _status(distdl.Partition, (8,) * 6, (1,) * 6) == 1                    # rank > 5
    assert _status(distdl.Partition, (1024, 1024), (32, 32)) == 4                # > 256 workers
    assert _status(distdl.Partition, (8, 8), (2, 2), (-1, 0), (0, 0)) == 2
    assert _status(distdl.halo_widths_1d, 4, 2, 9) == 2                          # kernel larger than the input


class _FakeTensor:
    """Stands in for a device tensor: only the address and the size are looked at before launch."""

    def __init__(self, addr, numel=16):
        self._addr, self._n = addr, numel
        import torch
        self.dtype = torch.float32

    def data_ptr(self):
        return self._addr

    def numel(self):
        return self._n


def test_operator_argument_validation_without_a_device():
    ok, odd = _FakeTensor(0x10000), _FakeTensor(0x10004)
    assert _status(distdl.broadcast_fwd, odd, [ok], stream=0) == 3               # alignment
    assert _status(distdl.broadcast_fwd, ok, [odd], stream=0) == 3
    assert _status(distdl.sumreduce_fwd, [ok, _FakeTensor(0)], ok, stream=0) == 1  # NULL source
    assert _status(distdl.sumreduce_fwd, [_FakeTensor(0x20000), ok], ok, stream=0) == 1  # dst aliases source 1
    part = distdl.Partition((8, 8), (2, 2), (1, 1), (1, 1))
    import torch
    if not torch.cuda.is_available():
        # created without a device: geometry works, operators refuse
        assert _status(distdl.halo_fwd, part, [ok] * 4, stream=0) == 5
    lib = distdl.lib()
    vp = ctypes.c_void_p
    arr = (vp * 4)(0x10000, 0x20000, 0x30000, 0x40000)
    assert lib.distdl_affine_fwd(16, 100, 128, 1, 1, arr, arr, None, arr, None) == 4   # block not a multiple of 8
    assert lib.distdl_affine_fwd(16, 256, 256, 3, 1, arr, arr, None, arr, None) == 2   # not divisible by the grid
    assert lib.distdl_conv_fwd(part.handle, arr, vp(0x50000), None, 3, 3, arr, None) == 2  # not a rank-4 partition
    p4 = distdl.Partition((1, 2, 16, 16), (1, 1, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
    assert lib.distdl_conv_fwd(p4.handle, arr, vp(0x50000), None, 3, 3, arr, None) == 2    # widths do not match 3x3
    assert lib.distdl_conv_fwd(p4.handle, arr, vp(0x50000), None, 4, 4, arr, None) == 4    # even kernel
    assert lib.distdl_last_error().decode() != ""


def test_validation_of_the_gradient_stencil_and_dtype_entry_points():
    lib = distdl.lib()
    vp = ctypes.c_void_p
    arr = (vp * 16)(*[0x10000 * (i + 1) for i in range(16)])
    # affine parameter gradients
    assert lib.distdl_affine_adj_params(16, 100, 128, 1, 1, arr, arr, arr, None, None) == 4   # block not a multiple of 8
    assert lib.distdl_affine_adj_params(16, 256, 256, 3, 1, arr, arr, arr, None, None) == 2   # not divisible by the grid
    assert lib.distdl_affine_adj_params(16, 256, 256, 1, 1, None, arr, arr, None, None) == 1  # NULL argument
    odd = (vp * 1)(0x10004)
    assert lib.distdl_affine_adj_params(16, 128, 128, 1, 1, odd, arr, arr, None, None) == 3   # alignment
    # convolution parameter gradients: the geometry is checked before anything touches a device
    p2 = distdl.Partition((8, 8), (2, 2), (1, 1), (1, 1))
    p4 = distdl.Partition((1, 2, 16, 16), (1, 1, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
    n = ctypes.c_int64(0)
    assert lib.distdl_conv_adj_params_workspace(p2.handle, 3, 3, ctypes.byref(n)) == 2          # not rank 4
    assert lib.distdl_conv_adj_params_workspace(p4.handle, 3, 3, ctypes.byref(n)) == 2          # widths do not match 3x3
    assert lib.distdl_conv_adj_params_workspace(p4.handle, 4, 4, ctypes.byref(n)) == 4          # even kernel
    assert lib.distdl_conv_adj_params_workspace(p4.handle, 5, 5, None) == 1
    assert lib.distdl_conv_adj_params(p4.handle, arr, arr, 5, 5, vp(0x50000), None, None, 0, None) == 1   # no workspace
    # star stencil
    taps = (ctypes.c_float * 27)(*([0.5] * 27))
    p3 = distdl.Partition((8, 8, 8), (2, 1, 1), (2, 2, 2), (2, 2, 2))
    assert lib.distdl_stencil3d_fwd(p2.handle, arr, taps, 1, arr, None) == 2                    # not rank 3
    assert lib.distdl_stencil3d_fwd(p3.handle, arr, taps, 5, arr, None) == 4                    # radius beyond 4
    assert lib.distdl_stencil3d_fwd(p3.handle, arr, taps, 1, arr, None) == 2                    # halo width is not the radius
    assert lib.distdl_stencil3d_adj(p3.handle, arr, None, 2, arr, None) == 1
    odd8 = (vp * 2)(0x10008, 0x20000)
    assert lib.distdl_stencil3d_fwd(p3.handle, odd8, taps, 2, arr, None) == 3                   # alignment
    with pytest.raises(ValueError):
        distdl.stencil3d_fwd(p3, [], [[1.0, 2.0]] * 3, [])                                      # even tap count
    # element types
    assert lib.distdl_sumreduce_fwd(arr, vp(0x90000), 2, 8, 7, None) == 1                       # unknown dtype
    assert lib.distdl_broadcast_fwd(vp(0x90000), arr, 2, 8, 7, None) == 1
    p64 = distdl.Partition((9, 9), (2, 2), (1, 1), (1, 1), dtype=distdl.F64)
    assert p64.halo_stats(False)[2] == 2 * distdl.Partition((9, 9), (2, 2), (1, 1), (1, 1)).halo_stats(False)[2]
    r64 = distdl.Repartition((12, 8), (3, 1), (1, 2), distdl.F64)
    assert r64.shard_shape(0) == (4, 8) and r64.shard_shape(1, destination=True) == (12, 4)


def test_periodic_partition_geometry_and_refusals():
    lib = distdl.lib()
    vp = ctypes.c_void_p
    # 8 x 8 on 2 x 2 workers, width 1: 20 ghost cells per shard; all of them have an owner when both
    # dimensions wrap (20 reads + 20 writes of 4 bytes per shard), only 9 of them (a row, a column, a corner) otherwise
    per = distdl.Partition((8, 8), (2, 2), (1, 1), (1, 1), periodic=(True, True))
    flat = distdl.Partition((8, 8), (2, 2), (1, 1), (1, 1))
    assert per.halo_stats(False)[2] == 4 * (20 + 20) * 4
    assert flat.halo_stats(False)[2] == 4 * (20 + 9) * 4
    # adjoint: every ghost read and cleared (8 B), every bulk cell in reach of a face read and written (8 B):
    # all 12 cells of the bulk's rim with both dimensions periodic, 7 of them (one row, one column) otherwise
    assert per.halo_stats(True)[2] == 4 * (20 * 8 + 12 * 8)
    assert flat.halo_stats(True)[2] == 4 * (20 * 4 + 9 * 4 + 7 * 8)
    # the ghost-width rule holds across the seam as well
    assert _status(distdl.Partition, (6,), (2,), (4,), (0,), periodic=(True,)) == 2
    # a worker alone along a periodic dimension is its own neighbour
    one = distdl.Partition((7,), (1,), (2,), (3,), periodic=(True,))
    assert one.halo_stats(False)[2] == (5 + 5) * 4 and one.halo_stats(True)[0] >= 1
    # fused layers take no periodic partitions
    arr = (vp * 16)(*[0x10000 * (i + 1) for i in range(16)])
    p4 = distdl.Partition((1, 2, 16, 16), (1, 1, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2), periodic=(False, False, True, True))
    assert lib.distdl_conv_fwd(p4.handle, arr, vp(0x50000), None, 5, 5, arr, None) == 4
    p3 = distdl.Partition((8, 8, 8), (2, 1, 1), (2, 2, 2), (2, 2, 2), periodic=(True, False, False))
    taps = (ctypes.c_float * 15)(*([0.5] * 15))
    assert lib.distdl_stencil3d_fwd(p3.handle, arr, taps, 2, arr, None) == 4


def test_validation_of_the_generalized_convolution():
    lib = distdl.lib()
    vp = ctypes.c_void_p
    arr = (vp * 64)(*[0x10000 * (i + 1) for i in range(64)])
    px = distdl.Partition((1, 4, 16, 16), (1, 2, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
    assert lib.distdl_convg_fwd(px.handle, 6, 2, arr, arr, None, 3, 3, arr, None) == 2          # widths do not match 3x3
    assert lib.distdl_convg_fwd(px.handle, 6, 2, arr, arr, None, 4, 4, arr, None) == 4          # even kernel
    assert lib.distdl_convg_fwd(px.handle, 1, 2, arr, arr, None, 5, 5, arr, None) == 2          # fewer channels than blocks
    assert lib.distdl_convg_fwd(px.handle, 18, 9, arr, arr, None, 5, 5, arr, None) == 4         # more than 8 channel blocks
    assert lib.distdl_convg_adj(px.handle, 6, 2, None, arr, 5, 5, arr, None) == 1
    pb = distdl.Partition((2, 4, 16, 16), (2, 1, 2, 2), (0, 0, 2, 2), (0, 0, 2, 2))
    assert lib.distdl_convg_fwd(pb.handle, 6, 2, arr, arr, None, 5, 5, arr, None) == 4          # batch partitioned
    odd = (vp * 8)(*[0x10004 + 0x10000 * i for i in range(8)])
    assert lib.distdl_convg_fwd(px.handle, 6, 2, odd, arr, None, 5, 5, arr, None) == 3          # alignment


def test_header_compiles_as_c_and_the_library_links_from_c(tmp_path):
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    exe = str(tmp_path / "host_check")
    libdir = os.path.dirname(distdl.LIB_PATH)
    subprocess.check_call([gcc, "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c_abi", "host_check.c"), "-o", exe,
                           "-L", libdir, "-ldistdl", "-Wl,-rpath," + libdir])
    out = subprocess.run([exe], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip().endswith("ok"), out.stdout + out.stderr


@pytest.mark.parametrize("gs,ps,lo,hi", [
    ((512, 512, 512), (4, 4, 4), (4, 4, 4), (4, 4, 4)),
    ((256, 256), (2, 2), (1, 1), (1, 1)),
    ((70, 66, 72), (2, 3, 2), (4, 2, 3), (1, 4, 2)),
    ((37, 45), (3, 2), (2, 1), (1, 3)),
    ((9, 40), (4, 1), (2, 3), (2, 0)),            # shards as thin as their neighbours' ghosts
    ((16, 16, 1024, 1024), (1, 1, 4, 4), (0, 0, 2, 2), (0, 0, 2, 2)),
])
def test_bench_byte_counts_from_oracle_geometry_match_the_planner(gs, ps, lo, hi):
    """bench.py counts the algorithmic bytes of H, H* and the convolution from partition geometry alone (the
    oracle's Partition, or its own extents-only stand-in); the library's planner counts them from its box lists."""
    import bench
    gp = distdl.Partition(gs, ps, lo, hi)
    want = (gp.halo_stats(False)[2], gp.halo_stats(True)[2])
    assert bench.halo_algorithmic_bytes(oracle.Partition(gs, ps, lo, hi)) == want
    assert bench.halo_algorithmic_bytes(bench._Geometry(gs, ps, lo, hi)) == want
    if len(gs) == 4:
        a = bench.conv_algorithmic_bytes(oracle.Partition(gs, ps, lo, hi))
        assert a == bench.conv_algorithmic_bytes(bench._Geometry(gs, ps, lo, hi)) == 2172796928


def test_bench_reference_arm_does_not_load_the_cuda_library():
    """`bench.py --impl reference` and the CPU-baseline leg time the oracle alone."""
    import subprocess, sys
    code = ("import sys, bench; b, s, per = bench.oracle_sample_step(bench.ORACLE_LEVELS[2]); "
            "import paper_2006_03108_b200 as d; assert d._lib is None, 'library was loaded'; "
            "assert b > 0 and s > 0; print('ok')")
    r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == "ok", r.stderr


def test_partition_broadcast_rejects_shapes_that_do_not_broadcast():
    lib = distdl.lib()
    one = ctypes.c_void_p(256)
    ptrs = (ctypes.c_void_p * 8)(*[256] * 8)
    elems = (ctypes.c_int64 * 8)(*[4] * 8)

    def call(src_p, dst_p):
        r = len(src_p)
        return lib.distdl_partition_broadcast_fwd(r, (ctypes.c_int32 * r)(*src_p), (ctypes.c_int32 * r)(*dst_p), elems,
                                                  ptrs, ptrs, distdl.F32, None)
    assert call((2, 2), (4, 2)) == 2 and b"dimension 0" in lib.distdl_last_error()       # DISTDL_ERR_SHAPE
    assert call((2, 1), (1, 2)) == 2
    assert call((1,), (512,)) == 4                                                        # DISTDL_ERR_UNSUPPORTED
    assert lib.distdl_partition_broadcast_fwd(1, None, None, elems, ptrs, ptrs, distdl.F32, None) == 1
