"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration that
bench.py times.  B, R, H, H*, the all-to-all and the affine layer are compared in full; the convolution
and the pooling layer on sampled (n, c) planes, the star stencil and the generalized convolution on sampled boxes,
the parameter gradients on
sampled channels / worker blocks, which the oracle computes one by one; properties that hold at any size
(zero ghosts, dot test) over everything."""

import numpy as np
import pytest

import oracle
import paper_2006_03108_b200 as distdl
from paper_2006_03108_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

DEV = "cuda:0"
dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
host = lambda t: t.cpu().numpy()


def _need_free_gb(gb):
    """The largest-size cases hold tens of GB on the device; they are skipped where that much is not free."""
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < gb * (1 << 30):
        pytest.skip("needs %d GB of free device memory, %.0f GB are free" % (gb, free / (1 << 30)))


def test_broadcast_and_sumreduce_full_size():
    k, shape = 8, (4096, 4096)
    x = inputs.uniform_pm1(shape, 2001)
    dst = [torch.empty(shape, device=DEV) for _ in range(k)]
    distdl.broadcast_fwd(dev(x), dst)
    torch.cuda.synchronize()
    for d in dst:
        assert host(d).tobytes() == x.tobytes()
    parts = [inputs.uniform_pm1(shape, 2010 + i) for i in range(k)]
    out = torch.empty(shape, device=DEV)
    distdl.sumreduce_fwd([dev(p) for p in parts], out)
    torch.cuda.synchronize()
    assert host(out).tobytes() == oracle.sumreduce_fwd(parts).tobytes()


def _long_vector(n, seed):
    """n fp32 values on the device: a seeded block of 2^24 values repeated, plus the number of the repeat
    (exact in fp32), so that no two positions 2^24 k apart, and none 2^31 or 2^32 apart, hold the same value."""
    blk = 1 << 24
    block = dev(inputs.uniform_pm1((blk,), seed))
    x = torch.empty(n, device=DEV)
    for seg in range((n + blk - 1) // blk):
        lo, hi = seg * blk, min(n, (seg + 1) * blk)
        torch.add(block[: hi - lo], float(seg), out=x[lo:hi])
    return x


def test_broadcast_and_sumreduce_beyond_2_to_31_elements():
    """Element counts above 2^31 (and byte counts above 2^33) with a ragged tail: the copies are compared
    in full as bit patterns on the device, the fold against the oracle on windows at the start, around
    element 2^31 and at the end, and against the single correctly rounded fp32 sum everywhere."""
    _need_free_gb(40)
    n = (1 << 31) + (1 << 20) + 3
    windows = [(0, 1 << 16), ((1 << 31) - (1 << 16), (1 << 31) + (1 << 16)), (n - (1 << 16) - 3, n)]
    x = _long_vector(n, 2101)
    dst = [torch.empty(n, device=DEV) for _ in range(2)]
    distdl.broadcast_fwd(x, dst)
    torch.cuda.synchronize()
    for d in dst:
        assert torch.equal(d.view(torch.int32), x.view(torch.int32))
        for lo, hi in windows:
            assert host(d[lo:hi]).tobytes() == host(x[lo:hi]).tobytes()
    del dst
    y = _long_vector(n, 2102)
    out = torch.empty(n, device=DEV)
    distdl.sumreduce_fwd([x, y], out)
    torch.cuda.synchronize()
    for lo, hi in windows:
        ref = oracle.sumreduce_fwd([host(x[lo:hi]), host(y[lo:hi])])
        assert host(out[lo:hi]).tobytes() == ref.tobytes()
    y.add_(x)                        # fp32 addition of two values has one correctly rounded result
    assert torch.equal(out.view(torch.int32), y.view(torch.int32))


def test_halo_on_shards_just_below_2_to_31_elements():
    """Two padded shards of 32770 x 65530 cells (2,147,418,100 each, 8.6 GB: cell offsets up to 2^31, byte
    offsets above 2^33), one interface between them.  The rows next to the interface are compared with
    the oracle run on those rows alone (a problem with one bulk row per worker has the same exchange);
    everything else by what H and H* leave behind: exterior ghosts zero, the rest of the bulk untouched."""
    _need_free_gb(40)
    R, C = 32770, 65530
    gs, ps = (2 * (R - 2), C - 2), (2, 1)
    gpart = distdl.Partition(gs, ps, (1, 1), (1, 1))
    mini = oracle.Partition((2, C - 2), ps, 1, 1)
    rows = [slice(R - 3, R), slice(0, 3)]           # worker 0: its last three rows; worker 1: its first three

    def check(call, seq, seed, adjoint):
        x = [_long_vector(R * C, seed + w).view(R, C) for w in range(2)]
        small = [host(x[w][rows[w]]) for w in range(2)]
        call(gpart, x)
        torch.cuda.synchronize()
        ref = seq(mini, small)
        # the mini problem's own exterior row (row 0 of worker 0, row 2 of worker 1) is a bulk row here
        assert host(x[0][R - 2:R]).tobytes() == ref[0][1:3].tobytes()
        assert host(x[1][0:2]).tobytes() == ref[1][0:2].tobytes()
        for w in range(2):
            keep = _long_vector(R * C, seed + w).view(R, C)
            inner = slice(1, R - 2) if w == 0 else slice(2, R - 1)      # bulk rows away from the interface
            assert torch.equal(x[w][inner, 1:C - 1].view(torch.int32), keep[inner, 1:C - 1].view(torch.int32))
            del keep
            assert not x[w][:, 0].any() and not x[w][:, C - 1].any()
            assert not x[w][0 if w == 0 else R - 1].any()
            if adjoint:
                assert not x[w][R - 1 if w == 0 else 0].any()

    check(distdl.halo_fwd, oracle.halo_fwd_sequence, 2201, False)
    check(distdl.halo_adj, oracle.halo_adj_sequence, 2211, True)


def test_halo_row_plan_on_shards_just_below_2_to_31_elements():
    """The row plan at its largest: two padded shards of 32760 x 65544 cells (2,147,221,440 each; unit offsets up to
    2^29, byte offsets above 2^33) side by side along the rows, ghost width 4 along the rows and 2 across them.  Ghost
    rows and the row ends next to the tensor's boundary must come out zero, the row ends at the interface must hold
    the neighbour's bulk columns (H) or be added into them (H*), the rest of the bulk must be untouched; windows of
    rows at the top, around cell 2^31 / 2 and at the bottom are also compared with the oracle run on those rows."""
    _need_free_gb(45)
    R, C, hr, hc = 32760, 65544, 2, 4
    gs, ps = (R - 2 * hr, 2 * (C - 2 * hc)), (1, 2)
    gpart = distdl.Partition(gs, ps, (hr, hc), (hr, hc))
    assert gpart.uses_row_plan() and gpart.uses_row_plan(adjoint=True)
    windows = [2, 16380, R - 5]                      # first bulk row of each three-row window
    mini = oracle.Partition((3, gs[1]), ps, (hr, hc), (hr, hc))

    def window(t, r0):                                # three bulk rows with two rows of (zero) ghost above and below
        out = np.zeros((7, C), dtype=np.float32)
        out[2:5] = host(t[r0:r0 + 3])
        return out

    for adjoint, seed in ((False, 2301), (True, 2311)):
        x = [_long_vector(R * C, seed + w).view(R, C) for w in range(2)]
        before = [[window(x[w], r0) for w in range(2)] for r0 in windows]
        if adjoint:
            distdl.halo_adj(gpart, x)
        else:
            distdl.halo_fwd(gpart, x)
        torch.cuda.synchronize()
        for r0, small in zip(windows, before):
            ref = (oracle.halo_adj_sequence if adjoint else oracle.halo_fwd_sequence)(mini, small)
            for w in range(2):
                assert host(x[w][r0:r0 + 3]).tobytes() == ref[w][2:5].tobytes(), "window at row %d, worker %d" % (r0, w)
        for w in range(2):
            keep = _long_vector(R * C, seed + w).view(R, C)
            # ghost rows, and the row ends on the tensor's boundary
            assert not x[w][:hr].any() and not x[w][R - hr:].any()
            assert not (x[w][:, :hc] if w == 0 else x[w][:, C - hc:]).any()
            inner = (slice(hr, R - hr), slice(2 * hc, C - 2 * hc))       # bulk cells away from both row ends
            assert torch.equal(x[w][inner].view(torch.int32), keep[inner].view(torch.int32))
            other = _long_vector(R * C, seed + 1 - w).view(R, C)
            rows = slice(hr, R - hr)
            mine = (slice(C - hc, C) if w == 0 else slice(0, hc))        # this worker's ghost columns at the interface
            theirs = (slice(hc, 2 * hc) if w == 0 else slice(C - 2 * hc, C - hc))   # the neighbour's bulk columns they mirror
            if adjoint:
                assert not x[w][rows, mine].any()
                recv = (slice(C - 2 * hc, C - hc) if w == 0 else slice(hc, 2 * hc))      # own bulk columns that receive
                from_ghost = (slice(0, hc) if w == 0 else slice(C - hc, C))              # the neighbour's ghost columns
                assert torch.equal(x[w][rows, recv], keep[rows, recv] + other[rows, from_ghost])
            else:
                assert torch.equal(x[w][rows, mine].view(torch.int32), other[rows, theirs].view(torch.int32))
                edge = (slice(C - 2 * hc, C - hc) if w == 0 else slice(hc, 2 * hc))
                assert torch.equal(x[w][rows, edge].view(torch.int32), keep[rows, edge].view(torch.int32))
            del keep, other
        del x


def test_halo_3d_full_size():
    gs, ps, h = (512,) * 3, (4,) * 3, 4
    opart = oracle.Partition(gs, ps, h, h)
    gpart = distdl.Partition(gs, ps, (h,) * 3, (h,) * 3)
    x = [inputs.uniform_pm1(opart.padded_shape(w), 3000 + w) for w in range(64)]
    xd = [dev(a) for a in x]
    distdl.halo_fwd(gpart, xd)
    torch.cuda.synchronize()
    ref = oracle.halo_fwd_sequence(opart, x)
    hx = [host(t) for t in xd]
    for w in range(64):
        assert hx[w].tobytes() == ref[w].tobytes(), "H differs on worker %d" % w
    del ref
    y = [inputs.uniform_pm1(opart.padded_shape(w), 4000 + w) for w in range(64)]
    yd = [dev(a) for a in y]
    distdl.halo_adj(gpart, yd)
    torch.cuda.synchronize()
    refa = oracle.halo_adj_sequence(opart, y)
    hy = [host(t) for t in yd]
    for w in range(64):
        assert hy[w].tobytes() == refa[w].tobytes(), "H* differs on worker %d" % w
    assert oracle.adjoint_test_ratio(hx, y, x, hy) < 1e-5


def test_conv_full_size_on_sampled_planes():
    gs, ps = (16, 16, 1024, 1024), (1, 1, 4, 4)
    gpart = distdl.Partition(gs, ps, (0, 0, 2, 2), (0, 0, 2, 2))
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    # full-size inputs are drawn on the device (seeded); the sampled planes are read back for the oracle
    xs = [torch.randn(16, 16, 260, 260, device=DEV, generator=g) for _ in range(16)]
    dys = [torch.randn(16, 16, 256, 256, device=DEV, generator=g) for _ in range(16)]
    w = inputs.normal((16, 5, 5), 5001, 0.1)
    ys = [torch.empty(16, 16, 256, 256, device=DEV) for _ in range(16)]
    dxs = [torch.full((16, 16, 260, 260), 7.0, device=DEV) for _ in range(16)]
    distdl.conv_fwd(gpart, xs, dev(w), None, ys)
    distdl.conv_adj(gpart, dys, dev(w), dxs)
    distdl.device_status()
    planes = [(0, 0), (3, 7), (9, 15), (15, 2), (15, 15)]
    # tolerance: 25 FMA roundings + one add of the kernel's two partial sums + the oracle's rounding to fp32
    sub = (1, 1, 1024, 1024)
    op = oracle.Partition(sub, ps, (0, 0, 2, 2), (0, 0, 2, 2))
    ob = oracle.Partition(sub, ps)
    for n, c in planes:
        x1 = [host(t[n:n + 1, c:c + 1]) for t in xs]
        dy1 = [host(t[n:n + 1, c:c + 1]) for t in dys]
        yref = oracle.conv_fwd(op, x1, w[c:c + 1])
        dxref = oracle.conv_adj(op, dy1, w[c:c + 1])
        ybound = oracle.conv_fwd(op, [np.abs(a) for a in x1], np.abs(w[c:c + 1]))
        dxbound = oracle.conv_adj(op, [np.abs(a) for a in dy1], np.abs(w[c:c + 1]))
        for k in range(16):
            got = host(ys[k][n:n + 1, c:c + 1]).astype(np.float64)
            assert np.all(np.abs(got - yref[k]) <= 27 * 2.0 ** -24 * ybound[k] + 1e-30)
            gotx = host(dxs[k][n:n + 1, c:c + 1])
            assert np.all(np.abs(gotx.astype(np.float64) - dxref[k]) <= 27 * 2.0 ** -24 * dxbound[k] + 1e-30)
            mask = np.ones(gotx.shape, dtype=bool)
            mask[op.bulk_slices(k)] = False
            assert not gotx[mask].any()
    # ghosts of every plane of dx are zero (property that holds at any size)
    for k in range(16):
        t = dxs[k]
        assert float(t[:, :, :2, :].abs().max()) == 0.0 and float(t[:, :, -2:, :].abs().max()) == 0.0
        assert float(t[:, :, :, :2].abs().max()) == 0.0 and float(t[:, :, :, -2:].abs().max()) == 0.0


def test_conv_on_shards_just_below_2_to_31_elements():
    """Four padded shards of 1982 x 16 planes of 260 x 260 cells (2,143,731,200 cells, 8.6 GB each): the
    last planes start at cell offsets just below 2^31.  Sampled planes against the oracle, as above."""
    _need_free_gb(80)
    N, C = 1982, 16
    gs, ps = (N, C, 512, 512), (1, 1, 2, 2)
    gpart = distdl.Partition(gs, ps, (0, 0, 2, 2), (0, 0, 2, 2))
    g = torch.Generator(device=DEV)
    g.manual_seed(6)
    w = inputs.normal((C, 5, 5), 5002, 0.1)
    planes = [(0, 0), (1000, 7), (N - 1, 0), (N - 1, C - 1)]
    sub = (1, 1, 512, 512)
    op = oracle.Partition(sub, ps, (0, 0, 2, 2), (0, 0, 2, 2))

    xs = [torch.randn(N, C, 260, 260, device=DEV, generator=g) for _ in range(4)]
    ys = [torch.empty(N, C, 256, 256, device=DEV) for _ in range(4)]
    distdl.conv_fwd(gpart, xs, dev(w), None, ys)
    distdl.device_status()
    for n, c in planes:
        x1 = [host(t[n:n + 1, c:c + 1]) for t in xs]
        yref = oracle.conv_fwd(op, x1, w[c:c + 1])
        ybound = oracle.conv_fwd(op, [np.abs(a) for a in x1], np.abs(w[c:c + 1]))
        for k in range(4):
            got = host(ys[k][n:n + 1, c:c + 1]).astype(np.float64)
            assert np.all(np.abs(got - yref[k]) <= 27 * 2.0 ** -24 * ybound[k] + 1e-30)
    del xs, ys
    torch.cuda.empty_cache()

    dys = [torch.randn(N, C, 256, 256, device=DEV, generator=g) for _ in range(4)]
    dxs = [torch.full((N, C, 260, 260), 7.0, device=DEV) for _ in range(4)]
    distdl.conv_adj(gpart, dys, dev(w), dxs)
    distdl.device_status()
    for n, c in planes:
        dy1 = [host(t[n:n + 1, c:c + 1]) for t in dys]
        dxref = oracle.conv_adj(op, dy1, w[c:c + 1])
        dxbound = oracle.conv_adj(op, [np.abs(a) for a in dy1], np.abs(w[c:c + 1]))
        for k in range(4):
            gotx = host(dxs[k][n:n + 1, c:c + 1])
            assert np.all(np.abs(gotx.astype(np.float64) - dxref[k]) <= 27 * 2.0 ** -24 * dxbound[k] + 1e-30)
    for t in dxs:
        assert float(t[:, :, :2, :].abs().max()) == 0.0 and float(t[:, :, -2:, :].abs().max()) == 0.0
        assert float(t[:, :, :, :2].abs().max()) == 0.0 and float(t[:, :, :, -2:].abs().max()) == 0.0


def test_affine_full_size():
    nb, nf, pf = 256, 8192, 4
    blk = nf // pf
    xb = inputs.f32_to_bf16_bits(inputs.normal((nb, nf), 6000))
    wb = inputs.f32_to_bf16_bits(inputs.normal((nf, nf), 6001, nf ** -0.5))
    dyb = inputs.f32_to_bf16_bits(inputs.normal((nb, nf), 6002))
    bf = lambda a: dev(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    xs, dys = np.split(xb, pf, axis=1), np.split(dyb, pf, axis=1)
    ws = [b for row in np.split(wb, pf, axis=0) for b in np.split(row, pf, axis=1)]
    w_d = [bf(a) for a in ws]
    y = [torch.empty(nb, blk, device=DEV) for _ in range(pf)]
    dx = [torch.empty(nb, blk, device=DEV) for _ in range(pf)]
    distdl.affine_fwd(nb, nf, nf, pf, pf, [bf(a) for a in xs], w_d, None, y)
    distdl.affine_adj(nb, nf, nf, pf, pf, [bf(a) for a in dys], w_d, dx)
    distdl.device_status()
    f64 = oracle.bf16_bits_to_f64
    xf, wf, dyf = [f64(a) for a in xs], [f64(a) for a in ws], [f64(a) for a in dys]
    yref, dxref = oracle.affine_fwd(xf, wf, pf, pf), oracle.affine_adj(dyf, wf, pf, pf)
    for got, ref in ((y, yref), (dx, dxref)):
        g = np.concatenate([host(t).astype(np.float64) for t in got], axis=1)
        r = np.concatenate([a.astype(np.float64) for a in ref], axis=1)
        assert np.max(np.abs(g - r)) / np.max(np.abs(r)) < 2e-2
        assert np.linalg.norm(g - r) / np.linalg.norm(r) < 1e-4
    assert oracle.adjoint_test_ratio([host(t) for t in y], dyf, xf, [host(t) for t in dx]) < 1e-4


def test_affine_on_the_largest_batch():
    """nb = 2^20 rows (the most the layer accepts), 4096 x 4096 weights on 2 x 2 workers: every output block
    holds 2^31 values (8.6 GB).  Rows of the batch are independent, so windows of rows at the start, the middle
    and the end are compared with the oracle run on those rows."""
    _need_free_gb(70)
    nb, nf, pf = 1 << 20, 4096, 2
    blk = nf // pf
    wb = inputs.f32_to_bf16_bits(inputs.normal((nf, nf), 6011, nf ** -0.5))
    bf = lambda a: dev(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    ws = [b for row in np.split(wb, pf, axis=0) for b in np.split(row, pf, axis=1)]
    w_d = [bf(a) for a in ws]
    g = torch.Generator(device=DEV)
    g.manual_seed(13)
    xs = [torch.randn(nb, blk, device=DEV, generator=g).to(torch.bfloat16) for _ in range(pf)]
    dys = [torch.randn(nb, blk, device=DEV, generator=g).to(torch.bfloat16) for _ in range(pf)]
    y = [torch.full((nb, blk), float("nan"), device=DEV) for _ in range(pf)]
    dx = [torch.full((nb, blk), float("nan"), device=DEV) for _ in range(pf)]
    distdl.affine_fwd(nb, nf, nf, pf, pf, xs, w_d, None, y)
    distdl.affine_adj(nb, nf, nf, pf, pf, dys, w_d, dx)
    distdl.device_status()
    f64 = oracle.bf16_bits_to_f64
    bits = lambda t: host(t.view(torch.int16)).view(np.uint16)
    wf = [f64(a) for a in ws]
    for lo, hi in [(0, 128), (nb // 2 - 64, nb // 2 + 64), (nb - 128, nb)]:
        xf = [f64(bits(t[lo:hi])) for t in xs]
        dyf = [f64(bits(t[lo:hi])) for t in dys]
        yref, dxref = oracle.affine_fwd(xf, wf, pf, pf), oracle.affine_adj(dyf, wf, pf, pf)
        for got, ref in ((y, yref), (dx, dxref)):
            gg = np.concatenate([host(t[lo:hi]).astype(np.float64) for t in got], axis=1)
            r = np.concatenate([a.astype(np.float64) for a in ref], axis=1)
            assert np.max(np.abs(gg - r)) / np.max(np.abs(r)) < 2e-2
            assert np.linalg.norm(gg - r) / np.linalg.norm(r) < 1e-4
    # every one of the 2^31 values of a block was written (the blocks were filled with NaN)
    for t in y + dx:
        assert bool(torch.isfinite(t).all())


def _pool_on_sampled_planes(N, C, image, ps, planes, seed):
    # 3 x 3 max pooling, stride 2, padding 1: ghost widths (1, 0) per worker
    gs, k, s, pad = (N, C) + image, (3, 3), (2, 2), ((1, 1), (1, 1))
    sub = (1, 1) + image
    P = ps[2] * ps[3]
    opart, geo = oracle.pool_partition(sub, ps, k, s, pad)
    gpart = distdl.Partition(gs, ps, [list(h) for h in opart.hlo], [list(h) for h in opart.hhi])
    oshape = (N, C, image[0] // 2 // ps[2], image[1] // 2 // ps[3])
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    xs = [torch.randn(*gpart.padded_shape(w), device=DEV, generator=g) for w in range(P)]
    ys = [torch.empty(oshape, device=DEV) for _ in range(P)]
    args = [torch.full(oshape, -1, dtype=torch.int32, device=DEV) for _ in range(P)]
    dys = [torch.randn(oshape, device=DEV, generator=g) for _ in range(P)]
    dxs = [torch.full(tuple(gpart.padded_shape(w)), 7.0, device=DEV) for w in range(P)]
    x_before = {(n, c): [host(t[n:n + 1, c:c + 1]) for t in xs] for n, c in planes}
    distdl.pool_fwd(gpart, xs, k, s, pad, distdl.POOL_MAX, ys, args)
    distdl.pool_adj(gpart, dys, args, k, s, pad, distdl.POOL_MAX, dxs)
    torch.cuda.synchronize()
    for (n, c), x1 in x_before.items():
        yref, aref = oracle.pool_fwd(opart, geo, x1, k, s, pad, "max")
        dy1 = [host(t[n:n + 1, c:c + 1]) for t in dys]
        dxref = oracle.pool_adj(opart, geo, dy1, k, s, pad, "max", aref)
        for w in range(P):
            assert host(ys[w][n:n + 1, c:c + 1]).tobytes() == yref[w].tobytes()
            assert np.array_equal(host(args[w][n:n + 1, c:c + 1]), aref[w])
            got = host(dxs[w][n:n + 1, c:c + 1])
            # up to four routed values per cell summed in fp32, then the fixed-order sums of H*
            assert np.max(np.abs(got - dxref[w])) <= 8 * 2.0 ** -24 * 4 * float(np.max(np.abs(dy1[w])))
    # properties at full size: every recorded position is a window position, ghosts of dx are zero,
    # and the adjoint routes all of dy (sum preserved up to fp32 rounding)
    for w in range(P):
        assert int(args[w].min()) >= 0 and int(args[w].max()) <= 8
        lo, hi = opart.widths(w)
        t = dxs[w]
        if lo[2]:
            assert float(t[:, :, :lo[2], :].abs().max()) == 0.0
        if lo[3]:
            assert float(t[:, :, :, :lo[3]].abs().max()) == 0.0
    total_dx = sum(float(t.sum(dtype=torch.float64)) for t in dxs)
    total_dy = sum(float(t.sum(dtype=torch.float64)) for t in dys)
    assert abs(total_dx - total_dy) <= 1e-6 * sum(float(t.abs().sum(dtype=torch.float64)) for t in dys)


def test_pool_full_size_on_sampled_planes():
    # the configuration bench.py times
    _pool_on_sampled_planes(16, 16, (1024, 1024), (1, 1, 4, 4), [(0, 0), (5, 11), (15, 15)], 7)


def test_pool_on_shards_just_below_2_to_31_elements():
    # four padded shards of 2031 x 16 planes of 257 x 257 cells: 2,146,328,304 cells (8.6 GB) each
    _need_free_gb(120)
    _pool_on_sampled_planes(2031, 16, (512, 512), (1, 1, 2, 2), [(0, 0), (1017, 5), (2030, 0), (2030, 15)], 8)


def _stencil3d_on_sampled_boxes(gs, ps, R, boxes, seed, dot_test):
    P = ps[0] * ps[1] * ps[2]
    bk = tuple(g // q for g, q in zip(gs, ps))                     # bulk extents (the splits are even)
    pad = tuple(v + 2 * R for v in bk)
    gpart = distdl.Partition(gs, ps, (R,) * 3, (R,) * 3)
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    xs = [torch.randn(*pad, device=DEV, generator=g) for _ in range(P)]
    dys = [torch.randn(*bk, device=DEV, generator=g) for _ in range(P)]
    w = inputs.normal((3, 2 * R + 1), 7001, 0.5)
    ys = [torch.empty(*bk, device=DEV) for _ in range(P)]
    dxs = [torch.full(pad, 7.0, device=DEV) for _ in range(P)]
    distdl.stencil3d_fwd(gpart, xs, w, ys)
    distdl.stencil3d_adj(gpart, dys, w, dxs)
    torch.cuda.synchronize()

    def gather(shards, off, lo, hi):
        """Global box [lo, hi) put together from the bulks of the device shards (bulk offset `off` inside a shard)."""
        out = np.zeros(tuple(b - a for a, b in zip(lo, hi)), dtype=np.float32)
        for s in range(P):
            c = (s // (ps[1] * ps[2]), (s // ps[2]) % ps[1], s % ps[2])
            a = [max(lo[k], bk[k] * c[k]) for k in range(3)]
            b = [min(hi[k], bk[k] * c[k] + bk[k]) for k in range(3)]
            if any(a[k] >= b[k] for k in range(3)):
                continue
            src = tuple(slice(a[k] - bk[k] * c[k] + off, b[k] - bk[k] * c[k] + off) for k in range(3))
            dst = tuple(slice(a[k] - lo[k], b[k] - lo[k]) for k in range(3))
            out[dst] = host(shards[s][src])
        return out

    eps = (6 * R + 5) * 2.0 ** -24
    for lo in boxes:
        hi = tuple(v + 20 for v in lo)
        elo = tuple(max(v - R, 0) for v in lo)
        ehi = tuple(min(v + R, n) for v, n in zip(hi, gs))
        one = oracle.Partition(tuple(b - a for a, b in zip(elo, ehi)), (1, 1, 1), R, R)
        inner = tuple(slice(l - e, l - e + 20) for l, e in zip(lo, elo))
        for shards_in, off_in, got_shards, off_out, fn in ((xs, R, ys, 0, oracle.stencil3d_fwd), (dys, 0, dxs, R, oracle.stencil3d_adj)):
            sub = gather(shards_in, off_in, elo, ehi)
            if fn is oracle.stencil3d_fwd:
                ref = fn(one, oracle.scatter_global(one, sub), w)[0][inner]
                mag = fn(one, oracle.scatter_global(one, np.abs(sub)), np.abs(w))[0][inner]
            else:
                ref = fn(one, [sub], w)[0][one.bulk_slices(0)][inner]
                mag = fn(one, [np.abs(sub)], np.abs(w))[0][one.bulk_slices(0)][inner]
            # the extended box is cut R cells beyond the sampled one (or at the tensor's own boundary, where the
            # oracle's zero padding is the right one), so the sampled cells see exactly their global neighbours
            got = gather(got_shards, off_out, lo, hi)
            assert np.all(np.abs(got.astype(np.float64) - ref) <= eps * mag + 1e-30)
    # properties at full size: x untouched is checked in the small tests; ghosts of every dx shard are zero
    for t in dxs:
        assert float(t[:R].abs().max()) == 0.0 and float(t[-R:].abs().max()) == 0.0
        assert float(t[:, :R].abs().max()) == 0.0 and float(t[:, -R:].abs().max()) == 0.0
        assert float(t[:, :, :R].abs().max()) == 0.0 and float(t[:, :, -R:].abs().max()) == 0.0
    if dot_test:
        # dot test over the whole volume, fp64 on the device (x's ghost storage does not take part)
        lhs = sum(float((a.double() * b.double()).sum()) for a, b in zip(ys, dys))
        rhs = sum(float((a[R:-R, R:-R, R:-R].double() * b[R:-R, R:-R, R:-R].double()).sum()) for a, b in zip(xs, dxs))
        ny = sum(float((a.double() ** 2).sum()) for a in ys) ** 0.5
        ndy = sum(float((a.double() ** 2).sum()) for a in dys) ** 0.5
        assert abs(lhs - rhs) <= 1e-5 * ny * ndy


def test_stencil3d_full_size_on_sampled_boxes():
    # the configuration bench.py times: 512^3 on 4 x 4 x 4 workers, radius 4; boxes at a corner of the
    # tensor, where eight shards meet, across a face, and at the far corner
    _stencil3d_on_sampled_boxes((512,) * 3, (4,) * 3, 4, [(0, 0, 0), (120, 120, 120), (250, 380, 120), (492, 492, 492)],
                                11, True)


def test_stencil3d_on_shards_just_below_2_to_31_elements():
    # two padded shards of 1288^3 = 2,136,719,872 cells (8.5 GB each); boxes at the first cells, across the
    # interface between the two workers (the last planes of worker 0, the first of worker 1) and at the far corner
    _need_free_gb(80)
    _stencil3d_on_sampled_boxes((2560, 1280, 1280), (2, 1, 1), 4,
                                [(0, 0, 0), (1270, 600, 1260), (1270, 1260, 1260), (2540, 1260, 1260)], 12, False)


def test_parameter_gradients_full_size():
    # convolution: dw, db of two channels of the 16 x 16 x 1024 x 1024 case, each over all 16 batch entries
    gs, ps = (16, 16, 1024, 1024), (1, 1, 4, 4)
    gpart = distdl.Partition(gs, ps, (0, 0, 2, 2), (0, 0, 2, 2))
    g = torch.Generator(device=DEV)
    g.manual_seed(13)
    xs = [torch.randn(16, 16, 260, 260, device=DEV, generator=g) for _ in range(16)]
    dys = [torch.randn(16, 16, 256, 256, device=DEV, generator=g) for _ in range(16)]
    dw, db = torch.empty(16, 5, 5, device=DEV), torch.empty(16, device=DEV)
    ws = torch.empty(distdl.conv_adj_params_workspace(gpart, 5, 5), dtype=torch.uint8, device=DEV)
    distdl.conv_adj_params(gpart, xs, dys, (5, 5), dw, db, ws)
    distdl.device_status()
    sub = (16, 1, 1024, 1024)
    op = oracle.Partition(sub, ps, (0, 0, 2, 2), (0, 0, 2, 2))
    for c in (0, 11):
        x1 = [host(t[:, c:c + 1]) for t in xs]
        dy1 = [host(t[:, c:c + 1]) for t in dys]
        dw_ref, db_ref = oracle.conv_adj_params(op, x1, dy1, 5, 5)
        # 16.8 M terms per tap; a running sum has 16 terms per tile of the channel (4096 tiles), then the folds
        mag_w, mag_b = oracle.conv_adj_params(op, [np.abs(a) for a in oracle.halo_fwd_sequence(op, x1)],
                                              [np.abs(a) for a in dy1], 5, 5)
        eps = (16 * 4096 + 64) * 2.0 ** -24
        assert np.all(np.abs(host(dw[c:c + 1]).astype(np.float64) - dw_ref) <= eps * mag_w)
        assert np.all(np.abs(host(db[c:c + 1]).astype(np.float64) - db_ref) <= eps * mag_b)
        assert np.linalg.norm(host(dw[c:c + 1]).astype(np.float64) - dw_ref) <= 1e-5 * np.linalg.norm(mag_w)
    del xs, dys

    # affine: dW blocks of three workers and every db of the 256 x 8192 x 8192 case
    nb, nf, pf = 256, 8192, 4
    blk = nf // pf
    xb = inputs.f32_to_bf16_bits(inputs.normal((nb, nf), 6100))
    dyb = inputs.f32_to_bf16_bits(inputs.normal((nb, nf), 6102))
    bf = lambda a: dev(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    xp, dyp = np.split(xb, pf, axis=1), np.split(dyb, pf, axis=1)
    dW = [torch.empty(blk, blk, device=DEV) for _ in range(pf * pf)]
    dB = [torch.empty(blk, device=DEV) for _ in range(pf)]
    distdl.affine_adj_params(nb, nf, nf, pf, pf, [bf(a) for a in dyp], [bf(a) for a in xp], dW, dB)
    distdl.device_status()
    f64 = oracle.bf16_bits_to_f64
    for i, j in ((0, 0), (2, 3), (3, 1)):
        ref, dbref = oracle.affine_adj_params([f64(dyp[i])], [f64(xp[j])], 1, 1)
        got = host(dW[i * pf + j]).astype(np.float64)
        assert np.max(np.abs(got - ref[0])) / np.max(np.abs(ref[0])) < 1e-4
        assert np.linalg.norm(got - ref[0]) / np.linalg.norm(ref[0]) < 1e-5
        assert np.max(np.abs(host(dB[i]).astype(np.float64) - dbref[0])) <= 1e-5 * np.max(np.abs(dbref[0]))


def test_repartition_full_size():
    # the all-to-all bench.py times: fp32 8192 x 8192, 8 row blocks -> 8 column blocks and back
    n = 8192
    rep = distdl.Repartition((n, n), (8, 1), (1, 8))
    rows = [inputs.uniform_pm1((n // 8, n), 8000 + i) for i in range(8)]
    src = [dev(a) for a in rows]
    dst = [torch.empty(n, n // 8, device=DEV) for _ in range(8)]
    distdl.repartition_fwd(rep, src, dst)
    back = [torch.empty(n // 8, n, device=DEV) for _ in range(8)]
    distdl.repartition_adj(rep, dst, back)
    torch.cuda.synchronize()
    ref = oracle.repartition_fwd(oracle.Partition((n, n), (8, 1)), oracle.Partition((n, n), (1, 8)), rows)
    for a, b in zip(dst, ref):
        assert host(a).tobytes() == b.tobytes()
    for a, b in zip(back, rows):
        assert host(a).tobytes() == b.tobytes()


def test_repartition_on_shards_just_below_2_to_31_elements():
    """Two row blocks <-> two column blocks of a 46340 x 92672 matrix: every shard holds 2,147,210,240
    cells (8.6 GB).  The sixteen rows and columns around the point where all four shards meet are compared
    with the oracle on that window alone (its even split falls on the same lines); every cell with the
    plain definition, a re-slicing of the matrix, on the device."""
    _need_free_gb(70)
    nr, nc = 46340, 92672
    rep = distdl.Repartition((nr, nc), (2, 1), (1, 2))
    src = [_long_vector(nr // 2 * nc, 8100 + i).view(nr // 2, nc) for i in range(2)]
    dst = [torch.empty(nr, nc // 2, device=DEV) for _ in range(2)]
    distdl.repartition_fwd(rep, src, dst)
    torch.cuda.synchronize()
    h = 8
    win = [host(src[0][-h:, nc // 2 - h:nc // 2 + h]), host(src[1][:h, nc // 2 - h:nc // 2 + h])]
    ref = oracle.repartition_fwd(oracle.Partition((2 * h, 2 * h), (2, 1)), oracle.Partition((2 * h, 2 * h), (1, 2)), win)
    assert host(dst[0][nr // 2 - h:nr // 2 + h, -h:]).tobytes() == ref[0].tobytes()
    assert host(dst[1][nr // 2 - h:nr // 2 + h, :h]).tobytes() == ref[1].tobytes()
    for j in range(2):
        for i in range(2):
            a = dst[j][i * (nr // 2):(i + 1) * (nr // 2)]
            b = src[i][:, j * (nc // 2):(j + 1) * (nc // 2)]
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    back = [torch.empty(nr // 2, nc, device=DEV) for _ in range(2)]
    distdl.repartition_adj(rep, dst, back)
    torch.cuda.synchronize()
    for a, b in zip(back, src):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_generalized_conv_full_size_on_samples():
    # the configuration bench.py times: 16 -> 16 channels, 5 x 5, fp32 4 x 16 x 1024 x 1024, channel partitions 2 x 2,
    # feature space 2 x 2
    N, C, S, k, h = 4, 16, 1024, 5, 2
    gpart = distdl.Partition((N, C, S, S), (1, 2, 2, 2), (0, 0, h, h), (0, 0, h, h))
    g = torch.Generator(device=DEV)
    g.manual_seed(17)
    xs = [torch.randn(N, 8, 516, 516, device=DEV, generator=g) for _ in range(8)]
    dys = [torch.randn(N, 8, 512, 512, device=DEV, generator=g) for _ in range(8)]
    wb = [inputs.normal((8, 8, k, k), 9000 + q, 0.05) for q in range(4)]
    wd = [dev(a) for a in wb]
    ys = [torch.empty(N, 8, 512, 512, device=DEV) for _ in range(8)]
    dxs = [torch.full((N, 8, 516, 516), 7.0, device=DEV) for _ in range(8)]
    dws = [torch.empty(8, 8, k, k, device=DEV) for _ in range(4)]
    dbs = [torch.empty(8, device=DEV) for _ in range(2)]
    ws = torch.empty(distdl.convg_adj_params_workspace(gpart, C, 2, k, k), dtype=torch.uint8, device=DEV)
    distdl.convg_fwd(gpart, C, 2, xs, wd, None, ys)
    distdl.convg_adj(gpart, C, 2, dys, wd, dxs)
    distdl.convg_adj_params(gpart, C, 2, xs, dys, (k, k), dws, dbs, ws)
    distdl.device_status()

    def gather(shards, off, n, lo, hi):
        """[16, rows, cols] of batch entry n over the global box [lo, hi) from the bulks of the eight shards."""
        out = np.zeros((C, hi[0] - lo[0], hi[1] - lo[1]), dtype=np.float32)
        for b in range(2):
            for r in range(2):
                for c in range(2):
                    a = [max(lo[0], 512 * r), max(lo[1], 512 * c)]
                    e = [min(hi[0], 512 * r + 512), min(hi[1], 512 * c + 512)]
                    if a[0] >= e[0] or a[1] >= e[1]:
                        continue
                    t = shards[(b * 2 + r) * 2 + c]
                    out[8 * b:8 * b + 8, a[0] - lo[0]:e[0] - lo[0], a[1] - lo[1]:e[1] - lo[1]] = host(
                        t[n, :, a[0] - 512 * r + off:e[0] - 512 * r + off, a[1] - 512 * c + off:e[1] - 512 * c + off])
        return out

    # boxes where the four feature-space shards meet, at a corner of the tensor, and inside a shard
    for n, lo in ((2, (500, 490)), (0, (0, 0)), (3, (984, 960)), (1, (130, 700))):
        hi = (lo[0] + 40, lo[1] + 64)
        elo = tuple(max(v - h, 0) for v in lo)
        ehi = tuple(min(v + h, S) for v in hi)
        shape = (1, C, ehi[0] - elo[0], ehi[1] - elo[1])
        sub = oracle.Partition(shape, (1, 2, 1, 1), (0, 0, h, h), (0, 0, h, h))
        suby = oracle.Partition(shape, (1, 2, 1, 1))
        inner = (slice(None), slice(lo[0] - elo[0], lo[0] - elo[0] + 40), slice(lo[1] - elo[1], lo[1] - elo[1] + 64))
        xbox = gather(xs, h, n, elo, ehi)[None]
        yref = oracle.assemble_global(suby, oracle.convg_fwd(sub, C, 2, oracle.scatter_global(sub, xbox), wb))[0][inner]
        ymag = oracle.assemble_global(suby, oracle.convg_fwd(sub, C, 2, oracle.scatter_global(sub, np.abs(xbox)),
                                                              [np.abs(a) for a in wb]))[0][inner]
        got = gather(ys, 0, n, lo, hi)
        assert np.all(np.abs(got.astype(np.float64) - yref) <= (C * k * k + 2) * 2.0 ** -24 * ymag + 1e-30)
        dybox = gather(dys, 0, n, elo, ehi)[None]
        dxref = oracle.assemble_global(sub, oracle.convg_adj(sub, C, 2, oracle.scatter_global(suby, dybox), wb))[0][inner]
        dxmag = oracle.assemble_global(sub, oracle.convg_adj(sub, C, 2, oracle.scatter_global(suby, np.abs(dybox)),
                                                             [np.abs(a) for a in wb]))[0][inner]
        gotx = gather(dxs, h, n, lo, hi)
        # the adjoint oracle rounds to fp32 before its halo sums: two more roundings at the box's own cut edges
        assert np.all(np.abs(gotx.astype(np.float64) - dxref) <= (C * k * k + 6) * 2.0 ** -24 * dxmag + 1e-30)
    for t in dxs:                                         # ghosts of dx are zero
        assert float(t[:, :, :h].abs().max()) == 0.0 and float(t[:, :, -h:].abs().max()) == 0.0
        assert float(t[:, :, :, :h].abs().max()) == 0.0 and float(t[:, :, :, -h:].abs().max()) == 0.0
    # parameter gradients of sampled channel pairs (o, c): the oracle on those two channels alone
    one = oracle.Partition((N, 1, S, S), (1, 1, 2, 2), (0, 0, h, h), (0, 0, h, h))
    for o, c in ((0, 0), (5, 12), (11, 3), (15, 15)):
        x1 = [host(xs[((c // 8) * 2 + r) * 2 + q][:, c % 8:c % 8 + 1]) for r in range(2) for q in range(2)]
        dy1 = [host(dys[((o // 8) * 2 + r) * 2 + q][:, o % 8:o % 8 + 1]) for r in range(2) for q in range(2)]
        dw_ref, db_ref = oracle.convg_adj_params(one, 1, 1, x1, dy1, k, k)
        xh = oracle.halo_fwd_sequence(one, x1)
        mag, _ = oracle.convg_adj_params(one, 1, 1, [np.abs(a) for a in xh], [np.abs(a) for a in dy1], k, k)
        got = host(dws[(o // 8) * 2 + c // 8][o % 8, c % 8]).astype(np.float64)
        tiles = N * 4 * 16 * 4
        assert np.all(np.abs(got - dw_ref[0][0, 0]) <= (16 * tiles + 64) * 2.0 ** -24 * mag[0][0, 0])
        assert np.linalg.norm(got - dw_ref[0][0, 0]) <= 1e-5 * np.linalg.norm(mag[0][0, 0])
        if c == 0:
            sum_abs = float(sum(np.abs(a.astype(np.float64)).sum() for a in dy1))
            assert abs(float(host(dbs[o // 8])[o % 8]) - float(db_ref[0][0])) <= (16 * tiles + 64) * 2.0 ** -24 * sum_abs
