"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration that
bench.py times.  B, R, H, H* and the affine layer are compared in full; the convolution on sampled
(n, c) planes, which the oracle computes one by one."""

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


def test_pool_full_size_on_sampled_planes():
    # the configuration bench.py times: 3 x 3 max pooling, stride 2, padding 1, ghost widths (1, 0) per worker
    gs, ps, k, s, pad = (16, 16, 1024, 1024), (1, 1, 4, 4), (3, 3), (2, 2), ((1, 1), (1, 1))
    sub = (1, 1, 1024, 1024)
    opart, geo = oracle.pool_partition(sub, ps, k, s, pad)
    gpart = distdl.Partition(gs, ps, [list(h) for h in opart.hlo], [list(h) for h in opart.hhi])
    g = torch.Generator(device=DEV)
    g.manual_seed(7)
    xs = [torch.randn(*gpart.padded_shape(w), device=DEV, generator=g) for w in range(16)]
    ys = [torch.empty(16, 16, 128, 128, device=DEV) for _ in range(16)]
    args = [torch.full((16, 16, 128, 128), -1, dtype=torch.int32, device=DEV) for _ in range(16)]
    dys = [torch.randn(16, 16, 128, 128, device=DEV, generator=g) for _ in range(16)]
    dxs = [torch.full(tuple(gpart.padded_shape(w)), 7.0, device=DEV) for w in range(16)]
    x_before = {(n, c): [host(t[n:n + 1, c:c + 1]) for t in xs] for n, c in [(0, 0), (5, 11), (15, 15)]}
    distdl.pool_fwd(gpart, xs, k, s, pad, distdl.POOL_MAX, ys, args)
    distdl.pool_adj(gpart, dys, args, k, s, pad, distdl.POOL_MAX, dxs)
    torch.cuda.synchronize()
    for (n, c), x1 in x_before.items():
        yref, aref = oracle.pool_fwd(opart, geo, x1, k, s, pad, "max")
        dy1 = [host(t[n:n + 1, c:c + 1]) for t in dys]
        dxref = oracle.pool_adj(opart, geo, dy1, k, s, pad, "max", aref)
        for w in range(16):
            assert host(ys[w][n:n + 1, c:c + 1]).tobytes() == yref[w].tobytes()
            assert np.array_equal(host(args[w][n:n + 1, c:c + 1]), aref[w])
            got = host(dxs[w][n:n + 1, c:c + 1])
            # up to four routed values per cell summed in fp32, then the fixed-order sums of H*
            assert np.max(np.abs(got - dxref[w])) <= 8 * 2.0 ** -24 * 4 * float(np.max(np.abs(dy1[w])))
    # properties at full size: every recorded position is a window position, ghosts of dx are zero,
    # and the adjoint routes all of dy (sum preserved up to fp32 rounding)
    for w in range(16):
        assert int(args[w].min()) >= 0 and int(args[w].max()) <= 8
        lo, hi = opart.widths(w)
        t = dxs[w]
        if lo[2]:
            assert float(t[:, :, :lo[2], :].abs().max()) == 0.0
        if lo[3]:
            assert float(t[:, :, :, :lo[3]].abs().max()) == 0.0
    total_dx = sum(float(t.double().sum()) for t in dxs)
    total_dy = sum(float(t.double().sum()) for t in dys)
    assert abs(total_dx - total_dy) <= 1e-6 * sum(float(t.double().abs().sum()) for t in dys)
