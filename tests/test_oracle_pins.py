"""CPU pins for the oracle: each function is checked against something other than itself.

Pins used: values printed in the figures of Appendix B (tests/golden), operator matrices
built cell by cell with a brute-force owner search, closed forms (R after B = k * identity),
library routines on the unpartitioned tensor (numpy.pad, scipy correlate2d, a plain matmul),
and a hand-evaluated worked case for the order of the adjoint halo sums.
"""

import itertools
import os

import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle
from oracle import Partition
from paper_2006_03108_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# Appendix B figures
# --------------------------------------------------------------------------

def _load_appendix_b():
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "appendix_b_halo_1d.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "case":
            cur = dict(name=tok[1], workers=[])
            cur.update({k: int(v) for k, v in (t.split("=") for t in tok[2:])})
            cases.append(cur)
        else:
            kv = dict(t.split("=") for t in tok[2:])
            rng = lambda s: tuple(int(v) for v in s.split(":"))
            pair = lambda s: tuple(int(v) for v in s.split(","))
            cur["workers"].append(dict(inp=rng(kv["in"]), out=rng(kv["out"]), halo=pair(kv["halo"]),
                                       unused=pair(kv["unused"]), view=kv["view"].split(",")))
    return cases


APPENDIX_B = _load_appendix_b()


@pytest.mark.parametrize("case", APPENDIX_B, ids=[c["name"] for c in APPENDIX_B])
def test_halo_geometry_matches_appendix_b_figures(case):
    got = oracle.halo_widths_1d(case["n"], case["p"], case["kernel"], case["stride"],
                                case["dilation"], case["pad_lo"], case["pad_hi"])
    assert len(got) == len(case["workers"]) == case["p"]
    for g, w in zip(got, case["workers"]):
        assert (g["in_start"], g["in_start"] + g["in_size"]) == w["inp"]
        assert (g["out_start"], g["out_start"] + g["out_size"]) == w["out"]
        assert (g["halo_lo"], g["halo_hi"]) == w["halo"]
        assert (g["unused_lo"], g["unused_hi"]) == w["unused"]


@pytest.mark.parametrize("case", APPENDIX_B, ids=[c["name"] for c in APPENDIX_B])
@pytest.mark.parametrize("form", ["definition", "sequence"])
def test_halo_fwd_reproduces_appendix_b_views(case, form):
    """With x[g] = g + 1 the exchanged padded rows must show the indices the figures print."""
    ws = case["workers"]
    part = Partition((case["n"],), (case["p"],), [[w["halo"][0] for w in ws]], [[w["halo"][1] for w in ws]])
    x = np.arange(1, case["n"] + 1, dtype=np.float32)
    shards = oracle.scatter_global(part, x, fill=lambda w: np.full(part.padded_shape(w), 77.0))
    H = oracle.halo_fwd_definition if form == "definition" else oracle.halo_fwd_sequence
    out = H(part, shards)
    for w, o in zip(ws, out):
        expect = [0.0 if v == "-" else float(int(v) + 1) for v in w["view"]]
        # the figures of the pooling cases draw unused inputs too: they are part of the bulk
        assert o.tolist() == expect


def test_balanced_split_from_appendix_b():
    assert oracle.balanced_split(11, 3)[1] == [4, 4, 3]
    assert oracle.balanced_split(7, 3)[1] == [3, 2, 2]
    assert oracle.balanced_split(10, 3)[1] == [4, 3, 3]
    assert oracle.balanced_split(20, 6) == ([0, 4, 8, 11, 14, 17], [4, 4, 3, 3, 3, 3])
    assert oracle.balanced_split(10, 6)[1] == [2, 2, 2, 2, 1, 1]


def test_worker_numbering_is_row_major():
    # Appendix B.2: workers 0,1 are the top row of a 2 x 2 partition, 2,3 the bottom row.
    part = Partition((4, 4), (2, 2))
    assert [part.coords(w) for w in range(4)] == [(0, 0), (0, 1), (1, 0), (1, 1)]
    assert part.bulk_start(1) == (0, 2) and part.bulk_start(2) == (2, 0)


# --------------------------------------------------------------------------
# Broadcast / sum-reduce
# --------------------------------------------------------------------------

def test_broadcast_and_sumreduce_dense_matrices():
    n, k = 5, 3
    Bm = np.vstack([np.eye(n)] * k)                      # [I; I; I]
    x = inputs.uniform_pm1((n,), 1)
    got = np.concatenate(oracle.broadcast_fwd(x, k))
    assert np.array_equal(got, (Bm @ x.astype(np.float64)).astype(np.float32))
    ys = [inputs.integers((n,), 10 + i) for i in range(k)]
    got = oracle.sumreduce_fwd(ys)
    assert np.array_equal(got, (Bm.T @ np.concatenate(ys).astype(np.float64)).astype(np.float32))
    # operator matrices from unit vectors are each other's transpose
    MB = np.stack([np.concatenate(oracle.broadcast_fwd(e, k)) for e in np.eye(n, dtype=np.float32)], 1)
    MR = np.stack([oracle.sumreduce_fwd(np.split(e, k)) for e in np.eye(n * k, dtype=np.float32)], 1)
    assert np.array_equal(MB, Bm) and np.array_equal(MR, Bm.T)


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_reduce_after_broadcast_is_k_times_identity(k):
    x = inputs.uniform_pm1((1000,), 2)
    got = oracle.sumreduce_fwd(oracle.broadcast_fwd(x, k))
    if k <= 2:
        assert np.array_equal(got, x * np.float32(k))    # x + x is exact
    # the left fold rounds the odd multiples (3x, 5x, ...): at most k-2 roundings of 2^-24 each
    assert np.all(np.abs(got.astype(np.float64) - k * x.astype(np.float64))
                  <= (k - 1) * 2.0 ** -24 * k * np.abs(x.astype(np.float64)))
    xi = inputs.integers((1000,), 2)
    assert np.array_equal(oracle.sumreduce_fwd(oracle.broadcast_fwd(xi, k)), xi * np.float32(k))


def test_sumreduce_order_and_signed_zero():
    # fixed worker order: ((a + b) + c), not (a + (b + c))
    a, b, c = np.float32(1e8), np.float32(-1e8), np.float32(1.0)
    assert oracle.sumreduce_fwd([np.array([a]), np.array([b]), np.array([c])])[0] == np.float32(1.0)
    assert oracle.sumreduce_fwd([np.array([c]), np.array([a]), np.array([b])])[0] == np.float32(0.0)
    # the fold starts from y_0, so k = 1 keeps -0.0
    z = oracle.sumreduce_fwd([np.array([-0.0], dtype=np.float32)])
    assert np.signbit(z[0])
    x = inputs.uniform_pm1((7,), 3)
    assert oracle.sumreduce_fwd([x]).tobytes() == x.tobytes()


def test_broadcast_dot_test_closed_form():
    # <Bx, y> = <x, sum_i y_i>
    k, n = 4, 257
    x = inputs.uniform_pm1((n,), 4)
    ys = [inputs.uniform_pm1((n,), 20 + i) for i in range(k)]
    r = oracle.adjoint_test_ratio(oracle.broadcast_fwd(x, k), ys, [x], [oracle.broadcast_adj(ys)])
    assert r < 1e-6


def test_adjoint_ratio_known_values():
    x = [np.array([1.0, 2.0])]
    assert oracle.adjoint_test_ratio(x, x, x, x) == 0.0          # F = I
    # F = 2I claimed adjoint I: <Fx,y> = 2*5, <x,F*y> = 5, norms: |Fx||y| = 10, |x||F*y| = 5
    Fx = [np.array([2.0, 4.0])]
    assert oracle.adjoint_test_ratio(Fx, x, x, x) == pytest.approx(0.5)


# --------------------------------------------------------------------------
# Halo exchange: brute-force matrices
# --------------------------------------------------------------------------

HALO_CASES = [
    # global shape, partition, hlo, hhi
    ((11,), (3,), 2, 2),
    ((7,), (1,), 1, 2),
    ((10,), (4,), [[0, 1, 2, 1]], [[1, 0, 2, 0]]),
    ((6, 6), (2, 2), 1, 1),
    ((7, 5), (3, 2), (1, 2), (2, 1)),
    ((9, 8), (2, 2), [[0, 4], [3, 0]], [[2, 0], [0, 3]]),      # Appendix B.2 style widths
    ((5, 6, 7), (2, 1, 3), (1, 2, 1), (1, 0, 2)),
    ((4, 4, 4), (2, 2, 2), 1, 1),
    ((6, 4), (3, 1), 2, 2),                                   # bulk 2 = halo: both-side receivers
    ((3, 3, 2, 4), (1, 1, 2, 2), (0, 0, 1, 1), (0, 0, 1, 1)),
]
HALO_IDS = ["1d", "1d_p1", "1d_asym", "2d", "2d_uneven", "2d_appB2", "3d_uneven", "3d_corner", "thin", "4d"]


def _cells(part):
    """Flat list of (worker, padded-local index) and the offset of each worker's block."""
    cells, off = [], []
    for w in range(part.num_workers):
        off.append(len(cells))
        for l in itertools.product(*[range(v) for v in part.padded_shape(w)]):
            cells.append((w, l))
    return cells, off


def _brute_force_H_matrix(part):
    """0/1 matrix of H built cell by cell: each ghost cell looks for the worker owning its
    global index by testing every worker's bulk box."""
    cells, off = _cells(part)
    index = {c: i for i, c in enumerate(cells)}
    M = np.zeros((len(cells), len(cells)))
    for i, (w, l) in enumerate(cells):
        st, sh = part.bulk_start(w), part.bulk_shape(w)
        lo, _ = part.widths(w)
        g = tuple(st[k] - lo[k] + l[k] for k in range(part.rank))
        in_bulk = all(lo[k] <= l[k] < lo[k] + sh[k] for k in range(part.rank))
        if in_bulk:
            M[i, i] = 1.0
            continue
        for v in range(part.num_workers):
            vs, vh = part.bulk_start(v), part.bulk_shape(v)
            if all(vs[k] <= g[k] < vs[k] + vh[k] for k in range(part.rank)):
                vlo, _ = part.widths(v)
                M[i, index[(v, tuple(g[k] - vs[k] + vlo[k] for k in range(part.rank)))]] = 1.0
                break
    return M


def _flatten(shards):
    return np.concatenate([np.asarray(s).ravel() for s in shards])


def _unflatten(part, v, dtype=np.float32):
    out, o = [], 0
    for w in range(part.num_workers):
        n = int(np.prod(part.padded_shape(w)))
        out.append(np.array(v[o:o + n], dtype=dtype).reshape(part.padded_shape(w)))
        o += n
    return out


def _operator_matrix(part, op):
    n = sum(int(np.prod(part.padded_shape(w))) for w in range(part.num_workers))
    cols = []
    for i in range(n):
        e = np.zeros(n, dtype=np.float32)
        e[i] = 1.0
        cols.append(_flatten(op(part, _unflatten(part, e))))
    return np.stack(cols, 1)


@pytest.mark.parametrize("case", HALO_CASES, ids=HALO_IDS)
def test_halo_matrices_match_brute_force_and_transpose(case):
    part = Partition(*case)
    M = _brute_force_H_matrix(part)
    assert np.array_equal(_operator_matrix(part, oracle.halo_fwd_definition), M)
    assert np.array_equal(_operator_matrix(part, oracle.halo_fwd_sequence), M)
    assert np.array_equal(_operator_matrix(part, oracle.halo_adj_sequence), M.T)


def _random_shards(part, seed, kind="uniform"):
    out = []
    for w in range(part.num_workers):
        gen = inputs.uniform_pm1 if kind == "uniform" else inputs.integers
        out.append(gen(part.padded_shape(w), seed * 1000 + w))
    return out


@pytest.mark.parametrize("case", HALO_CASES, ids=HALO_IDS)
def test_halo_forms_agree_bitwise_and_match_numpy_pad(case):
    part = Partition(*case)
    x = _random_shards(part, 5)                      # garbage in the ghosts
    a = oracle.halo_fwd_definition(part, x)
    b = oracle.halo_fwd_sequence(part, x)
    g = oracle.assemble_global(part, x)
    for w in range(part.num_workers):
        assert a[w].tobytes() == b[w].tobytes()
        # library pin: a window of the zero-padded global tensor
        lo, hi = part.widths(w)
        mlo, mhi = max(max(part.hlo[k]) for k in range(part.rank)), max(max(part.hhi[k]) for k in range(part.rank))
        gp = np.pad(g, [(mlo, mhi)] * part.rank)
        st, ps = part.bulk_start(w), part.padded_shape(w)
        win = tuple(slice(st[k] - lo[k] + mlo, st[k] - lo[k] + mlo + ps[k]) for k in range(part.rank))
        assert np.array_equal(a[w], gp[win])


def test_halo_special_cases():
    # a single worker: H only zeroes the ghosts
    part = Partition((5, 4), (1, 1), 2, 1)
    x = _random_shards(part, 6)
    out = oracle.halo_fwd_sequence(part, x)[0]
    ref = np.zeros_like(x[0])
    ref[part.bulk_slices(0)] = x[0][part.bulk_slices(0)]
    assert np.array_equal(out, ref)
    # zero widths: H and H* are the identity
    part = Partition((5, 4), (2, 2), 0, 0)
    x = _random_shards(part, 7)
    for op in (oracle.halo_fwd_definition, oracle.halo_fwd_sequence, oracle.halo_adj_sequence):
        assert all(np.array_equal(a, b) for a, b in zip(op(part, x), x))


@pytest.mark.parametrize("case", HALO_CASES, ids=HALO_IDS)
def test_halo_adjoint_invariants(case):
    part = Partition(*case)
    M = _brute_force_H_matrix(part)
    # integer-valued inputs: every summation order gives the same fp32 result
    y = _random_shards(part, 8, "int")
    got = oracle.halo_adj_sequence(part, y)
    assert np.array_equal(_flatten(got), (M.T @ _flatten(y).astype(np.float64)).astype(np.float32))
    # all ghosts are zero on exit
    y = _random_shards(part, 9)
    got = oracle.halo_adj_sequence(part, y)
    for w in range(part.num_workers):
        mask = np.ones(part.padded_shape(w), dtype=bool)
        mask[part.bulk_slices(w)] = False
        assert not got[w][mask].any()
    # dot-product test
    x = _random_shards(part, 10)
    r = oracle.adjoint_test_ratio(oracle.halo_fwd_sequence(part, x), y, x, got)
    assert r < 1e-6
    # the sum over all cells is kept, up to what sits in exterior ghosts (dropped)
    total = float(np.sum(M.T @ _flatten(y).astype(np.float64)))
    assert float(np.sum(_flatten(got).astype(np.float64))) == pytest.approx(total, rel=1e-5, abs=1e-4)


def test_halo_adjoint_order_worked_case():
    """2 x 2 partition of a 2 x 2 tensor, width 1 everywhere: the single bulk cell of worker 0
    receives from the ghosts of workers 1, 2 and 3.  The adjoint undoes dimension 1 first
    (Appendix B.2: "adjoint of second phase" comes first), so
        result = (own + w1's ghost) + (w2's ghost + w3's corner ghost),
    evaluated here by hand in fp32 with values for which other orders differ."""
    part = Partition((2, 2), (2, 2), 1, 1)
    y = [np.zeros((3, 3), dtype=np.float32) for _ in range(4)]
    own, g1, g2, g3 = np.float32(1.0), np.float32(1e8), np.float32(-1e8), np.float32(3.0)
    y[0][1, 1] = own        # worker 0's bulk cell (global (0,0))
    y[1][1, 0] = g1         # worker 1 (right of 0): its low ghost in dim 1
    y[2][0, 1] = g2         # worker 2 (below 0): its low ghost in dim 0
    y[3][0, 0] = g3         # worker 3 (diagonal): corner ghost
    got = oracle.halo_adj_sequence(part, y)[0][1, 1]
    expect = np.float32(np.float32(own + g1) + np.float32(g2 + g3))
    assert got == expect == np.float32(0.0)
    # a different association would not give this
    assert np.float32(np.float32(np.float32(own + g1) + g2) + g3) == np.float32(3.0)


def test_halo_adjoint_both_sides_low_first():
    # 1-D, 3 workers, bulk 1, width 1: the middle cell receives from both neighbours, low first
    part = Partition((3,), (3,), 1, 1)
    y = [np.zeros(3, dtype=np.float32) for _ in range(3)]
    y[1][1] = np.float32(1.0)
    y[0][2] = np.float32(1e8)      # low neighbour's high ghost
    y[2][0] = np.float32(-1e8)     # high neighbour's low ghost
    got = oracle.halo_adj_sequence(part, y)[1][1]
    assert got == np.float32(np.float32(np.float32(1.0) + np.float32(1e8)) + np.float32(-1e8)) == np.float32(0.0)


def test_appendix_b2_unbalanced_2d_exchange():
    """Appendix B.2 in words: 2 x 2 partition; workers 0 and 2 need nothing from 1 and 3 but
    give them width 3; workers 0,1 need width 2 from 2,3; workers 2,3 need width 4 from 0,1."""
    part = Partition((9, 8), (2, 2), [[0, 4], [0, 3]], [[2, 0], [0, 0]])
    g = np.arange(72, dtype=np.float32).reshape(9, 8) + 1
    x = oracle.scatter_global(part, g, fill=lambda w: np.full(part.padded_shape(w), -5.0))
    a = oracle.halo_fwd_sequence(part, x)
    assert a[0].shape == (5 + 2, 4) and a[1].shape == (5 + 2, 4 + 3)
    assert a[2].shape == (4 + 4, 4) and a[3].shape == (4 + 4, 4 + 3)
    assert np.array_equal(a[3], g[1:9, 1:8])          # rows 5-4.., cols 4-3..: a plain window
    assert np.array_equal(a[1], g[0:7, 1:8])
    assert np.array_equal(a[0], g[0:7, 0:4]) and np.array_equal(a[2], g[1:9, 0:4])


# --------------------------------------------------------------------------
# Convolution layer
# --------------------------------------------------------------------------

CONV_PARTS = [(1, 1, 1, 1), (1, 1, 2, 2), (1, 1, 3, 2), (1, 1, 1, 4)]


def _conv_problem(pshape, shape=(2, 3, 12, 13), k=(5, 5), seed=11):
    part = Partition(shape, pshape, (0, 0, k[0] // 2, k[1] // 2), (0, 0, k[0] // 2, k[1] // 2))
    xg = inputs.normal(shape, seed)
    w = inputs.normal((shape[1],) + k, seed + 1, 0.1)
    return part, xg, w


@pytest.mark.parametrize("pshape", CONV_PARTS)
def test_conv_fwd_matches_scipy_on_global_tensor(pshape):
    part, xg, w = _conv_problem(pshape)
    bias = inputs.normal((xg.shape[1],), 13)
    x = oracle.scatter_global(part, xg, fill=lambda wk: np.full(part.padded_shape(wk), 9.0))
    y = oracle.assemble_global(Partition(xg.shape, pshape), oracle.conv_fwd(part, x, w, bias))
    for n in range(xg.shape[0]):
        for c in range(xg.shape[1]):
            ref = correlate2d(xg[n, c].astype(np.float64), w[c].astype(np.float64), mode="same") + float(bias[c])
            assert np.allclose(y[n, c], ref, rtol=0, atol=2e-6)


@pytest.mark.parametrize("pshape", CONV_PARTS)
def test_conv_adj_is_transpose_and_matches_stepwise_form(pshape):
    part, xg, w = _conv_problem(pshape, shape=(1, 2, 7, 6), k=(5, 3))
    ypart = Partition(xg.shape, pshape)
    dyg = inputs.normal(xg.shape, 14)
    dy = oracle.scatter_global(ypart, dyg)
    dx = oracle.conv_adj(part, dy, w)
    # library pin: the adjoint of a same-size correlation is the same-size convolution,
    # i.e. correlation with the kernel rotated by 180 degrees
    dxg = oracle.assemble_global(part, dx)
    for c in range(xg.shape[1]):
        ref = correlate2d(dyg[0, c].astype(np.float64), w[c, ::-1, ::-1].astype(np.float64), mode="same")
        assert np.allclose(dxg[0, c], ref, rtol=0, atol=2e-6)
    # ghosts are zero
    for wk in range(part.num_workers):
        mask = np.ones(part.padded_shape(wk), dtype=bool)
        mask[part.bulk_slices(wk)] = False
        assert not dx[wk][mask].any()
    # step-by-step algorithm (local adjoint into padded shards, then H*)
    dx2 = oracle.conv_adj_scatter_then_halo(part, dy, w)
    for a, b in zip(dx, dx2):
        assert np.allclose(a, b, rtol=0, atol=5e-6)
    # dot-product test <Conv x, dy> = <x, Conv* dy> on the bulk
    x = oracle.scatter_global(part, xg)
    y = oracle.conv_fwd(part, x, w)
    assert oracle.adjoint_test_ratio(y, dy, x, dx) < 1e-6


def test_conv_unit_impulse_orientation():
    # cross-correlation: an impulse at (i0, j0) puts w[a, b] at output (i0 - a + ph, j0 - b + pw)
    part, _, w = _conv_problem((1, 1, 2, 2), shape=(1, 1, 8, 8))
    xg = np.zeros((1, 1, 8, 8), dtype=np.float32)
    xg[0, 0, 4, 3] = 1.0
    y = oracle.assemble_global(Partition(xg.shape, part.pshape), oracle.conv_fwd(part, oracle.scatter_global(part, xg), w))
    for a in range(5):
        for b in range(5):
            assert y[0, 0, 4 - a + 2, 3 - b + 2] == w[0, a, b]


# --------------------------------------------------------------------------
# Affine layer
# --------------------------------------------------------------------------

def _affine_problem(nb, nfi, nfo, pfo, pfi, seed, integer=False):
    if integer:
        xg = inputs.integers((nb, nfi), seed)
        wg = inputs.integers((nfo, nfi), seed + 1)
    else:
        xg = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(inputs.normal((nb, nfi), seed)))
        wg = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(inputs.normal((nfo, nfi), seed + 1, nfi ** -0.5)))
    xs = np.split(xg, pfi, axis=1)
    ws = [blk for row in np.split(wg, pfo, axis=0) for blk in np.split(row, pfi, axis=1)]
    return xg, wg, xs, ws


@pytest.mark.parametrize("pfo,pfi", [(1, 1), (2, 2), (4, 2), (1, 4)])
def test_affine_matches_plain_matmul(pfo, pfi):
    xg, wg, xs, ws = _affine_problem(6, 16, 8, pfo, pfi, 21, integer=True)
    bias = inputs.integers((8,), 23)
    y = np.concatenate(oracle.affine_fwd(xs, ws, pfo, pfi, np.split(bias, pfo)), axis=1)
    assert np.array_equal(y, xg @ wg.T + bias[None, :])            # integers: exact, bias once
    dyg = inputs.integers((6, 8), 24)
    dx = np.concatenate(oracle.affine_adj(np.split(dyg, pfo, axis=1), ws, pfo, pfi), axis=1)
    assert np.array_equal(dx, dyg @ wg)


def test_affine_bf16_inputs_against_fp64_and_dot_test():
    pfo = pfi = 2
    xg, wg, xs, ws = _affine_problem(8, 64, 32, pfo, pfi, 25)
    y = oracle.affine_fwd(xs, ws, pfo, pfi)
    ref = xg.astype(np.float64) @ wg.astype(np.float64).T
    assert np.allclose(np.concatenate(y, axis=1), ref, rtol=1e-6, atol=1e-6)
    dyg = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(inputs.normal((8, 32), 26)))
    dys = np.split(dyg, pfo, axis=1)
    dx = oracle.affine_adj(dys, ws, pfo, pfi)
    assert np.allclose(np.concatenate(dx, axis=1), dyg.astype(np.float64) @ wg.astype(np.float64), rtol=1e-6, atol=1e-6)
    assert oracle.adjoint_test_ratio(y, dys, xs, dx) < 1e-6


def test_bf16_helpers_round_to_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 (even mantissa) and 1 + 2^-7: goes to 1.0
    a = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0], dtype=np.float32)
    bits = inputs.f32_to_bf16_bits(a)
    assert bits.tolist() == [0x3F80, 0x3F82, 0xC020, 0x0000]
    assert oracle.bf16_bits_to_f64(bits).tolist() == [1.0, 1.0 + 2.0 ** -6, -2.5, 0.0]
    assert inputs.bf16_bits_to_f32(bits).tolist() == [1.0, 1.0 + 2.0 ** -6, -2.5, 0.0]


# --------------------------------------------------------------------------
# Distributed pooling layer (Section 4 "Sparse layers" + Appendix B halos)
# --------------------------------------------------------------------------

POOL_CASES = [
    # global shape, partition, kernel, stride, padding
    ((2, 3, 11, 10), (1, 1, 3, 2), (2, 2), (2, 2), ((0, 0), (0, 0))),
    ((1, 2, 20, 17), (1, 1, 6, 3), (3, 3), (2, 2), ((1, 1), (1, 1))),
    ((1, 1, 12, 12), (1, 1, 2, 2), (3, 2), (1, 2), ((1, 0), (0, 1))),
    ((1, 1, 1, 20), (1, 1, 1, 6), (1, 2), (1, 2), ((0, 0), (0, 0))),     # Fig. B4 along the last dimension
    ((1, 1, 1, 10), (1, 1, 1, 3), (1, 2), (1, 2), ((0, 0), (0, 0))),     # Fig. B3
    ((1, 2, 9, 9), (1, 1, 1, 1), (3, 3), (3, 3), ((0, 0), (0, 0))),
]


def _pool_setup(case, seed):
    gs, ps, k, s, pad = case
    part, geo = oracle.layers.pool_partition(gs, ps, k, s, pad)
    xg = inputs.normal(gs, seed)
    garbage = lambda w: inputs.normal(part.padded_shape(w), seed + 100 + w)
    return part, geo, xg, oracle.scatter_global(part, xg, fill=garbage)


def _out_block(geo, part, w):
    c = part.coords(w)
    return (slice(None), slice(None)) + tuple(
        slice(geo[k][c[2 + k]]["out_start"], geo[k][c[2 + k]]["out_start"] + geo[k][c[2 + k]]["out_size"]) for k in range(2))


@pytest.mark.parametrize("mode", ["avg", "max"])
def test_pool_global_matches_library_routine(mode):
    import torch
    import torch.nn.functional as F
    xg = inputs.normal((2, 3, 13, 14), 71)
    t = torch.from_numpy(xg)
    for k, s, p in [((3, 3), (2, 2), 1), ((2, 2), (2, 2), 0), ((3, 2), (1, 2), 0), ((5, 5), (3, 3), 2)]:
        pad = ((p, p), (p, p))
        y, arg = oracle.layers.pool_fwd_global(xg, k, s, pad, mode)
        if mode == "avg":
            ref = F.avg_pool2d(t, k, s, p).numpy()           # padding counts in the divisor by default
            assert np.max(np.abs(y - ref)) <= 4 * 2.0 ** -24 * np.max(np.abs(xg))
        else:
            ref, idx = F.max_pool2d(t, k, s, p, return_indices=True)
            assert np.array_equal(y, ref.numpy())
            # position inside the window -> flat index into the input plane (no ties in random data)
            Ho, Wo = y.shape[2:]
            i = np.arange(Ho)[:, None] * s[0] - p + arg // k[1]
            j = np.arange(Wo)[None, :] * s[1] - p + arg % k[1]
            assert np.array_equal(i * xg.shape[3] + j, idx.numpy())


def test_pool_max_takes_first_of_equal_values_and_skips_padding():
    xg = np.zeros((1, 1, 4, 4), np.float32)
    y, arg = oracle.layers.pool_fwd_global(xg, (2, 2), (2, 2), ((0, 0), (0, 0)), "max")
    assert np.all(arg == 0)
    xg = -np.ones((1, 1, 4, 4), np.float32)                   # padding must not win over negative data
    y, arg = oracle.layers.pool_fwd_global(xg, (3, 3), (2, 2), ((1, 1), (1, 1)), "max")
    assert np.all(y == -1.0) and arg[0, 0, 0, 0] == 4 and arg[0, 0, 1, 1] == 0


@pytest.mark.parametrize("case", POOL_CASES, ids=[str(c[:2]) for c in POOL_CASES])
@pytest.mark.parametrize("mode", ["avg", "max"])
def test_pool_distributed_forward_equals_sequential_layer(case, mode):
    gs, ps, k, s, pad = case
    part, geo, xg, xs = _pool_setup(case, 5)
    yg, ag = oracle.layers.pool_fwd_global(xg, k, s, pad, mode)
    ys, ar = oracle.layers.pool_fwd(part, geo, xs, k, s, pad, mode)
    for w in range(part.num_workers):
        assert np.array_equal(ys[w], yg[_out_block(geo, part, w)])
        if mode == "max":
            assert np.array_equal(ar[w], ag[_out_block(geo, part, w)])


@pytest.mark.parametrize("case", POOL_CASES, ids=[str(c[:2]) for c in POOL_CASES])
@pytest.mark.parametrize("mode", ["avg", "max"])
def test_pool_adjoint_is_transpose_and_partition_invariant(case, mode):
    gs, ps, k, s, pad = case
    part, geo, xg, xs = _pool_setup(case, 9)
    yg, ag = oracle.layers.pool_fwd_global(xg, k, s, pad, mode)
    dyg = inputs.integers(yg.shape, 33)
    dxg = oracle.layers.pool_adj_global(dyg, gs[2:], k, s, pad, mode, ag)
    # brute force: column e of the forward operator (for max: of its Jacobian) applied to dy
    if np.prod(gs) <= 400:
        for e in range(0, int(np.prod(gs)), 7):
            if mode == "avg":
                u = np.zeros(gs, np.float32)
                u.reshape(-1)[e] = 1.0
                col, _ = oracle.layers.pool_fwd_global(u, k, s, pad, "avg")
                want = float(np.sum(col.astype(np.float64) * dyg))
            else:
                idx = np.unravel_index(e, gs)
                Ho, Wo = yg.shape[2:]
                i = np.arange(Ho)[:, None] * s[0] - pad[0][0] + ag[idx[0], idx[1]] // k[1]
                j = np.arange(Wo)[None, :] * s[1] - pad[1][0] + ag[idx[0], idx[1]] % k[1]
                want = float(np.sum(dyg[idx[0], idx[1]][(i == idx[2]) & (j == idx[3])]))
            assert abs(float(dxg.reshape(-1)[e]) - want) <= 1e-6 * max(1.0, abs(want))
    # the distributed adjoint (local adjoint, then H*) gives the same tensor for every partition
    dys = [dyg[_out_block(geo, part, w)] for w in range(part.num_workers)]
    ars = None if mode == "avg" else [ag[_out_block(geo, part, w)] for w in range(part.num_workers)]
    dxs = oracle.layers.pool_adj(part, geo, dys, k, s, pad, mode, ars)
    got = oracle.assemble_global(part, dxs)
    assert np.max(np.abs(got - dxg)) <= 4 * 2.0 ** -24 * max(1.0, np.max(np.abs(dxg)))
    for w in range(part.num_workers):                          # ghosts are zero on exit
        g = dxs[w].copy()
        g[part.bulk_slices(w)] = 0
        assert not g.any()
    if mode == "max":                                          # every dy lands in exactly one cell
        assert np.sum(got.astype(np.float64)) == np.sum(dyg.astype(np.float64))


@pytest.mark.parametrize("case", POOL_CASES[:4], ids=[str(c[:2]) for c in POOL_CASES[:4]])
def test_pool_avg_dot_test(case):
    gs, ps, k, s, pad = case
    part, geo, xg, xs = _pool_setup(case, 21)
    xs = oracle.scatter_global(part, xg)                       # the operator acts on the bulk; ghosts are overwritten
    ys, _ = oracle.layers.pool_fwd(part, geo, xs, k, s, pad, "avg")
    dys = [inputs.normal(y.shape, 40 + w) for w, y in enumerate(ys)]
    dxs = oracle.layers.pool_adj(part, geo, dys, k, s, pad, "avg")
    assert oracle.adjoint_test_ratio(ys, dys, xs, dxs) < 1e-6


# --------------------------------------------------------------------------
# Generalized all-to-all, scatter / gather, all-reduce (Section 3)
# --------------------------------------------------------------------------

REPART_CASES = [
    # global shape, source partition, destination partition
    ((7, 9), (2, 1), (1, 3)),
    ((6, 10), (3, 2), (2, 5)),
    ((5, 4, 6), (1, 2, 3), (5, 1, 1)),
    ((12,), (1,), (5,)),            # scatter
    ((12,), (4,), (1,)),            # gather
    ((4, 6), (2, 2), (2, 2)),       # identity
]


@pytest.mark.parametrize("case", REPART_CASES, ids=[str(c) for c in REPART_CASES])
def test_repartition_is_a_permutation_with_inverse_adjoint(case):
    gs, sp, dp = case
    src, dst = Partition(gs, sp), Partition(gs, dp)
    n = int(np.prod(gs))
    sizes_s = [int(np.prod(src.padded_shape(w))) for w in range(src.num_workers)]
    sizes_d = [int(np.prod(dst.padded_shape(w))) for w in range(dst.num_workers)]
    assert sum(sizes_s) == n and sum(sizes_d) == n

    def apply(fn, a, b, vec, sizes):
        parts, at = [], 0
        for w, z in enumerate(sizes):
            parts.append(vec[at:at + z].reshape(a.padded_shape(w)))
            at += z
        return np.concatenate([p.reshape(-1) for p in fn(a, b, parts)]) if fn is oracle.repartition_fwd else \
            np.concatenate([p.reshape(-1) for p in fn(b, a, parts)])

    eye = np.eye(n, dtype=np.float32)
    F = np.stack([apply(oracle.repartition_fwd, src, dst, eye[e], sizes_s) for e in range(n)], axis=1)
    A = np.stack([apply(oracle.repartition_adj, dst, src, eye[e], sizes_d) for e in range(n)], axis=1)
    assert np.all(F.sum(axis=0) == 1) and np.all(F.sum(axis=1) == 1) and set(np.unique(F)) <= {0.0, 1.0}
    assert np.array_equal(A, F.T)                       # adjoint = transpose
    assert np.array_equal(A @ F, eye)                   # = inverse: the round trip is the identity


def test_repartition_transpose_scatter_gather_against_numpy_splits():
    g = inputs.uniform_pm1((8, 12), 3)
    rows, cols = Partition((8, 12), (4, 1)), Partition((8, 12), (1, 3))
    out = oracle.repartition_fwd(rows, cols, np.split(g, 4, axis=0))      # row blocks -> column blocks
    for got, ref in zip(out, np.split(g, 3, axis=1)):
        assert np.array_equal(got, ref)
    one, many = Partition((10,), (1,)), Partition((10,), (3,))
    v = inputs.uniform_pm1((10,), 4)
    sc = oracle.repartition_fwd(one, many, [v])                            # scatter: blocks 4, 3, 3
    assert [a.shape[0] for a in sc] == [4, 3, 3] and np.array_equal(np.concatenate(sc), v)
    assert np.array_equal(oracle.repartition_fwd(many, one, sc)[0], v)     # gather


def test_allreduce_is_symmetric_and_gives_every_worker_the_sum():
    k, n = 3, 4
    cols = []
    for e in range(k * n):
        u = np.zeros(k * n, np.float32)
        u[e] = 1
        cols.append(np.concatenate(oracle.allreduce([u[i * n:(i + 1) * n] for i in range(k)])))
    M = np.stack(cols, axis=1)
    assert np.array_equal(M, M.T)                                          # self-adjoint
    assert np.array_equal(M, np.kron(np.ones((k, k), np.float32), np.eye(n, dtype=np.float32)))
    parts = [inputs.uniform_pm1((1000,), 50 + i) for i in range(5)]
    out = oracle.allreduce(parts)
    ref = parts[0]
    for p in parts[1:]:
        ref = ref + p                                                      # fp32 left fold
    assert all(o.tobytes() == ref.tobytes() for o in out)


# --------------------------------------------------------------------------
# Broadcast / sum-reduce along partition dimensions (Section 4: the B and R of the layer algorithms)
# --------------------------------------------------------------------------

PARTITION_BROADCAST_CASES = [
    # source partition, destination partition, elements of every source realisation
    ((1,), (4,), [5]),
    ((1, 3), (2, 3), [2, 3, 1]),                       # the affine layer's x: 1 x P_fi -> P_fo x P_fi
    ((2, 1), (2, 3), [2, 3]),                          # its y: P_fo x 1 <- P_fo x P_fi
    ((1, 1, 2, 2, 1), (1, 3, 2, 2, 1), [1, 2, 3, 2]),  # the convolution's x: 1 x 1 x P_ci x P_0 x P_1 -> 1 x P_co x P_ci x P_0 x P_1
    ((1, 2, 1, 2), (1, 2, 3, 2), [2, 1, 1, 3]),        # its y: 1 x P_co x 1 x P_0 <- 1 x P_co x P_ci x P_0
    ((2, 2), (2, 2), [1, 2, 3, 4]),                    # equal partitions: the identity
]


def _pb_matrix(src_p, dst_p, sizes, adjoint):
    """The operator as a dense matrix, one column per unit vector, through the oracle."""
    src_of = oracle.primitives._partition_sources(src_p, dst_p)
    in_sizes = [sizes[j] for j in src_of] if adjoint else sizes
    total = sum(in_sizes)
    cols = []
    for e in range(total):
        u = np.zeros(total, np.float32)
        u[e] = 1
        parts, at = [], 0
        for n in in_sizes:
            parts.append(u[at:at + n])
            at += n
        out = (oracle.partition_broadcast_adj(src_p, dst_p, parts) if adjoint
               else oracle.partition_broadcast_fwd(src_p, dst_p, parts))
        cols.append(np.concatenate(out))
    return np.stack(cols, axis=1)


@pytest.mark.parametrize("case", PARTITION_BROADCAST_CASES, ids=[str(c[0]) + "->" + str(c[1]) for c in PARTITION_BROADCAST_CASES])
def test_partition_broadcast_is_the_stacked_identity_matrix_and_its_adjoint_the_transpose(case):
    src_p, dst_p, sizes = case
    B = _pb_matrix(src_p, dst_p, sizes, False)
    # built by hand, without the oracle: destination worker w (row-major coordinates) copies source worker j, whose
    # coordinates are w's where the source partition has several workers and 0 where it has one
    offs = np.concatenate([[0], np.cumsum(sizes)])
    blocks = []
    for w in np.ndindex(*dst_p):
        j = int(np.ravel_multi_index([c if p > 1 else 0 for c, p in zip(w, src_p)], src_p))
        blk = np.zeros((sizes[j], offs[-1]), np.float32)
        blk[:, offs[j]:offs[j + 1]] = np.eye(sizes[j], dtype=np.float32)
        blocks.append(blk)
    assert np.array_equal(B, np.concatenate(blocks, axis=0))
    assert np.array_equal(_pb_matrix(src_p, dst_p, sizes, True), B.T)
    copies = int(np.prod(dst_p)) // int(np.prod(src_p))
    assert np.array_equal(B.T @ B, copies * np.eye(offs[-1], dtype=np.float32))       # R B = k I


def test_partition_broadcast_special_cases_order_of_the_sum_and_dot_test():
    x = inputs.uniform_pm1((1000,), 5)
    out = oracle.partition_broadcast_fwd((1,), (5,), [x])                   # one source worker: the plain broadcast
    assert all(a.tobytes() == b.tobytes() for a, b in zip(out, oracle.broadcast_fwd(x, 5)))
    ys = [inputs.uniform_pm1((1000,), 60 + i) for i in range(5)]
    assert oracle.partition_broadcast_adj((1,), (5,), ys)[0].tobytes() == oracle.sumreduce_fwd(ys).tobytes()
    # order of the sum: in a 1 x 2 -> 3 x 2 partition pair source worker 1 gets (y1 + y3) + y5
    big, one = np.float32(2.0 ** 24), np.float32(1.0)
    ys = [np.zeros(1, np.float32), np.array([big]), np.zeros(1, np.float32), np.array([one]), np.zeros(1, np.float32),
          np.array([one])]
    got = oracle.partition_broadcast_adj((1, 2), (3, 2), ys)
    assert got[1][0] == big                                                 # (2^24 + 1) + 1 stays 2^24 in fp32 ...
    ys[1], ys[5] = ys[5], ys[1]
    assert oracle.partition_broadcast_adj((1, 2), (3, 2), ys)[1][0] == big + np.float32(2.0)   # ... (1 + 1) + 2^24 does not
    # bfloat16 sums through the same hook as the other folds
    b = [oracle.round_to_bf16_bits(inputs.uniform_pm1((64,), 70 + i).astype(np.float64)) for i in range(4)]
    ref = oracle.sumreduce_fwd([b[0], b[2]], add=oracle.bf16_add)
    assert np.array_equal(oracle.partition_broadcast_adj((1, 2), (2, 2), b, add=oracle.bf16_add)[0], ref)
    # adjoint test on random data
    src_p, dst_p, sizes = (1, 3), (4, 3), [50, 70, 30]
    xs = [inputs.uniform_pm1((n,), 80 + i) for i, n in enumerate(sizes)]
    ys = [inputs.uniform_pm1((sizes[w % 3],), 90 + w) for w in range(12)]
    r = oracle.adjoint_test_ratio(oracle.partition_broadcast_fwd(src_p, dst_p, xs), ys, xs,
                                  oracle.partition_broadcast_adj(src_p, dst_p, ys))
    assert r < 1e-6


# --------------------------------------------------------------------------
# Parameter gradients of the two layers (adjoint algorithms of Section 4: dW, db / dw, db)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("pfo,pfi", [(1, 1), (2, 2), (4, 2), (1, 4)])
def test_affine_param_gradients_exact_on_integers_and_against_autograd(pfo, pfi):
    import torch
    nb, nfi, nfo = 6, 16, 8
    xg, wg, xs, ws = _affine_problem(nb, nfi, nfo, pfo, pfi, 61, integer=True)
    dyg = inputs.integers((nb, nfo), 63)
    dw, db = oracle.affine_adj_params(np.split(dyg, pfo, axis=1), xs, pfo, pfi)
    dwg = np.concatenate([np.concatenate(dw[i * pfi:(i + 1) * pfi], axis=1) for i in range(pfo)], axis=0)
    # library routine on the unpartitioned operands: reverse-mode derivative of the framework's linear layer
    W = torch.tensor(wg, dtype=torch.float64, requires_grad=True)
    b = torch.zeros(nfo, dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.linear(torch.tensor(xg, dtype=torch.float64), W, b)
    y.backward(torch.tensor(dyg, dtype=torch.float64))
    assert np.array_equal(dwg, W.grad.numpy().astype(np.float32))
    assert np.array_equal(np.concatenate(db), b.grad.numpy().astype(np.float32))


def test_affine_param_gradients_brute_force_columns_and_dot_test():
    pfo, pfi, nb, nfi, nfo = 2, 2, 5, 8, 6
    xg, wg, xs, ws = _affine_problem(nb, nfi, nfo, pfo, pfi, 65)
    dyg = inputs.bf16_bits_to_f32(inputs.f32_to_bf16_bits(inputs.normal((nb, nfo), 66)))
    dys = np.split(dyg, pfo, axis=1)
    dw, db = oracle.affine_adj_params(dys, xs, pfo, pfi)
    bo, bi = nfo // pfo, nfi // pfi
    # the layer is linear in (W, b) for a fixed x: the gradient entry of one weight is <Affine(E; x), dy>
    # with E the unit weight tensor -- evaluated through the (separately pinned) forward oracle
    zero_w = [np.zeros((bo, bi), np.float32) for _ in range(pfo * pfi)]
    for i, j, o, f in itertools.product(range(pfo), range(pfi), range(bo), range(bi)):
        unit = [z.copy() for z in zero_w]
        unit[i * pfi + j][o, f] = 1.0
        y = oracle.affine_fwd(xs, unit, pfo, pfi)
        ref = sum(float((a.astype(np.float64) * d).sum()) for a, d in zip(y, dys))
        assert abs(float(dw[i * pfi + j][o, f]) - ref) <= 1e-6 * max(1.0, abs(ref))
    for i, o in itertools.product(range(pfo), range(bo)):
        unit_b = [np.zeros(bo, np.float32) for _ in range(pfo)]
        unit_b[i][o] = 1.0
        y = oracle.affine_fwd([np.zeros_like(x) for x in xs], zero_w, pfo, pfi, unit_b)
        ref = sum(float((a.astype(np.float64) * d).sum()) for a, d in zip(y, dys))
        assert abs(float(db[i][o]) - ref) <= 1e-6 * max(1.0, abs(ref))
    # dot test in parameter space: <Affine(W, b; x), dy> = <W, dW> + <b, db>
    bias = np.split(inputs.normal((nfo,), 67), pfo)
    y = oracle.affine_fwd(xs, ws, pfo, pfi, bias)
    assert oracle.adjoint_test_ratio(y, dys, list(ws) + bias, list(dw) + list(db)) < 1e-6


@pytest.mark.parametrize("pshape", CONV_PARTS)
def test_conv_param_gradients_against_autograd_and_partition_invariance(pshape):
    import torch
    part, xg, w = _conv_problem(pshape, shape=(2, 3, 12, 13), k=(5, 5), seed=71)
    dyg = inputs.normal(xg.shape, 73)
    x = oracle.scatter_global(part, xg, fill=lambda wk: np.full(part.padded_shape(wk), 7.0))   # garbage ghosts
    dy = oracle.scatter_global(Partition(xg.shape, pshape), dyg)
    dw, db = oracle.conv_adj_params(part, x, dy, 5, 5)
    W = torch.tensor(w[:, None], dtype=torch.float64, requires_grad=True)
    b = torch.zeros(xg.shape[1], dtype=torch.float64, requires_grad=True)
    y = torch.nn.functional.conv2d(torch.tensor(xg, dtype=torch.float64), W, b, padding=2, groups=xg.shape[1])
    y.backward(torch.tensor(dyg, dtype=torch.float64))
    assert np.allclose(dw, W.grad.numpy()[:, 0], rtol=1e-6, atol=1e-5)
    assert np.allclose(db, b.grad.numpy(), rtol=1e-6, atol=1e-5)
    # same result for every partition, 1 x 1 included
    one = Partition(xg.shape, (1, 1, 1, 1), (0, 0, 2, 2), (0, 0, 2, 2))
    dw1, db1 = oracle.conv_adj_params(one, oracle.scatter_global(one, xg), [dyg], 5, 5)
    assert np.allclose(dw, dw1, rtol=1e-6, atol=1e-5) and np.allclose(db, db1, rtol=1e-6, atol=1e-5)


def test_conv_param_gradients_brute_force_taps_and_dot_test():
    part, xg, w = _conv_problem((1, 1, 2, 2), shape=(1, 2, 7, 6), k=(5, 3), seed=75)
    ypart = Partition(xg.shape, part.pshape)
    dyg = inputs.normal(xg.shape, 77)
    x, dy = oracle.scatter_global(part, xg), oracle.scatter_global(ypart, dyg)
    dw, db = oracle.conv_adj_params(part, x, dy, 5, 3)
    # linear in (w, b): the gradient of tap (c, a, b) is <Conv(E_cab; x), dy> through the forward oracle
    for c, a, b in itertools.product(range(2), range(5), range(3)):
        unit = np.zeros_like(w)
        unit[c, a, b] = 1.0
        y = oracle.conv_fwd(part, x, unit)
        ref = sum(float((u.astype(np.float64) * v).sum()) for u, v in zip(y, dy))
        assert abs(float(dw[c, a, b]) - ref) <= 2e-6 * max(1.0, abs(ref))
    bias = inputs.normal((2,), 78)
    y = oracle.conv_fwd(part, x, w, bias)
    assert oracle.adjoint_test_ratio(y, dy, [w, bias], [dw, db]) < 1e-6


# --------------------------------------------------------------------------
# 3-D star-stencil layer (halo exchange + local sliding kernel on a rank-3 tensor)
# --------------------------------------------------------------------------

STENCIL_CASES = [
    # global shape, partition, radius
    ((6, 7, 8), (1, 1, 1), 2),
    ((9, 8, 10), (2, 2, 2), 2),
    ((12, 9, 13), (3, 1, 2), 4),
    ((5, 6, 7), (1, 2, 3), 1),
]


def _stencil_problem(case, seed):
    gs, ps, R = case
    part = Partition(gs, ps, R, R)
    xg = inputs.normal(gs, seed)
    w = inputs.normal((3, 2 * R + 1), seed + 1, 0.5)
    return part, xg, w


@pytest.mark.parametrize("case", STENCIL_CASES, ids=[str(c) for c in STENCIL_CASES])
def test_stencil3d_matches_library_correlation_and_stepwise_form(case):
    from scipy.ndimage import correlate1d
    part, xg, w = _stencil_problem(case, 81)
    x = oracle.scatter_global(part, xg, fill=lambda wk: np.full(part.padded_shape(wk), 5.0))    # garbage ghosts
    y = oracle.assemble_global(Partition(xg.shape, part.pshape), oracle.stencil3d_fwd(part, x, w))
    ref = sum(correlate1d(xg.astype(np.float64), w[d].astype(np.float64), axis=d, mode="constant", cval=0.0)
              for d in range(3))
    assert np.allclose(y, ref, rtol=0, atol=5e-6)
    # the distributed algorithm itself: exchange, then the local kernel on every padded shard
    for a, b in zip(oracle.stencil3d_fwd(part, x, w), oracle.stencil3d_fwd_exchange_then_local(part, x, w)):
        assert np.allclose(a, b, rtol=0, atol=5e-6)


def test_stencil3d_adjoint_is_the_transpose_matrix():
    gs, ps, R = (3, 4, 5), (1, 2, 2), 1
    part, ypart = Partition(gs, ps, R, R), Partition(gs, ps)
    w = inputs.normal((3, 3), 83, 0.5)
    n = int(np.prod(gs))
    F = np.zeros((n, n))
    A = np.zeros((n, n))
    for e in range(n):
        u = np.zeros(n, np.float32)
        u[e] = 1.0
        ug = u.reshape(gs)
        F[:, e] = oracle.assemble_global(ypart, oracle.stencil3d_fwd(part, oracle.scatter_global(part, ug), w)).reshape(-1)
        A[:, e] = oracle.assemble_global(part, oracle.stencil3d_adj(part, oracle.scatter_global(ypart, ug), w)).reshape(-1)
    assert np.array_equal(A, F.T)
    # the matrix itself, entry by entry: F[i, j] = sum of w[d][k + R] over (d, k) with j = i + k e_d
    idx = np.arange(n).reshape(gs)
    G = np.zeros((n, n))
    for i in itertools.product(*[range(v) for v in gs]):
        for d in range(3):
            for k in (-1, 0, 1):
                j = list(i)
                j[d] += k
                if 0 <= j[d] < gs[d]:
                    G[idx[i], idx[tuple(j)]] += float(np.float64(w[d][k + 1]))
    assert np.allclose(F, G.astype(np.float32), rtol=0, atol=1e-7)


@pytest.mark.parametrize("case", STENCIL_CASES[1:], ids=[str(c) for c in STENCIL_CASES[1:]])
def test_stencil3d_dot_test_and_zero_ghosts(case):
    part, xg, w = _stencil_problem(case, 85)
    ypart = Partition(xg.shape, part.pshape)
    x = oracle.scatter_global(part, xg)
    dy = oracle.scatter_global(ypart, inputs.normal(xg.shape, 87))
    y, dx = oracle.stencil3d_fwd(part, x, w), oracle.stencil3d_adj(part, dy, w)
    assert oracle.adjoint_test_ratio(y, dy, x, dx) < 1e-6
    for wk in range(part.num_workers):
        mask = np.ones(part.padded_shape(wk), dtype=bool)
        mask[part.bulk_slices(wk)] = False
        assert not dx[wk][mask].any()


# --------------------------------------------------------------------------
# bfloat16 and fp64 arithmetic of the sums (R, H*, all-reduce)
# --------------------------------------------------------------------------

def test_bf16_rounding_against_library_conversion_and_ties():
    import torch
    rng = np.random.Generator(np.random.Philox(97))
    vals = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-39).astype(np.float32),          # bfloat16 subnormals
        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 0.0, -0.0, 2.0 ** -133, 1.5 * 2.0 ** -133,
                  2.5 * 2.0 ** -133, 255.5, 256.5], dtype=np.float32)])
    ref = torch.from_numpy(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oracle.round_to_bf16_bits(vals.astype(np.float64))
    assert np.array_equal(got, ref)
    assert got[22000:22003].tolist() == [0x3F80, 0x3F82, 0xBF80]           # ties go to the even mantissa
    assert np.array_equal(oracle.bf16_bits_to_f64(got), oracle.bf16_bits_to_f64(ref))


def test_bf16_add_is_the_exact_sum_rounded_once():
    import torch
    rng = np.random.Generator(np.random.Philox(98))
    a = inputs.f32_to_bf16_bits((rng.standard_normal(50000) * 10.0 ** rng.integers(-6, 6, 50000)).astype(np.float32))
    b = inputs.f32_to_bf16_bits((rng.standard_normal(50000) * 10.0 ** rng.integers(-6, 6, 50000)).astype(np.float32))
    ta = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    tb = torch.from_numpy(b.view(np.int16)).view(torch.bfloat16)
    ref = (ta + tb).view(torch.int16).numpy().view(np.uint16)              # library bfloat16 addition
    assert np.array_equal(oracle.bf16_add(a, b), ref)
    # brute force on a few pairs: the nearest bfloat16 to the exact rational sum
    from fractions import Fraction
    for i in range(40):
        exact = Fraction(float(oracle.bf16_bits_to_f64(a[i:i + 1])[0])) + Fraction(float(oracle.bf16_bits_to_f64(b[i:i + 1])[0]))
        got = int(oracle.bf16_add(a[i:i + 1], b[i:i + 1])[0])
        gv = Fraction(float(oracle.bf16_bits_to_f64(np.array([got], np.uint16))[0]))
        for nb in (got - 1, got + 1):                                      # neighbours in the bit pattern order
            nv = Fraction(float(oracle.bf16_bits_to_f64(np.array([nb & 0xFFFF], np.uint16))[0]))
            assert abs(gv - exact) <= abs(nv - exact)


def test_sums_in_bf16_and_fp64_follow_the_fold_order():
    import torch
    k, n = 5, 3000
    parts32 = [inputs.uniform_pm1((n,), 300 + i) for i in range(k)]
    # bfloat16: left fold with library additions
    bits = [inputs.f32_to_bf16_bits(p) for p in parts32]
    acc = torch.from_numpy(bits[0].view(np.int16)).view(torch.bfloat16)
    for b in bits[1:]:
        acc = acc + torch.from_numpy(b.view(np.int16)).view(torch.bfloat16)
    assert np.array_equal(oracle.sumreduce_fwd(bits, add=oracle.bf16_add), acc.view(torch.int16).numpy().view(np.uint16))
    assert all(np.array_equal(o, oracle.sumreduce_fwd(bits, add=oracle.bf16_add)) for o in oracle.allreduce(bits, add=oracle.bf16_add))
    # fp64: a plain Python left fold
    parts64 = [p.astype(np.float64) * (1.0 + 2.0 ** -40 * i) for i, p in enumerate(parts32)]
    ref = [float(parts64[0][e]) for e in range(n)]
    for p in parts64[1:]:
        ref = [r + float(p[e]) for e, r in enumerate(ref)]
    assert oracle.sumreduce_fwd(parts64).tolist() == ref


def test_halo_adjoint_in_bf16_and_fp64_on_integer_data():
    # small integers: every sum is exact in all three types, so they must agree cell by cell
    part = Partition((9, 10), (2, 3), 2, 1)
    y32 = [inputs.integers(part.padded_shape(w), 400 + w) for w in range(part.num_workers)]
    ref = oracle.halo_adj_sequence(part, y32)
    got64 = oracle.halo_adj_sequence(part, [a.astype(np.float64) for a in y32])
    gotbf = oracle.halo_adj_sequence(part, [inputs.f32_to_bf16_bits(a) for a in y32], add=oracle.bf16_add)
    for a, b, c in zip(ref, got64, gotbf):
        assert np.array_equal(a.astype(np.float64), b)
        assert np.array_equal(a.astype(np.float64), oracle.bf16_bits_to_f64(c))


# --------------------------------------------------------------------------
# Periodic dimensions of the halo exchange
# --------------------------------------------------------------------------

PERIODIC_CASES = [
    # global shape, partition, hlo, hhi, periodic
    ((7,), (1,), 2, 3, (True,)),                       # one worker: its own neighbour on both sides
    ((9,), (2,), 2, 1, (True,)),                       # two workers: the same neighbour low and high
    ((10,), (3,), [[1, 2, 0]], [[2, 0, 1]], (True,)),
    ((6, 8), (2, 2), 1, 2, (True, False)),
    ((6, 8), (1, 3), (2, 1), (1, 2), (True, True)),
    ((4, 5, 6), (2, 1, 2), 1, 1, (False, True, True)),
]


@pytest.mark.parametrize("case", PERIODIC_CASES, ids=[str(c[0]) + str(c[1]) + str(c[4]) for c in PERIODIC_CASES])
def test_periodic_halo_matches_wrapped_padding_and_has_transpose_adjoint(case):
    gs, ps, hlo, hhi, per = case
    part = Partition(gs, ps, hlo, hhi, per)
    x = _random_shards(part, 9)                      # garbage in the ghosts
    a = oracle.halo_fwd_definition(part, x)
    b = oracle.halo_fwd_sequence(part, x)
    g = oracle.assemble_global(part, x)
    # library pin: a window of the global tensor padded by wrapping (periodic dimensions) or with zeros
    mlo = [max(part.hlo[k]) for k in range(part.rank)]
    mhi = [max(part.hhi[k]) for k in range(part.rank)]
    gp = g
    for k in range(part.rank):
        width = [(0, 0)] * part.rank
        width[k] = (mlo[k], mhi[k])
        gp = np.pad(gp, width, mode="wrap") if per[k] else np.pad(gp, width)
    for w in range(part.num_workers):
        assert a[w].tobytes() == b[w].tobytes()
        lo, _ = part.widths(w)
        st, pshape = part.bulk_start(w), part.padded_shape(w)
        win = tuple(slice(st[k] - lo[k] + mlo[k], st[k] - lo[k] + mlo[k] + pshape[k]) for k in range(part.rank))
        assert np.array_equal(a[w], gp[win])
    # operator matrices: 0/1 entries, one per ghost row; the adjoint sequence is the exact transpose
    M = _operator_matrix(part, oracle.halo_fwd_sequence)
    assert set(np.unique(M)) <= {0.0, 1.0} and np.all(M.sum(axis=1) <= 1)
    if all(per):
        assert np.all(M.sum(axis=1) == 1)                  # no zero padding anywhere
    assert np.array_equal(_operator_matrix(part, oracle.halo_adj_sequence), M.T)
    y = _random_shards(part, 10)
    assert oracle.adjoint_test_ratio(b, y, x, oracle.halo_adj_sequence(part, y)) < 1e-6


# --------------------------------------------------------------------------
# Generalized convolution: channel partitions P_co x P_ci besides the feature space
# --------------------------------------------------------------------------

CONVG_CASES = [
    # N, n_ci, n_co, H, W, P_ci, P_co, P_0, P_1, k
    (2, 4, 6, 9, 10, 2, 3, 2, 2, 3),
    (1, 5, 3, 8, 7, 2, 2, 1, 2, 5),        # uneven channel blocks (3 + 2, 2 + 1)
    (1, 3, 4, 6, 6, 1, 1, 1, 1, 3),
    (2, 2, 2, 12, 9, 2, 1, 3, 1, 5),
]


def _convg_problem(case, seed):
    N, nci, nco, H, W, pci, pco, p0, p1, k = case
    h = k // 2
    xpart = Partition((N, nci, H, W), (1, pci, p0, p1), (0, 0, h, h), (0, 0, h, h))
    ypart = Partition((N, nco, H, W), (1, pco, p0, p1))
    xg = inputs.normal((N, nci, H, W), seed)
    wg = inputs.normal((nco, nci, k, k), seed + 1, 0.2)
    bg = inputs.normal((nco,), seed + 2)
    cs_i, cz_i = oracle.balanced_split(nco, pco)
    cs_j, cz_j = oracle.balanced_split(nci, pci)
    wb = [wg[cs_i[i]:cs_i[i] + cz_i[i], cs_j[j]:cs_j[j] + cz_j[j]] for i in range(pco) for j in range(pci)]
    bb = [bg[cs_i[i]:cs_i[i] + cz_i[i]] for i in range(pco)]
    return xpart, ypart, xg, wg, bg, wb, bb


@pytest.mark.parametrize("case", CONVG_CASES, ids=[str(c) for c in CONVG_CASES])
def test_generalized_conv_matches_the_sequential_layer_and_its_autograd(case):
    import torch
    xpart, ypart, xg, wg, bg, wb, bb = _convg_problem(case, 101)
    nco, pco, k = case[2], case[6], case[9]
    x = oracle.scatter_global(xpart, xg, fill=lambda wk: np.full(xpart.padded_shape(wk), 3.0))     # garbage ghosts
    y = oracle.assemble_global(ypart, oracle.convg_fwd(xpart, nco, pco, x, wb, bb))
    X = torch.tensor(xg, dtype=torch.float64, requires_grad=True)
    Y = torch.nn.functional.conv2d(X, torch.tensor(wg, dtype=torch.float64), torch.tensor(bg, dtype=torch.float64), padding=k // 2)
    assert np.allclose(y, Y.detach().numpy(), rtol=1e-6, atol=1e-5)
    dyg = inputs.normal(Y.shape, 105)
    Y.backward(torch.tensor(dyg, dtype=torch.float64))
    dx = oracle.convg_adj(xpart, nco, pco, oracle.scatter_global(ypart, dyg), wb)
    assert np.allclose(oracle.assemble_global(xpart, dx), X.grad.numpy(), rtol=1e-6, atol=1e-5)
    for wk in range(xpart.num_workers):
        mask = np.ones(xpart.padded_shape(wk), dtype=bool)
        mask[xpart.bulk_slices(wk)] = False
        assert not dx[wk][mask].any()
    # dot test of the pair (no bias)
    y0 = oracle.convg_fwd(xpart, nco, pco, oracle.scatter_global(xpart, xg), wb)
    assert oracle.adjoint_test_ratio(y0, oracle.scatter_global(ypart, dyg), oracle.scatter_global(xpart, xg), dx) < 1e-6


def test_generalized_conv_reduces_to_the_depthwise_layer_on_diagonal_weights():
    # weights that couple channel c only to itself: the layer is the depthwise one, which is pinned separately
    N, C, H, W, k = 1, 4, 10, 8, 5
    xpart = Partition((N, C, H, W), (1, 2, 2, 1), (0, 0, 2, 2), (0, 0, 2, 2))
    dpart = Partition((N, C, H, W), (1, 1, 2, 1), (0, 0, 2, 2), (0, 0, 2, 2))
    xg = inputs.normal((N, C, H, W), 111)
    wd = inputs.normal((C, k, k), 112, 0.2)
    wg = np.zeros((C, C, k, k), np.float32)
    for c in range(C):
        wg[c, c] = wd[c]
    wb = [wg[2 * i:2 * i + 2, 2 * j:2 * j + 2] for i in range(2) for j in range(2)]
    y = oracle.assemble_global(Partition((N, C, H, W), (1, 2, 2, 1)), oracle.convg_fwd(xpart, C, 2, oracle.scatter_global(xpart, xg), wb))
    yd = oracle.assemble_global(Partition((N, C, H, W), (1, 1, 2, 1)), oracle.conv_fwd(dpart, oracle.scatter_global(dpart, xg), wd))
    assert np.allclose(y, yd, rtol=0, atol=2e-6)


@pytest.mark.parametrize("case", CONVG_CASES, ids=[str(c) for c in CONVG_CASES])
def test_generalized_conv_param_gradients_against_autograd_and_dot_test(case):
    import torch
    xpart, ypart, xg, wg, bg, wb, bb = _convg_problem(case, 121)
    N, nci, nco, H, W, pci, pco, p0, p1, k = case
    dyg = inputs.normal((N, nco, H, W), 125)
    x = oracle.scatter_global(xpart, xg, fill=lambda wk: np.full(xpart.padded_shape(wk), 4.0))     # garbage ghosts
    dy = oracle.scatter_global(ypart, dyg)
    dw, db = oracle.convg_adj_params(xpart, nco, pco, x, dy, k, k)
    Wt = torch.tensor(wg, dtype=torch.float64, requires_grad=True)
    Bt = torch.tensor(bg, dtype=torch.float64, requires_grad=True)
    Y = torch.nn.functional.conv2d(torch.tensor(xg, dtype=torch.float64), Wt, Bt, padding=k // 2)
    Y.backward(torch.tensor(dyg, dtype=torch.float64))
    cs_i, cz_i = oracle.balanced_split(nco, pco)
    cs_j, cz_j = oracle.balanced_split(nci, pci)
    for i in range(pco):
        for j in range(pci):
            ref = Wt.grad.numpy()[cs_i[i]:cs_i[i] + cz_i[i], cs_j[j]:cs_j[j] + cz_j[j]]
            assert np.allclose(dw[i * pci + j], ref, rtol=1e-6, atol=1e-5)
        assert np.allclose(db[i], Bt.grad.numpy()[cs_i[i]:cs_i[i] + cz_i[i]], rtol=1e-6, atol=1e-5)
    # parameter-space dot test through the (separately pinned) forward oracle: <Conv(w, b; x), dy> = <w, dw> + <b, db>
    y = oracle.convg_fwd(xpart, nco, pco, x, wb, bb)
    assert oracle.adjoint_test_ratio(y, dy, list(wb) + list(bb), list(dw) + list(db)) < 1e-6
