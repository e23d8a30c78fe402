"""Host-side replay of the row plan of H and of the row ends of H* (CPU, no kernel launched).

The row-plan kernels derive every address from one small record per (dimension, worker coordinate).  This test
fetches those records from the library (include/distdl_selftest.h), replays the kernels' index arithmetic block
by block in Python -- the same row classes, divisions by multiply-and-shift, neighbour lookups and staging
slots -- checks that every unit it touches lies inside its worker's array, that the units handled are exactly
the ones the kernel is responsible for, each once, and that their values equal the oracle's H / H* bit for bit.
"""

import numpy as np
import pytest

import oracle
import paper_2006_03108_b200 as distdl
from paper_2006_03108_b200 import inputs


class Rec:
    def __init__(self, w):
        u = [v & 0xFFFFFFFF for v in w]
        (self.n, self.hlo, self.b, self.lo_c, self.hi_c, self.lo_shift, self.hi_shift, self.rlo, self.rhi) = w[:9]
        self.magic_n, self.magic_b, self.magic_g, self.magic_bi, self.magic_rr = u[9:14]
        sh = u[14]
        self.shift_n, self.shift_b, self.shift_g, self.shift_bi, self.shift_rr = [(sh >> (6 * i)) & 63 for i in range(5)]


class Header:
    def __init__(self, h):
        self.rank, self.nw = h[0], h[1]
        self.pshape, self.base, self.wstride = h[2:7], h[7:12], h[12:17]
        self.nrec, self.nlines = h[17], h[18]
        self.rows, self.tiles, self.group = h[19:21], h[21:23], h[23:25]
        self.ngroups = h[25]


def fdiv(x, magic, shift, e):
    assert 0 <= x < 2 ** 31
    q = ((x * magic) >> 32) >> shift if magic else x
    assert q == x // max(e, 1), (x, e)
    return q


def blocks(H):
    per = sum(H.group)
    for blk in range(H.ngroups * per):
        group, ing = divmod(blk, per)
        kind = 0
        if ing >= H.group[0]:
            ing -= H.group[0]
            kind = 1
        yield kind, group * H.group[kind] + ing


def worker(H, dims, w):
    c = []
    for k in range(H.rank):
        c.append(w // H.wstride[k])
        w -= c[k] * H.wstride[k]
    return c, [dims[H.base[k] + c[k]] for k in range(H.rank)]


def ghost_rows(H, dims, src, out, written, s, t):
    d = H.rank
    c, e = worker(H, dims, s)
    cls = []
    for j in range(d - 1):
        r = e[j].n - e[j].b
        for k in range(d - 1):
            if k != j:
                r *= e[k].b if k < j else e[k].n
        cls.append(r)
    total, row0 = sum(cls), t * H.rows[0]
    if row0 >= total:
        return
    nrows = min(H.rows[0], total - row0)
    assert nrows <= 256
    ex, nx = e[d - 1], e[d - 1].n
    for rl in range(nrows):
        idx, j = row0 + rl, 0
        while j < d - 2 and idx >= cls[j]:
            idx -= cls[j]
            j += 1
        dst_lin = src_lin = 0
        dp = sp = 1
        outer_w, zero = 0, False
        for k in range(d - 2, -1, -1):
            f = e[k]
            if k == 0:
                coord = idx
            else:
                ext, mg, sf = ((f.n, f.magic_n, f.shift_n) if k > j else
                               (f.n - f.b, f.magic_g, f.shift_g) if k == j else (f.b, f.magic_b, f.shift_b))
                q = fdiv(idx, mg, sf, ext)
                coord, idx = idx - q * ext, q
            i = coord if k > j else ((coord if coord < f.hlo else coord + f.b) if k == j else f.hlo + coord)
            assert 0 <= i < f.n
            nc, si = c[k], i
            if i < f.hlo:
                nc, si = f.lo_c, i + f.lo_shift
            elif i >= f.hlo + f.b:
                nc, si = f.hi_c, i + f.hi_shift
            dst_lin += i * dp
            dp *= f.n
            if nc < 0:
                zero = True
            else:
                src_lin += si * sp
                sp *= dims[H.base[k] + nc].n
                outer_w += nc * H.wstride[k]
        for col in range(nx):
            assert fdiv(rl * nx + col, ex.magic_n, ex.shift_n, nx) == rl
            reg = 0 if col < ex.hlo else (1 if col < ex.hlo + ex.b else 2)
            ncx = (ex.lo_c, c[d - 1], ex.hi_c)[reg]
            shift = (ex.lo_shift, 0, ex.hi_shift)[reg]
            doff = dst_lin * nx + col
            assert 0 <= doff < len(out[s])
            if zero or ncx < 0:
                out[s][doff] = 0
                written[s][doff] += 1
            else:
                w = outer_w + ncx * H.wstride[d - 1]
                soff = src_lin * dims[H.base[d - 1] + ncx].n + shift + col
                assert 0 <= w < H.nw and 0 <= soff < len(src[w])
                out[s][doff] = src[w][soff]
                written[s][doff] += 1


def line_rows(H, e, inner, row0, nrows):
    d, rowlin = H.rank, []
    for rl in range(nrows):
        idx, lin, pitch = row0 + rl, 0, 1
        for k in range(d - 2, -1, -1):
            f = e[k]
            coord = idx
            ext = f.b - f.rlo - f.rhi if inner else f.b
            if k > 0:
                q = fdiv(idx, f.magic_bi, f.shift_bi, ext) if inner else fdiv(idx, f.magic_b, f.shift_b, ext)
                coord, idx = idx - q * ext, q
            assert 0 <= coord < ext
            lin += (f.hlo + (f.rlo if inner else 0) + coord) * pitch
            pitch *= f.n
        rowlin.append(lin)
    return rowlin


def replay_forward(hdr, recs, units):
    H, dims = Header(hdr), [Rec(r) for r in recs]
    d = H.rank
    out = [u.copy() for u in units]
    written = [np.zeros(len(u), dtype=np.int32) for u in units]
    for kind, tile in blocks(H):
        if kind == 0:
            s, t = divmod(tile, H.tiles[0])
            if s < H.nw:
                ghost_rows(H, dims, units, out, written, s, t)
            continue
        assert kind == 1
        line, t = divmod(tile, H.tiles[1])
        if line >= H.nlines:
            continue
        px = H.pshape[d - 1]
        first = line * px
        _, e = worker(H, dims, first)
        total = int(np.prod([e[k].b for k in range(d - 1)])) if d > 1 else 1
        row0 = t * H.rows[1]
        if row0 >= total:
            continue
        nrows = min(H.rows[1], total - row0)
        assert nrows <= 128
        xd = dims[H.base[d - 1]:H.base[d - 1] + px]
        cum_g, cum_p = [0], [0]
        for a in range(px):
            cum_g.append(cum_g[-1] + xd[a].n - xd[a].b)
            cum_p.append(cum_p[-1] + xd[a].rlo + xd[a].rhi)
        rowlin = line_rows(H, e, False, row0, nrows)
        GC, PC = cum_g[px], cum_p[px]
        assert nrows * GC <= 1024
        slots = {}
        for q in range(nrows * PC):
            a = 0
            while q >= nrows * cum_p[a + 1]:
                a += 1
            qa = q - nrows * cum_p[a]
            f = xd[a]
            rl, piece = divmod(qa, f.rlo + f.rhi)
            if piece < f.rlo:
                g = xd[f.lo_c]
                col = f.hlo + piece
                slot = nrows * cum_g[f.lo_c] + rl * (g.n - g.b) + g.hlo + piece
            else:
                g = xd[f.hi_c]
                u = piece - f.rlo
                col = f.hlo + f.b - f.rhi + u
                slot = nrows * cum_g[f.hi_c] + rl * (g.n - g.b) + u
            assert f.hlo <= col < f.hlo + f.b and 0 <= slot < nrows * GC and slot not in slots
            off = rowlin[rl] * f.n + col
            assert 0 <= off < len(units[first + a])
            slots[slot] = units[first + a][off].copy()
        for q in range(nrows * GC):
            a = 0
            while q >= nrows * cum_g[a + 1]:
                a += 1
            qa = q - nrows * cum_g[a]
            f = xd[a]
            rl, g = divmod(qa, f.n - f.b)
            low = g < f.hlo
            has = (f.lo_c >= 0) if low else (f.hi_c >= 0)
            col = g if low else g + f.b
            off = rowlin[rl] * f.n + col
            assert 0 <= off < len(out[first + a])
            out[first + a][off] = slots[nrows * cum_g[a] + qa] if has else 0
            written[first + a][off] += 1
    return out, written


def replay_adjoint_row_ends(hdr, recs, units, add):
    """The launch that handles the row ends of H*: in place, every unit read once and written once."""
    H, dims = Header(hdr), [Rec(r) for r in recs]
    d = H.rank
    mem = [u.copy() for u in units]
    touched = [np.zeros(len(u), dtype=np.int32) for u in units]
    for kind, tile in blocks(H):
        assert kind == 1
        line, t = divmod(tile, H.tiles[1])
        if line >= H.nlines:
            continue
        px = H.pshape[d - 1]
        first = line * px
        _, e = worker(H, dims, first)
        total = int(np.prod([e[k].b - e[k].rlo - e[k].rhi for k in range(d - 1)])) if d > 1 else 1
        row0 = t * H.rows[1]
        if row0 >= total:
            continue
        nrows = min(H.rows[1], total - row0)
        assert nrows <= 128
        xd = dims[H.base[d - 1]:H.base[d - 1] + px]
        cum_e = [0]
        for a in range(px):
            cum_e.append(cum_e[-1] + xd[a].n - xd[a].b + xd[a].rlo + xd[a].rhi)
        rowlin = line_rows(H, e, True, row0, nrows)
        EC = cum_e[px]
        assert nrows * EC <= 1024
        slots = {}

        def item(q):
            a = 0
            while q >= nrows * cum_e[a + 1]:
                a += 1
            qa = q - nrows * cum_e[a]
            f = xd[a]
            ec, lo_end = f.n - f.b + f.rlo + f.rhi, f.hlo + f.rlo
            rl, u = divmod(qa, ec)
            col = u if u < lo_end else u - lo_end + f.hlo + f.b - f.rhi
            assert 0 <= col < f.n
            return a, f, rl, u, col, lo_end

        for q in range(nrows * EC):
            a, f, rl, u, col, lo_end = item(q)
            ghost = col < f.hlo or col >= f.hlo + f.b
            outside = ghost and (f.lo_c < 0 if col < f.hlo else f.hi_c < 0)
            off = rowlin[rl] * f.n + col
            assert 0 <= off < len(mem[first + a])
            if not outside:
                slots[q] = mem[first + a][off].copy()
        for q in range(nrows * EC):
            a, f, rl, u, col, lo_end = item(q)
            v = 0
            if f.hlo <= col < f.hlo + f.b:
                v = slots[q]
                if u < lo_end:
                    if f.lo_c >= 0:
                        g = xd[f.lo_c]
                        gec = g.n - g.b + g.rlo + g.rhi
                        v = add(v, slots[nrows * cum_e[f.lo_c] + rl * gec + g.hlo + g.rlo + g.rhi + (u - f.hlo)])
                elif f.hi_c >= 0:
                    g = xd[f.hi_c]
                    gec = g.n - g.b + g.rlo + g.rhi
                    v = add(v, slots[nrows * cum_e[f.hi_c] + rl * gec + (u - lo_end)])
            off = rowlin[rl] * f.n + col
            mem[first + a][off] = v
            touched[first + a][off] += 1
    return mem, touched


CASES = [
    # global shape, workers, low widths, high widths, periodic, element type
    ((40,), (2,), 4, 4, None, np.float32),
    ((12, 16), (3, 1), (1, 4), (1, 4), None, np.float32),
    ((13, 48), (3, 2), (1, 4), (2, 8), None, np.float32),
    ((9, 7, 64), (2, 3, 4), [[1, 2], [0, 1, 2], [4, 0, 8, 4]], [[2, 0], [1, 1, 0], [4, 8, 0, 4]], None, np.float32),
    ((10, 10, 72), (3, 2, 3), (1, 2, 4), (2, 1, 4), None, np.float32),
    ((3, 3, 6, 16), (1, 1, 2, 2), (0, 0, 1, 4), (0, 0, 1, 4), None, np.float32),
    ((4, 5, 6, 4, 16), (2, 1, 2, 1, 2), (1, 0, 1, 1, 4), (0, 1, 1, 0, 4), None, np.float32),
    ((64, 48), (4, 4), (2, 0), (2, 0), None, np.float32),
    ((4, 4, 1040), (2, 2, 2), (1, 1, 260), (1, 1, 260), None, np.float32),
    ((16,), (1,), (4,), (8,), (True,), np.float32),
    ((12, 32), (1, 2), (2, 4), (1, 8), (True, True), np.float32),
    ((6, 10, 48), (2, 1, 3), (1, 2, 4), (2, 1, 4), (True, False, True), np.float32),
    ((9, 11, 12), (2, 3, 2), (1, 2, 2), (2, 1, 4), None, np.float64),
    ((7, 48), (2, 3), (2, 8), (1, 8), (False, True), np.uint16),
    ((36, 34, 40), (2, 2, 2), 4, 4, None, np.float32),          # several blocks per worker
    ((6, 6, 8), (3, 3, 2), (1, 1, 4), (1, 1, 0), None, np.float32),     # bulks exactly as wide as the two reaches together
]


def _make(case):
    gs, ps, lo, hi, per, dt = case
    code = {np.float32: distdl.F32, np.float64: distdl.F64, np.uint16: distdl.BF16}[dt]
    rank = len(gs)
    w = lambda h: [h] * rank if isinstance(h, int) else list(h)
    opart = oracle.Partition(gs, ps, lo, hi, per)
    gpart = distdl.Partition(gs, ps, w(lo), w(hi), dtype=code, periodic=per)
    x = []
    for k in range(opart.num_workers):
        a = inputs.uniform_pm1(opart.padded_shape(k), 400 + k)
        a = (a * np.float32(10.0) ** inputs.integers(opart.padded_shape(k), 450 + k, -3, 4)).astype(np.float32)
        x.append(inputs.f32_to_bf16_bits(a) if dt == np.uint16 else a.astype(dt))
    return opart, gpart, x, 16 // np.dtype(dt).itemsize


@pytest.mark.parametrize("case", CASES, ids=[str(c[0]) + str(c[1]) for c in CASES])
def test_row_plan_replay_of_the_forward_kernel_matches_the_oracle(case):
    opart, gpart, x, per_unit = _make(case)
    assert gpart.uses_row_plan()
    hdr, recs = distdl.selftest_row_plan(gpart)
    got, written = replay_forward(hdr, recs, [a.reshape(-1, per_unit) for a in x])
    ref = oracle.halo_fwd_definition(opart, x)
    for k in range(opart.num_workers):
        assert got[k].reshape(x[k].shape).tobytes() == ref[k].tobytes(), "worker %d" % k
        ghost = np.ones(x[k].shape, dtype=bool)
        ghost[opart.bulk_slices(k)] = False
        # every ghost unit written exactly once, no bulk unit written
        assert np.array_equal(written[k], ghost.reshape(-1, per_unit).all(axis=1).astype(np.int32))


def _row_end_units(opart, k, per_unit):
    """The 16-byte units of worker k that the row-end launch of H* owns: in the bulk rows out of every outer
    neighbour's reach, the ghost units at both ends and the bulk units within reach of the neighbours along the row."""
    rank = opart.rank
    c = opart.coords(k)
    lo, hi = opart.widths(k)
    b = opart.bulk_shape(k)

    def reach(dim):
        p, per = opart.pshape[dim], opart.periodic[dim]
        rl = opart.hhi[dim][(c[dim] - 1) % p] if (c[dim] > 0 or per) else 0
        rh = opart.hlo[dim][(c[dim] + 1) % p] if (c[dim] + 1 < p or per) else 0
        return rl, rh
    mask = np.zeros(opart.padded_shape(k), dtype=bool)
    rows = tuple(slice(lo[dim] + reach(dim)[0], lo[dim] + b[dim] - reach(dim)[1]) for dim in range(rank - 1))
    rl, rh = reach(rank - 1)
    x = rank - 1
    mask[rows + (slice(0, lo[x] + rl),)] = True
    mask[rows + (slice(lo[x] + b[x] - rh, lo[x] + b[x] + hi[x]),)] = True
    return mask.reshape(-1, per_unit).all(axis=1)


@pytest.mark.parametrize("case", CASES, ids=[str(c[0]) + str(c[1]) for c in CASES])
def test_row_plan_replay_of_the_row_ends_of_the_adjoint_matches_the_oracle(case):
    opart, gpart, x, per_unit = _make(case)
    if case[0] in ((9, 7, 64), (12, 16), (64, 48), (6, 10, 48)):
        # a bulk of 2 cells whose neighbours reach 1 and 2 cells into it; one worker along the rows; no ghosts along
        # the rows; no row out of reach of the (periodic) neighbours in dimension 0: the box plan does all of H*
        assert not gpart.uses_row_plan(adjoint=True)
        return
    assert gpart.uses_row_plan(adjoint=True)
    hdr, recs = distdl.selftest_row_plan(gpart, adjoint=True)
    assert Header(hdr).group[0] == 0
    if case[5] == np.uint16:
        add = lambda a, b: oracle.bf16_add(a, b)
        ref = oracle.halo_adj_sequence(opart, x, add=oracle.bf16_add)
    else:
        add = lambda a, b: a + b
        ref = oracle.halo_adj_sequence(opart, x)
    got, touched = replay_adjoint_row_ends(hdr, recs, [a.reshape(-1, per_unit) for a in x], add)
    for k in range(opart.num_workers):
        own = _row_end_units(opart, k, per_unit)
        assert np.array_equal(touched[k], own.astype(np.int32)), "worker %d: units handled" % k
        want = ref[k].reshape(-1, per_unit)
        assert got[k][own].tobytes() == want[own].tobytes(), "worker %d: values" % k
        assert got[k][~own].tobytes() == x[k].reshape(-1, per_unit)[~own].tobytes()      # nothing else is touched


def test_geometries_outside_the_row_plan():
    for gs, ps, lo, hi in [((11,), (3,), (2,), (2,)), ((67, 61, 68), (3, 2, 2), (2, 4, 4), (3, 4, 4)), ((256, 256), (2, 2), (1, 1), (1, 1))]:
        assert not distdl.Partition(gs, ps, lo, hi).uses_row_plan()
    thin = distdl.Partition((6, 32), (3, 2), (2, 4), (2, 4))      # the middle worker's bulk is thinner than the two reaches
    assert thin.uses_row_plan() and not thin.uses_row_plan(adjoint=True)
