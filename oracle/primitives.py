"""Oracle data-movement primitives: B, R, H, H* and the adjoint test.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Shards are numpy arrays
of the padded shape `bulk + hlo + hhi`, listed in worker order.  Operators that
the paper describes as in-place (the halo exchange, Section 3) return new arrays
here so that the caller keeps its input.
"""

import numpy as np

from .partition import Partition


# --------------------------------------------------------------------------
# Broadcast and sum-reduce (Section 3, "Broadcast", "Sum-reduce and all-reduce")
# --------------------------------------------------------------------------

def broadcast_fwd(src, k):
    """B_{a->{k}}: k copies of one realisation (the broadcast equation)."""
    return [np.array(src, copy=True) for _ in range(k)]


def round_to_bf16_bits(x):
    """fp64 values -> bfloat16 bit patterns (uint16), one rounding to nearest, ties to even.

    bfloat16 has 8 significant bits and the exponent range of fp32: the spacing of
    representable values at |x| in [2^(e-1), 2^e) is 2^(e-8), and never finer than
    2^-133 (subnormals).  The value is divided by its spacing, rounded to the nearest
    integer with ties to even (numpy.rint), and scaled back; the result is exactly
    representable in fp32, whose upper 16 bits are the answer.  Values beyond the
    largest finite bfloat16 are not handled (the operators here never produce them).
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                                  # |x| = m * 2^e with m in [0.5, 1)
    q = np.maximum(e - 8, -133).astype(np.int64)
    r = np.ldexp(np.rint(np.ldexp(x, -q)), q)
    return (r.astype(np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits):
    """bfloat16 bit patterns (uint16) -> the same values in fp64 (exact)."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def bf16_add(a_bits, b_bits):
    """a + b in bfloat16 arithmetic on bit patterns: the exact sum, rounded once.

    The sum of two bfloat16 values is exact in fp64 unless their exponents differ by
    more than 44, in which case the fp64 sum already rounds to the larger operand, as
    the bfloat16 result does.
    """
    return round_to_bf16_bits(bf16_bits_to_f64(a_bits) + bf16_bits_to_f64(b_bits))


def sumreduce_fwd(parts, add=None):
    """R_{{k}->a} = B*: sum of the k realisations (adjoint-of-broadcast equation).

    The sum is taken in worker order 0, 1, ..., k-1 in the arithmetic of the
    inputs: acc = y_0; acc = acc + y_i.  Starting from y_0 makes k = 1 an exact
    copy.  `add` replaces the addition of the arrays' own type (bf16_add for
    bfloat16 bit patterns).
    """
    acc = np.array(parts[0], copy=True)
    for i in range(1, len(parts)):
        acc = acc + parts[i] if add is None else add(acc, parts[i])
    return acc


def broadcast_adj(parts):
    """B* = R (Section 3: the adjoint of the broadcast is a sum-reduction)."""
    return sumreduce_fwd(parts)


def sumreduce_adj(src, k):
    """R* = B (Section 3)."""
    return broadcast_fwd(src, k)


# --------------------------------------------------------------------------
# Global <-> shard helpers (bookkeeping, no arithmetic)
# --------------------------------------------------------------------------

def scatter_global(part: Partition, g, fill=None, dtype=None):
    """Cut a global array into padded shards; bulk = the owner's block.

    Ghost cells are filled with `fill` (a callable worker -> array of padded
    shape, or None for zeros) so tests can plant garbage there.
    """
    g = np.asarray(g)
    dtype = dtype or g.dtype
    shards = []
    for w in range(part.num_workers):
        if fill is None:
            a = np.zeros(part.padded_shape(w), dtype=dtype)
        else:
            a = np.array(fill(w), dtype=dtype, copy=True)
            assert a.shape == part.padded_shape(w)
        st, sh = part.bulk_start(w), part.bulk_shape(w)
        src = tuple(slice(st[k], st[k] + sh[k]) for k in range(part.rank))
        a[part.bulk_slices(w)] = g[src]
        shards.append(a)
    return shards


def assemble_global(part: Partition, shards):
    """Put every shard's bulk back at its place in the global array."""
    g = np.zeros(part.global_shape, dtype=shards[0].dtype)
    for w in range(part.num_workers):
        st, sh = part.bulk_start(w), part.bulk_shape(w)
        dst = tuple(slice(st[k], st[k] + sh[k]) for k in range(part.rank))
        g[dst] = shards[w][part.bulk_slices(w)]
    return g


# --------------------------------------------------------------------------
# Halo exchange H (Section 3, "Halo exchange")
# --------------------------------------------------------------------------

def halo_fwd_definition(part: Partition, shards):
    """H by its plain meaning.

    After the exchange every ghost cell of every worker holds a copy of the bulk
    cell, owned by some other worker, that has the same global index (Section 3:
    the halo region "must contain copies of the current data owned by
    neighboring workers").  Ghost cells whose global index falls outside the
    tensor hold +0 (the implicit zero padding of Fig. B1).  The bulk is not
    touched and whatever the ghosts held before is discarded.
    """
    g = assemble_global(part, shards)
    out = []
    for w in range(part.num_workers):
        st = part.bulk_start(w)
        lo, _ = part.widths(w)
        pshape = part.padded_shape(w)
        # global index of padded-local index l is st - lo + l; taken modulo the extent in a periodic
        # dimension, otherwise cells outside the tensor stay zero
        a = g
        keep = []
        for k in range(part.rank):
            idx = np.arange(st[k] - lo[k], st[k] - lo[k] + pshape[k])
            n = part.global_shape[k]
            if part.periodic[k]:
                keep.append(np.ones(pshape[k], dtype=bool))
                idx = idx % n
            else:
                keep.append((idx >= 0) & (idx < n))
                idx = np.clip(idx, 0, n - 1)
            a = np.take(a, idx, axis=k)
        mask = keep[0]
        for k in range(1, part.rank):
            mask = np.multiply.outer(mask, keep[k])
        a = np.where(mask, a, np.zeros((), dtype=a.dtype)).astype(shards[w].dtype)
        a[part.bulk_slices(w)] = shards[w][part.bulk_slices(w)]
        out.append(a)
    return out


def _slab(part, w, k, lo_range, upto_padded):
    """Index tuple of a slab of worker w that spans `lo_range` in dimension k,
    the full padded extent in dimensions < k and the bulk extent in dimensions
    > k (corner data travels with the later dimensions of the nested exchange).
    """
    idx = []
    bs = part.bulk_slices(w)
    for j in range(part.rank):
        if j == k:
            idx.append(slice(lo_range[0], lo_range[1]))
        elif j < k and upto_padded:
            idx.append(slice(None))
        else:
            idx.append(bs[j])
    return tuple(idx)


def _neighbour(part, w, k, step):
    c = list(part.coords(w))
    c[k] += step
    if c[k] < 0 or c[k] >= part.pshape[k]:
        if not part.periodic[k]:
            return None
        c[k] %= part.pshape[k]           # across the seam; the worker itself when it is alone along k
    return part.worker(c)


def halo_fwd_sequence(part: Partition, shards):
    """H as the paper's operator sequence (the two halo-exchange equations).

    For dimension k = 0, 1, ..., d-1 and for every worker: K_S clears the send
    and receive buffers, C_P packs the boundary slab of the bulk into the send
    buffer, C_E copies it into the neighbour's receive buffer, C_U unpacks the
    receive buffer into the ghost slab, K_T clears the buffers again.  A side
    with no neighbour (the tensor's own boundary) gets zeros.
    """
    x = [np.array(s, copy=True) for s in shards]
    for k in range(part.rank):
        recv = {}
        for w in range(part.num_workers):
            lo, hi = part.widths(w)
            b = part.bulk_shape(w)
            for side, step in (("lo", -1), ("hi", +1)):
                n = _neighbour(part, w, k, step)
                width = lo[k] if side == "lo" else hi[k]
                if n is None or width == 0:
                    continue
                nlo, _ = part.widths(n)
                nb = part.bulk_shape(n)
                assert width <= nb[k], "halo reaches beyond the adjacent worker"
                # the neighbour packs the part of its bulk that borders w
                if side == "lo":
                    rng = (nlo[k] + nb[k] - width, nlo[k] + nb[k])
                else:
                    rng = (nlo[k], nlo[k] + width)
                send = np.zeros_like(x[n][_slab(part, n, k, rng, True)])   # K_S
                send[...] = x[n][_slab(part, n, k, rng, True)]             # C_P
                buf = np.zeros_like(send)                                  # K_S
                buf[...] = send                                            # C_E
                recv[(w, side)] = buf
        for w in range(part.num_workers):
            lo, hi = part.widths(w)
            b = part.bulk_shape(w)
            for side in ("lo", "hi"):
                width = lo[k] if side == "lo" else hi[k]
                if width == 0:
                    continue
                rng = (0, lo[k]) if side == "lo" else (lo[k] + b[k], lo[k] + b[k] + hi[k])
                ghost = _slab(part, w, k, rng, True)
                if (w, side) in recv:
                    buf = recv.pop((w, side))
                    # slabs of the two workers must agree in the other dimensions
                    assert buf.shape == x[w][ghost].shape
                    x[w][ghost] = buf                                      # C_U
                else:
                    x[w][ghost] = 0
        # K_T: the buffers go out of scope here
    # Every ghost cell is written exactly once: at the stage of the highest
    # dimension in which it is a ghost index.
    return x


# --------------------------------------------------------------------------
# Adjoint halo exchange H* (Section 3, the H* equation; Appendix B.2)
# --------------------------------------------------------------------------

def halo_adj_sequence(part: Partition, shards, add=None):
    """H* as the paper's reversed operator sequence (`add`: see sumreduce_fwd).

    Ghosts on the tensor's own boundary are cleared (the adjoint of writing a
    zero).  Then for dimension k = d-1 down to 0 and every worker: the ghost
    slab each neighbour holds of this worker's boundary is added into that
    boundary slab of the bulk (C*_U, C*_E, C*_P: "an add operation into the
    bulk tensor"), and the ghost slab is cleared (K*_T / in-place copy adjoint
    C* = K_b S_{b->a}).  When one bulk cell receives from both sides of a
    dimension the low-coordinate neighbour is added first.
    """
    y = [np.array(s, copy=True) for s in shards]
    # exterior ghosts carry nothing back
    for w in range(part.num_workers):
        lo, hi = part.widths(w)
        b = part.bulk_shape(w)
        for k in range(part.rank):
            if _neighbour(part, w, k, -1) is None and lo[k] > 0:
                idx = [slice(None)] * part.rank
                idx[k] = slice(0, lo[k])
                y[w][tuple(idx)] = 0
            if _neighbour(part, w, k, +1) is None and hi[k] > 0:
                idx = [slice(None)] * part.rank
                idx[k] = slice(lo[k] + b[k], lo[k] + b[k] + hi[k])
                y[w][tuple(idx)] = 0
    for k in reversed(range(part.rank)):
        for step in (-1, +1):            # low neighbour first, then high
            for w in range(part.num_workers):
                n = _neighbour(part, w, k, step)
                if n is None:
                    continue
                lo, hi = part.widths(w)
                b = part.bulk_shape(w)
                nlo, nhi = part.widths(n)
                nb = part.bulk_shape(n)
                if step == -1:
                    width = nhi[k]       # n's high ghost mirrors w's low boundary
                    if width == 0:
                        continue
                    mine = (lo[k], lo[k] + width)
                    theirs = (nlo[k] + nb[k], nlo[k] + nb[k] + width)
                else:
                    width = nlo[k]       # n's low ghost mirrors w's high boundary
                    if width == 0:
                        continue
                    mine = (lo[k] + b[k] - width, lo[k] + b[k])
                    theirs = (0, width)
                assert width <= b[k], "halo reaches beyond the adjacent worker"
                dst = _slab(part, w, k, mine, True)
                src = _slab(part, n, k, theirs, True)
                y[w][dst] = y[w][dst] + y[n][src] if add is None else add(y[w][dst], y[n][src])
                y[n][src] = 0
    return y


# --------------------------------------------------------------------------
# Adjoint (dot-product) test (Section 3, "Implementation")
# --------------------------------------------------------------------------

def _dot(a_list, b_list):
    s = 0.0
    for a, b in zip(a_list, b_list):
        s += float(np.dot(np.asarray(a, dtype=np.float64).ravel(),
                          np.asarray(b, dtype=np.float64).ravel()))
    return s


def adjoint_test_ratio(Fx, y, x, Fsy):
    """|<Fx,y> - <x,F*y>| / max(||Fx|| ||y||, ||x|| ||F*y||)  (the adjoint test).

    Arguments are lists of arrays (one per realisation); inner products and
    norms are Euclidean over every cell, accumulated in fp64.
    """
    lhs = _dot(Fx, y)
    rhs = _dot(x, Fsy)
    nFx = np.sqrt(_dot(Fx, Fx))
    ny = np.sqrt(_dot(y, y))
    nx = np.sqrt(_dot(x, x))
    nFsy = np.sqrt(_dot(Fsy, Fsy))
    den = max(nFx * ny, nx * nFsy)
    if den == 0.0:
        return 0.0
    return abs(lhs - rhs) / den


# --------------------------------------------------------------------------
# Generalized all-to-all (repartition), scatter / gather, all-reduce
# (Section 3, "Scatter and Gather", "Sum-reduce and all-reduce", "Generalized all-to-all")
# --------------------------------------------------------------------------

def repartition_fwd(src_part: Partition, dst_part: Partition, shards):
    """Generalized all-to-all: the same tensor, re-cut from one partition to another.

    Every cell of the tensor is moved from the worker that owns it in `src_part`
    to the worker that owns it in `dst_part` (a block permutation whose blocks are
    send-receive copies).  Written as its plain meaning: put the source blocks
    together, cut along the destination partition.  Both partitions carry no ghosts.
    A source partition of a single worker gives the scatter, a destination
    partition of a single worker the gather.
    """
    assert src_part.global_shape == dst_part.global_shape
    return scatter_global(dst_part, assemble_global(src_part, shards))


def repartition_adj(src_part: Partition, dst_part: Partition, dy_shards):
    """Adjoint of the generalized all-to-all.

    The operator is a permutation of cells (every copy is a move), so its adjoint
    is its inverse: the all-to-all back from `dst_part` to `src_part`.
    """
    return scatter_global(src_part, assemble_global(dst_part, dy_shards))


def allreduce(parts, add=None):
    """All-reduce = broadcast after sum-reduce (self-adjoint): every worker ends up with
    the fixed-order sum of all k realisations."""
    return broadcast_fwd(sumreduce_fwd(parts, add), len(parts))


# --------------------------------------------------------------------------
# Partition broadcast / sum-reduce along partition dimensions
# (Section 4, "Sparse layers": the forward and adjoint convolution algorithms and the two
# footnotes on broadcasting along partitions; "Dense layers": the affine algorithms)
# --------------------------------------------------------------------------

def _partition_sources(src_pshape, dst_pshape):
    """For every worker of the destination partition (row-major id) the worker of the source
    partition whose realisation it receives.

    The rule is NumPy's broadcasting rule applied to the two partition shapes, from source to
    destination only: along a partition dimension where the source has one worker and the
    destination has several, that one worker's realisation goes to all of them; along every other
    dimension both partitions have the same number of workers and coordinates correspond.
    """
    src_pshape, dst_pshape = tuple(int(v) for v in src_pshape), tuple(int(v) for v in dst_pshape)
    assert len(src_pshape) == len(dst_pshape)
    for a, b in zip(src_pshape, dst_pshape):
        assert a == b or a == 1, "a partition dimension broadcasts only from one worker"
    out = []
    for w in range(int(np.prod(dst_pshape))):
        coords, rest = [], w
        for p in reversed(dst_pshape):
            coords.append(rest % p)
            rest //= p
        coords.reverse()
        src = 0
        for k, c in enumerate(coords):
            src = src * src_pshape[k] + (c if src_pshape[k] > 1 else 0)
        out.append(src)
    return out


def partition_broadcast_fwd(src_pshape, dst_pshape, shards):
    """B_{{P_x} -> {P_w}}: every worker of the destination partition gets a copy of the realisation
    held by its source worker (x^ <- B x in the forward algorithms; dy^ <- B dy in the adjoint ones)."""
    src_of = _partition_sources(src_pshape, dst_pshape)
    assert len(shards) == int(np.prod(src_pshape))
    return [np.array(shards[j], copy=True) for j in src_of]


def partition_broadcast_adj(src_pshape, dst_pshape, dy_shards, add=None):
    """R_{{P_w} -> {P_x}} = B*: every worker of the smaller partition gets the sum of the realisations
    of the workers that its own realisation was (or would be) broadcast to, taken in the order of
    their worker ids, in the arithmetic of the inputs (y <- R y^ in the forward algorithms; dx <- R dx^
    in the adjoint ones)."""
    src_of = _partition_sources(src_pshape, dst_pshape)
    assert len(dy_shards) == len(src_of)
    out = []
    for j in range(int(np.prod(src_pshape))):
        out.append(sumreduce_fwd([dy_shards[w] for w in range(len(src_of)) if src_of[w] == j], add))
    return out
