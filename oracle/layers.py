"""Oracle distributed layers: depthwise convolution, pooling and affine (Section 4).

TEST INFRASTRUCTURE ONLY (see the package docstring).

The paper's experiment rests on one principle: a distributed layer gives the
same result as the sequential layer applied to the unpartitioned tensor
(Section 5).  The convolution oracle is therefore the sequential layer written
out on the global tensor; the affine oracle follows the three steps of the
forward / adjoint affine algorithms literally (broadcast, local contraction,
sum-reduce in worker order).
"""

import numpy as np

from .partition import Partition
from .primitives import (
    bf16_bits_to_f64,
    assemble_global,
    scatter_global,
    halo_adj_sequence,
    broadcast_fwd,
    sumreduce_fwd,
)


# --------------------------------------------------------------------------
# Distributed depthwise convolution (Section 4, "Sparse layers": forward /
# adjoint convolution algorithms, feature-space-only partition)
# --------------------------------------------------------------------------

def _check_conv_partition(part: Partition, kh, kw):
    assert part.rank == 4 and part.pshape[0] == 1 and part.pshape[1] == 1
    assert kh % 2 == 1 and kw % 2 == 1


def conv_fwd(part: Partition, x_shards, w, bias=None):
    """y = Conv(w, b; H x) for a depthwise, centred, stride-1 kernel.

    Forward convolution algorithm with the tensor partitioned over the feature
    space only, where the broadcasts and reductions drop out (closing remark of
    the convolution paragraph).  Written as the sequential layer on the global
    tensor: y[n,c,i,j] = b[c] + sum_{a,b} w[c,a,b] * x[n,c,i+a-ph,j+b-pw] with
    x = 0 outside the tensor ("Conv" is the framework's layer, i.e. a
    cross-correlation).  Accumulated in fp64, rounded once to fp32.
    Returns bulk-shaped fp32 output shards (no ghosts).
    """
    w = np.asarray(w, dtype=np.float64)
    C, kh, kw = w.shape
    _check_conv_partition(part, kh, kw)
    ph, pw = kh // 2, kw // 2
    xg = assemble_global(part, x_shards).astype(np.float64)
    N, Cx, Hg, Wg = xg.shape
    assert Cx == C
    xp = np.zeros((N, C, Hg + 2 * ph, Wg + 2 * pw), dtype=np.float64)
    xp[:, :, ph:ph + Hg, pw:pw + Wg] = xg
    acc = np.zeros((N, C, Hg, Wg), dtype=np.float64)
    for a in range(kh):
        for b in range(kw):
            acc += w[None, :, a, b, None, None] * xp[:, :, a:a + Hg, b:b + Wg]
    if bias is not None:
        acc += np.asarray(bias, dtype=np.float64)[None, :, None, None]
    yg = acc.astype(np.float32)
    ypart = Partition(part.global_shape, part.pshape, 0, 0)
    return scatter_global(ypart, yg)


def conv_adj(part: Partition, dy_shards, w):
    """dx = H* [dConv]* dy, written as the transpose of conv_fwd on the global tensor.

    dx[n,c,p,q] = sum_{a,b} w[c,a,b] * dy[n,c,p-a+ph,q-b+pw], dy = 0 outside.
    fp64 accumulation, one rounding to fp32.  Returned as padded shards of
    `part` whose ghosts are zero (what H* leaves behind).
    """
    w = np.asarray(w, dtype=np.float64)
    C, kh, kw = w.shape
    _check_conv_partition(part, kh, kw)
    ph, pw = kh // 2, kw // 2
    ypart = Partition(part.global_shape, part.pshape, 0, 0)
    dyg = assemble_global(ypart, dy_shards).astype(np.float64)
    N, Cy, Hg, Wg = dyg.shape
    assert Cy == C
    dyp = np.zeros((N, C, Hg + 2 * ph, Wg + 2 * pw), dtype=np.float64)
    dyp[:, :, ph:ph + Hg, pw:pw + Wg] = dyg
    acc = np.zeros((N, C, Hg, Wg), dtype=np.float64)
    for a in range(kh):
        for b in range(kw):
            # dy index p - a + ph  ->  padded index p - a + 2*ph
            acc += w[None, :, a, b, None, None] * \
                dyp[:, :, 2 * ph - a:2 * ph - a + Hg, 2 * pw - b:2 * pw - b + Wg]
    return scatter_global(part, acc.astype(np.float32))


def conv_adj_scatter_then_halo(part: Partition, dy_shards, w):
    """The adjoint convolution algorithm taken step by step (cross-check form).

    Each worker applies the adjoint of its local convolution to its own dy
    block, which scatters into its whole padded input shard (ghosts included);
    H* then adds the ghost parts into the neighbours' bulk and clears them.
    Local scatter in fp64, rounded to fp32 before H* (so the result agrees with
    conv_adj only to fp32 rounding).
    """
    w = np.asarray(w, dtype=np.float64)
    C, kh, kw = w.shape
    _check_conv_partition(part, kh, kw)
    ph, pw = kh // 2, kw // 2
    for k, h in ((2, ph), (3, pw)):
        assert all(v == h for v in part.hlo[k]) and all(v == h for v in part.hhi[k])
    local = []
    for wk in range(part.num_workers):
        dy = np.asarray(dy_shards[wk], dtype=np.float64)
        N, Cy, hb, wb = dy.shape
        dx = np.zeros((N, C, hb + 2 * ph, wb + 2 * pw), dtype=np.float64)
        for a in range(kh):
            for b in range(kw):
                # forward: y[i,j] += w[a,b] * xpad[i+a, j+b]  =>  transpose
                dx[:, :, a:a + hb, b:b + wb] += w[None, :, a, b, None, None] * dy
        local.append(dx.astype(np.float32))
    return halo_adj_sequence(part, local)


def conv_adj_params(part: Partition, x_shards, dy_shards, kh, kw):
    """Parameter part of the adjoint convolution algorithm: (dw, db), depthwise kernel.

    With the tensor partitioned over the feature space only, every worker holds
    a copy of the kernel (w^ <- B w), so its local gradients are summed over the
    workers (dw <- R dw^, db <- R db^, in worker order).  Step by step:
      x <- H x            (the exchanged input saved by the forward pass)
      dw^_k[c,a,b] = sum_{n,i,j} dy_k[n,c,i,j] * x_k[n,c,i+a,j+b]   (padded-local indices)
      db^_k[c]     = sum_{n,i,j} dy_k[n,c,i,j]
      dw = R_k dw^_k,  db = R_k db^_k
    Local sums and the fold over workers in fp64, rounded once to fp32.
    """
    _check_conv_partition(part, kh, kw)
    from .primitives import halo_fwd_sequence
    xh = halo_fwd_sequence(part, x_shards)
    dws, dbs = [], []
    for wk in range(part.num_workers):
        x = np.asarray(xh[wk], dtype=np.float64)
        dy = np.asarray(dy_shards[wk], dtype=np.float64)
        N, C, hb, wb = dy.shape
        assert x.shape == (N, C, hb + kh - 1, wb + kw - 1)
        dwk = np.zeros((C, kh, kw), dtype=np.float64)
        for a in range(kh):
            for b in range(kw):
                dwk[:, a, b] = (dy * x[:, :, a:a + hb, b:b + wb]).sum(axis=(0, 2, 3))
        dws.append(dwk)
        dbs.append(dy.sum(axis=(0, 2, 3)))
    return sumreduce_fwd(dws).astype(np.float32), sumreduce_fwd(dbs).astype(np.float32)


# --------------------------------------------------------------------------
# Generalized distributed convolution: channels partitioned as well
# (Section 4, "Sparse layers": forward / adjoint convolution algorithms with
# P_x = 1 x P_ci x P_0 x P_1, P_y = 1 x P_co x P_0 x P_1, weights on P_co x P_ci,
# work partition 1 x P_co x P_ci x P_0 x P_1)
# --------------------------------------------------------------------------

def _channel_blocks(n, p):
    from .partition import balanced_split
    return balanced_split(n, p)


def convg_fwd(xpart: Partition, nco, pco, x_shards, w_blocks, bias_blocks=None):
    """Forward convolution algorithm, step by step.

    xpart: partition 1 x P_ci x P_0 x P_1 of x [N, n_ci, H, W] with ghost widths
    (0, 0, ph, pw); worker (j, r, c) has id (j * P_0 + r) * P_1 + c.
    w_blocks[i * P_ci + j]: [n_co/P_co, n_ci/P_ci, kh, kw] (the block of worker (i, j)
    of P_r); bias_blocks[i]: [n_co/P_co] or None, present on the j = 0 subpartition only.
      x <- H x;  w^ <- B w, b^ <- B b (to every spatial worker);  x^ <- B x (to the
      P_co copies of the work partition);  y^_{ijs} <- Conv(w^_{ij}, b^_i if j = 0; x^_{js});
      y_{is} <- R over j = 0..P_ci-1 in order.
    Local convolutions and the fold in fp64, rounded once to fp32.  Returns the
    bulk-shaped shards of y on 1 x P_co x P_0 x P_1, id (i * P_0 + r) * P_1 + c.
    """
    from .primitives import halo_fwd_sequence
    assert xpart.rank == 4 and xpart.pshape[0] == 1
    _, pci, p0, p1 = xpart.pshape
    kh, kw = np.asarray(w_blocks[0]).shape[2:]
    ph, pw = kh // 2, kw // 2
    xh = halo_fwd_sequence(xpart, x_shards)
    xhat = [broadcast_fwd(np.asarray(a, dtype=np.float64), pco) for a in xh]        # copies for i = 0..P_co-1
    y = []
    for i in range(pco):
        for r in range(p0):
            for c in range(p1):
                partial = []
                for j in range(pci):
                    x = xhat[(j * p0 + r) * p1 + c][i]
                    w = np.asarray(w_blocks[i * pci + j], dtype=np.float64)
                    N, cib, hp, wp = x.shape
                    cob = w.shape[0]
                    assert w.shape[1] == cib
                    hb, wb = hp - 2 * ph, wp - 2 * pw
                    acc = np.zeros((N, cob, hb, wb), dtype=np.float64)
                    for a in range(kh):
                        for b in range(kw):
                            # sum over the block's input channels, in channel order
                            acc += np.einsum("oc,nchw->nohw", w[:, :, a, b], x[:, :, a:a + hb, b:b + wb])
                    if bias_blocks is not None and j == 0:
                        acc += np.asarray(bias_blocks[i], dtype=np.float64)[None, :, None, None]
                    partial.append(acc)
                y.append(sumreduce_fwd(partial).astype(np.float32))
    return y


def convg_adj(xpart: Partition, nco, pco, dy_shards, w_blocks):
    """Adjoint convolution algorithm, dx output, step by step.

      dy^_{ijs} <- B dy_{is} (to the P_ci copies);  dx^_{ijs} <- [dConv]*(dy^_{ijs}) with
      w^_{ij}: the local adjoint scatters into the whole padded input shard;
      dx_{js} <- R over i = 0..P_co-1 in order;  dx <- H* dx.
    fp64 up to the end of R, rounded to fp32 before H* (whose sums are then fp32, as in
    the halo oracle).  Returns padded shards of xpart with zero ghosts.
    """
    assert xpart.rank == 4 and xpart.pshape[0] == 1
    _, pci, p0, p1 = xpart.pshape
    kh, kw = np.asarray(w_blocks[0]).shape[2:]
    local = []
    for j in range(pci):
        for r in range(p0):
            for c in range(p1):
                wk = (j * p0 + r) * p1 + c
                partial = []
                for i in range(pco):
                    dy = np.asarray(dy_shards[(i * p0 + r) * p1 + c], dtype=np.float64)
                    w = np.asarray(w_blocks[i * pci + j], dtype=np.float64)
                    N, cob, hb, wb = dy.shape
                    dx = np.zeros((N, w.shape[1], hb + kh - 1, wb + kw - 1), dtype=np.float64)
                    for a in range(kh):
                        for b in range(kw):
                            dx[:, :, a:a + hb, b:b + wb] += np.einsum("oc,nohw->nchw", w[:, :, a, b], dy)
                    partial.append(dx)
                got = sumreduce_fwd(partial).astype(np.float32)
                assert got.shape == xpart.padded_shape(wk)
                local.append(got)
    return halo_adj_sequence(xpart, local)


def convg_adj_params(xpart: Partition, nco, pco, x_shards, dy_shards, kh, kw):
    """Parameter part of the adjoint convolution algorithm with channel partitions: (dw blocks, db blocks).

      x <- H x (the exchanged input of the forward pass);  dy^_{ijs} <- B dy_{is};
      dw^_{ijs}[o,c,a,b] = sum_{n,p} dy^_{ijs}[n,o,p] * x^_{js}[n,c,p + (a,b)]   (padded-local indices),
      db^_{ijs}[o]       = sum_{n,p} dy^_{ijs}[n,o,p]                            (j = 0 only);
      dw_{ij} <- R over the feature-space workers s in order,  db_i <- R over s (from the j = 0 workers).
    fp64 throughout, rounded once to fp32.  Returns (dw, db): dw[i * P_ci + j] of shape
    [nco_i, nci_j, kh, kw], db[i] of shape [nco_i].
    """
    from .primitives import halo_fwd_sequence
    assert xpart.rank == 4 and xpart.pshape[0] == 1
    _, pci, p0, p1 = xpart.pshape
    xh = halo_fwd_sequence(xpart, x_shards)
    dw, db = [], []
    for i in range(pco):
        for j in range(pci):
            per_worker = []
            for r in range(p0):
                for c in range(p1):
                    x = np.asarray(xh[(j * p0 + r) * p1 + c], dtype=np.float64)
                    dy = np.asarray(dy_shards[(i * p0 + r) * p1 + c], dtype=np.float64)
                    N, cob, hb, wb = dy.shape
                    g = np.zeros((cob, x.shape[1], kh, kw), dtype=np.float64)
                    for a in range(kh):
                        for b in range(kw):
                            g[:, :, a, b] = np.einsum("nohw,nchw->oc", dy, x[:, :, a:a + hb, b:b + wb])
                    per_worker.append(g)
            dw.append(sumreduce_fwd(per_worker).astype(np.float32))
        sums = [np.asarray(dy_shards[(i * p0 + r) * p1 + c], dtype=np.float64).sum(axis=(0, 2, 3))
                for r in range(p0) for c in range(p1)]
        db.append(sumreduce_fwd(sums).astype(np.float32))
    return dw, db


# --------------------------------------------------------------------------
# Distributed star-stencil layer on a rank-3 tensor (Section 4, "Sparse layers":
# a sliding-kernel layer on a feature-space partition = halo exchange, then the
# local kernel; Section 6 names large volumetric data as the target)
# --------------------------------------------------------------------------

def _star_apply(g, w, flip):
    """sum over axes d and offsets k = -R..R of w[d][k + R] * g shifted by k along d (zeros outside).

    flip = False: out[i] = sum w[d][k + R] * g[i + k e_d]   (cross-correlation, as for Conv)
    flip = True:  out[i] = sum w[d][k + R] * g[i - k e_d]   (its transpose)
    fp64 throughout.
    """
    w = np.asarray(w, dtype=np.float64)
    assert w.ndim == 2 and w.shape[0] == 3 and w.shape[1] % 2 == 1
    R = w.shape[1] // 2
    g = np.asarray(g, dtype=np.float64)
    gp = np.zeros(tuple(n + 2 * R for n in g.shape), dtype=np.float64)
    gp[R:R + g.shape[0], R:R + g.shape[1], R:R + g.shape[2]] = g
    out = np.zeros(g.shape, dtype=np.float64)
    for d in range(3):
        for k in range(-R, R + 1):
            off = [R, R, R]
            off[d] += -k if flip else k
            out += w[d][k + R] * gp[off[0]:off[0] + g.shape[0], off[1]:off[1] + g.shape[1], off[2]:off[2] + g.shape[2]]
    return out


def stencil3d_fwd(part: Partition, x_shards, w):
    """y = Stencil(w; H x): the sequential layer written out on the global tensor.

    w[d][k + R], d = 0..2, k = -R..R: one 1-D kernel per dimension (a star);
    y[i] = sum_d sum_k w[d][k + R] * x[i + k e_d], x = 0 outside the tensor.
    fp64 accumulation, rounded once to fp32.  Returns bulk-shaped shards.
    """
    assert part.rank == 3
    yg = _star_apply(assemble_global(part, x_shards), w, flip=False).astype(np.float32)
    return scatter_global(Partition(part.global_shape, part.pshape, 0, 0), yg)


def stencil3d_adj(part: Partition, dy_shards, w):
    """dx = H* [dStencil]* dy as the transpose of stencil3d_fwd on the global tensor.

    dx[i] = sum_d sum_k w[d][k + R] * dy[i - k e_d], dy = 0 outside.  Returned as
    padded shards of `part` whose ghosts are zero (what H* leaves behind).
    """
    assert part.rank == 3
    ypart = Partition(part.global_shape, part.pshape, 0, 0)
    dxg = _star_apply(assemble_global(ypart, dy_shards), w, flip=True).astype(np.float32)
    return scatter_global(part, dxg)


def stencil3d_fwd_exchange_then_local(part: Partition, x_shards, w):
    """The layer taken step by step (cross-check form): x <- H x, then every worker
    applies the kernel to its own padded shard, producing its bulk-shaped block."""
    w = np.asarray(w, dtype=np.float64)
    R = w.shape[1] // 2
    from .primitives import halo_fwd_sequence
    out = []
    for wk, xh in enumerate(halo_fwd_sequence(part, x_shards)):
        xh = np.asarray(xh, dtype=np.float64)
        assert all(part.hlo[d][c] == R and part.hhi[d][c] == R for d in range(3) for c in range(part.pshape[d]))
        b = tuple(n - 2 * R for n in xh.shape)
        acc = np.zeros(b, dtype=np.float64)
        for d in range(3):
            for k in range(-R, R + 1):
                off = [R, R, R]
                off[d] += k
                acc += w[d][k + R] * xh[off[0]:off[0] + b[0], off[1]:off[1] + b[1], off[2]:off[2] + b[2]]
        out.append(acc.astype(np.float32))
    return out


# --------------------------------------------------------------------------
# Distributed affine layer (Section 4, "Dense layers")
# --------------------------------------------------------------------------

def affine_fwd(x_parts, w_parts, pfo, pfi, bias_parts=None):
    """Forward affine algorithm on a P_fo x P_fi worker grid.

    x_parts[j]   (n_b, n_fi/P_fi) fp64 values, j = 0..P_fi-1 (partition 1 x P_fi)
    w_parts[i*P_fi + j]  (n_fo/P_fo, n_fi/P_fi), worker (i, j) in row-major order
    bias_parts[i]  (n_fo/P_fo,) or None; lives on grid column j = 0 only (Section 4,
                 "Dense layers": the bias sits on a single column of the grid so that it is
                 counted once; cf. Table C1: workers 0 and 2 of a 2 x 2)
    Steps: x^_{ij} <- B x_j;  y^_{ij} <- Affine(w_{ij}, b_{ij}; x^_{ij});
           y_i <- R over j = 0..P_fi-1 in order.
    Local contraction in fp64; the fold over j is done in fp64 as well and the
    result is rounded once to fp32.
    """
    y = []
    xhat = [broadcast_fwd(np.asarray(x_parts[j], dtype=np.float64), pfo) for j in range(pfi)]
    for i in range(pfo):
        partial = []
        for j in range(pfi):
            wij = np.asarray(w_parts[i * pfi + j], dtype=np.float64)
            yij = xhat[j][i] @ wij.T
            if bias_parts is not None and j == 0:
                yij = yij + np.asarray(bias_parts[i], dtype=np.float64)[None, :]
            partial.append(yij)
        y.append(sumreduce_fwd(partial).astype(np.float32))
    return y


def affine_adj(dy_parts, w_parts, pfo, pfi):
    """Adjoint affine algorithm, dx output only.

    dy^_{ij} <- B dy_i;  dx^_{ij} <- dy^_{ij} w_{ij};  dx_j <- R over
    i = 0..P_fo-1 in order.  fp64 throughout, rounded once to fp32.
    """
    dx = []
    dyhat = [broadcast_fwd(np.asarray(dy_parts[i], dtype=np.float64), pfi) for i in range(pfo)]
    for j in range(pfi):
        partial = []
        for i in range(pfo):
            wij = np.asarray(w_parts[i * pfi + j], dtype=np.float64)
            partial.append(dyhat[i][j] @ wij)
        dx.append(sumreduce_fwd(partial).astype(np.float32))
    return dx


def affine_adj_params(dy_parts, x_parts, pfo, pfi):
    """Parameter part of the adjoint affine algorithm: (dW, db).

    dy^_{ij} <- B dy_i (along grid rows); worker (i, j) holds x^_{ij} = x_j from
    the forward pass and applies [dAffine]* to dy^_{ij}:
        dW_{ij}[o, f] = sum_b dy^_{ij}[b, o] * x^_{ij}[b, f]
        db_{ij}[o]    = sum_b dy^_{ij}[b, o]      (only where the bias lives: j = 0)
    The weights are distributed on P_w itself, so no reduction follows: the
    result is one block per worker, in worker order i * P_fi + j, and one bias
    gradient per grid row.  fp64 sums over b in ascending order, rounded once
    to fp32.
    """
    dyhat = [broadcast_fwd(np.asarray(dy_parts[i], dtype=np.float64), pfi) for i in range(pfo)]
    xhat = [broadcast_fwd(np.asarray(x_parts[j], dtype=np.float64), pfo) for j in range(pfi)]
    dw, db = [], []
    for i in range(pfo):
        for j in range(pfi):
            dw.append((dyhat[i][j].T @ xhat[j][i]).astype(np.float32))
        db.append(dyhat[i][0].sum(axis=0).astype(np.float32))
    return dw, db


# --------------------------------------------------------------------------
# Distributed pooling layer (Section 4, "Sparse layers": pooling layers follow
# the convolution algorithms without weights; Appendix B: unbalanced halos of
# strided kernels)
# --------------------------------------------------------------------------

def pool_partition(global_shape, pshape, kernel, stride, pad):
    """Partition of a rank-4 NCHW input whose ghost widths are those of a pooling kernel.

    kernel = (kh, kw), stride = (sh, sw), pad = ((lo_h, hi_h), (lo_w, hi_w)).
    Only the two feature dimensions may be partitioned.  The widths of every
    worker follow from the range of inputs its block of the evenly split output
    needs (Section 3; Figs. B1-B4).  Returns (partition, geometry) where
    geometry[k] (k = 0 for H, 1 for W) is the list of per-worker-coordinate
    dicts of `halo_widths_1d`.
    """
    from .partition import halo_widths_1d
    assert len(global_shape) == 4 and pshape[0] == 1 and pshape[1] == 1
    geo = [halo_widths_1d(global_shape[2 + k], pshape[2 + k], kernel[k], stride[k], 1, pad[k][0], pad[k][1])
           for k in range(2)]
    hlo = [0, 0] + [[g["halo_lo"] for g in geo[k]] for k in range(2)]
    hhi = [0, 0] + [[g["halo_hi"] for g in geo[k]] for k in range(2)]
    return Partition(global_shape, pshape, hlo, hhi), geo


def _pool_windows(xg, kernel, stride, pad, fill):
    """All windows of the padded global tensor: array [N, C, Ho, Wo, kh, kw] (fp64)."""
    N, C, Hg, Wg = xg.shape
    (kh, kw), (sh, sw) = kernel, stride
    (plh, phh), (plw, phw) = pad
    Ho = (Hg + plh + phh - kh) // sh + 1
    Wo = (Wg + plw + phw - kw) // sw + 1
    xp = np.full((N, C, Hg + plh + phh, Wg + plw + phw), fill, dtype=np.float64)
    xp[:, :, plh:plh + Hg, plw:plw + Wg] = xg
    win = np.empty((N, C, Ho, Wo, kh, kw), dtype=np.float64)
    for a in range(kh):
        for b in range(kw):
            win[..., a, b] = xp[:, :, a:a + (Ho - 1) * sh + 1:sh, b:b + (Wo - 1) * sw + 1:sw]
    return win


def pool_fwd_global(xg, kernel, stride, pad, mode):
    """The sequential pooling layer on the unpartitioned tensor.

    mode "avg": y = mean over the kh x kw window of the zero-padded input (padding
    cells count in the divisor), fp64 sum rounded once to fp32.
    mode "max": y = largest value of the window, padding excluded (the window is
    clipped to the tensor); also returns, per output, the position a*kw + b inside
    the unclipped window of the first largest value in row-major window order.
    Returns (y, argmax or None).
    """
    xg = np.asarray(xg)
    kh, kw = kernel
    if mode == "avg":
        win = _pool_windows(xg.astype(np.float64), kernel, stride, pad, 0.0)
        return (win.sum(axis=(4, 5)) / (kh * kw)).astype(np.float32), None
    assert mode == "max"
    win = _pool_windows(xg.astype(np.float64), kernel, stride, pad, -np.inf)
    flat = win.reshape(win.shape[:4] + (kh * kw,))
    arg = flat.argmax(axis=4)            # first occurrence of the maximum
    return flat.max(axis=4).astype(np.float32), arg.astype(np.int32)


def pool_adj_global(dyg, in_hw, kernel, stride, pad, mode, argmax=None):
    """Adjoint of the pooling layer (for "max": of its Jacobian at the recorded argmax).

    dx[p, q] = sum over the outputs (i, j) whose window holds (p, q) of
    dy[i, j] / (kh*kw)  (avg), or of dy[i, j] where the recorded position of the
    maximum is (p, q)  (max).  fp64 sums rounded once to fp32.
    """
    dyg = np.asarray(dyg, dtype=np.float64)
    N, C, Ho, Wo = dyg.shape
    (kh, kw), (sh, sw) = kernel, stride
    (plh, phh), (plw, phw) = pad
    Hg, Wg = in_hw
    dxp = np.zeros((N, C, Hg + plh + phh, Wg + plw + phw), dtype=np.float64)
    for a in range(kh):
        for b in range(kw):
            if mode == "avg":
                contrib = dyg / (kh * kw)
            else:
                contrib = np.where(argmax == a * kw + b, dyg, 0.0)
            dxp[:, :, a:a + (Ho - 1) * sh + 1:sh, b:b + (Wo - 1) * sw + 1:sw] += contrib
    return dxp[:, :, plh:plh + Hg, plw:plw + Wg].astype(np.float32)


def _pool_out_slices(geo, coords):
    return tuple(slice(geo[k][coords[2 + k]]["out_start"],
                       geo[k][coords[2 + k]]["out_start"] + geo[k][coords[2 + k]]["out_size"]) for k in range(2))


def pool_fwd(part: Partition, geo, x_shards, kernel, stride, pad, mode):
    """Distributed pooling, forward: y = Pool(H x), in the steps of the forward algorithm.

    1. halo exchange on the padded input shards (ghosts on the tensor boundary
       hold the implicit zero padding; for "max" they are excluded from the window),
    2. every worker applies the sequential layer to its padded shard, starting at the
       first input its outputs need (owned inputs before it are unused, Fig. B3).
    Returns (y shards, argmax shards or None); worker c owns the c-th block of the
    evenly split output.
    """
    from .primitives import halo_fwd_definition
    xs = halo_fwd_definition(part, x_shards)
    (kh, kw), (sh, sw) = kernel, stride
    ys, args = [], []
    for w in range(part.num_workers):
        c = part.coords(w)
        gh, gw = geo[0][c[2]], geo[1][c[3]]
        st = part.bulk_start(w)
        lo, _ = part.widths(w)
        x = xs[w].astype(np.float64)
        oh, ow = gh["out_size"], gw["out_size"]
        # padded-local index of the first input of the first local output
        i0 = gh["out_start"] * sh - pad[0][0] - (st[2] - lo[2])
        j0 = gw["out_start"] * sw - pad[1][0] - (st[3] - lo[3])
        assert oh == 0 or (i0 >= 0 and i0 + (oh - 1) * sh + kh <= x.shape[2])
        assert ow == 0 or (j0 >= 0 and j0 + (ow - 1) * sw + kw <= x.shape[3])
        win = np.empty(x.shape[:2] + (oh, ow, kh, kw), dtype=np.float64)
        for a in range(kh):
            for b in range(kw):
                win[..., a, b] = x[:, :, i0 + a:i0 + a + max(oh - 1, 0) * sh + 1:sh,
                                   j0 + b:j0 + b + max(ow - 1, 0) * sw + 1:sw] if oh and ow else 0.0
        if mode == "avg":
            ys.append((win.sum(axis=(4, 5)) / (kh * kw)).astype(np.float32))
            args.append(None)
        else:
            # cells outside the tensor are not candidates
            gi = (st[2] - lo[2]) + i0 + np.arange(oh)[:, None] * sh + np.arange(kh)[None, :]
            gj = (st[3] - lo[3]) + j0 + np.arange(ow)[:, None] * sw + np.arange(kw)[None, :]
            out_i = (gi < 0) | (gi >= part.global_shape[2])
            out_j = (gj < 0) | (gj >= part.global_shape[3])
            mask = out_i[:, None, :, None] | out_j[None, :, None, :]
            win = np.where(mask[None, None], -np.inf, win)
            flat = win.reshape(win.shape[:4] + (kh * kw,))
            ys.append(flat.max(axis=4).astype(np.float32) if oh and ow else np.zeros(win.shape[:4], np.float32))
            args.append(flat.argmax(axis=4).astype(np.int32) if oh and ow else np.zeros(win.shape[:4], np.int32))
    return ys, (None if mode == "avg" else args)


def pool_adj(part: Partition, geo, dy_shards, kernel, stride, pad, mode, arg_shards=None):
    """Distributed pooling, adjoint: dx = H* Pool* dy, in the steps of the adjoint algorithm.

    1. every worker applies the adjoint of its local layer: each cell of its padded
       shard (ghosts included) receives the contributions of the worker's own outputs,
    2. adjoint halo exchange: ghost contributions are added into the owners' bulk
       and the ghosts are cleared.
    Returns padded fp32 shards.  (Local sums in fp64, rounded to fp32 before H*, whose
    sums are fp32 in the nested order -- the rounding points of the method.)
    """
    (kh, kw), (sh, sw) = kernel, stride
    dxs = []
    for w in range(part.num_workers):
        c = part.coords(w)
        gh, gw = geo[0][c[2]], geo[1][c[3]]
        st = part.bulk_start(w)
        lo, _ = part.widths(w)
        pshape = part.padded_shape(w)
        dx = np.zeros(pshape, dtype=np.float64)
        oh, ow = gh["out_size"], gw["out_size"]
        if oh and ow:
            i0 = gh["out_start"] * sh - pad[0][0] - (st[2] - lo[2])
            j0 = gw["out_start"] * sw - pad[1][0] - (st[3] - lo[3])
            dy = np.asarray(dy_shards[w], dtype=np.float64)
            for a in range(kh):
                for b in range(kw):
                    contrib = dy / (kh * kw) if mode == "avg" else np.where(arg_shards[w] == a * kw + b, dy, 0.0)
                    dx[:, :, i0 + a:i0 + a + (oh - 1) * sh + 1:sh, j0 + b:j0 + b + (ow - 1) * sw + 1:sw] += contrib
        dxs.append(dx.astype(np.float32))
    return halo_adj_sequence(part, dxs)
