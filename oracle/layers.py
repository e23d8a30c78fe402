"""Oracle distributed layers: depthwise convolution and affine (Section 4).

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


# --------------------------------------------------------------------------
# Distributed affine layer (Section 4, "Dense layers")
# --------------------------------------------------------------------------

def bf16_bits_to_f64(bits):
    """Widen bfloat16 bit patterns (uint16) exactly to fp64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def affine_fwd(x_parts, w_parts, pfo, pfi, bias_parts=None):
    """Forward affine algorithm on a P_fo x P_fi worker grid.

    x_parts[j]   (n_b, n_fi/P_fi) fp64 values, j = 0..P_fi-1 (partition 1 x P_fi)
    w_parts[i*P_fi + j]  (n_fo/P_fo, n_fi/P_fi), worker (i, j) in row-major order
    bias_parts[i]  (n_fo/P_fo,) or None; lives on grid column j = 0 only (the
                 "one P_fo x 1 subset", cf. Table C1: workers 0 and 2 of a 2 x 2)
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
