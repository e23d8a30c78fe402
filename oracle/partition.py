"""Oracle-side partition and halo geometry (test infrastructure only).

Section 4: a rank-d tensor is partitioned along each dimension by a d-length
partition vector giving the number of workers per dimension.  Appendix B shows
worked 1-D examples from which the balanced split rule and the halo-width rule
are read: the *output* tensor is split evenly, and each worker's halo widths
follow from the smallest and largest global input index its outputs touch
(Section 3, "Halo exchange").
"""

import numpy as np


def balanced_split(n, p):
    """Split extent n over p workers: n = q*p + r, the first r workers get q+1.

    Read from the index lists of the Appendix B figures (11 -> 4,4,3;
    7 -> 3,2,2; 20 -> 4,4,3,3,3,3; 10 -> 2,2,2,2,1,1).
    Returns (starts, sizes) as Python lists.
    """
    q, r = divmod(int(n), int(p))
    sizes = [q + 1 if c < r else q for c in range(p)]
    starts = [0] * p
    for c in range(1, p):
        starts[c] = starts[c - 1] + sizes[c - 1]
    return starts, sizes


def halo_widths_1d(n, p, kernel, stride=1, dilation=1, pad_lo=0, pad_hi=0):
    """Per-worker halo widths of a 1-D sliding kernel (Section 3, Appendix B).

    Input of length n and output of length
        m = floor((n + pad_lo + pad_hi - dilation*(kernel-1) - 1) / stride) + 1
    are both split evenly over p workers.  Output index o reads the inputs
    o*stride - pad_lo + t*dilation, t = 0..kernel-1.  For worker c with outputs
    [o0, o1] the needed input range is [o0*stride - pad_lo,
    o1*stride - pad_lo + dilation*(kernel-1)]; whatever lies left/right of its own
    input block is halo, whatever part of its own block lies outside the needed
    range is unused input.

    Returns a list of dicts with keys in_start, in_size, out_start, out_size,
    halo_lo, halo_hi, unused_lo, unused_hi.
    """
    m = (n + pad_lo + pad_hi - dilation * (kernel - 1) - 1) // stride + 1
    in_starts, in_sizes = balanced_split(n, p)
    out_starts, out_sizes = balanced_split(m, p)
    res = []
    for c in range(p):
        b0 = in_starts[c]
        b1 = in_starts[c] + in_sizes[c] - 1
        o0 = out_starts[c]
        o1 = out_starts[c] + out_sizes[c] - 1
        if out_sizes[c] == 0:
            need0, need1 = b0, b0 - 1
        else:
            need0 = o0 * stride - pad_lo
            need1 = o1 * stride - pad_lo + dilation * (kernel - 1)
        res.append(
            dict(
                in_start=b0,
                in_size=in_sizes[c],
                out_start=o0,
                out_size=out_sizes[c],
                halo_lo=max(0, b0 - need0),
                halo_hi=max(0, need1 - b1),
                unused_lo=max(0, min(need0, b1 + 1) - b0),
                unused_hi=max(0, b1 - max(need1, b0 - 1)),
            )
        )
    return res


class Partition:
    """Cartesian partition of a rank-d tensor with per-side halo widths.

    global_shape[k]  extent of dimension k
    pshape[k]        workers along dimension k (Section 4, partition vector)
    hlo[k][c], hhi[k][c]  ghost widths of the workers whose coordinate in
                     dimension k is c (Section 3: every side of every dimension
                     may have its own thickness).  An int, or a per-dimension
                     int, means "the same width for every worker".
    periodic[k]      True: dimension k wraps around (not in the paper, whose
                     exchange stops at the tensor's boundary; the same operator
                     sequence with the first and last worker as neighbours).

    Worker ids are the row-major index of the partition coordinate, last
    dimension fastest (Appendix B.2: in a 2 x 2 partition workers 0,1 are the
    top row and 2,3 the bottom row).
    """

    def __init__(self, global_shape, pshape, hlo=0, hhi=0, periodic=None):
        self.global_shape = tuple(int(v) for v in global_shape)
        self.pshape = tuple(int(v) for v in pshape)
        self.rank = len(self.global_shape)
        assert len(self.pshape) == self.rank
        # periodic[k]: dimension k wraps around (the first and the last worker are neighbours, and the
        # ghosts on the tensor's boundary hold the cells from the other end instead of zeros)
        self.periodic = tuple(bool(v) for v in periodic) if periodic is not None else (False,) * self.rank
        assert len(self.periodic) == self.rank
        self.start, self.size = [], []
        for k in range(self.rank):
            s, z = balanced_split(self.global_shape[k], self.pshape[k])
            self.start.append(s)
            self.size.append(z)
        self.hlo = self._widths(hlo)
        self.hhi = self._widths(hhi)
        self.num_workers = int(np.prod(self.pshape))

    def _widths(self, h):
        out = []
        for k in range(self.rank):
            hk = h[k] if isinstance(h, (list, tuple)) else h
            if isinstance(hk, (list, tuple)):
                assert len(hk) == self.pshape[k]
                out.append([int(v) for v in hk])
            else:
                out.append([int(hk)] * self.pshape[k])
        return out

    def coords(self, worker):
        """Partition coordinate of a worker id (row-major, last dim fastest)."""
        c = []
        for k in reversed(range(self.rank)):
            c.append(worker % self.pshape[k])
            worker //= self.pshape[k]
        return tuple(reversed(c))

    def worker(self, coords):
        w = 0
        for k in range(self.rank):
            w = w * self.pshape[k] + coords[k]
        return w

    def bulk_start(self, worker):
        c = self.coords(worker)
        return tuple(self.start[k][c[k]] for k in range(self.rank))

    def bulk_shape(self, worker):
        c = self.coords(worker)
        return tuple(self.size[k][c[k]] for k in range(self.rank))

    def widths(self, worker):
        c = self.coords(worker)
        lo = tuple(self.hlo[k][c[k]] for k in range(self.rank))
        hi = tuple(self.hhi[k][c[k]] for k in range(self.rank))
        return lo, hi

    def padded_shape(self, worker):
        lo, hi = self.widths(worker)
        b = self.bulk_shape(worker)
        return tuple(b[k] + lo[k] + hi[k] for k in range(self.rank))

    def bulk_slices(self, worker):
        """Slices selecting the bulk inside the padded shard array."""
        lo, _ = self.widths(worker)
        b = self.bulk_shape(worker)
        return tuple(slice(lo[k], lo[k] + b[k]) for k in range(self.rank))
