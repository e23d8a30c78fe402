"""Thin Python binding of the C-ABI library (include/distdl.h).

Argument marshalling only: tensors are turned into device pointers and sizes, every step of
every operator runs in the CUDA kernels of libdistdl.so.  There is no CPU or PyTorch fallback:
if the library is missing or a call fails, an exception is raised.

PyTorch is used by callers for device memory and streams; this module only reads
`tensor.data_ptr()` and the current stream handle.
"""

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdistdl.so")

F32 = 0
BF16 = 1
F64 = 2
MAX_RANK = 5

STATUS_NAMES = {
    0: "DISTDL_OK", 1: "DISTDL_ERR_INVALID_ARG", 2: "DISTDL_ERR_SHAPE", 3: "DISTDL_ERR_ALIGNMENT",
    4: "DISTDL_ERR_UNSUPPORTED", 5: "DISTDL_ERR_CUDA", 6: "DISTDL_ERR_TIMEOUT", 7: "DISTDL_ERR_NOMEM",
}


class DistdlError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status


_lib = None


def lib():
    """Loads libdistdl.so (once) and declares the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libdistdl.so is not built: run `python -m paper_2006_03108_b200.build` "
            "(there is no fallback path)")
    L = ctypes.CDLL(LIB_PATH)
    c_i32, c_i64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
    pi32, pi64, pvp = ctypes.POINTER(c_i32), ctypes.POINTER(c_i64), ctypes.POINTER(vp)
    ppi32 = ctypes.POINTER(pi32)
    L.distdl_last_error.restype = ctypes.c_char_p
    L.distdl_last_error.argtypes = []
    L.distdl_partition_create.argtypes = [c_i32, pi64, pi32, pi32, pi32, c_i32, pvp]
    L.distdl_partition_create_general.argtypes = [c_i32, pi64, pi32, ppi32, ppi32, c_i32, pvp]
    L.distdl_partition_create_periodic.argtypes = [c_i32, pi64, pi32, pi32, pi32, pi32, c_i32, pvp]
    L.distdl_partition_destroy.argtypes = [vp]
    L.distdl_partition_destroy.restype = None
    L.distdl_partition_num_workers.argtypes = [vp]
    L.distdl_partition_shard_extents.argtypes = [vp, c_i32, pi64, pi64, pi64, pi32, pi32]
    L.distdl_partition_halo_stats.argtypes = [vp, c_i32, pi64, pi64, pi64]
    L.distdl_partition_uses_row_plan.argtypes = [vp, c_i32]
    L.distdl_halo_widths_1d.argtypes = [c_i64, c_i32, c_i32, c_i32, c_i32, c_i32, c_i32, pi32, pi32, pi32, pi32]
    L.distdl_broadcast_fwd.argtypes = [vp, pvp, c_i32, c_i64, c_i32, vp]
    L.distdl_sumreduce_adj.argtypes = [vp, pvp, c_i32, c_i64, c_i32, vp]
    L.distdl_sumreduce_fwd.argtypes = [pvp, vp, c_i32, c_i64, c_i32, vp]
    L.distdl_broadcast_adj.argtypes = [pvp, vp, c_i32, c_i64, c_i32, vp]
    L.distdl_partition_broadcast_fwd.argtypes = [c_i32, pi32, pi32, pi64, pvp, pvp, c_i32, vp]
    L.distdl_partition_broadcast_adj.argtypes = [c_i32, pi32, pi32, pi64, pvp, pvp, c_i32, vp]
    L.distdl_halo_fwd.argtypes = [vp, pvp, vp]
    L.distdl_halo_adj.argtypes = [vp, pvp, vp]
    L.distdl_halo_fwd_noalloc.argtypes = [c_i32, pi64, pi32, pi32, pi32, c_i32, pvp, vp]
    L.distdl_conv_fwd.argtypes = [vp, pvp, vp, vp, c_i32, c_i32, pvp, vp]
    L.distdl_conv_adj.argtypes = [vp, pvp, vp, c_i32, c_i32, pvp, vp]
    L.distdl_repartition_create.argtypes = [c_i32, pi64, pi32, pi32, c_i32, pvp]
    L.distdl_repartition_destroy.argtypes = [vp]
    L.distdl_repartition_destroy.restype = None
    L.distdl_repartition_shard_shape.argtypes = [vp, c_i32, c_i32, pi64]
    L.distdl_repartition_fwd.argtypes = [vp, pvp, pvp, vp]
    L.distdl_repartition_adj.argtypes = [vp, pvp, pvp, vp]
    L.distdl_allreduce.argtypes = [pvp, c_i32, c_i64, c_i32, vp]
    L.distdl_pool_fwd.argtypes = [vp, pvp] + [c_i32] * 9 + [pvp, pvp, vp]
    L.distdl_pool_adj.argtypes = [vp, pvp, pvp] + [c_i32] * 9 + [pvp, vp]
    L.distdl_affine_fwd.argtypes = [c_i64, c_i64, c_i64, c_i32, c_i32, pvp, pvp, pvp, pvp, vp]
    L.distdl_affine_adj.argtypes = [c_i64, c_i64, c_i64, c_i32, c_i32, pvp, pvp, pvp, vp]
    L.distdl_affine_adj_params.argtypes = [c_i64, c_i64, c_i64, c_i32, c_i32, pvp, pvp, pvp, pvp, vp]
    L.distdl_conv_adj_params_workspace.argtypes = [vp, c_i32, c_i32, pi64]
    L.distdl_conv_adj_params.argtypes = [vp, pvp, pvp, c_i32, c_i32, vp, vp, vp, c_i64, vp]
    L.distdl_stencil3d_fwd.argtypes = [vp, pvp, ctypes.POINTER(ctypes.c_float), c_i32, pvp, vp]
    L.distdl_stencil3d_adj.argtypes = [vp, pvp, ctypes.POINTER(ctypes.c_float), c_i32, pvp, vp]
    L.distdl_convg_fwd.argtypes = [vp, c_i64, c_i32, pvp, pvp, pvp, c_i32, c_i32, pvp, vp]
    L.distdl_convg_adj.argtypes = [vp, c_i64, c_i32, pvp, pvp, c_i32, c_i32, pvp, vp]
    L.distdl_convg_adj_params_workspace.argtypes = [vp, c_i64, c_i32, c_i32, c_i32, pi64]
    L.distdl_convg_adj_params.argtypes = [vp, c_i64, c_i32, pvp, pvp, c_i32, c_i32, pvp, pvp, vp, c_i64, vp]
    L.distdl_device_status.argtypes = [vp]
    L.distdl_selftest_wait_timeout.argtypes = [c_i64, vp]
    L.distdl_selftest_row_plan.argtypes = [vp, c_i32, pi32, c_i32, pi32, c_i32, pi32]
    _lib = L
    return L


def _check(status):
    if status != 0:
        raise DistdlError(status, lib().distdl_last_error().decode())


def _ptr(t):
    """Device (or host) address of a tensor-like, or of a raw int."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _ptr_array(ts):
    arr = (ctypes.c_void_p * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = _ptr(t)
    return arr


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float64:
        return F64
    raise TypeError("unsupported dtype %s" % t.dtype)


class Partition:
    """Handle of a distdl_partition_t (see distdl_partition_create in include/distdl.h)."""

    def __init__(self, global_shape, partition_shape, halo_lo=None, halo_hi=None, dtype=F32, periodic=None):
        L = lib()
        rank = len(global_shape)
        if len(partition_shape) != rank:
            raise ValueError("global_shape and partition_shape differ in rank")
        self.rank = rank
        self.global_shape = tuple(int(v) for v in global_shape)
        self.partition_shape = tuple(int(v) for v in partition_shape)
        self._h = ctypes.c_void_p()
        gs = (ctypes.c_int64 * rank)(*self.global_shape)
        ps = (ctypes.c_int32 * rank)(*self.partition_shape)

        def general(h):
            return h is not None and any(isinstance(v, (list, tuple)) for v in h)

        if periodic is not None and any(periodic):
            if general(halo_lo) or general(halo_hi):
                raise ValueError("periodic partitions take one halo width per side and dimension")
            lo = None if halo_lo is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_lo])
            hi = None if halo_hi is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_hi])
            per = (ctypes.c_int32 * rank)(*[1 if v else 0 for v in periodic])
            _check(L.distdl_partition_create_periodic(rank, gs, ps, lo, hi, per, dtype, ctypes.byref(self._h)))
        elif general(halo_lo) or general(halo_hi):
            keep = []

            def rows(h):
                out = (ctypes.POINTER(ctypes.c_int32) * rank)()
                for k in range(rank):
                    hk = 0 if h is None else h[k]
                    vals = list(hk) if isinstance(hk, (list, tuple)) else [int(hk)] * self.partition_shape[k]
                    if len(vals) != self.partition_shape[k]:
                        raise ValueError("halo width list %d has the wrong length" % k)
                    a = (ctypes.c_int32 * len(vals))(*vals)
                    keep.append(a)
                    out[k] = ctypes.cast(a, ctypes.POINTER(ctypes.c_int32))
                return out

            _check(L.distdl_partition_create_general(rank, gs, ps, rows(halo_lo), rows(halo_hi), dtype,
                                                     ctypes.byref(self._h)))
        else:
            lo = None if halo_lo is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_lo])
            hi = None if halo_hi is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_hi])
            _check(L.distdl_partition_create(rank, gs, ps, lo, hi, dtype, ctypes.byref(self._h)))
        self.dtype = dtype
        self.num_workers = L.distdl_partition_num_workers(self._h)

    @property
    def handle(self):
        return self._h

    def shard_extents(self, worker):
        """(bulk_start, bulk_shape, padded_shape, halo_lo, halo_hi) of one worker, as tuples."""
        r = self.rank
        a, b, c = (ctypes.c_int64 * r)(), (ctypes.c_int64 * r)(), (ctypes.c_int64 * r)()
        lo, hi = (ctypes.c_int32 * r)(), (ctypes.c_int32 * r)()
        _check(lib().distdl_partition_shard_extents(self._h, worker, a, b, c, lo, hi))
        return tuple(a), tuple(b), tuple(c), tuple(lo), tuple(hi)

    def padded_shape(self, worker):
        return self.shard_extents(worker)[2]

    def bulk_shape(self, worker):
        return self.shard_extents(worker)[1]

    def halo_stats(self, adjoint=False):
        """(boxes, tiles, algorithmic bytes) of the H (or H*) plan."""
        a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        _check(lib().distdl_partition_halo_stats(self._h, 1 if adjoint else 0, ctypes.byref(a),
                                                 ctypes.byref(b), ctypes.byref(c)))
        return a.value, b.value, c.value

    def uses_row_plan(self, adjoint=False):
        """True if H of this partition runs through the row plan (rows of whole 16-byte units), or, with adjoint, if
        H* hands the row ends to it."""
        return lib().distdl_partition_uses_row_plan(self._h, 1 if adjoint else 0) == 1

    def close(self):
        if self._h:
            lib().distdl_partition_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def partition_create(global_shape, partition_shape, halo_lo=None, halo_hi=None, dtype=F32):
    return Partition(global_shape, partition_shape, halo_lo, halo_hi, dtype)


def halo_widths_1d(n, p, kernel, stride=1, dilation=1, pad_lo=0, pad_hi=0):
    """Per-worker (halo_lo, halo_hi, unused_lo, unused_hi) lists of a 1-D sliding kernel."""
    arrs = [(ctypes.c_int32 * p)() for _ in range(4)]
    _check(lib().distdl_halo_widths_1d(n, p, kernel, stride, dilation, pad_lo, pad_hi, *arrs))
    return tuple(list(a) for a in arrs)


def broadcast_fwd(src, dsts, stream=None):
    _check(lib().distdl_broadcast_fwd(_ptr(src), _ptr_array(dsts), len(dsts), src.numel(), _dtype_code(src),
                                      _stream(stream)))


def sumreduce_adj(dy, dxs, stream=None):
    _check(lib().distdl_sumreduce_adj(_ptr(dy), _ptr_array(dxs), len(dxs), dy.numel(), _dtype_code(dy),
                                      _stream(stream)))


def sumreduce_fwd(srcs, dst, stream=None):
    _check(lib().distdl_sumreduce_fwd(_ptr_array(srcs), _ptr(dst), len(srcs), dst.numel(), _dtype_code(dst),
                                      _stream(stream)))


def broadcast_adj(dys, dx, stream=None):
    _check(lib().distdl_broadcast_adj(_ptr_array(dys), _ptr(dx), len(dys), dx.numel(), _dtype_code(dx),
                                      _stream(stream)))


def _partition_pair(src_pshape, dst_pshape, small):
    rank = len(src_pshape)
    if len(dst_pshape) != rank:
        raise ValueError("partition shapes differ in rank")
    sp = (ctypes.c_int32 * rank)(*[int(v) for v in src_pshape])
    dp = (ctypes.c_int32 * rank)(*[int(v) for v in dst_pshape])
    el = (ctypes.c_int64 * len(small))(*[t.numel() for t in small])
    return rank, sp, dp, el


def partition_broadcast_fwd(src_pshape, dst_pshape, src, dst, stream=None):
    """dst[w] <- src[source of w]: broadcast along the partition dimensions where src_pshape is 1."""
    rank, sp, dp, el = _partition_pair(src_pshape, dst_pshape, src)
    _check(lib().distdl_partition_broadcast_fwd(rank, sp, dp, el, _ptr_array(src), _ptr_array(dst), _dtype_code(src[0]),
                                                _stream(stream)))


def partition_broadcast_adj(src_pshape, dst_pshape, dy, dx, stream=None):
    """dx[j] <- sum, in worker order, of the dy[w] whose source is j: the sum-reduce back to the smaller partition."""
    rank, sp, dp, el = _partition_pair(src_pshape, dst_pshape, dx)
    _check(lib().distdl_partition_broadcast_adj(rank, sp, dp, el, _ptr_array(dy), _ptr_array(dx), _dtype_code(dx[0]),
                                                _stream(stream)))


def halo_fwd(part, shards, stream=None):
    _check(lib().distdl_halo_fwd(part.handle, _ptr_array(shards), _stream(stream)))


def halo_adj(part, shards, stream=None):
    _check(lib().distdl_halo_adj(part.handle, _ptr_array(shards), _stream(stream)))


def halo_fwd_noalloc(global_shape, partition_shape, halo_lo, halo_hi, shards, dtype=F32, stream=None):
    """H for callers that must not allocate device memory: same result as halo_fwd, but the plan
    tables go into a fixed 1 MiB device array of the library instead of a cudaMalloc'd block
    (see distdl_halo_fwd_noalloc in include/distdl.h for the limits and the sharing rules)."""
    rank = len(global_shape)
    gs = (ctypes.c_int64 * rank)(*[int(v) for v in global_shape])
    ps = (ctypes.c_int32 * rank)(*[int(v) for v in partition_shape])
    lo = None if halo_lo is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_lo])
    hi = None if halo_hi is None else (ctypes.c_int32 * rank)(*[int(v) for v in halo_hi])
    _check(lib().distdl_halo_fwd_noalloc(rank, gs, ps, lo, hi, dtype, _ptr_array(shards), _stream(stream)))


def conv_fwd(part, x, w, bias, y, stream=None):
    kh, kw = int(w.shape[-2]), int(w.shape[-1])
    _check(lib().distdl_conv_fwd(part.handle, _ptr_array(x), _ptr(w), _ptr(bias), kh, kw, _ptr_array(y),
                                 _stream(stream)))


def conv_adj(part, dy, w, dx, stream=None):
    kh, kw = int(w.shape[-2]), int(w.shape[-1])
    _check(lib().distdl_conv_adj(part.handle, _ptr_array(dy), _ptr(w), kh, kw, _ptr_array(dx), _stream(stream)))


def _taps(w):
    """Host array of the 3 x (2R+1) taps (any nested sequence or numpy array) and the radius."""
    rows = [[float(v) for v in row] for row in w]
    if len(rows) != 3 or len(set(len(r) for r in rows)) != 1 or len(rows[0]) % 2 != 1:
        raise ValueError("taps must have shape [3][2R+1]")
    n = len(rows[0])
    return (ctypes.c_float * (3 * n))(*[v for row in rows for v in row]), n // 2


def stencil3d_fwd(part, x, w, y, stream=None):
    arr, radius = _taps(w)
    _check(lib().distdl_stencil3d_fwd(part.handle, _ptr_array(x), arr, radius, _ptr_array(y), _stream(stream)))


def stencil3d_adj(part, dy, w, dx, stream=None):
    arr, radius = _taps(w)
    _check(lib().distdl_stencil3d_adj(part.handle, _ptr_array(dy), arr, radius, _ptr_array(dx), _stream(stream)))


def convg_fwd(px, nco, pco, x, w, bias, y, stream=None):
    """Channel-partitioned convolution layer; w: list of blocks [nco_i, nci_j, kh, kw] in order i * P_ci + j."""
    kh, kw = int(w[0].shape[-2]), int(w[0].shape[-1])
    b = None if bias is None else _ptr_array(bias)
    _check(lib().distdl_convg_fwd(px.handle, nco, pco, _ptr_array(x), _ptr_array(w), b, kh, kw, _ptr_array(y),
                                  _stream(stream)))


def convg_adj(px, nco, pco, dy, w, dx, stream=None):
    kh, kw = int(w[0].shape[-2]), int(w[0].shape[-1])
    _check(lib().distdl_convg_adj(px.handle, nco, pco, _ptr_array(dy), _ptr_array(w), kh, kw, _ptr_array(dx),
                                  _stream(stream)))


def convg_adj_params_workspace(px, nco, pco, kh, kw):
    n = ctypes.c_int64(0)
    _check(lib().distdl_convg_adj_params_workspace(px.handle, nco, pco, kh, kw, ctypes.byref(n)))
    return n.value


def convg_adj_params(px, nco, pco, x, dy, kernel, dw, db, workspace, stream=None):
    """dw: list of blocks [nco_i, nci_j, kh, kw] in order i * P_ci + j; db: list of [nco_i] or None."""
    b = None if db is None else _ptr_array(db)
    _check(lib().distdl_convg_adj_params(px.handle, nco, pco, _ptr_array(x), _ptr_array(dy), kernel[0], kernel[1],
                                         _ptr_array(dw), b, _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


class Repartition:
    """Handle of a distdl_repartition_t: one tensor under a source and a destination partition."""

    def __init__(self, global_shape, src_partition_shape, dst_partition_shape, dtype=F32):
        rank = len(global_shape)
        if len(src_partition_shape) != rank or len(dst_partition_shape) != rank:
            raise ValueError("shapes differ in rank")
        self.rank = rank
        self._h = ctypes.c_void_p()
        gs = (ctypes.c_int64 * rank)(*[int(v) for v in global_shape])
        sp = (ctypes.c_int32 * rank)(*[int(v) for v in src_partition_shape])
        dp = (ctypes.c_int32 * rank)(*[int(v) for v in dst_partition_shape])
        _check(lib().distdl_repartition_create(rank, gs, sp, dp, dtype, ctypes.byref(self._h)))
        self.num_src = self.num_dst = 1
        for a, b in zip(src_partition_shape, dst_partition_shape):
            self.num_src *= int(a)
            self.num_dst *= int(b)

    @property
    def handle(self):
        return self._h

    def shard_shape(self, worker, destination=False):
        out = (ctypes.c_int64 * self.rank)()
        _check(lib().distdl_repartition_shard_shape(self._h, 1 if destination else 0, worker, out))
        return tuple(out)

    def __del__(self):
        try:
            if self._h:
                lib().distdl_repartition_destroy(self._h)
                self._h = ctypes.c_void_p()
        except Exception:
            pass


def repartition_fwd(rep, src, dst, stream=None):
    _check(lib().distdl_repartition_fwd(rep.handle, _ptr_array(src), _ptr_array(dst), _stream(stream)))


def repartition_adj(rep, dy, dx, stream=None):
    _check(lib().distdl_repartition_adj(rep.handle, _ptr_array(dy), _ptr_array(dx), _stream(stream)))


def allreduce(bufs, stream=None):
    _check(lib().distdl_allreduce(_ptr_array(bufs), len(bufs), bufs[0].numel(), _dtype_code(bufs[0]), _stream(stream)))


POOL_AVG, POOL_MAX = 0, 1


def pool_fwd(part, x, kernel, stride, pad, mode, y, argmax=None, stream=None):
    """kernel = (kh, kw), stride = (sh, sw), pad = ((lo_h, hi_h), (lo_w, hi_w)); x is updated in place by H."""
    a = None if argmax is None else _ptr_array(argmax)
    _check(lib().distdl_pool_fwd(part.handle, _ptr_array(x), kernel[0], kernel[1], stride[0], stride[1], pad[0][0],
                                 pad[0][1], pad[1][0], pad[1][1], mode, _ptr_array(y), a, _stream(stream)))


def pool_adj(part, dy, argmax, kernel, stride, pad, mode, dx, stream=None):
    a = None if argmax is None else _ptr_array(argmax)
    _check(lib().distdl_pool_adj(part.handle, _ptr_array(dy), a, kernel[0], kernel[1], stride[0], stride[1], pad[0][0],
                                 pad[0][1], pad[1][0], pad[1][1], mode, _ptr_array(dx), _stream(stream)))


def affine_fwd(nb, nfi, nfo, pfo, pfi, x, w, bias, y, stream=None):
    b = None if bias is None else _ptr_array(bias)
    _check(lib().distdl_affine_fwd(nb, nfi, nfo, pfo, pfi, _ptr_array(x), _ptr_array(w), b, _ptr_array(y),
                                   _stream(stream)))


def affine_adj(nb, nfi, nfo, pfo, pfi, dy, w, dx, stream=None):
    _check(lib().distdl_affine_adj(nb, nfi, nfo, pfo, pfi, _ptr_array(dy), _ptr_array(w), _ptr_array(dx),
                                   _stream(stream)))


def affine_adj_params(nb, nfi, nfo, pfo, pfi, dy, x, dw, db=None, stream=None):
    """dW blocks (worker order i * pfi + j) and, if given, the db blocks of the adjoint affine algorithm."""
    b = None if db is None else _ptr_array(db)
    _check(lib().distdl_affine_adj_params(nb, nfi, nfo, pfo, pfi, _ptr_array(dy), _ptr_array(x), _ptr_array(dw), b,
                                          _stream(stream)))


def conv_adj_params_workspace(part, kh, kw):
    """Bytes of device scratch conv_adj_params needs for this partition on the current device."""
    n = ctypes.c_int64(0)
    _check(lib().distdl_conv_adj_params_workspace(part.handle, kh, kw, ctypes.byref(n)))
    return n.value


def conv_adj_params(part, x, dy, kernel, dw, db, workspace, stream=None):
    """dw [C, kh, kw] and db [C] (or None) of the adjoint convolution algorithm; workspace: a uint8 tensor."""
    _check(lib().distdl_conv_adj_params(part.handle, _ptr_array(x), _ptr_array(dy), kernel[0], kernel[1], _ptr(dw),
                                        _ptr(db), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                        _stream(stream)))


def device_status(stream=None):
    """Synchronises the stream and raises DistdlError(DISTDL_ERR_TIMEOUT) if an affine kernel gave up."""
    _check(lib().distdl_device_status(_stream(stream)))


def selftest_wait_timeout(limit_cycles, stream=None):
    """Runs the bounded wait of the tensor-core kernels on a barrier nobody signals (include/distdl_selftest.h);
    the following device_status() raises DistdlError(DISTDL_ERR_TIMEOUT) once."""
    _check(lib().distdl_selftest_wait_timeout(int(limit_cycles), _stream(stream)))


def selftest_row_plan(part, adjoint=False):
    """(header words, list of 16-word records) of a partition's row plan (include/distdl_selftest.h): of H, or of
    the row ends of H*."""
    hdr = (ctypes.c_int32 * 64)()
    rec = (ctypes.c_int32 * (16 * 64))()
    n = ctypes.c_int32(0)
    _check(lib().distdl_selftest_row_plan(part.handle, 1 if adjoint else 0, hdr, 64, rec, 16 * 64, ctypes.byref(n)))
    return list(hdr), [list(rec[16 * i:16 * i + 16]) for i in range(n.value)]
