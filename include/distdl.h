/*
 * distdl.h -- C ABI of the linear data-movement operators of Hewett & Grady,
 * "A Linear Algebraic Approach to Model Parallelism in Deep Learning", and of
 * the two distributed layers built from them, for P virtual workers whose
 * shards all live in the memory of one GPU (sm_100a).
 *
 * General conventions
 *   - Every data buffer is DEVICE memory owned by the caller.  Arrays of
 *     pointers (`void *const *`) and arrays of shapes are HOST arrays; they are
 *     read during the call and need not outlive it.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Operator calls validate on the host, enqueue their kernels on
 *     that stream and return without synchronising.
 *   - Every function returns a distdl_status_t.  On any error nothing is
 *     launched; distdl_last_error() gives a thread-local message.  No function
 *     aborts, throws or traps on the device.
 *   - Every data pointer must be 16-byte aligned (DISTDL_ERR_ALIGNMENT).
 *   - Workers are numbered by the row-major index of their partition
 *     coordinate, last dimension fastest (Appendix B.2: in a 2 x 2 partition
 *     workers 0,1 are the top row, 2,3 the bottom row).
 *   - A shard is one contiguous row-major array of the padded shape
 *     bulk[k] + halo_lo[k] + halo_hi[k]; the bulk (the part the worker owns,
 *     Section 3 "Halo exchange") starts at index halo_lo[k] in each dimension.
 *   - The library allocates device memory only inside distdl_partition_create* and
 *     distdl_repartition_create (plan tables of a few KB to a few hundred KB, freed by the
 *     matching destroy call).  The calls that need scratch (the *_adj_params of the
 *     convolution layers) take it from the caller.
 */
#ifndef DISTDL_H
#define DISTDL_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DISTDL_OK = 0,
    DISTDL_ERR_INVALID_ARG = 1, /* NULL pointer, bad count, forbidden aliasing           */
    DISTDL_ERR_SHAPE = 2,       /* shapes / partition / halo widths inconsistent          */
    DISTDL_ERR_ALIGNMENT = 3,   /* a data pointer is not 16-byte aligned                  */
    DISTDL_ERR_UNSUPPORTED = 4, /* valid request outside what is implemented              */
    DISTDL_ERR_CUDA = 5,        /* a CUDA runtime call failed (message has the detail)    */
    DISTDL_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out (affine kernels)    */
    DISTDL_ERR_NOMEM = 7
} distdl_status_t;

typedef enum { DISTDL_F32 = 0, DISTDL_BF16 = 1, DISTDL_F64 = 2 } distdl_dtype_t;

#define DISTDL_MAX_RANK 5
#define DISTDL_MAX_WORKERS 256

typedef struct distdl_partition distdl_partition_t; /* opaque, immutable after create */

/* ------------------------------------------------------------------------
 * Partition and halo geometry (host planner).
 *
 * Section 4: a rank-d tensor is partitioned along each dimension by a d-length
 * partition vector of worker counts.  Section 3 / Appendix B: each extent is
 * split evenly (n = q*p + r, the first r workers get q+1 -- the rule read from
 * the index lists of Figs. B1-B4) and every side of every dimension of every
 * worker may carry its own ghost width.
 *
 * distdl_partition_create: the same width halo_lo[k] / halo_hi[k] on the low /
 *   high side of dimension k for every worker (NULL = all zero).  Ghosts on the
 *   tensor's own boundary exist too and stand for zero padding (Fig. B1).
 * distdl_partition_create_general: halo_lo[k] / halo_hi[k] point to
 *   partition_shape[k] widths, one per worker coordinate along dimension k
 *   (the unbalanced halos of Figs. B2-B4 and Appendix B.2).
 *
 * rank 1..DISTDL_MAX_RANK; product of partition_shape <= DISTDL_MAX_WORKERS;
 * global_shape[k] >= partition_shape[k]; a ghost may not be wider than the
 * adjacent worker's bulk (the paper assumes data from directly adjacent
 * workers only) -> DISTDL_ERR_SHAPE.  The plan tables are uploaded with a
 * synchronous copy on the current device.  *out is written only on success.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_partition_create(int32_t rank, const int64_t *global_shape,
                                        const int32_t *partition_shape,
                                        const int32_t *halo_lo, const int32_t *halo_hi,
                                        distdl_dtype_t dtype, distdl_partition_t **out);
distdl_status_t distdl_partition_create_general(int32_t rank, const int64_t *global_shape,
                                                const int32_t *partition_shape,
                                                const int32_t *const *halo_lo,
                                                const int32_t *const *halo_hi,
                                                distdl_dtype_t dtype, distdl_partition_t **out);
/* The same as distdl_partition_create with periodic[k] != 0 marking dimensions that wrap around: the
 * first and the last worker along such a dimension are neighbours (a worker alone along it is its own
 * neighbour), and the ghosts on that boundary of the tensor receive the cells from the other end
 * instead of zeros; H* adds them back there.  The paper's exchange stops at the tensor's boundary;
 * this is the same operator sequence with one more pair of neighbours per periodic dimension.
 * periodic == NULL: no dimension is periodic.  The fused layers (conv, pool, stencil3d) do not take
 * periodic partitions (DISTDL_ERR_UNSUPPORTED). */
distdl_status_t distdl_partition_create_periodic(int32_t rank, const int64_t *global_shape,
                                                 const int32_t *partition_shape,
                                                 const int32_t *halo_lo, const int32_t *halo_hi,
                                                 const int32_t *periodic, distdl_dtype_t dtype,
                                                 distdl_partition_t **out);
void distdl_partition_destroy(distdl_partition_t *p); /* NULL is allowed */
int32_t distdl_partition_num_workers(const distdl_partition_t *p); /* -1 if p is NULL */

/* Extents of one worker's shard; each output array has `rank` entries and may be NULL. */
distdl_status_t distdl_partition_shard_extents(const distdl_partition_t *p, int32_t worker,
                                               int64_t *bulk_start, int64_t *bulk_shape,
                                               int64_t *padded_shape, int32_t *halo_lo,
                                               int32_t *halo_hi);

/* Size of the host-built plan of H (adjoint = 0) or H* (adjoint != 0): number of boxes (one per
 * shard and neighbour direction), number of thread-block tiles, and the algorithmic bytes of one
 * application of the in-place method (H: every interior ghost cell read once from its owner and
 * every ghost cell written once; H*: every receiving bulk cell read and written once, every
 * interior ghost read once, every ghost cleared once).  Host only; outputs may be NULL. */
distdl_status_t distdl_partition_halo_stats(const distdl_partition_t *p, int32_t adjoint,
                                            int64_t *boxes, int64_t *tiles, int64_t *bytes);

/* Halo widths of a 1-D sliding kernel (Section 3, "Halo exchange": the widths follow from the first
 * and the last input index that a worker's own outputs touch, hence from the kernel's size, stride,
 * dilation and padding; worked cases: Figs. B1-B4).  Input length n and the output length
 * floor((n + pad_lo + pad_hi - dilation*(kernel-1) - 1)/stride) + 1 are both split evenly over p
 * workers.  Host only.  Each output array has p entries and may be NULL: halo widths, and the
 * count of owned inputs at either end that the worker's outputs never read. */
distdl_status_t distdl_halo_widths_1d(int64_t n, int32_t p, int32_t kernel, int32_t stride,
                                      int32_t dilation, int32_t pad_lo, int32_t pad_hi,
                                      int32_t *halo_lo, int32_t *halo_hi,
                                      int32_t *unused_lo, int32_t *unused_hi);

/* ------------------------------------------------------------------------
 * Broadcast B and sum-reduce R = B* (Section 3, "Broadcast", "Sum-reduce").
 *
 * broadcast_fwd:  dst[i][e] = src[e], i < k          (B = k copies)
 * sumreduce_fwd:  dst[e] = ((src[0][e] + src[1][e]) + ...) + src[k-1][e]
 *                 in the arithmetic of `t`, fixed worker order, starting from src[0]
 *                 (k = 1 is an exact copy).
 * broadcast_adj == sumreduce_fwd, sumreduce_adj == broadcast_fwd (R = B*, R* = B).
 *
 * n = elements per realisation (n = 0 is a no-op), 1 <= k.  In broadcast a dst[i] equal to
 * src is the in-place form (identity copy, skipped); any other overlap between buffers is not
 * detected and gives undefined results.  In sum-reduce dst may equal src[0] only.
 * F32, BF16 and F64, for the copies and for the sums: every addition is the exact sum of its two
 * operands rounded once to the type, to nearest even (fp32 / fp64 IEEE addition; bfloat16: add.rn.bf16).
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_broadcast_fwd(const void *src, void *const *dst, int32_t k, int64_t n,
                                     distdl_dtype_t t, void *stream);
distdl_status_t distdl_broadcast_adj(const void *const *dy, void *dx, int32_t k, int64_t n,
                                     distdl_dtype_t t, void *stream);
distdl_status_t distdl_sumreduce_fwd(const void *const *src, void *dst, int32_t k, int64_t n,
                                     distdl_dtype_t t, void *stream);
distdl_status_t distdl_sumreduce_adj(const void *dy, void *const *dx, int32_t k, int64_t n,
                                     distdl_dtype_t t, void *stream);

/* ------------------------------------------------------------------------
 * Broadcast and sum-reduce along partition dimensions (Section 4, "Sparse layers": the broadcasts
 * B_{P_x -> P_w} and reductions R_{P_w -> P_y} of the forward and adjoint convolution algorithms and
 * the two footnotes on broadcasting along partitions; "Dense layers": the same operators in the
 * affine algorithms).
 *
 * Two Cartesian worker partitions of the same rank: along every dimension the destination has as
 * many workers as the source, or the source has exactly one (NumPy's broadcasting rule on the two
 * partition shapes, from source to destination only).  Worker ids are row-major in both.  The
 * destination worker with coordinates c copies the source worker whose coordinates are c where
 * the source partition has several workers and 0 where it has one.
 *   partition_broadcast_fwd: dst[w] <- src[source of w]  for every w < Pdst (bit copies)
 *   partition_broadcast_adj: dx[j] <- sum of dy[w] over the destination workers w whose source is
 *       j, in ascending w, starting from the first (one addition per element and term, rounded
 *       once to the type): the sum-reduce R = B*, e.g. y <- R y^ with the roles of the two
 *       partitions as here (the smaller one receives).
 * elems[j]: elements of source worker j's realisation (its copies have the same size), j < Psrc.
 * src / dx: Psrc device pointers; dst / dy: Pdst device pointers (host arrays); all 16-byte
 * aligned.  A dst[w] equal to its source is left alone (the in-place form of the broadcast); dx[j]
 * may alias the first of its terms only.  rank 1..DISTDL_MAX_RANK, Pdst <= DISTDL_MAX_WORKERS.
 * Errors: DISTDL_ERR_SHAPE for partition shapes that do not broadcast, else as broadcast_fwd.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_partition_broadcast_fwd(int32_t rank, const int32_t *src_partition_shape,
                                               const int32_t *dst_partition_shape, const int64_t *elems,
                                               const void *const *src, void *const *dst, distdl_dtype_t t,
                                               void *stream);
distdl_status_t distdl_partition_broadcast_adj(int32_t rank, const int32_t *src_partition_shape,
                                               const int32_t *dst_partition_shape, const int64_t *elems,
                                               const void *const *dy, void *const *dx, distdl_dtype_t t,
                                               void *stream);

/* ------------------------------------------------------------------------
 * Halo exchange H and its adjoint H* (Section 3, "Halo exchange": the H and H* operator
 * sequences; Appendix B.2), in place on the P padded shards.
 *
 * halo_fwd: every ghost cell <- the bulk cell with the same global index (owned by a
 *   neighbouring worker), or +0 where that index lies outside the tensor.  Bulk cells are
 *   not written; previous ghost contents are never read.
 * halo_adj: every bulk cell that some neighbour holds ghost copies of <- itself plus those
 *   copies, summed in the nested order of H* (dimension d-1 undone first, so the sum is
 *   grouped by dimension 0 outermost; within a dimension: own, low neighbour, high neighbour);
 *   then every ghost cell <- 0.  Additions in the partition's type (F32, BF16 or F64), each rounded once.
 * shards[w] = device pointer of worker w's padded shard, w < P (host array).
 * Shards must not overlap one another.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_halo_fwd(const distdl_partition_t *p, void *const *shards, void *stream);
distdl_status_t distdl_halo_adj(const distdl_partition_t *p, void *const *shards, void *stream);
/* 1 if H (adjoint = 0) of this partition runs through the row plan -- every ghost width and bulk extent of
 * the innermost dimension is a whole number of 16-byte units, so ghost rows are moved end to end as aligned
 * vectors and the ghosts at the row ends are staged through shared memory -- or (adjoint != 0) if H* hands
 * the row ends to it: besides the above, every bulk is at least as wide as the ghosts its two neighbours
 * hold of it together, and the innermost dimension has neighbours.  0 if the general box plan does all the
 * work, -1 for a NULL partition.  Same results, bit for bit, either way. */
int32_t         distdl_partition_uses_row_plan(const distdl_partition_t *p, int32_t adjoint);

/* ------------------------------------------------------------------------
 * distdl_halo_fwd_noalloc: the halo exchange H for callers that must not allocate device memory.
 * (An addition of this library; the paper has no counterpart.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits -- inside a service whose
 * device memory was handed out in full at start-up, in a latency-critical loop where the implicit
 * device synchronisation of an allocation is not acceptable, or in a plug-in that is only given
 * buffers and a stream.  distdl_partition_create allocates a few KB of plan tables on the device;
 * this call does not: it computes the same plan on the host and copies it, on `stream`, into a
 * fixed array of 1 MiB that is part of the library image (so every GPU that loads the library
 * holds that 1 MiB until the process exits).  It calls no cudaMalloc, no cudaFree and no
 * allocating library routine; its only host-side scratch is ordinary heap memory, freed on return.
 *
 * Arguments: the geometry arguments of distdl_partition_create (uniform widths) and the shard
 * pointers of distdl_halo_fwd; same result as distdl_halo_fwd, bit for bit.
 * Limits: the plan tables (128 B per box, 48 B per copy source, 32 B per 64 KB tile) must fit in
 * the 1 MiB array, else DISTDL_ERR_UNSUPPORTED with the sizes in the message -- e.g. 64 workers
 * in 3-D with 128^3 shards need about 0.36 MiB, 256 workers in 3-D do not fit.
 * The first call on a device looks up the device address of the array (one cudaGetSymbolAddress
 * with that device current).  No call may be made on a stream that is being captured: the tables
 * are copied from host memory that is freed on return, so the call answers DISTDL_ERR_UNSUPPORTED
 * there and records nothing.  Like any copy from pageable host memory, the table copies may also
 * keep the host waiting until earlier work on `stream` has drained.
 * All calls share the one array: the tables of the previous call stay in it and are overwritten,
 * entry by entry as far as the new plan reaches, before the kernel of this call reads them.  Two
 * calls whose work overlaps on the GPU (different streams, no ordering between them) race on the
 * array and give undefined results; calls on one stream are safe.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_halo_fwd_noalloc(int32_t rank, const int64_t *global_shape,
                                        const int32_t *partition_shape, const int32_t *halo_lo,
                                        const int32_t *halo_hi, distdl_dtype_t dtype,
                                        void *const *shards, void *stream);

/* ------------------------------------------------------------------------
 * Generalized all-to-all, scatter / gather, all-reduce (Section 3, "Scatter and Gather",
 * "Sum-reduce and all-reduce", "Generalized all-to-all").
 *
 * A repartition object describes one tensor under two Cartesian partitions without ghosts, both
 * split evenly (src_partition_shape -> dst_partition_shape; at most DISTDL_MAX_WORKERS workers in
 * both together).  The all-to-all moves every cell from the worker that owns it in the source
 * partition to its owner in the destination partition: a block permutation whose blocks are
 * send-receive copies, one per pair of workers whose blocks intersect.  A source partition of one
 * worker is the scatter, a destination partition of one worker the gather.
 *   repartition_fwd: dst[Pdst] <- src[Psrc]   (contiguous row-major blocks, bit copies)
 *   repartition_adj: dx[Psrc] <- dy[Pdst]     (every copy is a move, so the adjoint is the
 *                                              inverse: the all-to-all back)
 * Outputs may overlap neither each other nor any input (DISTDL_ERR_INVALID_ARG).  F32, BF16 and F64.
 * repartition_shard_shape: extents of one worker's block (destination != 0: in the destination
 * partition); `shape` has rank entries.
 *
 * allreduce: A = B R on k buffers of n elements in place: every buffer ends up holding
 * ((b[0] + b[1]) + ...) + b[k-1] (fixed order, in the arithmetic of `t`); self-adjoint.  Two launches.
 * ---------------------------------------------------------------------- */
typedef struct distdl_repartition distdl_repartition_t; /* opaque, immutable after create */
distdl_status_t distdl_repartition_create(int32_t rank, const int64_t *global_shape,
                                          const int32_t *src_partition_shape,
                                          const int32_t *dst_partition_shape, distdl_dtype_t dtype,
                                          distdl_repartition_t **out);
void distdl_repartition_destroy(distdl_repartition_t *r); /* NULL is allowed */
distdl_status_t distdl_repartition_shard_shape(const distdl_repartition_t *r, int32_t destination,
                                               int32_t worker, int64_t *shape);
distdl_status_t distdl_repartition_fwd(const distdl_repartition_t *r, const void *const *src,
                                       void *const *dst, void *stream);
distdl_status_t distdl_repartition_adj(const distdl_repartition_t *r, const void *const *dy,
                                       void *const *dx, void *stream);
distdl_status_t distdl_allreduce(void *const *bufs, int32_t k, int64_t n, distdl_dtype_t t,
                                 void *stream);

/* ------------------------------------------------------------------------
 * Distributed convolution layer, feature-space partition only (Section 4, "Sparse layers":
 * forward / adjoint convolution algorithms and the closing remark that the broadcasts and
 * reductions drop out when only the feature space is partitioned).
 *
 * p: rank-4 NCHW F32 partition of shape 1 x 1 x Ph x Pw whose halo widths are (kh-1)/2 rows and
 *    (kw-1)/2 columns on every side (else DISTDL_ERR_SHAPE).  Depthwise, centred, stride 1,
 *    kh = kw in {3, 5, 7} (else DISTDL_ERR_UNSUPPORTED).
 * conv_fwd = H then the local cross-correlation, fused: y[n,c,i,j] = bias[c] +
 *    sum_{a,b} w[c,a,b] * x[n,c,i+a-ph,j+b-pw] over the GLOBAL tensor with zeros outside.
 *    x[w]: padded shards (only their bulk is read; ghost storage is neither read for its value
 *    nor written).  y[w]: bulk-shaped shards (no ghosts).  w: [C,kh,kw] F32.  bias: [C] or NULL.
 * conv_adj = local adjoint then H*, fused: dx[n,c,p,q] = sum_{a,b} w[c,a,b] *
 *    dy[n,c,p-a+ph,q-b+pw] (zeros outside), written to the bulk of the padded shards dx[w],
 *    whose ghosts are set to zero.  dy[w]: bulk-shaped shards.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_conv_fwd(const distdl_partition_t *p, const void *const *x, const void *w,
                                const void *bias, int32_t kh, int32_t kw, void *const *y,
                                void *stream);
distdl_status_t distdl_conv_adj(const distdl_partition_t *p, const void *const *dy, const void *w,
                                int32_t kh, int32_t kw, void *const *dx, void *stream);


/* Parameter gradients of the convolution layer (Section 4, "Sparse layers", adjoint convolution
 * algorithm: dw^, db^ <- [dConv]*(dy^) on every worker, then dw <- R dw^, db <- R db^; with a
 * feature-space partition every worker holds a copy of the kernel, so the sum runs over all workers).
 *   dw[c,a,b] = sum over workers k and n,i,j of dy_k[n,c,i,j] * (H x)_k[n,c,i+a,j+b]   (padded-local i+a, j+b)
 *             = sum_{n,i,j} dy[n,c,i,j] * x[n,c,i+a-ph,j+b-pw] on the global tensor, zeros outside;
 *   db[c]     = sum_{n,i,j} dy[n,c,i,j].
 * Same partition and kernel restrictions as conv_fwd.  x[w]: padded shards (only the bulk is read: the
 * halo exchange is fused, ghost storage is not touched); dy[w]: bulk-shaped shards; dw: [C,kh,kw] F32;
 * db: [C] F32 or NULL.  Sums are taken in fp32 in a fixed order that depends only on the shapes and
 * on the device (number of SMs): per-thread running sums over a static set of tiles, a tree over the
 * threads of a block, then the blocks' partial results in order -- the same bits on every run.
 * workspace: device scratch of at least the size conv_adj_params_workspace reports (a few hundred
 * KB), overwritten by the call; the caller may reuse it once the call's work on `stream` is done.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_conv_adj_params_workspace(const distdl_partition_t *p, int32_t kh, int32_t kw,
                                                 int64_t *bytes);
distdl_status_t distdl_conv_adj_params(const distdl_partition_t *p, const void *const *x,
                                       const void *const *dy, int32_t kh, int32_t kw, void *dw,
                                       void *db, void *workspace, int64_t workspace_bytes,
                                       void *stream);

/* ------------------------------------------------------------------------
 * Generalized convolution layer: channels partitioned as well (Section 4, "Sparse layers": the forward /
 * adjoint convolution algorithms with x on 1 x P_ci x P_0 x P_1, y on 1 x P_co x P_0 x P_1, the weights on
 * P_co x P_ci and the work partition 1 x P_co x P_ci x P_0 x P_1).
 *
 * px: rank-4 NCHW F32 partition of x, shape 1 x P_ci x P_0 x P_1, halo widths (0, 0, (kh-1)/2, (kw-1)/2) on
 *     every side; worker (j, r, c) has id (j*P_0 + r)*P_1 + c.  nco output channels are split evenly over pco
 *     blocks; y / dy live on 1 x pco x P_0 x P_1, worker (i, r, c) has id (i*P_0 + r)*P_1 + c.
 *     P_ci, pco <= 8; at most 64 shards per tensor; kh = kw in {3, 5, 7}, stride 1, centred.
 * w[i*P_ci + j]: F32 [nco_i, nci_j, kh, kw], the block of worker (i, j) of the weight partition.
 * bias[i]: F32 [nco_i], or bias == NULL (the bias lives on the j = 0 subpartition: added once).
 * convg_fwd: x <- H x; x^ <- B x (to the pco copies of the work partition); y^_{ijs} <- Conv(w_ij, b_i on j = 0;
 *     x^_js); y_is <- R over j = 0..P_ci-1 in order -- fused: y[n,o,p] = b[o] + sum over input channels c
 *     (block after block, channel after channel) and taps of w[o,c,a,b] * x[n,c,p + (a,b) - pad] on the
 *     GLOBAL tensor, zeros outside.  x[.]: padded shards (bulk read only); y[.]: bulk-shaped shards.
 * convg_adj: dy^ <- B dy; dx^_{ijs} <- [dConv]*(dy^_{ijs}); dx_js <- R over i in order; dx <- H* dx -- fused in
 *     gather form: dx[n,c,p] = sum over output channels o and taps of w[o,c,a,b] * dy[n,o,p - (a,b) + pad];
 *     dy[.]: bulk-shaped shards; dx[.]: padded shards whose ghosts are set to zero.
 * convg_adj_params: the parameter part of the adjoint algorithm: dw^_{ijs}, db^_{ijs} <- [dConv]*(dy^_{ijs}) with the
 *     exchanged x^_{js} of the forward pass, then dw_ij <- R over the feature-space workers s, db_i <- R over s
 *     (from the j = 0 workers): dw[i*P_ci + j] F32 [nco_i, nci_j, kh, kw] with
 *     dw[o,c,a,b] = sum_{n,p} dy[n,o,p] * x[n,c,p + (a,b) - pad] on the GLOBAL tensors; db[i] F32 [nco_i] (db may be
 *     NULL).  x[.]: padded shards (bulk read only, the exchange is fused); dy[.]: bulk-shaped shards.  Sums in
 *     fp32 in a fixed order (running sums over a static set of tiles, lanes, warps, then the slices of a
 *     channel pair in order).  workspace: device scratch of the size convg_adj_params_workspace reports.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_convg_fwd(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                 const void *const *x, const void *const *w, const void *const *bias,
                                 int32_t kh, int32_t kw, void *const *y, void *stream);
distdl_status_t distdl_convg_adj(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                 const void *const *dy, const void *const *w, int32_t kh, int32_t kw,
                                 void *const *dx, void *stream);
distdl_status_t distdl_convg_adj_params_workspace(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                                  int32_t kh, int32_t kw, int64_t *bytes);
distdl_status_t distdl_convg_adj_params(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                        const void *const *x, const void *const *dy, int32_t kh,
                                        int32_t kw, void *const *dw, void *const *db, void *workspace,
                                        int64_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------
 * Distributed star-stencil layer on a rank-3 tensor (Section 4, "Sparse layers": on a feature-space
 * partition a sliding-kernel layer is the halo exchange followed by the local kernel, its adjoint the
 * local adjoint followed by H*; Section 6 names large volumetric data as the target).
 *
 * p: rank-3 F32 partition, at most 8 workers along a dimension and 64 in all, whose halo widths equal
 *    `radius` (1..4) on every side of every dimension (else DISTDL_ERR_SHAPE).
 * w: HOST array [3][2*radius+1]: w[d][k+radius] is the tap at offset k along dimension d.
 * stencil3d_fwd = H then the local kernel, fused:
 *    y[i] = sum_d sum_{k=-radius..radius} w[d][k+radius] * x[i + k e_d] over the GLOBAL tensor, zeros outside.
 *    x[w]: padded shards (only their bulk is read; ghost storage is neither read nor written);
 *    y[w]: bulk-shaped shards.  6*radius+3 fp32 FMAs per output, z taps first, then y, then x.
 * stencil3d_adj = local adjoint then H*, fused (gather form):
 *    dx[i] = sum_d sum_k w[d][k+radius] * dy[i - k e_d] (zeros outside), written to the bulk of the
 *    padded shards dx[w], whose ghosts are set to zero.  dy[w]: bulk-shaped shards.
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_stencil3d_fwd(const distdl_partition_t *p, const void *const *x, const float *w,
                                     int32_t radius, void *const *y, void *stream);
distdl_status_t distdl_stencil3d_adj(const distdl_partition_t *p, const void *const *dy, const float *w,
                                     int32_t radius, void *const *dx, void *stream);

/* ------------------------------------------------------------------------
 * Distributed pooling layer, feature-space partition only (Section 4, "Sparse layers": pooling
 * layers follow the convolution algorithms; Section 3 / Appendix B: for a strided kernel the halo
 * widths differ from worker to worker and owned inputs may go unused, Figs. B2-B4).
 *
 * p: rank-4 NCHW F32 partition of shape 1 x 1 x Ph x Pw (at most 32 workers) made by
 *    distdl_partition_create_general with, in each feature dimension, exactly the widths
 *    distdl_halo_widths_1d gives for (kernel, stride, dilation 1, padding) -- else
 *    DISTDL_ERR_SHAPE.  Kernel extents up to 16.  Worker (r, c) owns block r / c of the evenly
 *    split output rows / columns.
 * pool_fwd = H on x in place (its ghosts are overwritten), then the local layer:
 *    AVG: y = mean of the kh x kw window of the zero-padded tensor (padding counts in the
 *         divisor), summed in fp32 in row-major window order, times 1/(kh*kw);
 *    MAX: y = largest value of the window clipped to the tensor; argmax (may be NULL) receives
 *         a*kw + b of the first largest value in row-major order of the unclipped window.
 *    x[w]: padded shards.  y[w], argmax[w]: [N, C, oh, ow] F32 / int32.
 * pool_adj = adjoint of the local layer into every cell of the padded dx[w] (a cell sums, in
 *    ascending output order and in fp32, dy/(kh*kw) over the local outputs whose window holds it;
 *    for MAX: dy of the outputs whose recorded position is that cell), then H* on dx in place:
 *    ghost contributions are added into the owners' bulk and the ghosts are cleared.
 * ---------------------------------------------------------------------- */
typedef enum { DISTDL_POOL_AVG = 0, DISTDL_POOL_MAX = 1 } distdl_pool_mode_t;
distdl_status_t distdl_pool_fwd(const distdl_partition_t *p, void *const *x, int32_t kh, int32_t kw,
                                int32_t sh, int32_t sw, int32_t pad_h_lo, int32_t pad_h_hi,
                                int32_t pad_w_lo, int32_t pad_w_hi, int32_t mode, void *const *y,
                                void *const *argmax, void *stream);
distdl_status_t distdl_pool_adj(const distdl_partition_t *p, const void *const *dy,
                                const void *const *argmax, int32_t kh, int32_t kw, int32_t sh,
                                int32_t sw, int32_t pad_h_lo, int32_t pad_h_hi, int32_t pad_w_lo,
                                int32_t pad_w_hi, int32_t mode, void *const *dx, void *stream);

/* ------------------------------------------------------------------------
 * Distributed affine layer on a Pfo x Pfi worker grid (Section 4, "Dense layers": forward and
 * adjoint affine algorithms).
 *
 * affine_fwd: x^_{ij} <- B x_j (along grid columns); y^_{ij} <- x^_{ij} W_{ij}^T (+ b_i on
 *   column j = 0 only: the "one Pfo x 1 subset"); y_i <- R over j = 0..Pfi-1 in order.
 * affine_adj: dy^_{ij} <- B dy_i (along grid rows); dx^_{ij} <- dy^_{ij} W_{ij};
 *   dx_j <- R over i = 0..Pfo-1 in order.  (dW, db are not computed.)
 * x[j]  BF16 [nb, nfi/Pfi]      w[i*Pfi+j]  BF16 [nfo/Pfo, nfi/Pfi]  (row-major)
 * y[i]  F32  [nb, nfo/Pfo]      bias[i] F32 [nfo/Pfo] or bias == NULL
 * dy[i] BF16 [nb, nfo/Pfo]      dx[j] F32 [nb, nfi/Pfi]
 * The contraction runs on the tensor cores with fp32 accumulation; the sums of R continue in the
 * same fp32 accumulator in the stated order.  nfi % Pfi == 0, nfo % Pfo == 0 (else
 * DISTDL_ERR_SHAPE); the per-worker block sizes nfi/Pfi and nfo/Pfo must be multiples of 8 (rows of
 * whole 16-byte units; tiles that reach past a block are filled with zeros on the way in and clipped
 * on the way out), Pfo, Pfi <= 8 and Pfo * Pfi <= 16 (else DISTDL_ERR_UNSUPPORTED); nb >= 1 is arbitrary.
 * A launch whose device-side waits ran out reports through distdl_device_status().
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_affine_fwd(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                  const void *const *x, const void *const *w,
                                  const void *const *bias, void *const *y, void *stream);
distdl_status_t distdl_affine_adj(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                  const void *const *dy, const void *const *w, void *const *dx,
                                  void *stream);

/* Parameter gradients of the affine layer (Section 4, "Dense layers", adjoint affine algorithm:
 * dW^, db^ <- [dAffine]*(dy^) with dy^_{ij} = dy_i and the x^_{ij} = x_j of the forward pass; the
 * weights are distributed on the worker grid itself, so no reduction follows).
 *   dw[i*Pfi+j]  F32 [nfo/Pfo, nfi/Pfi]   dW_{ij}[o,f] = sum_b dy_i[b,o] * x_j[b,f]
 *   db[i]        F32 [nfo/Pfo] (db may be NULL)   db_i[o] = sum_b dy_i[b,o]   (bias lives on column j = 0)
 * dy[i] BF16 [nb, nfo/Pfo], x[j] BF16 [nb, nfi/Pfi].  Tensor cores with fp32 accumulation over the
 * batch in ascending order (dW); db in fp32, eight contiguous chunks of the batch added in order.
 * Same shape restrictions as affine_fwd.  Bounded waits report through distdl_device_status().
 * ---------------------------------------------------------------------- */
distdl_status_t distdl_affine_adj_params(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo,
                                         int32_t pfi, const void *const *dy, const void *const *x,
                                         void *const *dw, void *const *db, void *stream);

/* Synchronises `stream`, then reads and clears the device status word that the affine kernels set
 * when one of their bounded waits (on a shared-memory barrier fed by TMA or by the tensor cores)
 * ran out: DISTDL_ERR_TIMEOUT in that case (the outputs of that launch are then undefined),
 * DISTDL_OK otherwise.  The only call of this library that blocks the host. */
distdl_status_t distdl_device_status(void *stream);

/* Thread-local message of the last error returned on this thread ("" if none). */
const char *distdl_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DISTDL_H */
