// Halo exchange H and adjoint halo exchange H* (Section 3, "Halo exchange") as gather kernels
// over a host-planned list of boxes.
//
// The paper runs the exchange as d nested pack / exchange / unpack phases so that corner data
// reaches its destination in d hops between distributed memories.  Here every shard sits in the
// same device memory, so each ghost cell is fetched straight from the bulk cell that owns its
// global index (one read, one write), and the adjoint is evaluated per receiving bulk cell as the
// same nested sum the d reversed phases would produce -- own value, low neighbour, high
// neighbour within a dimension; dimension 0 outermost -- so the result is bit-identical to the
// phase-by-phase order.  Each ghost cell is read by exactly one thread, which also clears it.
#include <cstdlib>
#include <cstring>

#include "common.h"

namespace distdl {

struct ShardPointers {
    void *p[DISTDL_MAX_WORKERS];
};

constexpr int kHaloThreads = 256;

// Element and 16-byte vector types of the sums, one addition per element, each the exact sum rounded
// once to the type (fp32 / fp64 IEEE addition, add.rn.bf16).
struct bf16x1 {
    unsigned short v;
};
struct bf16x8 {
    uint4 v;
};
__device__ __forceinline__ uint32_t halo_add_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ float4 vadd(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float vadd(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ double2 vadd(double2 a, double2 b) { return make_double2(__dadd_rn(a.x, b.x), __dadd_rn(a.y, b.y)); }
__device__ __forceinline__ double vadd(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ bf16x8 vadd(bf16x8 a, bf16x8 b) {
    bf16x8 r;
    r.v.x = halo_add_bf16x2(a.v.x, b.v.x);
    r.v.y = halo_add_bf16x2(a.v.y, b.v.y);
    r.v.z = halo_add_bf16x2(a.v.z, b.v.z);
    r.v.w = halo_add_bf16x2(a.v.w, b.v.w);
    return r;
}
__device__ __forceinline__ bf16x1 vadd(bf16x1 a, bf16x1 b) {
    bf16x1 r;
    asm("add.rn.bf16 %0, %1, %2;" : "=h"(r.v) : "h"(a.v), "h"(b.v));
    return r;
}

template <typename T> __device__ __forceinline__ T zero_of();
template <> __device__ __forceinline__ float4 zero_of<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float zero_of<float>() { return 0.f; }
template <> __device__ __forceinline__ uint4 zero_of<uint4>() { return make_uint4(0, 0, 0, 0); }
template <> __device__ __forceinline__ unsigned short zero_of<unsigned short>() { return 0; }
template <> __device__ __forceinline__ unsigned long long zero_of<unsigned long long>() { return 0ull; }
template <> __device__ __forceinline__ double2 zero_of<double2>() { return make_double2(0.0, 0.0); }
template <> __device__ __forceinline__ double zero_of<double>() { return 0.0; }
template <> __device__ __forceinline__ bf16x8 zero_of<bf16x8>() { return bf16x8{make_uint4(0, 0, 0, 0)}; }
template <> __device__ __forceinline__ bf16x1 zero_of<bf16x1>() { return bf16x1{0}; }

// Coordinates of flattened unit n inside the box (innermost dimension last).
__device__ __forceinline__ void decompose(const HaloBox &box, uint32_t n, uint32_t *coord) {
#pragma unroll
    for (int k = kMaxBoxDims - 1; k >= 1; --k) {
        coord[k] = 0;
        if (k < box.ndim) {
            const uint32_t q = __umulhi(n, box.magic[k]) >> box.shift[k];
            coord[k] = n - q * box.shape[k];
            n = q;
        }
    }
    coord[0] = n;
}

__device__ __forceinline__ uint32_t dot_stride(const uint32_t *coord, const uint32_t *stride, int nd) {
    uint32_t o = 0;
#pragma unroll
    for (int k = 0; k < kMaxBoxDims; ++k)
        if (k < nd) o += coord[k] * stride[k];
    return o;
}

// ---------------------------------------------------------------------------------------------
// Copy / clear tile (H, and the ghost clears of H*): T = uint4 (16 bytes), float, unsigned short.
// Each thread keeps kCopyBatch independent loads in flight.
// ---------------------------------------------------------------------------------------------
constexpr int kCopyBatch = 8;

template <typename T>
__device__ __forceinline__ void run_copy_tile(const HaloBox &box, const HaloSource *src, int nsrc,
                                              const ShardPointers &sh, uint32_t first, uint32_t count) {
    T *dst = reinterpret_cast<T *>(sh.p[box.dst_shard]) + box.dst_offset;
    const int nd = box.ndim;
    if (nsrc == 0) {
        for (uint32_t i = threadIdx.x; i < count; i += kHaloThreads) {
            uint32_t c[kMaxBoxDims];
            decompose(box, first + i, c);
            dst[dot_stride(c, box.dst_stride, nd)] = zero_of<T>();
        }
        return;
    }
    const T *s0 = reinterpret_cast<const T *>(sh.p[src[0].shard]) + src[0].offset;
    for (uint32_t base = threadIdx.x; base < count; base += kHaloThreads * kCopyBatch) {
        T v[kCopyBatch];
        uint32_t doff[kCopyBatch];
#pragma unroll
        for (int u = 0; u < kCopyBatch; ++u) {
            const uint32_t i = base + u * kHaloThreads;
            if (i < count) {
                uint32_t c[kMaxBoxDims];
                decompose(box, first + i, c);
                doff[u] = dot_stride(c, box.dst_stride, nd);
                v[u] = s0[dot_stride(c, src[0].stride, nd)];
            }
        }
#pragma unroll
        for (int u = 0; u < kCopyBatch; ++u)
            if (base + u * kHaloThreads < count) dst[doff[u]] = v[u];
    }
}

// ---------------------------------------------------------------------------------------------
// Nested sum of H*.  Balanced case (every level has two terms, NSRC = 2^levels): all loads are
// issued first, then the ghost clears, then a fixed binary tree in source order -- which is the
// left-to-right nested fold when each level has exactly two terms.
// ---------------------------------------------------------------------------------------------
// Orders the stores that follow after the arrival of `v`: a store issued to a line whose load is
// still in flight stalls the memory pipeline badly (measured: 4x lower throughput), so every
// store of a batch waits until the batch's sums -- and with them all of its loads -- are done.
__device__ __forceinline__ void stores_after(const float4 &v) {
    asm volatile("" ::"f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void stores_after(const float &v) { asm volatile("" ::"f"(v) : "memory"); }
__device__ __forceinline__ void stores_after(const double2 &v) { asm volatile("" ::"d"(v.x), "d"(v.y) : "memory"); }
__device__ __forceinline__ void stores_after(const double &v) { asm volatile("" ::"d"(v) : "memory"); }
__device__ __forceinline__ void stores_after(const bf16x8 &v) { asm volatile("" ::"r"(v.v.x), "r"(v.v.y), "r"(v.v.z), "r"(v.v.w) : "memory"); }
__device__ __forceinline__ void stores_after(const bf16x1 &v) { asm volatile("" ::"h"(v.v) : "memory"); }

template <typename T, int NSRC>
__device__ __forceinline__ void run_sum_tile_balanced(const HaloBox &box, const HaloSource *src,
                                                      const ShardPointers &sh, uint32_t first, uint32_t count) {
    constexpr int U = NSRC >= 8 ? 1 : (NSRC == 4 ? 2 : 8);   // units per thread per batch
    const int nd = box.ndim;
    T *base[NSRC];
#pragma unroll
    for (int j = 0; j < NSRC; ++j) base[j] = reinterpret_cast<T *>(sh.p[src[j].shard]) + src[j].offset;
    for (uint32_t b0 = threadIdx.x; b0 < count; b0 += kHaloThreads * U) {
        T *ptr[U][NSRC];
        T v[U][NSRC];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = b0 + u * kHaloThreads;
            if (i < count) {
                uint32_t c[kMaxBoxDims];
                decompose(box, first + i, c);
#pragma unroll
                for (int j = 0; j < NSRC; ++j) {
                    ptr[u][j] = base[j] + dot_stride(c, src[j].stride, nd);
                    v[u][j] = *ptr[u][j];
                }
            }
        }
        // fixed binary tree in source order
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int width = 1; width < NSRC; width *= 2)
#pragma unroll
                for (int j = 0; j < NSRC; j += 2 * width) v[u][j] = vadd(v[u][j], v[u][j + width]);
#pragma unroll
        for (int u = 0; u < U; ++u) stores_after(v[u][0]);
        // source 0 is the receiving bulk cell itself; every other source is a ghost cell
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (b0 + u * kHaloThreads < count) {
                *ptr[u][0] = v[u][0];
#pragma unroll
                for (int j = 1; j < NSRC; ++j) *ptr[u][j] = zero_of<T>();
            }
        }
    }
}

// General case (a level with three terms, i.e. a shard thinner than its two neighbours' ghosts).
template <typename T>
__device__ __forceinline__ void run_sum_tile_general(const HaloBox &box, const HaloSource *src, int nsrc,
                                                     const ShardPointers &sh, uint32_t first, uint32_t count) {
    T *dst = reinterpret_cast<T *>(sh.p[box.dst_shard]) + box.dst_offset;
    const int nd = box.ndim;
    const int top = box.levels - 1;
    for (uint32_t i = threadIdx.x; i < count; i += kHaloThreads) {
        uint32_t c[kMaxBoxDims];
        decompose(box, first + i, c);
        T acc[kMaxLevels];
#pragma unroll
        for (int l = 0; l < kMaxLevels; ++l) acc[l] = zero_of<T>();
        unsigned has = 0;
#pragma unroll 4
        for (int j = 0; j < nsrc; ++j) {
            const HaloSource &s = src[j];
            const T v = *(reinterpret_cast<const T *>(sh.p[s.shard]) + s.offset + dot_stride(c, s.stride, nd));
            // absent terms are skipped, never added as zero
            acc[0] = (has & 1u) ? vadd(acc[0], v) : v;
            has |= 1u;
            const int close = s.close;
#pragma unroll
            for (int l = 0; l < kMaxLevels - 1; ++l) {
                if (l < close) {
                    acc[l + 1] = ((has >> (l + 1)) & 1u) ? vadd(acc[l + 1], acc[l]) : acc[l];
                    has |= 2u << l;
                    has &= ~(1u << l);
                }
            }
        }
        T res = acc[0];
#pragma unroll
        for (int l = 1; l < kMaxLevels; ++l)
            if (l == top) res = acc[l];
        stores_after(res);
        dst[dot_stride(c, box.dst_stride, nd)] = res;
        for (int j = 0; j < nsrc; ++j) {
            const HaloSource &s = src[j];
            if (s.clear_after)
                *(reinterpret_cast<T *>(sh.p[s.shard]) + s.offset + dot_stride(c, s.stride, nd)) = zero_of<T>();
        }
    }
}

template <typename T>
__device__ __forceinline__ void run_sum_tile(const HaloBox &box, const HaloSource *src, int nsrc,
                                             const ShardPointers &sh, uint32_t first, uint32_t count) {
    if (box.balanced && nsrc == 2) run_sum_tile_balanced<T, 2>(box, src, sh, first, count);
    else if (box.balanced && nsrc == 4) run_sum_tile_balanced<T, 4>(box, src, sh, first, count);
    else if (box.balanced && nsrc == 8) run_sum_tile_balanced<T, 8>(box, src, sh, first, count);
    else run_sum_tile_general<T>(box, src, nsrc, sh, first, count);
}

// One thread block per tile.  SUMS = false: the forward plan (copies and clears only).
template <bool SUMS>
__global__ void __launch_bounds__(kHaloThreads, SUMS ? 2 : 4)
halo_box_kernel(const HaloBox *__restrict__ boxes, const HaloSource *__restrict__ sources,
                const HaloTile *__restrict__ tiles, int32_t elem_bytes,
                const __grid_constant__ ShardPointers sh) {
    __shared__ __align__(16) HaloBox s_box;
    __shared__ __align__(16) HaloSource s_src[kMaxSources];
    // every thread reads the (uniform) tile record; box and sources are staged in shared memory
    const uint4 t0 = __ldg(reinterpret_cast<const uint4 *>(tiles + blockIdx.x));
    const uint32_t count = __ldg(&tiles[blockIdx.x].count);
    const int box_id = (int)t0.x, src_begin = (int)t0.y, nsrc = (int)t0.z;
    const uint32_t first = t0.w;
    {
        const uint32_t *g = reinterpret_cast<const uint32_t *>(boxes + box_id);
        uint32_t *s = reinterpret_cast<uint32_t *>(&s_box);
        const uint32_t bw = sizeof(HaloBox) / 4, sw = (uint32_t)nsrc * (sizeof(HaloSource) / 4);
        const uint32_t *gs = reinterpret_cast<const uint32_t *>(sources + src_begin);
        uint32_t *ss = reinterpret_cast<uint32_t *>(s_src);
        for (uint32_t i = threadIdx.x; i < bw + sw; i += kHaloThreads) {
            if (i < bw) s[i] = __ldg(g + i);
            else ss[i - bw] = __ldg(gs + (i - bw));
        }
    }
    __syncthreads();
    if (!SUMS || nsrc <= 1) {
        if (s_box.vec) run_copy_tile<uint4>(s_box, s_src, nsrc, sh, first, count);
        else if (elem_bytes == 4) run_copy_tile<float>(s_box, s_src, nsrc, sh, first, count);
        else if (elem_bytes == 8) run_copy_tile<unsigned long long>(s_box, s_src, nsrc, sh, first, count);
        else run_copy_tile<unsigned short>(s_box, s_src, nsrc, sh, first, count);
    } else if (elem_bytes == 4) {
        if (s_box.vec) run_sum_tile<float4>(s_box, s_src, nsrc, sh, first, count);
        else run_sum_tile<float>(s_box, s_src, nsrc, sh, first, count);
    } else if (elem_bytes == 8) {
        if (s_box.vec) run_sum_tile<double2>(s_box, s_src, nsrc, sh, first, count);
        else run_sum_tile<double>(s_box, s_src, nsrc, sh, first, count);
    } else {
        if (s_box.vec) run_sum_tile<bf16x8>(s_box, s_src, nsrc, sh, first, count);
        else run_sum_tile<bf16x1>(s_box, s_src, nsrc, sh, first, count);
    }
}


// ---------------------------------------------------------------------------------------------
// Row plan kernels (see FastDim): H, and the row ends of H*, for partitions whose innermost
// dimension is made of whole 16-byte units.  Kinds of block, dealt out interleaved:
//
//  * ghost-row blocks: a range of one worker's *ghost rows* -- rows of the padded array whose index
//    is a ghost index in some outer dimension.  Such a row is ghost from end to end, and consecutive
//    ghost rows are contiguous in memory, so the block writes whole runs of memory; each row is
//    fetched as (low ghost columns | bulk columns | high ghost columns) from up to three neighbours.
//  * line blocks: a range of bulk rows of all the workers that sit next to each other along the
//    innermost dimension.  There the ghosts are a few units at both ends of every row.  The ghost
//    units at the end of row r and at the start of row r + 1 are adjacent in memory, and so are the
//    bulk units that the two neighbours want from (H) or add to (H*) those rows; loads are issued in
//    the order of the source rows and stores in the order of the destination rows, with shared
//    memory in between, so that a warp touches each 128-byte line once per direction.
// ---------------------------------------------------------------------------------------------
constexpr int kFastThreads = 256;
constexpr int kFastMaxRows = 256;      // row records per block
constexpr int kFastMaxSlots = 1024;    // staged units per line block (16 KB)

struct FastRowRec {
    uint32_t dst_off;      // unit offset of the row inside the worker's array
    int32_t shard[3];      // source worker of the low ghost / bulk / high ghost columns, -1: zeros
    uint32_t off[3];       // unit offset of the source row plus the column shift
};

__device__ __forceinline__ uint32_t fast_div(uint32_t x, uint32_t magic, uint32_t shift) {
    return magic ? (__umulhi(x, magic) >> shift) : x;
}

// Which kind of block this is, and its index among the blocks of that kind.
__device__ __forceinline__ int fast_block_kind(const FastHeader &H, uint32_t *tile_id) {
    const uint32_t per_group = (uint32_t)(H.group[0] + H.group[1]);
    const uint32_t group = blockIdx.x / per_group;
    uint32_t in_group = blockIdx.x - group * per_group;
    int kind = 0;
    if (in_group >= (uint32_t)H.group[0]) {
        in_group -= (uint32_t)H.group[0];
        kind = 1;
    }
    *tile_id = group * (uint32_t)H.group[kind] + in_group;
    return kind;
}

__device__ __forceinline__ void fast_load_records(const FastHeader &H, const FastDim *dims_g, FastDim *dims) {
    for (int i = threadIdx.x; i < H.num_records * (int)(sizeof(FastDim) / 4); i += kFastThreads)
        reinterpret_cast<uint32_t *>(dims)[i] = __ldg(reinterpret_cast<const uint32_t *>(dims_g) + i);
    __syncthreads();
}

// Coordinates of worker w and its record in every dimension.
__device__ __forceinline__ void fast_worker(const FastHeader &H, const FastDim *dims, uint32_t w, int *c, const FastDim **e) {
#pragma unroll
    for (int k = 0; k < kMaxBoxDims; ++k) {
        c[k] = 0;
        e[k] = dims;
        if (k < H.rank) {
            c[k] = (int)(w / (uint32_t)H.wstride[k]);
            w -= (uint32_t)c[k] * (uint32_t)H.wstride[k];
            e[k] = dims + H.dim_base[k] + c[k];
        }
    }
}

// Ghost-row block of worker s: rows [row0, ...) of its ghost rows.
__device__ __forceinline__ void fast_ghost_rows(const FastHeader &H, const FastDim *dims, const ShardPointers &sh,
                                                unsigned char *scratch, uint32_t s, uint32_t t) {
    const int d = H.rank;
    int c[kMaxBoxDims];
    const FastDim *e[kMaxBoxDims];
    fast_worker(H, dims, s, c, e);
    // class j holds the rows whose index is a bulk index in the dimensions before j, a ghost index in dimension j
    // and anything after it
    uint32_t cls_rows[kMaxBoxDims];
    uint32_t total_rows = 0;
#pragma unroll
    for (int j = 0; j < kMaxBoxDims - 1; ++j) {
        cls_rows[j] = 0;
        if (j < d - 1) {
            uint32_t r = (uint32_t)(e[j]->n - e[j]->b);
#pragma unroll
            for (int k = 0; k < kMaxBoxDims - 1; ++k)
                if (k < d - 1 && k != j) r *= (uint32_t)(k < j ? e[k]->b : e[k]->n);
            cls_rows[j] = r;
            total_rows += r;
        }
    }
    const uint32_t row0 = t * (uint32_t)H.rows_per_tile[0];
    if (row0 >= total_rows) return;
    const uint32_t nrows = min((uint32_t)H.rows_per_tile[0], total_rows - row0);
    const FastDim *ex = e[d - 1];
    const uint32_t nx = (uint32_t)ex->n;
    FastRowRec *recs = reinterpret_cast<FastRowRec *>(scratch);
    static_assert(sizeof(FastRowRec) * kFastMaxRows <= kFastMaxSlots * 16, "row records fit the scratch array");
    for (uint32_t rl = threadIdx.x; rl < nrows; rl += kFastThreads) {
        uint32_t idx = row0 + rl;
        int j = 0;
#pragma unroll
        for (int q = 0; q < kMaxBoxDims - 2; ++q)
            if (j == q && q < d - 2 && idx >= cls_rows[q]) {
                idx -= cls_rows[q];
                ++j;
            }
        // coordinates of the row inside its class, innermost outer dimension first
        uint32_t dst_lin = 0, src_lin = 0, dst_pitch = 1, src_pitch = 1;
        int outer_w = 0;
        bool zero = false;
#pragma unroll
        for (int k = kMaxBoxDims - 2; k >= 0; --k) {
            if (k < d - 1) {
                const FastDim &f = *e[k];
                uint32_t coord;
                if (k == 0) {
                    coord = idx;
                } else {
                    const uint32_t ext = k > j ? (uint32_t)f.n : (k == j ? (uint32_t)(f.n - f.b) : (uint32_t)f.b);
                    const uint32_t mg = k > j ? f.magic_n : (k == j ? f.magic_g : f.magic_b);
                    const uint32_t sf = k > j ? fast_shift_n(f) : (k == j ? fast_shift_g(f) : fast_shift_b(f));
                    const uint32_t q = fast_div(idx, mg, sf);
                    coord = idx - q * ext;
                    idx = q;
                }
                const int i = k > j ? (int)coord : (k == j ? ((int)coord < f.hlo ? (int)coord : (int)coord + f.b) : f.hlo + (int)coord);
                int nc = c[k], si = i;
                if (i < f.hlo) {
                    nc = f.lo_c;
                    si = i + f.lo_shift;
                } else if (i >= f.hlo + f.b) {
                    nc = f.hi_c;
                    si = i + f.hi_shift;
                }
                dst_lin += (uint32_t)i * dst_pitch;
                dst_pitch *= (uint32_t)f.n;
                if (nc < 0) {
                    zero = true;
                } else {
                    src_lin += (uint32_t)si * src_pitch;
                    src_pitch *= (uint32_t)dims[H.dim_base[k] + nc].n;
                    outer_w += nc * H.wstride[k];
                }
            }
        }
        FastRowRec r;
        r.dst_off = dst_lin * nx;
#pragma unroll
        for (int reg = 0; reg < 3; ++reg) {
            const int ncx = reg == 0 ? ex->lo_c : (reg == 1 ? c[d - 1] : ex->hi_c);
            const int shift = reg == 0 ? ex->lo_shift : (reg == 1 ? 0 : ex->hi_shift);
            r.shard[reg] = -1;
            r.off[reg] = 0;
            if (!zero && ncx >= 0) {
                r.shard[reg] = outer_w + ncx * H.wstride[d - 1];
                r.off[reg] = src_lin * (uint32_t)dims[H.dim_base[d - 1] + ncx].n + (uint32_t)shift;
            }
        }
        recs[rl] = r;
    }
    __syncthreads();
    uint4 *dst = reinterpret_cast<uint4 *>(sh.p[s]);
    const uint32_t count = nrows * nx;
    const uint32_t xlo = (uint32_t)ex->hlo, xhi = (uint32_t)(ex->hlo + ex->b);
    const uint32_t shx = fast_shift_n(*ex);
    constexpr int U = 8;
    for (uint32_t base = threadIdx.x; base < count; base += kFastThreads * U) {
        uint4 v[U];
        uint32_t doff[U];
        bool wr[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * kFastThreads;
            wr[u] = false;
            v[u] = make_uint4(0, 0, 0, 0);
            doff[u] = 0;
            if (i < count) {
                const uint32_t rl = fast_div(i, ex->magic_n, shx);
                const uint32_t col = i - rl * nx;
                const FastRowRec &r = recs[rl];
                const int reg = col < xlo ? 0 : (col < xhi ? 1 : 2);
                const int src = r.shard[reg];
                doff[u] = r.dst_off + col;
                wr[u] = true;
                if (src >= 0) v[u] = __ldg(reinterpret_cast<const uint4 *>(sh.p[src]) + (r.off[reg] + col));
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (wr[u]) dst[doff[u]] = v[u];
    }
}

// Unit offsets of bulk rows [row0, row0 + nrows) of a line of workers (the same in all of them up to the row
// pitch): `inner` restricts the rows to those out of every outer neighbour's reach.
__device__ __forceinline__ void fast_line_rows(const FastHeader &H, const FastDim *const *e, bool inner, uint32_t row0,
                                               uint32_t nrows, uint32_t *rowlin) {
    const int d = H.rank;
    for (uint32_t rl = threadIdx.x; rl < nrows; rl += kFastThreads) {
        uint32_t idx = row0 + rl, lin = 0, pitch = 1;
#pragma unroll
        for (int k = kMaxBoxDims - 2; k >= 0; --k) {
            if (k < d - 1) {
                const FastDim &f = *e[k];
                uint32_t coord = idx;
                if (k > 0) {
                    const uint32_t ext = inner ? (uint32_t)(f.b - f.rlo - f.rhi) : (uint32_t)f.b;
                    const uint32_t q = inner ? fast_div(idx, f.magic_bi, fast_shift_bi(f)) : fast_div(idx, f.magic_b, fast_shift_b(f));
                    coord = idx - q * ext;
                    idx = q;
                }
                lin += ((uint32_t)f.hlo + (inner ? (uint32_t)f.rlo : 0u) + coord) * pitch;
                pitch *= (uint32_t)f.n;
            }
        }
        rowlin[rl] = lin;
    }
}

__global__ void __launch_bounds__(kFastThreads)
halo_fast_fwd_kernel(const __grid_constant__ FastHeader H, const FastDim *__restrict__ dims_g,
                     const __grid_constant__ ShardPointers sh) {
    __shared__ FastDim dims[kMaxFastCoords];
    __shared__ __align__(16) unsigned char scratch[kFastMaxSlots * 16];
    fast_load_records(H, dims_g, dims);
    const int d = H.rank;
    uint32_t tile_id;
    const int kind = fast_block_kind(H, &tile_id);
    if (kind == 0) {
        const uint32_t s = tile_id / (uint32_t)H.tiles_per_owner[0];
        if (s < (uint32_t)H.num_workers) fast_ghost_rows(H, dims, sh, scratch, s, tile_id - s * (uint32_t)H.tiles_per_owner[0]);
        return;
    }
    // ---------------------------------------------------------------------- line block
    const uint32_t line = tile_id / (uint32_t)H.tiles_per_owner[1];
    if (line >= (uint32_t)H.num_lines) return;
    const uint32_t t = tile_id - line * (uint32_t)H.tiles_per_owner[1];
    const int px = H.pshape[d - 1];
    const uint32_t first_worker = line * (uint32_t)px;        // the innermost dimension has worker stride 1
    int c[kMaxBoxDims];
    const FastDim *e[kMaxBoxDims];
    fast_worker(H, dims, first_worker, c, e);
    uint32_t total_rows = 1;
#pragma unroll
    for (int k = 0; k < kMaxBoxDims - 1; ++k)
        if (k < d - 1) total_rows *= (uint32_t)e[k]->b;
    const uint32_t row0 = t * (uint32_t)H.rows_per_tile[1];
    if (row0 >= total_rows) return;
    const uint32_t nrows = min((uint32_t)H.rows_per_tile[1], total_rows - row0);
    // per worker of the line: cumulative counts of ghost units (stores) and of wanted bulk units (loads)
    __shared__ uint32_t cum_g[kMaxFastCoords + 1], cum_p[kMaxFastCoords + 1];
    __shared__ uint32_t rowlin[128];
    const FastDim *xd = dims + H.dim_base[d - 1];
    if (threadIdx.x == 0) {
        uint32_t g = 0, pc = 0;
        for (int a = 0; a < px; ++a) {
            cum_g[a] = g;
            cum_p[a] = pc;
            g += (uint32_t)(xd[a].n - xd[a].b);
            pc += (uint32_t)(xd[a].rlo + xd[a].rhi);      // what the two neighbours' ghosts hold of this worker's rows
        }
        cum_g[px] = g;
        cum_p[px] = pc;
    }
    fast_line_rows(H, e, false, row0, nrows, rowlin);
    __syncthreads();
    uint4 *slots = reinterpret_cast<uint4 *>(scratch);
    const uint32_t GC = cum_g[px], PC = cum_p[px];
    // loads, in the order (worker, row, wanted unit): the last units of row r and the first units of
    // row r + 1 are neighbours in memory and in this order
    for (uint32_t q = threadIdx.x; q < nrows * PC; q += kFastThreads) {
        int a = 0;
        while (q >= nrows * cum_p[a + 1]) ++a;
        const uint32_t qa = q - nrows * cum_p[a];
        const FastDim &f = xd[a];
        const uint32_t pc = (uint32_t)(f.rlo + f.rhi);
        const uint32_t rl = qa / pc, piece = qa - rl * pc;
        uint32_t col, slot;
        if (piece < (uint32_t)f.rlo) {      // first bulk units -> high ghost of the low neighbour
            const FastDim &g = xd[f.lo_c];
            col = (uint32_t)f.hlo + piece;
            slot = nrows * cum_g[f.lo_c] + rl * (uint32_t)(g.n - g.b) + (uint32_t)g.hlo + piece;
        } else {                            // last bulk units -> low ghost of the high neighbour
            const FastDim &g = xd[f.hi_c];
            const uint32_t u = piece - (uint32_t)f.rlo;
            col = (uint32_t)(f.hlo + f.b - f.rhi) + u;
            slot = nrows * cum_g[f.hi_c] + rl * (uint32_t)(g.n - g.b) + u;
        }
        slots[slot] = __ldg(reinterpret_cast<const uint4 *>(sh.p[first_worker + a]) + (rowlin[rl] * (uint32_t)f.n + col));
    }
    __syncthreads();
    // stores, in the order (worker, row, ghost unit): the high ghost of row r is followed by the low ghost of row r + 1
    for (uint32_t q = threadIdx.x; q < nrows * GC; q += kFastThreads) {
        int a = 0;
        while (q >= nrows * cum_g[a + 1]) ++a;
        const uint32_t qa = q - nrows * cum_g[a];
        const FastDim &f = xd[a];
        const uint32_t gc = (uint32_t)(f.n - f.b);
        const uint32_t rl = qa / gc, g = qa - rl * gc;
        const bool low = g < (uint32_t)f.hlo;
        const bool has = low ? f.lo_c >= 0 : f.hi_c >= 0;
        const uint32_t col = low ? g : g + (uint32_t)f.b;
        uint4 *dst = reinterpret_cast<uint4 *>(sh.p[first_worker + a]) + (rowlin[rl] * (uint32_t)f.n + col);
        *dst = has ? slots[nrows * cum_g[a] + qa] : make_uint4(0, 0, 0, 0);
    }
}

// ---------------------------------------------------------------------------------------------
// H* at the row ends.  T: 16-byte vector of the element type (float4, double2, bf16x8).
//
// The box plan is at its best where rows are long; where a partition is split along the innermost
// dimension, most of its boxes are columns a few units wide.  For those H* runs in two launches that
// touch disjoint cells: the box kernel on a plan without the row-end columns of the bulk rows that no
// outer neighbour reaches, and this kernel on exactly those.  There a bulk unit near a row end receives
// from one ghost unit of the neighbour along the row, and every unit involved -- low ghost, low
// receiving, high receiving, high ghost of every worker of the line -- is read once and written once,
// in memory order, with the neighbour's ghost value taken from shared memory.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kFastThreads)
halo_fast_adj_lines_kernel(const __grid_constant__ FastHeader H, const FastDim *__restrict__ dims_g,
                           const __grid_constant__ ShardPointers sh) {
    __shared__ FastDim dims[kMaxFastCoords];
    __shared__ __align__(16) unsigned char scratch[kFastMaxSlots * 16];
    fast_load_records(H, dims_g, dims);
    const int d = H.rank;
    uint32_t tile_id;
    if (fast_block_kind(H, &tile_id) != 1) return;
    // both ends of the bulk rows that are out of reach in every outer dimension, for all workers of the line
    const uint32_t line = tile_id / (uint32_t)H.tiles_per_owner[1];
    if (line >= (uint32_t)H.num_lines) return;
    const uint32_t t = tile_id - line * (uint32_t)H.tiles_per_owner[1];
    const int px = H.pshape[d - 1];
    const uint32_t first_worker = line * (uint32_t)px;
    int c[kMaxBoxDims];
    const FastDim *e[kMaxBoxDims];
    fast_worker(H, dims, first_worker, c, e);
    uint32_t total_rows = 1;
#pragma unroll
    for (int k = 0; k < kMaxBoxDims - 1; ++k)
        if (k < d - 1) total_rows *= (uint32_t)(e[k]->b - e[k]->rlo - e[k]->rhi);
    const uint32_t row0 = t * (uint32_t)H.rows_per_tile[1];
    if (row0 >= total_rows) return;
    const uint32_t nrows = min((uint32_t)H.rows_per_tile[1], total_rows - row0);
    __shared__ uint32_t cum_e[kMaxFastCoords + 1];
    __shared__ uint32_t rowlin[128];
    const FastDim *xd = dims + H.dim_base[d - 1];
    if (threadIdx.x == 0) {
        uint32_t n = 0;
        for (int a = 0; a < px; ++a) {
            cum_e[a] = n;
            n += (uint32_t)(xd[a].n - xd[a].b + xd[a].rlo + xd[a].rhi);     // low ghost, low receiving, high receiving, high ghost
        }
        cum_e[px] = n;
    }
    fast_line_rows(H, e, true, row0, nrows, rowlin);
    __syncthreads();
    T *slots = reinterpret_cast<T *>(scratch);
    const uint32_t EC = cum_e[px];
    // pass 1: every unit of the row ends into shared memory, in memory order per worker
    for (uint32_t q = threadIdx.x; q < nrows * EC; q += kFastThreads) {
        int a = 0;
        while (q >= nrows * cum_e[a + 1]) ++a;
        const uint32_t qa = q - nrows * cum_e[a];
        const FastDim &f = xd[a];
        const uint32_t ec = (uint32_t)(f.n - f.b + f.rlo + f.rhi), lo_end = (uint32_t)(f.hlo + f.rlo);
        const uint32_t rl = qa / ec, u = qa - rl * ec;
        const uint32_t col = u < lo_end ? u : u - lo_end + (uint32_t)(f.hlo + f.b - f.rhi);
        const bool ghost = col < (uint32_t)f.hlo || col >= (uint32_t)(f.hlo + f.b);
        const bool outside = ghost && (col < (uint32_t)f.hlo ? f.lo_c < 0 : f.hi_c < 0);      // never read: only cleared
        if (!outside) slots[q] = reinterpret_cast<const T *>(sh.p[first_worker + a])[rowlin[rl] * (uint32_t)f.n + col];
    }
    __syncthreads();
    // pass 2: ghosts <- 0, receiving units <- own value + the neighbour's ghost copy, same order
    for (uint32_t q = threadIdx.x; q < nrows * EC; q += kFastThreads) {
        int a = 0;
        while (q >= nrows * cum_e[a + 1]) ++a;
        const uint32_t qa = q - nrows * cum_e[a];
        const FastDim &f = xd[a];
        const uint32_t ec = (uint32_t)(f.n - f.b + f.rlo + f.rhi), lo_end = (uint32_t)(f.hlo + f.rlo);
        const uint32_t rl = qa / ec, u = qa - rl * ec;
        const uint32_t col = u < lo_end ? u : u - lo_end + (uint32_t)(f.hlo + f.b - f.rhi);
        T v = zero_of<T>();
        if (col >= (uint32_t)f.hlo && col < (uint32_t)(f.hlo + f.b)) {
            v = slots[q];
            if (u < lo_end) {
                if (f.lo_c >= 0) {      // the low neighbour's high ghost unit of the same cell: the last units of its row ends
                    const FastDim &g = xd[f.lo_c];
                    const uint32_t gec = (uint32_t)(g.n - g.b + g.rlo + g.rhi);
                    const uint32_t gu = (uint32_t)(g.hlo + g.rlo + g.rhi) + (u - (uint32_t)f.hlo);
                    v = vadd(v, slots[nrows * cum_e[f.lo_c] + rl * gec + gu]);
                }
            } else if (f.hi_c >= 0) {   // the high neighbour's low ghost unit: the first units of its row
                const FastDim &g = xd[f.hi_c];
                const uint32_t gec = (uint32_t)(g.n - g.b + g.rlo + g.rhi);
                v = vadd(v, slots[nrows * cum_e[f.hi_c] + rl * gec + (u - lo_end)]);
            }
        }
        reinterpret_cast<T *>(sh.p[first_worker + a])[rowlin[rl] * (uint32_t)f.n + col] = v;
    }
}

static distdl_status_t launch(const distdl_partition *p, const HaloPlanDevice &plan, void *const *shards,
                              void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!p || !shards) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (!p->device_block) return fail(DISTDL_ERR_CUDA, "%s: the partition was created without a CUDA device", what);
    ShardPointers sh;
    for (int32_t w = 0; w < p->num_workers; ++w) {
        if (!shards[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shards[%d] is NULL", what, w);
        if (!aligned16(shards[w])) return fail(DISTDL_ERR_ALIGNMENT, "%s: shards[%d] is not 16-byte aligned", what, w);
        sh.p[w] = shards[w];
    }
    // shards must not overlap (each is written in place)
    {
        const int64_t es = elem_size(p->dtype);
        for (int32_t a = 0; a < p->num_workers; ++a)
            for (int32_t b = a + 1; b < p->num_workers; ++b) {
                const char *a0 = (const char *)shards[a], *a1 = a0 + p->shard_elems(a) * es;
                const char *b0 = (const char *)shards[b], *b1 = b0 + p->shard_elems(b) * es;
                if (a0 < b1 && b0 < a1) return fail(DISTDL_ERR_INVALID_ARG, "%s: shards %d and %d overlap", what, a, b);
            }
    }
    for (int32_t w = p->num_workers; w < DISTDL_MAX_WORKERS; ++w) sh.p[w] = nullptr;
    if (plan.num_tiles == 0) return DISTDL_OK;
    // DISTDL_HALO_PLAN=box in the environment sends every call through the general box plan (for comparisons)
    static const bool box_only = [] {
        const char *v = getenv("DISTDL_HALO_PLAN");
        return v && strcmp(v, "box") == 0;
    }();
    if (box_only) {
        if (adjoint)
            halo_box_kernel<true><<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(
                plan.boxes, plan.sources, plan.tiles, elem_size(p->dtype), sh);
        else
            halo_box_kernel<false><<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(
                plan.boxes, plan.sources, plan.tiles, elem_size(p->dtype), sh);
        DISTDL_CUDA_CHECK(cudaGetLastError());
        return DISTDL_OK;
    }
    if (!adjoint && p->fast.usable && p->fast_dims_dev) {
        const FastHeader &h = p->fast.hdr;
        halo_fast_fwd_kernel<<<(unsigned)h.num_groups * (unsigned)(h.group[0] + h.group[1]), kFastThreads, 0,
                               (cudaStream_t)stream>>>(h, p->fast_dims_dev, sh);
        DISTDL_CUDA_CHECK(cudaGetLastError());
        return DISTDL_OK;
    }
    if (adjoint && p->fast.adj_usable && p->fast_dims_dev) {
        cudaStream_t st = (cudaStream_t)stream;
        const HaloPlanDevice &rest = p->adj_rest_dev;      // everything but the row ends of the rows out of outer reach
        if (rest.num_tiles > 0) {
            halo_box_kernel<true><<<rest.num_tiles, kHaloThreads, 0, st>>>(rest.boxes, rest.sources, rest.tiles, elem_size(p->dtype), sh);
            DISTDL_CUDA_CHECK(cudaGetLastError());
        }
        const FastHeader &h = p->fast.adj_hdr;
        const unsigned grid = (unsigned)h.num_groups * (unsigned)(h.group[0] + h.group[1]);
        if (p->dtype == DISTDL_F32) halo_fast_adj_lines_kernel<float4><<<grid, kFastThreads, 0, st>>>(h, p->fast_dims_dev, sh);
        else if (p->dtype == DISTDL_F64) halo_fast_adj_lines_kernel<double2><<<grid, kFastThreads, 0, st>>>(h, p->fast_dims_dev, sh);
        else halo_fast_adj_lines_kernel<bf16x8><<<grid, kFastThreads, 0, st>>>(h, p->fast_dims_dev, sh);
        DISTDL_CUDA_CHECK(cudaGetLastError());
        return DISTDL_OK;
    }
    if (adjoint)
        halo_box_kernel<true><<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(
            plan.boxes, plan.sources, plan.tiles, elem_size(p->dtype), sh);
    else
        halo_box_kernel<false><<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(
            plan.boxes, plan.sources, plan.tiles, elem_size(p->dtype), sh);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

// ---------------------------------------------------------------------------------------------
// Halo exchange without any device allocation: the plan tables go into a fixed device array.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticPlanBytes = (size_t)1 << 20;   // 1 MiB, held by every device that loads the library
static __device__ __align__(256) unsigned char g_static_plan[kStaticPlanBytes];
constexpr int kMaxDevices = 64;

// Device address of g_static_plan on the current device.  In host code the array's name only
// stands for the symbol; the address a kernel can use has to be asked for, once per device.
static distdl_status_t static_plan_address(unsigned char **out) {
    static unsigned char *cached[kMaxDevices] = {nullptr};
    int dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(DISTDL_ERR_UNSUPPORTED, "halo_fwd_noalloc: device index %d", dev);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());
    if (!cached[dev]) {
        void *ptr = nullptr;
        DISTDL_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_static_plan));
        cached[dev] = static_cast<unsigned char *>(ptr);
    }
    *out = cached[dev];
    return DISTDL_OK;
}

static distdl_status_t halo_fwd_noalloc_impl(int32_t rank, const int64_t *global_shape, const int32_t *partition_shape,
                                             const int32_t *halo_lo, const int32_t *halo_hi, distdl_dtype_t dtype,
                                             void *const *shards, void *stream) {
    const char *what = "halo_fwd_noalloc";
    clear_error();
    if (!shards) return fail(DISTDL_ERR_INVALID_ARG, "%s: shards is NULL", what);
    // The plan tables below are copied from host memory that is freed when this call returns: a captured
    // copy would read it again at every replay.  So the call refuses a stream that is being captured.
    {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        DISTDL_CUDA_CHECK(cudaStreamIsCapturing((cudaStream_t)stream, &cap));
        if (cap != cudaStreamCaptureStatusNone)
            return fail(DISTDL_ERR_UNSUPPORTED, "%s: the stream is being captured; this call copies its plan tables from "
                        "temporary host memory and cannot be recorded in a graph (use distdl_partition_create + distdl_halo_fwd)", what);
    }
    distdl_partition *p = nullptr;
    distdl_status_t st = partition_create_host_only(rank, global_shape, partition_shape, halo_lo, halo_hi, dtype, &p);
    if (st != DISTDL_OK) return st;
    struct Guard {
        distdl_partition *p;
        ~Guard() { delete p; }
    } guard{p};
    const HaloPlanHost &h = p->fwd_host;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t bz = up(h.boxes.size() * sizeof(HaloBox)), sz = up(h.sources.size() * sizeof(HaloSource)),
                 tz = up(h.tiles.size() * sizeof(HaloTile));
    if (bz + sz + tz > kStaticPlanBytes)
        return fail(DISTDL_ERR_UNSUPPORTED,
                    "%s: the plan of this partition needs %zu bytes of tables, the fixed device array holds %zu "
                    "(use distdl_partition_create + distdl_halo_fwd for larger partitions)",
                    what, bz + sz + tz, kStaticPlanBytes);
    ShardPointers sh;
    const int64_t es = elem_size(p->dtype);
    for (int32_t w = 0; w < p->num_workers; ++w) {
        if (!shards[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shards[%d] is NULL", what, w);
        if (!aligned16(shards[w])) return fail(DISTDL_ERR_ALIGNMENT, "%s: shards[%d] is not 16-byte aligned", what, w);
        sh.p[w] = shards[w];
    }
    for (int32_t a = 0; a < p->num_workers; ++a)
        for (int32_t b = a + 1; b < p->num_workers; ++b) {
            const char *a0 = (const char *)shards[a], *a1 = a0 + p->shard_elems(a) * es;
            const char *b0 = (const char *)shards[b], *b1 = b0 + p->shard_elems(b) * es;
            if (a0 < b1 && b0 < a1) return fail(DISTDL_ERR_INVALID_ARG, "%s: shards %d and %d overlap", what, a, b);
        }
    for (int32_t w = p->num_workers; w < DISTDL_MAX_WORKERS; ++w) sh.p[w] = nullptr;
    if (h.tiles.empty()) return DISTDL_OK;
    unsigned char *base = nullptr;
    st = static_plan_address(&base);
    if (st != DISTDL_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    // Every table entry the kernel reads is rewritten here, so nothing of an earlier call is used.
    // The copies are stream-ordered before the kernel; pageable sources are staged before the call
    // returns, so the host tables may go away right after it.
    DISTDL_CUDA_CHECK(cudaMemcpyAsync(base, h.boxes.data(), h.boxes.size() * sizeof(HaloBox), cudaMemcpyHostToDevice, s));
    if (!h.sources.empty())
        DISTDL_CUDA_CHECK(cudaMemcpyAsync(base + bz, h.sources.data(), h.sources.size() * sizeof(HaloSource), cudaMemcpyHostToDevice, s));
    DISTDL_CUDA_CHECK(cudaMemcpyAsync(base + bz + sz, h.tiles.data(), h.tiles.size() * sizeof(HaloTile), cudaMemcpyHostToDevice, s));
    halo_box_kernel<false><<<(unsigned)h.tiles.size(), kHaloThreads, 0, s>>>(
        reinterpret_cast<const HaloBox *>(base), reinterpret_cast<const HaloSource *>(base + bz),
        reinterpret_cast<const HaloTile *>(base + bz + sz), elem_size(p->dtype), sh);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

}  // namespace distdl

extern "C" distdl_status_t distdl_halo_fwd_noalloc(int32_t rank, const int64_t *global_shape,
                                                   const int32_t *partition_shape, const int32_t *halo_lo,
                                                   const int32_t *halo_hi, distdl_dtype_t dtype, void *const *shards,
                                                   void *stream) {
    return distdl::halo_fwd_noalloc_impl(rank, global_shape, partition_shape, halo_lo, halo_hi, dtype, shards, stream);
}

namespace distdl {
// The all-to-all runs the copy path of the box kernel on the pointer table [source shards, destination shards].
static distdl_status_t repartition_launch(const distdl_repartition *r, const void *const *from, void *const *to,
                                          void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!r || !from || !to) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (!r->device_block) return fail(DISTDL_ERR_CUDA, "%s: the object was created without a CUDA device", what);
    // forward: from = source shards, to = destination shards; adjoint: from = destination shards, to = source shards
    const int32_t nfrom = adjoint ? r->num_dst : r->num_src, nto = adjoint ? r->num_src : r->num_dst;
    const int32_t from_base = adjoint ? r->num_src : 0, to_base = adjoint ? 0 : r->num_src;
    ShardPointers sh;
    for (int32_t w = 0; w < DISTDL_MAX_WORKERS; ++w) sh.p[w] = nullptr;
    const int64_t es = elem_size(r->dtype);
    for (int32_t w = 0; w < nfrom; ++w) {
        if (!from[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: input shard %d is NULL", what, w);
        if (!aligned16(from[w])) return fail(DISTDL_ERR_ALIGNMENT, "%s: input shard %d is not 16-byte aligned", what, w);
        sh.p[from_base + w] = const_cast<void *>(from[w]);
    }
    for (int32_t w = 0; w < nto; ++w) {
        if (!to[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: output shard %d is NULL", what, w);
        if (!aligned16(to[w])) return fail(DISTDL_ERR_ALIGNMENT, "%s: output shard %d is not 16-byte aligned", what, w);
        sh.p[to_base + w] = to[w];
    }
    // an output shard may overlap neither another output nor any input (the copy is not in place)
    for (int32_t a = 0; a < nto; ++a) {
        const char *a0 = (const char *)to[a], *a1 = a0 + r->shard_elems[to_base + a] * es;
        for (int32_t b = a + 1; b < nto; ++b) {
            const char *b0 = (const char *)to[b], *b1 = b0 + r->shard_elems[to_base + b] * es;
            if (a0 < b1 && b0 < a1) return fail(DISTDL_ERR_INVALID_ARG, "%s: output shards %d and %d overlap", what, a, b);
        }
        for (int32_t b = 0; b < nfrom; ++b) {
            const char *b0 = (const char *)from[b], *b1 = b0 + r->shard_elems[from_base + b] * es;
            if (a0 < b1 && b0 < a1) return fail(DISTDL_ERR_INVALID_ARG, "%s: output shard %d overlaps input shard %d", what, a, b);
        }
    }
    const HaloPlanDevice &plan = adjoint ? r->adj_dev : r->fwd_dev;
    if (plan.num_tiles == 0) return DISTDL_OK;
    halo_box_kernel<false><<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(plan.boxes, plan.sources, plan.tiles,
                                                                                       elem_size(r->dtype), sh);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}
}  // namespace distdl

extern "C" distdl_status_t distdl_repartition_fwd(const distdl_repartition_t *r, const void *const *src, void *const *dst,
                                                  void *stream) {
    return distdl::repartition_launch(r, src, dst, stream, false, "repartition_fwd");
}

extern "C" distdl_status_t distdl_repartition_adj(const distdl_repartition_t *r, const void *const *dy, void *const *dx,
                                                  void *stream) {
    return distdl::repartition_launch(r, dy, dx, stream, true, "repartition_adj");
}

extern "C" distdl_status_t distdl_halo_fwd(const distdl_partition_t *p, void *const *shards, void *stream) {
    return distdl::launch(p, p ? p->fwd_dev : distdl::HaloPlanDevice(), shards, stream, false, "halo_fwd");
}

extern "C" distdl_status_t distdl_halo_adj(const distdl_partition_t *p, void *const *shards, void *stream) {
    return distdl::launch(p, p ? p->adj_dev : distdl::HaloPlanDevice(), shards, stream, true, "halo_adj");
}
