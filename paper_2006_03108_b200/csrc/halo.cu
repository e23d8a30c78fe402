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
