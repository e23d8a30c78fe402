// Halo exchange H and adjoint halo exchange H* (Section 3, "Halo exchange") as one gather
// kernel over a host-planned list of boxes.
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

__device__ __forceinline__ float4 add4(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ float add4(float a, float b) { return __fadd_rn(a, b); }

template <typename T> __device__ __forceinline__ T zero_of();
template <> __device__ __forceinline__ float4 zero_of<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float zero_of<float>() { return 0.f; }
template <> __device__ __forceinline__ uint4 zero_of<uint4>() { return make_uint4(0, 0, 0, 0); }
template <> __device__ __forceinline__ unsigned short zero_of<unsigned short>() { return 0; }

// Copy / clear of one tile with element type T (uint4 = 16 bytes, float, or unsigned short).
template <typename T>
__device__ __forceinline__ void run_copy_tile(const HaloBox &box, const HaloSource *src, const ShardPointers &sh,
                                              uint32_t first, uint32_t count) {
    T *dst = reinterpret_cast<T *>(sh.p[box.dst_shard]) + box.dst_offset;
    const T *s0 = box.nsrc ? reinterpret_cast<const T *>(sh.p[src[0].shard]) + src[0].offset : nullptr;
    const int nd = box.ndim;
    for (uint32_t i = threadIdx.x; i < count; i += kHaloThreads) {
        uint32_t rem = first + i;
        int64_t doff = 0, soff = 0;
        for (int k = nd - 1; k >= 0; --k) {
            const uint32_t e = (uint32_t)box.shape[k];
            const uint32_t q = rem / e, c = rem - q * e;
            rem = q;
            doff += (int64_t)c * box.dst_stride[k];
            if (s0) soff += (int64_t)c * src[0].stride[k];
        }
        dst[doff] = s0 ? s0[soff] : zero_of<T>();
    }
}

// Nested sum of one tile (H*): T is float4 or float.
template <typename T>
__device__ __forceinline__ void run_sum_tile(const HaloBox &box, const HaloSource *src, const ShardPointers &sh,
                                             uint32_t first, uint32_t count) {
    T *dst = reinterpret_cast<T *>(sh.p[box.dst_shard]) + box.dst_offset;
    const int nd = box.ndim;
    const int nsrc = box.nsrc;
    const int top = box.levels - 1;
    for (uint32_t i = threadIdx.x; i < count; i += kHaloThreads) {
        uint32_t rem = first + i;
        uint32_t coord[kMaxBoxDims];
#pragma unroll
        for (int k = kMaxBoxDims - 1; k >= 0; --k) {
            coord[k] = 0;
            if (k < nd) {
                const uint32_t e = (uint32_t)box.shape[k];
                const uint32_t q = rem / e;
                coord[k] = rem - q * e;
                rem = q;
            }
        }
        int64_t doff = 0;
#pragma unroll
        for (int k = 0; k < kMaxBoxDims; ++k)
            if (k < nd) doff += (int64_t)coord[k] * box.dst_stride[k];

        T acc[kMaxLevels];
        unsigned has = 0;
        for (int j = 0; j < nsrc; ++j) {
            const HaloSource &s = src[j];
            int64_t soff = s.offset;
#pragma unroll
            for (int k = 0; k < kMaxBoxDims; ++k)
                if (k < nd) soff += (int64_t)coord[k] * s.stride[k];
            T *sp = reinterpret_cast<T *>(sh.p[s.shard]) + soff;
            const T v = *sp;
            if (s.clear_after) *sp = zero_of<T>();
            // absent terms are skipped, never added as zero
            acc[0] = (has & 1u) ? add4(acc[0], v) : v;
            has |= 1u;
            const int close = s.close;
#pragma unroll
            for (int l = 0; l < kMaxLevels - 1; ++l) {
                if (l < close) {
                    acc[l + 1] = ((has >> (l + 1)) & 1u) ? add4(acc[l + 1], acc[l]) : acc[l];
                    has |= 2u << l;
                    has &= ~(1u << l);
                }
            }
        }
        T res = acc[0];
#pragma unroll
        for (int l = 1; l < kMaxLevels; ++l)
            if (l == top) res = acc[l];
        dst[doff] = res;
    }
}

__global__ void __launch_bounds__(kHaloThreads)
halo_box_kernel(const HaloBox *__restrict__ boxes, const HaloSource *__restrict__ sources,
                const HaloTile *__restrict__ tiles, int32_t num_tiles, int32_t elem_bytes,
                const __grid_constant__ ShardPointers sh) {
    __shared__ HaloBox s_box;
    __shared__ HaloSource s_src[kMaxSources];
    __shared__ HaloTile s_tile;
    for (int32_t t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        __syncthreads();
        if (threadIdx.x == 0) s_tile = tiles[t];
        __syncthreads();
        const HaloBox *gb = boxes + s_tile.box;
        // cooperative copy of the descriptors (4-byte words)
        {
            const uint32_t *g = reinterpret_cast<const uint32_t *>(gb);
            uint32_t *s = reinterpret_cast<uint32_t *>(&s_box);
            for (uint32_t i = threadIdx.x; i < sizeof(HaloBox) / 4; i += kHaloThreads) s[i] = g[i];
        }
        __syncthreads();
        {
            const uint32_t *g = reinterpret_cast<const uint32_t *>(sources + s_box.src_begin);
            uint32_t *s = reinterpret_cast<uint32_t *>(s_src);
            const uint32_t words = (uint32_t)s_box.nsrc * (sizeof(HaloSource) / 4);
            for (uint32_t i = threadIdx.x; i < words; i += kHaloThreads) s[i] = g[i];
        }
        __syncthreads();
        const uint32_t first = s_tile.first, count = s_tile.count;
        if (s_box.nsrc <= 1) {
            if (s_box.vec) run_copy_tile<uint4>(s_box, s_src, sh, first, count);
            else if (elem_bytes == 4) run_copy_tile<float>(s_box, s_src, sh, first, count);
            else run_copy_tile<unsigned short>(s_box, s_src, sh, first, count);
        } else {
            if (s_box.vec) run_sum_tile<float4>(s_box, s_src, sh, first, count);
            else run_sum_tile<float>(s_box, s_src, sh, first, count);
        }
    }
}

static distdl_status_t launch(const distdl_partition *p, const HaloPlanDevice &plan, void *const *shards,
                              void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!p || !shards) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (adjoint && p->dtype != DISTDL_F32) return fail(DISTDL_ERR_UNSUPPORTED, "%s: F32 only", what);
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
    halo_box_kernel<<<plan.num_tiles, kHaloThreads, 0, (cudaStream_t)stream>>>(
        plan.boxes, plan.sources, plan.tiles, plan.num_tiles, elem_size(p->dtype), sh);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

}  // namespace distdl

extern "C" distdl_status_t distdl_halo_fwd(const distdl_partition_t *p, void *const *shards, void *stream) {
    return distdl::launch(p, p ? p->fwd_dev : distdl::HaloPlanDevice(), shards, stream, false, "halo_fwd");
}

extern "C" distdl_status_t distdl_halo_adj(const distdl_partition_t *p, void *const *shards, void *stream) {
    return distdl::launch(p, p ? p->adj_dev : distdl::HaloPlanDevice(), shards, stream, true, "halo_adj");
}
