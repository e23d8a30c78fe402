// Broadcast B (k copies of one realisation) and sum-reduce R = B* (fixed-order sum of k
// realisations).  Section 3, "Broadcast" and "Sum-reduce and all-reduce".
//
// Both are pure streaming kernels: every input byte is read once and every output byte written
// once, several independent loads in flight per thread; 16-byte accesses, and 32-byte ones in the
// broadcast when every pointer allows them.
#include <algorithm>
#include <vector>

#include "common.h"

namespace distdl {

constexpr int kMaxFan = 16;         // destinations (B) or sources (R) handled by one launch
constexpr int kStreamThreads = 256;
constexpr int kUnroll = 4;          // 16-byte vectors per thread per step

struct FanPointers {
    void *p[kMaxFan];
};

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// coherent variant: the buffer may also be written by this kernel (in-place fold)
__device__ __forceinline__ uint4 ld_stream_coherent(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// dst[j][i] = src[i] for j < k; nvec 16-byte vectors, then `tail` trailing bytes.
__global__ void __launch_bounds__(kStreamThreads)
broadcast_kernel(const uint4 *__restrict__ src, const __grid_constant__ FanPointers dst, int k, size_t nvec, int tail) {
    const size_t stride = (size_t)gridDim.x * kStreamThreads;
    size_t i = (size_t)blockIdx.x * kStreamThreads + threadIdx.x;
    for (; i + (kUnroll - 1) * stride < nvec; i += kUnroll * stride) {
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream(src + i + u * stride);
        for (int j = 0; j < k; ++j) {
            uint4 *d = reinterpret_cast<uint4 *>(dst.p[j]);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) st_stream(d + i + u * stride, v[u]);
        }
    }
    for (; i < nvec; i += stride) {
        const uint4 v = ld_stream(src + i);
        for (int j = 0; j < k; ++j) st_stream(reinterpret_cast<uint4 *>(dst.p[j]) + i, v);
    }
    if (blockIdx.x == 0 && (int)threadIdx.x < tail) {
        const unsigned char b = reinterpret_cast<const unsigned char *>(src + nvec)[threadIdx.x];
        for (int j = 0; j < k; ++j) (reinterpret_cast<unsigned char *>(reinterpret_cast<uint4 *>(dst.p[j]) + nvec))[threadIdx.x] = b;
    }
}

// One addition per element of a 16-byte vector, each the exact sum rounded once to the type.
// DT: 0 = four fp32, 1 = eight bfloat16, 2 = two fp64.
__device__ __forceinline__ uint32_t add_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ unsigned short add_bf16(unsigned short a, unsigned short b) {
    unsigned short r;
    asm("add.rn.bf16 %0, %1, %2;" : "=h"(r) : "h"(a), "h"(b));
    return r;
}
template <int DT>
__device__ __forceinline__ uint4 add_vec(uint4 a, uint4 b) {
    uint4 r;
    if (DT == 0) {
        r.x = __float_as_uint(__fadd_rn(__uint_as_float(a.x), __uint_as_float(b.x)));
        r.y = __float_as_uint(__fadd_rn(__uint_as_float(a.y), __uint_as_float(b.y)));
        r.z = __float_as_uint(__fadd_rn(__uint_as_float(a.z), __uint_as_float(b.z)));
        r.w = __float_as_uint(__fadd_rn(__uint_as_float(a.w), __uint_as_float(b.w)));
    } else if (DT == 1) {
        r.x = add_bf16x2(a.x, b.x);
        r.y = add_bf16x2(a.y, b.y);
        r.z = add_bf16x2(a.z, b.z);
        r.w = add_bf16x2(a.w, b.w);
    } else {
        const double lo = __dadd_rn(__hiloint2double((int)a.y, (int)a.x), __hiloint2double((int)b.y, (int)b.x));
        const double hi = __dadd_rn(__hiloint2double((int)a.w, (int)a.z), __hiloint2double((int)b.w, (int)b.z));
        r.x = (uint32_t)__double2loint(lo);
        r.y = (uint32_t)__double2hiint(lo);
        r.z = (uint32_t)__double2loint(hi);
        r.w = (uint32_t)__double2hiint(hi);
    }
    return r;
}

// dst[i] = ((src[0][i] + src[1][i]) + ...) + src[k-1][i]   (left fold in source order, in the type's arithmetic)
// nvec 16-byte vectors, then `tail` trailing elements.
template <int K, int DT>
__global__ void __launch_bounds__(kStreamThreads)
sumreduce_kernel(const __grid_constant__ FanPointers src, void *__restrict__ dst, int k_runtime, size_t nvec, int tail) {
    const int k = K > 0 ? K : k_runtime;
    const size_t stride = (size_t)gridDim.x * kStreamThreads;
    for (size_t i = (size_t)blockIdx.x * kStreamThreads + threadIdx.x; i < nvec; i += stride) {
        uint4 v[K > 0 ? K : kMaxFan];
#pragma unroll
        for (int j = 0; j < (K > 0 ? K : kMaxFan); ++j)
            if (j < k) v[j] = ld_stream_coherent(reinterpret_cast<const uint4 *>(src.p[j]) + i);
        uint4 acc = v[0];
#pragma unroll
        for (int j = 1; j < (K > 0 ? K : kMaxFan); ++j)
            if (j < k) acc = add_vec<DT>(acc, v[j]);
        st_stream(reinterpret_cast<uint4 *>(dst) + i, acc);
    }
    if (blockIdx.x == 0 && (int)threadIdx.x < tail) {
        if (DT == 0) {
            const size_t e = nvec * 4 + threadIdx.x;
            float acc = reinterpret_cast<const float *>(src.p[0])[e];
            for (int j = 1; j < k; ++j) acc = __fadd_rn(acc, reinterpret_cast<const float *>(src.p[j])[e]);
            reinterpret_cast<float *>(dst)[e] = acc;
        } else if (DT == 1) {
            const size_t e = nvec * 8 + threadIdx.x;
            unsigned short acc = reinterpret_cast<const unsigned short *>(src.p[0])[e];
            for (int j = 1; j < k; ++j) acc = add_bf16(acc, reinterpret_cast<const unsigned short *>(src.p[j])[e]);
            reinterpret_cast<unsigned short *>(dst)[e] = acc;
        } else {
            const size_t e = nvec * 2 + threadIdx.x;
            double acc = reinterpret_cast<const double *>(src.p[0])[e];
            for (int j = 1; j < k; ++j) acc = __dadd_rn(acc, reinterpret_cast<const double *>(src.p[j])[e]);
            reinterpret_cast<double *>(dst)[e] = acc;
        }
    }
}

// 32-byte vectors (256-bit accesses): half as many memory instructions and requests per byte.
struct Vec32 {
    uint32_t v[8];
};
__device__ __forceinline__ Vec32 ld_stream32(const Vec32 *p) {
    Vec32 r;
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}
__device__ __forceinline__ Vec32 ld_stream32_coherent(const Vec32 *p) {
    Vec32 r;
    asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ void st_stream32(Vec32 *p, const Vec32 &r) {
    asm volatile("st.global.cs.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r.v[0]), "r"(r.v[1]), "r"(r.v[2]),
                 "r"(r.v[3]), "r"(r.v[4]), "r"(r.v[5]), "r"(r.v[6]), "r"(r.v[7]) : "memory");
}
inline bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// 32-byte form of the broadcast: nvec32 vectors; the caller handles what is left with the 16-byte kernel.
constexpr int kUnroll32 = 4;
__global__ void __launch_bounds__(kStreamThreads)
broadcast_kernel32(const Vec32 *__restrict__ src, const __grid_constant__ FanPointers dst, int k, size_t nvec32) {
    const size_t stride = (size_t)gridDim.x * kStreamThreads;
    size_t i = (size_t)blockIdx.x * kStreamThreads + threadIdx.x;
    for (; i + (kUnroll32 - 1) * stride < nvec32; i += kUnroll32 * stride) {
        Vec32 v[kUnroll32];
#pragma unroll
        for (int u = 0; u < kUnroll32; ++u) v[u] = ld_stream32(src + i + u * stride);
        for (int j = 0; j < k; ++j) {
            Vec32 *d = reinterpret_cast<Vec32 *>(dst.p[j]);
#pragma unroll
            for (int u = 0; u < kUnroll32; ++u) st_stream32(d + i + u * stride, v[u]);
        }
    }
    for (; i < nvec32; i += stride) {
        const Vec32 v = ld_stream32(src + i);
        for (int j = 0; j < k; ++j) st_stream32(reinterpret_cast<Vec32 *>(dst.p[j]) + i, v);
    }
}

static int stream_grid(size_t nvec, int per_thread) {
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t want = (nvec + (size_t)kStreamThreads * per_thread - 1) / ((size_t)kStreamThreads * per_thread);
    const size_t cap = (size_t)sms * 8;   // 8 resident blocks of 256 threads per SM
    return (int)std::max<size_t>(1, std::min(want, cap));
}

static distdl_status_t broadcast_impl(const void *src, void *const *dst, int32_t k, int64_t n, distdl_dtype_t t,
                                      void *stream, const char *what) {
    clear_error();
    if (!src || !dst) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (k < 1 || n < 0) return fail(DISTDL_ERR_INVALID_ARG, "%s: k = %d, n = %lld", what, k, (long long)n);
    if (!valid_dtype(t)) return fail(DISTDL_ERR_INVALID_ARG, "%s: bad dtype", what);
    if (!aligned16(src)) return fail(DISTDL_ERR_ALIGNMENT, "%s: src is not 16-byte aligned", what);
    for (int32_t j = 0; j < k; ++j) {
        if (!dst[j]) return fail(DISTDL_ERR_INVALID_ARG, "%s: destination %d is NULL", what, j);
        if (!aligned16(dst[j])) return fail(DISTDL_ERR_ALIGNMENT, "%s: destination %d is not 16-byte aligned", what, j);
    }
    if (n == 0) return DISTDL_OK;
    const size_t bytes = (size_t)n * elem_size(t);
    const size_t nvec = bytes / 16;
    const int tail = (int)(bytes % 16);
    const int grid = stream_grid(nvec, kUnroll);
    // destinations in groups of kMaxFan; a destination equal to the source is the in-place form
    FanPointers fp;
    int filled = 0;
    for (int32_t j = 0; j <= k; ++j) {
        if (j < k && dst[j] != src) fp.p[filled++] = dst[j];
        if (filled == kMaxFan || (j == k && filled > 0)) {
            for (int r = filled; r < kMaxFan; ++r) fp.p[r] = nullptr;
            bool wide = aligned32(src) && bytes >= 32;
            for (int r = 0; r < filled; ++r) wide = wide && aligned32(fp.p[r]);
            if (wide) {
                // 256-bit accesses for the body, the 16-byte kernel for what is left (under 32 bytes)
                const size_t nvec32 = bytes / 32;
                broadcast_kernel32<<<stream_grid(nvec32, kUnroll32), kStreamThreads, 0, (cudaStream_t)stream>>>(
                    (const Vec32 *)src, fp, filled, nvec32);
                DISTDL_CUDA_CHECK(cudaGetLastError());
                const size_t done = nvec32 * 32;
                if (done < bytes) {
                    FanPointers rest;
                    for (int r = 0; r < kMaxFan; ++r) rest.p[r] = fp.p[r] ? (char *)fp.p[r] + done : nullptr;
                    broadcast_kernel<<<1, kStreamThreads, 0, (cudaStream_t)stream>>>(
                        (const uint4 *)((const char *)src + done), rest, filled, (bytes - done) / 16, tail);
                    DISTDL_CUDA_CHECK(cudaGetLastError());
                }
            } else {
                broadcast_kernel<<<grid, kStreamThreads, 0, (cudaStream_t)stream>>>((const uint4 *)src, fp, filled, nvec, tail);
                DISTDL_CUDA_CHECK(cudaGetLastError());
            }
            filled = 0;
        }
    }
    return DISTDL_OK;
}

template <int K>
static void launch_sum(const FanPointers &fp, void *dst, int k, size_t nvec, int tail, int grid, distdl_dtype_t t,
                       cudaStream_t s) {
    if (t == DISTDL_F32) sumreduce_kernel<K, 0><<<grid, kStreamThreads, 0, s>>>(fp, dst, k, nvec, tail);
    else if (t == DISTDL_BF16) sumreduce_kernel<K, 1><<<grid, kStreamThreads, 0, s>>>(fp, dst, k, nvec, tail);
    else sumreduce_kernel<K, 2><<<grid, kStreamThreads, 0, s>>>(fp, dst, k, nvec, tail);
}

static distdl_status_t sumreduce_impl(const void *const *src, void *dst, int32_t k, int64_t n, distdl_dtype_t t,
                                      void *stream, const char *what) {
    clear_error();
    if (!src || !dst) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (k < 1 || n < 0) return fail(DISTDL_ERR_INVALID_ARG, "%s: k = %d, n = %lld", what, k, (long long)n);
    if (!valid_dtype(t)) return fail(DISTDL_ERR_INVALID_ARG, "%s: bad dtype", what);
    if (!aligned16(dst)) return fail(DISTDL_ERR_ALIGNMENT, "%s: dst is not 16-byte aligned", what);
    for (int32_t j = 0; j < k; ++j) {
        if (!src[j]) return fail(DISTDL_ERR_INVALID_ARG, "%s: source %d is NULL", what, j);
        if (!aligned16(src[j])) return fail(DISTDL_ERR_ALIGNMENT, "%s: source %d is not 16-byte aligned", what, j);
        if (j > 0 && src[j] == dst) return fail(DISTDL_ERR_INVALID_ARG, "%s: dst may alias source 0 only", what);
    }
    if (n == 0) return DISTDL_OK;
    const int per = 16 / elem_size(t);
    const size_t nvec = (size_t)n / per;
    const int tail = (int)(n % per);
    const int grid = stream_grid(nvec, 1);
    // sources in groups of kMaxFan; later groups continue the fold from dst, which keeps the order
    int32_t done = 0;
    while (done < k) {
        FanPointers fp;
        int filled = 0;
        if (done > 0) fp.p[filled++] = dst;
        while (filled < kMaxFan && done < k) fp.p[filled++] = const_cast<void *>(src[done++]);
        for (int r = filled; r < kMaxFan; ++r) fp.p[r] = nullptr;
        cudaStream_t s = (cudaStream_t)stream;
        switch (filled) {
            case 1: launch_sum<1>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 2: launch_sum<2>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 3: launch_sum<3>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 4: launch_sum<4>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 5: launch_sum<5>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 6: launch_sum<6>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 7: launch_sum<7>(fp, dst, filled, nvec, tail, grid, t, s); break;
            case 8: launch_sum<8>(fp, dst, filled, nvec, tail, grid, t, s); break;
            default: launch_sum<0>(fp, dst, filled, nvec, tail, grid, t, s); break;
        }
        DISTDL_CUDA_CHECK(cudaGetLastError());
    }
    return DISTDL_OK;
}

// Broadcast / sum-reduce along partition dimensions (Section 4, the B and R of the layer algorithms): the
// destination partition repeats the source partition along the dimensions where the source has one worker.
// For every worker of the destination partition (row-major id) the worker of the source partition it copies.
static distdl_status_t partition_sources(int32_t rank, const int32_t *src_p, const int32_t *dst_p, std::vector<int32_t> *src_of,
                                         int32_t *num_src, const char *what) {
    if (!src_p || !dst_p) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL partition shape", what);
    if (rank < 1 || rank > DISTDL_MAX_RANK) return fail(DISTDL_ERR_INVALID_ARG, "%s: rank %d outside 1..%d", what, rank, DISTDL_MAX_RANK);
    int64_t ns = 1, nd = 1;
    for (int k = 0; k < rank; ++k) {
        if (src_p[k] < 1 || dst_p[k] < 1) return fail(DISTDL_ERR_SHAPE, "%s: partition dimension %d is not positive", what, k);
        if (src_p[k] != dst_p[k] && src_p[k] != 1)
            return fail(DISTDL_ERR_SHAPE, "%s: partition dimension %d has %d source and %d destination workers (equal, or one source worker)",
                        what, k, src_p[k], dst_p[k]);
        ns *= src_p[k];
        nd *= dst_p[k];
        if (nd > DISTDL_MAX_WORKERS) return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d workers", what, DISTDL_MAX_WORKERS);
    }
    src_of->resize((size_t)nd);
    for (int64_t w = 0; w < nd; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        int64_t rest = w;
        for (int k = rank - 1; k >= 0; --k) {
            c[k] = (int32_t)(rest % dst_p[k]);
            rest /= dst_p[k];
        }
        int32_t j = 0;
        for (int k = 0; k < rank; ++k) j = j * src_p[k] + (src_p[k] > 1 ? c[k] : 0);
        (*src_of)[(size_t)w] = j;
    }
    *num_src = (int32_t)ns;
    return DISTDL_OK;
}

static distdl_status_t partition_broadcast_impl(int32_t rank, const int32_t *src_p, const int32_t *dst_p, const int64_t *elems,
                                                const void *const *small, const void *const *big, distdl_dtype_t t,
                                                void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!elems || !small || !big) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    std::vector<int32_t> src_of;
    int32_t ns = 0;
    distdl_status_t st = partition_sources(rank, src_p, dst_p, &src_of, &ns, what);
    if (st != DISTDL_OK) return st;
    for (int32_t j = 0; j < ns; ++j) {
        if (elems[j] < 0) return fail(DISTDL_ERR_INVALID_ARG, "%s: negative element count for source worker %d", what, j);
        if (!small[j]) return fail(DISTDL_ERR_INVALID_ARG, "%s: buffer of source-partition worker %d is NULL", what, j);
    }
    for (size_t w = 0; w < src_of.size(); ++w)
        if (!big[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: buffer of destination-partition worker %zu is NULL", what, w);
    std::vector<void *> group;
    for (int32_t j = 0; j < ns; ++j) {
        group.clear();
        for (size_t w = 0; w < src_of.size(); ++w)
            if (src_of[w] == j) group.push_back(const_cast<void *>(big[w]));      // ascending worker id: the order of the sum
        st = adjoint ? sumreduce_impl(group.data(), const_cast<void *>(small[j]), (int32_t)group.size(), elems[j], t, stream, what)
                     : broadcast_impl(small[j], group.data(), (int32_t)group.size(), elems[j], t, stream, what);
        if (st != DISTDL_OK) return st;
    }
    return DISTDL_OK;
}

}  // namespace distdl

extern "C" distdl_status_t distdl_partition_broadcast_fwd(int32_t rank, const int32_t *src_partition_shape,
                                                          const int32_t *dst_partition_shape, const int64_t *elems,
                                                          const void *const *src, void *const *dst, distdl_dtype_t t,
                                                          void *stream) {
    return distdl::partition_broadcast_impl(rank, src_partition_shape, dst_partition_shape, elems, src,
                                            reinterpret_cast<const void *const *>(dst), t, stream, false, "partition_broadcast_fwd");
}
extern "C" distdl_status_t distdl_partition_broadcast_adj(int32_t rank, const int32_t *src_partition_shape,
                                                          const int32_t *dst_partition_shape, const int64_t *elems,
                                                          const void *const *dy, void *const *dx, distdl_dtype_t t,
                                                          void *stream) {
    return distdl::partition_broadcast_impl(rank, src_partition_shape, dst_partition_shape, elems,
                                            reinterpret_cast<const void *const *>(dx), dy, t, stream, true, "partition_broadcast_adj");
}

extern "C" distdl_status_t distdl_broadcast_fwd(const void *src, void *const *dst, int32_t k, int64_t n,
                                                distdl_dtype_t t, void *stream) {
    return distdl::broadcast_impl(src, dst, k, n, t, stream, "broadcast_fwd");
}
extern "C" distdl_status_t distdl_sumreduce_adj(const void *dy, void *const *dx, int32_t k, int64_t n,
                                                distdl_dtype_t t, void *stream) {
    return distdl::broadcast_impl(dy, dx, k, n, t, stream, "sumreduce_adj");
}
extern "C" distdl_status_t distdl_sumreduce_fwd(const void *const *src, void *dst, int32_t k, int64_t n,
                                                distdl_dtype_t t, void *stream) {
    return distdl::sumreduce_impl(src, dst, k, n, t, stream, "sumreduce_fwd");
}
extern "C" distdl_status_t distdl_broadcast_adj(const void *const *dy, void *dx, int32_t k, int64_t n,
                                                distdl_dtype_t t, void *stream) {
    return distdl::sumreduce_impl(dy, dx, k, n, t, stream, "broadcast_adj");
}

extern "C" distdl_status_t distdl_allreduce(void *const *bufs, int32_t k, int64_t n, distdl_dtype_t t, void *stream) {
    // A = B R: the fixed-order sum lands in bufs[0] (a sum may be written over its first source), then goes out
    // to the other k - 1 buffers (the broadcast skips a destination equal to the source)
    distdl_status_t st = distdl::sumreduce_impl(reinterpret_cast<const void *const *>(bufs), bufs ? bufs[0] : nullptr, k, n, t,
                                                stream, "allreduce");
    if (st != DISTDL_OK) return st;
    return distdl::broadcast_impl(bufs[0], bufs, k, n, t, stream, "allreduce");
}
