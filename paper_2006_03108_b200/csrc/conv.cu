// Distributed depthwise convolution layer on a feature-space partition (Section 4, "Sparse
// layers"): forward = halo exchange H followed by the local sliding-kernel layer, adjoint =
// local adjoint followed by H*.  Both are fused: a thread block stages its input tile, ghost
// rows and columns included, in shared memory straight from the bulk of the neighbouring shards
// (or zeros outside the tensor), so ghost data never makes a round trip through device memory.
// The adjoint is evaluated in gather form (a correlation of dy with the kernel rotated by 180
// degrees), which equals "scatter locally, then add the ghosts into the neighbours' bulk" without
// any atomics, and it leaves the ghosts of dx zero as H* does.
#include <algorithm>
#include <cstring>

#include "common.h"

namespace distdl {

constexpr int kConvMaxWorkers = 64;
constexpr int kConvThreads = 256;
constexpr int kTileH = 64;    // output rows per block
constexpr int kTileW = 128;   // output columns per block
constexpr int kRowsPerThread = 8;

struct ConvParams {
    const float *in[kConvMaxWorkers];
    float *out[kConvMaxWorkers];
    int32_t bh[kConvMaxWorkers];   // bulk rows per worker-row coordinate
    int32_t bw[kConvMaxWorkers];   // bulk columns per worker-column coordinate
    const float *w;                // [C, K, K]
    const float *bias;             // [C] or nullptr
    int32_t ph_workers, pw_workers;
    int32_t channels;
    int32_t tiles_x;
};

// Row pitch (floats) of the shared-memory tile: wide enough for the staged columns (outputs plus
// PADL columns on the left and PH on the right, rounded up to whole float4s) and for the last
// thread's float4 window.
__host__ __device__ constexpr int conv_pitch(int K, bool adj) {
    const int ph = K / 2;
    const int padl = adj ? ((ph + 3) / 4) * 4 : ph;
    const int nv = (padl - ph + K + 3 + 3) / 4;
    const int staged = ((kTileW + padl + ph + 3) / 4) * 4;
    const int window = kTileW - 4 + 4 * nv;
    return staged > window ? staged : window;
}

__device__ __forceinline__ void cp_async16(float *smem, const float *gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// K: kernel extent (odd).  ADJ: false = forward (padded x -> bulk-shaped y), true = adjoint
// (bulk-shaped dy -> padded dx, rotated kernel, ghosts of dx cleared).
template <int K, bool ADJ>
__global__ void __launch_bounds__(kConvThreads, 2)
conv_depthwise_kernel(const __grid_constant__ ConvParams P) {
    constexpr int PH = K / 2;                    // halo rows = halo columns
    constexpr int PADL = ADJ ? ((PH + 3) / 4) * 4 : PH;   // shared-memory columns left of the first output
    constexpr int WOFF = PADL - PH;              // first column a thread needs, relative to its float4 slot
    constexpr int NV = (WOFF + K + 3 + 3) / 4;   // float4 loads per thread per input row
    constexpr int PITCH = conv_pitch(K, ADJ);
    extern __shared__ __align__(16) float tile[];   // [kTileH + K - 1][PITCH]

    const int shard = blockIdx.z;
    const int plane = blockIdx.y;
    const int r = shard / P.pw_workers, c = shard % P.pw_workers;
    const int bh = P.bh[r], bw = P.bw[c];
    const int i0 = (blockIdx.x / P.tiles_x) * kTileH;
    const int j0 = (blockIdx.x % P.tiles_x) * kTileW;
    if (i0 >= bh || j0 >= bw) return;
    const int ch = plane % P.channels;

    // input layout of a shard with bulk (h, w): forward = padded (h + 2PH, w + 2PH), bulk at
    // (PH, PH); adjoint = bulk-shaped.
    constexpr int IOFF = ADJ ? 0 : PH;
    // ---------------------------------------------------------------- stage the input tile
    // shared column s  <->  bulk column j0 - PADL + s ;  shared row ry  <->  bulk row i0 - PH + ry
    const int need_cols = min(kTileW, bw - j0) + PADL + PH;           // columns that can be read
    const int nvec_row = (need_cols + 3) / 4;
    const int need_rows = min(kTileH, bh - i0) + 2 * PH;
    for (int idx = threadIdx.x; idx < need_rows * nvec_row; idx += kConvThreads) {
        const int ry = idx / nvec_row, v = idx - ry * nvec_row;
        float *dst = tile + ry * PITCH + 4 * v;
        // resolve the row: which worker row owns bulk row i, or none (outside the tensor)
        int i = i0 - PH + ry, rr = r;
        bool row_ok = true;
        if (i < 0) {
            rr = r - 1;
            row_ok = rr >= 0;
            if (row_ok) i += P.bh[rr];
        } else if (i >= bh) {
            rr = r + 1;
            row_ok = rr < P.ph_workers;
            i -= bh;
            if (row_ok) row_ok = i < P.bh[rr];
        }
        if (!row_ok) {
            *reinterpret_cast<float4 *>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
            continue;
        }
        const int rbh = P.bh[rr];
        const int jfirst = j0 - PADL + 4 * v;        // bulk column of the vector's first element
        // fast path: the four columns lie in this worker column's bulk and the address is aligned
        const int pitch_c = bw + 2 * IOFF;
        const size_t plane_c = (size_t)(rbh + 2 * IOFF) * pitch_c;
        const float *row_c = P.in[rr * P.pw_workers + c] + plane * plane_c + (size_t)(i + IOFF) * pitch_c + IOFF;
        if (jfirst >= 0 && jfirst + 3 < bw && ((reinterpret_cast<uintptr_t>(row_c + jfirst) & 15u) == 0)) {
            cp_async16(dst, row_c + jfirst);
            continue;
        }
        float vals[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int j = jfirst + e, cc = c;
            bool ok = true;
            if (j < 0) {
                cc = c - 1;
                ok = cc >= 0;
                if (ok) j += P.bw[cc];
                if (ok) ok = j >= 0;
            } else if (j >= bw) {
                cc = c + 1;
                ok = cc < P.pw_workers;
                j -= bw;
                if (ok) ok = j < P.bw[cc];
            }
            float val = 0.f;
            if (ok) {
                const int pitch_n = P.bw[cc] + 2 * IOFF;
                const size_t plane_n = (size_t)(rbh + 2 * IOFF) * pitch_n;
                val = __ldg(P.in[rr * P.pw_workers + cc] + plane * plane_n + (size_t)(i + IOFF) * pitch_n + IOFF + j);
            }
            vals[e] = val;
        }
        *reinterpret_cast<float4 *>(dst) = make_float4(vals[0], vals[1], vals[2], vals[3]);
    }

    // ---------------------------------------------------------------- weights to registers
    float wreg[K * K];
#pragma unroll
    for (int t = 0; t < K * K; ++t) {
        // adjoint: kernel rotated by 180 degrees
        wreg[t] = __ldg(P.w + (size_t)ch * K * K + (ADJ ? K * K - 1 - t : t));
    }
    const float b0 = (!ADJ && P.bias) ? __ldg(P.bias + ch) : 0.f;

    // ---------------------------------------------------------------- clear the ghosts of dx
    if (ADJ) {
        const int pitch_o = bw + 2 * PH;
        float *oplane = P.out[shard] + (size_t)plane * (bh + 2 * PH) * pitch_o;
        const int i1 = min(i0 + kTileH, bh), j1 = min(j0 + kTileW, bw);
        // padded row / column ranges this block is responsible for (ring included at the edges)
        const int R0 = i0 == 0 ? 0 : i0 + PH, R1 = i1 == bh ? bh + 2 * PH : i1 + PH;
        const int C0 = j0 == 0 ? 0 : j0 + PH, C1 = j1 == bw ? bw + 2 * PH : j1 + PH;
        const int ncol = C1 - C0;
        if (i0 == 0)
            for (int t = threadIdx.x; t < PH * ncol; t += kConvThreads) oplane[(size_t)(t / ncol) * pitch_o + C0 + t % ncol] = 0.f;
        if (i1 == bh)
            for (int t = threadIdx.x; t < PH * ncol; t += kConvThreads) oplane[(size_t)(bh + PH + t / ncol) * pitch_o + C0 + t % ncol] = 0.f;
        const int Rb0 = max(R0, PH), Rb1 = min(R1, bh + PH);   // rows of the bulk band
        if (j0 == 0)
            for (int t = threadIdx.x; t < (Rb1 - Rb0) * PH; t += kConvThreads) oplane[(size_t)(Rb0 + t / PH) * pitch_o + t % PH] = 0.f;
        if (j1 == bw)
            for (int t = threadIdx.x; t < (Rb1 - Rb0) * PH; t += kConvThreads) oplane[(size_t)(Rb0 + t / PH) * pitch_o + bw + PH + t % PH] = 0.f;
    }

    cp_async_wait_all();
    __syncthreads();

    // ---------------------------------------------------------------- register-tiled stencil
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    float acc[kRowsPerThread][4];
#pragma unroll
    for (int a = 0; a < kRowsPerThread; ++a)
#pragma unroll
        for (int t = 0; t < 4; ++t) acc[a][t] = b0;

    const float *trow = tile + (ty * kRowsPerThread) * PITCH + 4 * tx;
#pragma unroll
    for (int ry = 0; ry < kRowsPerThread + K - 1; ++ry) {
        float in[4 * NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float4 q = *reinterpret_cast<const float4 *>(trow + ry * PITCH + 4 * v);
            in[4 * v + 0] = q.x; in[4 * v + 1] = q.y; in[4 * v + 2] = q.z; in[4 * v + 3] = q.w;
        }
#pragma unroll
        for (int a = 0; a < K; ++a) {
            const int orow = ry - a;       // output row (within the thread's strip) fed by tap row a
            if (orow >= 0 && orow < kRowsPerThread) {
#pragma unroll
                for (int b = 0; b < K; ++b)
#pragma unroll
                    for (int t = 0; t < 4; ++t)
                        acc[orow][t] = fmaf(wreg[a * K + b], in[WOFF + t + b], acc[orow][t]);
            }
        }
    }

    // ---------------------------------------------------------------- store
    constexpr int OOFF = ADJ ? PH : 0;
    const int pitch_o = bw + 2 * OOFF;
    float *oplane = P.out[shard] + (size_t)plane * (bh + 2 * OOFF) * pitch_o;
    const int jo = j0 + 4 * tx;
#pragma unroll
    for (int a = 0; a < kRowsPerThread; ++a) {
        const int io = i0 + ty * kRowsPerThread + a;
        if (io >= bh || jo >= bw) continue;
        float *o = oplane + (size_t)(io + OOFF) * pitch_o + OOFF + jo;
        if (jo + 3 < bw && (reinterpret_cast<uintptr_t>(o) & 15u) == 0) {
            *reinterpret_cast<float4 *>(o) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        } else if (jo + 3 < bw && (reinterpret_cast<uintptr_t>(o) & 7u) == 0) {
            *reinterpret_cast<float2 *>(o) = make_float2(acc[a][0], acc[a][1]);
            *reinterpret_cast<float2 *>(o + 2) = make_float2(acc[a][2], acc[a][3]);
        } else {
#pragma unroll
            for (int t = 0; t < 4; ++t)
                if (jo + t < bw) o[t] = acc[a][t];
        }
    }
}

template <int K, bool ADJ>
static constexpr int conv_smem_bytes() {
    return (kTileH + K - 1) * conv_pitch(K, ADJ) * (int)sizeof(float);
}

template <int K, bool ADJ>
static distdl_status_t launch_conv(const ConvParams &P, dim3 grid, cudaStream_t s) {
    constexpr int smem = conv_smem_bytes<K, ADJ>();
    static bool configured = false;
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_depthwise_kernel<K, ADJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        configured = true;
    }
    conv_depthwise_kernel<K, ADJ><<<grid, kConvThreads, smem, s>>>(P);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

static distdl_status_t conv_impl(const distdl_partition *p, const void *const *in, const void *w, const void *bias,
                                 int32_t kh, int32_t kw, void *const *out, void *stream, bool adj, const char *what) {
    clear_error();
    if (!p || !in || !w || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (p->rank != 4 || p->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (p->pshape[0] != 1 || p->pshape[1] != 1)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: only the feature-space dimensions may be partitioned", what);
    if (kh != kw || (kh != 3 && kh != 5 && kh != 7))
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: kernel %d x %d (supported: 3x3, 5x5, 7x7)", what, kh, kw);
    if (p->num_workers > kConvMaxWorkers) return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d workers", what, kConvMaxWorkers);
    const int h = kh / 2;
    for (int k = 0; k < 4; ++k)
        for (int32_t c = 0; c < p->pshape[k]; ++c) {
            const int want = k < 2 ? 0 : h;
            if (p->hlo[k][c] != want || p->hhi[k][c] != want)
                return fail(DISTDL_ERR_SHAPE, "%s: halo widths must be 0,0,%d,%d on every side", what, h, h);
        }
    if (!aligned16(w) || (bias && !aligned16(bias))) return fail(DISTDL_ERR_ALIGNMENT, "%s: w / bias not 16-byte aligned", what);
    const int64_t planes = p->global_shape[0] * p->global_shape[1];
    if (planes > 65535) return fail(DISTDL_ERR_UNSUPPORTED, "%s: N*C > 65535", what);
    ConvParams P;
    memset(&P, 0, sizeof(P));
    int64_t max_bh = 0, max_bw = 0;
    for (int32_t r = 0; r < p->pshape[2]; ++r) {
        P.bh[r] = (int32_t)p->size[2][r];
        max_bh = std::max<int64_t>(max_bh, p->size[2][r]);
    }
    for (int32_t c = 0; c < p->pshape[3]; ++c) {
        P.bw[c] = (int32_t)p->size[3][c];
        max_bw = std::max<int64_t>(max_bw, p->size[3][c]);
    }
    for (int32_t wk = 0; wk < p->num_workers; ++wk) {
        if (!in[wk] || !out[wk]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shard pointer %d is NULL", what, wk);
        if (!aligned16(in[wk]) || !aligned16(out[wk])) return fail(DISTDL_ERR_ALIGNMENT, "%s: shard %d is not 16-byte aligned", what, wk);
        P.in[wk] = (const float *)in[wk];
        P.out[wk] = (float *)out[wk];
    }
    P.w = (const float *)w;
    P.bias = (const float *)bias;
    P.ph_workers = p->pshape[2];
    P.pw_workers = p->pshape[3];
    P.channels = (int32_t)p->global_shape[1];
    P.tiles_x = (int32_t)((max_bw + kTileW - 1) / kTileW);
    const int tiles_y = (int)((max_bh + kTileH - 1) / kTileH);
    dim3 grid((unsigned)(P.tiles_x * tiles_y), (unsigned)planes, (unsigned)p->num_workers);
    cudaStream_t s = (cudaStream_t)stream;
    if (!adj) {
        if (kh == 3) return launch_conv<3, false>(P, grid, s);
        if (kh == 5) return launch_conv<5, false>(P, grid, s);
        return launch_conv<7, false>(P, grid, s);
    }
    if (kh == 3) return launch_conv<3, true>(P, grid, s);
    if (kh == 5) return launch_conv<5, true>(P, grid, s);
    return launch_conv<7, true>(P, grid, s);
}

}  // namespace distdl

extern "C" distdl_status_t distdl_conv_fwd(const distdl_partition_t *p, const void *const *x, const void *w,
                                           const void *bias, int32_t kh, int32_t kw, void *const *y, void *stream) {
    return distdl::conv_impl(p, x, w, bias, kh, kw, y, stream, false, "conv_fwd");
}
extern "C" distdl_status_t distdl_conv_adj(const distdl_partition_t *p, const void *const *dy, const void *w,
                                           int32_t kh, int32_t kw, void *const *dx, void *stream) {
    return distdl::conv_impl(p, dy, w, nullptr, kh, kw, dx, stream, true, "conv_adj");
}
