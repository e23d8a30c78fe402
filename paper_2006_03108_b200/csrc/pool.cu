// Distributed pooling layer on a feature-space partition with unbalanced halos (Section 4,
// "Sparse layers": pooling follows the convolution algorithms without weights; Section 3 and
// Appendix B: the halo widths of a strided kernel differ from worker to worker and some owned
// inputs may go unused).
//
// forward = halo exchange H (the library's in-place kernel), then the local sliding kernel over
// each worker's padded shard, starting at the first input the worker's block of the evenly split
// output needs; adjoint = local adjoint into every cell of the padded shard (ghosts included),
// then H*.  The local adjoint is evaluated in gather form -- a cell sums over the outputs whose
// window holds it, in ascending output order -- so overlapping windows need no atomics.
#include <algorithm>
#include <cstring>
#include <vector>

#include "common.h"

namespace distdl {

constexpr int kPoolMaxWorkers = 32;
constexpr int kPoolThreadsX = 32, kPoolThreadsY = 8;

struct PoolShard {
    const float *in;       // forward: padded x;   adjoint: dy
    float *out;            // forward: y;          adjoint: padded dx
    int32_t *arg;          // position of the maximum inside the window (a * kw + b), or nullptr
    int32_t ph, pw;        // padded extents of the shard (rows, columns)
    int32_t oh, ow;        // this worker's block of the output
    int32_t i0, j0;        // padded-local index of the first input of output (0, 0)
    int32_t g0h, g0w;      // global index of padded-local index 0
};

struct PoolParams {
    PoolShard s[kPoolMaxWorkers];
    int32_t planes, kh, kw, sh, sw, hg, wg, mode;
};

// One thread per output.  blockIdx.y = worker, blockIdx.x = (plane, row tile, column tile).
__global__ void __launch_bounds__(kPoolThreadsX *kPoolThreadsY)
pool_fwd_kernel(const __grid_constant__ PoolParams P, int tiles_x, int tiles_y) {
    const PoolShard &S = P.s[blockIdx.y];
    int rest = blockIdx.x;
    const int tx = rest % tiles_x;
    rest /= tiles_x;
    const int ty = rest % tiles_y;
    const int plane = rest / tiles_y;
    const int j = tx * kPoolThreadsX + threadIdx.x, i = ty * kPoolThreadsY + threadIdx.y;
    if (i >= S.oh || j >= S.ow || plane >= P.planes) return;
    const int r0 = S.i0 + i * P.sh, c0 = S.j0 + j * P.sw;
    const float *src = S.in + ((size_t)plane * S.ph + r0) * S.pw + c0;
    const size_t o = ((size_t)plane * S.oh + i) * S.ow + j;
    if (P.mode == DISTDL_POOL_AVG) {
        float acc = 0.f;
        for (int a = 0; a < P.kh; ++a)
            for (int b = 0; b < P.kw; ++b) acc = __fadd_rn(acc, src[a * S.pw + b]);
        S.out[o] = __fmul_rn(acc, 1.0f / (float)(P.kh * P.kw));
    } else {
        // largest value of the window clipped to the tensor; the first one in row-major order wins
        float best = 0.f;
        int where = -1;
        for (int a = 0; a < P.kh; ++a) {
            const int gi = S.g0h + r0 + a;
            if (gi < 0 || gi >= P.hg) continue;
            for (int b = 0; b < P.kw; ++b) {
                const int gj = S.g0w + c0 + b;
                if (gj < 0 || gj >= P.wg) continue;
                const float v = src[a * S.pw + b];
                if (where < 0 || v > best) {
                    best = v;
                    where = a * P.kw + b;
                }
            }
        }
        S.out[o] = best;
        if (S.arg) S.arg[o] = where < 0 ? 0 : where;
    }
}

__device__ __forceinline__ int div_floor(int a, int b) { return a >= 0 ? a / b : -((-a + b - 1) / b); }

// One thread per cell of the padded dx.  A cell (p, q) lies in the window of output (i, j) iff
// 0 <= p - i0 - i*sh < kh and likewise for the columns.
__global__ void __launch_bounds__(kPoolThreadsX *kPoolThreadsY)
pool_adj_kernel(const __grid_constant__ PoolParams P, int tiles_x, int tiles_y) {
    const PoolShard &S = P.s[blockIdx.y];
    int rest = blockIdx.x;
    const int tx = rest % tiles_x;
    rest /= tiles_x;
    const int ty = rest % tiles_y;
    const int plane = rest / tiles_y;
    const int q = tx * kPoolThreadsX + threadIdx.x, p = ty * kPoolThreadsY + threadIdx.y;
    if (p >= S.ph || q >= S.pw || plane >= P.planes) return;
    const int dp = p - S.i0, dq = q - S.j0;
    const int i_lo = max(0, div_floor(dp - P.kh + P.sh, P.sh)), i_hi = min(S.oh - 1, div_floor(dp, P.sh));
    const int j_lo = max(0, div_floor(dq - P.kw + P.sw, P.sw)), j_hi = min(S.ow - 1, div_floor(dq, P.sw));
    const float *dy = S.in + (size_t)plane * S.oh * S.ow;
    const int32_t *arg = S.arg ? S.arg + (size_t)plane * S.oh * S.ow : nullptr;
    float acc = 0.f;
    for (int i = i_lo; i <= i_hi; ++i)
        for (int j = j_lo; j <= j_hi; ++j) {
            if (P.mode == DISTDL_POOL_AVG) {
                acc = __fadd_rn(acc, dy[i * S.ow + j]);
            } else {
                const int a = dp - i * P.sh, b = dq - j * P.sw;
                if (arg[i * S.ow + j] == a * P.kw + b) acc = __fadd_rn(acc, dy[i * S.ow + j]);
            }
        }
    if (P.mode == DISTDL_POOL_AVG) acc = __fmul_rn(acc, 1.0f / (float)(P.kh * P.kw));
    S.out[((size_t)plane * S.ph + p) * S.pw + q] = acc;
}

// ---------------------------------------------------------------------------------------------
// Variants with the kernel and stride fixed at compile time (2 x 2 / 2 and 3 x 3 / 2, the pooling
// layers of the usual networks): index arithmetic in shifts, and four outputs (forward) or cells
// (adjoint) per thread, 32 columns apart, so that the lanes of a warp always touch neighbouring
// addresses.  Same sums in the same order as the general kernels above.
// ---------------------------------------------------------------------------------------------
constexpr int kPoolPerThread = 4;

template <int KH, int KW, int SH, int SW, int MODE>
__global__ void __launch_bounds__(kPoolThreadsX *kPoolThreadsY)
pool_fwd_fixed(const __grid_constant__ PoolParams P, int tiles_x, int tiles_y) {
    const PoolShard &S = P.s[blockIdx.y];
    int rest = blockIdx.x;
    const int tx = rest % tiles_x;
    rest /= tiles_x;
    const int ty = rest % tiles_y;
    const int plane = rest / tiles_y;
    const int jb = tx * kPoolThreadsX * kPoolPerThread + threadIdx.x, i = ty * kPoolThreadsY + threadIdx.y;
    if (i >= S.oh) return;
    const int r0 = S.i0 + i * SH;
    const float *row = S.in + ((size_t)plane * S.ph + r0) * S.pw + S.j0;
    float *orow = S.out + ((size_t)plane * S.oh + i) * S.ow;
    int32_t *arow = (MODE == DISTDL_POOL_MAX && S.arg) ? S.arg + ((size_t)plane * S.oh + i) * S.ow : nullptr;
    bool row_in[KH];
#pragma unroll
    for (int a = 0; a < KH; ++a) row_in[a] = S.g0h + r0 + a >= 0 && S.g0h + r0 + a < P.hg;
    bool rows_inside = true;
#pragma unroll
    for (int a = 0; a < KH; ++a) rows_inside = rows_inside && row_in[a];
#pragma unroll
    for (int u = 0; u < kPoolPerThread; ++u) {
        const int j = jb + u * kPoolThreadsX;
        if (j >= S.ow) break;
        const float *src = row + j * SW;
        const int gj0 = S.g0w + S.j0 + j * SW;
        float acc = 0.f;
        int where = -1;
        if (MODE == DISTDL_POOL_AVG) {
#pragma unroll
            for (int a = 0; a < KH; ++a)
#pragma unroll
                for (int b = 0; b < KW; ++b) acc = __fadd_rn(acc, src[a * S.pw + b]);
            acc = __fmul_rn(acc, 1.0f / (float)(KH * KW));
        } else if (rows_inside && gj0 >= 0 && gj0 + KW <= P.wg) {
            // the whole window lies inside the tensor: no cell to exclude
            acc = src[0];
            where = 0;
#pragma unroll
            for (int a = 0; a < KH; ++a)
#pragma unroll
                for (int b = 0; b < KW; ++b) {
                    if (a == 0 && b == 0) continue;
                    const float v = src[a * S.pw + b];
                    if (v > acc) {
                        acc = v;
                        where = a * KW + b;
                    }
                }
        } else {
#pragma unroll
            for (int a = 0; a < KH; ++a)
#pragma unroll
                for (int b = 0; b < KW; ++b) {
                    const float v = src[a * S.pw + b];
                    if (row_in[a] && gj0 + b >= 0 && gj0 + b < P.wg && (where < 0 || v > acc)) {
                        acc = v;
                        where = a * KW + b;
                    }
                }
        }
        orow[j] = acc;
        if (arow) arow[j] = where < 0 ? 0 : where;
    }
}

// Adjoint: a thread owns the SH x SW cells {i0 + SH*gi + r, j0 + SW*gj + c}.  The outputs whose window holds
// cell (r, c) of the group are (gi - t, gj - v) with window positions a = r + t*SH < KH, b = c + v*SW < KW, all
// known at compile time; the thread loads the NI x NJ candidate outputs once and every cell picks its terms
// (ascending output order = descending t, v).  tiles count groups: row group = first group + tile row, and so on.
template <int KH, int KW, int SH, int SW, int MODE>
__global__ void __launch_bounds__(kPoolThreadsX *kPoolThreadsY)
pool_adj_fixed(const __grid_constant__ PoolParams P, int tiles_x, int tiles_y) {
    const PoolShard &S = P.s[blockIdx.y];
    int rest = blockIdx.x;
    const int tx = rest % tiles_x;
    rest /= tiles_x;
    const int ty = rest % tiles_y;
    const int plane = rest / tiles_y;
    constexpr int NI = (KH + SH - 1) / SH, NJ = (KW + SW - 1) / SW;
    // the first group holds padded row / column 0
    const int gi = div_floor(-S.i0, SH) + ty * kPoolThreadsY + (int)threadIdx.y;
    const int gjb = div_floor(-S.j0, SW) + tx * kPoolThreadsX * kPoolPerThread + (int)threadIdx.x;
    const int p0 = S.i0 + gi * SH;
    if (p0 >= S.ph) return;
    const float *dy = S.in + (size_t)plane * S.oh * S.ow;
    const int32_t *arg = MODE == DISTDL_POOL_MAX ? S.arg + (size_t)plane * S.oh * S.ow : nullptr;
    float *oplane = S.out + (size_t)plane * S.ph * S.pw;
#pragma unroll
    for (int u = 0; u < kPoolPerThread; ++u) {
        const int gj = gjb + u * kPoolThreadsX;
        const int q0 = S.j0 + gj * SW;
        if (q0 >= S.pw) break;
        float g[NI][NJ];
        int code[NI][NJ];          // MAX: recorded position, -1 for an absent output; AVG: 0 present, -1 absent
        const bool interior = gi - (NI - 1) >= 0 && gi < S.oh && gj - (NJ - 1) >= 0 && gj < S.ow && p0 >= 0 &&
                              p0 + SH <= S.ph && q0 >= 0 && q0 + SW <= S.pw;
        if (interior) {
            // every candidate output exists and every cell of the group lies in the shard: no tests, 32-bit offsets
            const uint32_t o = (uint32_t)(gi * S.ow + gj);
#pragma unroll
            for (int t = 0; t < NI; ++t)
#pragma unroll
                for (int v = 0; v < NJ; ++v) {
                    g[t][v] = dy[o - (uint32_t)(t * S.ow + v)];
                    code[t][v] = MODE == DISTDL_POOL_MAX ? arg[o - (uint32_t)(t * S.ow + v)] : 0;
                }
            float *dst = oplane + (uint32_t)(p0 * S.pw + q0);
#pragma unroll
            for (int r = 0; r < SH; ++r)
#pragma unroll
                for (int c = 0; c < SW; ++c) {
                    float acc = 0.f;
#pragma unroll
                    for (int t = NI - 1; t >= 0; --t)
#pragma unroll
                        for (int v = NJ - 1; v >= 0; --v) {
                            if (r + t * SH >= KH || c + v * SW >= KW) continue;      // compile-time
                            if (MODE == DISTDL_POOL_AVG) acc = __fadd_rn(acc, g[t][v]);
                            else if (code[t][v] == (r + t * SH) * KW + (c + v * SW)) acc = __fadd_rn(acc, g[t][v]);
                        }
                    if (MODE == DISTDL_POOL_AVG) acc = __fmul_rn(acc, 1.0f / (float)(KH * KW));
                    dst[r * S.pw + c] = acc;
                }
            continue;
        }
#pragma unroll
        for (int t = 0; t < NI; ++t)
#pragma unroll
            for (int v = 0; v < NJ; ++v) {
                const int i = gi - t, j = gj - v;
                const bool in = i >= 0 && i < S.oh && j >= 0 && j < S.ow;
                g[t][v] = in ? dy[i * S.ow + j] : 0.f;
                code[t][v] = !in ? -1 : (MODE == DISTDL_POOL_MAX ? arg[i * S.ow + j] : 0);
            }
#pragma unroll
        for (int r = 0; r < SH; ++r) {
            const int p = p0 + r;
            if (p < 0 || p >= S.ph) continue;
#pragma unroll
            for (int c = 0; c < SW; ++c) {
                const int q = q0 + c;
                if (q < 0 || q >= S.pw) continue;
                float acc = 0.f;
#pragma unroll
                for (int t = NI - 1; t >= 0; --t)
#pragma unroll
                    for (int v = NJ - 1; v >= 0; --v) {
                        if (r + t * SH >= KH || c + v * SW >= KW) continue;      // compile-time
                        const bool take = MODE == DISTDL_POOL_AVG ? code[t][v] == 0
                                                                  : code[t][v] == (r + t * SH) * KW + (c + v * SW);
                        if (take) acc = __fadd_rn(acc, g[t][v]);
                    }
                if (MODE == DISTDL_POOL_AVG) acc = __fmul_rn(acc, 1.0f / (float)(KH * KW));
                oplane[(size_t)p * S.pw + q] = acc;
            }
        }
    }
}

template <int KH, int KW, int SH, int SW>
static void launch_pool_fixed(const PoolParams &P, dim3 grid, dim3 block, int tiles_x, int tiles_y, bool adjoint, cudaStream_t s) {
    if (!adjoint) {
        if (P.mode == DISTDL_POOL_AVG) pool_fwd_fixed<KH, KW, SH, SW, DISTDL_POOL_AVG><<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
        else pool_fwd_fixed<KH, KW, SH, SW, DISTDL_POOL_MAX><<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
    } else {
        if (P.mode == DISTDL_POOL_AVG) pool_adj_fixed<KH, KW, SH, SW, DISTDL_POOL_AVG><<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
        else pool_adj_fixed<KH, KW, SH, SW, DISTDL_POOL_MAX><<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
    }
}

struct PoolDim {
    std::vector<int64_t> out_start, out_size;
    std::vector<int32_t> hlo, hhi;
};

static distdl_status_t pool_dim(int64_t n, int32_t p, int32_t k, int32_t s, int32_t pad_lo, int32_t pad_hi, PoolDim &d,
                                const char *what) {
    d.hlo.resize(p);
    d.hhi.resize(p);
    const distdl_status_t st = distdl_halo_widths_1d(n, p, k, s, 1, pad_lo, pad_hi, d.hlo.data(), d.hhi.data(), nullptr, nullptr);
    if (st != DISTDL_OK) return st;
    const int64_t m = (n + pad_lo + pad_hi - k) / s + 1;
    const int64_t q = m / p, r = m % p;
    d.out_start.resize(p);
    d.out_size.resize(p);
    int64_t at = 0;
    for (int32_t c = 0; c < p; ++c) {
        d.out_size[c] = q + (c < r ? 1 : 0);
        d.out_start[c] = at;
        at += d.out_size[c];
    }
    (void)what;
    return DISTDL_OK;
}

static distdl_status_t pool_impl(const distdl_partition *p, const void *const *in, void *const *out, void *const *arg,
                                 int32_t kh, int32_t kw, int32_t sh, int32_t sw, int32_t plh, int32_t phh, int32_t plw,
                                 int32_t phw, int32_t mode, void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!p || !in || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (p->rank != 4 || p->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (p->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
    if (p->pshape[0] != 1 || p->pshape[1] != 1)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: only the feature-space dimensions may be partitioned", what);
    if (p->num_workers > kPoolMaxWorkers) return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d workers", what, kPoolMaxWorkers);
    if (mode != DISTDL_POOL_AVG && mode != DISTDL_POOL_MAX) return fail(DISTDL_ERR_INVALID_ARG, "%s: bad mode", what);
    if (kh < 1 || kw < 1 || sh < 1 || sw < 1 || plh < 0 || phh < 0 || plw < 0 || phw < 0)
        return fail(DISTDL_ERR_INVALID_ARG, "%s: bad kernel, stride or padding", what);
    if (kh > 16 || kw > 16) return fail(DISTDL_ERR_UNSUPPORTED, "%s: kernels beyond 16 x 16", what);
    if (mode == DISTDL_POOL_MAX && adjoint && !arg) return fail(DISTDL_ERR_INVALID_ARG, "%s: max pooling needs argmax", what);
    PoolDim dh, dw;
    distdl_status_t st = pool_dim(p->global_shape[2], p->pshape[2], kh, sh, plh, phh, dh, what);
    if (st != DISTDL_OK) return st;
    st = pool_dim(p->global_shape[3], p->pshape[3], kw, sw, plw, phw, dw, what);
    if (st != DISTDL_OK) return st;
    for (int32_t c = 0; c < p->pshape[2]; ++c)
        if (p->hlo[2][c] != dh.hlo[c] || p->hhi[2][c] != dh.hhi[c])
            return fail(DISTDL_ERR_SHAPE, "%s: ghost rows of worker row %d are (%d, %d), this kernel needs (%d, %d)", what, c,
                        p->hlo[2][c], p->hhi[2][c], dh.hlo[c], dh.hhi[c]);
    for (int32_t c = 0; c < p->pshape[3]; ++c)
        if (p->hlo[3][c] != dw.hlo[c] || p->hhi[3][c] != dw.hhi[c])
            return fail(DISTDL_ERR_SHAPE, "%s: ghost columns of worker column %d are (%d, %d), this kernel needs (%d, %d)", what,
                        c, p->hlo[3][c], p->hhi[3][c], dw.hlo[c], dw.hhi[c]);
    for (int k = 0; k < 2; ++k)
        if (p->hlo[k][0] != 0 || p->hhi[k][0] != 0) return fail(DISTDL_ERR_SHAPE, "%s: ghosts along batch or channels", what);

    PoolParams P;
    memset(&P, 0, sizeof(P));
    P.planes = (int32_t)(p->global_shape[0] * p->global_shape[1]);
    P.kh = kh;
    P.kw = kw;
    P.sh = sh;
    P.sw = sw;
    P.hg = (int32_t)p->global_shape[2];
    P.wg = (int32_t)p->global_shape[3];
    P.mode = mode;
    int64_t max_rows = 0, max_cols = 0;
    for (int32_t w = 0; w < p->num_workers; ++w) {
        const int32_t r = w / p->pshape[3], c = w % p->pshape[3];
        if (!in[w] || !out[w]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shard pointer %d is NULL", what, w);
        PoolShard &S = P.s[w];
        S.in = (const float *)in[w];
        S.out = (float *)out[w];
        S.arg = arg ? (int32_t *)arg[w] : nullptr;
        if (mode == DISTDL_POOL_MAX && adjoint && !S.arg) return fail(DISTDL_ERR_INVALID_ARG, "%s: argmax[%d] is NULL", what, w);
        S.ph = (int32_t)p->padded_extent(2, r);
        S.pw = (int32_t)p->padded_extent(3, c);
        S.oh = (int32_t)dh.out_size[r];
        S.ow = (int32_t)dw.out_size[c];
        S.g0h = (int32_t)(p->start[2][r] - p->hlo[2][r]);
        S.g0w = (int32_t)(p->start[3][c] - p->hlo[3][c]);
        S.i0 = (int32_t)(dh.out_start[r] * sh - plh - S.g0h);
        S.j0 = (int32_t)(dw.out_start[c] * sw - plw - S.g0w);
        if (S.oh > 0 && (S.i0 < 0 || S.i0 + (int64_t)(S.oh - 1) * sh + kh > S.ph))
            return fail(DISTDL_ERR_SHAPE, "%s: worker row %d does not hold the inputs of its outputs", what, r);
        if (S.ow > 0 && (S.j0 < 0 || S.j0 + (int64_t)(S.ow - 1) * sw + kw > S.pw))
            return fail(DISTDL_ERR_SHAPE, "%s: worker column %d does not hold the inputs of its outputs", what, c);
        max_rows = std::max<int64_t>(max_rows, adjoint ? S.ph : S.oh);
        max_cols = std::max<int64_t>(max_cols, adjoint ? S.pw : S.ow);
    }
    cudaStream_t s = (cudaStream_t)stream;
    // the compile-time variants handle four outputs / cells per thread along a row
    const int fixed = (kh == 2 && kw == 2 && sh == 2 && sw == 2) ? 1 : (kh == 3 && kw == 3 && sh == 2 && sw == 2) ? 2 : 0;
    const int per_thread = fixed ? kPoolPerThread : 1;
    if (fixed && adjoint) {
        // the compile-time adjoint walks groups of sh x sw cells; the group lattice starts up to one group before cell 0
        max_rows = max_rows / sh + 2;
        max_cols = max_cols / sw + 2;
    }
    const int tiles_x = (int)((max_cols + kPoolThreadsX * per_thread - 1) / (kPoolThreadsX * per_thread));
    const int tiles_y = (int)((max_rows + kPoolThreadsY - 1) / kPoolThreadsY);
    const int64_t blocks = (int64_t)tiles_x * tiles_y * P.planes;
    if (blocks >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);
    const dim3 grid((unsigned)blocks, (unsigned)p->num_workers), block(kPoolThreadsX, kPoolThreadsY);
    if (!adjoint) {
        // H in place on the padded input, then the local layer
        st = distdl_halo_fwd(p, const_cast<void *const *>(reinterpret_cast<const void *const *>(in)), stream);
        if (st != DISTDL_OK) return st;
    }
    if (blocks > 0) {
        if (fixed == 1) launch_pool_fixed<2, 2, 2, 2>(P, grid, block, tiles_x, tiles_y, adjoint, s);
        else if (fixed == 2) launch_pool_fixed<3, 3, 2, 2>(P, grid, block, tiles_x, tiles_y, adjoint, s);
        else if (!adjoint) pool_fwd_kernel<<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
        else pool_adj_kernel<<<grid, block, 0, s>>>(P, tiles_x, tiles_y);
    }
    DISTDL_CUDA_CHECK(cudaGetLastError());
    if (!adjoint) return DISTDL_OK;
    return distdl_halo_adj(p, out, stream);
}

}  // namespace distdl

extern "C" distdl_status_t distdl_pool_fwd(const distdl_partition_t *p, void *const *x, int32_t kh, int32_t kw, int32_t sh,
                                           int32_t sw, int32_t pad_h_lo, int32_t pad_h_hi, int32_t pad_w_lo,
                                           int32_t pad_w_hi, int32_t mode, void *const *y, void *const *argmax,
                                           void *stream) {
    return distdl::pool_impl(p, reinterpret_cast<const void *const *>(x), y, argmax, kh, kw, sh, sw, pad_h_lo, pad_h_hi,
                             pad_w_lo, pad_w_hi, mode, stream, false, "pool_fwd");
}

extern "C" distdl_status_t distdl_pool_adj(const distdl_partition_t *p, const void *const *dy, const void *const *argmax,
                                           int32_t kh, int32_t kw, int32_t sh, int32_t sw, int32_t pad_h_lo,
                                           int32_t pad_h_hi, int32_t pad_w_lo, int32_t pad_w_hi, int32_t mode,
                                           void *const *dx, void *stream) {
    // the positions are only read here; pool_impl shares one pointer type with the forward call
    return distdl::pool_impl(p, dy, dx, (void *const *)argmax, kh, kw, sh, sw, pad_h_lo, pad_h_hi, pad_w_lo, pad_w_hi, mode,
                             stream, true, "pool_adj");
}
