// Distributed star-stencil layer on a rank-3 tensor (Section 4, "Sparse layers": a sliding-kernel
// layer on a feature-space partition is the halo exchange H followed by the local kernel; its
// adjoint is the local adjoint followed by H*).  The kernel is a star: one 1-D kernel of radius R
// per dimension,
//   y[i] = sum_d sum_{k=-R..R} w[d][k+R] * x[i + k e_d],     x = 0 outside the tensor,
// which is the shape of the finite-difference operators of the volumetric problems the paper
// names as its target.  Both directions are fused with their exchange: a thread block reads the
// planes, rows and columns it needs straight from the bulk of whichever shard owns them, so no
// ghost cell is ever written to or read from device memory by the forward pass.  The adjoint is
// the same star with every 1-D kernel reversed, evaluated in gather form on the bulk-shaped dy,
// written into the bulk of the padded dx shards whose ghosts are cleared as H* leaves them.
//
// Blocking: a block (four warps) owns 8 rows x 128 columns of one shard and marches through a chunk
// of planes.  A thread owns 4 consecutive columns of two consecutive rows; the 2R+1 planes around the
// current one live in its registers (z neighbours), the current plane with R extra rows above /
// below and R extra columns left / right lives in shared memory (y and x neighbours; a star needs
// no corners).  The two rows of a thread share their y neighbours: 2R + 2 plane rows, two of them its
// own, serve both, which halves the shared-memory reads per output.  The values of the next plane --
// the thread's own cells R planes ahead, its vectors of the extra rows, one cell of an extra column
// -- are fetched one step early, so their latency is covered by the arithmetic of the current plane.
// Two plane buffers, one barrier per plane.
#include <algorithm>
#include <cstring>

#include "common.h"

namespace distdl {

constexpr int kStMaxWorkers = 64;
constexpr int kStMaxPerDim = 8;
constexpr int kStMaxR = 4;
constexpr int kStRpt = 2;             // consecutive rows per thread
constexpr int kStThreads = 128;
constexpr int kStRows = kStRpt * (kStThreads / 32);   // rows of a tile: 8
constexpr int kStCols = 128;          // columns of a tile = 32 lanes x 4
constexpr int kStChunk = 64;          // planes a block marches through
constexpr int kStLead = 4;            // shared-memory column of the tile's first column (keeps rows 16-byte aligned)
constexpr int kStPitch = kStLead + kStCols + 4;   // 136 floats

struct StencilParams {
    const float *in[kStMaxWorkers];
    float *out[kStMaxWorkers];
    int32_t bz[kStMaxPerDim], by[kStMaxPerDim], bx[kStMaxPerDim];   // bulk extents per worker coordinate
    int32_t pz, py, px;
    int32_t in_off, out_off;          // ghost width of the input / output layout (R or 0)
    int32_t tiles_y, tiles_x, chunks_z;
    int32_t clear_ghosts;             // adjoint: the ghosts of the output shards are set to zero
    float w[3][2 * kStMaxR + 1];      // taps; [d][k + R], already reversed for the adjoint
};

// Owner of coordinate c along one dimension, seen from worker coordinate s: the worker itself, or the
// one below / above (a ghost is never wider than the neighbour's bulk).  Returns false outside the tensor.
__device__ __forceinline__ bool st_owner(const int32_t *b, int p, int s, int c, int &so, int &co) {
    so = s;
    co = c;
    if (c < 0) {
        so = s - 1;
        if (so < 0) return false;
        co = c + b[so];
        return co >= 0;
    }
    if (c >= b[s]) {
        so = s + 1;
        if (so >= p) return false;
        co = c - b[s];
        return co < b[so];
    }
    return true;
}

template <int R, bool VEC>
__global__ void __launch_bounds__(kStThreads, 4)
stencil3d_kernel(const __grid_constant__ StencilParams P) {
    __shared__ __align__(16) float plane[2][kStRows + 2 * R][kStPitch];
    constexpr int N = 2 * R + 1;
    constexpr int kWarps = kStThreads / 32;
    constexpr int HR = (2 * R + kWarps - 1) / kWarps;     // extra rows a warp fetches per plane
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // block -> (shard, plane chunk, row tile, column tile), column tile fastest
    int rest = blockIdx.x;
    const int tx = rest % P.tiles_x;
    rest /= P.tiles_x;
    const int ty = rest % P.tiles_y;
    rest /= P.tiles_y;
    const int cz = rest % P.chunks_z;
    const int shard = rest / P.chunks_z;
    const int sx = shard % P.px, sy = (shard / P.px) % P.py, sz = shard / (P.px * P.py);
    const int bz = P.bz[sz], by = P.by[sy], bx = P.bx[sx];
    const int x0 = tx * kStCols, y0 = ty * kStRows, z0 = cz * kStChunk;
    if (x0 >= bx || y0 >= by || z0 >= bz) return;
    const int z1 = min(z0 + kStChunk, bz);
    const int th = min(kStRows, by - y0), tw = min(kStCols, bx - x0);
    const int io = P.in_off;
    const int ipx = bx + 2 * io;                       // input row pitch of every shard in this worker column

    const int rw = kStRpt * warp;                      // first of this warp's rows inside the tile
    const int x = x0 + 4 * lane;
    const bool col_ok = x < bx;
    bool row_ok[kStRpt];
#pragma unroll
    for (int r = 0; r < kStRpt; ++r) row_ok[r] = y0 + rw + r < by;

    // Everything that does not change from plane to plane is resolved once: for each kind of load a
    // base pointer (plane 0 of the owning shard, the thread's row and column; nullptr = zeros) and the
    // plane stride of that shard, in elements (a shard holds fewer than 2^31 of them).
    auto load4 = [&](const float *src) -> float4 {
        if (VEC) return __ldg(reinterpret_cast<const float4 *>(src));
        float4 v = make_float4(__ldg(src), 0.f, 0.f, 0.f);
        if (x + 1 < bx) v.y = __ldg(src + 1);
        if (x + 2 < bx) v.z = __ldg(src + 2);
        if (x + 3 < bx) v.w = __ldg(src + 3);
        return v;
    };
    const uint32_t ipy = (uint32_t)(by + 2 * io);
    const uint32_t own_stride = ipy * (uint32_t)ipx;                   // the same in the shards below and above
    const uint32_t own_off = (uint32_t)(y0 + rw + io) * (uint32_t)ipx + (uint32_t)(x + io);   // row 0 of the thread
    const float *own_mid = col_ok ? P.in[shard] + own_off : nullptr;
    const float *own_lo = col_ok && sz > 0 ? P.in[shard - P.py * P.px] + own_off : nullptr;
    const float *own_hi = col_ok && sz + 1 < P.pz ? P.in[shard + P.py * P.px] + own_off : nullptr;
    const int bz_lo = sz > 0 ? P.bz[sz - 1] : 0, bz_hi = sz + 1 < P.pz ? P.bz[sz + 1] : 0;
    // this thread's cells of plane zp (any plane within R of the chunk), zeros outside the tensor
    auto load_own = [&](int zp, float4 (&v)[kStRpt]) {
        const float *base = own_mid;
        if (zp < 0) {
            base = own_lo;
            zp += bz_lo;
            if (zp < 0) base = nullptr;
        } else if (zp >= bz) {
            base = own_hi;
            zp -= bz;
            if (zp >= bz_hi) base = nullptr;
        }
#pragma unroll
        for (int r = 0; r < kStRpt; ++r) {
            v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (base && row_ok[r]) v[r] = load4(base + (uint32_t)(zp + io) * own_stride + (uint32_t)(r * ipx));
        }
    };
    // extra rows of the current plane: row h of the 2R (R above the tile, R below) goes to warp h % kWarps
    const float *hrow_base[HR];
    uint32_t hrow_stride[HR];
    int hrow_s[HR];
#pragma unroll
    for (int i = 0; i < HR; ++i) {
        const int h = warp + kWarps * i;
        hrow_base[i] = nullptr;
        hrow_stride[i] = 0;
        hrow_s[i] = h < R ? h : R + th + (h - R);                      // its row in the shared-memory plane
        const int hy = h < R ? y0 - R + h : y0 + th + (h - R);
        int so, yo;
        if (h < 2 * R && col_ok && st_owner(P.by, P.py, sy, hy, so, yo)) {
            hrow_stride[i] = (uint32_t)(P.by[so] + 2 * io) * (uint32_t)ipx;
            hrow_base[i] = P.in[(sz * P.py + so) * P.px + sx] + (uint32_t)(yo + io) * (uint32_t)ipx + (uint32_t)(x + io);
        }
    }
    auto load_hrow = [&](int zp, float4 (&v)[HR]) {
#pragma unroll
        for (int i = 0; i < HR; ++i)
            v[i] = hrow_base[i] ? load4(hrow_base[i] + (uint32_t)(zp + io) * hrow_stride[i]) : make_float4(0.f, 0.f, 0.f, 0.f);
    };
    // threads 0 .. 8 * 2R - 1: one cell of an extra column of plane zp
    const int hc_row = threadIdx.x / (2 * R), hc_c = threadIdx.x % (2 * R);
    const bool hc_active = (int)threadIdx.x < kStRows * 2 * R && y0 + hc_row < by;
    const int hc_x = hc_c < R ? x0 - R + hc_c : x0 + tw + (hc_c - R);
    const int hc_s = kStLead + (hc_x - x0);                               // its column in the shared-memory plane
    const float *hcol_base = nullptr;
    uint32_t hcol_stride = 0;
    {
        int so, xo;
        if (hc_active && st_owner(P.bx, P.px, sx, hc_x, so, xo)) {
            const uint32_t pitch = (uint32_t)(P.bx[so] + 2 * io);
            hcol_stride = ipy * pitch;
            hcol_base = P.in[(sz * P.py + sy) * P.px + so] + (uint32_t)(y0 + hc_row + io) * pitch + (uint32_t)(xo + io);
        }
    }
    auto load_hcol = [&](int zp) -> float {
        return hcol_base ? __ldg(hcol_base + (uint32_t)(zp + io) * hcol_stride) : 0.f;
    };

    // prime: planes z0 - R .. z0 + R, extra rows / column of plane z0
    float4 q[N][kStRpt];
#pragma unroll
    for (int i = 0; i < N; ++i) load_own(z0 - R + i, q[i]);
    float4 hrow[HR];
    load_hrow(z0, hrow);
    float hcol = load_hcol(z0);

    const int oo = P.out_off;
    const int opy = by + 2 * oo, opx = bx + 2 * oo;
    float *optr = P.out[shard] + ((size_t)(z0 + oo) * opy + (size_t)(y0 + rw + oo)) * opx + (x + oo);
    const size_t oplane = (size_t)opy * opx;
    const bool clear_x = P.clear_ghosts && oo > 0;

    auto put4 = [&](float *d, const float4 &v) {      // own / extra-row cells into the shared-memory plane
        if (VEC) {
            *reinterpret_cast<float4 *>(d) = v;
        } else {
            d[0] = v.x;
            if (x + 1 < bx) d[1] = v.y;
            if (x + 2 < bx) d[2] = v.z;
            if (x + 3 < bx) d[3] = v.w;
        }
    };

    // One plane per turn; q[j] is the plane j - R away from the current one.  The queue is shifted by
    // register moves at the end of a turn: rotating it at compile time instead needs 2R+1 copies of the
    // loop body, which no longer fit the instruction cache (measured: 13 % slower).
    for (int z = z0; z < z1; ++z) {
        float(*pl)[kStPitch] = plane[(z - z0) & 1];
        // current plane into shared memory: own cells, the extra-row vectors, one extra-column cell.
        // Cells beyond the bulk are written by the extra-row / extra-column threads only.
        if (col_ok) {
#pragma unroll
            for (int r = 0; r < kStRpt; ++r)
                if (row_ok[r]) put4(&pl[R + rw + r][kStLead + 4 * lane], q[R][r]);
#pragma unroll
            for (int i = 0; i < HR; ++i)
                if (warp + kWarps * i < 2 * R) put4(&pl[hrow_s[i]][kStLead + 4 * lane], hrow[i]);
        }
        if (hc_active) pl[R + hc_row][hc_s] = hcol;
        // next plane's values, one step early
        float4 lead[kStRpt], hrow_n[HR];
        float hcol_n = 0.f;
        if (z + 1 < z1) {
            load_own(z + 1 + R, lead);
            load_hrow(z + 1, hrow_n);
            hcol_n = load_hcol(z + 1);
        } else {
#pragma unroll
            for (int r = 0; r < kStRpt; ++r) lead[r] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < HR; ++i) hrow_n[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        __syncthreads();

        if (col_ok && row_ok[0]) {
            float o[kStRpt][4];
#pragma unroll
            for (int r = 0; r < kStRpt; ++r)
#pragma unroll
                for (int e = 0; e < 4; ++e) o[r][e] = 0.f;
            // z neighbours: registers
#pragma unroll
            for (int k = 0; k < N; ++k) {
                const float wz = P.w[0][k];
#pragma unroll
                for (int r = 0; r < kStRpt; ++r) {
                    const float4 v = q[k][r];
                    o[r][0] = fmaf(wz, v.x, o[r][0]);
                    o[r][1] = fmaf(wz, v.y, o[r][1]);
                    o[r][2] = fmaf(wz, v.z, o[r][2]);
                    o[r][3] = fmaf(wz, v.w, o[r][3]);
                }
            }
            // y neighbours: the rows rw .. rw + 2R + RPT - 1 of the plane, each read once and used by every
            // row of the thread it is a neighbour of (tap k of row r is plane row rw + r + k)
#pragma unroll
            for (int j = 0; j < N + kStRpt - 1; ++j) {
                float4 v;
                // the thread's own rows come from its registers -- unless such a row lies beyond the bulk (a ragged
                // last tile): then that plane row holds an extra row fetched from the shard below
                const bool own = j >= R && j < R + kStRpt && row_ok[j >= R && j < R + kStRpt ? j - R : 0];
                if (own) v = q[R][j >= R && j < R + kStRpt ? j - R : 0];
                else if (VEC) v = *reinterpret_cast<const float4 *>(&pl[rw + j][kStLead + 4 * lane]);
                else {
                    const float *s = &pl[rw + j][kStLead + 4 * lane];
                    v = make_float4(s[0], s[1], s[2], s[3]);
                }
#pragma unroll
                for (int r = 0; r < kStRpt; ++r) {
                    const int k = j - r;
                    if (k < 0 || k >= N) continue;
                    const float wy = P.w[1][k];
                    o[r][0] = fmaf(wy, v.x, o[r][0]);
                    o[r][1] = fmaf(wy, v.y, o[r][1]);
                    o[r][2] = fmaf(wy, v.z, o[r][2]);
                    o[r][3] = fmaf(wy, v.w, o[r][3]);
                }
            }
            // x neighbours: the vectors left and right of the own one
#pragma unroll
            for (int r = 0; r < kStRpt; ++r) {
                float xs[12];
                const float4 l = *reinterpret_cast<const float4 *>(&pl[R + rw + r][4 * lane]);
                const float4 rt = *reinterpret_cast<const float4 *>(&pl[R + rw + r][4 * lane + 8]);
                xs[0] = l.x; xs[1] = l.y; xs[2] = l.z; xs[3] = l.w;
                if (VEC) {
                    const float4 c = q[R][r];
                    xs[4] = c.x; xs[5] = c.y; xs[6] = c.z; xs[7] = c.w;
                } else {
                    // a ragged last vector: its cells beyond the bulk are extra-column cells, not the thread's own
                    const float4 c = *reinterpret_cast<const float4 *>(&pl[R + rw + r][kStLead + 4 * lane]);
                    xs[4] = c.x; xs[5] = c.y; xs[6] = c.z; xs[7] = c.w;
                }
                xs[8] = rt.x; xs[9] = rt.y; xs[10] = rt.z; xs[11] = rt.w;
#pragma unroll
                for (int k = 0; k < N; ++k) {
                    const float wx = P.w[2][k];
#pragma unroll
                    for (int e = 0; e < 4; ++e) o[r][e] = fmaf(wx, xs[4 + e + k - R], o[r][e]);
                }
            }
#pragma unroll
            for (int r = 0; r < kStRpt; ++r) {
                if (!row_ok[r]) continue;
                float *op = optr + (size_t)r * opx;
                if (VEC) {
                    *reinterpret_cast<float4 *>(op) = make_float4(o[r][0], o[r][1], o[r][2], o[r][3]);
                } else {
                    op[0] = o[r][0];
                    if (x + 1 < bx) op[1] = o[r][1];
                    if (x + 2 < bx) op[2] = o[r][2];
                    if (x + 3 < bx) op[3] = o[r][3];
                }
                // adjoint: the ghost columns beside this row are cleared by the threads that write the row's
                // ends, so that they land in the same lines of memory as the row itself
                if (clear_x) {
                    if (x == 0) {
                        if (VEC && R == 4) *reinterpret_cast<float4 *>(op - 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                        else
                            for (int c = 1; c <= oo; ++c) op[-c] = 0.f;
                    }
                    if (x + 4 >= bx) {
                        if (VEC && R == 4) *reinterpret_cast<float4 *>(op + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                        else
                            for (int c = 0; c < oo; ++c) op[bx - x + c] = 0.f;
                    }
                }
            }
        }
        optr += oplane;
#pragma unroll
        for (int i = 0; i + 1 < N; ++i)
#pragma unroll
            for (int r = 0; r < kStRpt; ++r) q[i][r] = q[i + 1][r];
#pragma unroll
        for (int r = 0; r < kStRpt; ++r) q[N - 1][r] = lead[r];
#pragma unroll
        for (int i = 0; i < HR; ++i) hrow[i] = hrow_n[i];
        hcol = hcol_n;
    }

    if (P.clear_ghosts && oo > 0) {
        // this block's part of the ghost shell of the output shard: its box of bulk cells, extended
        // through the ghost layers wherever it touches a face of the shard
        const int zl = z0 == 0 ? 0 : z0 + oo, zh = z1 == bz ? bz + 2 * oo : z1 + oo;
        const int yl = y0 == 0 ? 0 : y0 + oo, yh = y0 + th == by ? by + 2 * oo : y0 + th + oo;
        const int xl = x0 == 0 ? 0 : x0 + oo, xh = x0 + tw == bx ? bx + 2 * oo : x0 + tw + oo;
        float *ob = P.out[shard];
        const int ny = yh - yl, nx = xh - xl;
        // whole planes of the ghost layers below / above
        for (int pz = zl; pz < zh; ++pz) {
            if (pz >= oo && pz < bz + oo) continue;
            for (int idx = threadIdx.x; idx < ny * nx; idx += kStThreads)
                ob[((size_t)pz * opy + (yl + idx / nx)) * opx + (xl + idx % nx)] = 0.f;
        }
        // planes of the bulk: ghost rows over the whole width (the ghost columns beside bulk rows were
        // cleared together with those rows)
        const int gy_lo = y0 == 0 ? oo : 0, gy = gy_lo + (y0 + th == by ? oo : 0);
        const int per_plane = gy * nx;
        if (per_plane > 0) {
            const int total = (z1 - z0) * per_plane;
            for (int idx = threadIdx.x; idx < total; idx += kStThreads) {
                const int pz = z0 + oo + idx / per_plane;
                const int e = idx % per_plane, r = e / nx;
                const int py = r < gy_lo ? r : by + oo + (r - gy_lo);
                ob[((size_t)pz * opy + py) * opx + (xl + e % nx)] = 0.f;
            }
        }
    }
}

template <int R>
static distdl_status_t launch_stencil(const StencilParams &P, unsigned grid, bool vec, cudaStream_t s) {
    if (vec) stencil3d_kernel<R, true><<<grid, kStThreads, 0, s>>>(P);
    else stencil3d_kernel<R, false><<<grid, kStThreads, 0, s>>>(P);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

static distdl_status_t stencil_impl(const distdl_partition *p, const void *const *in, const float *w, int32_t radius,
                                    void *const *out, void *stream, bool adj, const char *what) {
    clear_error();
    if (!p || !in || !w || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (p->rank != 3 || p->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-3 F32 partition", what);
    if (p->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
    if (radius < 1 || radius > kStMaxR) return fail(DISTDL_ERR_UNSUPPORTED, "%s: radius %d (supported: 1..%d)", what, radius, kStMaxR);
    if (p->num_workers > kStMaxWorkers) return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d workers", what, kStMaxWorkers);
    for (int k = 0; k < 3; ++k) {
        if (p->pshape[k] > kStMaxPerDim)
            return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d workers along a dimension", what, kStMaxPerDim);
        for (int32_t c = 0; c < p->pshape[k]; ++c)
            if (p->hlo[k][c] != radius || p->hhi[k][c] != radius)
                return fail(DISTDL_ERR_SHAPE, "%s: halo widths must equal the radius %d on every side", what, radius);
    }
    StencilParams P;
    memset(&P, 0, sizeof(P));
    int64_t mz = 0, my = 0, mx = 0;
    for (int32_t c = 0; c < p->pshape[0]; ++c) mz = std::max<int64_t>(mz, P.bz[c] = (int32_t)p->size[0][c]);
    for (int32_t c = 0; c < p->pshape[1]; ++c) my = std::max<int64_t>(my, P.by[c] = (int32_t)p->size[1][c]);
    for (int32_t c = 0; c < p->pshape[2]; ++c) mx = std::max<int64_t>(mx, P.bx[c] = (int32_t)p->size[2][c]);
    P.pz = p->pshape[0];
    P.py = p->pshape[1];
    P.px = p->pshape[2];
    P.in_off = adj ? 0 : radius;
    P.out_off = adj ? radius : 0;
    P.clear_ghosts = adj ? 1 : 0;
    P.tiles_x = (int32_t)((mx + kStCols - 1) / kStCols);
    P.tiles_y = (int32_t)((my + kStRows - 1) / kStRows);
    P.chunks_z = (int32_t)((mz + kStChunk - 1) / kStChunk);
    for (int d = 0; d < 3; ++d)
        for (int k = 0; k <= 2 * radius; ++k) P.w[d][k] = adj ? w[d * (2 * radius + 1) + (2 * radius - k)] : w[d * (2 * radius + 1) + k];
    // 16-byte accesses: every row of every layout starts on a 16-byte boundary and holds whole vectors
    bool vec = (P.in_off % 4) == 0 && (P.out_off % 4) == 0;
    for (int32_t c = 0; c < p->pshape[2]; ++c) vec = vec && (P.bx[c] % 4) == 0;
    for (int32_t wk = 0; wk < p->num_workers; ++wk) {
        if (!in[wk] || !out[wk]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shard pointer %d is NULL", what, wk);
        if (!aligned16(in[wk]) || !aligned16(out[wk])) return fail(DISTDL_ERR_ALIGNMENT, "%s: shard %d is not 16-byte aligned", what, wk);
        if (p->shard_elems(wk) >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: shard %d too large", what, wk);
        P.in[wk] = (const float *)in[wk];
        P.out[wk] = (float *)out[wk];
    }
    const int64_t blocks = (int64_t)p->num_workers * P.chunks_z * P.tiles_y * P.tiles_x;
    if (blocks >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);
    cudaStream_t s = (cudaStream_t)stream;
    switch (radius) {
        case 1: return launch_stencil<1>(P, (unsigned)blocks, vec, s);
        case 2: return launch_stencil<2>(P, (unsigned)blocks, vec, s);
        case 3: return launch_stencil<3>(P, (unsigned)blocks, vec, s);
        default: return launch_stencil<4>(P, (unsigned)blocks, vec, s);
    }
}

}  // namespace distdl

extern "C" distdl_status_t distdl_stencil3d_fwd(const distdl_partition_t *p, const void *const *x, const float *w,
                                                int32_t radius, void *const *y, void *stream) {
    return distdl::stencil_impl(p, x, w, radius, y, stream, false, "stencil3d_fwd");
}
extern "C" distdl_status_t distdl_stencil3d_adj(const distdl_partition_t *p, const void *const *dy, const float *w,
                                                int32_t radius, void *const *dx, void *stream) {
    return distdl::stencil_impl(p, dy, w, radius, dx, stream, true, "stencil3d_adj");
}
