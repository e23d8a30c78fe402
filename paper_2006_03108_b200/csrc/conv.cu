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
#include <vector>

#include "common.h"
#include "tma.h"

namespace distdl {

constexpr int kConvMaxWorkers = 64;
constexpr int kConvThreads = 128;
constexpr int kTileH = 32;    // output rows per block (8 thread rows x 4)
constexpr int kTileW = 128;   // output columns per block
constexpr int kRowsPerThread = 4;   // each thread: 4 rows x 8 columns of outputs
constexpr int kColsPerThread = 8;

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
    // n / d for the four divisors of the tile decoding (tiles_x, pw_workers, tiles_y, ph_workers):
    // umulhi(n, magic) >> shift for any n < 2^31; magic = 0 stands for d = 1
    uint32_t div_magic[4], div_shift[4];
};

// magic = ceil(2^(31+s) / d) with s = ceil(log2 d) is below 2^32 and divides every n < 2^31 exactly.
inline void conv_set_divisor(ConvParams &P, int which, uint32_t d) {
    if (d < 2) {
        P.div_magic[which] = 0;
        P.div_shift[which] = 0;
        return;
    }
    uint32_t sh = 0;
    while ((1u << sh) < d) ++sh;
    const uint64_t num = (uint64_t)1 << (31 + sh);
    P.div_magic[which] = (uint32_t)((num + d - 1) / d);
    P.div_shift[which] = sh - 1;
}
__device__ __forceinline__ uint32_t conv_div(const ConvParams &P, int which, uint32_t n) {
    const uint32_t m = P.div_magic[which];
    return m ? __umulhi(n, m) >> P.div_shift[which] : n;
}

// Row pitch (floats) of the shared-memory tile: wide enough for the staged columns (outputs plus
// PADL columns on the left and PH on the right, rounded up to whole float4s) and for the float4
// window of the last thread across (8 outputs, K - 1 more inputs, WOFF floats of lead-in).
__host__ __device__ constexpr int conv_padl(int K, bool adj) {
    // forward: the halo width; adjoint: the next multiple of four of twice the halo width, so that a
    // thread whose eight outputs start two columns to the left (see compute_tile) still reads an
    // aligned window
    return adj ? ((2 * (K / 2) + 3) / 4) * 4 : K / 2;
}
__host__ __device__ constexpr int conv_woff(int K, bool adj) { return adj ? conv_padl(K, adj) - 2 * (K / 2) : 0; }
__host__ __device__ constexpr int conv_pitch(int K, bool adj) {
    const int ph = K / 2;
    const int padl = conv_padl(K, adj);
    const int nf = ((conv_woff(K, adj) + kColsPerThread + K - 1 + 3) / 4) * 4;
    const int staged = ((kTileW + padl + ph + 3) / 4) * 4;
    const int window = kTileW - kColsPerThread + nf;
    const int p = staged > window ? staged : window;
    // an odd number of float4s per row: 16-byte loads whose lanes walk down a column (the edge pass
    // of the adjoint) then fall into eight different bank groups per quarter warp
    return (p / 4) % 2 ? p : p + 4;
}

__device__ __forceinline__ void cp_async16(float *smem, const float *gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Packed fp32 pair arithmetic (two FMAs per instruction on sm_100).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void cp_async4(float *smem, const float *gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8(float *smem, const float *gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

struct ConvTile {
    int shard, plane, r, c, bh, bw, i0, j0;
    bool valid;
};

__device__ __forceinline__ ConvTile decode_tile(const ConvParams &P, int tile, int tiles_y, int planes) {
    // tile id = (((plane * Ph + r) * tiles_y + ty) * Pw + c) * tiles_x + tx : consecutive ids sweep
    // one row of tiles of the global image from left to right across the worker columns, the next
    // row of tiles follows.  Blocks that run together therefore work on neighbouring tiles, and the
    // halo cells a tile takes from the shard next door sit in lines that the block working on that
    // shard's edge tile has just brought into L2.
    ConvTile t;
    uint32_t rest = (uint32_t)tile, q;
    q = conv_div(P, 0, rest);
    const int tx = (int)(rest - q * (uint32_t)P.tiles_x);
    rest = q;
    q = conv_div(P, 1, rest);
    t.c = (int)(rest - q * (uint32_t)P.pw_workers);
    rest = q;
    q = conv_div(P, 2, rest);
    const int ty = (int)(rest - q * (uint32_t)tiles_y);
    rest = q;
    q = conv_div(P, 3, rest);
    t.r = (int)(rest - q * (uint32_t)P.ph_workers);
    t.plane = (int)q;
    (void)planes;
    t.shard = t.r * P.pw_workers + t.c;
    t.bh = P.bh[t.r];
    t.bw = P.bw[t.c];
    t.i0 = ty * kTileH;
    t.j0 = tx * kTileW;
    t.valid = t.i0 < t.bh && t.j0 < t.bw;
    return t;
}

// Tile that a persistent block takes in turn `it` when its strided walk has reached id `walk`.  With an even grid a
// block would see only even or only odd ids, i.e. only left or only right tiles of a two-tile-wide shard, and the
// adjoint's extra pass over the last padded columns would always fall to the same blocks (and, with blocks dealt out
// to the SMs in order, to the same SMs).  In odd turns the two blocks of a pair of neighbouring ids swap their tiles.
__device__ __forceinline__ int conv_walk_tile(int walk, int it, int total) {
    if ((gridDim.x & 1u) == 0 && (it & 1) && (walk ^ 1) < total) return walk ^ 1;
    return walk;
}

// K: kernel extent (odd).  ADJ: false = forward (padded x -> bulk-shaped y), true = adjoint
// (bulk-shaped dy -> padded dx, rotated kernel, ghosts of dx cleared).
//
// Persistent blocks walk over the output tiles; the input tile of the next step is fetched with
// cp.async into the second shared-memory buffer while the current one is being consumed.
template <int K, bool ADJ>
struct ConvCfg {
    static constexpr int PH = K / 2;                                   // halo rows = halo columns
    static constexpr int PADL = conv_padl(K, ADJ);                     // tile column of bulk column j0
    static constexpr int WOFF = conv_woff(K, ADJ);                     // first column a thread needs in its slot
    static constexpr int NF = ((WOFF + kColsPerThread + K - 1 + 3) / 4) * 4;   // floats a thread loads per input row
    static constexpr int PITCH = conv_pitch(K, ADJ);
    static constexpr int ROWS = kTileH + K - 1;
    static constexpr int IOFF = ADJ ? 0 : PH;                          // offset of the bulk in the input layout
    static constexpr int OOFF = ADJ ? PH : 0;                          // offset of the bulk in the output layout
    static constexpr int TILE_FLOATS = ROWS * PITCH;
};

// Issues the asynchronous copies (and the direct zero stores) that fill `tile` for output tile t.
// wofs: first entry of P.in of the group of Ph x Pw shards the tile belongs to (the channel-partitioned
// layer keeps one such group per block of input channels).
template <int K, bool ADJ>
__device__ __forceinline__ void stage_tile(const ConvParams &P, const ConvTile &t, float *tile, int wofs = 0) {
    using C = ConvCfg<K, ADJ>;
    if (!t.valid) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int need_cols = min(kTileW, t.bw - t.j0) + C::PADL + C::PH;
    const int nvec_row = (need_cols + 3) / 4;
    const int need_rows = min(kTileH, t.bh - t.i0) + 2 * C::PH;
    // vectors [v_lo, v_hi) of a row lie inside this worker column's bulk; whether they can be copied 16 or 8 bytes
    // at a time depends on where the row starts in memory (a pitch of 4 k + 2 floats alternates between the two)
    const int first_col = t.j0 - C::PADL;                               // bulk column of tile column 0
    const int v_lo_in = first_col < 0 ? (-first_col + 3) / 4 : 0;
    const int v_hi_in = max(v_lo_in, min(nvec_row, (t.bw - first_col) / 4));
    for (int ry = warp; ry < need_rows; ry += kConvThreads / 32) {
        // which worker row owns bulk row i (warp-uniform), or none: outside the tensor
        int i = t.i0 - C::PH + ry, rr = t.r;
        bool row_ok = true;
        if (i < 0) {
            rr = t.r - 1;
            row_ok = rr >= 0;
            if (row_ok) i += P.bh[rr];
        } else if (i >= t.bh) {
            rr = t.r + 1;
            row_ok = rr < P.ph_workers;
            i -= t.bh;
            if (row_ok) row_ok = i < P.bh[rr];
        }
        float *srow = tile + ry * C::PITCH;
        if (!row_ok) {
            for (int v = lane; v < nvec_row; v += 32)
                *reinterpret_cast<float4 *>(srow + 4 * v) = make_float4(0.f, 0.f, 0.f, 0.f);
            continue;
        }
        const int rbh = P.bh[rr];
        const int pitch_c = t.bw + 2 * C::IOFF;
        const float *grow = P.in[wofs + rr * P.pw_workers + t.c] + (size_t)t.plane * (rbh + 2 * C::IOFF) * pitch_c +
                            (size_t)(i + C::IOFF) * pitch_c + C::IOFF + first_col;
        const uint32_t mis = (uint32_t)reinterpret_cast<uintptr_t>(grow) & 15u;
        int v_lo = v_lo_in, v_hi = v_hi_in;
        if (mis == 0) {
            for (int v = v_lo + lane; v < v_hi; v += 32) cp_async16(srow + 4 * v, grow + 4 * v);
        } else if (mis == 8) {
            for (int u = 2 * v_lo + lane; u < 2 * v_hi; u += 32) cp_async8(srow + 2 * u, grow + 2 * u);
        } else {
            v_lo = v_hi = 0;            // element by element below
        }
        // edge columns: left of v_lo and right of v_hi, element by element (neighbour columns or zero)
        const int n_left = 4 * v_lo, n_right = 4 * (nvec_row - v_hi);
        for (int e = lane; e < n_left + n_right; e += 32) {
            const int s = e < n_left ? e : 4 * v_hi + (e - n_left);
            int j = first_col + s, cc = t.c;
            bool ok = true;
            if (j < 0) {
                cc = t.c - 1;
                ok = cc >= 0;
                if (ok) {
                    j += P.bw[cc];
                    ok = j >= 0;
                }
            } else if (j >= t.bw) {
                cc = t.c + 1;
                ok = cc < P.pw_workers;
                j -= t.bw;
                if (ok) ok = j < P.bw[cc];
            }
            if (ok) {
                const int pitch_n = P.bw[cc] + 2 * C::IOFF;
                cp_async4(srow + s, P.in[wofs + rr * P.pw_workers + cc] + (size_t)t.plane * (rbh + 2 * C::IOFF) * pitch_n +
                                        (size_t)(i + C::IOFF) * pitch_n + C::IOFF + j);
            } else {
                srow[s] = 0.f;
            }
        }
    }
}

// Register-tiled stencil of one staged tile: each thread produces 4 rows x 8 columns with packed
// fp32 pair FMAs and no register shuffling.  A thread's input row arrives as aligned pairs
// P[i] = (x[2i], x[2i+1]).  Taps whose first input index is even feed the output pairs (o0,o1),
// (o2,o3), (o4,o5), (o6,o7) from P directly; taps whose first index is odd feed the shifted pairs
// (o1,o2), (o3,o4), (o5,o6), again from aligned P, plus o0 and o7 as two scalar FMAs.  The two
// sets of partial sums are added once at the end.
// wk2: K*K weights as (w, w) pairs (already rotated for the adjoint), then the bias.
template <int K, bool ADJ>
__device__ __forceinline__ void compute_tile(const ConvParams &P, const ConvTile &t, const float *tile, const float *wk2,
                                             int extra_warp = 0) {
    using C = ConvCfg<K, ADJ>;
    if (!t.valid) return;
    const float b0 = ADJ ? 0.f : wk2[2 * K * K];

    // Adjoint: a thread's eight outputs start PH columns to the left of its slot, i.e. they are the
    // padded columns j0 + 8 tx .. + 7 of dx -- 32-byte aligned stores, an aligned input window, and
    // the left ghost columns come out of the main pass as zeros.  The last 2 PH padded columns of the
    // shard (PH outputs and the right ghost) are done by a small extra pass of the last tile.
    const bool last_tile_x = t.j0 + kTileW >= t.bw;
    if (ADJ) {
        // top / bottom ghost rows above and below this tile's padded column range
        const int pitch_o = t.bw + 2 * C::PH;
        float *oplane = P.out[t.shard] + (uint32_t)t.plane * (uint32_t)(t.bh + 2 * C::PH) * (uint32_t)pitch_o;
        const int c0 = t.j0, c1 = last_tile_x ? pitch_o : t.j0 + kTileW;
        if (t.i0 == 0)
            for (int r = 0; r < C::PH; ++r)
                for (int q = c0 + threadIdx.x; q < c1; q += kConvThreads) oplane[r * pitch_o + q] = 0.f;
        if (t.i0 + kTileH >= t.bh)
            for (int r = 0; r < C::PH; ++r)
                for (int q = c0 + threadIdx.x; q < c1; q += kConvThreads) oplane[(t.bh + C::PH + r) * pitch_o + q] = 0.f;
        if (last_tile_x) {
            // padded columns bw .. bw + 2 PH - 1: the outputs bw - PH .. bw - 1, then the right ghost.
            // One thread per tile row (a single warp, extra_warp: the caller rotates it from tile to tile so that the
            // four schedulers of an SM share this work), so the other warps go straight to the main pass.
            const int out_rows = min(kTileH, t.bh - t.i0);
            if ((int)(threadIdx.x >> 5) == extra_warp && (int)(threadIdx.x & 31) < out_rows) {
                const int row = threadIdx.x & 31;
                const int first = t.bw - 2 * C::PH - (t.j0 - C::PADL);     // tile column of the window's first input
                float acc[C::PH];
#pragma unroll
                for (int c = 0; c < C::PH; ++c) acc[c] = 0.f;
                constexpr int LEAD = C::WOFF % 4;                          // first % 4 when bw is a multiple of four
                if (((first - LEAD) & 3) == 0) {
                    // aligned window: float4 loads (conflict-free down a column thanks to the odd pitch)
                    constexpr int NV = (LEAD + 3 * C::PH + 3) / 4;
                    const float4 *src = reinterpret_cast<const float4 *>(tile + row * C::PITCH + (first - LEAD));
#pragma unroll
                    for (int a = 0; a < K; ++a) {
                        float in[4 * NV];
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            const float4 q = src[a * (C::PITCH / 4) + v];
                            in[4 * v] = q.x;
                            in[4 * v + 1] = q.y;
                            in[4 * v + 2] = q.z;
                            in[4 * v + 3] = q.w;
                        }
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float w = wk2[2 * (a * K + b)];
#pragma unroll
                            for (int c = 0; c < C::PH; ++c) acc[c] = fmaf(w, in[LEAD + c + b], acc[c]);
                        }
                    }
                } else {
                    const float *src = tile + row * C::PITCH + first;
#pragma unroll
                    for (int a = 0; a < K; ++a) {
                        float in[3 * C::PH];
#pragma unroll
                        for (int j = 0; j < 3 * C::PH; ++j) in[j] = src[a * C::PITCH + j];
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float w = wk2[2 * (a * K + b)];
#pragma unroll
                            for (int c = 0; c < C::PH; ++c) acc[c] = fmaf(w, in[c + b], acc[c]);
                        }
                    }
                }
                float *dst = oplane + ((t.i0 + row + C::PH) * pitch_o + t.bw);
                // every lane writes to another row, so each store instruction costs 32 separate
                // memory requests: use as few and as wide stores as the alignment allows
                float e[2 * C::PH];
#pragma unroll
                for (int c = 0; c < C::PH; ++c) {
                    e[c] = acc[c];
                    e[C::PH + c] = 0.f;
                }
                const uintptr_t da = reinterpret_cast<uintptr_t>(dst);
                if (C::PH % 2 == 0 && (da & 15u) == 0) {
#pragma unroll
                    for (int c = 0; c < 2 * C::PH; c += 4)
                        *reinterpret_cast<float4 *>(dst + c) = make_float4(e[c], e[c + 1], e[c + 2], e[c + 3]);
                } else if ((da & 7u) == 0) {
#pragma unroll
                    for (int c = 0; c < 2 * C::PH; c += 2) *reinterpret_cast<float2 *>(dst + c) = make_float2(e[c], e[c + 1]);
                } else {
#pragma unroll
                    for (int c = 0; c < 2 * C::PH; ++c) dst[c] = e[c];
                }
            }
        }
    }

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    constexpr int NP = C::NF / 2;                      // aligned input pairs per row
    uint64_t acc_e[kRowsPerThread][4];                 // (o0,o1) (o2,o3) (o4,o5) (o6,o7)
    uint64_t acc_o[kRowsPerThread][3];                 // (o1,o2) (o3,o4) (o5,o6)
    float acc_s[kRowsPerThread][2];                    // o0, o7 from the odd-aligned taps
#pragma unroll
    for (int r = 0; r < kRowsPerThread; ++r) {
#pragma unroll
        for (int p2 = 0; p2 < 4; ++p2) acc_e[r][p2] = pack2(b0, b0);
#pragma unroll
        for (int p2 = 0; p2 < 3; ++p2) acc_o[r][p2] = 0ull;
        acc_s[r][0] = acc_s[r][1] = 0.f;
    }
    const float *tbase = tile + (ty * kRowsPerThread) * C::PITCH + kColsPerThread * tx;
    const uint64_t *wpairs = reinterpret_cast<const uint64_t *>(wk2);
#pragma unroll
    for (int a = 0; a < K; ++a) {
        uint64_t wp[K];
#pragma unroll
        for (int b = 0; b < K; ++b) wp[b] = wpairs[a * K + b];
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r) {
            uint64_t Pr[NP];
            const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(tbase + (r + a) * C::PITCH);
#pragma unroll
            for (int v = 0; v < NP / 2; ++v) {
                const ulonglong2 q = src[v];
                Pr[2 * v] = q.x;
                Pr[2 * v + 1] = q.y;
            }
#pragma unroll
            for (int b = 0; b < K; ++b) {
                constexpr int dummy = 0;
                (void)dummy;
                const int j0 = C::WOFF + b;            // array index of the first input of output 0
                if ((j0 & 1) == 0) {
#pragma unroll
                    for (int p2 = 0; p2 < 4; ++p2) acc_e[r][p2] = fma2(wp[b], Pr[j0 / 2 + p2], acc_e[r][p2]);
                } else {
#pragma unroll
                    for (int p2 = 0; p2 < 3; ++p2) acc_o[r][p2] = fma2(wp[b], Pr[(j0 + 1) / 2 + p2], acc_o[r][p2]);
                    float wlo, whi, xlo, xhi;
                    unpack2(wp[b], wlo, whi);
                    unpack2(Pr[(j0 - 1) / 2], xlo, xhi);              // x[j0] is the high half
                    acc_s[r][0] = fmaf(wlo, xhi, acc_s[r][0]);
                    unpack2(Pr[(j0 + 7) / 2], xlo, xhi);              // x[j0 + 7] is the low half
                    acc_s[r][1] = fmaf(wlo, xlo, acc_s[r][1]);
                }
            }
        }
    }

    const uint32_t pitch_o = (uint32_t)(t.bw + 2 * C::OOFF);
    float *oplane = P.out[t.shard] + (uint32_t)t.plane * (uint32_t)(t.bh + 2 * C::OOFF) * pitch_o;   // below 2^31 elements per shard
    // column of the first output inside an output row: forward = bulk column, adjoint = padded column
    const int jo = t.j0 + kColsPerThread * tx;
    const int jlim = t.bw;                      // forward: bulk width; adjoint: the main pass ends at padded column bw
#pragma unroll
    for (int r = 0; r < kRowsPerThread; ++r) {
        const int io = t.i0 + ty * kRowsPerThread + r;
        if (io >= t.bh || jo >= jlim) continue;
        float e[8], o[8];
#pragma unroll
        for (int p2 = 0; p2 < 4; ++p2) unpack2(acc_e[r][p2], e[2 * p2], e[2 * p2 + 1]);
        o[0] = acc_s[r][0];
        o[7] = acc_s[r][1];
#pragma unroll
        for (int p2 = 0; p2 < 3; ++p2) unpack2(acc_o[r][p2], o[2 * p2 + 1], o[2 * p2 + 2]);
        float v[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = e[q] + o[q];
        if (ADJ) {
#pragma unroll
            for (int q = 0; q < C::PH; ++q)
                if (jo + q < C::PH) v[q] = 0.f;   // left ghost columns of dx
        }
        float *dst = oplane + ((uint32_t)(io + C::OOFF) * pitch_o + (uint32_t)jo);
        if (jo + 7 < jlim && (reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
            // one 256-bit store: a half warp then writes 512 contiguous bytes of a row in one request
            asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "f"(v[0]), "f"(v[1]), "f"(v[2]),
                         "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
        } else if (jo + 7 < jlim && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
            *reinterpret_cast<float4 *>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4 *>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
        } else if (jo + 7 < jlim && (reinterpret_cast<uintptr_t>(dst) & 7u) == 0) {
#pragma unroll
            for (int q = 0; q < 8; q += 2) *reinterpret_cast<float2 *>(dst + q) = make_float2(v[q], v[q + 1]);
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (jo + q < jlim) dst[q] = v[q];
        }
    }
}

// Fills the (w, w) pair table and the bias of one channel from raw weights (global or shared).
template <int K, bool ADJ>
__device__ __forceinline__ void fill_weight_pairs(float *wk2, const float *wraw, float bias) {
    if (threadIdx.x < K * K) {
        const float w = wraw[ADJ ? K * K - 1 - (int)threadIdx.x : (int)threadIdx.x];   // adjoint: rotated kernel
        reinterpret_cast<float2 *>(wk2)[threadIdx.x] = make_float2(w, w);
    } else if (threadIdx.x == K * K) {
        wk2[2 * K * K] = bias;
    }
}

template <int K, bool ADJ>
__global__ void __launch_bounds__(kConvThreads, 4)
conv_depthwise_kernel(const __grid_constant__ ConvParams P, int total_tiles, int tiles_y, int planes) {
    using C = ConvCfg<K, ADJ>;
    extern __shared__ __align__(16) float smem[];   // two tile buffers
    __shared__ __align__(16) float wk[2 * K * K + 2];
    int buf = 0;
    int tile = blockIdx.x;
    if (tile >= total_tiles) return;
    int turn = 0;
    ConvTile cur = decode_tile(P, conv_walk_tile(tile, turn, total_tiles), tiles_y, planes);
    stage_tile<K, ADJ>(P, cur, smem);
    cp_async_commit();
    while (true) {
        const int next = tile + gridDim.x;
        const bool has_next = next < total_tiles;
        ConvTile nxt = cur;
        ++turn;
        if (has_next) {
            nxt = decode_tile(P, conv_walk_tile(next, turn, total_tiles), tiles_y, planes);
            stage_tile<K, ADJ>(P, nxt, smem + (buf ^ 1) * C::TILE_FLOATS);
        }
        cp_async_commit();
        cp_async_wait_group<1>();          // everything but the newest group: the current tile is here
        if (cur.valid) {
            const int ch = cur.plane % P.channels;
            fill_weight_pairs<K, ADJ>(wk, P.w + (size_t)ch * K * K, P.bias ? __ldg(P.bias + ch) : 0.f);
        }
        __syncthreads();
        compute_tile<K, ADJ>(P, cur, smem + buf * C::TILE_FLOATS, wk);
        __syncthreads();                   // the buffer may be refilled from now on
        if (!has_next) break;
        cur = nxt;
        tile = next;
        buf ^= 1;
    }
    cp_async_wait_group<0>();
}

// ---------------------------------------------------------------------------------------------
// TMA variant (up to 16 workers, 16-byte aligned row pitch): the tile body is fetched by one
// bulk tensor copy per tile from the shard's own storage; only the halo strips that come from
// neighbouring shards (or are zero outside the tensor) are fetched cell by cell into a small side
// buffer and patched into the tile before it is consumed.  Staging then costs a handful of
// instructions per thread, which leaves the issue slots to the packed FMAs.
// ---------------------------------------------------------------------------------------------
constexpr int kConvTmaMaxWorkers = 16;
constexpr uint64_t kConvWaitLimitNs = 2000000000ull;

__device__ int g_conv_status = 0;

struct ConvTmaParams {
    ConvParams base;
    CUtensorMap in_map[kConvTmaMaxWorkers];
    int32_t total_tiles, tiles_y, planes;
};

template <int K, bool ADJ>
struct ConvTmaCfg {
    using C = ConvCfg<K, ADJ>;
    static constexpr int TILE_STRIDE = ((C::TILE_FLOATS * 4 + 127) / 128) * 32;     // floats, 128-byte multiple
    static constexpr int SIDE = 2 * C::PH * C::PITCH + 2 * C::PH * C::ROWS;         // patch cells, upper bound
    static constexpr int SIDE_STRIDE = ((SIDE + 31) / 32) * 32;
    static constexpr int BOX_BYTES = C::PITCH * C::ROWS * 4;
    static constexpr int WK_STRIDE = 64 + 128;                                      // raw weights + bias, (w,w) pairs + bias
    static constexpr int SMEM_BYTES = 2 * TILE_STRIDE * 4 + 2 * SIDE_STRIDE * 4 + 2 * WK_STRIDE * 4 + 64 + 128;
};

// The halo strips of a tile -- top / bottom rows and left / right columns that lie outside the
// shard's own bulk -- are enumerated by every thread the same way at staging and at patching
// time: f(q, ry, s) gets the cell's slot q in the side buffer and its tile coordinates.
template <int K, bool ADJ, typename F>
__device__ __forceinline__ void for_each_patch_cell(const ConvTile &t, F f) {
    using C = ConvCfg<K, ADJ>;
    const int out_rows = min(kTileH, t.bh - t.i0), out_cols = min(kTileW, t.bw - t.j0);
    const int H = out_rows + 2 * C::PH;
    const int colL = C::PADL - C::PH, colR = C::PADL + out_cols, rowB = C::PH + out_rows;
    // the row strips span every column the tile's threads read: in the adjoint the threads' outputs
    // start PH columns further left, so their windows start at tile column WOFF = PADL - 2 PH
    const int colS = C::WOFF, W = colR + C::PH - colS;
    int q0 = 0;
    if (t.i0 == 0) {
#pragma unroll
        for (int r = 0; r < C::PH; ++r)
            for (int s = threadIdx.x; s < W; s += kConvThreads) f(q0 + r * W + s, r, colS + s);
        q0 += C::PH * W;
    }
    // rows / columns of the tile that lie beyond the shard's bulk: all PH of them in the last tile, and
    // some already in the tile before it when the last one holds fewer than PH rows / columns
    const int nbot = min(C::PH, max(0, t.i0 + out_rows + C::PH - t.bh));
    const int nright = min(C::PH, max(0, t.j0 + out_cols + C::PH - t.bw));
    if (nbot > 0) {
#pragma unroll
        for (int r = 0; r < C::PH; ++r)
            if (r < nbot)
                for (int s = threadIdx.x; s < W; s += kConvThreads) f(q0 + r * W + s, rowB + C::PH - nbot + r, colS + s);
        q0 += C::PH * W;
    }
    if (t.j0 == 0) {
        for (int ry = threadIdx.x; ry < H; ry += kConvThreads)
#pragma unroll
            for (int c = 0; c < C::PH; ++c) f(q0 + ry * C::PH + c, ry, colL + c);
        q0 += C::PH * H;
    }
    if (nright > 0) {
        for (int ry = threadIdx.x; ry < H; ry += kConvThreads)
#pragma unroll
            for (int c = 0; c < C::PH; ++c)
                if (c < nright) f(q0 + ry * C::PH + c, ry, colR + C::PH - nright + c);
    }
}

// Fetches the halo strips of tile t (cells that belong to neighbouring shards, or zeros outside the
// tensor) into the side buffer, cell by cell.
template <int K, bool ADJ>
__device__ __forceinline__ void stage_halo_strips(const ConvParams &P, const ConvTile &t, float *side, int wofs = 0) {
    using C = ConvCfg<K, ADJ>;
    for_each_patch_cell<K, ADJ>(t, [&](int q, int ry, int s) {
        int i = t.i0 - C::PH + ry, rr = t.r;
        bool ok = true;
        if (i < 0) {
            rr = t.r - 1;
            ok = rr >= 0;
            if (ok) i += P.bh[rr];
        } else if (i >= t.bh) {
            rr = t.r + 1;
            ok = rr < P.ph_workers;
            i -= t.bh;
            if (ok) ok = i < P.bh[rr];
        }
        int j = t.j0 - C::PADL + s, cc = t.c;
        if (j < 0) {
            cc = t.c - 1;
            ok = ok && cc >= 0;
            if (ok) {
                j += P.bw[cc];
                ok = j >= 0;
            }
        } else if (j >= t.bw) {
            cc = t.c + 1;
            ok = ok && cc < P.pw_workers;
            j -= t.bw;
            if (ok) ok = j < P.bw[cc];
        }
        if (ok) {
            // a shard holds fewer than 2^31 elements: 32-bit offsets
            const uint32_t pitch_n = (uint32_t)(P.bw[cc] + 2 * C::IOFF);
            const uint32_t off = ((uint32_t)t.plane * (uint32_t)(P.bh[rr] + 2 * C::IOFF) + (uint32_t)(i + C::IOFF)) * pitch_n +
                                 (uint32_t)(C::IOFF + j);
            cp_async4(side + q, P.in[wofs + rr * P.pw_workers + cc] + off);
        } else {
            side[q] = 0.f;
        }
    });
}

template <int K, bool ADJ>
__device__ __forceinline__ void stage_tile_tma(const ConvTmaParams &Q, const ConvTile &t, float *tile, float *side,
                                               float *wk, uint32_t bar) {
    using C = ConvCfg<K, ADJ>;
    using T = ConvTmaCfg<K, ADJ>;
    const ConvParams &P = Q.base;
    if (!t.valid) return;
    if (threadIdx.x == 0) {
        fence_proxy_async();     // earlier generic-proxy accesses to this buffer are ordered before the bulk copy
        mbar_expect_tx(bar, T::BOX_BYTES);
        // forward: padded coordinates (bulk column j sits at j + PH); adjoint: bulk coordinates
        const int x = ADJ ? t.j0 - C::PADL : t.j0;
        const int y = ADJ ? t.i0 - C::PH : t.i0;
        tma_load_3d(smem_u32(tile), &Q.in_map[t.shard], x, y, t.plane, bar);
    }
    // this channel's weights and bias
    if (threadIdx.x <= K * K) {
        const int ch = t.plane % P.channels;
        if (threadIdx.x < K * K) cp_async4(wk + threadIdx.x, P.w + (size_t)ch * K * K + threadIdx.x);
        else if (P.bias) cp_async4(wk + K * K, P.bias + ch);
        else wk[K * K] = 0.f;
    }
    stage_halo_strips<K, ADJ>(P, t, side);
}

template <int K, bool ADJ>
__global__ void __launch_bounds__(kConvThreads, 4)
conv_tma_kernel(const __grid_constant__ ConvTmaParams Q) {
    using C = ConvCfg<K, ADJ>;
    using T = ConvTmaCfg<K, ADJ>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    float *tiles = reinterpret_cast<float *>(smem_raw + (((raw + 127u) & ~127u) - raw));
    float *sides = tiles + 2 * T::TILE_STRIDE;
    float *wks = sides + 2 * T::SIDE_STRIDE;
    const uint32_t bars = smem_u32(wks + 2 * T::WK_STRIDE);
    if (threadIdx.x == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 8, 1);
        fence_barrier_init();
    }
    __syncthreads();

    int tile = blockIdx.x;
    if (tile >= Q.total_tiles) return;
    int buf = 0;
    uint32_t phase0 = 0, phase1 = 0;          // parity of the next completion of each buffer's barrier
    int turn = 0;
    ConvTile cur = decode_tile(Q.base, conv_walk_tile(tile, turn, Q.total_tiles), Q.tiles_y, Q.planes);
    stage_tile_tma<K, ADJ>(Q, cur, tiles, sides, wks, bars);
    cp_async_commit();
    while (true) {
        const int next = tile + gridDim.x;
        const bool has_next = next < Q.total_tiles;
        ConvTile nxt = cur;
        ++turn;
        if (has_next) {
            nxt = decode_tile(Q.base, conv_walk_tile(next, turn, Q.total_tiles), Q.tiles_y, Q.planes);
            stage_tile_tma<K, ADJ>(Q, nxt, tiles + (buf ^ 1) * T::TILE_STRIDE, sides + (buf ^ 1) * T::SIDE_STRIDE,
                                   wks + (buf ^ 1) * T::WK_STRIDE, bars + 8 * (buf ^ 1));
        }
        cp_async_commit();
        cp_async_wait_group<1>();
        bool ok = true;
        if (cur.valid) {
            const uint32_t bar = bars + 8 * buf, parity = buf ? phase1 : phase0;
            if (!mbar_try_wait(bar, parity)) {
                const uint64_t t0 = global_timer();
                while (!mbar_try_wait(bar, parity)) {
                    if (global_timer() - t0 > kConvWaitLimitNs) {
                        ok = false;
                        break;
                    }
                }
            }
            if (buf) phase1 ^= 1; else phase0 ^= 1;
        }
        if (__syncthreads_or(!ok)) {
            // the bulk copy never arrived: record it and leave (every thread takes this branch)
            if (threadIdx.x == 0) {
                atomicExch(&g_conv_status, (int)DISTDL_ERR_TIMEOUT);
                const uint64_t t0 = global_timer();
                while (global_timer() - t0 < 1000000ull) {}
            }
            break;
        }
        float *tl = tiles + buf * T::TILE_STRIDE;
        float *wraw = wks + buf * T::WK_STRIDE;
        if (cur.valid) {
            const float *sd = sides + buf * T::SIDE_STRIDE;
            for_each_patch_cell<K, ADJ>(cur, [&](int q, int ry, int s) { tl[ry * C::PITCH + s] = sd[q]; });
            fill_weight_pairs<K, ADJ>(wraw + 64, wraw, wraw[K * K]);
        }
        __syncthreads();
        compute_tile<K, ADJ>(Q.base, cur, tl, wraw + 64, (turn >> 1) & 3);
        __syncthreads();
        if (!has_next) break;
        cur = nxt;
        tile = next;
        buf ^= 1;
    }
    cp_async_wait_group<0>();
}

int conv_take_status() {
    int st = 0;
    if (cudaMemcpyFromSymbol(&st, g_conv_status, sizeof(int)) != cudaSuccess) return -1;
    if (st != 0) {
        const int zero = 0;
        cudaMemcpyToSymbol(g_conv_status, &zero, sizeof(int));
    }
    return st;
}

template <int K, bool ADJ>
static constexpr int conv_smem_bytes() {
    return 2 * (kTileH + K - 1) * conv_pitch(K, ADJ) * (int)sizeof(float);
}

template <int K, bool ADJ>
static distdl_status_t launch_conv(const ConvParams &P, int total_tiles, int tiles_y, int planes, cudaStream_t s) {
    constexpr int smem = conv_smem_bytes<K, ADJ>();
    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    static int blocks_on[kMaxDevicesPerProcess] = {0};
    int &blocks = blocks_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_depthwise_kernel<K, ADJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        int dev = 0, sms = 0, per_sm = 0;
        DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
        DISTDL_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, conv_depthwise_kernel<K, ADJ>, kConvThreads, smem));
        blocks = sms * (per_sm > 0 ? per_sm : 1);
        configured = true;
    }
    const int grid = total_tiles < blocks ? total_tiles : blocks;
    conv_depthwise_kernel<K, ADJ><<<grid, kConvThreads, smem, s>>>(P, total_tiles, tiles_y, planes);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

template <int K, bool ADJ>
static distdl_status_t launch_conv_tma(const distdl_partition *p, ConvTmaParams &Q, const void *const *in, cudaStream_t s) {
    using C = ConvCfg<K, ADJ>;
    using T = ConvTmaCfg<K, ADJ>;
    EncodeTiledFn enc = tensor_map_encoder();
    const int64_t planes = Q.planes;
    for (int32_t wk = 0; wk < p->num_workers; ++wk) {
        const int r = wk / Q.base.pw_workers, c = wk % Q.base.pw_workers;
        const cuuint64_t pitch = (cuuint64_t)(Q.base.bw[c] + 2 * C::IOFF), rows = (cuuint64_t)(Q.base.bh[r] + 2 * C::IOFF);
        const cuuint64_t dims[3] = {pitch, rows, (cuuint64_t)planes};
        const cuuint64_t strides[2] = {pitch * 4, pitch * rows * 4};
        const cuuint32_t box[3] = {(cuuint32_t)C::PITCH, (cuuint32_t)C::ROWS, 1};
        const cuuint32_t estr[3] = {1, 1, 1};
        if (enc(&Q.in_map[wk], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(in[wk]), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return fail(DISTDL_ERR_CUDA, "conv: tensor map of shard %d failed", wk);
    }
    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    static int blocks_on[kMaxDevicesPerProcess] = {0};
    int &blocks = blocks_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_tma_kernel<K, ADJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM_BYTES));
        int dev = 0, sms = 0, per_sm = 0;
        DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
        DISTDL_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, conv_tma_kernel<K, ADJ>, kConvThreads, T::SMEM_BYTES));
        blocks = sms * (per_sm > 0 ? per_sm : 1);
        configured = true;
    }
    const int grid = Q.total_tiles < blocks ? Q.total_tiles : blocks;
    conv_tma_kernel<K, ADJ><<<grid, kConvThreads, T::SMEM_BYTES, s>>>(Q);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

static distdl_status_t conv_impl(const distdl_partition *p, const void *const *in, const void *w, const void *bias,
                                 int32_t kh, int32_t kw, void *const *out, void *stream, bool adj, const char *what) {
    clear_error();
    if (!p || !in || !w || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (p->rank != 4 || p->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (p->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
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
    conv_set_divisor(P, 0, (uint32_t)P.tiles_x);
    conv_set_divisor(P, 1, (uint32_t)P.pw_workers);
    conv_set_divisor(P, 2, (uint32_t)tiles_y);
    conv_set_divisor(P, 3, (uint32_t)P.ph_workers);
    const int64_t total = (int64_t)P.tiles_x * tiles_y * planes * p->num_workers;
    if (total >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);
    cudaStream_t s = (cudaStream_t)stream;
    const int tt = (int)total, pl = (int)planes;
    // TMA variant: few enough workers for the tensor maps to travel as kernel parameters, and a row
    // pitch of whole 16-byte units in every shard's input layout
    bool tma_ok = p->num_workers <= kConvTmaMaxWorkers && tensor_map_encoder() != nullptr;
    for (int32_t c = 0; c < p->pshape[3] && tma_ok; ++c) tma_ok = ((P.bw[c] + (adj ? 0 : 2 * h)) % 4) == 0;
    if (tma_ok) {
        ConvTmaParams Q;
        memset(&Q, 0, sizeof(Q));
        Q.base = P;
        Q.total_tiles = tt;
        Q.tiles_y = tiles_y;
        Q.planes = pl;
        if (!adj) {
            if (kh == 3) return launch_conv_tma<3, false>(p, Q, in, s);
            if (kh == 5) return launch_conv_tma<5, false>(p, Q, in, s);
            return launch_conv_tma<7, false>(p, Q, in, s);
        }
        if (kh == 3) return launch_conv_tma<3, true>(p, Q, in, s);
        if (kh == 5) return launch_conv_tma<5, true>(p, Q, in, s);
        return launch_conv_tma<7, true>(p, Q, in, s);
    }
    if (!adj) {
        if (kh == 3) return launch_conv<3, false>(P, tt, tiles_y, pl, s);
        if (kh == 5) return launch_conv<5, false>(P, tt, tiles_y, pl, s);
        return launch_conv<7, false>(P, tt, tiles_y, pl, s);
    }
    if (kh == 3) return launch_conv<3, true>(P, tt, tiles_y, pl, s);
    if (kh == 5) return launch_conv<5, true>(P, tt, tiles_y, pl, s);
    return launch_conv<7, true>(P, tt, tiles_y, pl, s);
}

// ---------------------------------------------------------------------------------------------
// Generalized convolution layer: channels partitioned as well (Section 4, "Sparse layers": forward /
// adjoint convolution algorithms with x on 1 x P_ci x P_0 x P_1, y on 1 x P_co x P_0 x P_1, weights on
// P_co x P_ci and the work partition 1 x P_co x P_ci x P_0 x P_1).
//   forward:  x <- H x;  x^ <- B x (to the P_co copies);  y^_{ijs} <- Conv(w_{ij}, b_i on j = 0; x^_{js});
//             y_{is} <- R over j, in order.
//   adjoint:  dy^ <- B dy (to the P_ci copies);  dx^_{ijs} <- [dConv]*(dy^_{ijs});  dx_{js} <- R over i, in
//             order;  dx <- H* dx  (gather form: a correlation of dy with the rotated kernels).
// With every shard in one memory the broadcasts are implicit and the sum-reduce is the running sum of
// the block that owns an output tile: it walks through the blocks of the reduced channel partition in
// worker order and through the channels of a block in channel order, so the order of the sum is fixed.
// H / H* are fused as in the depthwise kernels (tiles staged with their ghost rows and columns from
// the neighbouring shards' bulk).  A block owns 32 x 128 pixels of kCob output channels; a thread
// 4 x 8 pixels of them, as packed pairs of neighbouring pixels.
// ---------------------------------------------------------------------------------------------
constexpr int kCob = 2;                 // output channels per block
constexpr int kMaxChanBlocks = 8;       // P_co, P_ci
constexpr int kMaxGroups = 128;         // groups of kCob output channels

struct ConvGParams {
    ConvParams base;                        // in = shards of the input tensor, out = shards of the output tensor
    const float *w[kMaxChanBlocks * kMaxChanBlocks];   // weight blocks, worker order i * P_ci + j
    const float *bias[kMaxChanBlocks];      // forward only; per block of output channels, may be null
    int32_t cnt_out[kMaxChanBlocks], cnt_in[kMaxChanBlocks];   // channels per block of the output / input partition
    int32_t p_out, p_in, pci;               // blocks of the output / input channel partition; P_ci
    int32_t groups;                         // groups of up to kCob output channels, all blocks together
    uint8_t grp_block[kMaxGroups], grp_first[kMaxGroups], grp_count[kMaxGroups];
    int32_t tiles_y, total_tiles;
    int32_t ooff;                           // ghost width of the output layout
};

// One input channel's contribution to the block's kCob x 32 x 128 outputs: per thread 4 x 8 pixels of kCob
// channels as packed pairs.  wp: K * K * kCob (w, w) pairs of this input channel, [tap][channel].
template <int K, bool ADJ>
__device__ __forceinline__ void convg_accumulate(const float *tile, const uint64_t *wp, uint64_t (&acc)[kCob][kRowsPerThread][4]) {
    using C = ConvCfg<K, ADJ>;
    constexpr int XO = C::PADL - C::PH;                         // tile column of the first input of output column 0
    constexpr int NF2 = ((XO + kColsPerThread + K - 1 + 3) / 4) * 4;   // floats of a thread's (aligned) window
    constexpr int NP = NF2 / 2;
    static_assert(kTileW - kColsPerThread + NF2 <= C::PITCH, "window beyond the tile row");
    static_assert(kCob % 2 == 0, "weight pairs are read two channels at a time");
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const float *tbase = tile + (ty * kRowsPerThread) * C::PITCH + kColsPerThread * tx;
#pragma unroll
    for (int rho = 0; rho < kRowsPerThread + K - 1; ++rho) {
        uint64_t Pr[NP], Qr[NP - 1];
        const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(tbase + rho * C::PITCH);
#pragma unroll
        for (int v = 0; v < NP / 2; ++v) {
            const ulonglong2 q = src[v];
            Pr[2 * v] = q.x;
            Pr[2 * v + 1] = q.y;
        }
#pragma unroll
        for (int i = 0; i < NP - 1; ++i) {
            float a0, a1, b0, b1;
            unpack2(Pr[i], a0, a1);
            unpack2(Pr[i + 1], b0, b1);
            Qr[i] = pack2(a1, b0);
        }
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r) {
            const int a = rho - r;
            if (a < 0 || a >= K) continue;
#pragma unroll
            for (int b = 0; b < K; ++b) {
                // the pairs of all kCob channels of one tap sit side by side: one 16-byte read for two channels
                uint64_t w2[kCob];
#pragma unroll
                for (int o = 0; o < kCob; o += 2) {
                    const ulonglong2 q = *reinterpret_cast<const ulonglong2 *>(wp + (a * K + b) * kCob + o);
                    w2[o] = q.x;
                    w2[o + 1] = q.y;
                }
                // outputs (2 p2, 2 p2 + 1) read window floats XO + 2 p2 + b, + 1
                const int j0 = XO + b;
#pragma unroll
                for (int p2 = 0; p2 < 4; ++p2) {
                    const uint64_t X = (j0 & 1) ? Qr[p2 + (j0 - 1) / 2] : Pr[p2 + j0 / 2];
#pragma unroll
                    for (int o = 0; o < kCob; ++o) acc[o][r][p2] = fma2(w2[o], X, acc[o][r][p2]);
                }
            }
        }
    }
}

// (w, w) pairs of input channel (ib, cl) for the output channels of group (ob, o0, oc); layout [tap][channel]
template <int K, bool ADJ>
__device__ __forceinline__ void convg_stage_weights(const ConvGParams &G, int ob, int o0, int oc, int ib, int cl, uint64_t *dst) {
    if ((int)threadIdx.x < kCob * K * K) {
        const int tap = threadIdx.x / kCob, o = threadIdx.x - tap * kCob;
        float w = 0.f;
        if (o < oc) {
            const float *blk = ADJ ? G.w[ib * G.pci + ob] : G.w[ob * G.pci + ib];
            const int s_out = ADJ ? K * K : G.cnt_in[ib] * K * K, s_in = ADJ ? G.cnt_out[ob] * K * K : K * K;
            w = __ldg(blk + (size_t)(o0 + o) * s_out + (size_t)cl * s_in + (ADJ ? K * K - 1 - tap : tap));   // adjoint: rotated
        }
        reinterpret_cast<float2 *>(dst)[threadIdx.x] = make_float2(w, w);
    }
}

template <int K, bool ADJ>
__device__ __forceinline__ void convg_store(const ConvGParams &G, const ConvTile &t, int n, int ob, int o0, int oc,
                                            const uint64_t (&acc)[kCob][kRowsPerThread][4]) {
    const ConvParams &P = G.base;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int spatial = P.ph_workers * P.pw_workers;
    const int oo = G.ooff;
    const uint32_t pitch_o = (uint32_t)(t.bw + 2 * oo), rows_o = (uint32_t)(t.bh + 2 * oo);
    const int jo = t.j0 + kColsPerThread * tx;
#pragma unroll
    for (int o = 0; o < kCob; ++o) {
        if (o >= oc) continue;
        float *oplane = P.out[ob * spatial + t.shard] + ((size_t)n * G.cnt_out[ob] + (size_t)(o0 + o)) * rows_o * pitch_o;
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r) {
            const int io = t.i0 + ty * kRowsPerThread + r;
            if (io >= t.bh || jo >= t.bw) continue;
            float v[8];
#pragma unroll
            for (int p2 = 0; p2 < 4; ++p2) unpack2(acc[o][r][p2], v[2 * p2], v[2 * p2 + 1]);
            float *dst = oplane + ((size_t)(io + oo) * pitch_o + (size_t)(jo + oo));
            if (jo + 7 < t.bw && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
                *reinterpret_cast<float4 *>(dst) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4 *>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (jo + q < t.bw) dst[q] = v[q];
            }
        }
    }
}

template <int K, bool ADJ>
__device__ __forceinline__ void convg_init(const ConvGParams &G, int ob, int o0, int oc, uint64_t (&acc)[kCob][kRowsPerThread][4]) {
#pragma unroll
    for (int o = 0; o < kCob; ++o) {
        float b = 0.f;
        if (!ADJ && G.bias[ob] && o < oc) b = __ldg(G.bias[ob] + o0 + o);
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r)
#pragma unroll
            for (int p2 = 0; p2 < 4; ++p2) acc[o][r][p2] = pack2(b, b);
    }
}

// General variant: tiles staged by per-thread asynchronous copies (any row pitch, any number of shards).
template <int K, bool ADJ>
__global__ void __launch_bounds__(kConvThreads, 3)
convg_kernel(const __grid_constant__ ConvGParams G) {
    using C = ConvCfg<K, ADJ>;
    extern __shared__ __align__(16) float smem[];               // two x tiles, then two weight tables
    float *tiles = smem;
    uint64_t *wtab = reinterpret_cast<uint64_t *>(smem + 2 * C::TILE_FLOATS);   // [2][K * K][kCob] (w, w) pairs
    const ConvParams &P = G.base;
    const int spatial = P.ph_workers * P.pw_workers;

    for (int tile = blockIdx.x; tile < G.total_tiles; tile += gridDim.x) {
        ConvTile t = decode_tile(P, tile, G.tiles_y, 0);
        if (!t.valid) continue;                                  // the same for every thread of the block
        const int n = t.plane / G.groups, g = t.plane - n * G.groups;
        const int ob = G.grp_block[g], o0 = G.grp_first[g], oc = G.grp_count[g];
        uint64_t acc[kCob][kRowsPerThread][4];
        convg_init<K, ADJ>(G, ob, o0, oc, acc);
        // the channels of the reduced partition: block after block, channel after channel
        auto stage = [&](int ib, int cl, int buf) {
            ConvTile ti = t;
            ti.plane = n * G.cnt_in[ib] + cl;
            stage_tile<K, ADJ>(P, ti, tiles + buf * C::TILE_FLOATS, ib * spatial);
            convg_stage_weights<K, ADJ>(G, ob, o0, oc, ib, cl, wtab + buf * (kCob * K * K));
        };
        int ib = 0, cl = 0, buf = 0;
        stage(0, 0, 0);
        cp_async_commit();
        while (true) {
            int nib = ib, ncl = cl + 1;
            if (ncl == G.cnt_in[ib]) {
                ncl = 0;
                ++nib;
            }
            const bool has_next = nib < G.p_in;
            if (has_next) stage(nib, ncl, buf ^ 1);
            cp_async_commit();
            cp_async_wait_group<1>();
            __syncthreads();
            convg_accumulate<K, ADJ>(tiles + buf * C::TILE_FLOATS, wtab + buf * (kCob * K * K), acc);
            __syncthreads();
            if (!has_next) break;
            ib = nib;
            cl = ncl;
            buf ^= 1;
        }
        cp_async_wait_group<0>();
        convg_store<K, ADJ>(G, t, n, ob, o0, oc, acc);
        __syncthreads();
    }
}

// TMA variant (at most kConvGTmaShards input shards, rows of whole 16-byte units): the tile body of every
// input channel arrives by one bulk tensor copy, the halo strips cell by cell into a side buffer.
constexpr int kConvGTmaShards = 32;
struct ConvGTmaParams {
    ConvGParams g;
    CUtensorMap in_map[kConvGTmaShards];
};

// Four blocks per SM where the register tile allows it without spills (5 x 5), three otherwise.
template <int K, bool ADJ>
__global__ void __launch_bounds__(kConvThreads, K == 5 ? 4 : 3)
convg_tma_kernel(const __grid_constant__ ConvGTmaParams Q) {
    using C = ConvCfg<K, ADJ>;
    using T = ConvTmaCfg<K, ADJ>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    float *tiles = reinterpret_cast<float *>(smem_raw + (((raw + 127u) & ~127u) - raw));
    float *sides = tiles + 2 * T::TILE_STRIDE;
    uint64_t *wtab = reinterpret_cast<uint64_t *>(sides + 2 * T::SIDE_STRIDE);          // [2][K * K][kCob]
    const uint32_t bars = smem_u32(wtab + 2 * kCob * K * K);
    const ConvGParams &G = Q.g;
    const ConvParams &P = G.base;
    const int spatial = P.ph_workers * P.pw_workers;
    if (threadIdx.x == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 8, 1);
        fence_barrier_init();
    }
    __syncthreads();
    uint32_t phase0 = 0, phase1 = 0;
    bool failed = false;

    for (int tile = blockIdx.x; tile < G.total_tiles && !failed; tile += gridDim.x) {
        ConvTile t = decode_tile(P, tile, G.tiles_y, 0);
        if (!t.valid) continue;
        const int n = t.plane / G.groups, g = t.plane - n * G.groups;
        const int ob = G.grp_block[g], o0 = G.grp_first[g], oc = G.grp_count[g];
        uint64_t acc[kCob][kRowsPerThread][4];
        convg_init<K, ADJ>(G, ob, o0, oc, acc);
        auto stage = [&](int ib, int cl, int buf) {
            ConvTile ti = t;
            ti.plane = n * G.cnt_in[ib] + cl;
            if (threadIdx.x == 0) {
                fence_proxy_async();
                mbar_expect_tx(bars + 8 * buf, T::BOX_BYTES);
                // forward: padded coordinates (bulk column j sits at j + PH); adjoint: bulk coordinates
                const int x = ADJ ? t.j0 - C::PADL : t.j0;
                const int y = ADJ ? t.i0 - C::PH : t.i0;
                tma_load_3d(smem_u32(tiles + buf * T::TILE_STRIDE), &Q.in_map[ib * spatial + t.shard], x, y, ti.plane, bars + 8 * buf);
            }
            stage_halo_strips<K, ADJ>(P, ti, sides + buf * T::SIDE_STRIDE, ib * spatial);
            convg_stage_weights<K, ADJ>(G, ob, o0, oc, ib, cl, wtab + buf * (kCob * K * K));
        };
        int ib = 0, cl = 0, buf = 0;
        stage(0, 0, 0);
        cp_async_commit();
        while (true) {
            int nib = ib, ncl = cl + 1;
            if (ncl == G.cnt_in[ib]) {
                ncl = 0;
                ++nib;
            }
            const bool has_next = nib < G.p_in;
            if (has_next) stage(nib, ncl, buf ^ 1);
            cp_async_commit();
            cp_async_wait_group<1>();
            bool ok = true;
            {
                const uint32_t bar = bars + 8 * buf, parity = buf ? phase1 : phase0;
                if (!mbar_try_wait(bar, parity)) {
                    const uint64_t t0 = global_timer();
                    while (!mbar_try_wait(bar, parity)) {
                        if (global_timer() - t0 > kConvWaitLimitNs) {
                            ok = false;
                            break;
                        }
                    }
                }
                if (buf) phase1 ^= 1; else phase0 ^= 1;
            }
            if (__syncthreads_or(!ok)) {
                if (threadIdx.x == 0) {
                    atomicExch(&g_conv_status, (int)DISTDL_ERR_TIMEOUT);
                    const uint64_t t0 = global_timer();
                    while (global_timer() - t0 < 1000000ull) {}
                }
                failed = true;
                break;
            }
            float *tl = tiles + buf * T::TILE_STRIDE;
            {
                const float *sd = sides + buf * T::SIDE_STRIDE;
                for_each_patch_cell<K, ADJ>(t, [&](int q, int ry, int s2) { tl[ry * C::PITCH + s2] = sd[q]; });
            }
            __syncthreads();
            convg_accumulate<K, ADJ>(tl, wtab + buf * (kCob * K * K), acc);
            __syncthreads();
            if (!has_next) break;
            ib = nib;
            cl = ncl;
            buf ^= 1;
        }
        cp_async_wait_group<0>();
        if (failed) break;
        convg_store<K, ADJ>(G, t, n, ob, o0, oc, acc);
        __syncthreads();
    }
}

// Clears the ghost frame of every plane of the padded output shards (what H* leaves behind).
struct GhostFrameParams {
    float *shard[kConvMaxWorkers];
    int32_t planes[kConvMaxWorkers], bh[kConvMaxWorkers], bw[kConvMaxWorkers];
    int32_t h;
};
__global__ void clear_ghost_frame_kernel(const __grid_constant__ GhostFrameParams Q) {
    const int s = blockIdx.y;
    const int bh = Q.bh[s], bw = Q.bw[s], h = Q.h;
    const int pw = bw + 2 * h, ph = bh + 2 * h;
    const int frame = ph * pw - bh * bw;                  // ghost cells per plane
    const long long total = (long long)Q.planes[s] * frame;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        const int plane = (int)(idx / frame);
        int e = (int)(idx - (long long)plane * frame), row, col;
        if (e < h * pw) {                                 // rows above the bulk
            row = e / pw;
            col = e - row * pw;
        } else if (e < 2 * h * pw) {                      // rows below
            e -= h * pw;
            row = h + bh + e / pw;
            col = e % pw;
        } else {                                          // columns beside the bulk rows
            e -= 2 * h * pw;
            row = h + e / (2 * h);
            const int c = e % (2 * h);
            col = c < h ? c : bw + c;
        }
        Q.shard[s][((size_t)plane * ph + row) * pw + col] = 0.f;
    }
}

template <int K, bool ADJ>
static distdl_status_t launch_convg(const ConvGParams &G, int in_shards, const int64_t *in_planes, cudaStream_t s) {
    using C = ConvCfg<K, ADJ>;
    using T = ConvTmaCfg<K, ADJ>;
    constexpr int smem_plain = 2 * C::TILE_FLOATS * 4 + 2 * kCob * K * K * 8;
    constexpr int smem_tma = 2 * T::TILE_STRIDE * 4 + 2 * T::SIDE_STRIDE * 4 + 2 * kCob * K * K * 8 + 64 + 128;
    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    static int blocks_plain_on[kMaxDevicesPerProcess] = {0}, blocks_tma_on[kMaxDevicesPerProcess] = {0};
    int &blocks_plain = blocks_plain_on[cur_dev], &blocks_tma = blocks_tma_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(convg_kernel<K, ADJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_plain));
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(convg_tma_kernel<K, ADJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_tma));
        int dev = 0, sms = 0, a = 0, b = 0;
        DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
        DISTDL_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, convg_kernel<K, ADJ>, kConvThreads, smem_plain));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, convg_tma_kernel<K, ADJ>, kConvThreads, smem_tma));
        blocks_plain = sms * std::max(a, 1);
        blocks_tma = sms * std::max(b, 1);
        configured = true;
    }
    const ConvParams &P = G.base;
    EncodeTiledFn enc = tensor_map_encoder();
    bool tma = enc != nullptr && in_shards <= kConvGTmaShards;
    for (int32_t c = 0; c < P.pw_workers; ++c) tma = tma && ((P.bw[c] + 2 * C::IOFF) % 4) == 0;
    if (tma) {
        ConvGTmaParams Q;
        memset(&Q, 0, sizeof(Q));
        Q.g = G;
        const int spatial = P.ph_workers * P.pw_workers;
        const cuuint32_t estr[3] = {1, 1, 1};
        for (int k = 0; k < in_shards; ++k) {
            const int r = (k % spatial) / P.pw_workers, c = k % P.pw_workers;
            const cuuint64_t pitch = (cuuint64_t)(P.bw[c] + 2 * C::IOFF), rows = (cuuint64_t)(P.bh[r] + 2 * C::IOFF);
            const cuuint64_t dims[3] = {pitch, rows, (cuuint64_t)in_planes[k / spatial]};
            const cuuint64_t strides[2] = {pitch * 4, pitch * rows * 4};
            const cuuint32_t box[3] = {(cuuint32_t)C::PITCH, (cuuint32_t)C::ROWS, 1};
            if (enc(&Q.in_map[k], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(P.in[k]), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return fail(DISTDL_ERR_CUDA, "convg: tensor map of input shard %d failed", k);
        }
        const int grid = G.total_tiles < blocks_tma ? G.total_tiles : blocks_tma;
        convg_tma_kernel<K, ADJ><<<grid, kConvThreads, smem_tma, s>>>(Q);
    } else {
        const int grid = G.total_tiles < blocks_plain ? G.total_tiles : blocks_plain;
        convg_kernel<K, ADJ><<<grid, kConvThreads, smem_plain, s>>>(G);
    }
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

// px: partition of the tensor with n_ci channels (x, dx); the other tensor (y, dy) has n_co channels on pco
// blocks and the same spatial partition.  Forward: in = x (padded), out = y (bulk-shaped); adjoint: in = dy
// (bulk-shaped), out = dx (padded, ghosts cleared).
static distdl_status_t convg_impl(const distdl_partition *px, int64_t nco, int32_t pco, const void *const *in,
                                  const void *const *w, const void *const *bias, int32_t kh, int32_t kw,
                                  void *const *out, void *stream, bool adj, const char *what) {
    clear_error();
    if (!px || !in || !w || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (px->rank != 4 || px->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (px->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
    if (px->pshape[0] != 1) return fail(DISTDL_ERR_UNSUPPORTED, "%s: the batch dimension may not be partitioned", what);
    if (kh != kw || (kh != 3 && kh != 5 && kh != 7))
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: kernel %d x %d (supported: 3x3, 5x5, 7x7)", what, kh, kw);
    const int32_t pci = px->pshape[1], ph = px->pshape[2], pw = px->pshape[3];
    if (pco < 1 || nco < pco) return fail(DISTDL_ERR_SHAPE, "%s: %lld output channels on %d blocks", what, (long long)nco, pco);
    if (pci > kMaxChanBlocks || pco > kMaxChanBlocks)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d blocks of a channel partition", what, kMaxChanBlocks);
    if ((int64_t)std::max(pci, pco) * ph * pw > kConvMaxWorkers)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d shards of one tensor", what, kConvMaxWorkers);
    const int h = kh / 2;
    for (int k = 0; k < 4; ++k)
        for (int32_t c = 0; c < px->pshape[k]; ++c) {
            const int want = k < 2 ? 0 : h;
            if (px->hlo[k][c] != want || px->hhi[k][c] != want)
                return fail(DISTDL_ERR_SHAPE, "%s: halo widths must be 0,0,%d,%d on every side", what, h, h);
        }
    ConvGParams G;
    memset(&G, 0, sizeof(G));
    ConvParams &P = G.base;
    int64_t max_bh = 0, max_bw = 0;
    for (int32_t r = 0; r < ph; ++r) max_bh = std::max<int64_t>(max_bh, P.bh[r] = (int32_t)px->size[2][r]);
    for (int32_t c = 0; c < pw; ++c) max_bw = std::max<int64_t>(max_bw, P.bw[c] = (int32_t)px->size[3][c]);
    P.ph_workers = ph;
    P.pw_workers = pw;
    P.tiles_x = (int32_t)((max_bw + kTileW - 1) / kTileW);
    G.tiles_y = (int32_t)((max_bh + kTileH - 1) / kTileH);
    conv_set_divisor(P, 0, (uint32_t)P.tiles_x);
    conv_set_divisor(P, 1, (uint32_t)pw);
    conv_set_divisor(P, 2, (uint32_t)G.tiles_y);
    conv_set_divisor(P, 3, (uint32_t)ph);
    // channel blocks: the evenly split n_ci (from the partition) and n_co
    std::vector<int64_t> co_start, co_size;
    split_evenly(nco, pco, co_start, co_size);
    const int32_t p_out = adj ? pci : pco, p_in = adj ? pco : pci;
    for (int32_t b = 0; b < pci; ++b) (adj ? G.cnt_out : G.cnt_in)[b] = (int32_t)px->size[1][b];
    for (int32_t b = 0; b < pco; ++b) (adj ? G.cnt_in : G.cnt_out)[b] = (int32_t)co_size[b];
    G.p_out = p_out;
    G.p_in = p_in;
    G.pci = pci;
    int groups = 0;
    for (int32_t b = 0; b < p_out; ++b)
        for (int32_t f = 0; f < G.cnt_out[b]; f += kCob) {
            if (groups == kMaxGroups || f > 255) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many output channels", what);
            G.grp_block[groups] = (uint8_t)b;
            G.grp_first[groups] = (uint8_t)f;
            G.grp_count[groups] = (uint8_t)std::min<int32_t>(kCob, G.cnt_out[b] - f);
            ++groups;
        }
    G.groups = groups;
    G.ooff = adj ? h : 0;
    const int64_t total = (int64_t)P.tiles_x * G.tiles_y * ph * pw * px->global_shape[0] * groups;
    if (total >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);
    G.total_tiles = (int32_t)total;
    const int spatial = ph * pw;
    for (int32_t k = 0; k < p_in * spatial; ++k) {
        if (!in[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: input shard %d is NULL", what, k);
        if (!aligned16(in[k])) return fail(DISTDL_ERR_ALIGNMENT, "%s: input shard %d is not 16-byte aligned", what, k);
        P.in[k] = (const float *)in[k];
    }
    for (int32_t k = 0; k < p_out * spatial; ++k) {
        if (!out[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: output shard %d is NULL", what, k);
        if (!aligned16(out[k])) return fail(DISTDL_ERR_ALIGNMENT, "%s: output shard %d is not 16-byte aligned", what, k);
        P.out[k] = (float *)out[k];
    }
    for (int32_t k = 0; k < pco * pci; ++k) {
        if (!w[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: weight block %d is NULL", what, k);
        G.w[k] = (const float *)w[k];
    }
    if (!adj && bias)
        for (int32_t b = 0; b < pco; ++b) G.bias[b] = (const float *)bias[b];
    cudaStream_t s = (cudaStream_t)stream;
    distdl_status_t st;
    int64_t in_planes[kMaxChanBlocks];
    for (int32_t b = 0; b < p_in; ++b) in_planes[b] = px->global_shape[0] * G.cnt_in[b];
    const int ins = p_in * spatial;
    if (!adj) st = kh == 3 ? launch_convg<3, false>(G, ins, in_planes, s) : kh == 5 ? launch_convg<5, false>(G, ins, in_planes, s)
                                                                        : launch_convg<7, false>(G, ins, in_planes, s);
    else st = kh == 3 ? launch_convg<3, true>(G, ins, in_planes, s) : kh == 5 ? launch_convg<5, true>(G, ins, in_planes, s)
                                                                     : launch_convg<7, true>(G, ins, in_planes, s);
    if (st != DISTDL_OK || !adj) return st;
    // adjoint: the ghosts of dx are zero, as H* leaves them
    GhostFrameParams Q;
    memset(&Q, 0, sizeof(Q));
    Q.h = h;
    for (int32_t b = 0; b < pci; ++b)
        for (int32_t r = 0; r < ph; ++r)
            for (int32_t c = 0; c < pw; ++c) {
                const int k = (b * ph + r) * pw + c;
                Q.shard[k] = (float *)out[k];
                Q.planes[k] = (int32_t)(px->global_shape[0] * px->size[1][b]);
                Q.bh[k] = P.bh[r];
                Q.bw[k] = P.bw[c];
            }
    clear_ghost_frame_kernel<<<dim3(64, (unsigned)(pci * spatial)), 256, 0, s>>>(Q);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

// ---------------------------------------------------------------------------------------------
// Parameter gradients of the layer (adjoint convolution algorithm, Section 4 "Sparse layers"):
//   dw^_k[c,a,b] = sum_{n,i,j} dy_k[n,c,i,j] * (H x)_k[n,c,i+a,j+b],   db^_k[c] = sum dy_k[n,c,i,j],
//   dw = R_k dw^_k,  db = R_k db^_k      (every worker holds a copy of the kernel).
// H is fused as in the forward kernel: a block stages the x tile with its ghost rows and columns
// straight from the neighbouring shards' bulk, and the dy tile beside it.  A work item is one
// (channel, slice): the tiles slice, slice + S, slice + 2 S, ... of that channel's planes across all
// workers, so the K*K + 1 running sums stay in registers from tile to tile.  Every thread owns 4 x 8
// pixels of a tile and keeps each sum as a pair (even pixel column, odd pixel column) for the
// packed fp32 FMAs.  At the end of an item the block folds its sums (lanes by shuffles, warps in
// order) and writes one row of K*K + 1 values to the scratch table; a second small kernel adds the
// S rows of a channel in order.  The assignment of tiles to sums is static, so the result does not
// change from run to run.
// ---------------------------------------------------------------------------------------------
constexpr int kGradRow = 64;   // floats per (channel, slice) row of the scratch table (K*K + 1 <= 50 used)

struct ConvGradParams {
    ConvParams base;                        // in = padded x shards; out unused
    const float *dy[kConvMaxWorkers];       // bulk-shaped shards
    float *partial;                         // [channels][slices][kGradRow]
    int32_t slices;
    int32_t tiles_per_plane;                // Ph * tiles_y * Pw * tiles_x
    int32_t tiles_per_channel;              // batch * tiles_per_plane
    int32_t tiles_y;
    // Which planes an item reads.  pairs == 0 (depthwise layer): item channel ch, plane n * channels + ch of x
    // and of dy.  pairs = n_co * n_ci (generalized layer): item (o, c) reads input channel c of x and output
    // channel o of dy, each found in the group of Ph x Pw shards of its channel block.
    int32_t pairs, spatial, n_x;
    int32_t x_blocks, y_blocks;
    int32_t x_start[8], x_cnt[8], y_start[8], y_cnt[8];
};

// plane of batch entry n = n * mult + base, in the shards [wofs, wofs + Ph * Pw)
struct GradItem {
    int x_wofs, x_base, x_mult, dy_wofs, dy_base, dy_mult;
};
__device__ __forceinline__ GradItem grad_item(const ConvGradParams &G, int q) {
    GradItem it;
    if (G.pairs == 0) {
        it.x_wofs = it.dy_wofs = 0;
        it.x_base = it.dy_base = q;
        it.x_mult = it.dy_mult = G.base.channels;
        return it;
    }
    const int o = q / G.n_x, c = q - o * G.n_x;
    int jb = 0, ib = 0;
    for (int b = 1; b < G.x_blocks; ++b)
        if (c >= G.x_start[b]) jb = b;
    for (int b = 1; b < G.y_blocks; ++b)
        if (o >= G.y_start[b]) ib = b;
    it.x_wofs = jb * G.spatial;
    it.x_base = c - G.x_start[jb];
    it.x_mult = G.x_cnt[jb];
    it.dy_wofs = ib * G.spatial;
    it.dy_base = o - G.y_start[ib];
    it.dy_mult = G.y_cnt[ib];
    return it;
}

// dy tile: kTileH rows of kTileW floats, zero outside the shard's bulk
__device__ __forceinline__ void stage_dy_tile(const float *shard, int dy_plane, const ConvTile &t, float *dt) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = min(kTileH, t.bh - t.i0), cols = min(kTileW, t.bw - t.j0);
    const float *plane = shard + (size_t)dy_plane * t.bh * t.bw;
    const bool fast = (t.bw % 4) == 0;
    const int nv = fast ? cols / 4 : 0;
    for (int ry = warp; ry < kTileH; ry += kConvThreads / 32) {
        float *srow = dt + ry * kTileW;
        if (ry >= rows) {
            for (int v = lane; v < kTileW / 4; v += 32) *reinterpret_cast<float4 *>(srow + 4 * v) = make_float4(0.f, 0.f, 0.f, 0.f);
            continue;
        }
        const float *grow = plane + (size_t)(t.i0 + ry) * t.bw + t.j0;
        for (int v = lane; v < nv; v += 32) cp_async16(srow + 4 * v, grow + 4 * v);
        for (int e = 4 * nv + lane; e < kTileW; e += 32) {
            if (e < cols) cp_async4(srow + e, grow + e);
            else srow[e] = 0.f;
        }
    }
}

// Cells of the x tile that stage_tile leaves untouched when the tile is ragged: set to zero, so that
// the products with the zeros of the dy tile are zeros whatever an earlier tile left there.
template <int K>
__device__ __forceinline__ void clear_unstaged_x(const ConvTile &t, float *tile) {
    using C = ConvCfg<K, false>;
    const int out_rows = min(kTileH, t.bh - t.i0), out_cols = min(kTileW, t.bw - t.j0);
    if (out_rows == kTileH && out_cols == kTileW) return;
    const int need_rows = out_rows + 2 * C::PH;
    const int staged = ((out_cols + C::PADL + C::PH + 3) / 4) * 4;
    for (int idx = threadIdx.x; idx < C::ROWS * C::PITCH; idx += kConvThreads) {
        const int ry = idx / C::PITCH, s = idx - ry * C::PITCH;
        if (ry >= need_rows || s >= staged) tile[idx] = 0.f;
    }
}

template <int K>
__device__ __forceinline__ void grad_accumulate(const float *xt, const float *dt, uint64_t (&acc)[K][K], uint64_t &accb) {
    using C = ConvCfg<K, false>;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    constexpr int NP = C::NF / 2;
    uint64_t D[kRowsPerThread][4];
#pragma unroll
    for (int r = 0; r < kRowsPerThread; ++r) {
        const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(dt + (ty * kRowsPerThread + r) * kTileW + kColsPerThread * tx);
        const ulonglong2 q0 = src[0], q1 = src[1];
        D[r][0] = q0.x;
        D[r][1] = q0.y;
        D[r][2] = q1.x;
        D[r][3] = q1.y;
    }
    const uint64_t ones = pack2(1.f, 1.f);
#pragma unroll
    for (int r = 0; r < kRowsPerThread; ++r)
#pragma unroll
        for (int p2 = 0; p2 < 4; ++p2) accb = fma2(D[r][p2], ones, accb);
    const float *tbase = xt + (ty * kRowsPerThread) * C::PITCH + kColsPerThread * tx;
#pragma unroll
    for (int rho = 0; rho < kRowsPerThread + K - 1; ++rho) {
        // one input row: aligned pairs P[i] = (x[2i], x[2i+1]) and shifted pairs Q[i] = (x[2i+1], x[2i+2])
        uint64_t Pr[NP], Qr[NP - 1];
        const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(tbase + rho * C::PITCH);
#pragma unroll
        for (int v = 0; v < NP / 2; ++v) {
            const ulonglong2 q = src[v];
            Pr[2 * v] = q.x;
            Pr[2 * v + 1] = q.y;
        }
#pragma unroll
        for (int i = 0; i < NP - 1; ++i) {
            float a0, a1, b0, b1;
            unpack2(Pr[i], a0, a1);
            unpack2(Pr[i + 1], b0, b1);
            Qr[i] = pack2(a1, b0);
        }
        // pixel pair outermost, taps innermost: consecutive FMAs go to different running sums
#pragma unroll
        for (int p2 = 0; p2 < 4; ++p2) {
#pragma unroll
            for (int r = 0; r < kRowsPerThread; ++r) {
                const int a = rho - r;
                if (a < 0 || a >= K) continue;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    // pixels (2 p2, 2 p2 + 1) of output row r read x columns 2 p2 + b, 2 p2 + b + 1
                    const uint64_t X = (b & 1) ? Qr[p2 + (b - 1) / 2] : Pr[p2 + b / 2];
                    acc[a][b] = fma2(D[r][p2], X, acc[a][b]);
                }
            }
        }
    }
}

template <int K>
__global__ void __launch_bounds__(kConvThreads, 3)
conv_grad_kernel(const __grid_constant__ ConvGradParams G) {
    using C = ConvCfg<K, false>;
    extern __shared__ __align__(16) float smem[];        // two x tiles, then two dy tiles
    float *xts = smem;
    float *dts = smem + 2 * C::TILE_FLOATS;
    __shared__ float red[kConvThreads / 32][K * K + 1];
    const ConvParams &P = G.base;
    const int items = (G.pairs ? G.pairs : P.channels) * G.slices;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int ch = item / G.slices, sl = item - ch * G.slices;
        uint64_t acc[K][K];
        uint64_t accb = 0ull;
#pragma unroll
        for (int a = 0; a < K; ++a)
#pragma unroll
            for (int b = 0; b < K; ++b) acc[a][b] = 0ull;
        const GradItem it = grad_item(G, ch);
        // tile L of the item: its place (batch entry, shard, rows, columns); .plane = the plane of x, dyp = that of dy
        int dyp = 0;
        auto tile_of = [&](int L) {
            ConvTile t = decode_tile(P, L, G.tiles_y, 0);          // decodes the batch entry into .plane
            dyp = t.plane * it.dy_mult + it.dy_base;
            t.plane = t.plane * it.x_mult + it.x_base;
            return t;
        };
        auto stage = [&](const ConvTile &t, int b) {
            if (!t.valid) return;
            float *xt = xts + b * C::TILE_FLOATS;
            clear_unstaged_x<K>(t, xt);
            stage_tile<K, false>(P, t, xt, it.x_wofs);
            stage_dy_tile(G.dy[it.dy_wofs + t.shard], dyp, t, dts + b * (kTileH * kTileW));
        };
        int L = sl, buf = 0;
        if (L < G.tiles_per_channel) {
            ConvTile cur = tile_of(L);
            stage(cur, 0);
            cp_async_commit();
            while (true) {
                const int next = L + G.slices;
                const bool has_next = next < G.tiles_per_channel;
                ConvTile nxt = cur;
                if (has_next) {
                    nxt = tile_of(next);
                    stage(nxt, buf ^ 1);
                }
                cp_async_commit();
                cp_async_wait_group<1>();
                __syncthreads();
                if (cur.valid) grad_accumulate<K>(xts + buf * C::TILE_FLOATS, dts + buf * (kTileH * kTileW), acc, accb);
                __syncthreads();
                if (!has_next) break;
                cur = nxt;
                L = next;
                buf ^= 1;
            }
            cp_async_wait_group<0>();
        }
        // fold: pair halves, lanes (butterfly), then the warps in order
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
        for (int a = 0; a < K; ++a)
#pragma unroll
            for (int b = 0; b <= K; ++b) {
                if (b == K && a != 0) continue;
                float lo, hi;
                unpack2(b == K ? accb : acc[a][b], lo, hi);
                float v = lo + hi;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) red[warp][b == K ? K * K : a * K + b] = v;
            }
        __syncthreads();
        if (threadIdx.x <= K * K) {
            float v = red[0][threadIdx.x];
#pragma unroll
            for (int w2 = 1; w2 < kConvThreads / 32; ++w2) v += red[w2][threadIdx.x];
            G.partial[(size_t)item * kGradRow + threadIdx.x] = v;
        }
        __syncthreads();
    }
}

// TMA variant of the parameter-gradient kernel: the x tile body and (when every shard's rows are
// whole 16-byte units) the dy tile arrive by one bulk tensor copy each -- out-of-range parts of a
// ragged tile are filled with zeros by the copy -- and only the halo strips are fetched cell by cell.
struct ConvGradTmaParams {
    ConvGradParams g;
    CUtensorMap x_map[kConvTmaMaxWorkers];
    CUtensorMap dy_map[kConvTmaMaxWorkers];
};

template <int K, bool DYTMA>
__global__ void __launch_bounds__(kConvThreads, 3)
conv_grad_tma_kernel(const __grid_constant__ ConvGradTmaParams Q) {
    using C = ConvCfg<K, false>;
    using T = ConvTmaCfg<K, false>;
    constexpr int DY_FLOATS = kTileH * kTileW;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    float *tiles = reinterpret_cast<float *>(smem_raw + (((raw + 127u) & ~127u) - raw));
    float *sides = tiles + 2 * T::TILE_STRIDE;
    float *dts = sides + 2 * T::SIDE_STRIDE;
    const uint32_t bars = smem_u32(dts + 2 * DY_FLOATS);
    // the fold at the end of an item reuses the first x tile buffer (idle by then): no static shared memory,
    // which is what lets three blocks share an SM for K = 5
    float (*red)[K * K + 1] = reinterpret_cast<float (*)[K * K + 1]>(tiles);
    const ConvGradParams &G = Q.g;
    const ConvParams &P = G.base;
    if (threadIdx.x == 0) {
        mbar_init(bars, 1);
        mbar_init(bars + 8, 1);
        fence_barrier_init();
    }
    __syncthreads();
    uint32_t phase0 = 0, phase1 = 0;
    bool failed = false;
    const int items = (G.pairs ? G.pairs : P.channels) * G.slices;
    for (int item = blockIdx.x; item < items && !failed; item += gridDim.x) {
        const int ch = item / G.slices, sl = item - ch * G.slices;
        uint64_t acc[K][K];
        uint64_t accb = 0ull;
#pragma unroll
        for (int a = 0; a < K; ++a)
#pragma unroll
            for (int b = 0; b < K; ++b) acc[a][b] = 0ull;
        const GradItem it = grad_item(G, ch);
        // tile L of the item: its place (batch entry, shard, rows, columns); .plane = the plane of x, dyp = that of dy
        int dyp = 0;
        auto tile_of = [&](int L) {
            ConvTile t = decode_tile(P, L, G.tiles_y, 0);          // decodes the batch entry into .plane
            dyp = t.plane * it.dy_mult + it.dy_base;
            t.plane = t.plane * it.x_mult + it.x_base;
            return t;
        };
        auto stage = [&](const ConvTile &t, int b) {
            if (!t.valid) return;
            float *xt = tiles + b * T::TILE_STRIDE, *dt = dts + b * DY_FLOATS;
            if (threadIdx.x == 0) {
                fence_proxy_async();
                mbar_expect_tx(bars + 8 * b, T::BOX_BYTES + (DYTMA ? DY_FLOATS * 4 : 0));
                tma_load_3d(smem_u32(xt), &Q.x_map[it.x_wofs + t.shard], t.j0, t.i0, t.plane, bars + 8 * b);
                if (DYTMA) tma_load_3d(smem_u32(dt), &Q.dy_map[it.dy_wofs + t.shard], t.j0, t.i0, dyp, bars + 8 * b);
            }
            if (!DYTMA) stage_dy_tile(G.dy[it.dy_wofs + t.shard], dyp, t, dt);
            stage_halo_strips<K, false>(P, t, sides + b * T::SIDE_STRIDE, it.x_wofs);
        };
        int L = sl, buf = 0;
        if (L < G.tiles_per_channel) {
            ConvTile cur = tile_of(L);
            stage(cur, 0);
            cp_async_commit();
            while (true) {
                const int next = L + G.slices;
                const bool has_next = next < G.tiles_per_channel;
                ConvTile nxt = cur;
                if (has_next) {
                    nxt = tile_of(next);
                    stage(nxt, buf ^ 1);
                }
                cp_async_commit();
                cp_async_wait_group<1>();
                bool ok = true;
                if (cur.valid) {
                    const uint32_t bar = bars + 8 * buf, parity = buf ? phase1 : phase0;
                    if (!mbar_try_wait(bar, parity)) {
                        const uint64_t t0 = global_timer();
                        while (!mbar_try_wait(bar, parity)) {
                            if (global_timer() - t0 > kConvWaitLimitNs) {
                                ok = false;
                                break;
                            }
                        }
                    }
                    if (buf) phase1 ^= 1; else phase0 ^= 1;
                }
                if (__syncthreads_or(!ok)) {
                    if (threadIdx.x == 0) {
                        atomicExch(&g_conv_status, (int)DISTDL_ERR_TIMEOUT);
                        const uint64_t t0 = global_timer();
                        while (global_timer() - t0 < 1000000ull) {}
                    }
                    failed = true;
                    break;
                }
                float *tl = tiles + buf * T::TILE_STRIDE;
                if (cur.valid) {
                    const float *sd = sides + buf * T::SIDE_STRIDE;
                    for_each_patch_cell<K, false>(cur, [&](int q, int ry, int s2) { tl[ry * C::PITCH + s2] = sd[q]; });
                    // ragged tile: what the box holds beyond the cells the tile's own outputs read is ghost
                    // storage of unknown content; it only ever meets the zeros of the dy tile, but 0 * inf
                    // is not 0 -- clear it
                    const int out_rows = min(kTileH, cur.bh - cur.i0), out_cols = min(kTileW, cur.bw - cur.j0);
                    if (out_rows < kTileH || out_cols < kTileW) {
                        const int need_rows = out_rows + 2 * C::PH, need_cols = out_cols + 2 * C::PH;
                        for (int idx = threadIdx.x; idx < C::ROWS * C::PITCH; idx += kConvThreads) {
                            const int ry = idx / C::PITCH, s2 = idx - ry * C::PITCH;
                            if (ry >= need_rows || s2 >= need_cols) tl[idx] = 0.f;
                        }
                    }
                }
                __syncthreads();
                if (cur.valid) grad_accumulate<K>(tl, dts + buf * DY_FLOATS, acc, accb);
                __syncthreads();
                if (!has_next) break;
                cur = nxt;
                L = next;
                buf ^= 1;
            }
            cp_async_wait_group<0>();
        }
        if (failed) break;
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
        for (int a = 0; a < K; ++a)
#pragma unroll
            for (int b = 0; b <= K; ++b) {
                if (b == K && a != 0) continue;
                float lo, hi;
                unpack2(b == K ? accb : acc[a][b], lo, hi);
                float v = lo + hi;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) red[warp][b == K ? K * K : a * K + b] = v;
            }
        __syncthreads();
        if (threadIdx.x <= K * K) {
            float v = red[0][threadIdx.x];
#pragma unroll
            for (int w2 = 1; w2 < kConvThreads / 32; ++w2) v += red[w2][threadIdx.x];
            G.partial[(size_t)item * kGradRow + threadIdx.x] = v;
        }
        __syncthreads();
    }
}

// dw[c, :, :] and db[c] = the slices' rows of channel c added in order
__global__ void conv_grad_finish_kernel(const float *partial, int slices, int taps, float *dw, float *db) {
    const int ch = blockIdx.x, t = threadIdx.x;
    if (t > taps) return;
    const float *row = partial + (size_t)ch * slices * kGradRow + t;
    float v = row[0];
    for (int s = 1; s < slices; ++s) v += row[(size_t)s * kGradRow];
    if (t < taps) dw[(size_t)ch * taps + t] = v;
    else if (db) db[ch] = v;
}

// Generalized layer: item q = (o, c); the slices' rows added in order go to tap t of dw block (i, j) at
// [o_local][c_local], the last entry of the c = 0 items to db_i[o_local].
struct ConvGGradOut {
    float *dw[64];
    float *db[8];
};
__global__ void convg_grad_finish_kernel(const __grid_constant__ ConvGradParams G, const __grid_constant__ ConvGGradOut O, int taps) {
    const int q = blockIdx.x, t = threadIdx.x;
    if (t > taps) return;
    const float *row = G.partial + (size_t)q * G.slices * kGradRow + t;
    float v = row[0];
    for (int s = 1; s < G.slices; ++s) v += row[(size_t)s * kGradRow];
    const GradItem it = grad_item(G, q);
    const int ib = it.dy_wofs / G.spatial, jb = it.x_wofs / G.spatial;
    if (t < taps) O.dw[ib * G.x_blocks + jb][((size_t)it.dy_base * it.x_mult + it.x_base) * taps + t] = v;
    else if (O.db[ib] && q % G.n_x == 0) O.db[ib][it.dy_base] = v;
}

template <int K>
static constexpr int grad_smem_bytes(bool tma) {
    return tma ? 2 * ConvTmaCfg<K, false>::TILE_STRIDE * 4 + 2 * ConvTmaCfg<K, false>::SIDE_STRIDE * 4 + 2 * kTileH * kTileW * 4 + 64 + 128
               : 2 * ConvCfg<K, false>::TILE_FLOATS * 4 + 2 * kTileH * kTileW * 4;
}

// Resident blocks on the current device: the same number for the plain and the TMA kernels (the smaller
// of their occupancies), so that the slicing -- and with it the order of the sums and the size of the
// scratch table -- does not depend on which of them a call ends up using.
template <int K>
static distdl_status_t grad_config(int *blocks_out) {
    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    static int blocks_on[kMaxDevicesPerProcess] = {0};
    int &blocks = blocks_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_grad_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, grad_smem_bytes<K>(false)));
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_grad_tma_kernel<K, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, grad_smem_bytes<K>(true)));
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(conv_grad_tma_kernel<K, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, grad_smem_bytes<K>(true)));
        int dev = 0, sms = 0, a = 0, b = 0, c = 0;
        DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
        DISTDL_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, conv_grad_kernel<K>, kConvThreads, grad_smem_bytes<K>(false)));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, conv_grad_tma_kernel<K, true>, kConvThreads, grad_smem_bytes<K>(true)));
        DISTDL_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&c, conv_grad_tma_kernel<K, false>, kConvThreads, grad_smem_bytes<K>(true)));
        const int per_sm = std::max(1, std::min(a, std::min(b, c)));
        blocks = sms * per_sm;
        configured = true;
    }
    *blocks_out = blocks;
    return DISTDL_OK;
}

// Geometry shared by the workspace query and the launch: slices per channel and tile counts.
static distdl_status_t grad_plan(const distdl_partition *p, int32_t kh, int32_t kw, const char *what, ConvGradParams *G,
                                 int *grid) {
    if (!p) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL partition", what);
    if (p->rank != 4 || p->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (p->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
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
    ConvParams &P = G->base;
    int64_t max_bh = 0, max_bw = 0;
    for (int32_t r = 0; r < p->pshape[2]; ++r) {
        P.bh[r] = (int32_t)p->size[2][r];
        max_bh = std::max<int64_t>(max_bh, p->size[2][r]);
    }
    for (int32_t c = 0; c < p->pshape[3]; ++c) {
        P.bw[c] = (int32_t)p->size[3][c];
        max_bw = std::max<int64_t>(max_bw, p->size[3][c]);
    }
    P.ph_workers = p->pshape[2];
    P.pw_workers = p->pshape[3];
    P.channels = (int32_t)p->global_shape[1];
    P.tiles_x = (int32_t)((max_bw + kTileW - 1) / kTileW);
    const int tiles_y = (int)((max_bh + kTileH - 1) / kTileH);
    conv_set_divisor(P, 0, (uint32_t)P.tiles_x);
    conv_set_divisor(P, 1, (uint32_t)P.pw_workers);
    conv_set_divisor(P, 2, (uint32_t)tiles_y);
    conv_set_divisor(P, 3, (uint32_t)P.ph_workers);
    const int64_t per_plane = (int64_t)P.tiles_x * tiles_y * p->num_workers;
    const int64_t per_channel = per_plane * p->global_shape[0];
    if (per_channel * P.channels >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);
    int blocks = 0;
    distdl_status_t st = kh == 3 ? grad_config<3>(&blocks) : kh == 5 ? grad_config<5>(&blocks) : grad_config<7>(&blocks);
    if (st != DISTDL_OK) return st;
    // as many slices per channel as give every item a resident block of its own (one wave), never more
    // than tiles; with more channels than blocks, one slice per channel
    int64_t slices = blocks / P.channels;
    slices = std::max<int64_t>(1, std::min<int64_t>(slices, per_channel));
    G->slices = (int32_t)slices;
    G->tiles_per_plane = (int32_t)per_plane;
    G->tiles_per_channel = (int32_t)per_channel;
    G->tiles_y = tiles_y;
    *grid = (int)std::min<int64_t>(blocks, slices * P.channels);
    return DISTDL_OK;
}

template <int K>
static distdl_status_t launch_grad(const distdl_partition *p, const ConvGradParams &G, int grid, float *dw, float *db,
                                   cudaStream_t s, const ConvGGradOut *gout = nullptr) {
    const ConvParams &P = G.base;
    // shards of x and of dy: one group of Ph x Pw for the depthwise layer, one per channel block otherwise
    const int spatial = P.ph_workers * P.pw_workers;
    const int nx = G.pairs ? G.x_blocks * spatial : p->num_workers, ny = G.pairs ? G.y_blocks * spatial : p->num_workers;
    // TMA for the x tiles: few enough workers for the maps to travel as kernel parameters and padded rows
    // of whole 16-byte units; for the dy tiles as well when the bulk rows are
    EncodeTiledFn enc = tensor_map_encoder();
    bool x_tma = nx <= kConvTmaMaxWorkers && ny <= kConvTmaMaxWorkers && enc != nullptr, dy_tma = true;
    for (int32_t c = 0; c < P.pw_workers; ++c) {
        x_tma = x_tma && ((P.bw[c] + 2 * (K / 2)) % 4) == 0;
        dy_tma = dy_tma && (P.bw[c] % 4) == 0;
    }
    if (x_tma) {
        using C = ConvCfg<K, false>;
        ConvGradTmaParams Q;
        memset(&Q, 0, sizeof(Q));
        Q.g = G;
        const cuuint32_t estr[3] = {1, 1, 1};
        for (int32_t wk = 0; wk < std::max(nx, ny); ++wk) {
            const int r = (wk % spatial) / P.pw_workers, c = wk % P.pw_workers;
            const cuuint64_t batch = (cuuint64_t)p->global_shape[0];
            const cuuint64_t xplanes = batch * (cuuint64_t)(G.pairs ? G.x_cnt[std::min(wk / spatial, 7)] : p->global_shape[1]);
            const cuuint64_t planes = batch * (cuuint64_t)(G.pairs ? G.y_cnt[std::min(wk / spatial, 7)] : p->global_shape[1]);
            const cuuint64_t pitch = (cuuint64_t)(P.bw[c] + 2 * C::PH), rows = (cuuint64_t)(P.bh[r] + 2 * C::PH);
            const cuuint64_t dims[3] = {pitch, rows, xplanes};
            const cuuint64_t strides[2] = {pitch * 4, pitch * rows * 4};
            const cuuint32_t box[3] = {(cuuint32_t)C::PITCH, (cuuint32_t)C::ROWS, 1};
            if (wk < nx)
                if (enc(&Q.x_map[wk], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(P.in[wk]), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                    return fail(DISTDL_ERR_CUDA, "conv_adj_params: tensor map of x shard %d failed", wk);
            if (!dy_tma || wk >= ny) continue;
            const cuuint64_t ddims[3] = {(cuuint64_t)P.bw[c], (cuuint64_t)P.bh[r], planes};
            const cuuint64_t dstrides[2] = {(cuuint64_t)P.bw[c] * 4, (cuuint64_t)P.bw[c] * (cuuint64_t)P.bh[r] * 4};
            const cuuint32_t dbox[3] = {(cuuint32_t)kTileW, (cuuint32_t)kTileH, 1};
            if (enc(&Q.dy_map[wk], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(G.dy[wk]), ddims, dstrides, dbox, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return fail(DISTDL_ERR_CUDA, "conv_adj_params: tensor map of dy shard %d failed", wk);
        }
        if (dy_tma) conv_grad_tma_kernel<K, true><<<grid, kConvThreads, grad_smem_bytes<K>(true), s>>>(Q);
        else conv_grad_tma_kernel<K, false><<<grid, kConvThreads, grad_smem_bytes<K>(true), s>>>(Q);
    } else {
        conv_grad_kernel<K><<<grid, kConvThreads, grad_smem_bytes<K>(false), s>>>(G);
    }
    DISTDL_CUDA_CHECK(cudaGetLastError());
    if (G.pairs) convg_grad_finish_kernel<<<G.pairs, 64, 0, s>>>(G, *gout, K * K);
    else conv_grad_finish_kernel<<<G.base.channels, 64, 0, s>>>(G.partial, G.slices, K * K, dw, db);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

// Parameter gradients of the generalized layer: geometry, slices and the channel tables of the items.
static distdl_status_t convg_grad_plan(const distdl_partition *px, int64_t nco, int32_t pco, int32_t kh, int32_t kw,
                                       const char *what, ConvGradParams *G, int *grid) {
    if (!px) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL partition", what);
    if (px->rank != 4 || px->dtype != DISTDL_F32) return fail(DISTDL_ERR_SHAPE, "%s: needs a rank-4 F32 partition", what);
    if (px->any_periodic()) return fail(DISTDL_ERR_UNSUPPORTED, "%s: periodic partitions are not supported by the fused layers", what);
    if (px->pshape[0] != 1) return fail(DISTDL_ERR_UNSUPPORTED, "%s: the batch dimension may not be partitioned", what);
    if (kh != kw || (kh != 3 && kh != 5 && kh != 7))
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: kernel %d x %d (supported: 3x3, 5x5, 7x7)", what, kh, kw);
    const int32_t pci = px->pshape[1], ph = px->pshape[2], pw = px->pshape[3];
    if (pco < 1 || nco < pco) return fail(DISTDL_ERR_SHAPE, "%s: %lld output channels on %d blocks", what, (long long)nco, pco);
    if (pci > 8 || pco > 8) return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than 8 blocks of a channel partition", what);
    if ((int64_t)std::max(pci, pco) * ph * pw > kConvMaxWorkers)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: more than %d shards of one tensor", what, kConvMaxWorkers);
    const int h = kh / 2;
    for (int k = 0; k < 4; ++k)
        for (int32_t c = 0; c < px->pshape[k]; ++c) {
            const int want = k < 2 ? 0 : h;
            if (px->hlo[k][c] != want || px->hhi[k][c] != want)
                return fail(DISTDL_ERR_SHAPE, "%s: halo widths must be 0,0,%d,%d on every side", what, h, h);
        }
    ConvParams &P = G->base;
    int64_t max_bh = 0, max_bw = 0;
    for (int32_t r = 0; r < ph; ++r) max_bh = std::max<int64_t>(max_bh, P.bh[r] = (int32_t)px->size[2][r]);
    for (int32_t c = 0; c < pw; ++c) max_bw = std::max<int64_t>(max_bw, P.bw[c] = (int32_t)px->size[3][c]);
    P.ph_workers = ph;
    P.pw_workers = pw;
    P.channels = (int32_t)px->global_shape[1];
    P.tiles_x = (int32_t)((max_bw + kTileW - 1) / kTileW);
    const int tiles_y = (int)((max_bh + kTileH - 1) / kTileH);
    conv_set_divisor(P, 0, (uint32_t)P.tiles_x);
    conv_set_divisor(P, 1, (uint32_t)pw);
    conv_set_divisor(P, 2, (uint32_t)tiles_y);
    conv_set_divisor(P, 3, (uint32_t)ph);
    const int64_t per_plane = (int64_t)P.tiles_x * tiles_y * ph * pw;
    const int64_t per_item = per_plane * px->global_shape[0];
    const int64_t pairs = nco * px->global_shape[1];
    if (per_item >= ((int64_t)1 << 31) || pairs > 65536) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles or channel pairs", what);
    int blocks = 0;
    distdl_status_t st = kh == 3 ? grad_config<3>(&blocks) : kh == 5 ? grad_config<5>(&blocks) : grad_config<7>(&blocks);
    if (st != DISTDL_OK) return st;
    // about four items per resident block, handed out round-robin; never more slices than tiles
    int64_t slices = (4 * (int64_t)blocks + pairs - 1) / pairs;
    slices = std::max<int64_t>(1, std::min<int64_t>(slices, per_item));
    G->slices = (int32_t)slices;
    G->tiles_per_plane = (int32_t)per_plane;
    G->tiles_per_channel = (int32_t)per_item;
    G->tiles_y = tiles_y;
    G->pairs = (int32_t)pairs;
    G->spatial = ph * pw;
    G->n_x = (int32_t)px->global_shape[1];
    G->x_blocks = pci;
    G->y_blocks = pco;
    std::vector<int64_t> co_start, co_size;
    split_evenly(nco, pco, co_start, co_size);
    for (int32_t b = 0; b < pci; ++b) {
        G->x_start[b] = (int32_t)px->start[1][b];
        G->x_cnt[b] = (int32_t)px->size[1][b];
    }
    for (int32_t b = 0; b < pco; ++b) {
        G->y_start[b] = (int32_t)co_start[b];
        G->y_cnt[b] = (int32_t)co_size[b];
    }
    *grid = (int)std::min<int64_t>(blocks, slices * pairs);
    return DISTDL_OK;
}

}  // namespace distdl

extern "C" distdl_status_t distdl_convg_fwd(const distdl_partition_t *px, int64_t nco, int32_t pco, const void *const *x,
                                            const void *const *w, const void *const *bias, int32_t kh, int32_t kw,
                                            void *const *y, void *stream) {
    return distdl::convg_impl(px, nco, pco, x, w, bias, kh, kw, y, stream, false, "convg_fwd");
}
extern "C" distdl_status_t distdl_convg_adj(const distdl_partition_t *px, int64_t nco, int32_t pco, const void *const *dy,
                                            const void *const *w, int32_t kh, int32_t kw, void *const *dx, void *stream) {
    return distdl::convg_impl(px, nco, pco, dy, w, nullptr, kh, kw, dx, stream, true, "convg_adj");
}

extern "C" distdl_status_t distdl_convg_adj_params_workspace(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                                             int32_t kh, int32_t kw, int64_t *bytes) {
    using namespace distdl;
    clear_error();
    if (!bytes) return fail(DISTDL_ERR_INVALID_ARG, "convg_adj_params_workspace: NULL argument");
    ConvGradParams G;
    memset(&G, 0, sizeof(G));
    int grid = 0;
    const distdl_status_t st = convg_grad_plan(px, nco, pco, kh, kw, "convg_adj_params_workspace", &G, &grid);
    if (st != DISTDL_OK) return st;
    *bytes = (int64_t)G.pairs * G.slices * kGradRow * (int64_t)sizeof(float);
    return DISTDL_OK;
}

extern "C" distdl_status_t distdl_convg_adj_params(const distdl_partition_t *px, int64_t nco, int32_t pco,
                                                   const void *const *x, const void *const *dy, int32_t kh, int32_t kw,
                                                   void *const *dw, void *const *db, void *workspace,
                                                   int64_t workspace_bytes, void *stream) {
    using namespace distdl;
    clear_error();
    const char *what = "convg_adj_params";
    if (!px || !x || !dy || !dw || !workspace) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    ConvGradParams G;
    memset(&G, 0, sizeof(G));
    int grid = 0;
    const distdl_status_t st = convg_grad_plan(px, nco, pco, kh, kw, what, &G, &grid);
    if (st != DISTDL_OK) return st;
    const int64_t need = (int64_t)G.pairs * G.slices * kGradRow * (int64_t)sizeof(float);
    if (workspace_bytes < need) return fail(DISTDL_ERR_INVALID_ARG, "%s: workspace of %lld bytes, %lld needed", what,
                                            (long long)workspace_bytes, (long long)need);
    if (!aligned16(workspace)) return fail(DISTDL_ERR_ALIGNMENT, "%s: workspace not 16-byte aligned", what);
    for (int32_t k = 0; k < G.x_blocks * G.spatial; ++k) {
        if (!x[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: x shard %d is NULL", what, k);
        if (!aligned16(x[k])) return fail(DISTDL_ERR_ALIGNMENT, "%s: x shard %d is not 16-byte aligned", what, k);
        G.base.in[k] = (const float *)x[k];
    }
    for (int32_t k = 0; k < G.y_blocks * G.spatial; ++k) {
        if (!dy[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: dy shard %d is NULL", what, k);
        if (!aligned16(dy[k])) return fail(DISTDL_ERR_ALIGNMENT, "%s: dy shard %d is not 16-byte aligned", what, k);
        G.dy[k] = (const float *)dy[k];
    }
    ConvGGradOut O;
    memset(&O, 0, sizeof(O));
    for (int32_t k = 0; k < G.x_blocks * G.y_blocks; ++k) {
        if (!dw[k]) return fail(DISTDL_ERR_INVALID_ARG, "%s: dw block %d is NULL", what, k);
        O.dw[k] = (float *)dw[k];
    }
    if (db)
        for (int32_t b = 0; b < G.y_blocks; ++b) O.db[b] = (float *)db[b];
    G.partial = (float *)workspace;
    cudaStream_t s = (cudaStream_t)stream;
    if (kh == 3) return launch_grad<3>(px, G, grid, nullptr, nullptr, s, &O);
    if (kh == 5) return launch_grad<5>(px, G, grid, nullptr, nullptr, s, &O);
    return launch_grad<7>(px, G, grid, nullptr, nullptr, s, &O);
}

extern "C" distdl_status_t distdl_conv_adj_params_workspace(const distdl_partition_t *p, int32_t kh, int32_t kw,
                                                            int64_t *bytes) {
    using namespace distdl;
    clear_error();
    if (!bytes) return fail(DISTDL_ERR_INVALID_ARG, "conv_adj_params_workspace: NULL argument");
    ConvGradParams G;
    memset(&G, 0, sizeof(G));
    int grid = 0;
    const distdl_status_t st = grad_plan(p, kh, kw, "conv_adj_params_workspace", &G, &grid);
    if (st != DISTDL_OK) return st;
    *bytes = (int64_t)G.base.channels * G.slices * kGradRow * (int64_t)sizeof(float);
    return DISTDL_OK;
}

extern "C" distdl_status_t distdl_conv_adj_params(const distdl_partition_t *p, const void *const *x,
                                                  const void *const *dy, int32_t kh, int32_t kw, void *dw, void *db,
                                                  void *workspace, int64_t workspace_bytes, void *stream) {
    using namespace distdl;
    clear_error();
    const char *what = "conv_adj_params";
    if (!p || !x || !dy || !dw || !workspace) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    ConvGradParams G;
    memset(&G, 0, sizeof(G));
    int grid = 0;
    const distdl_status_t st = grad_plan(p, kh, kw, what, &G, &grid);
    if (st != DISTDL_OK) return st;
    const int64_t need = (int64_t)G.base.channels * G.slices * kGradRow * (int64_t)sizeof(float);
    if (workspace_bytes < need) return fail(DISTDL_ERR_INVALID_ARG, "%s: workspace of %lld bytes, %lld needed", what,
                                            (long long)workspace_bytes, (long long)need);
    if (!aligned16(dw) || !aligned16(workspace) || (db && !aligned16(db)))
        return fail(DISTDL_ERR_ALIGNMENT, "%s: dw / db / workspace not 16-byte aligned", what);
    for (int32_t wk = 0; wk < p->num_workers; ++wk) {
        if (!x[wk] || !dy[wk]) return fail(DISTDL_ERR_INVALID_ARG, "%s: shard pointer %d is NULL", what, wk);
        if (!aligned16(x[wk]) || !aligned16(dy[wk])) return fail(DISTDL_ERR_ALIGNMENT, "%s: shard %d is not 16-byte aligned", what, wk);
        G.base.in[wk] = (const float *)x[wk];
        G.dy[wk] = (const float *)dy[wk];
    }
    G.partial = (float *)workspace;
    cudaStream_t s = (cudaStream_t)stream;
    if (kh == 3) return launch_grad<3>(p, G, grid, (float *)dw, (float *)db, s);
    if (kh == 5) return launch_grad<5>(p, G, grid, (float *)dw, (float *)db, s);
    return launch_grad<7>(p, G, grid, (float *)dw, (float *)db, s);
}

namespace distdl {

}  // namespace distdl

extern "C" distdl_status_t distdl_conv_fwd(const distdl_partition_t *p, const void *const *x, const void *w,
                                           const void *bias, int32_t kh, int32_t kw, void *const *y, void *stream) {
    return distdl::conv_impl(p, x, w, bias, kh, kw, y, stream, false, "conv_fwd");
}
extern "C" distdl_status_t distdl_conv_adj(const distdl_partition_t *p, const void *const *dy, const void *w,
                                           int32_t kh, int32_t kw, void *const *dx, void *stream) {
    return distdl::conv_impl(p, dy, w, nullptr, kh, kw, dx, stream, true, "conv_adj");
}
