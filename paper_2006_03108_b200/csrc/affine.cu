// Distributed affine layer on a Pfo x Pfi worker grid (Section 4, "Dense layers"): forward
//   x^_{ij} <- B x_j ;  y^_{ij} <- x^_{ij} W_{ij}^T (+ b_i on column j = 0) ;  y_i <- R_j y^_{ij}
// and adjoint (dx only)
//   dy^_{ij} <- B dy_i ;  dx^_{ij} <- dy^_{ij} W_{ij} ;  dx_j <- R_i dx^_{ij}.
//
// All workers live in one device memory, so the broadcast is implicit (every thread block that
// needs a block of x reads it through L2 -- no copy is materialised) and the sum-reduce is the
// tensor-core accumulator itself: one thread block owns a 128 x 128 tile of the output and walks
// through the workers of its grid row (forward) or grid column (adjoint) in worker order, so the
// partial products y^_{ij} never exist in memory and the order of the sum is fixed.
//
// Kernel: warp-specialised, one TMA producer thread, one tcgen05.mma issuer thread, four epilogue
// warps.  Operands are staged by TMA (128-byte swizzle) into a ring of shared-memory stages; the
// fp32 accumulator lives in tensor memory and is read back with tcgen05.ld for the epilogue.
// The forward contraction takes W as the K-major operand ([out, in] rows are contiguous in K =
// in); the adjoint takes the same buffers as the MN-major operand, so no transposed copy of W is
// ever made.  Every wait is bounded: if one runs out, the block records DISTDL_ERR_TIMEOUT in a
// device status word, releases its tensor memory and returns.
#include <cuda.h>

#include <algorithm>
#include <cstring>

#include "common.h"
#include "tma.h"

namespace distdl {

constexpr int kTileM = 128;
constexpr int kTileN = 128;
constexpr int kBlockK = 64;                 // 64 bf16 = one 128-byte swizzle row
constexpr int kAffineThreads = 192;         // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue
constexpr int kMaxMaps = 24;                // tensor maps passed as kernel parameters

__device__ int g_affine_status = 0;         // 0 = ok, otherwise DISTDL_ERR_TIMEOUT

struct AffineParams {
    CUtensorMap a_map[8];                   // activation blocks (x_j forward, dy_i adjoint)
    CUtensorMap w_map[kMaxMaps - 8];        // weight blocks, worker order i * pfi + j
    float *out[8];                          // output blocks (y_i forward, dx_j adjoint)
    const float *bias[8];                   // forward only, may be all null
    int32_t nb;                             // batch rows
    int32_t pfo, pfi;
    int32_t blk_out;                        // columns of one output block
    int32_t blk_red;                        // length of the contraction inside one worker
    int32_t nred;                           // workers summed over (pfi forward, pfo adjoint)
    int32_t adjoint;
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
// Bounded wait: false if the limit ran out or another role already gave up.  The limit is counted
// in SM clock cycles (reading %globaltimer costs several hundred nanoseconds, which would serialise
// the pipeline when it sits on the critical path of every k-block), and the clock is only looked
// at once in a while.
constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit_cycles = kWaitLimitCycles) {
    long long t0 = 0;
    for (unsigned spins = 0;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 63u) == 63u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_cycles) {
                *abort_flag = 1;
                atomicExch(&g_affine_status, (int)DISTDL_ERR_TIMEOUT);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  Fields (bit positions): start address >> 4
// [0,14), leading byte offset >> 4 [16,30), stride byte offset >> 4 [32,46), descriptor version 1
// [46,48), layout type 2 = 128-byte swizzle [61,64).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: D = fp32 [4,6) = 1, A = B = bf16 [7,10) = [10,13) = 1,
// A major bit 15, B major bit 16 (0 = K-major, 1 = MN-major), N >> 3 in [17,23), M >> 4 in [24,29).
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------------------------------
// Cluster helpers for the two-SM variant
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int32_t c0, int32_t c1, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;   // both blocks of the pair
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// ------------------------------------------------------------------------------------------
// Kernel.  PAIR = false: one thread block owns a 128 x 128 output tile (used when the batch fits
// one 128-row tile).  PAIR = true: a cluster of two blocks owns a 256 x 128 tile; each block stages
// its own 128 activation rows and its own half of the weight tile, one tcgen05.mma.cta_group::2
// issued by the leader drives the tensor cores of both SMs and reads the weight halves from both
// shared memories -- a quarter less shared-memory fill per flop, which buys a deeper ring.  The
// leader's "full" barrier counts the bytes of both blocks' bulk copies; "empty" and "accumulator
// ready" are signalled in both blocks at once by a multicast commit.
//
// The producer and the MMA issuer are single threads, so their loops are kept to a few dozen
// instructions per k-block: counters advance incrementally (no divisions) and the shared-memory
// descriptors are a precomputed base plus an offset.
// Tiles are numbered row tile fastest, so blocks that share a weight tile run together.
// ------------------------------------------------------------------------------------------
template <bool PAIR>
struct AffineCfg {
    static constexpr int STAGES = PAIR ? 9 : 6;
    static constexpr int A_BYTES = kTileM * kBlockK * 2;                       // 16 KB
    static constexpr int B_BYTES = (PAIR ? kTileN / 2 : kTileN) * kBlockK * 2; // 8 or 16 KB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment*/ + 256 /*barriers*/;
};

template <bool PAIR>
__global__ void __launch_bounds__(kAffineThreads, 1)
affine_kernel(const __grid_constant__ AffineParams P) {
    using C = AffineCfg<PAIR>;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle pattern is a function of address bits [7,10)
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + C::STAGES * C::STAGE_BYTES);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * C::STAGES;
    const uint32_t bar_acc = bar_empty + 8 * C::STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * C::STAGES + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0;         // 0 = leader of the pair
    const int rows_per_tile = PAIR ? 2 * kTileM : kTileM;
    const int tile = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int row_tiles = (P.nb + rows_per_tile - 1) / rows_per_tile;
    const int m0 = (tile % row_tiles) * rows_per_tile + (int)rank * kTileM;   // this block's first row
    const int ntile = tile / row_tiles;
    const int tiles_per_block = (P.blk_out + kTileN - 1) / kTileN;   // the last tile of a block may be partly empty
    const int oblk = ntile / tiles_per_block;                  // output block (i forward, j adjoint)
    const int n0 = (ntile % tiles_per_block) * kTileN;         // first output column inside the block
    // the last k-block of a worker may reach past its block: TMA fills both operands with zeros there
    const int kblocks_per_worker = (P.blk_red + kBlockK - 1) / kBlockK;
    const int num_kblocks = P.nred * kblocks_per_worker;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);      // the (leader's) producer arrives once, with the byte count
            mbar_init(bar_empty + 8 * s, 1);     // one commit per use
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        // 128 columns of tensor memory: one fp32 accumulator of 128 lanes x 128 columns per block
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kTileN) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kTileN) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tcgen05_fence_before();
    if (PAIR) cluster_sync_all();    // both blocks' barriers exist before anyone signals them
    else __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const CUtensorMap *amap = &P.a_map[0];
            // forward: W_{oblk, r}, next worker = next map; adjoint: W_{r, oblk}, next worker = next grid row
            const CUtensorMap *wmap = P.adjoint ? &P.w_map[oblk] : &P.w_map[oblk * P.pfi];
            const int wstep = P.adjoint ? P.pfi : 1;
            const int nb0 = n0 + (PAIR ? (int)rank * (kTileN / 2) : 0);   // this block's part of the weight tile
            uint32_t s = 0, phase = 0, sa = base;
            int k0 = 0, kin = 0;
            for (int kb = 0; kb < num_kblocks; ++kb) {
                if (!mbar_wait(bar_empty + 8 * s, phase ^ 1, abort_flag)) break;
                const uint32_t full = bar_full + 8 * s;
                if (PAIR) {
                    const uint32_t full_leader = map_to_cta(full, 0);
                    if (rank == 0) mbar_expect_tx(full, 2 * C::STAGE_BYTES);      // both blocks' bytes
                    tma_load_2d_pair(sa, amap, k0, m0, full_leader);
                    if (!P.adjoint) tma_load_2d_pair(sa + C::A_BYTES, wmap, k0, nb0, full_leader);   // box {64 k, 64 rows}
                    else tma_load_2d_pair(sa + C::A_BYTES, wmap, nb0, k0, full_leader);              // box {64 n, 64 k}
                } else {
                    mbar_expect_tx(full, C::STAGE_BYTES);
                    tma_load_2d(sa, amap, k0, m0, full);                        // box {64 k, 128 rows}
                    if (!P.adjoint) {
                        tma_load_2d(sa + C::A_BYTES, wmap, k0, nb0, full);      // K-major: box {64 k, 128 rows}
                    } else {                                                    // MN-major: two boxes {64 n, 64 k}
                        tma_load_2d(sa + C::A_BYTES, wmap, nb0, k0, full);
                        tma_load_2d(sa + C::A_BYTES + C::B_BYTES / 2, wmap, nb0 + 64, k0, full);
                    }
                }
                k0 += kBlockK;
                if (++kin == kblocks_per_worker) {      // next worker of the grid row / column, in order
                    kin = 0;
                    k0 = 0;
                    ++amap;
                    wmap += wstep;
                }
                sa += C::STAGE_BYTES;
                if (++s == C::STAGES) {
                    s = 0;
                    sa = base;
                    phase ^= 1;
                }
            }
            if (*abort_flag) {
                // give copies that are still in flight time to land before the block retires
                const uint64_t t0 = global_timer();
                while (global_timer() - t0 < 1000000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc(PAIR ? 2 * kTileM : kTileM, kTileN, P.adjoint ? 1 : 0);
            // A, K-major: 8-row groups 1024 bytes apart; a K step of 16 elements is 32 bytes.
            // B forward, K-major: the same.  B adjoint, MN-major: 64-column atoms B_BYTES/2 apart
            // (leading offset; one atom per block in the pair variant), 8-k groups 1024 bytes apart; a
            // K step of 16 rows is 2048 bytes.  Descriptor addresses are in 16-byte units.
            const uint64_t a0 = smem_desc(base, 16, 1024);
            const uint64_t b0 = P.adjoint ? smem_desc(base + C::A_BYTES, PAIR ? C::B_BYTES : C::B_BYTES / 2, 1024)
                                          : smem_desc(base + C::A_BYTES, 16, 1024);
            const uint64_t bstep = P.adjoint ? (2048 >> 4) : (32 >> 4);
            uint32_t s = 0, phase = 0;
            uint64_t off = 0;
            bool ok = true;
            for (int kb = 0; kb < num_kblocks; ++kb) {
                ok = mbar_wait(bar_full + 8 * s, phase, abort_flag);
                if (!ok) break;
                tcgen05_fence_after();
                const uint64_t a = a0 + off, b = b0 + off;
                if (PAIR) {
                    umma_bf16_pair(tmem_acc, a, b, idesc, kb ? 1u : 0u);
                    umma_bf16_pair(tmem_acc, a + 2, b + bstep, idesc, 1u);
                    umma_bf16_pair(tmem_acc, a + 4, b + 2 * bstep, idesc, 1u);
                    umma_bf16_pair(tmem_acc, a + 6, b + 3 * bstep, idesc, 1u);
                    tcgen05_commit_pair(bar_empty + 8 * s);     // frees the stage in both blocks
                } else {
                    umma_bf16(tmem_acc, a, b, idesc, kb ? 1u : 0u);
                    umma_bf16(tmem_acc, a + 2, b + bstep, idesc, 1u);
                    umma_bf16(tmem_acc, a + 4, b + 2 * bstep, idesc, 1u);
                    umma_bf16(tmem_acc, a + 6, b + 3 * bstep, idesc, 1u);
                    tcgen05_commit(bar_empty + 8 * s);          // frees the stage once these MMAs retire
                }
                off += C::STAGE_BYTES >> 4;
                if (++s == C::STAGES) {
                    s = 0;
                    off = 0;
                    phase ^= 1;
                }
            }
            if (ok) {                                           // accumulator complete
                if (PAIR) tcgen05_commit_pair(bar_acc);
                else tcgen05_commit(bar_acc);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3;                  // tensor-memory lanes [32 q, 32 q + 32)
        // warp-uniform outcome: tcgen05.ld below is a warp-collective instruction
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar_acc, 0, abort_flag));
        tcgen05_fence_after();
        if (ok) {
            const int row = m0 + quarter * 32 + lane;
            float *out = P.out[oblk] + (size_t)row * P.blk_out + n0;
            const float *bias = P.bias[oblk];
#pragma unroll 1
            for (int c = 0; c < kTileN; c += 32) {
                uint32_t v[32];
                const uint32_t taddr = tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                    "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                      "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                      "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (row < P.nb) {
#pragma unroll
                    for (int q = 0; q < 32; q += 4) {
                        if (n0 + c + q >= P.blk_out) continue;      // columns past the block (whole float4s: blocks are multiples of 8)
                        float4 o;
                        o.x = __uint_as_float(v[q + 0]);
                        o.y = __uint_as_float(v[q + 1]);
                        o.z = __uint_as_float(v[q + 2]);
                        o.w = __uint_as_float(v[q + 3]);
                        if (bias) {
                            const float4 b = __ldg(reinterpret_cast<const float4 *>(bias + n0 + c + q));
                            o.x += b.x; o.y += b.y; o.z += b.z; o.w += b.w;
                        }
                        *reinterpret_cast<float4 *>(out + c + q) = o;
                    }
                }
            }
        }
    }
    // a block may not retire, or free its tensor memory, while its peer can still read its shared
    // memory or signal its barriers
    tcgen05_fence_before();
    if (PAIR) cluster_sync_all();
    else __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)kTileN) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)kTileN) : "memory");
    }
}

// ------------------------------------------------------------------------------------------
// Four-block variant: a cluster of two pairs owns a 256 x 256 output tile and splits the workers of
// the reduction between the pairs (pair 0 takes the first half of the grid row / column, pair 1
// the second half, each in worker order).  With tiles twice as wide every block of activations is
// streamed through L2 by half as many pairs, and splitting the reduction keeps all SMs busy.
//
// Epilogue: pair 0 finishes output columns [0, 128) of the tile, pair 1 columns [128, 256).  Every
// block spills its 128 x 256 fp32 accumulator to its own shared memory (the ring is free by then):
// the half it keeps into `own`, the other half into `send`, which one bulk copy through
// distributed shared memory moves into the `recv` buffer of the block with the same rows in the
// other pair.  Each block then adds (first half of the workers) + (second half), adds the bias and
// writes whole 512-byte row segments.
// ------------------------------------------------------------------------------------------
constexpr int kQuadThreads = 256;                           // warps 0/1: one lane each for TMA and MMA; all 8 in the epilogue
constexpr int kQuadN = 256;                                 // output columns per cluster
constexpr int kQuadStages = 7;
constexpr int kQuadABytes = kTileM * kBlockK * 2;           // 16 KB: this block's 128 activation rows
constexpr int kQuadBBytes = (kQuadN / 2) * kBlockK * 2;     // 16 KB: this block's half of the weight tile
constexpr int kQuadStageBytes = kQuadABytes + kQuadBBytes;
constexpr int kQuadSmemBytes = kQuadStages * kQuadStageBytes + 1024 + 256;
constexpr int kQuadPitch = kQuadN / 2 + 4;                  // floats per row of an epilogue buffer; staggers rows over the banks
constexpr int kQuadBufBytes = kTileM * kQuadPitch * 4;      // 67,584
static_assert(3 * kQuadBufBytes <= kQuadStages * kQuadStageBytes, "epilogue buffers must fit in the ring");
static_assert(kQuadBufBytes % 16 == 0, "bulk copies move multiples of 16 bytes");

__device__ __forceinline__ void tcgen05_commit_mask(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// shared memory of this block -> shared memory of another block of the cluster; the bytes are
// counted on a barrier of the destination block
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_cluster_addr, uint32_t src, uint32_t bytes, uint32_t bar_cluster_addr) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster_addr), "r"(src), "r"(bytes), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(kQuadThreads, 1)
affine_kernel_quad(const __grid_constant__ AffineParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + kQuadStages * kQuadStageBytes);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kQuadStages;
    const uint32_t bar_acc = bar_empty + 8 * kQuadStages;
    const uint32_t bar_recv = bar_acc + 8;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kQuadStages + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = cluster_ctarank();        // 0..3
    const uint32_t khalf = crank >> 1;               // which half of the reduction this pair takes
    const uint32_t prank = crank & 1;                // 0 = leader of its pair
    const uint32_t leader = crank & ~1u;
    const int tile = (int)(blockIdx.x >> 2);
    const int row_tiles = (P.nb + 2 * kTileM - 1) / (2 * kTileM);
    const int m0 = (tile % row_tiles) * 2 * kTileM + (int)prank * kTileM;
    const int ntile = tile / row_tiles;
    const int tiles_per_block = P.blk_out / kQuadN;
    const int oblk = ntile / tiles_per_block;
    const int n0 = (ntile % tiles_per_block) * kQuadN;
    const int kblocks_per_worker = (P.blk_red + kBlockK - 1) / kBlockK;
    const int workers = P.nred / 2;                  // workers summed by this pair
    const int r0 = (int)khalf * workers;             // first of them
    const int num_kblocks = workers * kblocks_per_worker;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQuadStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_recv, 1);
        *abort_flag = 0;
        fence_barrier_init();
        mbar_expect_tx(bar_recv, kQuadBufBytes);     // the other pair's half of this block's columns
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kQuadN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    cluster_sync_all();
    tcgen05_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            const CUtensorMap *amap = &P.a_map[r0];
            const CUtensorMap *wmap = P.adjoint ? &P.w_map[r0 * P.pfi + oblk] : &P.w_map[oblk * P.pfi + r0];
            const int wstep = P.adjoint ? P.pfi : 1;
            const int nb0 = n0 + (int)prank * (kQuadN / 2);
            uint32_t s = 0, phase = 0, sa = base;
            int k0 = 0, kin = 0;
            for (int kb = 0; kb < num_kblocks; ++kb) {
                if (!mbar_wait(bar_empty + 8 * s, phase ^ 1, abort_flag)) break;
                const uint32_t full = bar_full + 8 * s;
                const uint32_t full_leader = map_to_cta(full, leader);
                if (prank == 0) mbar_expect_tx(full, 2 * kQuadStageBytes);
                tma_load_2d_pair(sa, amap, k0, m0, full_leader);
                if (!P.adjoint) {
                    tma_load_2d_pair(sa + kQuadABytes, wmap, k0, nb0, full_leader);                  // box {64 k, 128 rows}
                } else {                                                                            // two boxes {64 n, 64 k}
                    tma_load_2d_pair(sa + kQuadABytes, wmap, nb0, k0, full_leader);
                    tma_load_2d_pair(sa + kQuadABytes + kQuadBBytes / 2, wmap, nb0 + 64, k0, full_leader);
                }
                k0 += kBlockK;
                if (++kin == kblocks_per_worker) {
                    kin = 0;
                    k0 = 0;
                    ++amap;
                    wmap += wstep;
                }
                sa += kQuadStageBytes;
                if (++s == kQuadStages) {
                    s = 0;
                    sa = base;
                    phase ^= 1;
                }
            }
            if (*abort_flag) {
                const uint64_t t0 = global_timer();
                while (global_timer() - t0 < 1000000ull) {}
            }
        }
        __syncwarp();       // the other lanes sleep here instead of polling beside the producer
    } else if (warp == 1) {
        if (lane == 0 && prank == 0) {
            const uint32_t idesc = instr_desc(2 * kTileM, kQuadN, P.adjoint ? 1 : 0);
            const uint64_t a0 = smem_desc(base, 16, 1024);
            const uint64_t b0 = P.adjoint ? smem_desc(base + kQuadABytes, kQuadBBytes / 2, 1024)
                                          : smem_desc(base + kQuadABytes, 16, 1024);
            const uint64_t bstep = P.adjoint ? (2048 >> 4) : (32 >> 4);
            const uint16_t mask = (uint16_t)(3u << leader);       // the two blocks of this pair
            uint32_t s = 0, phase = 0;
            uint64_t off = 0;
            bool ok = true;
            for (int kb = 0; kb < num_kblocks; ++kb) {
                ok = mbar_wait(bar_full + 8 * s, phase, abort_flag);
                if (!ok) break;
                tcgen05_fence_after();
                const uint64_t a = a0 + off, b = b0 + off;
                umma_bf16_pair(tmem_acc, a, b, idesc, kb ? 1u : 0u);
                umma_bf16_pair(tmem_acc, a + 2, b + bstep, idesc, 1u);
                umma_bf16_pair(tmem_acc, a + 4, b + 2 * bstep, idesc, 1u);
                umma_bf16_pair(tmem_acc, a + 6, b + 3 * bstep, idesc, 1u);
                tcgen05_commit_mask(bar_empty + 8 * s, mask);
                off += kQuadStageBytes >> 4;
                if (++s == kQuadStages) {
                    s = 0;
                    off = 0;
                    phase ^= 1;
                }
            }
            if (ok) tcgen05_commit_mask(bar_acc, mask);
        }
        __syncwarp();
    }

    // ---------------------------------------------------------------------- epilogue, all warps
    // this pair's accumulator is complete: its MMAs have retired, so the ring is free as well
    const bool acc_ok = mbar_wait(bar_acc, 0, abort_flag);
    const bool ok = __syncthreads_and(acc_ok) != 0;
    tcgen05_fence_after();
    tcgen05_fence_before();
    cluster_sync_all();                      // ... in all four blocks: `recv` may be written from outside

    const int quarter = warp & 3;            // tensor-memory lanes [32 q, 32 q + 32) belong to warps q and q + 4
    const int chalf = warp >> 2;             // column half of the tile this warp spills
    const uint32_t buf_own = base, buf_send = base + kQuadBufBytes, buf_recv = base + 2 * kQuadBufBytes;
    if (ok) {
        tcgen05_fence_after();
        const uint32_t dst = ((uint32_t)chalf == khalf ? buf_own : buf_send) +
                             (uint32_t)((quarter * 32 + lane) * kQuadPitch * 4);
#pragma unroll 1
        for (int c = 0; c < kQuadN / 2; c += 32) {
            uint32_t v[32];
            tmem_ld32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(chalf * (kQuadN / 2) + c), v);
#pragma unroll
            for (int q = 0; q < 32; q += 4)
                asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst + (uint32_t)((c + q) * 4)), "r"(v[q]),
                             "r"(v[q + 1]), "r"(v[q + 2]), "r"(v[q + 3]) : "memory");
        }
        fence_proxy_async();                 // the bulk copy below reads what was just written
    }
    __syncthreads();
    if (ok && threadIdx.x == 0)
        bulk_copy_to_cta(map_to_cta(buf_recv, crank ^ 2u), buf_send, kQuadBufBytes, map_to_cta(bar_recv, crank ^ 2u));
    const bool got = ok && mbar_wait(bar_recv, 0, abort_flag);
    if (got) {
        const float *own = reinterpret_cast<const float *>(aligned);
        const float *recv = reinterpret_cast<const float *>(aligned + 2 * kQuadBufBytes);
        const int col = n0 + (int)khalf * (kQuadN / 2) + 4 * lane;     // column inside the output block
        const float *bias = P.bias[oblk];
        float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
        if (bias) b = __ldg(reinterpret_cast<const float4 *>(bias + col));
        constexpr int kRowsPerWarp = kTileM / (kQuadThreads / 32);
#pragma unroll 4
        for (int i = 0; i < kRowsPerWarp; ++i) {
            const int rloc = warp * kRowsPerWarp + i;
            const int row = m0 + rloc;
            if (row >= P.nb) break;
            const float4 mine = *reinterpret_cast<const float4 *>(own + rloc * kQuadPitch + 4 * lane);
            const float4 other = *reinterpret_cast<const float4 *>(recv + rloc * kQuadPitch + 4 * lane);
            // (workers of the first half) + (workers of the second half), then the bias
            float4 o;
            o.x = (khalf == 0 ? mine.x + other.x : other.x + mine.x) + b.x;
            o.y = (khalf == 0 ? mine.y + other.y : other.y + mine.y) + b.y;
            o.z = (khalf == 0 ? mine.z + other.z : other.z + mine.z) + b.z;
            o.w = (khalf == 0 ? mine.w + other.w : other.w + mine.w) + b.w;
            *reinterpret_cast<float4 *>(P.out[oblk] + (size_t)row * P.blk_out + col) = o;
        }
    }
    // nobody retires while its outgoing copy may still read its shared memory or a peer may signal
    // its barriers; the peer's arrival here follows the end of that copy
    tcgen05_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)kQuadN) : "memory");
    }
}

// ------------------------------------------------------------------------------------------
// Parameter gradients of the adjoint affine algorithm (Section 4, "Dense layers"):
//   dW_{ij} = dy^_{ij}^T x^_{ij}  with dy^_{ij} = dy_i (B along grid rows), x^_{ij} = x_j (B along grid
//   columns, kept from the forward pass);  db_i = column sums of dy_i (the bias lives on grid column 0).
// The weights are distributed over the worker grid itself, so nothing is reduced afterwards: each
// thread block owns one 128 x 128 tile of one worker's dW block and contracts over the batch.
// Both operands are MN-major for the tensor cores (dy_i is [nb, out] row-major: the M index is
// contiguous; x_j is [nb, in]: the N index is contiguous), staged by TMA as 64 x 64 swizzled atoms.
// The output (fp32, nfo x nfi) dominates the traffic: the epilogue stages the tile in (swizzled)
// shared memory and hands it to TMA stores, so whole 128-byte lines leave the SM while the loads and
// MMAs of the next tile run.
// ------------------------------------------------------------------------------------------
constexpr int kDwThreads = 192;                              // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue
constexpr int kDwStages = 4;
constexpr int kDwOperandBytes = 2 * 64 * kBlockK * 2;        // two 64 x 64 bf16 atoms = 16 KB
constexpr int kDwStageBytes = 2 * kDwOperandBytes;           // A and B
constexpr int kDwOutBytes = kTileM * kTileN * 4;             // 64 KB: the fp32 tile as four 128 x 32 boxes
constexpr int kDwSmemBytes = kDwStages * kDwStageBytes + kDwOutBytes + 1024 + 128;
constexpr int kDwTmemCols = 2 * kTileN;                      // two accumulators

struct AffineDwParams {
    CUtensorMap dy_map[8];                  // dy_i  [nb, bfo] bf16, box {64 out, 64 batch}
    CUtensorMap x_map[8];                   // x_j   [nb, bfi] bf16, box {64 in, 64 batch}
    CUtensorMap dw_map[kMaxMaps - 8];       // dW_ij [bfo, bfi] fp32, box {32 in, 128 out}
    int32_t nb, pfi;
    int32_t tiles_m, tiles_n;               // 128 x 128 tiles per worker block
    int32_t total_tiles;
    int32_t bfi;                            // columns of a dW block
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int32_t c0, int32_t c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// barrier 1 of the four epilogue warps, combined with an AND over their predicates
__device__ __forceinline__ bool epilogue_all(bool pred) {
    uint32_t out;
    asm volatile(
        "{\n.reg .pred p, q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "barrier.cta.red.and.pred p, 1, 128, q;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(out) : "r"((uint32_t)pred) : "memory");
    return out != 0;
}

struct DwTile {
    int wi, wj, m0, n0;
};
__device__ __forceinline__ DwTile dw_tile(const AffineDwParams &P, int tile) {
    // tile id: column tile fastest, then row tile, then worker j, then worker i
    DwTile t;
    int rest = tile;
    t.n0 = (rest % P.tiles_n) * kTileN;
    rest /= P.tiles_n;
    t.m0 = (rest % P.tiles_m) * kTileM;
    rest /= P.tiles_m;
    t.wj = rest % P.pfi;
    t.wi = rest / P.pfi;
    return t;
}

// Persistent: one block per SM walks over tiles blockIdx.x, + gridDim.x, ...  The producer runs ahead
// through a four-stage ring (a whole tile at batch 256), the accumulator alternates between two
// 128-column halves of tensor memory, and the epilogue of tile t (tensor memory -> swizzled shared
// memory -> TMA stores) runs while the tensor cores work on tile t + 1.
__global__ void __launch_bounds__(kDwThreads, 1)
affine_dw_kernel(const __grid_constant__ AffineDwParams P) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *aligned = smem_raw + (base - raw);
    const uint32_t out_base = base + kDwStages * kDwStageBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(aligned + kDwStages * kDwStageBytes + kDwOutBytes);
    const uint32_t bar_full = smem_u32(bars);
    const uint32_t bar_empty = bar_full + 8 * kDwStages;
    const uint32_t bar_acc_full = bar_empty + 8 * kDwStages;     // two
    const uint32_t bar_acc_empty = bar_acc_full + 16;            // two
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * kDwStages + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kblocks = (P.nb + kBlockK - 1) / kBlockK;       // rows past nb are filled with zeros by TMA

    if (threadIdx.x == 0) {
        for (int s = 0; s < kDwStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 4);                  // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kDwTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t s = 0, phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x) {
                const DwTile t = dw_tile(P, tile);
                const CUtensorMap *amap = &P.dy_map[t.wi], *bmap = &P.x_map[t.wj];
                for (int kb = 0; kb < num_kblocks; ++kb) {
                    ok = mbar_wait(bar_empty + 8 * s, phase ^ 1, abort_flag);
                    if (!ok) break;
                    const uint32_t full = bar_full + 8 * s, sa = base + s * kDwStageBytes;
                    mbar_expect_tx(full, kDwStageBytes);
                    const int k0 = kb * kBlockK;
                    tma_load_2d(sa, amap, t.m0, k0, full);                                 // atom: out features m0 .. m0 + 63
                    tma_load_2d(sa + kDwOperandBytes / 2, amap, t.m0 + 64, k0, full);
                    tma_load_2d(sa + kDwOperandBytes, bmap, t.n0, k0, full);               // atom: in features n0 .. n0 + 63
                    tma_load_2d(sa + kDwOperandBytes + kDwOperandBytes / 2, bmap, t.n0 + 64, k0, full);
                    if (++s == kDwStages) {
                        s = 0;
                        phase ^= 1;
                    }
                }
            }
            if (*abort_flag) {
                const uint64_t t0 = global_timer();
                while (global_timer() - t0 < 1000000ull) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // both operands MN-major (bits 15 and 16): 64-wide atoms 8 KB apart (leading offset), groups of
            // eight batch rows 1024 bytes apart (stride offset), a K step of 16 batch rows is 2048 bytes
            const uint32_t idesc = instr_desc(kTileM, kTileN, 1) | (1u << 15);
            uint32_t s = 0, phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < P.total_tiles && ok; tile += gridDim.x, ++it) {
                const uint32_t buf = (uint32_t)it & 1u;
                // the epilogue has read this half's previous tile (passes at once the first two times)
                ok = mbar_wait(bar_acc_empty + 8 * buf, (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t tmem_acc = tmem_base + buf * (uint32_t)kTileN;
                for (int kb = 0; kb < num_kblocks; ++kb) {
                    ok = mbar_wait(bar_full + 8 * s, phase, abort_flag);
                    if (!ok) break;
                    tcgen05_fence_after();
                    const uint32_t sa = base + s * kDwStageBytes;
                    const uint64_t a = smem_desc(sa, kDwOperandBytes / 2, 1024);
                    const uint64_t b = smem_desc(sa + kDwOperandBytes, kDwOperandBytes / 2, 1024);
                    constexpr uint64_t kstep = 2048 >> 4;
                    umma_bf16(tmem_acc, a, b, idesc, kb ? 1u : 0u);
                    umma_bf16(tmem_acc, a + kstep, b + kstep, idesc, 1u);
                    umma_bf16(tmem_acc, a + 2 * kstep, b + 2 * kstep, idesc, 1u);
                    umma_bf16(tmem_acc, a + 3 * kstep, b + 3 * kstep, idesc, 1u);
                    tcgen05_commit(bar_empty + 8 * s);
                    if (++s == kDwStages) {
                        s = 0;
                        phase ^= 1;
                    }
                }
                if (ok) tcgen05_commit(bar_acc_full + 8 * buf);
            }
        }
        __syncwarp();
    } else {
        // epilogue.  Box q of the staging buffer (columns 32 q .. 32 q + 31) is a 128 x 32 fp32 array of
        // 128-byte rows with the 16-byte chunks of row r stored at chunk ^ (r & 7): the layout of a
        // 128-byte-swizzled tensor map.  Every decision to go on or to give up is taken by the four warps
        // together, so they always meet at the same barriers.
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const bool issuer = warp == 2 && lane == 0;
        int it = 0;
        for (int tile = blockIdx.x; tile < P.total_tiles; tile += gridDim.x, ++it) {
            const uint32_t buf = (uint32_t)it & 1u;
            const bool mine = mbar_wait(bar_acc_full + 8 * buf, ((uint32_t)it >> 1) & 1u, abort_flag);
            if (!epilogue_all(mine)) break;
            tcgen05_fence_after();
            const uint32_t tmem_acc = tmem_base + buf * (uint32_t)kTileN;
            const DwTile t = dw_tile(P, tile);
            const CUtensorMap *omap = &P.dw_map[t.wi * P.pfi + t.wj];
            // box by box, so that the read-out of one box by its store (which runs at the rate of the SM's
            // port into the memory system) overlaps the copy of the next box out of tensor memory
#pragma unroll 1
            for (int q = 0; q < kTileN / 32; ++q) {
                // at most three stores in flight: the one that read this box for the previous tile is done
                if (issuer) asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory");
                asm volatile("bar.sync 1, 128;" ::: "memory");
                uint32_t v[32];
                tmem_ld32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(32 * q), v);
                const uint32_t boxaddr = out_base + (uint32_t)q * (kTileM * 128);
                const uint32_t rowaddr = boxaddr + (uint32_t)row * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                 ::"r"(rowaddr + (uint32_t)((c ^ (row & 7)) << 4)), "r"(v[4 * c]), "r"(v[4 * c + 1]),
                                   "r"(v[4 * c + 2]), "r"(v[4 * c + 3]) : "memory");
                if (q == kTileN / 32 - 1) {
                    // this half of tensor memory may be overwritten by the tile after the next
                    tcgen05_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_acc_empty + 8 * buf);
                }
                fence_proxy_async();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (issuer) {
                    // a box that starts past the last column of the block has nothing to store (boxes that
                    // only reach past it are clipped by the copy); its group is committed empty
                    if (t.n0 + 32 * q < P.bfi) tma_store_2d(omap, boxaddr, t.n0 + 32 * q, t.m0);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        if (issuer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores done before the block retires
    }
    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kDwTmemCols) : "memory");
    }
}

// db_i[o] = sum over the batch of dy_i[b, o], fp32 sums of bf16 values in a fixed order: the batch is cut
// into eight contiguous chunks (one per warp, rows ascending inside a chunk) and the chunk sums are
// added in chunk order.  A block covers 64 columns of one dy block.
struct AffineDbParams {
    const uint16_t *dy[8];
    float *db[8];
    int32_t nb, bfo;
};
constexpr int kDbThreads = 256;
__global__ void __launch_bounds__(kDbThreads) affine_db_kernel(const AffineDbParams P) {
    __shared__ float part[kDbThreads / 32][64];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col = blockIdx.x * 64 + 2 * lane;
    const int i = blockIdx.y;
    const int chunk = (P.nb + kDbThreads / 32 - 1) / (kDbThreads / 32);
    const int b0 = warp * chunk, b1 = min(P.nb, b0 + chunk);
    const uint16_t *src = P.dy[i] + col;
    float s0 = 0.f, s1 = 0.f;
    if (col < P.bfo) {
#pragma unroll 8
        for (int b = b0; b < b1; ++b) {
            const uint32_t two = *reinterpret_cast<const uint32_t *>(src + (size_t)b * P.bfo);
            s0 += __uint_as_float(two << 16);
            s1 += __uint_as_float(two & 0xffff0000u);
        }
    }
    part[warp][2 * lane] = s0;
    part[warp][2 * lane + 1] = s1;
    __syncthreads();
    if (threadIdx.x < 64) {
        float v = part[0][threadIdx.x];
#pragma unroll
        for (int w = 1; w < kDbThreads / 32; ++w) v += part[w][threadIdx.x];
        if (blockIdx.x * 64 + (int)threadIdx.x < P.bfo) P.db[i][blockIdx.x * 64 + threadIdx.x] = v;
    }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
static EncodeTiledFn encode_fn() { return tensor_map_encoder(); }

// Row-major bf16 matrix [rows, cols]; box = {box_cols (inner), box_rows}; 128-byte swizzle.
static bool make_map(CUtensorMap *m, const void *ptr, int64_t rows, int64_t cols, int box_cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static distdl_status_t affine_impl(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                   const void *const *act, const void *const *w, const void *const *bias,
                                   void *const *out, void *stream, bool adjoint, const char *what) {
    clear_error();
    if (!act || !w || !out) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (nb < 1 || nfi < 1 || nfo < 1 || pfo < 1 || pfi < 1)
        return fail(DISTDL_ERR_INVALID_ARG, "%s: non-positive size", what);
    if (nfi % pfi || nfo % pfo) return fail(DISTDL_ERR_SHAPE, "%s: features not divisible by the worker grid", what);
    const int64_t bfi = nfi / pfi, bfo = nfo / pfo;
    if (bfi % 8 || bfo % 8)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: per-worker feature blocks must be multiples of 8 (rows of whole 16-byte units)", what);
    if (pfo > 8 || pfi > 8 || pfo * pfi > kMaxMaps - 8)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: worker grid larger than 8 per side or %d workers", what, kMaxMaps - 8);
    if (nb > (1 << 20)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: batch too large", what);
    const int nact = adjoint ? pfo : pfi, nout = adjoint ? pfi : pfo;
    for (int i = 0; i < nact; ++i) {
        if (!act[i]) return fail(DISTDL_ERR_INVALID_ARG, "%s: activation block %d is NULL", what, i);
        if (!aligned16(act[i])) return fail(DISTDL_ERR_ALIGNMENT, "%s: activation block %d not 16-byte aligned", what, i);
    }
    for (int i = 0; i < nout; ++i) {
        if (!out[i]) return fail(DISTDL_ERR_INVALID_ARG, "%s: output block %d is NULL", what, i);
        if (!aligned16(out[i])) return fail(DISTDL_ERR_ALIGNMENT, "%s: output block %d not 16-byte aligned", what, i);
        if (bias && bias[i] && !aligned16(bias[i])) return fail(DISTDL_ERR_ALIGNMENT, "%s: bias %d not 16-byte aligned", what, i);
    }
    for (int i = 0; i < pfo * pfi; ++i) {
        if (!w[i]) return fail(DISTDL_ERR_INVALID_ARG, "%s: weight block %d is NULL", what, i);
        if (!aligned16(w[i])) return fail(DISTDL_ERR_ALIGNMENT, "%s: weight block %d not 16-byte aligned", what, i);
    }
    if (!encode_fn()) return fail(DISTDL_ERR_CUDA, "%s: cuTensorMapEncodeTiled is not available", what);

    AffineParams P;
    memset(&P, 0, sizeof(P));
    const int64_t act_cols = adjoint ? bfo : bfi;
    for (int i = 0; i < nact; ++i)
        if (!make_map(&P.a_map[i], act[i], nb, act_cols, kBlockK, kTileM))
            return fail(DISTDL_ERR_CUDA, "%s: tensor map of activation block %d failed", what, i);
    // more than one 128-row tile of the batch: a pair of blocks shares each 256 x 128 output tile
    const bool pair = nb > kTileM;
    // four-block variant: an even number of workers to sum over and output blocks of whole 256-column tiles
    const bool quad = pair && ((adjoint ? pfo : pfi) % 2 == 0) && ((adjoint ? bfi : bfo) % kQuadN == 0);
    for (int i = 0; i < pfo * pfi; ++i) {
        // forward: box {64 along in-features (K), 128 out-feature rows} (64 rows per block of a pair);
        // adjoint: box {64 along in-features (N), 64 out-feature rows (K)} of the same row-major
        // [bfo, bfi] block
        const bool ok = adjoint ? make_map(&P.w_map[i], w[i], bfo, bfi, 64, kBlockK)
                                : make_map(&P.w_map[i], w[i], bfo, bfi, kBlockK, quad ? kQuadN / 2 : (pair ? kTileN / 2 : kTileN));
        if (!ok) return fail(DISTDL_ERR_CUDA, "%s: tensor map of weight block %d failed", what, i);
    }
    for (int i = 0; i < nout; ++i) {
        P.out[i] = (float *)out[i];
        P.bias[i] = (!adjoint && bias) ? (const float *)bias[i] : nullptr;
    }
    P.nb = (int32_t)nb;
    P.pfo = pfo;
    P.pfi = pfi;
    P.blk_out = (int32_t)(adjoint ? bfi : bfo);
    P.blk_red = (int32_t)(adjoint ? bfo : bfi);
    P.nred = adjoint ? pfo : pfi;
    P.adjoint = adjoint ? 1 : 0;

    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(affine_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               AffineCfg<false>::SMEM_BYTES));
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(affine_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               AffineCfg<true>::SMEM_BYTES));
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(affine_kernel_quad, cudaFuncAttributeMaxDynamicSharedMemorySize, kQuadSmemBytes));
        configured = true;
    }
    const int64_t blk_out = adjoint ? bfi : bfo;
    const int64_t ntiles = (adjoint ? pfi : pfo) * ((blk_out + kTileN - 1) / kTileN);
    if (quad) {
        const int64_t row_pairs = (nb + 2 * kTileM - 1) / (2 * kTileM);
        const int64_t qtiles = (adjoint ? nfi : nfo) / kQuadN;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)(4 * row_pairs * qtiles));
        cfg.blockDim = dim3(kQuadThreads);
        cfg.dynamicSmemBytes = kQuadSmemBytes;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 4;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        DISTDL_CUDA_CHECK(cudaLaunchKernelEx(&cfg, affine_kernel_quad, P));
    } else if (pair) {
        const int64_t row_pairs = (nb + 2 * kTileM - 1) / (2 * kTileM);
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)(2 * row_pairs * ntiles));
        cfg.blockDim = dim3(kAffineThreads);
        cfg.dynamicSmemBytes = AffineCfg<true>::SMEM_BYTES;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        DISTDL_CUDA_CHECK(cudaLaunchKernelEx(&cfg, affine_kernel<true>, P));
    } else {
        const int64_t row_tiles = (nb + kTileM - 1) / kTileM;
        affine_kernel<false><<<(unsigned)(row_tiles * ntiles), kAffineThreads, AffineCfg<false>::SMEM_BYTES,
                               (cudaStream_t)stream>>>(P);
    }
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

static bool make_map_f32(CUtensorMap *m, const void *ptr, int64_t rows, int64_t cols, int box_cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static distdl_status_t affine_params_impl(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                          const void *const *dy, const void *const *x, void *const *dw,
                                          void *const *db, void *stream) {
    const char *what = "affine_adj_params";
    clear_error();
    if (!dy || !x || !dw) return fail(DISTDL_ERR_INVALID_ARG, "%s: NULL argument", what);
    if (nb < 1 || nfi < 1 || nfo < 1 || pfo < 1 || pfi < 1) return fail(DISTDL_ERR_INVALID_ARG, "%s: non-positive size", what);
    if (nfi % pfi || nfo % pfo) return fail(DISTDL_ERR_SHAPE, "%s: features not divisible by the worker grid", what);
    const int64_t bfi = nfi / pfi, bfo = nfo / pfo;
    if (bfi % 8 || bfo % 8)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: per-worker feature blocks must be multiples of 8 (rows of whole 16-byte units)", what);
    if (pfo > 8 || pfi > 8 || pfo * pfi > kMaxMaps - 8)
        return fail(DISTDL_ERR_UNSUPPORTED, "%s: worker grid larger than 8 per side or %d workers", what, kMaxMaps - 8);
    if (nb > (1 << 20)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: batch too large", what);
    for (int i = 0; i < pfo; ++i) {
        if (!dy[i] || (db && !db[i])) return fail(DISTDL_ERR_INVALID_ARG, "%s: dy / db block %d is NULL", what, i);
        if (!aligned16(dy[i]) || (db && !aligned16(db[i]))) return fail(DISTDL_ERR_ALIGNMENT, "%s: dy / db block %d not 16-byte aligned", what, i);
    }
    for (int j = 0; j < pfi; ++j) {
        if (!x[j]) return fail(DISTDL_ERR_INVALID_ARG, "%s: x block %d is NULL", what, j);
        if (!aligned16(x[j])) return fail(DISTDL_ERR_ALIGNMENT, "%s: x block %d not 16-byte aligned", what, j);
    }
    for (int i = 0; i < pfo * pfi; ++i) {
        if (!dw[i]) return fail(DISTDL_ERR_INVALID_ARG, "%s: dW block %d is NULL", what, i);
        if (!aligned16(dw[i])) return fail(DISTDL_ERR_ALIGNMENT, "%s: dW block %d not 16-byte aligned", what, i);
    }
    if (!encode_fn()) return fail(DISTDL_ERR_CUDA, "%s: cuTensorMapEncodeTiled is not available", what);
    // tiles past the end of a block are partly empty: loads are zero-filled and stores clipped by TMA
    const int64_t tiles = ((bfo + kTileM - 1) / kTileM) * ((bfi + kTileN - 1) / kTileN) * pfo * pfi;
    if (tiles >= ((int64_t)1 << 31)) return fail(DISTDL_ERR_UNSUPPORTED, "%s: too many tiles", what);

    AffineDwParams P;
    memset(&P, 0, sizeof(P));
    for (int i = 0; i < pfo; ++i)
        if (!make_map(&P.dy_map[i], dy[i], nb, bfo, 64, kBlockK)) return fail(DISTDL_ERR_CUDA, "%s: tensor map of dy block %d failed", what, i);
    for (int j = 0; j < pfi; ++j)
        if (!make_map(&P.x_map[j], x[j], nb, bfi, 64, kBlockK)) return fail(DISTDL_ERR_CUDA, "%s: tensor map of x block %d failed", what, j);
    for (int i = 0; i < pfo * pfi; ++i)
        if (!make_map_f32(&P.dw_map[i], dw[i], bfo, bfi, 32, kTileM)) return fail(DISTDL_ERR_CUDA, "%s: tensor map of dW block %d failed", what, i);
    P.nb = (int32_t)nb;
    P.pfi = pfi;
    P.tiles_m = (int32_t)((bfo + kTileM - 1) / kTileM);
    P.tiles_n = (int32_t)((bfi + kTileN - 1) / kTileN);
    P.total_tiles = (int32_t)tiles;
    P.bfi = (int32_t)bfi;
    // one-time set-up per device (kernel attributes, occupancy): a process may drive several GPUs
    static bool configured_on[kMaxDevicesPerProcess] = {false};
    int cur_dev = 0;
    DISTDL_CUDA_CHECK(cudaGetDevice(&cur_dev));
    if (cur_dev < 0 || cur_dev >= kMaxDevicesPerProcess)
        return fail(DISTDL_ERR_UNSUPPORTED, "device index %d: at most %d devices per process", cur_dev, kMaxDevicesPerProcess);
    std::lock_guard<std::mutex> setup_lock(setup_mutex());      // first calls from several threads set up once
    bool &configured = configured_on[cur_dev];
    static int sms_on[kMaxDevicesPerProcess] = {0};
    int &sms = sms_on[cur_dev];
    if (!configured) {
        DISTDL_CUDA_CHECK(cudaFuncSetAttribute(affine_dw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemBytes));
        int dev = 0;
        DISTDL_CUDA_CHECK(cudaGetDevice(&dev));
        DISTDL_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        configured = true;
    }
    const unsigned grid = (unsigned)std::min<int64_t>(tiles, sms > 0 ? sms : 1);
    affine_dw_kernel<<<grid, kDwThreads, kDwSmemBytes, (cudaStream_t)stream>>>(P);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    if (db) {
        AffineDbParams B;
        memset(&B, 0, sizeof(B));
        for (int i = 0; i < pfo; ++i) {
            B.dy[i] = (const uint16_t *)dy[i];
            B.db[i] = (float *)db[i];
        }
        B.nb = (int32_t)nb;
        B.bfo = (int32_t)bfo;
        dim3 grid((unsigned)((bfo + 63) / 64), (unsigned)pfo);
        affine_db_kernel<<<grid, kDbThreads, 0, (cudaStream_t)stream>>>(B);
        DISTDL_CUDA_CHECK(cudaGetLastError());
    }
    return DISTDL_OK;
}

}  // namespace distdl

extern "C" distdl_status_t distdl_affine_fwd(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                             const void *const *x, const void *const *w, const void *const *bias,
                                             void *const *y, void *stream) {
    return distdl::affine_impl(nb, nfi, nfo, pfo, pfi, x, w, bias, y, stream, false, "affine_fwd");
}

extern "C" distdl_status_t distdl_affine_adj(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                             const void *const *dy, const void *const *w, void *const *dx,
                                             void *stream) {
    return distdl::affine_impl(nb, nfi, nfo, pfo, pfi, dy, w, nullptr, dx, stream, true, "affine_adj");
}

extern "C" distdl_status_t distdl_affine_adj_params(int64_t nb, int64_t nfi, int64_t nfo, int32_t pfo, int32_t pfi,
                                                    const void *const *dy, const void *const *x, void *const *dw,
                                                    void *const *db, void *stream) {
    return distdl::affine_params_impl(nb, nfi, nfo, pfo, pfi, dy, x, dw, db, stream);
}

namespace distdl {
int conv_take_status();   // conv.cu

// Self-test of the bounded wait: one thread waits, through the same mbar_wait as the kernels above, on a
// barrier that nobody arrives at.  The wait gives up after `limit_cycles`, records DISTDL_ERR_TIMEOUT in the
// status word and the kernel returns by itself.
__global__ void selftest_wait_kernel(long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
        mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_cycles);
    }
}
}

extern "C" distdl_status_t distdl_selftest_wait_timeout(int64_t limit_cycles, void *stream) {
    using namespace distdl;
    clear_error();
    // the limit of the self-test stays short: at most about a tenth of a second of SM clock cycles
    if (limit_cycles < 1 || limit_cycles > 200000000ll)
        return fail(DISTDL_ERR_INVALID_ARG, "selftest_wait_timeout: limit outside 1 .. 2e8 cycles");
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles);
    DISTDL_CUDA_CHECK(cudaGetLastError());
    return DISTDL_OK;
}

extern "C" distdl_status_t distdl_device_status(void *stream) {
    using namespace distdl;
    clear_error();
    DISTDL_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
    int st = 0;
    DISTDL_CUDA_CHECK(cudaMemcpyFromSymbol(&st, g_affine_status, sizeof(int)));
    if (st != 0) {
        const int zero = 0;
        DISTDL_CUDA_CHECK(cudaMemcpyToSymbol(g_affine_status, &zero, sizeof(int)));
    }
    const int cst = conv_take_status();
    if (cst < 0) return fail(DISTDL_ERR_CUDA, "device_status: reading the status word failed");
    if (st != 0 || cst != 0)
        return fail(DISTDL_ERR_TIMEOUT, "a bounded device-side wait of %s kernel ran out",
                    st != 0 ? "an affine" : "a convolution");
    return DISTDL_OK;
}
