// Shared host-side helpers of the library: error reporting and the partition object.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <string>
#include <vector>

#include "distdl.h"

namespace distdl {

// Records a thread-local message and returns `code`.
distdl_status_t fail(distdl_status_t code, const char *fmt, ...);
void clear_error();

#define DISTDL_CUDA_CHECK(expr)                                                          \
    do {                                                                                 \
        cudaError_t e__ = (expr);                                                        \
        if (e__ != cudaSuccess)                                                          \
            return ::distdl::fail(DISTDL_ERR_CUDA, "%s failed: %s", #expr,               \
                                  cudaGetErrorString(e__));                              \
    } while (0)

constexpr int kMaxDevicesPerProcess = 64;   // per-device one-time set-up flags are kept for this many devices
std::mutex &setup_mutex();                  // guards the one-time, per-device set-up of the operator entry points

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int elem_size(distdl_dtype_t t) { return t == DISTDL_F32 ? 4 : (t == DISTDL_F64 ? 8 : 2); }
inline bool valid_dtype(distdl_dtype_t t) { return t == DISTDL_F32 || t == DISTDL_BF16 || t == DISTDL_F64; }

// ---------------------------------------------------------------------------------------------
// Device-side plan tables of the halo kernels.
//
// A *box* is a rectangular set of cells of one destination shard together with the list of
// source boxes (same shape, possibly in other shards) whose values are combined into it.
// A box with no source is cleared; a box with one source is a copy; a box with several sources
// is the nested sum of H*.  A *tile* is a contiguous range of a box's flattened index space;
// one thread block processes one tile.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxBoxDims = DISTDL_MAX_RANK;
constexpr int kMaxLevels = DISTDL_MAX_RANK;   // nesting depth of the H* sum
constexpr int kMaxSources = 32;               // sources of one box (2^5, or 3^3 for thin shards)

// Offsets and strides are in *units* (16-byte vectors when `vec`, elements otherwise) and fit in
// 32 bits (a shard holds fewer than 2^31 elements).
struct HaloSource {
    int32_t shard;                 // shard the source cells live in
    int32_t close;                 // how many nesting levels are folded after adding this source
    int32_t clear_after;           // 1: source cells are set to zero once read (ghost sources)
    uint32_t offset;               // unit offset of the box origin inside the shard
    uint32_t stride[kMaxBoxDims];  // unit stride per box dimension (innermost last)
    uint32_t pad_[3];
};
static_assert(sizeof(HaloSource) == 48, "HaloSource layout");

struct HaloBox {
    int32_t dst_shard;
    int32_t ndim;                  // box dimensions kept after dropping extent-1 dimensions
    int32_t vec;                   // 1: every offset, stride and extent allows 16-byte accesses
    int32_t levels;                // nesting levels of the sum (>= 1)
    int32_t balanced;              // 1: every nesting level has exactly two terms (nsrc = 2^levels)
    uint32_t dst_offset;
    uint32_t shape[kMaxBoxDims];   // extents in units
    uint32_t magic[kMaxBoxDims];   // n / shape[k] == umulhi(n, magic[k]) >> shift[k] for n < 2^31
    uint32_t shift[kMaxBoxDims];
    uint32_t dst_stride[kMaxBoxDims];
    uint32_t pad_[6];
};
static_assert(sizeof(HaloBox) == 128, "HaloBox layout");

struct HaloTile {
    int32_t box;
    int32_t src_begin;             // index of the box's first source in the source table
    int32_t nsrc;                  // 0: clear, 1: copy, more: nested sum
    uint32_t first;                // first flattened unit of the tile
    uint32_t count;                // units in the tile
    uint32_t pad_[3];
};
static_assert(sizeof(HaloTile) == 32, "HaloTile layout");

struct HaloPlanHost {
    std::vector<HaloBox> boxes;
    std::vector<HaloSource> sources;
    std::vector<HaloTile> tiles;
    int64_t algorithmic_bytes = 0; // bytes read + written by the in-place method
};

struct HaloPlanDevice {
    HaloBox *boxes = nullptr;
    HaloSource *sources = nullptr;
    HaloTile *tiles = nullptr;
    int32_t num_tiles = 0;
};

// ---------------------------------------------------------------------------------------------
// Row plan of the halo kernels: used when every ghost width and bulk extent of the innermost
// dimension is a whole number of 16-byte units, so that all ghost cells can be moved as aligned
// vectors.  The geometry of a Cartesian partition is separable: where a ghost cell's value lives
// follows, dimension by dimension, from the worker's coordinate along that dimension alone.  The
// plan is therefore one small record per (dimension, worker coordinate); the kernels derive
// everything else (which rows are ghost rows, their source rows in the neighbours) from it.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxFastCoords = 64;    // sum over the dimensions of the workers along each

struct FastDim {
    int32_t n, hlo, b;                // padded extent, low ghost width, bulk extent (innermost dimension: in units)
    int32_t lo_c, hi_c;               // coordinate of the low / high neighbour along this dimension, -1: none
    int32_t lo_shift, hi_shift;       // index in that neighbour's padded range minus the own index of the same cell
    int32_t rlo, rhi;                 // bulk cells at the low / high end that the neighbour there holds ghost copies of
    // x / e == umulhi(x, magic) >> shift for x < 2^31 (magic 0: e <= 1, the quotient is x), for the extents
    // e = n, b, g = n - b (ghost cells), bi = b - rlo - rhi (bulk cells out of every neighbour's reach), rr = rlo + rhi
    uint32_t magic_n, magic_b, magic_g, magic_bi, magic_rr;
    uint32_t shifts;                  // shift of n | b << 6 | g << 12 | bi << 18 | rr << 24
    int32_t pad_;
};
static_assert(sizeof(FastDim) == 64, "FastDim layout");

__host__ __device__ inline uint32_t fast_shift_n(const FastDim &f) { return f.shifts & 63u; }
__host__ __device__ inline uint32_t fast_shift_b(const FastDim &f) { return (f.shifts >> 6) & 63u; }
__host__ __device__ inline uint32_t fast_shift_g(const FastDim &f) { return (f.shifts >> 12) & 63u; }
__host__ __device__ inline uint32_t fast_shift_bi(const FastDim &f) { return (f.shifts >> 18) & 63u; }
__host__ __device__ inline uint32_t fast_shift_rr(const FastDim &f) { return (f.shifts >> 24) & 63u; }

// Block counts of one kernel launch: blocks are dealt out in groups holding a fixed number of blocks of each kind.
struct FastHeader {
    int32_t rank;                     // dimensions (the innermost one in 16-byte units)
    int32_t num_workers;
    int32_t pshape[kMaxBoxDims];
    int32_t dim_base[kMaxBoxDims];    // index of (dimension k, coordinate 0) in the record table
    int32_t wstride[kMaxBoxDims];     // worker-id stride of a step along dimension k
    int32_t num_records;
    int32_t num_lines;                // workers / pshape[rank - 1]
    // kind 0: ghost rows, per worker (H only)
    // kind 1: row ends of bulk rows, per line of workers along the innermost dimension (H: all bulk rows; H*: the bulk
    //         rows out of every outer neighbour's reach)
    int32_t rows_per_tile[2];
    int32_t tiles_per_owner[2];       // per worker (kind 0) or per line (kind 1)
    int32_t group[2];                 // blocks of each kind per group
    int32_t num_groups;
};

struct FastPlanHost {
    bool usable = false;              // H runs through the row plan
    bool adj_usable = false;          // the row ends of H* too (needs bulks at least as wide as the two neighbours' reach together)
    FastHeader hdr;                   // H
    FastHeader adj_hdr;               // H*: line blocks only
    std::vector<FastDim> dims;
};

}  // namespace distdl

// The opaque partition object of the C ABI.
struct distdl_partition {
    int32_t rank = 0;
    distdl_dtype_t dtype = DISTDL_F32;
    int32_t num_workers = 0;
    int device = 0;
    int64_t global_shape[DISTDL_MAX_RANK] = {0};
    int32_t pshape[DISTDL_MAX_RANK] = {0};
    bool periodic[DISTDL_MAX_RANK] = {false, false, false, false, false};   // dimension wraps around
    bool any_periodic() const {
        for (int k = 0; k < rank; ++k)
            if (periodic[k]) return true;
        return false;
    }
    // per dimension, per worker coordinate along that dimension
    std::vector<int64_t> start[DISTDL_MAX_RANK];
    std::vector<int64_t> size[DISTDL_MAX_RANK];
    std::vector<int32_t> hlo[DISTDL_MAX_RANK];
    std::vector<int32_t> hhi[DISTDL_MAX_RANK];

    distdl::HaloPlanHost fwd_host, adj_host;
    distdl::HaloPlanDevice fwd_dev, adj_dev;
    // H* without the row ends that the row plan handles (built when fast.adj_usable)
    distdl::HaloPlanHost adj_rest_host;
    distdl::HaloPlanDevice adj_rest_dev;
    distdl::FastPlanHost fast;      // row plan (see FastDim); fast.usable says whether the geometry allows it
    distdl::FastDim *fast_dims_dev = nullptr;
    void *device_block = nullptr;   // one allocation holding all device tables

    void coords(int32_t worker, int32_t *c) const {
        for (int k = rank - 1; k >= 0; --k) {
            c[k] = worker % pshape[k];
            worker /= pshape[k];
        }
    }
    int32_t worker_of(const int32_t *c) const {
        int32_t w = 0;
        for (int k = 0; k < rank; ++k) w = w * pshape[k] + c[k];
        return w;
    }
    int64_t padded_extent(int k, int32_t c) const { return size[k][c] + hlo[k][c] + hhi[k][c]; }
    int64_t shard_elems(int32_t worker) const {
        int32_t c[DISTDL_MAX_RANK];
        coords(worker, c);
        int64_t n = 1;
        for (int k = 0; k < rank; ++k) n *= padded_extent(k, c[k]);
        return n;
    }
};

// The opaque object of the generalized all-to-all: the same tensor under two partitions without ghosts.
struct distdl_repartition {
    int32_t rank = 0;
    distdl_dtype_t dtype = DISTDL_F32;
    int device = 0;
    int64_t global_shape[DISTDL_MAX_RANK] = {0};
    int32_t src_pshape[DISTDL_MAX_RANK] = {0}, dst_pshape[DISTDL_MAX_RANK] = {0};
    int32_t num_src = 0, num_dst = 0;
    std::vector<int64_t> src_start[DISTDL_MAX_RANK], src_size[DISTDL_MAX_RANK];
    std::vector<int64_t> dst_start[DISTDL_MAX_RANK], dst_size[DISTDL_MAX_RANK];
    std::vector<int64_t> shard_elems;      // source workers first, then destination workers
    distdl::HaloPlanHost fwd_host, adj_host;
    distdl::HaloPlanDevice fwd_dev, adj_dev;
    void *device_block = nullptr;
};

namespace distdl {
// Box / tile lists of the all-to-all and of its adjoint (the all-to-all back).
distdl_status_t build_repartition_plans(distdl_repartition *r);
void split_evenly(int64_t n, int32_t p, std::vector<int64_t> &start, std::vector<int64_t> &size);
// One device allocation holding the tables of two plans; host-only when there is no CUDA device
// (*block stays nullptr).  Synchronous copies on the current device.
distdl_status_t upload_plan_pair(const HaloPlanHost &a, const HaloPlanHost &b, HaloPlanDevice *da, HaloPlanDevice *db,
                                 void **block, int *device, const char *what, const void *extra = nullptr,
                                 size_t extra_bytes = 0, void **extra_dev = nullptr);
// Builds the forward (H) and adjoint (H*) box/tile lists of a partition (host only).
distdl_status_t build_halo_plans(distdl_partition *p, bool forward_only = false);
// Fills p->fast (row plan) where the geometry allows it.
void build_fast_plan(distdl_partition *p);
// Geometry and halo plans only, no device memory.
distdl_status_t partition_create_host_only(int32_t rank, const int64_t *global_shape, const int32_t *partition_shape,
                                           const int32_t *halo_lo, const int32_t *halo_hi, distdl_dtype_t dtype,
                                           distdl_partition_t **out);
}  // namespace distdl
