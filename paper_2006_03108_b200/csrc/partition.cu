// Partition object of the C ABI: creation, queries, upload of the halo plan tables.
#include <cstring>
#include <new>

#include "common.h"

using namespace distdl;

distdl_status_t distdl::upload_plan_pair(const HaloPlanHost &a, const HaloPlanHost &b, HaloPlanDevice *da, HaloPlanDevice *db,
                                 void **block, int *device, const char *what, const void *extra, size_t extra_bytes,
                                 void **extra_dev) {
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) {
        cudaGetLastError();
        return DISTDL_OK;      // host-only object
    }
    cudaGetDevice(device);
    auto bytes_of = [](const HaloPlanHost &h, size_t *bz, size_t *sz, size_t *tz) {
        auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
        *bz = up(h.boxes.size() * sizeof(HaloBox));
        *sz = up(h.sources.size() * sizeof(HaloSource));
        *tz = up(h.tiles.size() * sizeof(HaloTile));
    };
    size_t fbz, fsz, ftz, abz, asz, atz;
    bytes_of(a, &fbz, &fsz, &ftz);
    bytes_of(b, &abz, &asz, &atz);
    const size_t ebz = (extra_bytes + 255) & ~(size_t)255;
    const size_t total = fbz + fsz + ftz + abz + asz + atz + ebz + 256;
    cudaError_t e = cudaMalloc(block, total);
    if (e != cudaSuccess) {
        *block = nullptr;
        return fail(DISTDL_ERR_NOMEM, "%s: cudaMalloc(%zu) failed: %s", what, total, cudaGetErrorString(e));
    }
    char *at = (char *)*block;
    auto put = [&](const void *src, size_t n, size_t reserved) -> void * {
        void *dst = at;
        if (n && e == cudaSuccess) e = cudaMemcpy(dst, src, n, cudaMemcpyHostToDevice);
        at += reserved;
        return dst;
    };
    da->boxes = (HaloBox *)put(a.boxes.data(), a.boxes.size() * sizeof(HaloBox), fbz);
    da->sources = (HaloSource *)put(a.sources.data(), a.sources.size() * sizeof(HaloSource), fsz);
    da->tiles = (HaloTile *)put(a.tiles.data(), a.tiles.size() * sizeof(HaloTile), ftz);
    da->num_tiles = (int32_t)a.tiles.size();
    db->boxes = (HaloBox *)put(b.boxes.data(), b.boxes.size() * sizeof(HaloBox), abz);
    db->sources = (HaloSource *)put(b.sources.data(), b.sources.size() * sizeof(HaloSource), asz);
    db->tiles = (HaloTile *)put(b.tiles.data(), b.tiles.size() * sizeof(HaloTile), atz);
    db->num_tiles = (int32_t)b.tiles.size();
    if (extra_dev) *extra_dev = extra_bytes ? put(extra, extra_bytes, ebz) : nullptr;
    if (e != cudaSuccess) {
        cudaFree(*block);
        *block = nullptr;
        return fail(DISTDL_ERR_CUDA, "%s: upload failed: %s", what, cudaGetErrorString(e));
    }
    return DISTDL_OK;
}

static distdl_status_t create_impl(int32_t rank, const int64_t *global_shape, const int32_t *partition_shape,
                                   const int32_t *const *hlo, const int32_t *const *hhi,
                                   const int32_t *ulo, const int32_t *uhi, distdl_dtype_t dtype,
                                   distdl_partition_t **out, bool upload = true, const int32_t *periodic = nullptr) {
    clear_error();
    if (!out) return fail(DISTDL_ERR_INVALID_ARG, "partition_create: out is NULL");
    if (rank < 1 || rank > DISTDL_MAX_RANK)
        return fail(DISTDL_ERR_INVALID_ARG, "partition_create: rank %d outside 1..%d", rank, DISTDL_MAX_RANK);
    if (!global_shape || !partition_shape) return fail(DISTDL_ERR_INVALID_ARG, "partition_create: NULL shape");
    if (!valid_dtype(dtype)) return fail(DISTDL_ERR_INVALID_ARG, "partition_create: bad dtype");
    int64_t workers = 1;
    for (int k = 0; k < rank; ++k) {
        if (partition_shape[k] < 1) return fail(DISTDL_ERR_SHAPE, "partition_create: partition_shape[%d] < 1", k);
        if (global_shape[k] < partition_shape[k])
            return fail(DISTDL_ERR_SHAPE, "partition_create: global_shape[%d] smaller than the worker count", k);
        workers *= partition_shape[k];
        if (workers > DISTDL_MAX_WORKERS)
            return fail(DISTDL_ERR_UNSUPPORTED, "partition_create: more than %d workers", DISTDL_MAX_WORKERS);
    }
    distdl_partition *p = new (std::nothrow) distdl_partition();
    if (!p) return fail(DISTDL_ERR_NOMEM, "partition_create: out of host memory");
    p->rank = rank;
    p->dtype = dtype;
    p->num_workers = (int32_t)workers;
    for (int k = 0; k < rank; ++k) {
        p->global_shape[k] = global_shape[k];
        p->pshape[k] = partition_shape[k];
        p->periodic[k] = periodic && periodic[k] != 0;
        const int32_t pk = partition_shape[k];
        const int64_t q = global_shape[k] / pk, r = global_shape[k] % pk;
        int64_t at = 0;
        for (int32_t c = 0; c < pk; ++c) {
            const int64_t sz = q + (c < r ? 1 : 0);   // first r workers get one more
            p->start[k].push_back(at);
            p->size[k].push_back(sz);
            at += sz;
            const int32_t lo = hlo ? (hlo[k] ? hlo[k][c] : 0) : (ulo ? ulo[k] : 0);
            const int32_t hi = hhi ? (hhi[k] ? hhi[k][c] : 0) : (uhi ? uhi[k] : 0);
            if (lo < 0 || hi < 0) {
                delete p;
                return fail(DISTDL_ERR_SHAPE, "partition_create: negative halo width in dimension %d", k);
            }
            p->hlo[k].push_back(lo);
            p->hhi[k].push_back(hi);
        }
        // a ghost may only hold cells of the directly adjacent worker (around the seam too, when the
        // dimension is periodic)
        if (p->periodic[k] && (p->hlo[k][0] > p->size[k][pk - 1] || p->hhi[k][pk - 1] > p->size[k][0])) {
            delete p;
            return fail(DISTDL_ERR_SHAPE, "partition_create: a halo across the periodic seam of dimension %d is wider than its neighbour's bulk", k);
        }
        for (int32_t c = 0; c < pk; ++c) {
            if (c > 0 && p->hlo[k][c] > p->size[k][c - 1]) {
                delete p;
                return fail(DISTDL_ERR_SHAPE, "partition_create: low halo of worker coordinate %d in dimension %d is wider than its neighbour's bulk", c, k);
            }
            if (c + 1 < pk && p->hhi[k][c] > p->size[k][c + 1]) {
                delete p;
                return fail(DISTDL_ERR_SHAPE, "partition_create: high halo of worker coordinate %d in dimension %d is wider than its neighbour's bulk", c, k);
            }
        }
    }
    for (int32_t w = 0; w < p->num_workers; ++w)
        if (p->shard_elems(w) >= (int64_t)1 << 31) {
            delete p;
            return fail(DISTDL_ERR_UNSUPPORTED, "partition_create: shard too large");
        }
    if (upload) build_fast_plan(p);
    distdl_status_t st = build_halo_plans(p, !upload);      // without an upload (the entry point that allocates nothing) only H is planned
    if (st != DISTDL_OK) {
        delete p;
        return st;
    }
    // Upload.  Without a CUDA device the object stays host-only: geometry queries work, operator
    // calls report DISTDL_ERR_CUDA.
    if (upload) {
        // one more blob behind the two box plans: the row plan's records and the box plan of the rest of H*
        std::vector<unsigned char> blob;
        size_t at_boxes = 0, at_sources = 0, at_tiles = 0;
        auto append = [&blob](const void *src, size_t n) {
            const size_t at = blob.size();
            blob.resize(at + ((n + 255) & ~(size_t)255));
            if (n) memcpy(blob.data() + at, src, n);
            return at;
        };
        if (p->fast.usable) {
            append(p->fast.dims.data(), p->fast.dims.size() * sizeof(FastDim));
            const HaloPlanHost &r = p->adj_rest_host;
            at_boxes = append(r.boxes.data(), r.boxes.size() * sizeof(HaloBox));
            at_sources = append(r.sources.data(), r.sources.size() * sizeof(HaloSource));
            at_tiles = append(r.tiles.data(), r.tiles.size() * sizeof(HaloTile));
        }
        void *blob_dev = nullptr;
        st = upload_plan_pair(p->fwd_host, p->adj_host, &p->fwd_dev, &p->adj_dev, &p->device_block, &p->device,
                              "partition_create", blob.data(), blob.size(), &blob_dev);
        if (st == DISTDL_OK && blob_dev) {
            unsigned char *base = static_cast<unsigned char *>(blob_dev);
            p->fast_dims_dev = reinterpret_cast<FastDim *>(base);
            p->adj_rest_dev.boxes = reinterpret_cast<HaloBox *>(base + at_boxes);
            p->adj_rest_dev.sources = reinterpret_cast<HaloSource *>(base + at_sources);
            p->adj_rest_dev.tiles = reinterpret_cast<HaloTile *>(base + at_tiles);
            p->adj_rest_dev.num_tiles = (int32_t)p->adj_rest_host.tiles.size();
        }
        if (st != DISTDL_OK) {
            delete p;
            return st;
        }
    }
    *out = p;
    return DISTDL_OK;
}

extern "C" distdl_status_t distdl_partition_create(int32_t rank, const int64_t *global_shape,
                                                   const int32_t *partition_shape, const int32_t *halo_lo,
                                                   const int32_t *halo_hi, distdl_dtype_t dtype,
                                                   distdl_partition_t **out) {
    return create_impl(rank, global_shape, partition_shape, nullptr, nullptr, halo_lo, halo_hi, dtype, out);
}

extern "C" distdl_status_t distdl_partition_create_general(int32_t rank, const int64_t *global_shape,
                                                           const int32_t *partition_shape,
                                                           const int32_t *const *halo_lo,
                                                           const int32_t *const *halo_hi, distdl_dtype_t dtype,
                                                           distdl_partition_t **out) {
    static const int32_t *const none[DISTDL_MAX_RANK] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    return create_impl(rank, global_shape, partition_shape, halo_lo ? halo_lo : none, halo_hi ? halo_hi : none,
                       nullptr, nullptr, dtype, out);
}

extern "C" distdl_status_t distdl_partition_create_periodic(int32_t rank, const int64_t *global_shape,
                                                            const int32_t *partition_shape, const int32_t *halo_lo,
                                                            const int32_t *halo_hi, const int32_t *periodic,
                                                            distdl_dtype_t dtype, distdl_partition_t **out) {
    return create_impl(rank, global_shape, partition_shape, nullptr, nullptr, halo_lo, halo_hi, dtype, out, true, periodic);
}

namespace distdl {
// Geometry and halo plans only, no device memory (used by the entry point that must not allocate).
distdl_status_t partition_create_host_only(int32_t rank, const int64_t *global_shape, const int32_t *partition_shape,
                                           const int32_t *halo_lo, const int32_t *halo_hi, distdl_dtype_t dtype,
                                           distdl_partition_t **out) {
    return create_impl(rank, global_shape, partition_shape, nullptr, nullptr, halo_lo, halo_hi, dtype, out, false);
}
}  // namespace distdl

extern "C" void distdl_partition_destroy(distdl_partition_t *p) {
    if (!p) return;
    if (p->device_block) cudaFree(p->device_block);
    delete p;
}

extern "C" int32_t distdl_partition_num_workers(const distdl_partition_t *p) { return p ? p->num_workers : -1; }

extern "C" distdl_status_t distdl_partition_shard_extents(const distdl_partition_t *p, int32_t worker,
                                                          int64_t *bulk_start, int64_t *bulk_shape,
                                                          int64_t *padded_shape, int32_t *halo_lo,
                                                          int32_t *halo_hi) {
    clear_error();
    if (!p) return fail(DISTDL_ERR_INVALID_ARG, "shard_extents: partition is NULL");
    if (worker < 0 || worker >= p->num_workers)
        return fail(DISTDL_ERR_INVALID_ARG, "shard_extents: worker %d outside 0..%d", worker, p->num_workers - 1);
    int32_t c[DISTDL_MAX_RANK];
    p->coords(worker, c);
    for (int k = 0; k < p->rank; ++k) {
        if (bulk_start) bulk_start[k] = p->start[k][c[k]];
        if (bulk_shape) bulk_shape[k] = p->size[k][c[k]];
        if (padded_shape) padded_shape[k] = p->padded_extent(k, c[k]);
        if (halo_lo) halo_lo[k] = p->hlo[k][c[k]];
        if (halo_hi) halo_hi[k] = p->hhi[k][c[k]];
    }
    return DISTDL_OK;
}

// Plan statistics (host): number of boxes and tiles and the algorithmic bytes of one H or H*.
extern "C" distdl_status_t distdl_partition_halo_stats(const distdl_partition_t *p, int32_t adjoint,
                                                       int64_t *boxes, int64_t *tiles, int64_t *bytes) {
    clear_error();
    if (!p) return fail(DISTDL_ERR_INVALID_ARG, "halo_stats: partition is NULL");
    const HaloPlanHost &h = adjoint ? p->adj_host : p->fwd_host;
    if (boxes) *boxes = (int64_t)h.boxes.size();
    if (tiles) *tiles = (int64_t)h.tiles.size();
    if (bytes) *bytes = h.algorithmic_bytes;
    return DISTDL_OK;
}

// Copies the row plan (header and per-coordinate records, as 32-bit words) to the caller: lets a host-side
// test replay the kernels' index arithmetic.
extern "C" distdl_status_t distdl_selftest_row_plan(const distdl_partition_t *p, int32_t adjoint, int32_t *header,
                                                    int32_t header_words, int32_t *records, int32_t record_words,
                                                    int32_t *num_records) {
    clear_error();
    if (!p || !header || !records || !num_records) return fail(DISTDL_ERR_INVALID_ARG, "selftest_row_plan: NULL argument");
    if (adjoint ? !p->fast.adj_usable : !p->fast.usable)
        return fail(DISTDL_ERR_UNSUPPORTED, "selftest_row_plan: this partition has no row plan for %s", adjoint ? "the row ends of H*" : "H");
    const size_t hw = sizeof(FastHeader) / 4, rw = p->fast.dims.size() * (sizeof(FastDim) / 4);
    if ((size_t)header_words < hw || (size_t)record_words < rw)
        return fail(DISTDL_ERR_INVALID_ARG, "selftest_row_plan: need %zu header words and %zu record words", hw, rw);
    memcpy(header, adjoint ? &p->fast.adj_hdr : &p->fast.hdr, hw * 4);
    memcpy(records, p->fast.dims.data(), rw * 4);
    *num_records = (int32_t)p->fast.dims.size();
    return DISTDL_OK;
}

extern "C" int32_t distdl_partition_uses_row_plan(const distdl_partition_t *p, int32_t adjoint) {
    return p ? ((adjoint ? p->fast.adj_usable : p->fast.usable) ? 1 : 0) : -1;
}

// ---------------------------------------------------------------------------------------------
// Generalized all-to-all
// ---------------------------------------------------------------------------------------------
extern "C" distdl_status_t distdl_repartition_create(int32_t rank, const int64_t *global_shape,
                                                     const int32_t *src_partition_shape,
                                                     const int32_t *dst_partition_shape, distdl_dtype_t dtype,
                                                     distdl_repartition_t **out) {
    clear_error();
    if (!global_shape || !src_partition_shape || !dst_partition_shape || !out)
        return fail(DISTDL_ERR_INVALID_ARG, "repartition_create: NULL argument");
    if (rank < 1 || rank > DISTDL_MAX_RANK) return fail(DISTDL_ERR_INVALID_ARG, "repartition_create: rank %d", rank);
    if (!valid_dtype(dtype)) return fail(DISTDL_ERR_INVALID_ARG, "repartition_create: bad dtype");
    distdl_repartition *r = new distdl_repartition();
    r->rank = rank;
    r->dtype = dtype;
    int64_t ns = 1, nd = 1;
    for (int k = 0; k < rank; ++k) {
        if (global_shape[k] < 1 || src_partition_shape[k] < 1 || dst_partition_shape[k] < 1 ||
            src_partition_shape[k] > global_shape[k] || dst_partition_shape[k] > global_shape[k]) {
            delete r;
            return fail(DISTDL_ERR_SHAPE, "repartition_create: dimension %d: extent %lld, workers %d -> %d", k,
                        (long long)global_shape[k], src_partition_shape[k], dst_partition_shape[k]);
        }
        r->global_shape[k] = global_shape[k];
        r->src_pshape[k] = src_partition_shape[k];
        r->dst_pshape[k] = dst_partition_shape[k];
        ns *= src_partition_shape[k];
        nd *= dst_partition_shape[k];
        split_evenly(global_shape[k], src_partition_shape[k], r->src_start[k], r->src_size[k]);
        split_evenly(global_shape[k], dst_partition_shape[k], r->dst_start[k], r->dst_size[k]);
    }
    if (ns + nd > DISTDL_MAX_WORKERS) {
        delete r;
        return fail(DISTDL_ERR_UNSUPPORTED, "repartition_create: %lld + %lld workers (at most %d together)", (long long)ns,
                    (long long)nd, DISTDL_MAX_WORKERS);
    }
    r->num_src = (int32_t)ns;
    r->num_dst = (int32_t)nd;
    auto elems = [&](const int32_t *pshape, const std::vector<int64_t> *size, int32_t w) {
        int64_t n = 1;
        for (int k = rank - 1; k >= 0; --k) {
            n *= size[k][w % pshape[k]];
            w /= pshape[k];
        }
        return n;
    };
    for (int32_t w = 0; w < r->num_src; ++w) r->shard_elems.push_back(elems(r->src_pshape, r->src_size, w));
    for (int32_t w = 0; w < r->num_dst; ++w) r->shard_elems.push_back(elems(r->dst_pshape, r->dst_size, w));
    for (int64_t n : r->shard_elems)
        if (n >= (int64_t)1 << 31) {
            delete r;
            return fail(DISTDL_ERR_UNSUPPORTED, "repartition_create: shard too large");
        }
    distdl_status_t st = build_repartition_plans(r);
    if (st == DISTDL_OK)
        st = upload_plan_pair(r->fwd_host, r->adj_host, &r->fwd_dev, &r->adj_dev, &r->device_block, &r->device,
                              "repartition_create");
    if (st != DISTDL_OK) {
        delete r;
        return st;
    }
    *out = r;
    return DISTDL_OK;
}

extern "C" void distdl_repartition_destroy(distdl_repartition_t *r) {
    if (!r) return;
    if (r->device_block) cudaFree(r->device_block);
    delete r;
}

extern "C" distdl_status_t distdl_repartition_shard_shape(const distdl_repartition_t *r, int32_t destination, int32_t worker,
                                                          int64_t *shape) {
    clear_error();
    if (!r || !shape) return fail(DISTDL_ERR_INVALID_ARG, "repartition_shard_shape: NULL argument");
    const int32_t *pshape = destination ? r->dst_pshape : r->src_pshape;
    const std::vector<int64_t> *size = destination ? r->dst_size : r->src_size;
    if (worker < 0 || worker >= (destination ? r->num_dst : r->num_src))
        return fail(DISTDL_ERR_INVALID_ARG, "repartition_shard_shape: worker %d", worker);
    for (int k = r->rank - 1; k >= 0; --k) {
        shape[k] = size[k][worker % pshape[k]];
        worker /= pshape[k];
    }
    return DISTDL_OK;
}
