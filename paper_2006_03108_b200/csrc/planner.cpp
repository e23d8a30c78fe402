// Host planner: partition geometry (balanced split, per-side ghost widths) and the box / tile
// lists that the halo kernels execute.  Section 3 "Halo exchange", Section 4 (partition vector),
// Appendix B (worked geometry examples).
#include <algorithm>
#include <array>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "common.h"

namespace distdl {

static thread_local char g_error[512] = "";

distdl_status_t fail(distdl_status_t code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
    return code;
}
void clear_error() { g_error[0] = 0; }

std::mutex &setup_mutex() {
    static std::mutex m;
    return m;
}

}  // namespace distdl

extern "C" const char *distdl_last_error(void) { return distdl::g_error; }

using namespace distdl;

// ---------------------------------------------------------------------------------------------
// Balanced split and 1-D halo widths
// ---------------------------------------------------------------------------------------------
static void balanced_split(int64_t n, int32_t p, std::vector<int64_t> &start, std::vector<int64_t> &size) {
    const int64_t q = n / p, r = n % p;
    start.resize(p);
    size.resize(p);
    int64_t at = 0;
    for (int32_t c = 0; c < p; ++c) {
        size[c] = q + (c < r ? 1 : 0);
        start[c] = at;
        at += size[c];
    }
}

extern "C" distdl_status_t distdl_halo_widths_1d(int64_t n, int32_t p, int32_t kernel, int32_t stride,
                                                 int32_t dilation, int32_t pad_lo, int32_t pad_hi,
                                                 int32_t *halo_lo, int32_t *halo_hi,
                                                 int32_t *unused_lo, int32_t *unused_hi) {
    clear_error();
    if (n < 1 || p < 1 || kernel < 1 || stride < 1 || dilation < 1 || pad_lo < 0 || pad_hi < 0)
        return fail(DISTDL_ERR_INVALID_ARG, "halo_widths_1d: non-positive argument");
    const int64_t reach = (int64_t)dilation * (kernel - 1);
    const int64_t span = n + pad_lo + pad_hi - reach - 1;
    if (span < 0) return fail(DISTDL_ERR_SHAPE, "halo_widths_1d: kernel larger than padded input");
    const int64_t m = span / stride + 1;
    std::vector<int64_t> is, iz, os, oz;
    balanced_split(n, p, is, iz);
    balanced_split(m, p, os, oz);
    for (int32_t c = 0; c < p; ++c) {
        const int64_t own_first = is[c], own_last = is[c] + iz[c] - 1;
        int64_t need_first = own_first, need_last = own_first - 1;   // empty range if no outputs
        if (oz[c] > 0) {
            need_first = os[c] * stride - pad_lo;
            need_last = (os[c] + oz[c] - 1) * stride - pad_lo + reach;
        }
        const int64_t hl = std::max<int64_t>(0, own_first - need_first);
        const int64_t hh = std::max<int64_t>(0, need_last - own_last);
        const int64_t ul = std::max<int64_t>(0, std::min(need_first, own_last + 1) - own_first);
        const int64_t uh = std::max<int64_t>(0, own_last - std::max(need_last, own_first - 1));
        if (halo_lo) halo_lo[c] = (int32_t)hl;
        if (halo_hi) halo_hi[c] = (int32_t)hh;
        if (unused_lo) unused_lo[c] = (int32_t)ul;
        if (unused_hi) unused_hi[c] = (int32_t)uh;
    }
    return DISTDL_OK;
}

// ---------------------------------------------------------------------------------------------
// Box construction
// ---------------------------------------------------------------------------------------------
namespace {

struct Region {             // a rectangular set of cells of one shard, in padded-local indices
    int32_t shard;
    int64_t start[DISTDL_MAX_RANK];
    int64_t extent[DISTDL_MAX_RANK];
};

struct PendingSource {
    Region r;
    int32_t close;
    int32_t clear_after;
};

constexpr uint32_t kTileUnits = 4096;

struct Builder {
    HaloPlanHost *plan;
    int esize;
    int rank;
    std::vector<std::array<int64_t, DISTDL_MAX_RANK>> shard_shape;   // extents of every shard's array
    std::vector<Region> dst_regions;                                   // for the disjointness check

    Builder(const distdl_partition *p, HaloPlanHost *plan_, int esize_) : plan(plan_), esize(esize_), rank(p->rank) {
        shard_shape.resize(p->num_workers);
        for (int32_t w = 0; w < p->num_workers; ++w) {
            int32_t c[DISTDL_MAX_RANK];
            p->coords(w, c);
            for (int k = 0; k < rank; ++k) shard_shape[w][k] = p->padded_extent(k, c[k]);
        }
    }
    Builder(int rank_, std::vector<std::array<int64_t, DISTDL_MAX_RANK>> shapes, HaloPlanHost *plan_, int esize_)
        : plan(plan_), esize(esize_), rank(rank_), shard_shape(std::move(shapes)) {}

    void strides_of(int32_t shard, int64_t *stride) const {
        int64_t s = 1;
        for (int k = rank - 1; k >= 0; --k) {
            stride[k] = s;
            s *= shard_shape[shard][k];
        }
    }
    bool inside(const Region &r) const {
        if (r.shard < 0 || r.shard >= (int32_t)shard_shape.size()) return false;
        for (int k = 0; k < rank; ++k)
            if (r.start[k] < 0 || r.extent[k] < 0 || r.start[k] + r.extent[k] > shard_shape[r.shard][k]) return false;
        return true;
    }

    // Adds one box; `srcs` may be empty (clear).  Returns false on an internal inconsistency.
    bool add(const Region &dst, const std::vector<PendingSource> &srcs, int levels) {
        const int d = rank;
        int64_t cells = 1;
        for (int k = 0; k < d; ++k) cells *= dst.extent[k];
        if (cells == 0) return true;
        if (!inside(dst)) return false;
        for (const auto &s : srcs) {
            if (!inside(s.r)) return false;
            for (int k = 0; k < d; ++k)
                if (s.r.extent[k] != dst.extent[k]) return false;
        }
        if ((int)srcs.size() > kMaxSources) return false;
        dst_regions.push_back(dst);

        // element offsets and strides, all dimensions
        int64_t dstride[DISTDL_MAX_RANK], doff = 0;
        strides_of(dst.shard, dstride);
        for (int k = 0; k < d; ++k) doff += dst.start[k] * dstride[k];
        std::vector<std::array<int64_t, DISTDL_MAX_RANK>> sstride(srcs.size());
        std::vector<int64_t> soff(srcs.size(), 0);
        for (size_t j = 0; j < srcs.size(); ++j) {
            strides_of(srcs[j].r.shard, sstride[j].data());
            for (int k = 0; k < d; ++k) soff[j] += srcs[j].r.start[k] * sstride[j][k];
        }
        // drop extent-1 dimensions, merge dimensions that are contiguous everywhere
        std::vector<int> keep;
        for (int k = 0; k < d; ++k)
            if (dst.extent[k] != 1) keep.push_back(k);
        if (keep.empty()) keep.push_back(d - 1);
        std::vector<int64_t> shape;
        std::vector<int64_t> ds;
        std::vector<std::vector<int64_t>> ss(srcs.size());
        for (int k : keep) {
            bool merged = false;
            if (!shape.empty()) {
                // previous kept dim (outer) merges with this one if outer stride == extent*stride
                bool ok = ds.back() == dst.extent[k] * dstride[k];
                for (size_t j = 0; j < srcs.size() && ok; ++j)
                    ok = ss[j].back() == dst.extent[k] * sstride[j][k];
                if (ok) {
                    shape.back() *= dst.extent[k];
                    ds.back() = dstride[k];
                    for (size_t j = 0; j < srcs.size(); ++j) ss[j].back() = sstride[j][k];
                    merged = true;
                }
            }
            if (!merged) {
                shape.push_back(dst.extent[k]);
                ds.push_back(dstride[k]);
                for (size_t j = 0; j < srcs.size(); ++j) ss[j].push_back(sstride[j][k]);
            }
        }
        const int nd = (int)shape.size();
        // 16-byte vector path: innermost dimension contiguous, everything a multiple of 16 bytes
        const int64_t per = 16 / esize;
        bool vec = ds[nd - 1] == 1 && shape[nd - 1] % per == 0 && doff % per == 0;
        for (int i = 0; i + 1 < nd && vec; ++i) vec = ds[i] % per == 0;
        for (size_t j = 0; j < srcs.size() && vec; ++j) {
            vec = ss[j][nd - 1] == 1 && soff[j] % per == 0;
            for (int i = 0; i + 1 < nd && vec; ++i) vec = ss[j][i] % per == 0;
        }
        const int64_t unit = vec ? per : 1;
        // to units; a dimension whose extent becomes one unit carries no coordinate and is dropped
        {
            shape[nd - 1] /= unit;
            for (int i = 0; i + 1 < nd; ++i) {
                ds[i] /= unit;
                for (size_t j = 0; j < srcs.size(); ++j) ss[j][i] /= unit;
            }
            doff /= unit;
            for (size_t j = 0; j < srcs.size(); ++j) soff[j] /= unit;
            int o = 0;
            for (int i = 0; i < nd; ++i) {
                if (shape[i] == 1 && !(o == 0 && i == nd - 1)) continue;
                shape[o] = shape[i];
                ds[o] = ds[i];
                for (size_t j = 0; j < srcs.size(); ++j) ss[j][o] = ss[j][i];
                ++o;
            }
            shape.resize(o);
        }
        const int nd_units = (int)shape.size();

        HaloBox b;
        memset(&b, 0, sizeof(b));
        b.dst_shard = dst.shard;
        b.vec = vec ? 1 : 0;
        b.levels = std::max(levels, 1);
        b.balanced = ((int64_t)srcs.size() == ((int64_t)1 << b.levels)) ? 1 : 0;
        b.ndim = nd_units;
        b.dst_offset = (uint32_t)doff;
        int64_t units = 1;
        for (int i = 0; i < nd_units; ++i) {
            const int64_t e = shape[i];
            if (e >= ((int64_t)1 << 31)) return false;
            b.shape[i] = (uint32_t)e;
            b.dst_stride[i] = (uint32_t)ds[i];
            // exact division of any n < 2^31 by e >= 2: q = (n * magic) >> (31 + s) with
            // s = ceil(log2 e), magic = ceil(2^(31+s) / e) < 2^32; evaluated as
            // umulhi(n, magic) >> (s - 1).  (e = 1 only for a one-unit box, never divided by.)
            if (e >= 2) {
                int sft = 0;
                while (((int64_t)1 << sft) < e) ++sft;
                const unsigned __int128 num = (unsigned __int128)1 << (31 + sft);
                b.magic[i] = (uint32_t)((num + (uint64_t)e - 1) / (uint64_t)e);
                b.shift[i] = (uint32_t)(sft - 1);
            }
            units *= e;
        }
        if (units >= ((int64_t)1 << 31)) return false;
        const int32_t src_begin = (int32_t)plan->sources.size();
        for (size_t j = 0; j < srcs.size(); ++j) {
            HaloSource s;
            memset(&s, 0, sizeof(s));
            s.shard = srcs[j].r.shard;
            s.close = srcs[j].close;
            s.clear_after = srcs[j].clear_after;
            s.offset = (uint32_t)soff[j];
            for (int i = 0; i < nd_units; ++i) s.stride[i] = (uint32_t)ss[j][i];
            plan->sources.push_back(s);
        }
        const int32_t box_id = (int32_t)plan->boxes.size();
        plan->boxes.push_back(b);
        for (int64_t at = 0; at < units; at += kTileUnits) {
            HaloTile t;
            memset(&t, 0, sizeof(t));
            t.box = box_id;
            t.src_begin = src_begin;
            t.nsrc = (int32_t)srcs.size();
            t.first = (uint32_t)at;
            t.count = (uint32_t)std::min<int64_t>(kTileUnits, units - at);
            plan->tiles.push_back(t);
        }
        // algorithmic traffic: destination written once; every source read once; cleared sources
        // written once; the destination's own previous value is source 0 of a sum (counted there).
        int64_t bytes = cells * esize;
        for (const auto &s : srcs) bytes += cells * esize * (1 + (s.clear_after ? 1 : 0));
        plan->algorithmic_bytes += bytes;
        return true;
    }

    bool destinations_disjoint() const {
        const int d = rank;
        for (size_t a = 0; a < dst_regions.size(); ++a)
            for (size_t b = a + 1; b < dst_regions.size(); ++b) {
                const Region &x = dst_regions[a], &y = dst_regions[b];
                if (x.shard != y.shard) continue;
                bool overlap = true;
                for (int k = 0; k < d && overlap; ++k)
                    overlap = x.start[k] < y.start[k] + y.extent[k] && y.start[k] < x.start[k] + x.extent[k];
                if (overlap) return false;
            }
        return true;
    }
};

// Iterates over {-1,0,+1}^d in row-major order of (delta + 1).
inline bool next_delta(int *delta, int d) {
    for (int k = d - 1; k >= 0; --k) {
        if (delta[k] < 1) {
            ++delta[k];
            return true;
        }
        delta[k] = -1;
    }
    return false;
}

}  // namespace

namespace distdl {

distdl_status_t build_halo_plans(distdl_partition *p, bool forward_only) {
    const int d = p->rank;
    const int esize = elem_size(p->dtype);

    // ---------------- forward: one box per (shard, direction) ----------------
    Builder fb(p, &p->fwd_host, esize);
    // exterior-ghost clear boxes are shared by the adjoint plan
    Builder ab(p, &p->adj_host, esize);
    // H* without the part that the row plan takes (p->fast.adj_usable): the row ends -- ghost cells and receiving bulk
    // cells along the innermost dimension -- of the bulk rows that no neighbour in an outer dimension reaches
    const bool split_adj = p->fast.adj_usable && !forward_only;
    Builder rb(p, &p->adj_rest_host, esize);
    // reach of the low / high neighbour into the bulk of the workers with coordinate c along dimension k
    auto reach_lo = [&](int k, int32_t c) -> int64_t {
        const int32_t pk = p->pshape[k];
        return (c > 0 || p->periodic[k]) ? p->hhi[k][(c + pk - 1) % pk] : 0;
    };
    auto reach_hi = [&](int k, int32_t c) -> int64_t {
        const int32_t pk = p->pshape[k];
        return (c + 1 < pk || p->periodic[k]) ? p->hlo[k][(c + 1) % pk] : 0;
    };
    for (int32_t w = 0; w < p->num_workers; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        p->coords(w, c);
        int delta[DISTDL_MAX_RANK];
        for (int k = 0; k < d; ++k) delta[k] = -1;
        do {
            bool centre = true, has_neighbour = true;
            for (int k = 0; k < d; ++k) {
                if (delta[k] != 0) centre = false;
                const int32_t nc = c[k] + delta[k];
                if ((nc < 0 || nc >= p->pshape[k]) && !p->periodic[k]) has_neighbour = false;
            }
            if (centre) continue;
            Region dst;
            dst.shard = w;
            int32_t nc[DISTDL_MAX_RANK];
            for (int k = 0; k < d; ++k) {
                const int64_t hl = p->hlo[k][c[k]], b = p->size[k][c[k]], hh = p->hhi[k][c[k]];
                dst.start[k] = delta[k] < 0 ? 0 : (delta[k] == 0 ? hl : hl + b);
                dst.extent[k] = delta[k] < 0 ? hl : (delta[k] == 0 ? b : hh);
                // a periodic dimension wraps around: the neighbour across the seam (the worker itself when
                // it is alone along that dimension)
                nc[k] = (c[k] + delta[k] + p->pshape[k]) % p->pshape[k];
            }
            std::vector<PendingSource> srcs;
            if (has_neighbour) {
                PendingSource s;
                s.r.shard = p->worker_of(nc);
                s.close = 0;
                s.clear_after = 0;
                for (int k = 0; k < d; ++k) {
                    const int64_t nhl = p->hlo[k][nc[k]], nb = p->size[k][nc[k]];
                    s.r.extent[k] = dst.extent[k];
                    // low ghost <- the last cells of the low neighbour's bulk; high ghost <- the
                    // first cells of the high neighbour's bulk; otherwise the same bulk range
                    s.r.start[k] = delta[k] < 0 ? nhl + nb - dst.extent[k] : nhl;
                }
                srcs.push_back(s);
                if (!fb.add(dst, srcs, 1)) return fail(DISTDL_ERR_SHAPE, "halo plan: forward box out of range");
            } else {
                if (!fb.add(dst, srcs, 1)) return fail(DISTDL_ERR_SHAPE, "halo plan: clear box out of range");
                if (forward_only) continue;
                if (!ab.add(dst, srcs, 1)) return fail(DISTDL_ERR_SHAPE, "halo plan: clear box out of range");
                if (split_adj) {
                    bool row_end = delta[d - 1] != 0;
                    for (int k = 0; k + 1 < d; ++k) row_end = row_end && delta[k] == 0;
                    if (!row_end) {
                        if (!rb.add(dst, srcs, 1)) return fail(DISTDL_ERR_SHAPE, "halo plan: clear box out of range");
                    } else {
                        // ghosts at the row ends of the bulk rows: only the rows within some outer neighbour's reach stay
                        // here, as one slab per outer dimension and side (out of reach before it, any bulk index after it)
                        for (int j = 0; j + 1 < d; ++j) {
                            for (int side = 0; side < 2; ++side) {
                                Region r = dst;
                                const int64_t hl = p->hlo[j][c[j]], b = p->size[j][c[j]];
                                const int64_t wl = reach_lo(j, c[j]), wh = reach_hi(j, c[j]);
                                r.start[j] = side == 0 ? hl : hl + b - wh;
                                r.extent[j] = side == 0 ? wl : wh;
                                for (int k = 0; k < j; ++k) {
                                    const int64_t kl = reach_lo(k, c[k]), kh = reach_hi(k, c[k]);
                                    r.start[k] = p->hlo[k][c[k]] + kl;
                                    r.extent[k] = p->size[k][c[k]] - kl - kh;
                                }
                                if (!rb.add(r, srcs, 1)) return fail(DISTDL_ERR_SHAPE, "halo plan: clear box out of range");
                            }
                        }
                    }
                }
            }
        } while (next_delta(delta, d));
    }
    // The forward-only form serves the entry point that builds its plan at every call: the pairwise check of the
    // destination boxes (quadratic in their number) is left to partition_create, which builds the same boxes.
    if (forward_only) return DISTDL_OK;
    if (!fb.destinations_disjoint()) return fail(DISTDL_ERR_SHAPE, "halo plan: forward boxes overlap");

    // ---------------- adjoint: receiving bulk boxes with their nested sources ----------------
    for (int32_t w = 0; w < p->num_workers; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        p->coords(w, c);
        // per dimension: up to three segments of the bulk with (from_lo, from_hi) flags
        struct Seg { int64_t s0, s1; bool from_lo, from_hi; };
        std::vector<Seg> segs[DISTDL_MAX_RANK];
        for (int k = 0; k < d; ++k) {
            const int64_t b = p->size[k][c[k]];
            const int32_t pk = p->pshape[k];
            const bool has_lo = c[k] > 0 || p->periodic[k], has_hi = c[k] + 1 < pk || p->periodic[k];
            const int64_t wl = has_lo ? p->hhi[k][(c[k] + pk - 1) % pk] : 0;   // low neighbour's high ghost
            const int64_t wh = has_hi ? p->hlo[k][(c[k] + 1) % pk] : 0;        // high neighbour's low ghost
            int64_t cuts[4] = {0, wl, b - wh, b};
            std::sort(cuts, cuts + 4);
            for (int i = 0; i < 3; ++i) {
                if (cuts[i] == cuts[i + 1]) continue;
                Seg s{cuts[i], cuts[i + 1], cuts[i] < wl, cuts[i] >= b - wh};
                segs[k].push_back(s);
            }
        }
        std::vector<size_t> pick(d, 0);
        while (true) {
            bool any = false;
            for (int k = 0; k < d; ++k) any = any || segs[k][pick[k]].from_lo || segs[k][pick[k]].from_hi;
            if (any) {
                Region dst;
                dst.shard = w;
                std::vector<int> options[DISTDL_MAX_RANK];
                std::vector<int> active;   // dimensions with more than one option, outermost first
                for (int k = 0; k < d; ++k) {
                    const Seg &s = segs[k][pick[k]];
                    dst.start[k] = p->hlo[k][c[k]] + s.s0;
                    dst.extent[k] = s.s1 - s.s0;
                    options[k].push_back(0);
                    if (s.from_lo) options[k].push_back(-1);   // low neighbour first,
                    if (s.from_hi) options[k].push_back(+1);   // then high
                    if (options[k].size() > 1) active.push_back(k);
                }
                const int levels = (int)active.size();
                std::vector<PendingSource> srcs;
                std::vector<size_t> o(d, 0);
                while (true) {
                    PendingSource s;
                    int32_t nc[DISTDL_MAX_RANK];
                    bool self = true;
                    for (int k = 0; k < d; ++k) {
                        nc[k] = (c[k] + options[k][o[k]] + p->pshape[k]) % p->pshape[k];   // wraps in a periodic dimension
                        if (options[k][o[k]] != 0) self = false;
                    }
                    s.r.shard = p->worker_of(nc);
                    s.clear_after = self ? 0 : 1;
                    for (int k = 0; k < d; ++k) {
                        // the same cell in the neighbour's padded-local index: offset s0 of this bulk is the
                        // low neighbour's high ghost cell s0 (right after its bulk), or lies b - s0 cells
                        // before the start of the high neighbour's bulk
                        const int64_t s0 = segs[k][pick[k]].s0, b = p->size[k][c[k]];
                        const int opt = options[k][o[k]];
                        s.r.start[k] = opt == 0 ? p->hlo[k][c[k]] + s0
                                     : opt < 0 ? p->hlo[k][nc[k]] + p->size[k][nc[k]] + s0
                                               : p->hlo[k][nc[k]] - (b - s0);
                        s.r.extent[k] = dst.extent[k];
                    }
                    // levels folded after this term: trailing active dimensions at their last option
                    int close = 0;
                    for (int i = levels - 1; i >= 1; --i) {
                        const int k = active[i];
                        if (o[k] + 1 == options[k].size()) ++close; else break;
                    }
                    s.close = close;
                    srcs.push_back(s);
                    int k = d - 1;
                    for (; k >= 0; --k) {
                        if (o[k] + 1 < options[k].size()) { ++o[k]; break; }
                        o[k] = 0;
                    }
                    if (k < 0) break;
                }
                if ((int)srcs.size() > kMaxSources)
                    return fail(DISTDL_ERR_UNSUPPORTED, "halo plan: a bulk cell receives from more than %d ghosts", kMaxSources);
                if (!ab.add(dst, srcs, levels)) return fail(DISTDL_ERR_SHAPE, "halo plan: adjoint box out of range");
                // the row plan takes the boxes that receive along the innermost dimension only
                const bool row_end_only = levels == 1 && active[0] == d - 1;
                if (split_adj && !row_end_only && !rb.add(dst, srcs, levels))
                    return fail(DISTDL_ERR_SHAPE, "halo plan: adjoint box out of range");
            }
            int k = d - 1;
            for (; k >= 0; --k) {
                if (pick[k] + 1 < segs[k].size()) { ++pick[k]; break; }
                pick[k] = 0;
            }
            if (k < 0) break;
        }
    }
    if (!ab.destinations_disjoint()) return fail(DISTDL_ERR_SHAPE, "halo plan: adjoint boxes overlap");
    if (split_adj && !rb.destinations_disjoint()) return fail(DISTDL_ERR_SHAPE, "halo plan: adjoint boxes overlap");
    return DISTDL_OK;
}

// ---------------------------------------------------------------------------------------------
// Generalized all-to-all: one copy box per pair (destination worker, source worker) whose blocks of
// the tensor intersect.  Shards are numbered source workers first, then destination workers; the
// adjoint plan is the same list with the roles of the two regions exchanged.
// ---------------------------------------------------------------------------------------------
distdl_status_t build_repartition_plans(distdl_repartition *r) {
    const int d = r->rank;
    const int esize = elem_size(r->dtype);
    const int32_t ns = r->num_src, nd = r->num_dst;
    std::vector<std::array<int64_t, DISTDL_MAX_RANK>> shapes(ns + nd);
    auto coords = [&](const int32_t *pshape, int32_t w, int32_t *c) {
        for (int k = d - 1; k >= 0; --k) {
            c[k] = w % pshape[k];
            w /= pshape[k];
        }
    };
    for (int32_t w = 0; w < ns; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        coords(r->src_pshape, w, c);
        for (int k = 0; k < d; ++k) shapes[w][k] = r->src_size[k][c[k]];
    }
    for (int32_t w = 0; w < nd; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        coords(r->dst_pshape, w, c);
        for (int k = 0; k < d; ++k) shapes[ns + w][k] = r->dst_size[k][c[k]];
    }
    Builder fb(d, shapes, &r->fwd_host, esize), ab(d, shapes, &r->adj_host, esize);
    for (int32_t wd = 0; wd < nd; ++wd) {
        int32_t cd[DISTDL_MAX_RANK];
        coords(r->dst_pshape, wd, cd);
        for (int32_t ws = 0; ws < ns; ++ws) {
            int32_t cs[DISTDL_MAX_RANK];
            coords(r->src_pshape, ws, cs);
            Region in_dst, in_src;
            in_dst.shard = ns + wd;
            in_src.shard = ws;
            bool empty = false;
            for (int k = 0; k < d; ++k) {
                const int64_t s0 = r->src_start[k][cs[k]], s1 = s0 + r->src_size[k][cs[k]];
                const int64_t d0 = r->dst_start[k][cd[k]], d1 = d0 + r->dst_size[k][cd[k]];
                const int64_t lo = std::max(s0, d0), hi = std::min(s1, d1);
                if (hi <= lo) {
                    empty = true;
                    break;
                }
                in_dst.start[k] = lo - d0;
                in_src.start[k] = lo - s0;
                in_dst.extent[k] = in_src.extent[k] = hi - lo;
            }
            if (empty) continue;
            PendingSource from_src{in_src, 0, 0}, from_dst{in_dst, 0, 0};
            if (!fb.add(in_dst, {from_src}, 1)) return fail(DISTDL_ERR_SHAPE, "repartition plan: box out of range");
            if (!ab.add(in_src, {from_dst}, 1)) return fail(DISTDL_ERR_SHAPE, "repartition plan: box out of range");
        }
    }
    if (!fb.destinations_disjoint() || !ab.destinations_disjoint())
        return fail(DISTDL_ERR_SHAPE, "repartition plan: boxes overlap");
    return DISTDL_OK;
}

// ---------------------------------------------------------------------------------------------
// Row plan: one record per (dimension, worker coordinate), see FastDim.
// ---------------------------------------------------------------------------------------------
static void magic_of(int64_t e, uint32_t *magic, uint32_t *shift) {
    // exact division of any x < 2^31 by e >= 2: x / e == umulhi(x, magic) >> shift with s = ceil(log2 e),
    // magic = ceil(2^(31+s) / e) < 2^32, shift = s - 1; e <= 1: magic 0 (the quotient is x itself)
    *magic = 0;
    *shift = 0;
    if (e < 2) return;
    int sft = 0;
    while (((int64_t)1 << sft) < e) ++sft;
    const unsigned __int128 num = (unsigned __int128)1 << (31 + sft);
    *magic = (uint32_t)((num + (uint64_t)e - 1) / (uint64_t)e);
    *shift = (uint32_t)(sft - 1);
}

// Deals `total[i]` blocks of kind i out in groups: the rarest kind present gets one block per group.
static bool fast_groups(const int64_t total[2], FastHeader *h) {
    int64_t least = 0;
    for (int i = 0; i < 2; ++i)
        if (total[i] > 0 && (least == 0 || total[i] < least)) least = total[i];
    if (least == 0) return false;
    int64_t groups = 0, per_group = 0;
    for (int i = 0; i < 2; ++i) {
        h->group[i] = total[i] > 0 ? (int32_t)std::min<int64_t>(64, total[i] / least) : 0;
        if (h->group[i]) groups = std::max(groups, (total[i] + h->group[i] - 1) / h->group[i]);
        per_group += h->group[i];
    }
    if (groups * per_group >= ((int64_t)1 << 31)) return false;
    h->num_groups = (int32_t)groups;
    return true;
}

void build_fast_plan(distdl_partition *p) {
    FastPlanHost &f = p->fast;
    f.usable = f.adj_usable = false;
    f.dims.clear();
    memset(&f.hdr, 0, sizeof(f.hdr));
    memset(&f.adj_hdr, 0, sizeof(f.adj_hdr));
    const int d = p->rank;
    const int esize = elem_size(p->dtype);
    const int64_t per = 16 / esize;
    int64_t coords = 0;
    for (int k = 0; k < d; ++k) coords += p->pshape[k];
    if (coords > kMaxFastCoords) return;
    // the innermost dimension in whole 16-byte units, for every worker coordinate along it
    for (int32_t c = 0; c < p->pshape[d - 1]; ++c)
        if (p->hlo[d - 1][c] % per || p->hhi[d - 1][c] % per || p->size[d - 1][c] % per) return;
    FastHeader &h = f.hdr;
    h.rank = d;
    h.num_workers = p->num_workers;
    int32_t stride = 1;
    for (int k = d - 1; k >= 0; --k) {
        h.wstride[k] = stride;
        stride *= p->pshape[k];
    }
    int64_t any_ghost = 0;
    bool wide_enough = true;          // every bulk at least as wide as its two neighbours' reach together
    for (int k = 0; k < d; ++k) {
        h.pshape[k] = p->pshape[k];
        h.dim_base[k] = (int32_t)f.dims.size();
        const int64_t unit = k == d - 1 ? per : 1;
        const int32_t pk = p->pshape[k];
        for (int32_t c = 0; c < pk; ++c) {
            FastDim e;
            memset(&e, 0, sizeof(e));
            e.hlo = (int32_t)(p->hlo[k][c] / unit);
            e.b = (int32_t)(p->size[k][c] / unit);
            e.n = (int32_t)(p->padded_extent(k, c) / unit);
            any_ghost += e.n - e.b;
            const bool has_lo = c > 0 || p->periodic[k], has_hi = c + 1 < pk || p->periodic[k];
            e.lo_c = has_lo ? (c + pk - 1) % pk : -1;
            e.hi_c = has_hi ? (c + 1) % pk : -1;
            if (has_lo) {
                e.lo_shift = (int32_t)((p->hlo[k][e.lo_c] + p->size[k][e.lo_c] - p->hlo[k][c]) / unit);
                e.rlo = (int32_t)(p->hhi[k][e.lo_c] / unit);
            }
            if (has_hi) {
                e.hi_shift = (int32_t)((p->hlo[k][e.hi_c] - p->hlo[k][c] - p->size[k][c]) / unit);
                e.rhi = (int32_t)(p->hlo[k][e.hi_c] / unit);
            }
            if (e.rlo + e.rhi > e.b) wide_enough = false;
            uint32_t sn, sb, sg, sbi, srr;
            magic_of(e.n, &e.magic_n, &sn);
            magic_of(e.b, &e.magic_b, &sb);
            magic_of(e.n - e.b, &e.magic_g, &sg);
            magic_of(e.b - e.rlo - e.rhi, &e.magic_bi, &sbi);
            magic_of(e.rlo + e.rhi, &e.magic_rr, &srr);
            e.shifts = sn | (sb << 6) | (sg << 12) | (sbi << 18) | (srr << 24);
            f.dims.push_back(e);
        }
    }
    h.num_records = (int32_t)f.dims.size();
    h.num_lines = p->num_workers / p->pshape[d - 1];
    if (any_ghost == 0) return;     // nothing to exchange: the box plan (empty) handles it
    // block sizes from the largest worker
    int64_t nx_max = 1, ghost_rows_max = 0, bulk_rows_max = 0, inner_rows_max = 0;
    int64_t gc = 0, ec = 0;         // per row of a line: ghost units, and units of the row ends that H* rewrites
    for (int32_t c = 0; c < p->pshape[d - 1]; ++c) {
        const FastDim &e = f.dims[h.dim_base[d - 1] + c];
        nx_max = std::max<int64_t>(nx_max, e.n);
        gc += e.n - e.b;
        ec += e.n - e.b + e.rlo + e.rhi;
    }
    for (int32_t w = 0; w < p->num_workers; ++w) {
        int32_t c[DISTDL_MAX_RANK];
        p->coords(w, c);
        int64_t all = 1, bulk = 1, inner = 1;
        for (int k = 0; k + 1 < d; ++k) {
            const FastDim &e = f.dims[h.dim_base[k] + c[k]];
            all *= e.n;
            bulk *= e.b;
            inner *= std::max(0, e.b - e.rlo - e.rhi);
        }
        ghost_rows_max = std::max(ghost_rows_max, all - bulk);   // rows with a ghost index in some outer dimension
        bulk_rows_max = std::max(bulk_rows_max, bulk);
        inner_rows_max = std::max(inner_rows_max, inner);
    }
    if (ghost_rows_max >= ((int64_t)1 << 31) || bulk_rows_max >= ((int64_t)1 << 31)) return;
    if (gc > 1024) return;          // staging of one row's ghost units for all workers of a line: 16 KB at most
    const int32_t rows_s = (int32_t)std::min<int64_t>(256, std::max<int64_t>(1, 4096 / nx_max));
    auto tiles = [](int64_t rows, int32_t per_tile) { return (int32_t)((rows + per_tile - 1) / per_tile); };
    // ---- H
    h.rows_per_tile[0] = rows_s;
    h.tiles_per_owner[0] = tiles(ghost_rows_max, rows_s);
    if (gc > 0) {
        h.rows_per_tile[1] = (int32_t)std::min<int64_t>(128, std::max<int64_t>(1, 512 / gc));
        h.tiles_per_owner[1] = tiles(bulk_rows_max, h.rows_per_tile[1]);
    }
    {
        const int64_t total[2] = {(int64_t)h.tiles_per_owner[0] * p->num_workers, (int64_t)h.tiles_per_owner[1] * h.num_lines};
        f.usable = fast_groups(total, &h);
    }
    // ---- row ends of H*: every bulk at least as wide as its two neighbours' reach together, some reach along the rows,
    // and some rows out of every outer neighbour's reach
    if (!f.usable || !wide_enough || ec == gc || ec > 1024 || inner_rows_max == 0) return;
    FastHeader &a = f.adj_hdr;
    a = h;
    memset(a.rows_per_tile, 0, sizeof(a.rows_per_tile));
    memset(a.tiles_per_owner, 0, sizeof(a.tiles_per_owner));
    a.rows_per_tile[1] = (int32_t)std::min<int64_t>(128, std::max<int64_t>(1, 512 / ec));
    a.tiles_per_owner[1] = tiles(inner_rows_max, a.rows_per_tile[1]);
    {
        const int64_t total[2] = {0, (int64_t)a.tiles_per_owner[1] * a.num_lines};
        f.adj_usable = fast_groups(total, &a);
    }
}

void split_evenly(int64_t n, int32_t p, std::vector<int64_t> &start, std::vector<int64_t> &size) {
    balanced_split(n, p, start, size);
}

}  // namespace distdl
