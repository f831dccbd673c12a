// Host side of the C ABI declared in speca.h: handle, arena layout, per-sample reference
// history, the host-computed scalars of Eq. 2-3, argument checks and kernel launches.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "speca_internal.h"

using namespace speca;

namespace {

constexpr size_t kAlign = 256;
// Planes start on 4 KB boundaries (relative to the arena base). A warp moves 1 KB per 32-byte vector
// instruction; streams whose starts differ by an odd multiple of 256 B split those across L2 / DRAM
// interleave boundaries and measured 3-5 % slower on B200.
constexpr size_t kPlaneAlign = 4096;
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
constexpr size_t kGaveUpWord = kVerifyTickets;  // index of the bulk path's flag among the counter words
constexpr size_t kCounterBytes = (kVerifyTickets + 1) * sizeof(uint32_t);

struct Layout {
    size_t segs_off, tiles_off[kNumTileSizes], partials_off, ticket_off, tables_off, total;
    std::vector<SegDesc> segs;
    std::vector<uint32_t> tiles[kNumTileSizes];  // per tile size: first tile of each segment, then the total
};

// Shape checks and arena layout shared by speca_cache_arena_bytes and speca_cache_create.
speca_status_t make_layout_impl(const speca_cache_config_t* cfg, Layout* L) {
    if (cfg == nullptr || cfg->entries == nullptr) return SPECA_ERR_INVALID_ARG;
    if (cfg->n_entries < 1 || cfg->n_entries > SPECA_MAX_ENTRIES) return SPECA_ERR_SHAPE;
    if (cfg->batch < 1 || cfg->batch > SPECA_MAX_BATCH) return SPECA_ERR_SHAPE;
    if (cfg->max_order < 0 || cfg->max_order > SPECA_MAX_ORDER) return SPECA_ERR_SHAPE;
    if (cfg->dtype != SPECA_F32 && cfg->dtype != SPECA_BF16) return SPECA_ERR_INVALID_ARG;
    if (cfg->basis != SPECA_BASIS_TAYLOR && cfg->basis != SPECA_BASIS_NEWTON &&
        cfg->basis != SPECA_BASIS_ADAMS_BASHFORTH)
        return SPECA_ERR_INVALID_ARG;
    if (cfg->path != SPECA_PATH_AUTO && cfg->path != SPECA_PATH_DIRECT && cfg->path != SPECA_PATH_BULK &&
        cfg->path != SPECA_PATH_WIDE)
        return SPECA_ERR_INVALID_ARG;
    if (cfg->verify_entry < -1 || cfg->verify_entry >= cfg->n_entries) return SPECA_ERR_INVALID_ARG;
    if (cfg->layout != SPECA_LAYOUT_TABLES && cfg->layout != SPECA_LAYOUT_HISTORY) return SPECA_ERR_INVALID_ARG;
    // the raw-feature cache runs on the default kernels only
    if (cfg->layout == SPECA_LAYOUT_HISTORY && cfg->path != SPECA_PATH_AUTO && cfg->path != SPECA_PATH_WIDE)
        return SPECA_ERR_UNSUPPORTED;
    const size_t esz = cfg->dtype == SPECA_BF16 ? 2 : 4;
    const size_t n_segs = static_cast<size_t>(cfg->n_entries) * cfg->batch;
    const int B = cfg->batch, m = cfg->max_order;

    size_t off = 0;
    L->segs_off = off;
    off = align_up(off + n_segs * sizeof(SegDesc), kAlign);
    for (int k = 0; k < kNumTileSizes; ++k) {
        L->tiles_off[k] = off;
        off = align_up(off + (n_segs + 1) * sizeof(uint32_t), kAlign);
    }
    L->partials_off = off;
    off = align_up(off + static_cast<size_t>(kMaxClusters) * B * 3 * sizeof(float), kAlign);  // up to 3 values per metric
    L->ticket_off = off;  // the verify kernel's arrival counters, then the bulk path's gave-up flag
    off = align_up(off + kCounterBytes, kPlaneAlign);
    L->tables_off = off;

    L->segs.resize(n_segs);
    uint64_t n_tiles[kNumTileSizes];
    for (int k = 0; k < kNumTileSizes; ++k) {
        L->tiles[k].assign(n_segs + 1, 0);
        n_tiles[k] = 0;
    }
    for (int e = 0; e < cfg->n_entries; ++e) {
        const int64_t tokens = cfg->entries[e].tokens;
        const int64_t dim = cfg->entries[e].dim;
        if (tokens < 1 || dim < 1) return SPECA_ERR_SHAPE;
        if (tokens > (int64_t(1) << 31) / dim) return SPECA_ERR_SHAPE;  // n_elems must stay below 2^31
        const uint64_t n = static_cast<uint64_t>(tokens) * dim;
        if (n >= (uint64_t(1) << 31)) return SPECA_ERR_SHAPE;
        const size_t stride = align_up(n * esz, kPlaneAlign);
        for (int b = 0; b < B; ++b) {
            SegDesc& s = L->segs[static_cast<size_t>(e) * B + b];
            s.plane0_off = off;
            s.plane_stride = stride;
            s.io_off = static_cast<uint64_t>(b) * n * esz;
            s.n_elems = static_cast<uint32_t>(n);
            s.entry = static_cast<uint16_t>(e);
            s.sample = static_cast<uint16_t>(b);
            off += stride * (m + 1);
            for (int k = 0; k < kNumTileSizes; ++k) {
                L->tiles[k][static_cast<size_t>(e) * B + b] = static_cast<uint32_t>(n_tiles[k]);
                n_tiles[k] += (n * esz + kTileSizes[k] - 1) / kTileSizes[k];
                if (n_tiles[k] >= (uint64_t(1) << 32)) return SPECA_ERR_SHAPE;
            }
        }
    }
    for (int k = 0; k < kNumTileSizes; ++k) L->tiles[k][n_segs] = static_cast<uint32_t>(n_tiles[k]);
    L->total = off;
    return SPECA_OK;
}

// The C ABI never lets an exception out: a failed host allocation becomes SPECA_ERR_NOMEM.
speca_status_t make_layout(const speca_cache_config_t* cfg, Layout* L) noexcept {
    try {
        return make_layout_impl(cfg, L);
    } catch (const std::bad_alloc&) {
        return SPECA_ERR_NOMEM;
    } catch (...) {
        return SPECA_ERR_INVALID_ARG;
    }
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

}  // namespace

struct speca_cache {
    int n_entries, B, m, dtype, basis, verify_entry, device, path, layout;
    double eps;
    char* arena;
    Layout L;
    int sm_count;
    int grid_verify, cluster;
    int tile_update, tile_forecast;  // indices into kTileSizes
    // per-sample reference history, most recent first
    int32_t n_refs[SPECA_MAX_BATCH];
    double t_hist[SPECA_MAX_BATCH][SPECA_MAX_ORDER + 1];
    // reference step in progress
    bool pending;
    double pend_t[SPECA_MAX_BATCH];
    uint8_t pend_mask[SPECA_MAX_BATCH];
    std::vector<uint8_t> entry_updated;
    uint64_t launches;
    speca_cache_stats_t stats;
    char last_error[256];
};

namespace {

speca_status_t fail(speca_cache* c, speca_status_t st, const char* fmt, ...) {
    if (c != nullptr) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->last_error, sizeof c->last_error, fmt, ap);
        va_end(ap);
    }
    return st;
}

// Reports a failed runtime call and takes its error out of the thread's last-error slot, so that a
// recoverable failure is not reported a second time by the next call (an error that broke the
// context is returned again by the runtime itself).
speca_status_t cuda_fail(speca_cache* c, cudaError_t err, const char* what) {
    (void)cudaGetLastError();
    return fail(c, SPECA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(err));
}

inline size_t elem_size(const speca_cache* c) { return c->dtype == SPECA_BF16 ? 2 : 4; }

// An error left by earlier work on this thread surfaces here, once, before new work is queued.
speca_status_t check_sticky(speca_cache* c) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(c, e, "earlier CUDA error");
    return SPECA_OK;
}

// The order a launch's kernel is compiled for: the highest among its samples.
int launch_order(const int8_t* order, int batch) {
    int v = 0;
    for (int b = 0; b < batch; ++b) v = order[b] > v ? order[b] : v;
    return v;
}

// Horner multipliers of Eq. 2 for sample b at time t: level i (1-based) multiplies by mu[i-1].
void forecast_scalars(const speca_cache* c, int b, double t, int* order, float* mu) {
    const int v = c->n_refs[b] < 1 ? -1 : (c->n_refs[b] - 1 < c->m ? c->n_refs[b] - 1 : c->m);
    *order = v;
    for (int i = 0; i < SPECA_MAX_ORDER; ++i) mu[i] = 0.f;
    if (c->basis == SPECA_BASIS_ADAMS_BASHFORTH) {
        // F + x (D_1 + h/2 (D_2 + 5h/6 (D_3 + 9h/10 D_4))): the v-step Adams-Bashforth sum over the
        // slopes g_j = sum_i C(j,i) (-h)^i D_{1+i}, collected by plane (coefficients 1, 1/2, 5/12, 3/8)
        static const double ratio[SPECA_MAX_ORDER] = {1.0, 1.0 / 2, 5.0 / 6, 9.0 / 10};
        const double h = v >= 2 ? c->t_hist[b][0] - c->t_hist[b][1] : 0.0;
        for (int i = 1; i <= v; ++i) mu[i - 1] = static_cast<float>(i == 1 ? t - c->t_hist[b][0] : ratio[i - 1] * h);
        return;
    }
    for (int i = 1; i <= v; ++i) {
        const double x = (c->basis == SPECA_BASIS_NEWTON) ? (t - c->t_hist[b][i - 1]) : (t - c->t_hist[b][0]) / i;
        mu[i - 1] = static_cast<float>(x);
    }
}

// SPECA_LAYOUT_HISTORY: the planes hold the features of the last references, the one of age j (0 =
// latest) in physical plane (references - 1 - j) mod (m + 1). The table a SPECA_LAYOUT_TABLES cache
// would hold is a linear map of those features: run Eq. 3's recursion on unit vectors, oldest feature
// first, to get the map; weigh its rows as the basis weighs the planes (Eq. 2); the result is one weight
// per stored feature, scattered to physical plane order. The forecast is sum_i w[i] * plane_i, i <= order.
void history_weights(const speca_cache* c, int b, double t, int* order, float* w) {
    const int refs = c->n_refs[b];
    const int v = refs < 1 ? -1 : (refs - 1 < c->m ? refs - 1 : c->m);
    *order = v;
    for (int i = 0; i < kCoef; ++i) w[i] = 0.f;
    if (v < 0) return;
    const double* th = c->t_hist[b];
    double rows[kCoef][kCoef] = {};  // rows[i][j]: share of the feature of age j in plane i
    rows[0][v] = 1.0;
    for (int k = v - 1; k >= 0; --k) {  // fold in the feature of age k; v - k references came before it
        double next[kCoef][kCoef] = {};
        next[0][k] = 1.0;
        for (int i = 0; i < v - k; ++i) {
            const double gap = th[k] - (c->basis == SPECA_BASIS_NEWTON ? th[k + 1 + i] : th[k + 1]);
            for (int j = 0; j <= v; ++j) next[i + 1][j] = (next[i][j] - rows[i][j]) / gap;
        }
        for (int i = 0; i <= v - k; ++i)
            for (int j = 0; j <= v; ++j) rows[i][j] = next[i][j];
    }
    double plane_w[kCoef];
    plane_w[0] = 1.0;
    if (c->basis == SPECA_BASIS_NEWTON) {
        for (int i = 1; i <= v; ++i) plane_w[i] = plane_w[i - 1] * (t - th[i - 1]);
    } else if (c->basis == SPECA_BASIS_ADAMS_BASHFORTH) {
        static const double collected[SPECA_MAX_ORDER] = {1.0, 1.0 / 2, 5.0 / 12, 3.0 / 8};
        const double x = t - th[0], h = v >= 2 ? th[0] - th[1] : 0.0;
        double hp = 1.0;
        for (int i = 1; i <= v; ++i) {
            plane_w[i] = x * collected[i - 1] * hp;
            hp *= h;
        }
    } else {
        const double x = t - th[0];
        for (int i = 1; i <= v; ++i) plane_w[i] = plane_w[i - 1] * x / i;
    }
    const int ring = c->m + 1;
    for (int j = 0; j <= v; ++j) {
        double a = 0.0;
        for (int i = 0; i <= v; ++i) a += plane_w[i] * rows[i][j];
        w[((refs - 1 - j) % ring + ring) % ring] = static_cast<float>(a);
    }
}

// Scalars of a forecast for sample b, whichever layout the cache has.
void forecast_coefficients(const speca_cache* c, int b, double t, int* order, float* coef) {
    if (c->layout == SPECA_LAYOUT_HISTORY)
        history_weights(c, b, t, order, coef);
    else
        forecast_scalars(c, b, t, order, coef);
}

}  // namespace

extern "C" {

speca_status_t speca_cache_arena_bytes(const speca_cache_config_t* cfg, size_t* out_bytes) {
    if (out_bytes == nullptr) return SPECA_ERR_INVALID_ARG;
    Layout L;
    speca_status_t st = make_layout(cfg, &L);
    if (st != SPECA_OK) return st;
    *out_bytes = L.total;
    return SPECA_OK;
}

speca_status_t speca_cache_create(const speca_cache_config_t* cfg, speca_cache_t** out) {
    if (out == nullptr) return SPECA_ERR_INVALID_ARG;
    *out = nullptr;
    speca_cache* c = new (std::nothrow) speca_cache();
    if (c == nullptr) return SPECA_ERR_NOMEM;
    speca_status_t st = make_layout(cfg, &c->L);
    if (st != SPECA_OK) {
        delete c;
        return st;
    }
    if (cfg->arena == nullptr) {
        delete c;
        return SPECA_ERR_INVALID_ARG;
    }
    if (reinterpret_cast<uintptr_t>(cfg->arena) % kAlign != 0) {
        delete c;
        return SPECA_ERR_ALIGNMENT;
    }
    if (cfg->arena_bytes < c->L.total) {
        delete c;
        return SPECA_ERR_NOMEM;
    }
    int n_dev = 0;
    cudaError_t ce = cudaGetDeviceCount(&n_dev);
    if (ce != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) {
        delete c;
        return ce != cudaSuccess ? SPECA_ERR_CUDA : SPECA_ERR_INVALID_ARG;
    }
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, cfg->device);
    if (major != 10) {  // the kernels are built for sm_100a only
        delete c;
        return SPECA_ERR_UNSUPPORTED;
    }
    c->n_entries = cfg->n_entries;
    c->B = cfg->batch;
    c->m = cfg->max_order;
    c->dtype = cfg->dtype;
    c->basis = cfg->basis;
    c->layout = cfg->layout;
    c->verify_entry = cfg->verify_entry < 0 ? cfg->n_entries - 1 : cfg->verify_entry;
    c->device = cfg->device;
    c->path = cfg->path == SPECA_PATH_AUTO ? SPECA_PATH_WIDE : cfg->path;
    c->eps = cfg->eps > 0.f ? static_cast<double>(cfg->eps) : 1e-8;  // Eq. 4
    c->arena = static_cast<char*>(cfg->arena);
    c->pending = false;
    c->launches = 0;
    std::memset(&c->stats, 0, sizeof c->stats);
    c->last_error[0] = 0;
    try {
        c->entry_updated.assign(c->n_entries, 0);
    } catch (const std::bad_alloc&) {
        delete c;
        return SPECA_ERR_NOMEM;
    }
    for (int b = 0; b < SPECA_MAX_BATCH; ++b) {
        c->n_refs[b] = 0;
        for (int i = 0; i <= SPECA_MAX_ORDER; ++i) c->t_hist[b][i] = std::numeric_limits<double>::quiet_NaN();
    }

    DeviceGuard guard(c->device);
    if (!guard.ok) {
        delete c;
        return SPECA_ERR_CUDA;
    }
    const Layout& L = c->L;
    ce = cudaMemcpy(c->arena + L.segs_off, L.segs.data(), L.segs.size() * sizeof(SegDesc), cudaMemcpyHostToDevice);
    for (int k = 0; k < kNumTileSizes && ce == cudaSuccess; ++k)
        ce = cudaMemcpy(c->arena + L.tiles_off[k], L.tiles[k].data(), L.tiles[k].size() * sizeof(uint32_t),
                        cudaMemcpyHostToDevice);
    if (ce == cudaSuccess) ce = cudaMemset(c->arena + L.ticket_off, 0, kCounterBytes);
    if (ce != cudaSuccess) {
        delete c;
        return SPECA_ERR_CUDA;
    }
    cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    c->tile_update = tile_size_index(stream_tile_bytes(c->path, true));
    c->tile_forecast = tile_size_index(stream_tile_bytes(c->path, false));
    if (c->tile_update < 0 || c->tile_forecast < 0) {
        delete c;
        return SPECA_ERR_UNSUPPORTED;
    }
    c->cluster = SPECA_VERIFY_CLUSTER;
    // the fewest over the orders a launch may have: samples below max_order run lower-order kernels
    int n_clusters = kMaxClusters;
    for (int v = 0; v <= c->m; ++v) {
        const int n = max_resident_verify_clusters(c->dtype, v, c->cluster);
        n_clusters = n < n_clusters ? n : n_clusters;
    }
    if (n_clusters > kMaxClusters) n_clusters = kMaxClusters;
    c->grid_verify = n_clusters * c->cluster;
    *out = c;
    return SPECA_OK;
}

speca_status_t speca_cache_destroy(speca_cache_t* c) {
    if (c == nullptr) return SPECA_OK;
    DeviceGuard guard(c->device);
    cudaError_t ce = cudaDeviceSynchronize();
    // the bulk path's kernels set this word when a bounded wait for a copy gave up
    uint32_t gave_up = 0;
    if (ce == cudaSuccess)
        ce = cudaMemcpy(&gave_up, c->arena + c->L.ticket_off + kGaveUpWord * sizeof(uint32_t), sizeof gave_up,
                        cudaMemcpyDeviceToHost);
    delete c;
    return (ce == cudaSuccess && gave_up == 0) ? SPECA_OK : SPECA_ERR_CUDA;
}

speca_status_t speca_cache_reset(speca_cache_t* c, const uint8_t* host_sample_mask) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (c->pending) return fail(c, SPECA_ERR_STATE, "reset while a reference step is open");
    for (int b = 0; b < c->B; ++b) {
        if (host_sample_mask != nullptr && host_sample_mask[b] == 0) continue;
        c->n_refs[b] = 0;
        c->stats.resets[b] += 1;
        for (int i = 0; i <= SPECA_MAX_ORDER; ++i) c->t_hist[b][i] = std::numeric_limits<double>::quiet_NaN();
    }
    return SPECA_OK;
}

}  // extern "C"

namespace {

// speca_cache_update, optionally re-arming the masked samples (act_spec / act_active non-null) in the
// same launch.
speca_status_t update_impl(speca_cache_t* c, const void* const* feats, const double* t_ref,
                           const uint8_t* host_sample_mask, void* stream, int32_t* act_spec, uint8_t* act_active) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (feats == nullptr || t_ref == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "update: null argument");
    uint8_t mask[SPECA_MAX_BATCH];
    bool any_sample = false;
    for (int b = 0; b < c->B; ++b) {
        mask[b] = (host_sample_mask == nullptr || host_sample_mask[b] != 0) ? 1 : 0;
        any_sample |= mask[b] != 0;
        if (mask[b] && !std::isfinite(t_ref[b])) return fail(c, SPECA_ERR_INVALID_ARG, "update: t_ref[%d] not finite", b);
    }
    if (c->pending) {
        for (int b = 0; b < c->B; ++b) {
            if (mask[b] != c->pend_mask[b] || (mask[b] && std::memcmp(&t_ref[b], &c->pend_t[b], sizeof(double)) != 0))
                return fail(c, SPECA_ERR_STATE, "update: mask or t_ref differ from the open reference step (sample %d)", b);
        }
    }
    StreamParams p;
    std::memset(&p, 0, sizeof p);
    // scalars of Eq. 3: reciprocal gaps
    for (int b = 0; b < c->B; ++b) {
        p.order[b] = -1;
        if (!mask[b]) continue;
        const int v_new = c->n_refs[b] < c->m ? c->n_refs[b] : c->m;
        for (int i = 0; i < v_new; ++i) {
            const double gap = t_ref[b] - (c->basis == SPECA_BASIS_NEWTON ? c->t_hist[b][i] : c->t_hist[b][0]);
            if (gap == 0.0) return fail(c, SPECA_ERR_ZERO_GAP, "update: sample %d repeats a reference time", b);
            p.coef[b][i] = static_cast<float>(1.0 / gap);
        }
        p.order[b] = static_cast<int8_t>(v_new);
        if (c->layout == SPECA_LAYOUT_HISTORY) {
            // nothing is differenced now: the feature is copied into the plane after the latest one
            // (the gaps above were only checked, so that no later forecast divides by zero)
            p.order[b] = 0;
            p.slot[b] = static_cast<uint8_t>(c->n_refs[b] % (c->m + 1));
        }
    }
    int e_lo = -1, e_hi = -1;
    const size_t esz = elem_size(c);
    for (int e = 0; e < c->n_entries; ++e) {
        if (feats[e] == nullptr) continue;
        if (c->entry_updated[e]) return fail(c, SPECA_ERR_STATE, "update: entry %d already updated in this step", e);
        if (feats[e] == SPECA_FEATURE_IN_PLACE) {
            if (c->layout != SPECA_LAYOUT_HISTORY)
                return fail(c, SPECA_ERR_INVALID_ARG, "update: SPECA_FEATURE_IN_PLACE needs a cache that keeps raw features");
            continue;  // the caller wrote every masked sample's feature into its next plane: nothing to copy
        }
        if (reinterpret_cast<uintptr_t>(feats[e]) % esz != 0)
            return fail(c, SPECA_ERR_ALIGNMENT, "update: feats[%d] not aligned to the element size", e);
        if (c->layout == SPECA_LAYOUT_HISTORY) {
            // The model may have written the feature straight into the plane that is next in the ring
            // (speca_cache_next_slot): then there is nothing to copy for this entry.
            bool in_place = any_sample;
            for (int b = 0; b < c->B && in_place; ++b) {
                if (!mask[b]) continue;
                const SegDesc& s = c->L.segs[static_cast<size_t>(e) * c->B + b];
                const char* slot_ptr = c->arena + s.plane0_off + static_cast<size_t>(p.slot[b]) * s.plane_stride;
                in_place = static_cast<const char*>(feats[e]) + s.io_off == slot_ptr;
            }
            if (in_place) continue;  // p.io[e] stays null: the launch skips the entry
        }
        if (e_lo < 0) e_lo = e;
        e_hi = e;
        p.io[e] = const_cast<void*>(feats[e]);
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    if (e_lo >= 0 && any_sample) {
        const Layout& L = c->L;
        const std::vector<uint32_t>& tiles = L.tiles[c->tile_update];
        p.segs = reinterpret_cast<const SegDesc*>(c->arena + L.segs_off);
        p.tile_start = reinterpret_cast<const uint32_t*>(c->arena + L.tiles_off[c->tile_update]);
        p.arena = c->arena;
        p.dev_mask = nullptr;
        p.err_flag = reinterpret_cast<uint32_t*>(c->arena + L.ticket_off) + kGaveUpWord;
        p.seg_lo = static_cast<uint32_t>(e_lo) * c->B;
        p.seg_hi = static_cast<uint32_t>(e_hi + 1) * c->B;
        p.tile_lo = tiles[p.seg_lo];
        p.tile_hi = tiles[p.seg_hi];
        const uint32_t n_tiles = p.tile_hi - p.tile_lo;
        const uint32_t full = static_cast<uint32_t>(c->sm_count * stream_ctas_per_sm(c->path, true, c->dtype, launch_order(p.order, c->B)));
        const int grid = static_cast<int>(n_tiles < full ? n_tiles : full);
        uint64_t bits = 0;
        for (int b = 0; b < c->B; ++b)
            if (mask[b]) bits |= uint64_t(1) << b;
        if (act_active != nullptr && c->path != SPECA_PATH_BULK) {  // the kernel's first CTA re-arms the samples
            p.act_spec = act_spec;
            p.act_active = act_active;
            p.act_bits = bits;
            act_active = nullptr;
        }
        cudaError_t ce = launch_update(p, c->dtype, c->path, grid, static_cast<cudaStream_t>(stream));
        if (ce != cudaSuccess) return cuda_fail(c, ce, "update launch");
        c->launches += 1;
        c->stats.update_launches += 1;
    }
    if (act_active != nullptr && any_sample) {  // nothing was copied (or the staged kernels ran): a launch of its own
        uint64_t bits = 0;
        for (int b = 0; b < c->B; ++b)
            if (mask[b]) bits |= uint64_t(1) << b;
        cudaError_t ce = launch_activate(bits, c->B, act_spec, act_active, static_cast<cudaStream_t>(stream));
        if (ce != cudaSuccess) return cuda_fail(c, ce, "activate launch");
        c->launches += 1;
        c->stats.activate_launches += 1;
    }
    if (!c->pending) {
        c->pending = true;
        for (int b = 0; b < c->B; ++b) {
            c->pend_mask[b] = mask[b];
            c->pend_t[b] = t_ref[b];
        }
    }
    for (int e = 0; e < c->n_entries; ++e)
        if (feats[e] != nullptr) c->entry_updated[e] = 1;
    return SPECA_OK;
}

}  // namespace

extern "C" {

speca_status_t speca_cache_update(speca_cache_t* c, const void* const* feats, const double* t_ref,
                                  const uint8_t* host_sample_mask, void* stream) {
    return update_impl(c, feats, t_ref, host_sample_mask, stream, nullptr, nullptr);
}

speca_status_t speca_cache_update_activate(speca_cache_t* c, const void* const* feats, const double* t_ref,
                                           const uint8_t* host_sample_mask, int32_t* dev_spec_count,
                                           uint8_t* dev_active_mask, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (dev_spec_count == nullptr || dev_active_mask == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "update_activate: null argument");
    if (reinterpret_cast<uintptr_t>(dev_spec_count) % 4 != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "update_activate: dev_spec_count must be 4-byte aligned");
    return update_impl(c, feats, t_ref, host_sample_mask, stream, dev_spec_count, dev_active_mask);
}

speca_status_t speca_cache_update_forecast(speca_cache_t* c, const void* const* feats, const double* t_ref,
                                           const uint8_t* host_sample_mask, const double* t_target,
                                           const uint8_t* dev_active_mask, void* const* outs, int32_t* dev_spec_count,
                                           uint8_t* dev_rearm_mask, void* stream) {
    return speca_cache_update_forecast_multi(c, feats, t_ref, host_sample_mask, 1, t_target, dev_active_mask, outs,
                                             dev_spec_count, dev_rearm_mask, stream);
}

speca_status_t speca_cache_update_forecast_multi(speca_cache_t* c, const void* const* feats, const double* t_ref,
                                                 const uint8_t* host_sample_mask, int32_t n_targets, const double* t_target,
                                                 const uint8_t* dev_active_mask, void* const* outs, int32_t* dev_spec_count,
                                                 uint8_t* dev_rearm_mask, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (feats == nullptr || t_ref == nullptr || t_target == nullptr || outs == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: null argument");
    if (n_targets < 1 || n_targets > SPECA_MAX_HORIZON)
        return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: n_targets must be 1..%d", SPECA_MAX_HORIZON);
    if ((dev_spec_count == nullptr) != (dev_rearm_mask == nullptr))
        return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: give both re-arming buffers or neither");
    if (reinterpret_cast<uintptr_t>(dev_spec_count) % 4 != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "update_forecast: dev_spec_count must be 4-byte aligned");
    if (c->path != SPECA_PATH_WIDE) return fail(c, SPECA_ERR_UNSUPPORTED, "update_forecast: the default kernel path only");
    const bool hist = c->layout == SPECA_LAYOUT_HISTORY;
    if (c->pending) return fail(c, SPECA_ERR_STATE, "update_forecast: a reference step is open (commit it first)");
    uint8_t mask[SPECA_MAX_BATCH];
    bool any_sample = false;
    for (int b = 0; b < c->B; ++b) {
        mask[b] = (host_sample_mask == nullptr || host_sample_mask[b] != 0) ? 1 : 0;
        any_sample |= mask[b] != 0;
        if (mask[b] && !std::isfinite(t_ref[b])) return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: t_ref[%d] not finite", b);
        for (int k = 0; k < n_targets; ++k)
            if (!std::isfinite(t_target[static_cast<size_t>(k) * c->B + b]))
                return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: t_target[%d][%d] not finite", k, b);
    }
    static thread_local FusedParams q;  // 20 KB: kept off the stack
    std::memset(&q, 0, sizeof q);
    StreamParams& p = q.up;
    uint64_t bits = 0;
    for (int b = 0; b < c->B; ++b) {  // scalars of Eq. 3, as in speca_cache_update
        p.order[b] = -1;
        if (!mask[b]) continue;
        bits |= uint64_t(1) << b;
        const int v_new = c->n_refs[b] < c->m ? c->n_refs[b] : c->m;
        for (int i = 0; i < v_new; ++i) {
            const double gap = t_ref[b] - (c->basis == SPECA_BASIS_NEWTON ? c->t_hist[b][i] : c->t_hist[b][0]);
            if (gap == 0.0) return fail(c, SPECA_ERR_ZERO_GAP, "update_forecast: sample %d repeats a reference time", b);
            p.coef[b][i] = static_cast<float>(1.0 / gap);
        }
        p.order[b] = static_cast<int8_t>(v_new);
        if (hist) {  // nothing is differenced: the feature goes into the ring plane after the latest one
            p.order[b] = 0;
            p.slot[b] = static_cast<uint8_t>(c->n_refs[b] % (c->m + 1));
        }
    }
    p.weighted = hist ? 1 : 0;
    const size_t esz = elem_size(c);
    bool any_out = false;
    for (int e = 0; e < c->n_entries; ++e) {
        if (feats[e] == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: feats[%d] is null (the call is a whole reference step)", e);
        if (reinterpret_cast<uintptr_t>(outs[e]) % esz != 0)
            return fail(c, SPECA_ERR_ALIGNMENT, "update_forecast: outs[%d] not aligned to the element size", e);
        q.out[e] = outs[e];
        any_out |= outs[e] != nullptr;
        if (feats[e] == SPECA_FEATURE_IN_PLACE) {
            if (!hist) return fail(c, SPECA_ERR_INVALID_ARG, "update_forecast: SPECA_FEATURE_IN_PLACE needs a cache that keeps raw features");
            continue;  // the features already sit in their ring planes: nothing to copy, the forecast reads them there
        }
        if (reinterpret_cast<uintptr_t>(feats[e]) % esz != 0)
            return fail(c, SPECA_ERR_ALIGNMENT, "update_forecast: feats[%d] not aligned to the element size", e);
        if (hist) {  // written straight into the next ring planes (speca_cache_next_slot): nothing to copy either
            bool in_place = any_sample;
            for (int b = 0; b < c->B && in_place; ++b) {
                if (!mask[b]) continue;
                const SegDesc& sg = c->L.segs[static_cast<size_t>(e) * c->B + b];
                in_place = static_cast<const char*>(feats[e]) + sg.io_off ==
                           c->arena + sg.plane0_off + static_cast<size_t>(p.slot[b]) * sg.plane_stride;
            }
            if (in_place) continue;
        }
        p.io[e] = const_cast<void*>(feats[e]);
    }
    // The forecast's scalars are those of the history AFTER this step: commit on a copy of the host
    // state, keep the copy if anything below fails.
    int32_t saved_refs[SPECA_MAX_BATCH];
    double saved_hist[SPECA_MAX_BATCH][SPECA_MAX_ORDER + 1];
    std::memcpy(saved_refs, c->n_refs, sizeof saved_refs);
    std::memcpy(saved_hist, c->t_hist, sizeof saved_hist);
    auto roll_back = [&]() {
        std::memcpy(c->n_refs, saved_refs, sizeof saved_refs);
        std::memcpy(c->t_hist, saved_hist, sizeof saved_hist);
    };
    for (int b = 0; b < c->B; ++b) {
        if (!mask[b]) continue;
        for (int i = SPECA_MAX_ORDER; i >= 1; --i) c->t_hist[b][i] = c->t_hist[b][i - 1];
        c->t_hist[b][0] = t_ref[b];
        c->n_refs[b] += 1;
    }
    bool any_forecast = false;
    q.n_targets = n_targets;
    q.batch = c->B;
    for (int b = 0; b < c->B; ++b) {
        int order = -1;
        for (int k = 0; k < n_targets; ++k)
            forecast_coefficients(c, b, t_target[static_cast<size_t>(k) * c->B + b], &order, q.fc_coef[k][b]);
        if (order < 0 && dev_active_mask == nullptr && any_out) {
            roll_back();
            return fail(c, SPECA_ERR_STATE, "update_forecast: sample %d has no reference, in this step or before", b);
        }
        q.fc_order[b] = static_cast<int8_t>(order);
        any_forecast |= order >= 0;
    }
    q.fc_mask = dev_active_mask;
    DeviceGuard guard(c->device);
    if (!guard.ok) {
        roll_back();
        return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    }
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) {
        roll_back();
        return st;
    }
    if (any_sample || (any_forecast && any_out)) {
        const Layout& L = c->L;
        const std::vector<uint32_t>& tiles = L.tiles[c->tile_update];
        p.segs = reinterpret_cast<const SegDesc*>(c->arena + L.segs_off);
        p.tile_start = reinterpret_cast<const uint32_t*>(c->arena + L.tiles_off[c->tile_update]);
        p.arena = c->arena;
        p.err_flag = reinterpret_cast<uint32_t*>(c->arena + L.ticket_off) + kGaveUpWord;
        p.seg_lo = 0;
        p.seg_hi = static_cast<uint32_t>(c->n_entries) * c->B;
        p.tile_lo = tiles[p.seg_lo];
        p.tile_hi = tiles[p.seg_hi];
        if (dev_rearm_mask != nullptr && any_sample) {  // the kernel's first CTA re-arms the updated samples
            p.act_spec = dev_spec_count;
            p.act_active = dev_rearm_mask;
            p.act_bits = bits;
        }
        int v = launch_order(p.order, c->B);
        const int vf = launch_order(q.fc_order, c->B);
        v = vf > v ? vf : v;
        const uint32_t n_tiles = p.tile_hi - p.tile_lo;
        const uint32_t full = static_cast<uint32_t>(c->sm_count * fused_ctas_per_sm(v, hist, c->dtype, n_targets));
        const int grid = static_cast<int>(n_tiles < full ? n_tiles : full);
        cudaError_t ce = launch_update_forecast(q, c->dtype, grid, static_cast<cudaStream_t>(stream));
        if (ce != cudaSuccess) {
            roll_back();
            return cuda_fail(c, ce, "update_forecast launch");
        }
        c->launches += 1;
        c->stats.update_forecast_launches += 1;
    }
    for (int b = 0; b < c->B; ++b)
        if (mask[b]) c->stats.reference_steps[b] += 1;
    return SPECA_OK;
}

speca_status_t speca_cache_commit_step(speca_cache_t* c) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (!c->pending) return fail(c, SPECA_ERR_STATE, "commit: no reference step is open");
    for (int e = 0; e < c->n_entries; ++e)
        if (!c->entry_updated[e]) return fail(c, SPECA_ERR_STATE, "commit: entry %d was not updated in this step", e);
    for (int b = 0; b < c->B; ++b) {
        if (!c->pend_mask[b]) continue;
        for (int i = SPECA_MAX_ORDER; i >= 1; --i) c->t_hist[b][i] = c->t_hist[b][i - 1];
        c->t_hist[b][0] = c->pend_t[b];
        c->n_refs[b] += 1;
        c->stats.reference_steps[b] += 1;
    }
    c->pending = false;
    std::fill(c->entry_updated.begin(), c->entry_updated.end(), 0);
    return SPECA_OK;
}

speca_status_t speca_forecast(speca_cache_t* c, const double* t_target, const uint8_t* dev_active_mask,
                              void* const* outs, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (t_target == nullptr || outs == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "forecast: null argument");
    if (c->pending) return fail(c, SPECA_ERR_STATE, "forecast: a reference step is open (commit it first)");
    StreamParams p;
    std::memset(&p, 0, sizeof p);
    bool any_sample = false;
    for (int b = 0; b < c->B; ++b) {
        if (!std::isfinite(t_target[b])) return fail(c, SPECA_ERR_INVALID_ARG, "forecast: t_target[%d] not finite", b);
        int order;
        forecast_coefficients(c, b, t_target[b], &order, p.coef[b]);
        if (order < 0 && dev_active_mask == nullptr)
            return fail(c, SPECA_ERR_STATE, "forecast: sample %d has no committed reference", b);
        p.order[b] = static_cast<int8_t>(order);
        any_sample |= order >= 0;
    }
    int e_lo = -1, e_hi = -1;
    const size_t esz = elem_size(c);
    for (int e = 0; e < c->n_entries; ++e) {
        if (outs[e] == nullptr) continue;
        if (reinterpret_cast<uintptr_t>(outs[e]) % esz != 0)
            return fail(c, SPECA_ERR_ALIGNMENT, "forecast: outs[%d] not aligned to the element size", e);
        if (e_lo < 0) e_lo = e;
        e_hi = e;
        p.io[e] = outs[e];
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    if (e_lo < 0 || !any_sample) return SPECA_OK;
    const Layout& L = c->L;
    const std::vector<uint32_t>& tiles = L.tiles[c->tile_forecast];
    p.segs = reinterpret_cast<const SegDesc*>(c->arena + L.segs_off);
    p.tile_start = reinterpret_cast<const uint32_t*>(c->arena + L.tiles_off[c->tile_forecast]);
    p.arena = c->arena;
    p.dev_mask = dev_active_mask;
    p.weighted = c->layout == SPECA_LAYOUT_HISTORY ? 1 : 0;
    p.err_flag = reinterpret_cast<uint32_t*>(c->arena + L.ticket_off) + kGaveUpWord;
    p.seg_lo = static_cast<uint32_t>(e_lo) * c->B;
    p.seg_hi = static_cast<uint32_t>(e_hi + 1) * c->B;
    p.tile_lo = tiles[p.seg_lo];
    p.tile_hi = tiles[p.seg_hi];
    const uint32_t n_tiles = p.tile_hi - p.tile_lo;
    const uint32_t full = static_cast<uint32_t>(c->sm_count * stream_ctas_per_sm(c->path, false, c->dtype, launch_order(p.order, c->B)));
    const int grid = static_cast<int>(n_tiles < full ? n_tiles : full);
    cudaError_t ce = launch_forecast(p, c->dtype, c->path, grid, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "forecast launch");
    c->launches += 1;
    c->stats.forecast_launches += 1;
    return SPECA_OK;
}

speca_status_t speca_forecast_multi(speca_cache_t* c, int32_t n_targets, const double* t_targets,
                                    const uint8_t* dev_active_mask, void* const* outs, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (t_targets == nullptr || outs == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "forecast_multi: null argument");
    if (n_targets < 1 || n_targets > SPECA_MAX_HORIZON)
        return fail(c, SPECA_ERR_INVALID_ARG, "forecast_multi: n_targets must be 1..%d", SPECA_MAX_HORIZON);
    if (c->pending) return fail(c, SPECA_ERR_STATE, "forecast_multi: a reference step is open (commit it first)");
    static thread_local MultiParams p;  // 13 KB: kept off the stack
    std::memset(&p, 0, sizeof p);
    bool any_sample = false;
    for (int b = 0; b < c->B; ++b) {
        int order = -1;
        for (int k = 0; k < n_targets; ++k) {
            const double t = t_targets[static_cast<size_t>(k) * c->B + b];
            if (!std::isfinite(t)) return fail(c, SPECA_ERR_INVALID_ARG, "forecast_multi: t_targets[%d][%d] not finite", k, b);
            forecast_coefficients(c, b, t, &order, p.coef[k][b]);
        }
        if (order < 0 && dev_active_mask == nullptr)
            return fail(c, SPECA_ERR_STATE, "forecast_multi: sample %d has no committed reference", b);
        p.order[b] = static_cast<int8_t>(order);
        any_sample |= order >= 0;
    }
    int e_lo = -1, e_hi = -1;
    const size_t esz = elem_size(c);
    for (int e = 0; e < c->n_entries; ++e) {
        if (outs[e] == nullptr) continue;
        if (reinterpret_cast<uintptr_t>(outs[e]) % esz != 0)
            return fail(c, SPECA_ERR_ALIGNMENT, "forecast_multi: outs[%d] not aligned to the element size", e);
        if (e_lo < 0) e_lo = e;
        e_hi = e;
        p.io[e] = outs[e];
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    if (e_lo < 0 || !any_sample) return SPECA_OK;
    const Layout& L = c->L;
    const int ti = tile_size_index(multi_tile_bytes());
    if (ti < 0) return fail(c, SPECA_ERR_UNSUPPORTED, "forecast_multi: no tile table for its tile size");
    const std::vector<uint32_t>& tiles = L.tiles[ti];
    p.segs = reinterpret_cast<const SegDesc*>(c->arena + L.segs_off);
    p.tile_start = reinterpret_cast<const uint32_t*>(c->arena + L.tiles_off[ti]);
    p.arena = c->arena;
    p.dev_mask = dev_active_mask;
    p.weighted = c->layout == SPECA_LAYOUT_HISTORY ? 1 : 0;
    p.n_targets = n_targets;
    p.seg_lo = static_cast<uint32_t>(e_lo) * c->B;
    p.seg_hi = static_cast<uint32_t>(e_hi + 1) * c->B;
    p.tile_lo = tiles[p.seg_lo];
    p.tile_hi = tiles[p.seg_hi];
    const uint32_t n_tiles = p.tile_hi - p.tile_lo;
    const uint32_t full = static_cast<uint32_t>(c->sm_count * multi_ctas_per_sm(n_targets));
    const int grid = static_cast<int>(n_tiles < full ? n_tiles : full);
    cudaError_t ce = launch_forecast_multi(p, c->dtype, c->B, grid, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "forecast_multi launch");
    c->launches += 1;
    c->stats.forecast_multi_launches += 1;
    return SPECA_OK;
}

speca_status_t speca_forecast_sum(speca_cache_t* c, const int32_t* entry_ids, int32_t n_ids, const double* t_target,
                                  const uint8_t* dev_active_mask, const void* base, void* out, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (entry_ids == nullptr || t_target == nullptr || out == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "forecast_sum: null argument");
    if (n_ids < 1 || n_ids > SPECA_MAX_ENTRIES) return fail(c, SPECA_ERR_INVALID_ARG, "forecast_sum: n_ids out of range");
    if (c->pending) return fail(c, SPECA_ERR_STATE, "forecast_sum: a reference step is open (commit it first)");
    static thread_local SumParams p;
    std::memset(&p, 0, sizeof p);
    const Layout& L = c->L;
    for (int j = 0; j < n_ids; ++j) {
        if (entry_ids[j] < 0 || entry_ids[j] >= c->n_entries)
            return fail(c, SPECA_ERR_INVALID_ARG, "forecast_sum: entry_ids[%d] out of range", j);
        const uint32_t n = L.segs[static_cast<size_t>(entry_ids[j]) * c->B].n_elems;
        if (j == 0) p.n_elems = n;
        if (n != p.n_elems) return fail(c, SPECA_ERR_SHAPE, "forecast_sum: entries %d and %d differ in size", entry_ids[0], entry_ids[j]);
        p.ids[j] = static_cast<uint16_t>(entry_ids[j]);
    }
    const size_t esz = elem_size(c);
    if (reinterpret_cast<uintptr_t>(out) % esz != 0 || reinterpret_cast<uintptr_t>(base) % esz != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "forecast_sum: base / out not aligned to the element size");
    bool any_sample = false;
    for (int b = 0; b < c->B; ++b) {
        if (!std::isfinite(t_target[b])) return fail(c, SPECA_ERR_INVALID_ARG, "forecast_sum: t_target[%d] not finite", b);
        int order;
        forecast_coefficients(c, b, t_target[b], &order, p.coef[b]);
        if (order < 0 && dev_active_mask == nullptr)
            return fail(c, SPECA_ERR_STATE, "forecast_sum: sample %d has no committed reference", b);
        p.order[b] = static_cast<int8_t>(order);
        any_sample |= order >= 0;
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    if (!any_sample) return SPECA_OK;
    const uint32_t te = sum_tile_bytes() / static_cast<uint32_t>(esz);
    p.segs = reinterpret_cast<const SegDesc*>(c->arena + L.segs_off);
    p.arena = c->arena;
    p.dev_mask = dev_active_mask;
    p.weighted = c->layout == SPECA_LAYOUT_HISTORY ? 1 : 0;
    p.base = static_cast<const char*>(base);
    p.out = static_cast<char*>(out);
    p.tiles_per_sample = (p.n_elems + te - 1) / te;
    p.batch = c->B;
    p.n_ids = n_ids;
    const uint64_t tiles = static_cast<uint64_t>(p.tiles_per_sample) * c->B;
    const uint64_t full = static_cast<uint64_t>(c->sm_count) * sum_ctas_per_sm();
    const int grid = static_cast<int>(tiles < full ? tiles : full);
    cudaError_t ce = launch_forecast_sum(p, c->dtype, grid, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "forecast_sum launch");
    c->launches += 1;
    c->stats.forecast_sum_launches += 1;
    return SPECA_OK;
}

speca_status_t speca_verify(speca_cache_t* c, const void* fresh, const double* t_target, const float* tau,
                            const uint8_t* dev_active_mask, void* out_pred, float* dev_err, uint8_t* dev_accept,
                            void* stream) {
    return speca_verify_metric(c, SPECA_METRIC_L2, fresh, t_target, tau, dev_active_mask, out_pred, dev_err, dev_accept,
                               stream);
}

// speca_verify_metric (dev_sums == nullptr) and speca_verify_partial (dev_sums given, no tau / err / accept).
struct SelectArgs {
    int32_t k_max, group;
    int32_t* spec_count;
    uint8_t* active;
    int32_t* idx;
    int32_t* n_active;
};

static speca_status_t verify_impl(speca_cache_t* c, int32_t metric, const void* fresh, const double* t_target,
                                  const float* tau, const uint8_t* dev_active_mask, void* out_pred, float* dev_err,
                                  uint8_t* dev_accept, double* dev_sums, void* stream, const SelectArgs* sel = nullptr) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (metric < SPECA_METRIC_L2 || metric > SPECA_METRIC_COSINE)
        return fail(c, SPECA_ERR_INVALID_ARG, "verify: unknown metric %d", metric);
    const bool partial = dev_sums != nullptr;
    if (fresh == nullptr || t_target == nullptr || (!partial && (tau == nullptr || dev_err == nullptr || dev_accept == nullptr)))
        return fail(c, SPECA_ERR_INVALID_ARG, "verify: null argument");
    if (reinterpret_cast<uintptr_t>(dev_sums) % sizeof(double) != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "verify: dev_sums not aligned");
    if (c->pending) return fail(c, SPECA_ERR_STATE, "verify: a reference step is open (commit it first)");
    const size_t esz = elem_size(c);
    if (reinterpret_cast<uintptr_t>(fresh) % esz != 0 || reinterpret_cast<uintptr_t>(out_pred) % esz != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "verify: fresh / out_pred not aligned to the element size");
    if (reinterpret_cast<uintptr_t>(dev_err) % sizeof(float) != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "verify: dev_err not aligned");
    VerifyParams p;
    std::memset(&p, 0, sizeof p);
    bool any_sample = false;
    int v_max = 0;
    for (int b = 0; b < c->B; ++b) {
        if (!std::isfinite(t_target[b])) return fail(c, SPECA_ERR_INVALID_ARG, "verify: t_target[%d] not finite", b);
        if (!partial && std::isnan(tau[b])) return fail(c, SPECA_ERR_INVALID_ARG, "verify: tau[%d] is NaN", b);
        int order;
        forecast_coefficients(c, b, t_target[b], &order, p.coef[b]);
        if (order < 0 && dev_active_mask == nullptr)
            return fail(c, SPECA_ERR_STATE, "verify: sample %d has no committed reference", b);
        p.order[b] = static_cast<int8_t>(order);
        p.tau[b] = partial ? 0.f : tau[b];
        any_sample |= order >= 0;
        v_max = order > v_max ? order : v_max;
    }
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    // No sample has a table: nothing to verify. The fused form still launches, so that the kernel's
    // early exit writes the next mask.
    if (!any_sample && sel == nullptr) return SPECA_OK;
    const Layout& L = c->L;
    const SegDesc& s0 = L.segs[static_cast<size_t>(c->verify_entry) * c->B];
    const uint32_t te = verify_tile_elems(c->dtype, v_max);
    // the entry's B tables follow one another in the arena, one table (max_order + 1 planes) apart
    p.plane0_off = s0.plane0_off;
    p.sample_pitch = s0.plane_stride * static_cast<uint64_t>(c->m + 1);
    p.plane_stride = s0.plane_stride;
    p.io_pitch = static_cast<uint64_t>(s0.n_elems) * esz;
    p.arena = c->arena;
    p.dev_mask = dev_active_mask;
    p.weighted = c->layout == SPECA_LAYOUT_HISTORY ? 1 : 0;
    p.fresh = static_cast<const char*>(fresh);
    p.out_pred = static_cast<char*>(out_pred);
    p.err = dev_err;
    p.accept = dev_accept;
    p.partials = reinterpret_cast<float*>(c->arena + L.partials_off);
    p.ticket = reinterpret_cast<uint32_t*>(c->arena + L.ticket_off);
    p.raw_sums = dev_sums;
    if (sel != nullptr) {
        p.sel_active = sel->active;
        p.sel_spec = sel->spec_count;
        p.sel_idx = sel->idx;
        p.sel_n = sel->n_active;
        p.sel_kmax = sel->k_max;
        p.sel_group = sel->group;
    }
    p.n_elems = s0.n_elems;
    p.tiles_per_sample = (s0.n_elems + te - 1) / te;
    p.units_per_sample = (p.tiles_per_sample + c->cluster - 1) / c->cluster;
    p.batch = c->B;
    p.metric = metric;
    p.eps = c->eps;
    const uint64_t units = static_cast<uint64_t>(p.units_per_sample) * c->B;
    int grid = c->grid_verify;
    if (units * c->cluster < static_cast<uint64_t>(grid)) grid = static_cast<int>(units) * c->cluster;
    cudaError_t ce = launch_verify(p, c->dtype, grid, c->cluster, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "verify launch");
    c->launches += 1;
    c->stats.verify_launches += 1;
    return SPECA_OK;
}

speca_status_t speca_verify_metric(speca_cache_t* c, int32_t metric, const void* fresh, const double* t_target,
                                   const float* tau, const uint8_t* dev_active_mask, void* out_pred, float* dev_err,
                                   uint8_t* dev_accept, void* stream) {
    return verify_impl(c, metric, fresh, t_target, tau, dev_active_mask, out_pred, dev_err, dev_accept, nullptr, stream);
}

speca_status_t speca_verify_select(speca_cache_t* c, int32_t metric, const void* fresh, const double* t_target,
                                   const float* tau, const uint8_t* dev_active_mask, uint8_t* dev_next_active_mask,
                                   void* out_pred, float* dev_err, uint8_t* dev_accept, int32_t k_max, int32_t group,
                                   int32_t* dev_spec_count, int32_t* dev_active_idx, int32_t* dev_n_active, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (dev_active_mask == nullptr || dev_next_active_mask == nullptr || dev_spec_count == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "verify_select: null argument");
    const uintptr_t a = reinterpret_cast<uintptr_t>(dev_active_mask), b = reinterpret_cast<uintptr_t>(dev_next_active_mask);
    if (a < b + static_cast<uintptr_t>(c->B) && b < a + static_cast<uintptr_t>(c->B))
        return fail(c, SPECA_ERR_INVALID_ARG, "verify_select: the next mask must not overlap this step's mask");
    if (k_max < 1 || group < 1 || c->B % group != 0)
        return fail(c, SPECA_ERR_INVALID_ARG, "verify_select: k_max >= 1 and group must divide the batch");
    if (reinterpret_cast<uintptr_t>(dev_spec_count) % 4 != 0 || reinterpret_cast<uintptr_t>(dev_active_idx) % 4 != 0 ||
        reinterpret_cast<uintptr_t>(dev_n_active) % 4 != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "verify_select: int32 buffers must be 4-byte aligned");
    const SelectArgs sel = {k_max, group, dev_spec_count, dev_next_active_mask, dev_active_idx, dev_n_active};
    return verify_impl(c, metric, fresh, t_target, tau, dev_active_mask, out_pred, dev_err, dev_accept, nullptr, stream, &sel);
}

speca_status_t speca_verify_partial(speca_cache_t* c, int32_t metric, const void* fresh, const double* t_target,
                                    const uint8_t* dev_active_mask, void* out_pred, double* dev_sums, void* stream) {
    if (c != nullptr && dev_sums == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "verify_partial: null dev_sums");
    return verify_impl(c, metric, fresh, t_target, nullptr, dev_active_mask, out_pred, nullptr, nullptr, dev_sums, stream);
}

speca_status_t speca_verify_decide(int32_t metric, const double* dev_sums, int32_t batch, const float* tau, float eps,
                                   const uint8_t* dev_active_mask, float* dev_err, uint8_t* dev_accept, void* stream) {
    if (dev_sums == nullptr || tau == nullptr || dev_err == nullptr || dev_accept == nullptr) return SPECA_ERR_INVALID_ARG;
    if (metric < SPECA_METRIC_L2 || metric > SPECA_METRIC_COSINE) return SPECA_ERR_INVALID_ARG;
    if (batch < 1 || batch > SPECA_MAX_BATCH) return SPECA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(dev_sums) % sizeof(double) != 0 || reinterpret_cast<uintptr_t>(dev_err) % sizeof(float) != 0)
        return SPECA_ERR_ALIGNMENT;
    DecideParams q;
    std::memset(&q, 0, sizeof q);
    q.eps = eps > 0.f ? static_cast<double>(eps) : 1e-8;
    for (int b = 0; b < batch; ++b) {
        if (std::isnan(tau[b])) return SPECA_ERR_INVALID_ARG;
        q.tau[b] = tau[b];
    }
    if (cudaGetLastError() != cudaSuccess) return SPECA_ERR_CUDA;  // an earlier error, reported once
    cudaError_t ce = launch_decide(metric, dev_sums, batch, q, dev_active_mask, dev_err, dev_accept,
                                   static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) (void)cudaGetLastError();
    return ce == cudaSuccess ? SPECA_OK : SPECA_ERR_CUDA;
}

speca_status_t speca_select_adaptive(speca_cache_t* c, const uint8_t* dev_accept, int32_t k_max, int32_t group,
                                     int32_t* dev_spec_count, uint8_t* dev_active_mask, int32_t* dev_active_idx,
                                     int32_t* dev_n_active, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (dev_accept == nullptr || dev_spec_count == nullptr || dev_active_mask == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "select: null argument");
    if (k_max < 1 || group < 1 || c->B % group != 0)
        return fail(c, SPECA_ERR_INVALID_ARG, "select: k_max >= 1 and group must divide the batch");
    if (reinterpret_cast<uintptr_t>(dev_spec_count) % 4 != 0 || reinterpret_cast<uintptr_t>(dev_active_idx) % 4 != 0 ||
        reinterpret_cast<uintptr_t>(dev_n_active) % 4 != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "select: int32 buffers must be 4-byte aligned");
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    cudaError_t ce = launch_select(dev_accept, k_max, group, c->B, dev_spec_count, dev_active_mask, dev_active_idx,
                                   dev_n_active, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "select launch");
    c->launches += 1;
    c->stats.select_launches += 1;
    return SPECA_OK;
}

speca_status_t speca_activate(speca_cache_t* c, const uint8_t* host_sample_mask, int32_t* dev_spec_count,
                              uint8_t* dev_active_mask, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (dev_spec_count == nullptr || dev_active_mask == nullptr)
        return fail(c, SPECA_ERR_INVALID_ARG, "activate: null argument");
    if (reinterpret_cast<uintptr_t>(dev_spec_count) % 4 != 0)
        return fail(c, SPECA_ERR_ALIGNMENT, "activate: dev_spec_count must be 4-byte aligned");
    uint64_t bits = 0;
    for (int b = 0; b < c->B; ++b)
        if (host_sample_mask == nullptr || host_sample_mask[b] != 0) bits |= (uint64_t(1) << b);
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    speca_status_t st = check_sticky(c);
    if (st != SPECA_OK) return st;
    cudaError_t ce = launch_activate(bits, c->B, dev_spec_count, dev_active_mask, static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) return cuda_fail(c, ce, "activate launch");
    c->launches += 1;
    c->stats.activate_launches += 1;
    return SPECA_OK;
}

double speca_tau(double tau0, double beta, double t, double T) {
    if (!(T > 0.0)) return std::numeric_limits<double>::quiet_NaN();
    return tau0 * std::pow(beta, (T - t) / T);
}

speca_status_t speca_cache_state(const speca_cache_t* c, int32_t* host_n_refs, double* host_t_last) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    for (int b = 0; b < c->B; ++b) {
        if (host_n_refs != nullptr) host_n_refs[b] = c->n_refs[b];
        if (host_t_last != nullptr) host_t_last[b] = c->t_hist[b][0];
    }
    return SPECA_OK;
}

speca_status_t speca_cache_get_history(const speca_cache_t* c, int32_t* host_n_refs, double* host_t_hist) {
    if (c == nullptr || host_n_refs == nullptr || host_t_hist == nullptr) return SPECA_ERR_INVALID_ARG;
    for (int b = 0; b < c->B; ++b) {
        host_n_refs[b] = c->n_refs[b];
        for (int i = 0; i <= SPECA_MAX_ORDER; ++i) host_t_hist[b * (SPECA_MAX_ORDER + 1) + i] = c->t_hist[b][i];
    }
    return SPECA_OK;
}

speca_status_t speca_cache_set_history(speca_cache_t* c, const int32_t* host_n_refs, const double* host_t_hist) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    if (host_n_refs == nullptr || host_t_hist == nullptr) return fail(c, SPECA_ERR_INVALID_ARG, "set_history: null argument");
    if (c->pending) return fail(c, SPECA_ERR_STATE, "set_history while a reference step is open");
    for (int b = 0; b < c->B; ++b) {
        if (host_n_refs[b] < 0) return fail(c, SPECA_ERR_INVALID_ARG, "set_history: n_refs[%d] negative", b);
        const int defined = host_n_refs[b] < SPECA_MAX_ORDER + 1 ? host_n_refs[b] : SPECA_MAX_ORDER + 1;
        for (int i = 0; i < defined; ++i)
            if (!std::isfinite(host_t_hist[b * (SPECA_MAX_ORDER + 1) + i]))
                return fail(c, SPECA_ERR_INVALID_ARG, "set_history: time %d of sample %d not finite", i, b);
    }
    for (int b = 0; b < c->B; ++b) {
        c->n_refs[b] = host_n_refs[b];
        for (int i = 0; i <= SPECA_MAX_ORDER; ++i) c->t_hist[b][i] = host_t_hist[b * (SPECA_MAX_ORDER + 1) + i];
    }
    return SPECA_OK;
}

speca_status_t speca_cache_plane(const speca_cache_t* c, int32_t entry, int32_t sample, void** plane0,
                                 size_t* plane_stride_bytes) {
    if (c == nullptr || plane0 == nullptr || plane_stride_bytes == nullptr) return SPECA_ERR_INVALID_ARG;
    if (entry < 0 || entry >= c->n_entries || sample < 0 || sample >= c->B) return SPECA_ERR_INVALID_ARG;
    const SegDesc& s = c->L.segs[static_cast<size_t>(entry) * c->B + sample];
    *plane0 = c->arena + s.plane0_off;
    *plane_stride_bytes = s.plane_stride;
    return SPECA_OK;
}

speca_status_t speca_forecast_weights(int32_t layout, int32_t basis, int32_t max_order, int32_t n_refs,
                                      const double* t_hist, double t_target, int32_t* out_order, float* out_coef) {
    if (t_hist == nullptr || out_order == nullptr || out_coef == nullptr) return SPECA_ERR_INVALID_ARG;
    if (layout != SPECA_LAYOUT_TABLES && layout != SPECA_LAYOUT_HISTORY) return SPECA_ERR_INVALID_ARG;
    if (basis != SPECA_BASIS_TAYLOR && basis != SPECA_BASIS_NEWTON && basis != SPECA_BASIS_ADAMS_BASHFORTH)
        return SPECA_ERR_INVALID_ARG;
    if (max_order < 0 || max_order > SPECA_MAX_ORDER || n_refs < 0 || !std::isfinite(t_target)) return SPECA_ERR_INVALID_ARG;
    speca_cache tmp;
    tmp.m = max_order;
    tmp.basis = basis;
    tmp.layout = layout;
    tmp.n_refs[0] = n_refs;
    const int known = n_refs < max_order + 1 ? n_refs : max_order + 1;
    for (int i = 0; i <= SPECA_MAX_ORDER; ++i)
        tmp.t_hist[0][i] = i < known ? t_hist[i] : std::numeric_limits<double>::quiet_NaN();
    for (int i = 0; i < known; ++i)
        if (!std::isfinite(t_hist[i])) return SPECA_ERR_INVALID_ARG;
    int order = -1;
    float coef[kCoef] = {};
    forecast_coefficients(&tmp, 0, t_target, &order, coef);
    *out_order = order;
    for (int i = 0; i < kCoef; ++i) out_coef[i] = coef[i];
    return SPECA_OK;
}

speca_status_t speca_cache_next_slot(const speca_cache_t* c, int32_t entry, int32_t sample, void** out) {
    if (c == nullptr || out == nullptr) return SPECA_ERR_INVALID_ARG;
    if (c->layout != SPECA_LAYOUT_HISTORY) return SPECA_ERR_UNSUPPORTED;
    if (entry < 0 || entry >= c->n_entries || sample < 0 || sample >= c->B) return SPECA_ERR_INVALID_ARG;
    const SegDesc& s = c->L.segs[static_cast<size_t>(entry) * c->B + sample];
    *out = c->arena + s.plane0_off + static_cast<size_t>(c->n_refs[sample] % (c->m + 1)) * s.plane_stride;
    return SPECA_OK;
}

speca_status_t speca_cache_stats(const speca_cache_t* c, speca_cache_stats_t* out) {
    if (c == nullptr || out == nullptr) return SPECA_ERR_INVALID_ARG;
    *out = c->stats;
    return SPECA_OK;
}

speca_status_t speca_cache_check(speca_cache_t* c, void* stream) {
    if (c == nullptr) return SPECA_ERR_INVALID_ARG;
    DeviceGuard guard(c->device);
    if (!guard.ok) return fail(c, SPECA_ERR_CUDA, "cudaSetDevice failed");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t ce = cudaStreamSynchronize(s);
    if (ce != cudaSuccess) return cuda_fail(c, ce, "check: stream");
    uint32_t* word = reinterpret_cast<uint32_t*>(c->arena + c->L.ticket_off) + kGaveUpWord;
    uint32_t gave_up = 0;
    ce = cudaMemcpyAsync(&gave_up, word, sizeof gave_up, cudaMemcpyDeviceToHost, s);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(s);
    if (ce != cudaSuccess) return cuda_fail(c, ce, "check: read-back");
    if (gave_up != 0) {
        ce = cudaMemsetAsync(word, 0, sizeof gave_up, s);
        if (ce != cudaSuccess) return cuda_fail(c, ce, "check: clear");
        return fail(c, SPECA_ERR_CUDA, "a staged copy never landed: results since the last check are incomplete");
    }
    return SPECA_OK;
}

speca_status_t speca_cache_launch_count(const speca_cache_t* c, uint64_t* out) {
    if (c == nullptr || out == nullptr) return SPECA_ERR_INVALID_ARG;
    *out = c->launches;
    return SPECA_OK;
}

const char* speca_status_string(speca_status_t status) {
    switch (status) {
        case SPECA_OK: return "ok";
        case SPECA_ERR_INVALID_ARG: return "invalid argument";
        case SPECA_ERR_SHAPE: return "shape outside supported limits";
        case SPECA_ERR_ALIGNMENT: return "pointer alignment";
        case SPECA_ERR_STATE: return "call order violated";
        case SPECA_ERR_ZERO_GAP: return "reference time repeats (zero gap)";
        case SPECA_ERR_NOMEM: return "out of memory / arena too small";
        case SPECA_ERR_CUDA: return "CUDA error";
        case SPECA_ERR_UNSUPPORTED: return "unsupported device or feature";
    }
    return "unknown status";
}

const char* speca_last_error(const speca_cache_t* c) { return c == nullptr ? "" : c->last_error; }

const char* speca_version(void) { return "speca-b200 0.1 (sm_100a)"; }

}  // extern "C"
