// Internal declarations shared by the host dispatch (speca_api.cpp) and the kernels
// (speca_kernels.cu). Not part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "speca.h"

namespace speca {

// A tile is the unit a CTA picks up from the flattened work list: a fixed number of bytes of one
// plane of one (entry, sample) table. Each stream kernel shape has its own tile size; the arena
// holds one tile-prefix table per size in kTileSizes.
constexpr uint32_t kTileSizes[] = {4096, 8192, 16384, 32768};
constexpr int kNumTileSizes = 4;
constexpr int kThreads = 256;       // verify kernel CTA size
// Launch shape of the verify kernel: 32-byte vectors per thread and plane for orders 0-2 (orders 3-4
// always hold one), the CTAs per SM the registers are capped for, and the cluster size.
#ifndef SPECA_VERIFY_U
#define SPECA_VERIFY_U 2
#endif
#ifndef SPECA_VERIFY_MINB
#define SPECA_VERIFY_MINB 2
#endif
#ifndef SPECA_VERIFY_CLUSTER
#define SPECA_VERIFY_CLUSTER 4
#endif
__host__ __device__ constexpr int verify_vectors(int v) { return v <= 2 ? SPECA_VERIFY_U : 1; }
// Tile of the verify kernel compiled for order v (the highest order among the launch's samples):
// 256 threads x verify_vectors(v) x 32 bytes per plane.
__host__ __device__ constexpr uint32_t verify_tile_bytes(int v) { return 8192u * verify_vectors(v); }
constexpr int kMaxClusters = 1024;  // upper bound on verify clusters (reduction scratch rows)
// Arrival counter of the verify kernel, zero between launches. (The word after it is the bulk
// path's gave-up flag in a cache's arena.)
constexpr int kVerifyTickets = 1;

inline int tile_size_index(uint32_t tile_bytes) {
    for (int i = 0; i < kNumTileSizes; ++i)
        if (kTileSizes[i] == tile_bytes) return i;
    return -1;
}

// One (entry, sample) table. Segments are ordered entry-major, sample-minor: seg = e * B + b.
struct SegDesc {
    uint64_t plane0_off;    // byte offset of plane 0 from the arena base (4 KB aligned)
    uint64_t plane_stride;  // bytes between consecutive planes (multiple of 4096)
    uint64_t io_off;        // byte offset of this sample's row inside the entry's [B, N_e, D] tensor
    uint32_t n_elems;       // N_e * D
    uint16_t entry;
    uint16_t sample;
};
static_assert(sizeof(SegDesc) == 32, "SegDesc layout");

// Per-sample scalars of a launch: Horner multipliers or reciprocal gaps (SPECA_MAX_ORDER of them), or the
// weights of a raw-feature cache (one per plane).
constexpr int kCoef = SPECA_MAX_ORDER + 1;

// Arguments of the streaming kernels (update, forecast), passed by value as one kernel parameter.
struct StreamParams {
    const SegDesc* segs;         // all segments of the cache
    const uint32_t* tile_start;  // [n_segs + 1] prefix of tiles per segment, for this path's tile size
    char* arena;
    const uint8_t* dev_mask;  // device, per sample, may be null
    uint32_t seg_lo, seg_hi;  // segment range this launch covers
    uint32_t tile_lo, tile_hi;
    uint32_t* err_flag;  // device word the bulk path sets if a wait gives up
    // update:   order = highest plane written (v_new), coef[b][i] = 1 / gap_i
    // forecast: order = highest plane read (v),        coef[b][i] = Horner multiplier of level i+1
    // order < 0: sample is skipped
    // A cache that keeps raw features (SPECA_LAYOUT_HISTORY):
    // update:   order = 0, slot[b] = plane that receives the feature
    // forecast: weighted = 1, coef[b][i] = weight of physical plane i (i <= order): out = sum_i coef_i * plane_i
    // update only, optional: samples (bits of act_bits) to re-arm for speculation in the same launch
    int32_t* act_spec;
    uint8_t* act_active;
    uint64_t act_bits;
    int8_t order[SPECA_MAX_BATCH];
    uint8_t slot[SPECA_MAX_BATCH];
    int32_t weighted;
    float coef[SPECA_MAX_BATCH][kCoef];
    void* io[SPECA_MAX_ENTRIES];  // per entry: feature (update) or output (forecast); null = skip
};

// Arguments of the fused reference step: Eq. 3 for the samples that were fully computed and, in the
// same pass over the tables, Eq. 2 at the next speculative time for them (from the planes just
// written) and for the samples that keep speculating (from their unchanged planes).
struct FusedParams {
    StreamParams up;                  // the update half: io = features, order / coef as for an update
    const uint8_t* fc_mask;           // device, per sample, may be null: consulted for samples NOT updated here
    int8_t fc_order[SPECA_MAX_BATCH]; // order of the forecast after this step (-1: nothing to forecast)
    int32_t n_targets;                // K speculative times forecast in this pass (1..SPECA_MAX_HORIZON)
    int32_t batch;
    float fc_coef[SPECA_MAX_HORIZON][SPECA_MAX_BATCH][kCoef];  // per target: Horner multipliers relative to the history after this step
    void* out[SPECA_MAX_ENTRIES];     // per entry: [K, B, N_e, D] forecast output; null = update only
};

// Arguments of the multi-horizon forecast: K targets evaluated from one read of the table.
struct MultiParams {
    const SegDesc* segs;
    const uint32_t* tile_start;  // prefix table for multi_tile_bytes()
    char* arena;
    const uint8_t* dev_mask;
    uint32_t seg_lo, seg_hi;
    uint32_t tile_lo, tile_hi;
    int32_t n_targets;                // K
    int32_t weighted;                 // raw-feature cache: coef = weights of the physical planes
    int8_t order[SPECA_MAX_BATCH];
    float coef[SPECA_MAX_HORIZON][SPECA_MAX_BATCH][kCoef];  // Horner multipliers (or plane weights) per target
    void* io[SPECA_MAX_ENTRIES];      // per entry: [K, B, N_e, D] output; null = skip
};

// Arguments of the summed forecast: out = base + sum over a list of equally shaped entries.
struct SumParams {
    const SegDesc* segs;  // all segments of the cache
    char* arena;
    const uint8_t* dev_mask;
    const char* base;     // [B, n_elems] or null
    char* out;            // [B, n_elems]
    uint32_t n_elems;     // per sample (common to the listed entries)
    uint32_t tiles_per_sample;
    int32_t batch;
    int32_t n_ids;
    int32_t weighted;  // raw-feature cache: coef = weights of the physical planes
    int8_t order[SPECA_MAX_BATCH];
    float coef[SPECA_MAX_BATCH][kCoef];
    uint16_t ids[SPECA_MAX_ENTRIES];  // entries to add, in this order
};

// Arguments of the fused forecast + relative-L2 kernel over the verification entry.
struct VerifyParams {
    // The verification entry's B tables are laid out evenly: sample b's plane 0 starts at
    // arena + plane0_off + b * sample_pitch, its planes are plane_stride bytes apart, and its row of
    // the [B, N_v, D] tensors (fresh, out_pred) starts b * io_pitch bytes in.
    uint64_t plane0_off, sample_pitch, plane_stride, io_pitch;
    char* arena;
    const uint8_t* dev_mask;
    const char* fresh;  // [B, N_v, D]
    char* out_pred;     // may be null
    float* err;
    uint8_t* accept;
    float* partials;     // [B][n_clusters][values of the metric: 2, or 3 for cosine]
    uint32_t* ticket;    // arrival counter, zero between launches
    double* raw_sums;    // [B][4] or null: write the combined running values instead of err / accept
    // fused per-sample continuation (speca_verify_select); sel_active == null: not fused
    uint8_t* sel_active;  // receives the next active mask once every decision is final; must not alias dev_mask
    int32_t* sel_spec;
    int32_t* sel_idx;
    int32_t* sel_n;
    int32_t sel_kmax, sel_group;
    uint32_t n_elems;    // per sample
    uint32_t tiles_per_sample;
    uint32_t units_per_sample;  // ceil(tiles_per_sample / cluster size): host-side grid sizing only
    int32_t batch;
    int32_t metric;  // speca_metric_t
    double eps;
    int32_t weighted;  // raw-feature cache: coef[b][i] = weight of physical plane i instead of Horner multipliers
    int8_t order[SPECA_MAX_BATCH];
    float coef[SPECA_MAX_BATCH][kCoef];
    float tau[SPECA_MAX_BATCH];
};

struct DecideParams {
    double eps;
    float tau[SPECA_MAX_BATCH];
};

// Launchers. `dtype` is a speca_dtype_t. All enqueue on `stream` and return the launch status.
cudaError_t launch_update(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream);
cudaError_t launch_forecast(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream);
cudaError_t launch_update_forecast(const FusedParams& p, int dtype, int grid, cudaStream_t stream);
int fused_ctas_per_sm(int order, bool raw_features, int dtype, int n_targets);
cudaError_t launch_verify(const VerifyParams& p, int dtype, int grid, int cluster, cudaStream_t stream);
cudaError_t launch_select(const uint8_t* accept, int32_t k_max, int32_t group, int32_t batch, int32_t* spec_count,
                          uint8_t* active, int32_t* idx, int32_t* n_active, cudaStream_t stream);
cudaError_t launch_activate(uint64_t mask_bits, int32_t batch, int32_t* spec_count, uint8_t* active,
                            cudaStream_t stream);

// Tile size and designed CTAs per SM of the stream kernel a path uses for update / forecast.
uint32_t stream_tile_bytes(int path, bool update);
int stream_ctas_per_sm(int path, bool update, int dtype, int order);
// Multi-horizon forecast kernel: tile size, designed CTAs per SM, launcher.
uint32_t multi_tile_bytes();
int multi_ctas_per_sm(int n_targets);
cudaError_t launch_forecast_multi(const MultiParams& p, int dtype, int batch, int grid, cudaStream_t stream);
cudaError_t launch_decide(int metric, const double* sums, int batch, const DecideParams& q, const uint8_t* mask, float* err,
                          uint8_t* accept, cudaStream_t stream);
uint32_t sum_tile_bytes();
int sum_ctas_per_sm();
cudaError_t launch_forecast_sum(const SumParams& p, int dtype, int grid, cudaStream_t stream);
// Clusters of the verify kernel that fit on the current device at once.
int max_resident_verify_clusters(int dtype, int order, int cluster);

inline uint32_t verify_tile_elems(int dtype, int v) { return verify_tile_bytes(v) / (dtype == SPECA_BF16 ? 2u : 4u); }

}  // namespace speca
