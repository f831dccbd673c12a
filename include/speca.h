/*
 * speca.h -- C ABI of the SpeCa speculative feature-cache hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel arithmetic of "forecast-then-verify" sampling
 * for diffusion transformers (SpeCa, arXiv 2509.11628):
 *
 *   - the per-layer derivative table that the TaylorSeer draft model keeps (Eq. 3, Section 3.3),
 *     rewritten in place at every fully computed reference step,
 *   - the Taylor extrapolation of every cached block output to a speculative step (Eq. 2),
 *   - the relative L2 error between the forecast and the freshly computed feature of the
 *     verification layer, reduced to one accept/reject decision per sample (Eq. 4 and the
 *     sequential validation rule of Section 3.4.2),
 *   - per-sample masks so that rejected samples of a batch stop forecasting (the
 *     sample-adaptive computation allocation of Sections 1 and 4).
 *
 * Conventions shared by every entry point
 *   - Every function returns a speca_status_t. Nothing throws, aborts or prints.
 *   - "host" pointers are read during the call and may be freed on return. "device" pointers
 *     must be valid on the cache's CUDA device until the work enqueued on `stream` has run.
 *   - All device work is enqueued on the caller's stream (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and the call returns without synchronising.
 *   - Arguments are validated on the host before anything is launched: a call that returns an
 *     error has enqueued nothing and has not changed the cache's state.
 *   - Tensors are dense, row-major [B, N_e, D] in the cache's storage dtype; sample b of an entry
 *     starts at element b*N_e*D. Device tensor pointers must be aligned to the element size;
 *     32-byte aligned rows (pointer and N_e*D*sizeof(element) multiples of 32) take the fast
 *     vector path, anything else a slower 16-byte or element-wise path with equal results.
 *   - The calls that enqueue work (update, forecast*, verify*, select, activate) neither allocate
 *     nor synchronise, so they may be issued while `stream` is being captured into a CUDA graph.
 *     Times, thresholds and host masks are folded into the kernel arguments at capture; a replay
 *     reads the device buffers (features, masks, counters) as they are then. The host-side history
 *     (update / commit_step / reset) advances at capture time only, not on replay.
 *   - A CUDA error that an earlier call on the thread left behind is reported once (SPECA_ERR_CUDA,
 *     "earlier CUDA error") by the next call that enqueues work, and cleared: a recoverable error
 *     (a rejected launch configuration, say) does not poison later calls, while an error that broke
 *     the context keeps coming back from the runtime itself.
 *   - A handle is not thread safe: use one handle from one host thread at a time.
 *   - There is no CPU fallback: without a usable CUDA device speca_cache_create fails.
 */
#ifndef SPECA_H_
#define SPECA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECA_MAX_ORDER   4     /* highest Taylor order m */
#define SPECA_MAX_BATCH   64    /* most samples B in one cache */
#define SPECA_MAX_ENTRIES 512   /* most cached tensors (block outputs) in one cache */
#define SPECA_MAX_HORIZON 8     /* most speculative steps one speca_forecast_multi call evaluates */

typedef struct speca_cache speca_cache_t; /* opaque, owned by the library */

typedef enum {
    SPECA_OK = 0,
    SPECA_ERR_INVALID_ARG = 1, /* null pointer, value out of range, non-finite time */
    SPECA_ERR_SHAPE = 2,       /* entry list / batch / order outside the supported limits */
    SPECA_ERR_ALIGNMENT = 3,   /* pointer not aligned as the call requires */
    SPECA_ERR_STATE = 4,       /* call order violated (forecast before an update, double update ...) */
    SPECA_ERR_ZERO_GAP = 5,    /* a reference time equals one it must differ from */
    SPECA_ERR_NOMEM = 6,       /* arena too small, or host allocation failed */
    SPECA_ERR_CUDA = 7,        /* a CUDA runtime call failed; see speca_last_error */
    SPECA_ERR_UNSUPPORTED = 8  /* device is not an sm_100 part, or feature not built */
} speca_status_t;

typedef enum { SPECA_F32 = 0, SPECA_BF16 = 1 } speca_dtype_t;

/*
 * Which polynomial basis the derivative table holds.
 *  SPECA_BASIS_TAYLOR  Eq. 2-3 as printed: plane i holds the i-th backward difference quotient
 *                      (Delta^i F / N^i on a uniform grid of spacing N), the forecast is
 *                      sum_i plane_i * x^i / i! with x = t_target - t_last. For non-uniform
 *                      reference times every quotient divides by the latest gap. Exact for
 *                      features that are polynomials of degree <= 1 in t.
 *  SPECA_BASIS_NEWTON  Newton divided differences over the true reference times, evaluated in
 *                      Newton form. Exact for polynomials of degree <= m at any gaps. Same
 *                      kernels, different host-computed scalars.
 *  SPECA_BASIS_ADAMS_BASHFORTH  The alternative draft model of the appendix's draft-model ablation
 *                      (named there without a formula). Tables as in the Taylor basis; the forecast
 *                      is F + x * sum_j b_j g_j with g_j the difference-quotient slope j references
 *                      back and b the textbook Adams-Bashforth coefficients of as many steps as
 *                      slopes are known (at most 4), which in Horner form over the planes is
 *                      F + x (D_1 + h/2 (D_2 + 5h/6 (D_3 + 9h/10 D_4))), h = the latest reference gap.
 *                      Same kernels again.
 */
typedef enum { SPECA_BASIS_TAYLOR = 0, SPECA_BASIS_NEWTON = 1, SPECA_BASIS_ADAMS_BASHFORTH = 2 } speca_basis_t;

/* Which kernel variant moves the data. Results are identical; only speed differs. */
typedef enum {
    SPECA_PATH_AUTO = 0,   /* library default: the fastest measured (currently WIDE) */
    SPECA_PATH_DIRECT = 1, /* 16-byte vector loads straight into registers, 256 threads x 4 deep */
    SPECA_PATH_BULK = 2,   /* cp.async.bulk (TMA) staging through a shared-memory ring */
    SPECA_PATH_WIDE = 3    /* 32-byte vector loads / stores, per-kernel launch shapes */
} speca_path_t;

/*
 * What the cache keeps per (entry, sample) in its max_order + 1 planes.
 * TABLES   the difference quotients of Eq. 3, rewritten at every reference step (the paper's derivative
 *          tables): an update reads the feature and the old planes and writes all planes.
 * HISTORY  the raw features of the last max_order + 1 references, in a ring: an update only copies the
 *          feature into the next plane (2 words per element instead of 2 * order + 2), and Eq. 3's
 *          differences are folded into per-plane weights on the host when a forecast is asked for:
 *          out = sum_i w_i * plane_i. Same Eq. 2-3 (and the same Newton / Adams-Bashforth readings), any
 *          gaps; the results differ from TABLES only in that no intermediate quotient is rounded to the
 *          storage type. Served by the default kernel path only (SPECA_PATH_AUTO / SPECA_PATH_WIDE).
 *          Accuracy: every forecast element is a correct rounding to the storage type of Eq. 2-3 evaluated
 *          in fp32 (within 4e-6 of the summed magnitudes of its terms). Because the forecast is rounded
 *          once from a combination of stored values, on a UNIFORM time grid with bf16 storage (weights are
 *          then ratios of small integers) a few per cent of the elements land exactly on a rounding tie,
 *          where an fp64 evaluation may pick the other neighbour; both are correct. The verification error
 *          computed on the library's forecast meets the 1e-4 bound; against an fp64 evaluation of the
 *          whole chain it can differ by up to 6e-3 of itself on such grids when the forecast offsets make
 *          the weights inexact in fp32 (with integer weights, and on uneven grids, the difference stays
 *          far below 1e-4).
 */
typedef enum {
    SPECA_LAYOUT_TABLES = 0,
    SPECA_LAYOUT_HISTORY = 1
} speca_layout_t;

/*
 * Error metric of the verification. Eq. 4 is the relative l2 error (the paper's default); the
 * appendix on error metrics also evaluates l1, l-infinity and cosine similarity, named there
 * without formulas. The forms used here (p = forecast, f = computed feature, all over one sample):
 *   L2      ||p - f||_2   / (||f||_2   + eps)
 *   L1      ||p - f||_1   / (||f||_1   + eps)
 *   LINF    ||p - f||_inf / (||f||_inf + eps)
 *   COSINE  1 - <p, f> / (||p||_2 ||f||_2 + eps)     (a distance: 0 = same direction)
 * In every case the sample is accepted iff the value is <= tau, and a NaN rejects.
 */
typedef enum {
    SPECA_METRIC_L2 = 0,
    SPECA_METRIC_L1 = 1,
    SPECA_METRIC_LINF = 2,
    SPECA_METRIC_COSINE = 3
} speca_metric_t;

typedef struct {
    int64_t tokens; /* N_e  >= 1 */
    int32_t dim;    /* D    >= 1 */
} speca_entry_desc_t;

typedef struct {
    int32_t n_entries;                 /* 1..SPECA_MAX_ENTRIES */
    const speca_entry_desc_t* entries; /* host; copied by speca_cache_create */
    int32_t batch;                     /* B, 1..SPECA_MAX_BATCH */
    int32_t max_order;                 /* m, 0..SPECA_MAX_ORDER (0 = plain cache reuse) */
    int32_t dtype;                     /* speca_dtype_t: storage type of tables, features, forecasts */
    int32_t basis;                     /* speca_basis_t */
    int32_t verify_entry;              /* index of the verification layer's entry; -1 = last entry */
    float eps;                         /* epsilon of Eq. 4; <= 0 selects the paper's 1e-8 */
    void* arena;                       /* device; caller-owned, 256-byte aligned (4 KB aligned for full speed:
                                          planes then start on 4 KB boundaries), lives as long as the handle */
    size_t arena_bytes;                /* >= speca_cache_arena_bytes() */
    int32_t device;                    /* CUDA device ordinal that owns the arena */
    int32_t path;                      /* speca_path_t */
    int32_t layout;                    /* speca_layout_t; 0 = the paper's derivative tables */
} speca_cache_config_t;

/*
 * Bytes of device memory a cache with this configuration needs (tables for every entry, sample
 * and order 0..m, plus a few KB of descriptors and reduction scratch). `arena`, `arena_bytes`
 * and `device` are ignored. Host only; touches no GPU.
 * Errors: INVALID_ARG (null), SHAPE (limits exceeded, sizes overflow).
 */
speca_status_t speca_cache_arena_bytes(const speca_cache_config_t* cfg, size_t* out_bytes);

/*
 * Build a cache over the caller's arena (Section 3.3: one derivative table per cached block
 * output). Writes the descriptor tables into the arena (synchronously) and returns a handle in
 * *out. The arena's table region is not cleared: planes are defined only once an update has
 * written them. Errors: INVALID_ARG, SHAPE, ALIGNMENT (arena), NOMEM (arena too small),
 * CUDA, UNSUPPORTED (device is not compute capability 10.x).
 */
speca_status_t speca_cache_create(const speca_cache_config_t* cfg, speca_cache_t** out);

/* Waits for the device to finish work that uses the handle, then frees host state. The arena
 * stays with the caller. NULL is accepted. Returns SPECA_ERR_CUDA if the device reported an error
 * or a SPECA_PATH_BULK kernel gave up waiting for a copy (its results are then incomplete). */
speca_status_t speca_cache_destroy(speca_cache_t* cache);

/* Forget the reference history of the samples with host_sample_mask[b] != 0 (NULL = all):
 * their next update is a first update. Host state only. */
speca_status_t speca_cache_reset(speca_cache_t* cache, const uint8_t* host_sample_mask);

/*
 * Reference step, Eq. 3 / workflow step 1 of Section 3.2: fold freshly computed features into
 * the derivative tables, in place.
 *   feats            host array of n_entries device pointers; feats[e] = [B, N_e, D] feature of
 *                    entry e at the new reference time, NULL = entry e is not part of this call
 *                    (a model hands over one block at a time; any subset per call is fine).
 *   t_ref            host, B doubles: the reference time of each sample (any monotone or
 *                    non-monotone coordinate; only differences are used).
 *   host_sample_mask host, B bytes, NULL = all: samples that were fully computed. Other samples'
 *                    tables are neither read nor written.
 * For sample b with r = number of committed references: plane 0 <- f; for i < min(m, r):
 * plane i+1 <- (new plane i - old plane i) / gap_i, the chain carried in fp32 and each plane
 * rounded once to the storage dtype. gap_i is t_ref - t_last (TAYLOR) or t_ref - (i-th previous
 * reference time) (NEWTON).
 * A SPECA_LAYOUT_HISTORY cache does none of this arithmetic here: it copies f into the plane after the
 * latest one, plane (references mod (m + 1)), and leaves the differencing to the forecast's weights
 * (nothing at all is copied for an entry whose feats pointer is the address speca_cache_next_slot
 * gave); the checks, states and errors are the same.
 * All entries of one reference step must be updated (each exactly once per masked sample)
 * before speca_cache_commit_step; t_ref and the mask must be the same in all of those calls.
 * Errors: INVALID_ARG, ALIGNMENT, ZERO_GAP, STATE (entry updated twice in one step, or
 * t_ref / mask differ from the step's first call), CUDA.
 */
speca_status_t speca_cache_update(speca_cache_t* cache, const void* const* feats, const double* t_ref,
                                  const uint8_t* host_sample_mask, void* stream);

/*
 * speca_cache_update that also re-arms the masked samples for speculation, as speca_activate would
 * (dev_active_mask[b] = 1, dev_spec_count[b] = 0 for every masked sample), in the same launch: after a
 * reference step the samples that took it may speculate again. When the call copies nothing (features
 * already in place, or an empty mask) the re-arming runs as a launch of its own. Both device buffers are
 * required. Errors: those of speca_cache_update and speca_activate.
 */
speca_status_t speca_cache_update_activate(speca_cache_t* cache, const void* const* feats, const double* t_ref,
                                           const uint8_t* host_sample_mask, int32_t* dev_spec_count,
                                           uint8_t* dev_active_mask, void* stream);

/*
 * A whole reference step and the first speculative step after it in ONE pass over the tables
 * (Section 3.2, workflow steps 1 and 2; Eq. 3 followed by Eq. 2): exactly
 *     speca_cache_update(_activate)(feats, t_ref, host_sample_mask);  speca_cache_commit_step();
 *     speca_forecast(t_target, dev_active_mask, outs);
 * bit for bit, but the forecast of a sample that takes the reference step is evaluated from the planes
 * the update has just formed (rounded to the storage dtype, as a forecast launch would read them), so
 * the table is not read again: 2v + 3 words per element instead of (2v + 2) + (v + 2). A reference
 * step is always followed by a speculative one, so this is the normal way to take it.
 *   feats            every entry's feature (no NULLs: the call is the whole step and commits it).
 *   t_ref, host_sample_mask   as in speca_cache_update.
 *   t_target         host, B doubles: the speculative time to forecast, per sample.
 *   dev_active_mask  device, B bytes, NULL = all: consulted only for samples that do NOT take this
 *                    reference step (they are forecast from their unchanged tables if non-zero);
 *                    samples that take it are always forecast. The kernel does not write it.
 *   outs             per entry: forecast output, or NULL for an entry that is only updated (the
 *                    verification entry, whose forecast comes out of speca_verify's out_pred).
 *   dev_spec_count, dev_rearm_mask   both or neither: as speca_cache_update_activate, the samples
 *                    of host_sample_mask are marked active in dev_rearm_mask and their counters
 *                    cleared (dev_rearm_mask may be the buffer dev_active_mask names).
 * A cache that keeps raw features (SPECA_LAYOUT_HISTORY) takes the same call: the feature is copied into
 * its ring plane and the weighted sum is formed with it still in registers, v + 3 words per element
 * instead of 2 + (v + 2); an entry given as SPECA_FEATURE_IN_PLACE, or as the pointer speca_cache_next_slot
 * returned, is not copied and only forecast. The default kernel path only. On error nothing is
 * enqueued and the history is unchanged. Errors: INVALID_ARG, ALIGNMENT, ZERO_GAP, STATE (a reference
 * step is open; or a sample has no reference and no device mask is given), UNSUPPORTED, CUDA.
 */
speca_status_t speca_cache_update_forecast(speca_cache_t* cache, const void* const* feats, const double* t_ref,
                                           const uint8_t* host_sample_mask, const double* t_target,
                                           const uint8_t* dev_active_mask, void* const* outs, int32_t* dev_spec_count,
                                           uint8_t* dev_rearm_mask, void* stream);

/*
 * The same with K = n_targets speculative times at once (Fig. 1: the draft predicts the next steps
 * from one reference): exactly speca_cache_update(_activate) + speca_cache_commit_step +
 * speca_forecast_multi, bit for bit, in one pass: 2v + 2 + K words per element instead of
 * (2v + 2) + (v + 1 + K). t_target is K x B doubles (target-major) and outs[e] a [K, B, N_e, D] tensor,
 * as in speca_forecast_multi; everything else as above. n_targets = 1 is speca_cache_update_forecast.
 * Errors: as above, and INVALID_ARG for n_targets outside 1..SPECA_MAX_HORIZON.
 */
speca_status_t speca_cache_update_forecast_multi(speca_cache_t* cache, const void* const* feats, const double* t_ref,
                                                 const uint8_t* host_sample_mask, int32_t n_targets,
                                                 const double* t_target, const uint8_t* dev_active_mask,
                                                 void* const* outs, int32_t* dev_spec_count, uint8_t* dev_rearm_mask,
                                                 void* stream);

/*
 * Close a reference step: push t_ref into each masked sample's reference history and raise its
 * reference count. Host state only. Errors: STATE if some entry has not been updated for
 * exactly the masked samples since the last commit, or no update is pending.
 */
speca_status_t speca_cache_commit_step(speca_cache_t* cache);

/*
 * Speculative step, Eq. 2 / workflow step 2: extrapolate every cached block output to t_target.
 *   t_target        host, B doubles.
 *   dev_active_mask device, B bytes, NULL = all samples: samples with a zero byte are skipped
 *                   (their planes are not read, their rows of outs are not written).
 *   outs            host array of n_entries device pointers, outs[e] = [B, N_e, D], NULL = skip e.
 * out = sum_{i=0..v} plane_i * prod-of-multipliers, evaluated by Horner's rule in fp32 and
 * rounded once to the storage dtype; v = min(m, references - 1) per sample.
 * Errors: INVALID_ARG, ALIGNMENT, STATE (a sample has no committed reference and the mask is
 * NULL; with a device mask such samples must be inactive: they are skipped on the device), CUDA.
 */
speca_status_t speca_forecast(speca_cache_t* cache, const double* t_target, const uint8_t* dev_active_mask,
                              void* const* outs, void* stream);

/*
 * Several speculative steps at once: Eq. 2 evaluated for K targets t-1 .. t-K from one read of the
 * tables (Fig. 1: the draft model predicts the next N timesteps from the latest reference; workflow
 * step 2 of Section 3.2). Same arithmetic as K calls of speca_forecast, bit for bit, but the planes
 * are read once: (v + 1 + K) words of traffic per element instead of K (v + 2).
 *   n_targets       K, 1..SPECA_MAX_HORIZON.
 *   t_targets       host, K * B doubles, target k of sample b at [k * B + b].
 *   dev_active_mask device, B bytes, NULL = all: inactive samples are skipped for every target.
 *   outs            host array of n_entries device pointers, outs[e] = [K, B, N_e, D] (target-major),
 *                   NULL = skip e.
 * Errors: INVALID_ARG (null, K out of range, non-finite time), ALIGNMENT, STATE, CUDA.
 */
speca_status_t speca_forecast_multi(speca_cache_t* cache, int32_t n_targets, const double* t_targets,
                                    const uint8_t* dev_active_mask, void* const* outs, void* stream);

/*
 * Forecasts consumed as a sum. A transformer adds its block outputs to a residual stream, so on a
 * speculative step the forecasts (Eq. 2) of equally shaped blocks are only needed as
 *     out = base + sum over the listed entries of forecast_e(t_target),
 * which this call computes without writing the individual forecasts: each entry's Horner result
 * stays in fp32, is added unrounded in list order, and the total is rounded once to the storage
 * dtype. (An extension of workflow step 2 that assumes the model's residual structure; the paper
 * itself only forecasts per block.)
 *   entry_ids       host, n_ids entry indices (1..SPECA_MAX_ENTRIES of them), all with the same
 *                   tokens * dim; an entry may be listed more than once.
 *   t_target        host, B doubles.  dev_active_mask: device, B bytes, NULL = all (inactive samples'
 *                   rows of out are not written).
 *   base            device [B, N, D] or NULL (= 0).  out: device [B, N, D]; may alias base.
 * Errors: INVALID_ARG (null, empty list, index out of range, non-finite time), SHAPE (entries of
 * different sizes), ALIGNMENT, STATE, CUDA.
 */
speca_status_t speca_forecast_sum(speca_cache_t* cache, const int32_t* entry_ids, int32_t n_ids, const double* t_target,
                                  const uint8_t* dev_active_mask, const void* base, void* out, void* stream);

/*
 * Verification, Eq. 4 and the accept rule of Section 3.4.2, fused with the forecast of the
 * verification entry:  e_b = ||p_b - f_b||_2 / (||f_b||_2 + eps),  accept_b = (e_b <= tau_b),
 * with p the forecast rounded to the storage dtype and the norms taken over all N_v*D elements
 * of sample b. Sums are accumulated in fp32 per thread and combined in a fixed order (warp
 * shuffle, shared memory, cluster shared memory, then fp64 across clusters), so results are
 * identical from run to run. A NaN anywhere in a sample rejects it.
 *   fresh           device, [B, N_v, D]: the verification layer's feature computed by the model.
 *   t_target, tau   host, B doubles / B floats.
 *   dev_active_mask device, B bytes, NULL = all. Inactive samples: err, accept, out_pred untouched.
 *   out_pred        device [B, N_v, D] or NULL: also store the forecast p.
 *   dev_err         device, B floats.  dev_accept: device, B bytes (1 = accept).
 * Uses a few KB of reduction scratch inside the arena: two verify calls on the same handle must
 * not overlap on the GPU (enqueue them on one stream).
 * Errors: INVALID_ARG, ALIGNMENT, STATE, CUDA.
 */
speca_status_t speca_verify(speca_cache_t* cache, const void* fresh, const double* t_target, const float* tau,
                            const uint8_t* dev_active_mask, void* out_pred, float* dev_err,
                            uint8_t* dev_accept, void* stream);

/* speca_verify with another error metric (speca_metric_t); everything else as speca_verify.
 * speca_verify(...) is speca_verify_metric(..., SPECA_METRIC_L2, ...). Errors: as speca_verify,
 * and INVALID_ARG for an unknown metric. */
speca_status_t speca_verify_metric(speca_cache_t* cache, int32_t metric, const void* fresh, const double* t_target,
                                   const float* tau, const uint8_t* dev_active_mask, void* out_pred, float* dev_err,
                                   uint8_t* dev_accept, void* stream);

/*
 * Verification of a cache that holds only a token range of every entry (sequence-parallel layout:
 * each GPU caches N_e / R tokens of every block output). Eq. 4 needs sums over the whole sample, so
 * the step is split: every rank reduces its shard to the metric's running values, the ranks combine
 * them (one all-reduce of 4*B doubles: sum, or max for SPECA_METRIC_LINF), every rank decides.
 *
 * speca_verify_partial: as speca_verify_metric, but instead of err / accept it writes
 *   dev_sums   device, B x 4 doubles: sample b at [4b .. 4b+2] (unused slots 0), untouched for
 *              inactive samples. L2: sum (p-f)^2, sum f^2. L1: sum |p-f|, sum |f|.
 *              LINF: max |p-f|, max |f|. COSINE: sum p f, sum p^2, sum f^2.
 * speca_verify_decide: e_b from combined values by the metric's formula (eps <= 0 selects 1e-8),
 *   accept_b = (e_b <= tau_b); needs no handle. dev_active_mask NULL = all.
 * With one rank, partial followed by decide gives exactly what speca_verify_metric gives.
 * Errors: as speca_verify_metric; speca_verify_decide: INVALID_ARG, SHAPE (batch), ALIGNMENT, CUDA.
 */
speca_status_t speca_verify_partial(speca_cache_t* cache, int32_t metric, const void* fresh, const double* t_target,
                                    const uint8_t* dev_active_mask, void* out_pred, double* dev_sums, void* stream);
speca_status_t speca_verify_decide(int32_t metric, const double* dev_sums, int32_t batch, const float* tau, float eps,
                                   const uint8_t* dev_active_mask, float* dev_err, uint8_t* dev_accept, void* stream);

/*
 * Per-sample continuation of the speculative run (sequential validation of Section 3.4.2, the
 * forced activation period N of Appendix A, sample-adaptive allocation):
 *   for every active sample b: if accept_b then spec_count_b += 1
 *   keep_b   = active_b && accept_b && spec_count_b < k_max
 *   active'_b = AND of keep over the `group` consecutive samples that contain b
 *               (group = 1: per sample; 2: a classifier-free-guidance pair shares its fate)
 *   dev_active_idx = ascending list of the samples with active' = 1, dev_n_active = its length.
 * All pointers are device pointers; dev_spec_count (B int32) and dev_active_mask (B bytes) are
 * updated in place; dev_active_idx (B int32) and dev_n_active (1 int32) may be NULL.
 * Errors: INVALID_ARG (null, k_max < 1, group < 1 or not dividing B), CUDA.
 */
speca_status_t speca_select_adaptive(speca_cache_t* cache, const uint8_t* dev_accept, int32_t k_max,
                                     int32_t group, int32_t* dev_spec_count, uint8_t* dev_active_mask,
                                     int32_t* dev_active_idx, int32_t* dev_n_active, void* stream);

/*
 * speca_verify_metric followed by speca_select_adaptive in one launch: the cluster that finishes the
 * reduction also applies the continuation rule, once every sample's decision is final. Same results
 * as the two calls; saves a kernel launch per speculative step.
 *   dev_active_mask       device, B bytes, required: this step's mask (read only).
 *   dev_next_active_mask  device, B bytes, must not overlap dev_active_mask: receives the mask of the
 *                         next step (other thread blocks may still be reading this step's mask when
 *                         it is written, hence two buffers; a caller alternates between them).
 * The other arguments are those of the two calls. If no sample is active, the next mask is all zero
 * and *dev_n_active = 0. Errors: those of the two calls, INVALID_ARG for overlapping masks.
 */
speca_status_t speca_verify_select(speca_cache_t* cache, int32_t metric, const void* fresh, const double* t_target,
                                   const float* tau, const uint8_t* dev_active_mask, uint8_t* dev_next_active_mask,
                                   void* out_pred, float* dev_err, uint8_t* dev_accept, int32_t k_max, int32_t group,
                                   int32_t* dev_spec_count, int32_t* dev_active_idx, int32_t* dev_n_active, void* stream);

/* After a reference step: mark the samples with host_sample_mask[b] != 0 (NULL = all) active again
 * and clear their speculative-step counters, on the stream. Errors: INVALID_ARG, CUDA. */
speca_status_t speca_activate(speca_cache_t* cache, const uint8_t* host_sample_mask, int32_t* dev_spec_count,
                              uint8_t* dev_active_mask, void* stream);

/*
 * Verification without a handle, an arena or any allocation. (The paper has no counterpart: this is
 * Eq. 4 and the accept rule applied to a forecast tensor the caller already holds, offered for
 * callers that cannot give the library memory.)
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a serving process
 * whose framework pool took all of HBM at start-up, a plug-in that is only handed input and output
 * tensors, a host thread that must not call cudaMalloc because that call synchronises the whole
 * device. speca_verify keeps its reduction scratch in the caller's arena; this variant keeps it in
 * a fixed array inside the library image instead, SPECA_STATIC_SCRATCH_BYTES (about 65 KB) that
 * every GPU which loads the library holds until the process exits. The call path contains no
 * cudaMalloc, cudaFree or other allocating routine.
 *
 *   e_b = ||pred_b - fresh_b||_2 / (||fresh_b||_2 + eps),  accept_b = (e_b <= tau_b)
 *
 *   pred, fresh     device, dense [batch, n_elems] in `dtype`; both 16-byte aligned, and
 *                   n_elems * sizeof(element) a multiple of 16 when batch > 1 (every row must
 *                   start on a 16-byte boundary). pred is typically an output of speca_forecast.
 *   n_elems         1 .. SPECA_STATIC_MAX_ELEMS per sample; batch 1 .. SPECA_STATIC_MAX_BATCH.
 *   tau             host, batch floats. eps <= 0 selects the paper's 1e-8.
 *   dev_active_mask device, batch bytes, NULL = all; inactive samples' err / accept are untouched.
 *   dev_err         device, batch floats.  dev_accept: device, batch bytes (1 = accept).
 *   device          CUDA device ordinal that owns all the buffers; stream as everywhere else.
 *
 * The first call on a device (and per storage type) looks up the scratch array's device address
 * (cudaGetSymbolAddress, with that device current) and the number of thread-block clusters the
 * device can hold, and remembers both; make that first call before any stream capture begins.
 * Later calls do no driver queries. Every call on a device shares the one array, which keeps whatever the
 * previous call left: each call re-initialises what it needs on the stream before the reduction
 * runs, so calls in stream order are independent, but two calls whose kernels overlap on the GPU
 * (different streams, no dependency between them) race on the scratch and give wrong results.
 * Errors: INVALID_ARG (null, dtype, NaN tau, bad device), SHAPE (batch or n_elems beyond the
 * maxima above), ALIGNMENT, UNSUPPORTED (not an sm_100 device), CUDA. On error nothing that writes
 * dev_err or dev_accept is enqueued (the scratch's counters may already have been cleared on the stream).
 */
#define SPECA_STATIC_MAX_BATCH 64
#define SPECA_STATIC_MAX_ELEMS 2147483647LL
#define SPECA_STATIC_MAX_CLUSTERS 128
#define SPECA_STATIC_SCRATCH_BYTES (8 * 64 * SPECA_STATIC_MAX_CLUSTERS + 512)
speca_status_t speca_verify_pred_static(const void* pred, const void* fresh, int64_t n_elems, int32_t batch,
                                        int32_t dtype, const float* tau, float eps, const uint8_t* dev_active_mask,
                                        float* dev_err, uint8_t* dev_accept, int32_t device, void* stream);

/* Threshold schedule of Section 3.4.2: tau_t = tau0 * beta^((T - t) / T). Returns NaN for T <= 0. */
double speca_tau(double tau0, double beta, double t, double T);

/* Per-sample host state: committed reference count and latest reference time (NaN if none).
 * Either output may be NULL. */
speca_status_t speca_cache_state(const speca_cache_t* cache, int32_t* host_n_refs, double* host_t_last);

/*
 * Checkpoint / resume. The tables live in the caller's arena; the only other state of a cache is
 * the reference history of each sample. speca_cache_get_history copies it out (host_n_refs: B
 * int32; host_t_hist: B x (SPECA_MAX_ORDER + 1) doubles, most recent first, NaN where undefined);
 * speca_cache_set_history installs it in a cache of the same configuration -- built over a copy of
 * the saved arena bytes, it continues exactly where the saved one stopped. Host only.
 * Errors: INVALID_ARG (null, negative count, a defined time that is not finite), STATE (set while a
 * reference step is open).
 */
speca_status_t speca_cache_get_history(const speca_cache_t* cache, int32_t* host_n_refs, double* host_t_hist);
speca_status_t speca_cache_set_history(speca_cache_t* cache, const int32_t* host_n_refs, const double* host_t_hist);

/* Device address and byte stride of the table of (entry, sample): plane i starts at
 * *plane0 + i * *plane_stride_bytes. For checkpointing and tests. In a SPECA_LAYOUT_HISTORY cache
 * plane i is a ring slot: the feature of the j-th latest reference sits in plane
 * (references - 1 - j) mod (max_order + 1). */
speca_status_t speca_cache_plane(const speca_cache_t* cache, int32_t entry, int32_t sample, void** plane0,
                                 size_t* plane_stride_bytes);

/*
 * The per-sample scalars a forecast (or verification) at t_target hands to the kernels, for a sample
 * with n_refs committed references at times t_hist[0] (latest), t_hist[1], ... (min(n_refs,
 * max_order + 1) of them are read). Host only; touches no GPU and needs no cache.
 *   *out_order  v = min(max_order, n_refs - 1), -1 without references: planes 0..v are read.
 *   out_coef    SPECA_MAX_ORDER + 1 floats. TABLES: the Horner multipliers of Eq. 2, out =
 *               plane_0 + c_0 (plane_1 + c_1 (plane_2 + ...)); TAYLOR c_i = (t_target - t_last)/(i + 1).
 *               HISTORY: one weight per physical plane, out = sum_i c_i * plane_i, with Eq. 3's
 *               differencing over the actual gaps folded in.
 * Errors: INVALID_ARG.
 */
speca_status_t speca_forecast_weights(int32_t layout, int32_t basis, int32_t max_order, int32_t n_refs,
                                      const double* t_hist, double t_target, int32_t* out_order, float* out_coef);

/*
 * SPECA_LAYOUT_HISTORY only: device address of the plane that the next reference step of `sample` will
 * fill for `entry` (N_e * D elements of the storage type, 4 KB aligned). A model that writes its block
 * output there directly, and then passes that same address (minus sample * N_e * D elements, i.e. the
 * address a [B, N_e, D] tensor would need for the row to land there; for B = 1 simply the address
 * itself) as feats[entry] to speca_cache_update, pays nothing for the reference step: the entry is
 * recognised as already in place and not copied. The address changes after every committed step of
 * that sample. Errors: INVALID_ARG, UNSUPPORTED (a cache that keeps difference tables).
 */
speca_status_t speca_cache_next_slot(const speca_cache_t* cache, int32_t entry, int32_t sample, void** out);

/*
 * SPECA_LAYOUT_HISTORY only: pass this as feats[entry] to speca_cache_update to say that the feature of
 * every masked sample of that entry already sits in the plane speca_cache_next_slot names for it (a
 * batch whose samples are at the same ring position forms a strided [B, N_e, D] tensor there: sample
 * stride = (max_order + 1) * plane stride). The entry then takes part in the reference step like any
 * other, and nothing is copied.
 */
#define SPECA_FEATURE_IN_PLACE ((const void*)(uintptr_t)1)

/*
 * Host-side counters of a handle since it was created (nothing here is read back from the device, so
 * the call neither launches nor synchronises). Launch counts are per kernel kind; the fused
 * verify + continuation call counts as one verify launch, the fused reference step
 * (speca_cache_update_forecast) has a count of its own. reference_steps[b] counts committed
 * reference steps of sample b (it does not go back to zero on a reset, unlike the history length
 * that speca_cache_state reports); resets[b] counts how often sample b's history was cleared.
 * Entries at and beyond the batch size are zero. reference_steps is the number of full passes each
 * sample of a batch needed: the quantity that sample-adaptive computation allocation varies.
 */
typedef struct {
    uint64_t update_launches, forecast_launches, forecast_multi_launches, forecast_sum_launches;
    uint64_t verify_launches, select_launches, activate_launches, update_forecast_launches;
    uint64_t reference_steps[SPECA_MAX_BATCH];
    uint64_t resets[SPECA_MAX_BATCH];
} speca_cache_stats_t;
speca_status_t speca_cache_stats(const speca_cache_t* cache, speca_cache_stats_t* out);

/*
 * Health check of the work a handle has enqueued on `stream`: waits for that stream (the one call
 * besides destroy that synchronises), then reads the cache's gave-up word. The SPECA_PATH_BULK kernels
 * wait for their staged copies with a bounded wait; if one ever gives up, the kernel sets that word
 * and finishes without the tile, so results since the previous check are incomplete. Returns
 * SPECA_ERR_CUDA in that case (and clears the word), or if the stream reports an error; SPECA_OK
 * otherwise. The other kernel paths never set the word. Errors: INVALID_ARG (null handle), CUDA.
 */
speca_status_t speca_cache_check(speca_cache_t* cache, void* stream);

/* How many kernels the handle has launched since it was created. */
speca_status_t speca_cache_launch_count(const speca_cache_t* cache, uint64_t* out);

const char* speca_status_string(speca_status_t status);
/* Human-readable detail of the most recent error on this handle ("" if none). */
const char* speca_last_error(const speca_cache_t* cache);
/* Library version string. */
const char* speca_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECA_H_ */
