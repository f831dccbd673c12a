// CUDA kernels of the SpeCa feature-cache hot path for sm_100a (B200).
//
//   update   : Eq. 3 -- fold a freshly computed feature into the derivative table, in place
//   forecast : Eq. 2 -- Horner evaluation of the table at a speculative time
//   verify   : Eq. 4 -- forecast of the verification entry fused with ||p - f||, ||f|| and the
//              accept rule of Section 3.4.2
//   select   : per-sample continuation of the speculative run (Section 3.4.2, Appendix A)
//
// Every kernel is a pure HBM stream (about half a flop per byte), so the design goal is bytes in
// flight, coalescing and no re-reads: 16-byte vectors, several independent loads per thread before
// the first use, persistent grids sized from the SM count, streaming cache hints (nothing is
// reused before it leaves L2). No tensor cores are involved.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "speca_internal.h"

namespace cg = cooperative_groups;

namespace speca {

// ------------------------------------------------------------------------------------------------
// element packing
// ------------------------------------------------------------------------------------------------

template <int DT>
struct Elem;
template <>
struct Elem<SPECA_F32> {
    static constexpr int kBytes = 4;
    static constexpr int kEPV = 4;  // elements per 16-byte vector
};
template <>
struct Elem<SPECA_BF16> {
    static constexpr int kBytes = 2;
    static constexpr int kEPV = 8;
};

template <int DT>
__device__ __forceinline__ void unpack(const uint4& v, float (&f)[Elem<DT>::kEPV]) {
    if constexpr (DT == SPECA_F32) {
        f[0] = __uint_as_float(v.x);
        f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z);
        f[3] = __uint_as_float(v.w);
    } else {
        // bfloat16 is the upper half of a binary32: widening is a shift
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            f[2 * k] = __uint_as_float(w[k] << 16);
            f[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
}

template <int DT>
__device__ __forceinline__ uint4 pack(const float (&f)[Elem<DT>::kEPV]) {
    uint4 v;
    if constexpr (DT == SPECA_F32) {
        v.x = __float_as_uint(f[0]);
        v.y = __float_as_uint(f[1]);
        v.z = __float_as_uint(f[2]);
        v.w = __float_as_uint(f[3]);
    } else {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);  // round to nearest even
            w[k] = *reinterpret_cast<uint32_t*>(&h);
        }
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    return v;
}

// value after a round trip through the storage type
template <int DT>
__device__ __forceinline__ float round_storage(float x) {
    if constexpr (DT == SPECA_F32)
        return x;
    else
        return __bfloat162float(__float2bfloat16_rn(x));
}

template <int DT>
__device__ __forceinline__ float load_scalar(const char* base, uint32_t idx) {
    if constexpr (DT == SPECA_F32)
        return reinterpret_cast<const float*>(base)[idx];
    else
        return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(base)[idx]) << 16);
}

template <int DT>
__device__ __forceinline__ void store_scalar(char* base, uint32_t idx, float x) {
    if constexpr (DT == SPECA_F32)
        reinterpret_cast<float*>(base)[idx] = x;
    else
        reinterpret_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(x);
}

// ------------------------------------------------------------------------------------------------
// work list: tile -> segment
// ------------------------------------------------------------------------------------------------

// Largest s in [lo, hi) with tile_start[s] <= tile. Every thread of the CTA runs the same search;
// the loads are warp-uniform and stay in L1.
__device__ __forceinline__ uint32_t find_segment(const uint32_t* __restrict__ tile_start, uint32_t lo, uint32_t hi,
                                                 uint32_t tile) {
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (__ldg(tile_start + mid) <= tile)
            lo = mid;
        else
            hi = mid;
    }
    return lo;
}

// ------------------------------------------------------------------------------------------------
// per-tile bodies, direct (register) path
// ------------------------------------------------------------------------------------------------

// Eq. 2 in Horner form: acc = D_v; acc = D_{i-1} + acc * mu_i for i = v..1.
template <int DT, int V, int U>
__device__ __forceinline__ void forecast_tile(const char* __restrict__ plane0, uint64_t stride,
                                              char* __restrict__ out, uint32_t cnt, const float (&mu)[SPECA_MAX_ORDER]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    uint4* __restrict__ dst = reinterpret_cast<uint4*>(out);
    for (uint32_t base = 0; base < nvec; base += kThreads * U) {
        uint4 d[V + 1][U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
#pragma unroll
                for (int i = 0; i <= V; ++i)
                    d[i][u] = __ldcs(reinterpret_cast<const uint4*>(plane0 + i * stride) + idx);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
                float acc[EPV];
                unpack<DT>(d[V][u], acc);
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[EPV];
                    unpack<DT>(d[i - 1][u], lo);
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
                }
                __stcs(dst + idx, pack<DT>(acc));
            }
        }
    }
    // ragged tail, or the whole tile when the output row is not 16-byte aligned
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float acc = load_scalar<DT>(plane0 + V * stride, j);
#pragma unroll
        for (int i = V; i >= 1; --i) acc = fmaf(acc, mu[i - 1], load_scalar<DT>(plane0 + (i - 1) * stride, j));
        store_scalar<DT>(out, j, acc);
    }
}

// Eq. 3 as a chain of difference quotients: c_0 = f; c_{i+1} = (c_i - D_i) * r_i; D_i <- c_i.
// V = highest plane written. Reads f and planes 0..V-1, writes planes 0..V, each element once.
template <int DT, int V, int U>
__device__ __forceinline__ void update_tile(char* __restrict__ plane0, uint64_t stride, const char* __restrict__ feat,
                                            uint32_t cnt, const float (&r)[SPECA_MAX_ORDER]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(feat) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t base = 0; base < nvec; base += kThreads * U) {
        uint4 fv[U];
        uint4 d[V > 0 ? V : 1][U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
                fv[u] = __ldcs(reinterpret_cast<const uint4*>(feat) + idx);
#pragma unroll
                for (int i = 0; i < V; ++i) d[i][u] = __ldcs(reinterpret_cast<const uint4*>(plane0 + i * stride) + idx);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
                float c[EPV];
                unpack<DT>(fv[u], c);
                // plane 0 is the feature itself: already in storage format
                __stcs(reinterpret_cast<uint4*>(plane0) + idx, fv[u]);
#pragma unroll
                for (int i = 0; i < V; ++i) {
                    float old[EPV];
                    unpack<DT>(d[i][u], old);
#pragma unroll
                    for (int k = 0; k < EPV; ++k) c[k] = (c[k] - old[k]) * r[i];
                    __stcs(reinterpret_cast<uint4*>(plane0 + (i + 1) * stride) + idx, pack<DT>(c));
                }
            }
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float c = load_scalar<DT>(feat, j);
        float old[V > 0 ? V : 1];
#pragma unroll
        for (int i = 0; i < V; ++i) old[i] = load_scalar<DT>(plane0 + i * stride, j);
        store_scalar<DT>(plane0, j, c);
#pragma unroll
        for (int i = 0; i < V; ++i) {
            c = (c - old[i]) * r[i];
            store_scalar<DT>(plane0 + (i + 1) * stride, j, c);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// streaming kernels: persistent CTAs stride over the flattened tile list
// ------------------------------------------------------------------------------------------------

// Runtime-order variants for the rare tiles whose sample has fewer references than the launch's
// common order (warm-up after a reset): one vector at a time, planes visited in a loop.
template <int DT>
__device__ __noinline__ void forecast_tile_any(const char* __restrict__ plane0, uint64_t stride, char* __restrict__ out,
                                               uint32_t cnt, int v, const float (&mu)[SPECA_MAX_ORDER]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += kThreads) {
        float acc[EPV];
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + v * stride) + idx), acc);
        for (int i = v; i >= 1; --i) {
            float lo[EPV];
            unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + (i - 1) * stride) + idx), lo);
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
        }
        __stcs(reinterpret_cast<uint4*>(out) + idx, pack<DT>(acc));
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float acc = load_scalar<DT>(plane0 + v * stride, j);
        for (int i = v; i >= 1; --i) acc = fmaf(acc, mu[i - 1], load_scalar<DT>(plane0 + (i - 1) * stride, j));
        store_scalar<DT>(out, j, acc);
    }
}

template <int DT>
__device__ __noinline__ void update_tile_any(char* __restrict__ plane0, uint64_t stride, const char* __restrict__ feat,
                                             uint32_t cnt, int v, const float (&r)[SPECA_MAX_ORDER]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(feat) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += kThreads) {
        const uint4 fv = __ldcs(reinterpret_cast<const uint4*>(feat) + idx);
        float c[EPV];
        unpack<DT>(fv, c);
        uint4 next = fv;  // value to store into plane i
        for (int i = 0; i < v; ++i) {
            float old[EPV];
            unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + i * stride) + idx), old);
            __stcs(reinterpret_cast<uint4*>(plane0 + i * stride) + idx, next);
#pragma unroll
            for (int k = 0; k < EPV; ++k) c[k] = (c[k] - old[k]) * r[i];
            next = pack<DT>(c);
        }
        __stcs(reinterpret_cast<uint4*>(plane0 + v * stride) + idx, next);
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float c = load_scalar<DT>(feat, j);
        for (int i = 0; i < v; ++i) {
            const float old = load_scalar<DT>(plane0 + i * stride, j);
            store_scalar<DT>(plane0 + i * stride, j, c);
            c = (c - old) * r[i];
        }
        store_scalar<DT>(plane0 + v * stride, j, c);
    }
}

// ------------------------------------------------------------------------------------------------
// streaming kernels: persistent CTAs stride over the flattened tile list
// ------------------------------------------------------------------------------------------------

// Independent 16-byte loads a thread issues per plane before it starts computing.
__host__ __device__ constexpr int unroll_for(int planes) { return planes <= 4 ? 4 : 2; }

// V = the order most samples of the launch have (the host passes the maximum over samples).
template <int DT, int V, bool UPDATE>
__global__ void __launch_bounds__(kThreads, 2) stream_direct_kernel(const __grid_constant__ StreamParams p) {
    constexpr uint32_t kTile = kTileBytesDirect / Elem<DT>::kBytes;
    constexpr int U = unroll_for(V + 1 + (UPDATE ? 0 : 0));
    uint32_t seg = p.seg_lo;
    for (uint32_t tile = p.tile_lo + blockIdx.x; tile < p.tile_hi; tile += gridDim.x) {
        seg = find_segment(p.tile_start, seg, p.seg_hi, tile);
        const SegDesc sd = p.segs[seg];
        const int v = p.order[sd.sample];
        char* io = static_cast<char*>(p.io[sd.entry]);
        if (v < 0 || io == nullptr) continue;
        if (p.dev_mask != nullptr && p.dev_mask[sd.sample] == 0) continue;
        const uint32_t elem0 = (tile - __ldg(p.tile_start + seg)) * kTile;
        const uint32_t cnt = min(kTile, sd.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        char* plane0 = p.arena + sd.plane0_off + byte0;
        char* row = io + sd.io_off + byte0;
        float coef[SPECA_MAX_ORDER];
#pragma unroll
        for (int i = 0; i < SPECA_MAX_ORDER; ++i) coef[i] = p.coef[sd.sample][i];
        if constexpr (UPDATE) {
            if (v == V)
                update_tile<DT, V, U>(plane0, sd.plane_stride, row, cnt, coef);
            else
                update_tile_any<DT>(plane0, sd.plane_stride, row, cnt, v, coef);
        } else {
            if (v == V)
                forecast_tile<DT, V, U>(plane0, sd.plane_stride, row, cnt, coef);
            else
                forecast_tile_any<DT>(plane0, sd.plane_stride, row, cnt, v, coef);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// verify: forecast of one entry fused with the two sums of squares of Eq. 4
// ------------------------------------------------------------------------------------------------

constexpr int kMaxClusterSize = 8;

template <int DT, int V, int U>
__device__ __forceinline__ void verify_tile(const char* __restrict__ plane0, uint64_t stride,
                                            const char* __restrict__ fresh, char* __restrict__ out_pred, uint32_t cnt,
                                            const float (&mu)[SPECA_MAX_ORDER], float& num, float& den) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(fresh) | reinterpret_cast<uintptr_t>(out_pred)) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t base = 0; base < nvec; base += kThreads * U) {
        uint4 d[V + 1][U];
        uint4 fv[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
#pragma unroll
                for (int i = 0; i <= V; ++i)
                    d[i][u] = __ldcs(reinterpret_cast<const uint4*>(plane0 + i * stride) + idx);
                fv[u] = __ldcs(reinterpret_cast<const uint4*>(fresh) + idx);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = base + u * kThreads + threadIdx.x;
            if (idx < nvec) {
                float acc[EPV], f[EPV];
                unpack<DT>(d[V][u], acc);
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[EPV];
                    unpack<DT>(d[i - 1][u], lo);
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
                }
                // the forecast as the model would consume it: rounded to the storage type
                const uint4 pv = pack<DT>(acc);
                unpack<DT>(pv, acc);
                unpack<DT>(fv[u], f);
#pragma unroll
                for (int k = 0; k < EPV; ++k) {
                    const float diff = acc[k] - f[k];
                    num = fmaf(diff, diff, num);
                    den = fmaf(f[k], f[k], den);
                }
                if (out_pred != nullptr) __stcs(reinterpret_cast<uint4*>(out_pred) + idx, pv);
            }
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float acc = load_scalar<DT>(plane0 + V * stride, j);
#pragma unroll
        for (int i = V; i >= 1; --i) acc = fmaf(acc, mu[i - 1], load_scalar<DT>(plane0 + (i - 1) * stride, j));
        acc = round_storage<DT>(acc);
        const float f = load_scalar<DT>(fresh, j);
        const float diff = acc - f;
        num = fmaf(diff, diff, num);
        den = fmaf(f, f, den);
        if (out_pred != nullptr) store_scalar<DT>(out_pred, j, acc);
    }
}

template <int DT>
__device__ __noinline__ void verify_tile_any(const char* __restrict__ plane0, uint64_t stride,
                                             const char* __restrict__ fresh, char* __restrict__ out_pred, uint32_t cnt,
                                             int v, const float (&mu)[SPECA_MAX_ORDER], float& num, float& den) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(fresh) | reinterpret_cast<uintptr_t>(out_pred)) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += kThreads) {
        float acc[EPV], f[EPV];
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + v * stride) + idx), acc);
        for (int i = v; i >= 1; --i) {
            float lo[EPV];
            unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + (i - 1) * stride) + idx), lo);
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
        }
        const uint4 pv = pack<DT>(acc);
        unpack<DT>(pv, acc);
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(fresh) + idx), f);
#pragma unroll
        for (int k = 0; k < EPV; ++k) {
            const float diff = acc[k] - f[k];
            num = fmaf(diff, diff, num);
            den = fmaf(f[k], f[k], den);
        }
        if (out_pred != nullptr) __stcs(reinterpret_cast<uint4*>(out_pred) + idx, pv);
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float acc = load_scalar<DT>(plane0 + v * stride, j);
        for (int i = v; i >= 1; --i) acc = fmaf(acc, mu[i - 1], load_scalar<DT>(plane0 + (i - 1) * stride, j));
        acc = round_storage<DT>(acc);
        const float f = load_scalar<DT>(fresh, j);
        const float diff = acc - f;
        num = fmaf(diff, diff, num);
        den = fmaf(f, f, den);
        if (out_pred != nullptr) store_scalar<DT>(out_pred, j, acc);
    }
}

// Does cluster q of Q own at least one work unit of sample b (units_per_sample units per sample,
// unit u belongs to cluster u mod Q)?
__device__ __forceinline__ bool cluster_touches(uint32_t q, uint32_t Q, uint32_t b, uint32_t units_per_sample) {
    const uint32_t lo = b * units_per_sample;
    const uint32_t first = lo + (q + Q - lo % Q) % Q;
    return first < lo + units_per_sample;
}

// Work unit = `cluster size` consecutive tiles of one sample, one per CTA of the cluster, so all
// CTAs of a cluster always work on the same sample and reach the reduction together.
// Reduction: registers -> warp shuffle -> shared memory (CTA) -> the leader CTA's shared memory
// through the cluster's distributed shared memory -> one partial per (cluster, sample) in global
// scratch -> the cluster that arrives last (ticket counter, no waiting) adds the partials in
// cluster order in fp64 and applies Eq. 4 and the accept rule.
template <int DT, int V>
__global__ void __launch_bounds__(kThreads, 2) verify_kernel(const __grid_constant__ VerifyParams p) {
    constexpr uint32_t kTile = kTileBytesDirect / Elem<DT>::kBytes;
    constexpr int U = unroll_for(V + 2);
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t csize = cluster.num_blocks();
    const uint32_t crank = cluster.block_rank();
    const uint32_t cid = blockIdx.x / csize;
    const uint32_t n_clusters = gridDim.x / csize;

    __shared__ float warp_part[2][kThreads / 32];
    __shared__ float cluster_slot[2][2][kMaxClusterSize];  // [parity][num|den][rank], leader's copy is used
    __shared__ bool is_last;

    float num = 0.f, den = 0.f;
    int cur_b = -1;
    uint32_t parity = 0;

    auto flush = [&](int b) {
        // warp level
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            num += __shfl_xor_sync(0xFFFFFFFFu, num, off);
            den += __shfl_xor_sync(0xFFFFFFFFu, den, off);
        }
        if ((threadIdx.x & 31) == 0) {
            warp_part[0][threadIdx.x >> 5] = num;
            warp_part[1][threadIdx.x >> 5] = den;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float n = 0.f, d = 0.f;
#pragma unroll
            for (int w = 0; w < kThreads / 32; ++w) {
                n += warp_part[0][w];
                d += warp_part[1][w];
            }
            // hand the CTA's sums to the cluster leader through distributed shared memory
            float* leader = cluster.map_shared_rank(&cluster_slot[parity][0][0], 0);
            leader[crank] = n;
            leader[kMaxClusterSize + crank] = d;
        }
        cluster.sync();
        if (crank == 0 && threadIdx.x == 0) {
            float n = 0.f, d = 0.f;
            for (uint32_t r = 0; r < csize; ++r) {
                n += cluster_slot[parity][0][r];
                d += cluster_slot[parity][1][r];
            }
            float* dst = p.partials + (static_cast<size_t>(cid) * p.batch + b) * 2;
            __stcg(dst, n);
            __stcg(dst + 1, d);
        }
        // Slots alternate between two buffers: a CTA can write the buffer of flush k+2 only after
        // the barrier of flush k+1, which the leader enters after it has read the buffer of flush k.
        parity ^= 1;
        num = 0.f;
        den = 0.f;
    };

    const uint32_t total_units = static_cast<uint32_t>(p.batch) * p.units_per_sample;
    for (uint32_t unit = cid; unit < total_units; unit += n_clusters) {
        const int b = static_cast<int>(unit / p.units_per_sample);
        const int v = p.order[b];
        if (v < 0 || (p.dev_mask != nullptr && p.dev_mask[b] == 0)) continue;  // uniform over the cluster
        if (b != cur_b) {
            if (cur_b >= 0) flush(cur_b);
            cur_b = b;
        }
        const uint32_t tile = (unit % p.units_per_sample) * csize + crank;
        if (tile >= p.tiles_per_sample) continue;
        const SegDesc sd = p.segs[b];
        const uint32_t elem0 = tile * kTile;
        const uint32_t cnt = min(kTile, p.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        const char* plane0 = p.arena + sd.plane0_off + byte0;
        const char* fresh = p.fresh + sd.io_off + byte0;
        char* pred = p.out_pred != nullptr ? p.out_pred + sd.io_off + byte0 : nullptr;
        float mu[SPECA_MAX_ORDER];
#pragma unroll
        for (int i = 0; i < SPECA_MAX_ORDER; ++i) mu[i] = p.coef[b][i];
        if (v == V)
            verify_tile<DT, V, U>(plane0, sd.plane_stride, fresh, pred, cnt, mu, num, den);
        else
            verify_tile_any<DT>(plane0, sd.plane_stride, fresh, pred, cnt, v, mu, num, den);
    }
    if (cur_b >= 0) flush(cur_b);

    if (crank != 0) return;  // nobody touches a non-leader's shared memory after its last barrier

    if (threadIdx.x == 0) {
        __threadfence();  // partials visible before the ticket
        const uint32_t t = atomicAdd(p.ticket, 1u);
        is_last = (t == n_clusters - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int b = threadIdx.x; b < p.batch; b += kThreads) {
        if (p.order[b] < 0 || (p.dev_mask != nullptr && p.dev_mask[b] == 0)) continue;
        double sn = 0.0, sd = 0.0;
        for (uint32_t q = 0; q < n_clusters; ++q) {
            if (!cluster_touches(q, n_clusters, b, p.units_per_sample)) continue;
            const float* src = p.partials + (static_cast<size_t>(q) * p.batch + b) * 2;
            sn += static_cast<double>(__ldcg(src));
            sd += static_cast<double>(__ldcg(src + 1));
        }
        const double e = sqrt(sn) / (sqrt(sd) + p.eps);
        p.err[b] = static_cast<float>(e);
        p.accept[b] = (e <= static_cast<double>(p.tau[b])) ? 1 : 0;  // NaN compares false: reject
    }
    __syncthreads();
    if (threadIdx.x == 0) *p.ticket = 0;  // ready for the next launch on this stream
}

// ------------------------------------------------------------------------------------------------
// select / activate: B <= 64 samples, one small CTA
// ------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(SPECA_MAX_BATCH) select_kernel(const uint8_t* __restrict__ accept, int32_t k_max,
                                                                  int32_t group, int32_t batch,
                                                                  int32_t* __restrict__ spec_count,
                                                                  uint8_t* __restrict__ active,
                                                                  int32_t* __restrict__ idx_out,
                                                                  int32_t* __restrict__ n_out) {
    __shared__ uint8_t keep[SPECA_MAX_BATCH];
    __shared__ uint8_t next[SPECA_MAX_BATCH];
    const int b = threadIdx.x;
    if (b < batch) {
        const bool a = active[b] != 0;
        const bool ok = a && accept[b] != 0;
        int32_t c = spec_count[b];
        if (ok) {
            c += 1;
            spec_count[b] = c;
        }
        keep[b] = (ok && c < k_max) ? 1 : 0;
    }
    __syncthreads();
    if (b < batch) {
        const int g0 = (b / group) * group;
        uint8_t all = 1;
        for (int i = 0; i < group; ++i) all &= keep[g0 + i];
        next[b] = all;
        active[b] = all;
    }
    __syncthreads();
    if (b == 0) {
        int32_t n = 0;
        for (int i = 0; i < batch; ++i)
            if (next[i]) {
                if (idx_out != nullptr) idx_out[n] = i;
                ++n;
            }
        if (n_out != nullptr) *n_out = n;
    }
}

__global__ void __launch_bounds__(SPECA_MAX_BATCH) activate_kernel(uint64_t mask_bits, int32_t batch,
                                                                    int32_t* __restrict__ spec_count,
                                                                    uint8_t* __restrict__ active) {
    const int b = threadIdx.x;
    if (b < batch && ((mask_bits >> b) & 1ull)) {
        active[b] = 1;
        spec_count[b] = 0;
    }
}

// ------------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------------

static_assert(kThreads * 4 * 16 == kTileBytesDirect, "a direct tile is one pass of the CTA at unroll 4");

template <int DT, bool UPDATE>
static const void* stream_kernel_for(int v) {
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&stream_direct_kernel<DT, 0, UPDATE>);
        case 1: return reinterpret_cast<const void*>(&stream_direct_kernel<DT, 1, UPDATE>);
        case 2: return reinterpret_cast<const void*>(&stream_direct_kernel<DT, 2, UPDATE>);
        case 3: return reinterpret_cast<const void*>(&stream_direct_kernel<DT, 3, UPDATE>);
        default: return reinterpret_cast<const void*>(&stream_direct_kernel<DT, 4, UPDATE>);
    }
}

template <int DT>
static const void* verify_kernel_for(int v) {
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&verify_kernel<DT, 0>);
        case 1: return reinterpret_cast<const void*>(&verify_kernel<DT, 1>);
        case 2: return reinterpret_cast<const void*>(&verify_kernel<DT, 2>);
        case 3: return reinterpret_cast<const void*>(&verify_kernel<DT, 3>);
        default: return reinterpret_cast<const void*>(&verify_kernel<DT, 4>);
    }
}

static int max_order(const int8_t* order) {
    int v = 0;
    for (int b = 0; b < SPECA_MAX_BATCH; ++b) v = order[b] > v ? order[b] : v;
    return v;
}

static cudaError_t launch_stream(const StreamParams& p, int dtype, bool update, int grid, cudaStream_t stream) {
    const int v = max_order(p.order);
    const void* fn;
    if (update)
        fn = dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, true>(v) : stream_kernel_for<SPECA_F32, true>(v);
    else
        fn = dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, false>(v) : stream_kernel_for<SPECA_F32, false>(v);
    void* args[1] = {const_cast<StreamParams*>(&p)};
    return cudaLaunchKernel(fn, dim3(grid), dim3(kThreads), args, 0, stream);
}

cudaError_t launch_update(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream) {
    if (path != SPECA_PATH_DIRECT) return cudaErrorNotSupported;
    return launch_stream(p, dtype, true, grid, stream);
}

cudaError_t launch_forecast(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream) {
    if (path != SPECA_PATH_DIRECT) return cudaErrorNotSupported;
    return launch_stream(p, dtype, false, grid, stream);
}

cudaError_t launch_verify(const VerifyParams& p, int dtype, int grid, int cluster, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int v = max_order(p.order);
    const void* fn = dtype == SPECA_BF16 ? verify_kernel_for<SPECA_BF16>(v) : verify_kernel_for<SPECA_F32>(v);
    void* args[1] = {const_cast<VerifyParams*>(&p)};
    return cudaLaunchKernelExC(&cfg, fn, args);
}

cudaError_t launch_select(const uint8_t* accept, int32_t k_max, int32_t group, int32_t batch, int32_t* spec_count,
                          uint8_t* active, int32_t* idx, int32_t* n_active, cudaStream_t stream) {
    select_kernel<<<1, SPECA_MAX_BATCH, 0, stream>>>(accept, k_max, group, batch, spec_count, active, idx, n_active);
    return cudaGetLastError();
}

cudaError_t launch_activate(uint64_t mask_bits, int32_t batch, int32_t* spec_count, uint8_t* active,
                            cudaStream_t stream) {
    activate_kernel<<<1, SPECA_MAX_BATCH, 0, stream>>>(mask_bits, batch, spec_count, active);
    return cudaGetLastError();
}

static int occupancy(const void* kernel) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, kThreads, 0) != cudaSuccess || n < 1) n = 1;
    return n;
}

int ctas_per_sm_update(int dtype, int order) {
    return occupancy(dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, true>(order)
                                         : stream_kernel_for<SPECA_F32, true>(order));
}
int ctas_per_sm_forecast(int dtype, int order) {
    return occupancy(dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, false>(order)
                                         : stream_kernel_for<SPECA_F32, false>(order));
}
int ctas_per_sm_verify(int dtype, int order) {
    return occupancy(dtype == SPECA_BF16 ? verify_kernel_for<SPECA_BF16>(order) : verify_kernel_for<SPECA_F32>(order));
}

}  // namespace speca
