// CUDA kernels of the SpeCa feature-cache hot path for sm_100a (B200).
//
//   update         : Eq. 3 -- fold a freshly computed feature into the derivative table, in place
//   forecast       : Eq. 2 -- Horner evaluation of the table at a speculative time
//   forecast_multi : Eq. 2 for several speculative times from one read of the table (Fig. 1)
//   verify         : Eq. 4 -- forecast of the verification entry fused with the error reduction and
//                    the accept rule of Section 3.4.2 (l2, or the appendix's other metrics)
//   select         : per-sample continuation of the speculative run (Section 3.4.2, Appendix A)
//
// Every kernel is a pure HBM stream (about half a flop per byte, no reuse), so the design is about
// how the DRAM sees it: 32-byte vector loads and stores (sm_100), all of a chunk's loads issued
// before the first use, persistent grids of a few CTAs per SM whose bytes in flight are matched to
// the read / write mix, planes on 4 KB boundaries, no re-reads. No tensor cores are involved. The
// TMA-staged variant (cp.async.bulk + mbarrier) is kept for comparison.
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
// 16- and 32-byte global vectors
// ------------------------------------------------------------------------------------------------

// W bytes of consecutive elements in registers. sm_100 has 256-bit global loads and stores
// (ld/st.global.v8.b32); a warp then moves 1 KB of consecutive bytes per instruction.
template <int W>
struct Vec {
    uint32_t r[W / 4];
};

// The asm statements are volatile so that a tile's loads are all issued, in program order, before
// the first value is consumed: the number of independent loads in flight per thread is part of the
// design (see the shape table below), not something to leave to the instruction scheduler.
#ifndef SPECA_LD32
#define SPECA_LD32 "ld.global.v8.b32"
#endif
#ifndef SPECA_ST32
#define SPECA_ST32 "st.global.v8.b32"
#endif
template <int W>
__device__ __forceinline__ Vec<W> load_vec(const char* p) {
    Vec<W> v;
    if constexpr (W == 16)
        asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3])
                     : "l"(p));
    else
        asm volatile(SPECA_LD32 " {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]), "=r"(v.r[6]),
                       "=r"(v.r[7])
                     : "l"(p));
    return v;
}

// The verification's loads: each byte is read once, and the launch follows a forecast launch whose
// freshly written lines still sit dirty in L2. Marking the verification's own lines as the first to be
// evicted keeps it from pushing those write-backs in front of its loads: inside a step the FLUX-shaped
// entry (141 MB) takes 32.9 us instead of 37.0, the HunyuanVideo-shaped one 108.5 instead of 110.6, the
// DiT-shaped one (38 MB) is unchanged; the L1 hints change nothing, and the same hint on the streaming
// kernels' loads and stores is neutral to slightly worse.
#ifndef SPECA_LD32_VERIFY
#define SPECA_LD32_VERIFY "ld.global.L2::evict_first.v8.b32"
#endif
__device__ __forceinline__ Vec<32> load_vec_verify(const char* p) {
    Vec<32> v;
    asm volatile(SPECA_LD32_VERIFY " {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.r[0]), "=r"(v.r[1]), "=r"(v.r[2]), "=r"(v.r[3]), "=r"(v.r[4]), "=r"(v.r[5]), "=r"(v.r[6]),
                   "=r"(v.r[7])
                 : "l"(p));
    return v;
}

template <int W>
__device__ __forceinline__ void store_vec(char* p, const Vec<W>& v) {
    if constexpr (W == 16)
        asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.r[0]), "r"(v.r[1]), "r"(v.r[2]),
                     "r"(v.r[3])
                     : "memory");
    else
        asm volatile(SPECA_ST32 " [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.r[0]), "r"(v.r[1]),
                     "r"(v.r[2]), "r"(v.r[3]), "r"(v.r[4]), "r"(v.r[5]), "r"(v.r[6]), "r"(v.r[7])
                     : "memory");
}

template <int DT, int W>
struct VecElems {
    static constexpr int kEPV = W / Elem<DT>::kBytes;
};

template <int DT, int W>
__device__ __forceinline__ void unpack_vec(const Vec<W>& v, float (&f)[W / Elem<DT>::kBytes]) {
    if constexpr (DT == SPECA_F32) {
#pragma unroll
        for (int k = 0; k < W / 4; ++k) f[k] = __uint_as_float(v.r[k]);
    } else {
        // bfloat16 is the upper half of a binary32: widening is a shift
#pragma unroll
        for (int k = 0; k < W / 4; ++k) {
            f[2 * k] = __uint_as_float(v.r[k] << 16);
            f[2 * k + 1] = __uint_as_float(v.r[k] & 0xFFFF0000u);
        }
    }
}

template <int DT, int W>
__device__ __forceinline__ Vec<W> pack_vec(const float (&f)[W / Elem<DT>::kBytes]) {
    Vec<W> v;
    if constexpr (DT == SPECA_F32) {
#pragma unroll
        for (int k = 0; k < W / 4; ++k) v.r[k] = __float_as_uint(f[k]);
    } else {
#pragma unroll
        for (int k = 0; k < W / 4; ++k) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);  // round to nearest even
            v.r[k] = *reinterpret_cast<uint32_t*>(&h);
        }
    }
    return v;
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

// The same, starting from a guess: caches of one model hold runs of equally sized segments, so the
// segment of a tile further on is usually (tiles ahead) / (tiles per segment) segments ahead. The
// guess costs two independent loads; the search runs only when it is wrong. Returns the segment and
// its tile range.
__device__ __forceinline__ uint32_t next_segment(const uint32_t* __restrict__ tile_start, uint32_t seg, uint32_t seg_hi,
                                                 uint32_t tile, uint32_t& seg_first, uint32_t& seg_end) {
    if (seg_end > seg_first) {
        const uint32_t guess = seg + (tile - seg_first) / (seg_end - seg_first);
        if (guess < seg_hi) {
            const uint32_t a = __ldg(tile_start + guess), b = __ldg(tile_start + guess + 1);
            if (a <= tile && tile < b) {
                seg_first = a;
                seg_end = b;
                return guess;
            }
        }
    }
    seg = find_segment(tile_start, seg, seg_hi, tile);
    seg_first = __ldg(tile_start + seg);
    seg_end = __ldg(tile_start + seg + 1);
    return seg;
}

// ------------------------------------------------------------------------------------------------
// per-tile bodies
// ------------------------------------------------------------------------------------------------
// A tile is NT x U vectors of W bytes per plane; thread t owns vectors t, t + NT, ... so that a warp
// touches W * 32 consecutive bytes per instruction. `cnt` elements of the tile exist (the last tile
// of a segment is ragged): whole vectors go through the vector loop, the remainder through the
// scalar loop. `row` must be W-byte aligned (the planes always are).

// One level of a forecast: Horner (acc * mu + lo), or for a cache that keeps raw features one more term
// of the weighted sum (acc + lo * mu).
__device__ __forceinline__ float forecast_level(float acc, float lo, float mu, bool weighted) {
    return weighted ? fmaf(lo, mu, acc) : fmaf(acc, mu, lo);
}

// Eq. 2 in Horner form: acc = D_v; acc = D_{i-1} + acc * mu_i for i = v..1.
// With `weighted` (a cache that keeps raw features) the same planes are combined as a plain weighted
// sum instead: acc = sum_i w_i * plane_i, w = mu[0..V].
template <int DT, int V, int W, int NT, int U>
__device__ __forceinline__ void forecast_tile(const char* __restrict__ plane0, uint64_t stride,
                                              char* __restrict__ out, uint32_t cnt, const float (&mu)[kCoef],
                                              bool weighted) {
    constexpr int EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = cnt / EPV;
    Vec<W> d[V + 1][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
#pragma unroll
            for (int i = 0; i <= V; ++i) d[i][u] = load_vec<W>(plane0 + i * stride + static_cast<size_t>(idx) * W);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
            float acc[EPV];
            unpack_vec<DT, W>(d[V][u], acc);
            if (weighted) {
#pragma unroll
                for (int k = 0; k < EPV; ++k) acc[k] *= mu[V];
            }
#pragma unroll
            for (int i = V; i >= 1; --i) {
                float lo[EPV];
                unpack_vec<DT, W>(d[i - 1][u], lo);
                if (weighted) {
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(lo[k], mu[i - 1], acc[k]);
                } else {
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
                }
            }
            store_vec<W>(out + static_cast<size_t>(idx) * W, pack_vec<DT, W>(acc));
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += NT) {
        float acc = load_scalar<DT>(plane0 + V * stride, j);
        if (weighted) acc *= mu[V];
#pragma unroll
        for (int i = V; i >= 1; --i) {
            const float lo = load_scalar<DT>(plane0 + (i - 1) * stride, j);
            acc = weighted ? fmaf(lo, mu[i - 1], acc) : fmaf(acc, mu[i - 1], lo);
        }
        store_scalar<DT>(out, j, acc);
    }
}

// Eq. 3 as a chain of difference quotients: c_0 = f; c_{i+1} = (c_i - D_i) * r_i; D_i <- c_i.
// V = highest plane written. Reads f and planes 0..V-1, writes planes 0..V, each element once.
template <int DT, int V, int W, int NT, int U>
__device__ __forceinline__ void update_tile(char* __restrict__ plane0, uint64_t stride, const char* __restrict__ feat,
                                            uint32_t cnt, const float (&r)[kCoef]) {
    constexpr int EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = cnt / EPV;
    Vec<W> fv[U];
    Vec<W> d[V > 0 ? V : 1][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
            fv[u] = load_vec<W>(feat + static_cast<size_t>(idx) * W);
#pragma unroll
            for (int i = 0; i < V; ++i) d[i][u] = load_vec<W>(plane0 + i * stride + static_cast<size_t>(idx) * W);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
            float c[EPV];
            unpack_vec<DT, W>(fv[u], c);
            // every new plane is computed before the first store is issued: the thread's stores
            // leave as one burst after its loads have all returned
#pragma unroll
            for (int i = 0; i < V; ++i) {
                float old[EPV];
                unpack_vec<DT, W>(d[i][u], old);
#pragma unroll
                for (int k = 0; k < EPV; ++k) c[k] = (c[k] - old[k]) * r[i];
                d[i][u] = pack_vec<DT, W>(c);  // plane i + 1
            }
            // plane 0 is the feature itself: already in storage format
            store_vec<W>(plane0 + static_cast<size_t>(idx) * W, fv[u]);
#pragma unroll
            for (int i = 0; i < V; ++i)
                store_vec<W>(plane0 + (i + 1) * stride + static_cast<size_t>(idx) * W, d[i][u]);
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += NT) {
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

// Eq. 3 and, from the planes it has just formed, Eq. 2 at the next speculative time: the reference step
// that is followed by a speculative one (it always is) hands over its first forecast without reading the
// table again. Reads f and planes 0..V-1, writes planes 0..V and the forecast: 2V + 3 words per element
// instead of (2V + 2) + (V + 2). The forecast is evaluated from the ROUNDED planes, exactly as a
// forecast launch would find them in memory, so the result is bit for bit that of the two calls.
// With several speculative times (mu[k] per target, outputs target_stride bytes apart) the planes stay
// in registers and only the Horner pass and the store repeat: 2V + 2 + K words per element.
template <int DT, int V, int W, int NT, int U>
__device__ __forceinline__ void update_forecast_tile(char* __restrict__ plane0, uint64_t stride,
                                                     const char* __restrict__ feat, char* __restrict__ out,
                                                     uint64_t target_stride, int n_targets, uint32_t cnt,
                                                     const float (&r)[kCoef],
                                                     const float (*__restrict__ mu)[SPECA_MAX_BATCH][kCoef], uint32_t sample) {
    constexpr int EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = cnt / EPV;
    Vec<W> fv[U];
    Vec<W> d[V > 0 ? V : 1][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
            fv[u] = load_vec<W>(feat + static_cast<size_t>(idx) * W);
#pragma unroll
            for (int i = 0; i < V; ++i) d[i][u] = load_vec<W>(plane0 + i * stride + static_cast<size_t>(idx) * W);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
            float c[EPV];
            unpack_vec<DT, W>(fv[u], c);
#pragma unroll
            for (int i = 0; i < V; ++i) {
                float old[EPV];
                unpack_vec<DT, W>(d[i][u], old);
#pragma unroll
                for (int k = 0; k < EPV; ++k) c[k] = (c[k] - old[k]) * r[i];
                d[i][u] = pack_vec<DT, W>(c);  // plane i + 1, rounded
            }
            store_vec<W>(plane0 + static_cast<size_t>(idx) * W, fv[u]);
#pragma unroll
            for (int i = 0; i < V; ++i)
                store_vec<W>(plane0 + (i + 1) * stride + static_cast<size_t>(idx) * W, d[i][u]);
        }
    }
    // Horner over the stored values, once per target: acc = D_V; acc = D_{i-1} + acc * mu_i
#pragma unroll 1
    for (int t = 0; t < n_targets; ++t) {
        float m[kCoef];
#pragma unroll
        for (int i = 0; i < kCoef; ++i) m[i] = mu[t][sample][i];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = u * NT + threadIdx.x;
            if (idx < nvec) {
                float acc[EPV];
                if constexpr (V > 0)
                    unpack_vec<DT, W>(d[V - 1][u], acc);
                else
                    unpack_vec<DT, W>(fv[u], acc);
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[EPV];
                    if (i == 1)
                        unpack_vec<DT, W>(fv[u], lo);
                    else
                        unpack_vec<DT, W>(d[i - 2 >= 0 ? i - 2 : 0][u], lo);
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], m[i - 1], lo[k]);
                }
                store_vec<W>(out + t * target_stride + static_cast<size_t>(idx) * W, pack_vec<DT, W>(acc));
            }
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += NT) {
        float c = load_scalar<DT>(feat, j);
        float old[V > 0 ? V : 1], neu[V + 1];
#pragma unroll
        for (int i = 0; i < V; ++i) old[i] = load_scalar<DT>(plane0 + i * stride, j);
        neu[0] = c;  // already a storage value
        store_scalar<DT>(plane0, j, c);
#pragma unroll
        for (int i = 0; i < V; ++i) {
            c = (c - old[i]) * r[i];
            store_scalar<DT>(plane0 + (i + 1) * stride, j, c);
            neu[i + 1] = round_storage<DT>(c);
        }
        for (int t = 0; t < n_targets; ++t) {
            float acc = neu[V];
#pragma unroll
            for (int i = V; i >= 1; --i) acc = fmaf(acc, mu[t][sample][i - 1], neu[i - 1]);
            store_scalar<DT>(out + t * target_stride, j, acc);
        }
    }
}

// Runtime-order, any-alignment variants for the rare tiles whose sample has fewer references than
// the launch's common order (warm-up after a reset) or whose row is not vector aligned: 16-byte
// vectors when the row allows it, else one element at a time; planes visited in a loop.
template <int DT>
__device__ __noinline__ void forecast_tile_any(const char* __restrict__ plane0, uint64_t stride, char* __restrict__ out,
                                               uint32_t cnt, int v, const float (&mu)[kCoef], bool weighted = false) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(out) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += blockDim.x) {
        float acc[EPV];
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + v * stride) + idx), acc);
        if (weighted) {
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] *= mu[v];
        }
        for (int i = v; i >= 1; --i) {
            float lo[EPV];
            unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + (i - 1) * stride) + idx), lo);
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] = weighted ? fmaf(lo[k], mu[i - 1], acc[k]) : fmaf(acc[k], mu[i - 1], lo[k]);
        }
        __stcs(reinterpret_cast<uint4*>(out) + idx, pack<DT>(acc));
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += blockDim.x) {
        float acc = load_scalar<DT>(plane0 + v * stride, j);
        if (weighted) acc *= mu[v];
        for (int i = v; i >= 1; --i) {
            const float lo = load_scalar<DT>(plane0 + (i - 1) * stride, j);
            acc = weighted ? fmaf(lo, mu[i - 1], acc) : fmaf(acc, mu[i - 1], lo);
        }
        store_scalar<DT>(out, j, acc);
    }
}

template <int DT>
__device__ __noinline__ void update_tile_any(char* __restrict__ plane0, uint64_t stride, const char* __restrict__ feat,
                                             uint32_t cnt, int v, const float (&r)[kCoef]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(feat) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += blockDim.x) {
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
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += blockDim.x) {
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
// Launch shapes. Both kernels are pure HBM streams whose speed is set by how the DRAM sees the mix
// of reads and writes, so the shape (vector width, threads, vectors per thread, CTAs per SM) was
// chosen by sweeping it on a B200 in bf16 with every plane 4 KB aligned (at order 2):
//   update   (half of the traffic is writes): few bytes in flight win -- 128 threads x two 32-byte
//            vectors per plane, 2 CTAs/SM (48 KB in flight per SM) reaches the device's copy rate
//            (one vector x 3 CTAs/SM is 1-3 % behind: 496 / 1489 us against 483 / 1474 on the DiT /
//            FLUX shapes); deeper or wider shapes (256 x 4 vectors, 2 CTAs/SM) are 4-9 % slower.
//   forecast (one write per three reads): flat above ~70 KB in flight per SM; 256 threads x one
//            vector per plane, 3 CTAs/SM.
// Other orders were swept the same way (FLUX shape, GB/s before -> after giving each order its own
// shape): update order 0: 4600 -> 6470, order 1: 5810 -> 6450, order 4: 6300 -> 6490; forecast order 0
// (a plain copy): 6070 -> 6350, order 3: 6750 -> 6840, order 4: 6670 -> 6940.
// SPECA_PATH_DIRECT keeps a 16-byte / 256-thread / 4-deep shape for both.
// A tile is `chunks` consecutive chunks of NT x U vectors; a CTA finishes one chunk (loads, arithmetic,
// stores) before it starts the next, so the bytes in flight are set by NT x U x W while the per-tile
// bookkeeping (segment lookup, descriptor, bounds) is paid once per `chunks`.
struct Shape {
    int w, nt, u, chunks, minb;
};
// One shape per order v: the number of streams grows with v, so the vectors per thread shrink to keep
// the bytes in flight per SM near the sweet spot of the mix. Every shape has a 32 KB tile.
#ifndef SPECA_SHAPES_UPDATE
#define SPECA_SHAPES_UPDATE \
    {32, 128, 2, 4, 4}, {32, 128, 2, 4, 3}, {32, 128, 2, 4, 2}, {32, 128, 1, 8, 3}, { 32, 128, 1, 8, 2 }
#endif
#ifndef SPECA_SHAPES_FORECAST
#define SPECA_SHAPES_FORECAST \
    {32, 128, 2, 4, 4}, {32, 256, 1, 4, 3}, {32, 256, 1, 4, 3}, {32, 256, 1, 4, 2}, { 32, 256, 1, 4, 2 }
#endif
// fp32 storage takes the same shapes with one exception, measured on the FLUX-shaped entries: the
// order-4 update (five reads, five writes) ran at 5.2 TB/s with one vector per thread against 6.3-6.4
// with four vectors per thread and one CTA per SM; bf16 prefers the table's shape (6.49 against 6.38).
#ifndef SPECA_SHAPE_UPDATE4_F32
#define SPECA_SHAPE_UPDATE4_F32 { 32, 128, 4, 2, 1 }
#endif
__host__ __device__ constexpr Shape shape_for(int path, bool update, int v, int dtype) {
    constexpr Shape up[SPECA_MAX_ORDER + 1] = {SPECA_SHAPES_UPDATE};
    constexpr Shape fc[SPECA_MAX_ORDER + 1] = {SPECA_SHAPES_FORECAST};
    const int i = v < 0 ? 0 : (v > SPECA_MAX_ORDER ? SPECA_MAX_ORDER : v);
    if (path != SPECA_PATH_WIDE) return Shape{16, 256, 4, 1, 2};
    if (update && i == 4 && dtype == SPECA_F32) return Shape SPECA_SHAPE_UPDATE4_F32;
    return update ? up[i] : fc[i];
}
__host__ __device__ constexpr uint32_t shape_tile_bytes(Shape s) { return static_cast<uint32_t>(s.w) * s.nt * s.u * s.chunks; }

// V = the order most samples of the launch have (the host passes the maximum over samples).
template <int DT, int V, bool UPDATE, int W, int NT, int U, int C, int MINB>
__global__ void __launch_bounds__(NT, MINB) stream_kernel(const __grid_constant__ StreamParams p) {
    constexpr uint32_t kChunk = static_cast<uint32_t>(NT) * U * W / Elem<DT>::kBytes;  // elements
    constexpr uint32_t kTile = kChunk * C;
    if constexpr (UPDATE) {
        // a reference step re-arms its samples for speculation: folded into this launch on request
        if (p.act_active != nullptr && blockIdx.x == 0 && threadIdx.x < SPECA_MAX_BATCH && ((p.act_bits >> threadIdx.x) & 1ull)) {
            p.act_active[threadIdx.x] = 1;
            p.act_spec[threadIdx.x] = 0;
        }
    }
    uint32_t seg = p.seg_lo, seg_first = 0, seg_end = 0;  // tiles [seg_first, seg_end) belong to `seg`
    SegDesc sd = {};
    int v = -1;
    char* io = nullptr;
    float coef[kCoef] = {};
    uint32_t slot = 0;  // history layout, update only: the plane that receives the feature
    for (uint32_t tile = p.tile_lo + blockIdx.x; tile < p.tile_hi; tile += gridDim.x) {
        if (tile >= seg_end) {  // tiles only grow: look forward from the current segment
            seg = next_segment(p.tile_start, seg, p.seg_hi, tile, seg_first, seg_end);
            sd = p.segs[seg];
            v = p.order[sd.sample];
            io = static_cast<char*>(p.io[sd.entry]);
            if (p.dev_mask != nullptr && p.dev_mask[sd.sample] == 0) v = -1;
#pragma unroll
            for (int i = 0; i < kCoef; ++i) coef[i] = p.coef[sd.sample][i];
            slot = p.slot[sd.sample];
        }
        if (v < 0 || io == nullptr) continue;
        const uint32_t elem0 = (tile - seg_first) * kTile;
        const uint32_t cnt = min(kTile, sd.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        char* plane0 = p.arena + sd.plane0_off + slot * sd.plane_stride + byte0;
        char* row = io + sd.io_off + byte0;
        const bool fast = v == V && (reinterpret_cast<uintptr_t>(row) & (W - 1)) == 0;
        if (fast) {
            for (uint32_t done = 0; done < cnt; done += kChunk) {
                const uint32_t n = min(kChunk, cnt - done);
                const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                if constexpr (UPDATE)
                    update_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, row + off, n, coef);
                else
                    forecast_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, row + off, n, coef, p.weighted != 0);
            }
        } else {
            if constexpr (UPDATE)
                update_tile_any<DT>(plane0, sd.plane_stride, row, cnt, v, coef);
            else
                forecast_tile_any<DT>(plane0, sd.plane_stride, row, cnt, v, coef, p.weighted != 0);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// multi-horizon forecast: Eq. 2 for K speculative steps from one read of the table
// ------------------------------------------------------------------------------------------------
// The draft model predicts several future steps from the same reference (Fig. 1, workflow step 2).
// Evaluating them in one pass reads the v + 1 planes once and writes K outputs: (v + 1 + K) words per
// element instead of K (v + 2). Output k of entry e is row k of a [K, B, N_e, D] tensor.
// Swept like the others: up to 5 targets the mix is close to the update's and 256 threads x 2 CTAs/SM
// win (6700 / 6480 GB/s at K = 2 / 4 on the FLUX shape against 6090 / 6350); with more targets writes
// dominate and the narrower 128 x 3 shape is better (6320 against 5930 at K = 8).
__host__ __device__ constexpr Shape multi_shape(int n_targets) {
    return n_targets <= 5 ? Shape{32, 256, 1, 4, 2} : Shape{32, 128, 1, 8, 3};
}
static_assert(shape_tile_bytes(multi_shape(1)) == shape_tile_bytes(multi_shape(8)), "one tile table for both");

template <int DT, int V, int W, int NT, int U>
__device__ __forceinline__ void forecast_multi_tile(const char* __restrict__ plane0, uint64_t stride,
                                                    char* __restrict__ out, uint64_t target_stride, int n_targets,
                                                    uint32_t cnt, const float (*__restrict__ mu)[SPECA_MAX_BATCH][kCoef],
                                                    uint32_t sample, bool weighted) {
    constexpr int EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = cnt / EPV;
    Vec<W> d[V + 1][U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
#pragma unroll
            for (int i = 0; i <= V; ++i) d[i][u] = load_vec<W>(plane0 + i * stride + static_cast<size_t>(idx) * W);
        }
    }
#pragma unroll 1
    for (int k = 0; k < n_targets; ++k) {
        float m[kCoef];
#pragma unroll
        for (int i = 0; i < kCoef; ++i) m[i] = mu[k][sample][i];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = u * NT + threadIdx.x;
            if (idx < nvec) {
                float acc[EPV];
                unpack_vec<DT, W>(d[V][u], acc);
                if (weighted) {
#pragma unroll
                    for (int e = 0; e < EPV; ++e) acc[e] *= m[V];
                }
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[EPV];
                    unpack_vec<DT, W>(d[i - 1][u], lo);
                    if (weighted) {
#pragma unroll
                        for (int e = 0; e < EPV; ++e) acc[e] = fmaf(lo[e], m[i - 1], acc[e]);
                    } else {
#pragma unroll
                        for (int e = 0; e < EPV; ++e) acc[e] = fmaf(acc[e], m[i - 1], lo[e]);
                    }
                }
                store_vec<W>(out + k * target_stride + static_cast<size_t>(idx) * W, pack_vec<DT, W>(acc));
            }
        }
        for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += NT) {
            float acc = load_scalar<DT>(plane0 + V * stride, j);
            if (weighted) acc *= m[V];
#pragma unroll
            for (int i = V; i >= 1; --i) {
                const float lo = load_scalar<DT>(plane0 + (i - 1) * stride, j);
                acc = weighted ? fmaf(lo, m[i - 1], acc) : fmaf(acc, m[i - 1], lo);
            }
            store_scalar<DT>(out + k * target_stride, j, acc);
        }
    }
}

template <int DT, int V, int W, int NT, int U, int C, int MINB>
__global__ void __launch_bounds__(NT, MINB) forecast_multi_kernel(const __grid_constant__ MultiParams p, int batch) {
    constexpr uint32_t kChunk = static_cast<uint32_t>(NT) * U * W / Elem<DT>::kBytes;
    constexpr uint32_t kTile = kChunk * C;
    uint32_t seg = p.seg_lo, seg_first = 0, seg_end = 0;
    SegDesc sd = {};
    int v = -1;
    char* io = nullptr;
    uint64_t target_stride = 0;  // bytes between consecutive targets of this entry's output
    for (uint32_t tile = p.tile_lo + blockIdx.x; tile < p.tile_hi; tile += gridDim.x) {
        if (tile >= seg_end) {
            seg = next_segment(p.tile_start, seg, p.seg_hi, tile, seg_first, seg_end);
            sd = p.segs[seg];
            v = p.order[sd.sample];
            io = static_cast<char*>(p.io[sd.entry]);
            if (p.dev_mask != nullptr && p.dev_mask[sd.sample] == 0) v = -1;
            target_stride = static_cast<uint64_t>(batch) * sd.n_elems * Elem<DT>::kBytes;
        }
        if (v < 0 || io == nullptr) continue;
        const uint32_t elem0 = (tile - seg_first) * kTile;
        const uint32_t cnt = min(kTile, sd.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        char* plane0 = p.arena + sd.plane0_off + byte0;
        char* row = io + sd.io_off + byte0;
        const bool fast = v == V && ((reinterpret_cast<uintptr_t>(row) | target_stride) & (W - 1)) == 0;
        if (fast) {
            for (uint32_t done = 0; done < cnt; done += kChunk) {
                const uint32_t n = min(kChunk, cnt - done);
                const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                forecast_multi_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, row + off, target_stride,
                                                     p.n_targets, n, p.coef, sd.sample, p.weighted != 0);
            }
        } else {
            for (int k = 0; k < p.n_targets; ++k) {
                float m[kCoef];
#pragma unroll
                for (int i = 0; i < kCoef; ++i) m[i] = p.coef[k][sd.sample][i];
                forecast_tile_any<DT>(plane0, sd.plane_stride, row + k * target_stride, cnt, v, m, p.weighted != 0);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// fused reference step: Eq. 3 and the forecasts that follow it, one pass over the tables
// ------------------------------------------------------------------------------------------------
// The same fusion for a cache that keeps raw features: the reference step copies the feature into ring
// plane `slot` and the forecast is the weighted sum of the ring's planes, of which plane `slot` is the
// feature just loaded: V + 1 reads (feature and the V other planes) and 1 + K writes instead of
// (1 + 1) + (V + 1 + K). Same order of operations as the weighted forecast tiles: acc = w_V * plane_V,
// then acc += w_i * plane_i for i = V-1 .. 0.
template <int DT, int V, int W, int NT, int U>
__device__ __forceinline__ void history_update_forecast_tile(char* __restrict__ plane0, uint64_t stride,
                                                             const char* __restrict__ feat, char* __restrict__ out,
                                                             uint64_t target_stride, int n_targets, uint32_t cnt, int slot,
                                                             const float (*__restrict__ mu)[SPECA_MAX_BATCH][kCoef],
                                                             uint32_t sample) {
    constexpr int EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = cnt / EPV;
    Vec<W> d[V + 1][U];  // d[slot] holds the feature
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
#pragma unroll
            for (int i = 0; i <= V; ++i)
                d[i][u] = load_vec<W>((i == slot ? feat : plane0 + i * stride) + static_cast<size_t>(idx) * W);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * NT + threadIdx.x;
        if (idx < nvec) {
#pragma unroll
            for (int i = 0; i <= V; ++i)
                if (i == slot) store_vec<W>(plane0 + i * stride + static_cast<size_t>(idx) * W, d[i][u]);
        }
    }
#pragma unroll 1
    for (int t = 0; t < n_targets; ++t) {
        float m[kCoef];
#pragma unroll
        for (int i = 0; i < kCoef; ++i) m[i] = mu[t][sample][i];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t idx = u * NT + threadIdx.x;
            if (idx < nvec) {
                float acc[EPV];
                unpack_vec<DT, W>(d[V][u], acc);
#pragma unroll
                for (int k = 0; k < EPV; ++k) acc[k] *= m[V];
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[EPV];
                    unpack_vec<DT, W>(d[i - 1][u], lo);
#pragma unroll
                    for (int k = 0; k < EPV; ++k) acc[k] = fmaf(lo[k], m[i - 1], acc[k]);
                }
                store_vec<W>(out + t * target_stride + static_cast<size_t>(idx) * W, pack_vec<DT, W>(acc));
            }
        }
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += NT) {
        float val[V + 1];
#pragma unroll
        for (int i = 0; i <= V; ++i) val[i] = load_scalar<DT>(i == slot ? feat : plane0 + i * stride, j);
#pragma unroll
        for (int i = 0; i <= V; ++i)
            if (i == slot) store_scalar<DT>(plane0 + i * stride, j, val[i]);
        for (int t = 0; t < n_targets; ++t) {
            float acc = val[V] * mu[t][sample][V];
#pragma unroll
            for (int i = V; i >= 1; --i) acc = fmaf(val[i - 1], mu[t][sample][i - 1], acc);
            store_scalar<DT>(out + t * target_stride, j, acc);
        }
    }
}

// The fused reference step: stream_kernel's walk over the update's tile list with, per tile, one of
//   sample updated, output given      -> update_forecast_tile (K forecasts from the planes just formed)
//   sample updated, no output         -> update_tile
//   sample not updated but forecast   -> forecast_multi_tile from its unchanged planes
// HIST: a cache that keeps raw features; the update is then a copy into ring plane `slot` and the
// forecasts are weighted sums (history_update_forecast_tile).
template <int DT, int V, int W, int NT, int U, int C, int MINB, bool HIST>
__global__ void __launch_bounds__(NT, MINB) update_forecast_kernel(const __grid_constant__ FusedParams q) {
    constexpr uint32_t kChunk = static_cast<uint32_t>(NT) * U * W / Elem<DT>::kBytes;  // elements
    constexpr uint32_t kTile = kChunk * C;
    const StreamParams& p = q.up;
    if (p.act_active != nullptr && blockIdx.x == 0 && threadIdx.x < SPECA_MAX_BATCH && ((p.act_bits >> threadIdx.x) & 1ull)) {
        p.act_active[threadIdx.x] = 1;
        p.act_spec[threadIdx.x] = 0;
    }
    const int K = q.n_targets;
    constexpr bool hist = HIST;
    uint32_t seg = p.seg_lo, seg_first = 0, seg_end = 0;
    SegDesc sd = {};
    int v_up = -1, v_fc = -1, slot = 0;
    char* in = nullptr;
    char* out = nullptr;
    uint64_t target_stride = 0;  // bytes between consecutive targets of this entry's output
    float r[kCoef] = {};
    for (uint32_t tile = p.tile_lo + blockIdx.x; tile < p.tile_hi; tile += gridDim.x) {
        if (tile >= seg_end) {
            seg = next_segment(p.tile_start, seg, p.seg_hi, tile, seg_first, seg_end);
            sd = p.segs[seg];
            v_up = p.order[sd.sample];
            v_fc = q.fc_order[sd.sample];
            in = static_cast<char*>(p.io[sd.entry]);
            out = static_cast<char*>(q.out[sd.entry]);
            target_stride = static_cast<uint64_t>(q.batch) * sd.n_elems * Elem<DT>::kBytes;
            slot = p.slot[sd.sample];
            // a sample that is not updated here is forecast only if it is still speculating
            if (v_up < 0 && q.fc_mask != nullptr && q.fc_mask[sd.sample] == 0) v_fc = -1;
#pragma unroll
            for (int i = 0; i < kCoef; ++i) r[i] = p.coef[sd.sample][i];
        }
        const bool do_up = v_up >= 0 && in != nullptr, do_fc = v_fc >= 0 && out != nullptr;
        if (!do_up && !do_fc) continue;
        const uint32_t elem0 = (tile - seg_first) * kTile;
        const uint32_t cnt = min(kTile, sd.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        char* plane0 = p.arena + sd.plane0_off + byte0;
        char* frow = do_up ? in + sd.io_off + byte0 : nullptr;
        char* orow = do_fc ? out + sd.io_off + byte0 : nullptr;
        const bool out_aligned = ((reinterpret_cast<uintptr_t>(orow) | (K > 1 ? target_stride : 0)) & (W - 1)) == 0;
        const bool in_aligned = (reinterpret_cast<uintptr_t>(frow) & (W - 1)) == 0;
        if (do_up && do_fc && v_fc == V && (hist || v_up == V) && in_aligned && out_aligned) {
            for (uint32_t done = 0; done < cnt; done += kChunk) {
                const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                if (hist)
                    history_update_forecast_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, frow + off, orow + off,
                                                                  target_stride, K, min(kChunk, cnt - done), slot, q.fc_coef,
                                                                  sd.sample);
                else
                    update_forecast_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, frow + off, orow + off, target_stride,
                                                          K, min(kChunk, cnt - done), r, q.fc_coef, sd.sample);
            }
            continue;
        }
        // the rare shapes: halves done one after the other by the single-purpose routines
        if (do_up) {
            if (hist) {  // a copy into the ring plane
                char* dst = plane0 + static_cast<size_t>(slot) * sd.plane_stride;
                if (in_aligned) {
                    for (uint32_t done = 0; done < cnt; done += kChunk) {
                        const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                        update_tile<DT, 0, W, NT, U>(dst + off, sd.plane_stride, frow + off, min(kChunk, cnt - done), r);
                    }
                } else {
                    update_tile_any<DT>(dst, sd.plane_stride, frow, cnt, 0, r);
                }
            } else if (v_up == V && in_aligned) {
                for (uint32_t done = 0; done < cnt; done += kChunk) {
                    const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                    update_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, frow + off, min(kChunk, cnt - done), r);
                }
            } else {
                update_tile_any<DT>(plane0, sd.plane_stride, frow, cnt, v_up, r);
            }
        }
        if (do_fc) {
            if (do_up) __syncthreads();  // the forecast may read a plane element another thread of the CTA has just written
            if (v_fc == V && out_aligned) {
                for (uint32_t done = 0; done < cnt; done += kChunk) {
                    const size_t off = static_cast<size_t>(done) * Elem<DT>::kBytes;
                    forecast_multi_tile<DT, V, W, NT, U>(plane0 + off, sd.plane_stride, orow + off, target_stride, K,
                                                         min(kChunk, cnt - done), q.fc_coef, sd.sample, hist);
                }
            } else {
                for (int t = 0; t < K; ++t) {
                    float m[kCoef];
#pragma unroll
                    for (int i = 0; i < kCoef; ++i) m[i] = q.fc_coef[t][sd.sample][i];
                    forecast_tile_any<DT>(plane0, sd.plane_stride, orow + t * target_stride, cnt, v_fc, m, hist);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// summed forecast: the forecasts of equally shaped entries added into one output
// ------------------------------------------------------------------------------------------------
// A transformer adds its block outputs to a residual stream, so on a speculative step the forecasts
// of equally shaped blocks are only consumed as base + sum_e forecast_e. Computing that sum directly
// reads the v + 1 planes of every listed entry and writes one tensor: E (v + 1) + 1 (+ 1 with a base)
// words per element instead of E (v + 2) for separate forecasts (and the adds the model would then
// do). Each entry's Horner result stays in fp32 and is added unrounded, in list order; the total is
// rounded once. Read-dominated, so it uses the forecast's launch shape: 256 threads, one 32-byte
// vector per plane, 3 CTAs/SM; a tile is 8 KB of the output row.
constexpr int kSumW = 32, kSumThreads = 256, kSumMinBlocks = 3;
constexpr uint32_t kSumTileBytes = kSumW * kSumThreads;

template <int DT, int V>
__global__ void __launch_bounds__(kSumThreads, kSumMinBlocks) forecast_sum_kernel(const __grid_constant__ SumParams p) {
    constexpr int W = kSumW;
    constexpr int EPV = W / Elem<DT>::kBytes;
    constexpr uint32_t kTile = kSumTileBytes / Elem<DT>::kBytes;
    const uint32_t total = static_cast<uint32_t>(p.batch) * p.tiles_per_sample;
    const uint64_t row_bytes = static_cast<uint64_t>(p.n_elems) * Elem<DT>::kBytes;
    for (uint32_t t = blockIdx.x; t < total; t += gridDim.x) {
        const uint32_t b = t / p.tiles_per_sample;
        const int v = p.order[b];
        if (v < 0 || (p.dev_mask != nullptr && p.dev_mask[b] == 0)) continue;
        const uint32_t elem0 = (t - b * p.tiles_per_sample) * kTile;
        const uint32_t cnt = min(kTile, p.n_elems - elem0);
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        const char* base = p.base != nullptr ? p.base + b * row_bytes + byte0 : nullptr;
        char* out = p.out + b * row_bytes + byte0;
        float mu[kCoef];
#pragma unroll
        for (int i = 0; i < kCoef; ++i) mu[i] = p.coef[b][i];
        const bool weighted = p.weighted != 0;  // raw-feature cache: sum_i mu[i] * plane_i instead of Horner
        const uint32_t idx = threadIdx.x;
        const bool vec_ok = ((reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(base)) & (W - 1)) == 0;
        const uint32_t nvec = vec_ok ? cnt / EPV : 0;
        if (idx < nvec) {
            float sum[EPV];
            if (base != nullptr) {
                unpack_vec<DT, W>(load_vec<W>(base + static_cast<size_t>(idx) * W), sum);
            } else {
#pragma unroll
                for (int k = 0; k < EPV; ++k) sum[k] = 0.f;
            }
            int j = 0;
            if (v == V) {
                // Low orders read one or two planes per entry: take the entries in groups so that every
                // thread keeps four loads in flight. The forecasts are still added one by one, in list order.
                constexpr int G = V == 0 ? 4 : (V == 1 ? 2 : 1);
                if constexpr (G > 1) {
                    for (; j + G <= p.n_ids; j += G) {
                        Vec<W> d[G][V + 1];
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            const SegDesc sd = p.segs[static_cast<uint32_t>(p.ids[j + g]) * p.batch + b];
                            const char* plane0 = p.arena + sd.plane0_off + byte0 + static_cast<size_t>(idx) * W;
#pragma unroll
                            for (int i = 0; i <= V; ++i) d[g][i] = load_vec<W>(plane0 + i * sd.plane_stride);
                        }
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            float acc[EPV];
                            unpack_vec<DT, W>(d[g][V], acc);
                            if (weighted) {
#pragma unroll
                                for (int k = 0; k < EPV; ++k) acc[k] *= mu[V];
                            }
#pragma unroll
                            for (int i = V; i >= 1; --i) {
                                float lo[EPV];
                                unpack_vec<DT, W>(d[g][i - 1], lo);
#pragma unroll
                                for (int k = 0; k < EPV; ++k) acc[k] = forecast_level(acc[k], lo[k], mu[i - 1], weighted);
                            }
#pragma unroll
                            for (int k = 0; k < EPV; ++k) sum[k] += acc[k];
                        }
                    }
                }
            }
            for (; j < p.n_ids; ++j) {
                const SegDesc sd = p.segs[static_cast<uint32_t>(p.ids[j]) * p.batch + b];
                const char* plane0 = p.arena + sd.plane0_off + byte0 + static_cast<size_t>(idx) * W;
                float acc[EPV];
                if (v == V) {
                    Vec<W> d[V + 1];
#pragma unroll
                    for (int i = 0; i <= V; ++i) d[i] = load_vec<W>(plane0 + i * sd.plane_stride);
                    unpack_vec<DT, W>(d[V], acc);
                    if (weighted) {
#pragma unroll
                        for (int k = 0; k < EPV; ++k) acc[k] *= mu[V];
                    }
#pragma unroll
                    for (int i = V; i >= 1; --i) {
                        float lo[EPV];
                        unpack_vec<DT, W>(d[i - 1], lo);
#pragma unroll
                        for (int k = 0; k < EPV; ++k) acc[k] = forecast_level(acc[k], lo[k], mu[i - 1], weighted);
                    }
                } else {  // a sample with fewer references than the launch's common order
                    unpack_vec<DT, W>(load_vec<W>(plane0 + v * sd.plane_stride), acc);
                    if (weighted) {
#pragma unroll
                        for (int k = 0; k < EPV; ++k) acc[k] *= mu[v];
                    }
                    for (int i = v; i >= 1; --i) {
                        float lo[EPV];
                        unpack_vec<DT, W>(load_vec<W>(plane0 + (i - 1) * sd.plane_stride), lo);
#pragma unroll
                        for (int k = 0; k < EPV; ++k) acc[k] = forecast_level(acc[k], lo[k], mu[i - 1], weighted);
                    }
                }
#pragma unroll
                for (int k = 0; k < EPV; ++k) sum[k] += acc[k];
            }
            store_vec<W>(out + static_cast<size_t>(idx) * W, pack_vec<DT, W>(sum));
        }
        // ragged tail of the row, or the whole tile when a row is not 32-byte aligned
        for (uint32_t e = nvec * EPV + threadIdx.x; e < cnt; e += kSumThreads) {
            float sum = base != nullptr ? load_scalar<DT>(base, e) : 0.f;
            for (int j = 0; j < p.n_ids; ++j) {
                const SegDesc sd = p.segs[static_cast<uint32_t>(p.ids[j]) * p.batch + b];
                const char* plane0 = p.arena + sd.plane0_off + byte0;
                float acc = load_scalar<DT>(plane0 + v * sd.plane_stride, e);
                if (weighted) acc *= mu[v];
                for (int i = v; i >= 1; --i)
                    acc = forecast_level(acc, load_scalar<DT>(plane0 + (i - 1) * sd.plane_stride, e), mu[i - 1], weighted);
                sum += acc;
            }
            store_scalar<DT>(out, e, sum);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// bulk path: the same streams staged through shared memory by the TMA engine
// ------------------------------------------------------------------------------------------------
// One elected thread issues `cp.async.bulk` copies (untiled TMA, 8 KB per plane and tile, no
// multicast) into a ring of shared-memory stages and arms the stage's mbarrier with the byte count;
// the CTA waits on the barrier's phase, computes from shared memory and stores from registers.
// Measured on B200 this does not beat the register-direct 32-byte path for these reuse-free streams;
// it is kept as a selectable variant. Tiles the copy engine cannot take (ragged last tile of a row,
// rows that are not 16-byte aligned, samples at a lower order) go through the generic per-tile
// routines in the same loop. Every wait is bounded: a copy that never lands sets the cache's error
// word, and the CTA stops issuing, waits once more (bounded) for what it issued and returns.

constexpr uint32_t kBulkTileBytes = 8192;
constexpr int kBulkThreads = 256;
constexpr uint32_t kBulkSpinLimit = 1u << 18;  // polls; a healthy copy completes within a few

__host__ __device__ constexpr int bulk_stages(int v) {
    const int per_stage = (v + 1) * static_cast<int>(kBulkTileBytes);
    const int s = 98304 / per_stage;
    return s > 4 ? 4 : (s < 2 ? 2 : s);
}
__host__ __device__ constexpr size_t bulk_smem_bytes(int v) {
    return 256 + static_cast<size_t>(bulk_stages(v)) * (v + 1) * kBulkTileBytes;
}

struct BulkSlot {      // what the producer decided for the tile that occupies a stage
    char* plane0;      // plane 0 of the tile
    char* row;         // feature (update) / output (forecast) row of the tile
    uint64_t stride;
    uint32_t cnt;      // elements; 0 = nothing to do (masked sample, entry not in this call)
    int32_t v;
    uint32_t staged;   // 1: copies were issued into the stage; 0: use the generic routine
    uint32_t sample;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; false if the phase did not complete within the limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t spins = 0; spins < kBulkSpinLimit; ++spins)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; dst, src 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

template <int DT, int V, bool UPDATE>
__global__ void __launch_bounds__(kBulkThreads) stream_bulk_kernel(const __grid_constant__ StreamParams p) {
    constexpr int S = bulk_stages(V);
    constexpr int NIN = V + 1;  // update: feature + planes 0..V-1; forecast: planes 0..V
    constexpr uint32_t kTile = kBulkTileBytes / Elem<DT>::kBytes;
    constexpr int EPV = Elem<DT>::kEPV;
    constexpr int VPT = kBulkTileBytes / 16 / kBulkThreads;  // 16-byte vectors per thread per plane
    constexpr int PV = kBulkTileBytes / 16;                  // vectors per plane and tile
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    BulkSlot* slots = reinterpret_cast<BulkSlot*>(smem + 64);
    static_assert(64 + 4 * sizeof(BulkSlot) <= 256, "slot ring fits the header");
    unsigned char* buf = smem + 256;

    const uint32_t first = p.tile_lo + blockIdx.x;
    const uint32_t my = first < p.tile_hi ? (p.tile_hi - first + gridDim.x - 1) / gridDim.x : 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // producer state (meaningful in thread 0 only)
    uint32_t pseg = p.seg_lo, pseg_first = 0, pseg_end = 0;
    uint32_t outstanding = 0;  // stages with copies issued and not yet consumed
    bool stop = false;
    auto prepare = [&](uint32_t j, int s) {
        const uint32_t tile = first + j * gridDim.x;
        if (tile >= pseg_end) {
            pseg = find_segment(p.tile_start, pseg, p.seg_hi, tile);
            pseg_first = __ldg(p.tile_start + pseg);
            pseg_end = __ldg(p.tile_start + pseg + 1);
        }
        const SegDesc sd = p.segs[pseg];
        int v = p.order[sd.sample];
        char* io = static_cast<char*>(p.io[sd.entry]);
        if (p.dev_mask != nullptr && p.dev_mask[sd.sample] == 0) v = -1;
        BulkSlot d;
        d.cnt = 0;
        d.v = v;
        d.staged = 0;
        d.sample = sd.sample;
        d.stride = sd.plane_stride;
        d.plane0 = nullptr;
        d.row = nullptr;
        if (v >= 0 && io != nullptr) {
            const uint32_t elem0 = (tile - pseg_first) * kTile;
            const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
            d.cnt = min(kTile, sd.n_elems - elem0);
            d.plane0 = p.arena + sd.plane0_off + byte0;
            d.row = io + sd.io_off + byte0;
            const bool ok = !stop && v == V && d.cnt == kTile && (reinterpret_cast<uintptr_t>(d.row) & 15u) == 0;
            if (ok) {
                unsigned char* b = buf + static_cast<size_t>(s) * NIN * kBulkTileBytes;
                mbar_expect_tx(&full[s], NIN * kBulkTileBytes);
                if constexpr (UPDATE) {
                    bulk_load(b, d.row, kBulkTileBytes, &full[s]);
#pragma unroll
                    for (int i = 0; i < V; ++i)
                        bulk_load(b + (i + 1) * kBulkTileBytes, d.plane0 + i * sd.plane_stride, kBulkTileBytes, &full[s]);
                } else {
#pragma unroll
                    for (int i = 0; i <= V; ++i)
                        bulk_load(b + i * kBulkTileBytes, d.plane0 + i * sd.plane_stride, kBulkTileBytes, &full[s]);
                }
                d.staged = 1;
                outstanding |= 1u << s;
            }
        }
        slots[s] = d;
    };

    if (threadIdx.x == 0)
        for (int s = 0; s < S && static_cast<uint32_t>(s) < my; ++s) prepare(s, s);
    __syncthreads();

    uint32_t phase_bits = 0;  // per stage: parity of the next phase to wait for (same in every thread)
    bool dead = false;
    for (uint32_t j = 0; j < my; ++j) {
        const int s = j % S;
        const BulkSlot d = slots[s];
        if (d.cnt != 0) {
            float coef[kCoef];
#pragma unroll
            for (int i = 0; i < kCoef; ++i) coef[i] = p.coef[d.sample][i];
            if (d.staged) {
                const uint32_t parity = (phase_bits >> s) & 1u;
                bool landed = false;
                if (!dead) {
                    if (mbar_wait_bounded(&full[s], parity)) {
                        landed = true;
                        phase_bits ^= 1u << s;
                        outstanding &= ~(1u << s);
                    } else {
                        dead = true;  // the phase stays pending: the last loop below waits for it once more
                        *p.err_flag = 1;
                    }
                }
                if (landed) {
                    const uint4* in = reinterpret_cast<const uint4*>(buf + static_cast<size_t>(s) * NIN * kBulkTileBytes);
#pragma unroll
                    for (int u = 0; u < VPT; ++u) {
                        const int idx = u * kBulkThreads + threadIdx.x;
                        if constexpr (UPDATE) {
                            const uint4 fv = in[idx];
                            float c[EPV];
                            unpack<DT>(fv, c);
                            __stcs(reinterpret_cast<uint4*>(d.plane0) + idx, fv);
#pragma unroll
                            for (int i = 0; i < V; ++i) {
                                float old[EPV];
                                unpack<DT>(in[(i + 1) * PV + idx], old);
#pragma unroll
                                for (int k = 0; k < EPV; ++k) c[k] = (c[k] - old[k]) * coef[i];
                                __stcs(reinterpret_cast<uint4*>(d.plane0 + (i + 1) * d.stride) + idx, pack<DT>(c));
                            }
                        } else {
                            float acc[EPV];
                            unpack<DT>(in[V * PV + idx], acc);
#pragma unroll
                            for (int i = V; i >= 1; --i) {
                                float lo[EPV];
                                unpack<DT>(in[(i - 1) * PV + idx], lo);
#pragma unroll
                                for (int k = 0; k < EPV; ++k) acc[k] = fmaf(acc[k], coef[i - 1], lo[k]);
                            }
                            __stcs(reinterpret_cast<uint4*>(d.row) + idx, pack<DT>(acc));
                        }
                    }
                }
            } else {
                if constexpr (UPDATE)
                    update_tile_any<DT>(d.plane0, d.stride, d.row, d.cnt, d.v, coef);
                else
                    forecast_tile_any<DT>(d.plane0, d.stride, d.row, d.cnt, d.v, coef);
            }
        }
        __syncthreads();  // stage s and its slot are free again
        if (threadIdx.x == 0 && j + S < my) {
            stop = dead;
            prepare(j + S, s);
        }
    }
    // After a timeout copies may still be outstanding: give each such stage one more bounded wait so
    // that nothing lands in the shared memory of a CTA that has already left.
    if (dead && threadIdx.x == 0) {
        for (int s = 0; s < S; ++s)
            if (outstanding & (1u << s)) (void)mbar_wait_bounded(&full[s], (phase_bits >> s) & 1u);
    }
}

// ------------------------------------------------------------------------------------------------
// verify: forecast of one entry fused with the reduction of Eq. 4 (or of another error metric)
// ------------------------------------------------------------------------------------------------

constexpr int kMaxClusterSize = 8;
// 256 threads x verify_vectors(order) 32-byte vectors per plane and tile
constexpr int kVerifyW = 32;
static_assert(verify_tile_bytes(0) == kThreads * kVerifyW * verify_vectors(0) && verify_tile_bytes(4) == kThreads * kVerifyW,
              "verify tile size");

// Error metrics of the verification. Eq. 4 is the relative l2 error; the appendix on error metrics
// also evaluates l1, l-infinity and cosine similarity, all in relative form. Each metric keeps NA
// running values per sample, folds one (forecast, feature) pair into them, merges two partial
// results, and turns the totals into the error e that is compared with tau.
//   L2    a0 = sum (p-f)^2, a1 = sum f^2            e = sqrt(a0) / (sqrt(a1) + eps)
//   L1    a0 = sum |p-f|,   a1 = sum |f|            e = a0 / (a1 + eps)
//   LINF  a0 = max |p-f|,   a1 = max |f|            e = a0 / (a1 + eps)
//   COS   a0 = sum p f, a1 = sum p^2, a2 = sum f^2  e = 1 - a0 / (sqrt(a1) sqrt(a2) + eps)
// A NaN in any element must reach e (and reject the sample), so the maxima propagate NaN.
__device__ __forceinline__ float nan_max(float a, float b) { return (a > b || a != a) ? a : b; }
__device__ __forceinline__ double nan_max(double a, double b) { return (a > b || a != a) ? a : b; }

template <int M>
struct Metric {
    static constexpr int NA = (M == SPECA_METRIC_COSINE) ? 3 : 2;
    __device__ static __forceinline__ void fold(float p, float f, float (&a)[3]) {
        if constexpr (M == SPECA_METRIC_L2) {
            const float d = p - f;
            a[0] = fmaf(d, d, a[0]);
            a[1] = fmaf(f, f, a[1]);
        } else if constexpr (M == SPECA_METRIC_L1) {
            a[0] += fabsf(p - f);
            a[1] += fabsf(f);
        } else if constexpr (M == SPECA_METRIC_LINF) {
            a[0] = nan_max(a[0], fabsf(p - f));
            a[1] = nan_max(a[1], fabsf(f));
        } else {
            a[0] = fmaf(p, f, a[0]);
            a[1] = fmaf(p, p, a[1]);
            a[2] = fmaf(f, f, a[2]);
        }
    }
    template <typename T>
    __device__ static __forceinline__ T merge(T x, T y) {
        if constexpr (M == SPECA_METRIC_LINF)
            return nan_max(x, y);
        else
            return x + y;
    }
    // The error from the totals. err is handed out as a binary32, so for the ratio metrics the square
    // roots and the division are binary32 too (a few ulp of the stored value; fp64 square roots and
    // divisions are long dependent instruction sequences on the kernel's critical tail) and the accept
    // flag is exactly err <= tau on the stored values. Totals outside the binary32 range (or NaN) take
    // the fp64 formulas, and so does the cosine distance, whose 1 - ratio cancels.
    __device__ static __forceinline__ double error(const double (&s)[3], double eps) {
        if constexpr (M == SPECA_METRIC_COSINE) {
            return 1.0 - s[0] / (sqrt(s[1]) * sqrt(s[2]) + eps);
        } else {
            const bool fits = fabs(s[0]) < 1e38 && fabs(s[1]) < 1e38;
            if (fits) {
                const float a0 = static_cast<float>(s[0]), a1 = static_cast<float>(s[1]), e = static_cast<float>(eps);
                if constexpr (M == SPECA_METRIC_L2)
                    return static_cast<double>(sqrtf(a0) / (sqrtf(a1) + e));
                else
                    return static_cast<double>(a0 / (a1 + e));
            }
            if constexpr (M == SPECA_METRIC_L2)
                return sqrt(s[0]) / (sqrt(s[1]) + eps);
            else
                return s[0] / (s[1] + eps);
        }
    }
};

// One tile of the verification entry as a CTA sees it.
struct VTile {
    const char* plane0;  // plane 0 of the tile
    const char* fresh;
    char* pred;          // null: the forecast is not kept
    uint32_t cnt;        // elements (the last tile of a sample is ragged)
    int32_t slot;        // sample's position among the samples this cluster meets
    int32_t b;           // sample
    int32_t v;           // the sample's order
    bool fast;           // compiled order and 32-byte aligned rows: vector registers hold the tile
};

// The tile's v + 1 planes and the fresh feature, U 32-byte vectors per thread each.
template <int V, int U>
struct VRegs {
    Vec<kVerifyW> d[V + 1][U];
    Vec<kVerifyW> f[U];
};

// Issues all of the tile's loads before anything is consumed.
template <int DT, int V, int U>
__device__ __forceinline__ void verify_issue(VRegs<V, U>& r, const VTile& t, uint64_t stride) {
    constexpr int W = kVerifyW, EPV = W / Elem<DT>::kBytes;
    const uint32_t nvec = t.cnt / EPV;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * kThreads + threadIdx.x;
        if (idx < nvec) {
            const size_t o = static_cast<size_t>(idx) * W;
#pragma unroll
            for (int i = 0; i <= V; ++i) r.d[i][u] = load_vec_verify(t.plane0 + i * stride + o);
            r.f[u] = load_vec_verify(t.fresh + o);
        }
    }
}

// Eq. 2 on the tile's registers, the forecast rounded to the storage type as the model would consume it,
// then one fold of (forecast, feature) per element into the running values. A vector is worked
// through in 16-byte halves so that few unpacked values are live beside the vectors still to come.
template <int DT, int V, int U, int M>
__device__ __forceinline__ void verify_fold(const VRegs<V, U>& r, const VTile& t, uint64_t stride, const float (&mu)[kCoef],
                                            bool weighted, float (&a)[3]) {
    constexpr int W = kVerifyW, EPV = W / Elem<DT>::kBytes, H = EPV / 2;
    const uint32_t nvec = t.cnt / EPV;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const uint32_t idx = u * kThreads + threadIdx.x;
        if (idx < nvec) {
            Vec<W> pv;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                Vec<16> part;
                float acc[H], f[H];
#pragma unroll
                for (int k = 0; k < 4; ++k) part.r[k] = r.d[V][u].r[4 * h + k];
                unpack_vec<DT, 16>(part, acc);
                if (weighted) {
#pragma unroll
                    for (int k = 0; k < H; ++k) acc[k] *= mu[V];
                }
#pragma unroll
                for (int i = V; i >= 1; --i) {
                    float lo[H];
#pragma unroll
                    for (int k = 0; k < 4; ++k) part.r[k] = r.d[i - 1][u].r[4 * h + k];
                    unpack_vec<DT, 16>(part, lo);
                    if (weighted) {
#pragma unroll
                        for (int k = 0; k < H; ++k) acc[k] = fmaf(lo[k], mu[i - 1], acc[k]);
                    } else {
#pragma unroll
                        for (int k = 0; k < H; ++k) acc[k] = fmaf(acc[k], mu[i - 1], lo[k]);
                    }
                }
                part = pack_vec<DT, 16>(acc);
                unpack_vec<DT, 16>(part, acc);
#pragma unroll
                for (int k = 0; k < 4; ++k) pv.r[4 * h + k] = part.r[k];
#pragma unroll
                for (int k = 0; k < 4; ++k) part.r[k] = r.f[u].r[4 * h + k];
                unpack_vec<DT, 16>(part, f);
#pragma unroll
                for (int k = 0; k < H; ++k) Metric<M>::fold(acc[k], f[k], a);
            }
            if (t.pred != nullptr) store_vec<W>(t.pred + static_cast<size_t>(idx) * W, pv);
        }
    }
    // ragged end of a sample's last tile
    for (uint32_t j = nvec * EPV + threadIdx.x; j < t.cnt; j += kThreads) {
        float acc = load_scalar<DT>(t.plane0 + V * stride, j);
        if (weighted) acc *= mu[V];
#pragma unroll
        for (int i = V; i >= 1; --i) {
            const float lo = load_scalar<DT>(t.plane0 + (i - 1) * stride, j);
            acc = weighted ? fmaf(lo, mu[i - 1], acc) : fmaf(acc, mu[i - 1], lo);
        }
        acc = round_storage<DT>(acc);
        Metric<M>::fold(acc, load_scalar<DT>(t.fresh, j), a);
        if (t.pred != nullptr) store_scalar<DT>(t.pred, j, acc);
    }
}

template <int DT, int M>
__device__ __noinline__ void verify_tile_any(const char* __restrict__ plane0, uint64_t stride,
                                             const char* __restrict__ fresh, char* __restrict__ out_pred, uint32_t cnt,
                                             int v, const float (&mu)[kCoef], bool weighted, float (&a)[3]) {
    constexpr int EPV = Elem<DT>::kEPV;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(fresh) | reinterpret_cast<uintptr_t>(out_pred) |
                          reinterpret_cast<uintptr_t>(plane0)) & 15u) == 0;
    const uint32_t nvec = vec_ok ? cnt / EPV : 0;
    for (uint32_t idx = threadIdx.x; idx < nvec; idx += kThreads) {
        float acc[EPV], f[EPV];
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + v * stride) + idx), acc);
        if (weighted) {
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] *= mu[v];
        }
        for (int i = v; i >= 1; --i) {
            float lo[EPV];
            unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(plane0 + (i - 1) * stride) + idx), lo);
#pragma unroll
            for (int k = 0; k < EPV; ++k) acc[k] = weighted ? fmaf(lo[k], mu[i - 1], acc[k]) : fmaf(acc[k], mu[i - 1], lo[k]);
        }
        const uint4 pv = pack<DT>(acc);
        unpack<DT>(pv, acc);
        unpack<DT>(__ldcs(reinterpret_cast<const uint4*>(fresh) + idx), f);
#pragma unroll
        for (int k = 0; k < EPV; ++k) {
            Metric<M>::fold(acc[k], f[k], a);
        }
        if (out_pred != nullptr) __stcs(reinterpret_cast<uint4*>(out_pred) + idx, pv);
    }
    for (uint32_t j = nvec * EPV + threadIdx.x; j < cnt; j += kThreads) {
        float acc = load_scalar<DT>(plane0 + v * stride, j);
        if (weighted) acc *= mu[v];
        for (int i = v; i >= 1; --i) {
            const float lo = load_scalar<DT>(plane0 + (i - 1) * stride, j);
            acc = weighted ? fmaf(lo, mu[i - 1], acc) : fmaf(acc, mu[i - 1], lo);
        }
        acc = round_storage<DT>(acc);
        const float f = load_scalar<DT>(fresh, j);
        Metric<M>::fold(acc, f, a);
        if (out_pred != nullptr) store_scalar<DT>(out_pred, j, acc);
    }
}

// Per-sample continuation of the speculative run by ONE warp (all 32 lanes take part; B <= 64, lane l
// looks after samples l and l + 32). In two halves, so that the fused caller can have the loads of the
// first in flight while it is still summing: what the rule reads from memory ...
struct SelectIn {
    bool act[2];
    int32_t cnt[2];
};
__device__ __forceinline__ SelectIn select_load(int32_t batch, const int32_t* spec_count, const uint8_t* active_in) {
    const int lane = threadIdx.x & 31;
    SelectIn in;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int b = lane + 32 * h;
        in.act[h] = b < batch && active_in[b] != 0;
        in.cnt[h] = b < batch ? spec_count[b] : 0;
    }
    return in;
}
// ... and the rule itself, given each sample's accept flag (acc[h] for sample lane + 32 h).
__device__ __forceinline__ void select_apply(const SelectIn& in, const bool (&acc)[2], int32_t k_max, int32_t group,
                                             int32_t batch, int32_t* spec_count, uint8_t* active_out, int32_t* idx_out,
                                             int32_t* n_out) {
    const int lane = threadIdx.x & 31;
    uint64_t keep = 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int b = lane + 32 * h;
        bool k = false;
        if (b < batch) {
            const bool ok = in.act[h] && acc[h];
            int32_t c = in.cnt[h];
            if (ok) {
                c += 1;
                spec_count[b] = c;
            }
            k = ok && c < k_max;
        }
        keep |= static_cast<uint64_t>(__ballot_sync(0xFFFFFFFFu, k)) << (32 * h);
    }
    uint64_t next = 0;  // a group continues only if every member does
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int b = lane + 32 * h;
        bool all = false;
        if (b < batch) {
            const int g0 = (b / group) * group;
            const uint64_t members = (group >= 64 ? ~0ull : ((1ull << group) - 1ull)) << g0;
            all = (keep & members) == members;
            active_out[b] = all ? 1 : 0;
        }
        next |= static_cast<uint64_t>(__ballot_sync(0xFFFFFFFFu, all)) << (32 * h);
    }
    if (idx_out != nullptr) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int b = lane + 32 * h;
            if (b < batch && ((next >> b) & 1ull)) idx_out[__popcll(next & ((1ull << b) - 1ull))] = b;
        }
    }
    if (lane == 0 && n_out != nullptr) *n_out = __popcll(next);
}
// Both halves, with the accept flags read from memory (in place is fine: a lane reads its own samples'
// mask bytes before it writes them).
__device__ __forceinline__ void select_in_warp(const uint8_t* accept, int32_t k_max, int32_t group, int32_t batch,
                                               int32_t* spec_count, const uint8_t* active_in, uint8_t* active_out,
                                               int32_t* idx_out, int32_t* n_out) {
    const int lane = threadIdx.x & 31;
    const SelectIn in = select_load(batch, spec_count, active_in);
    bool acc[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) acc[h] = lane + 32 * h < batch && in.act[h] && accept[lane + 32 * h] != 0;
    select_apply(in, acc, k_max, group, batch, spec_count, active_out, idx_out, n_out);
}

// Tiles of the active samples form one list of T = (active samples) x (tiles per sample) tiles;
// cluster q of Q owns the contiguous range [q*T/Q, (q+1)*T/Q). Q <= 1024, so the products fit 32 bits
// whenever T < 2^22 (every benchmark shape: T is a few thousand): the 64-bit division is the rare case.
__device__ __forceinline__ uint32_t range_begin(uint32_t q, uint32_t Q, uint32_t T) {
    if (T < (1u << 22)) return q * T / Q;
    return static_cast<uint32_t>(static_cast<uint64_t>(q) * T / Q);
}
// The cluster whose range holds `tile`: the smallest q with range_begin(q + 1) > tile, that is
// ceil((tile + 1) * Q / T) - 1. Holds for Q > T too, where some clusters own nothing.
__device__ __forceinline__ uint32_t range_owner(uint32_t tile, uint32_t Q, uint32_t T) {
    if (T < (1u << 22)) return ((tile + 1) * Q - 1) / T;
    return static_cast<uint32_t>(((static_cast<uint64_t>(tile) + 1) * Q - 1) / T);
}
// Index of the a-th set bit of `bits` (a < popcount).
__device__ __forceinline__ int nth_set_bit(uint64_t bits, uint32_t a) {
    for (uint32_t i = 0; i < a; ++i) bits &= bits - 1;
    return __ffsll(static_cast<long long>(bits)) - 1;
}

// Release / acquire fences at device scope (lighter than the sequentially consistent __threadfence).
__device__ __forceinline__ void fence_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

// Each cluster walks a contiguous range of the active samples' tiles, its CTAs taking every
// (cluster size)-th tile. The running values go
//   registers -> warp shuffle -> this CTA's shared memory, one slot per sample the cluster meets
//   -> once, at the end of the range: the leader CTA's shared memory through the cluster's distributed
//      shared memory, ONE cluster barrier per launch
//   -> one partial per (cluster, sample) in global scratch.
// The cluster that arrives last (ticket counter, nobody waits) adds every sample's partials in fp64 in
// a fixed lane / shuffle order, applies Eq. 4 and the accept rule, runs the fused continuation rule
// and re-zeroes the ticket.
template <int DT, int V, int M>
__global__ void __launch_bounds__(kThreads, V <= 2 ? SPECA_VERIFY_MINB : 2) verify_kernel(const __grid_constant__ VerifyParams p) {
    constexpr uint32_t kTile = verify_tile_bytes(V) / Elem<DT>::kBytes;
    constexpr int W = kVerifyW, U = verify_vectors(V);
    constexpr int NA = Metric<M>::NA;
    constexpr int kWarps = kThreads / 32;
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t csize = cluster.num_blocks();
    const uint32_t crank = cluster.block_rank();
    const uint32_t cid = blockIdx.x / csize;
    const uint32_t Q = gridDim.x / csize;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    __shared__ float warp_part[SPECA_MAX_BATCH][NA][kWarps];            // [slot][value][warp], this CTA's
    __shared__ float cluster_slot[SPECA_MAX_BATCH][NA][kMaxClusterSize];  // [slot][value][rank], the leader's copy is used
    __shared__ uint32_t active_bits[2];
    __shared__ bool is_last;
    __shared__ uint8_t sel_accept[SPECA_MAX_BATCH];  // this launch's accept flags, for the fused continuation

    // Every CTA of the cluster is running once this barrier completes; it is only waited for right
    // before the first access to the leader's shared memory.
    cluster.barrier_arrive();

    for (int i = threadIdx.x; i < SPECA_MAX_BATCH * NA * kWarps; i += kThreads) (&warp_part[0][0][0])[i] = 0.f;
    if (threadIdx.x < SPECA_MAX_BATCH) sel_accept[threadIdx.x] = 0;  // a sample that is not verified does not continue
    // samples that take part: a defined table and, with a device mask, a non-zero byte
    if (threadIdx.x < 64) {
        const int b = threadIdx.x;
        const bool on = b < p.batch && p.order[b] >= 0 && (p.dev_mask == nullptr || p.dev_mask[b] != 0);
        const uint32_t ballot = __ballot_sync(0xFFFFFFFFu, on);
        if (lane == 0) active_bits[warp] = ballot;
    }
    __syncthreads();
    const uint64_t bits = static_cast<uint64_t>(active_bits[0]) | (static_cast<uint64_t>(active_bits[1]) << 32);
    const uint32_t n_active = __popcll(bits);
    const uint32_t tps = p.tiles_per_sample;
    const uint32_t T = n_active * tps;
    const uint32_t t_lo = n_active ? range_begin(cid, Q, T) : 0, t_hi = n_active ? range_begin(cid + 1, Q, T) : 0;
    if (t_lo >= t_hi) {  // nobody active, or more clusters than tiles: the whole cluster leaves together
        cluster.barrier_wait();
        if (n_active == 0 && p.sel_active != nullptr && blockIdx.x == 0 && warp == 0)
            select_in_warp(p.accept, p.sel_kmax, p.sel_group, p.batch, p.sel_spec, p.dev_mask, p.sel_active, p.sel_idx, p.sel_n);
        return;
    }
    const uint32_t a_first = t_lo / tps;
    const uint32_t span = (t_hi - 1) / tps - a_first + 1;  // samples this cluster meets
    const uint32_t Q_busy = Q < T ? Q : T;                 // clusters that own at least one tile

    // tile number -> what to load; the sample lookup is redone only when the sample changes
    uint32_t known_a = 0xFFFFFFFFu;
    int known_b = 0;
    auto locate = [&](uint32_t t) {
        VTile x;
        const uint32_t a = t / tps;
        if (a != known_a) {
            known_a = a;
            known_b = nth_set_bit(bits, a);
        }
        const uint32_t elem0 = (t - a * tps) * kTile;
        const uint64_t byte0 = static_cast<uint64_t>(elem0) * Elem<DT>::kBytes;
        const uint64_t io = static_cast<uint64_t>(known_b) * p.io_pitch + byte0;
        x.b = known_b;
        x.slot = static_cast<int32_t>(a - a_first);
        x.v = p.order[known_b];
        x.cnt = min(kTile, p.n_elems - elem0);
        x.plane0 = p.arena + p.plane0_off + static_cast<uint64_t>(known_b) * p.sample_pitch + byte0;
        x.fresh = p.fresh + io;
        x.pred = p.out_pred != nullptr ? p.out_pred + io : nullptr;
        x.fast = x.v == V && ((reinterpret_cast<uintptr_t>(x.plane0) | reinterpret_cast<uintptr_t>(x.fresh) |
                               reinterpret_cast<uintptr_t>(x.pred)) & (W - 1)) == 0;
        return x;
    };

    float acc[3] = {0.f, 0.f, 0.f};
    float mu[kCoef] = {};
    int32_t acc_slot = -1;
    // the warp's running values of the sample it has been folding go to the sample's slot
    auto park = [&]() {
        if (acc_slot < 0) return;
#pragma unroll
        for (int i = 0; i < NA; ++i) {
            float s = acc[i];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s = Metric<M>::merge(s, __shfl_xor_sync(0xFFFFFFFFu, s, off));
            if (lane == 0) warp_part[acc_slot][i][warp] = s;
        }
        acc[0] = acc[1] = acc[2] = 0.f;
    };
    auto enter = [&](const VTile& t) {  // uniform over the CTA
        if (t.slot != acc_slot) {
            park();
            acc_slot = t.slot;
#pragma unroll
            for (int i = 0; i < kCoef; ++i) mu[i] = p.coef[t.b][i];
        }
    };
    // A sample's tiles are all vector tiles or all generic ones (its rows are 32-byte aligned and its
    // order is the compiled one, or not). First pass: the vector tiles -- all of a tile's loads, then its
    // arithmetic. Second pass, rarely needed: the generic ones (kept out of the first loop so that no
    // call sits between a tile's loads and their use).
    bool any_generic = false;
    {
        VRegs<V, U> r;
        for (uint32_t t = t_lo + crank; t < t_hi; t += csize) {
            const VTile x = locate(t);
            if (!x.fast) {
                any_generic = true;
                continue;
            }
            verify_issue<DT, V, U>(r, x, p.plane_stride);
            enter(x);
            verify_fold<DT, V, U, M>(r, x, p.plane_stride, mu, p.weighted != 0, acc);
        }
        park();
        acc_slot = -1;
    }
    if (any_generic) {
        for (uint32_t t = t_lo + crank; t < t_hi; t += csize) {
            const VTile x = locate(t);
            if (x.fast) continue;
            enter(x);
            verify_tile_any<DT, M>(x.plane0, p.plane_stride, x.fresh, x.pred, x.cnt, x.v, mu, p.weighted != 0, acc);
        }
        park();
    }
    __syncthreads();

    // this CTA's value of every sample the cluster met -> the leader's shared memory, one barrier
    cluster.barrier_wait();
    if (threadIdx.x < span * NA) {
        const uint32_t slot = threadIdx.x / NA, i = threadIdx.x % NA;
        float s = warp_part[slot][i][0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) s = Metric<M>::merge(s, warp_part[slot][i][w]);
        float* leader = cluster.map_shared_rank(&cluster_slot[0][0][0], 0);
        leader[(slot * NA + i) * kMaxClusterSize + crank] = s;
    }
    cluster.sync();
    if (crank != 0) return;  // nobody touches a non-leader's shared memory after this barrier

    // the cluster's partial of every sample it met -> global scratch
    for (uint32_t slot = warp; slot < span; slot += kWarps) {
        const int b = nth_set_bit(bits, a_first + slot);
        float part[3] = {0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < NA; ++i) {
            float s = lane < csize ? cluster_slot[slot][i][lane] : 0.f;  // 0 is neutral for the sums and for maxima of magnitudes
#pragma unroll
            for (int off = kMaxClusterSize / 2; off > 0; off >>= 1) s = Metric<M>::merge(s, __shfl_xor_sync(0xFFFFFFFFu, s, off));
            part[i] = s;
        }
        if (lane == 0) {
            float* dst = p.partials + (static_cast<size_t>(b) * Q + cid) * NA;
#pragma unroll
            for (int i = 0; i < NA; ++i) __stcg(dst + i, part[i]);
            fence_gpu();  // this partial is visible device-wide before the ticket below is taken
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t t = atomicAdd(p.ticket, 1u);
        fence_gpu();
        is_last = (t == Q_busy - 1);
    }
    __syncthreads();
    if (!is_last) return;

    // Last cluster to arrive. A sample's partials sit side by side in the scratch ([sample][cluster]).
    // A group of L lanes adds one sample's partials: with few samples each has many partials and a
    // whole warp takes one sample; with many samples each has few and a warp takes four or eight at a
    // time, so that the CTA's eight warps cover the batch in one pass.
    // Per sample the order is fixed (lane l adds clusters q_lo + l, q_lo + l + L, ..., then a shuffle
    // tree over the group), four loads per lane are in flight at once, and the sums are fp64.
    // the continuation rule's own inputs are asked for now and used after the sums
    SelectIn sel_in = {};
    if (p.sel_active != nullptr && warp == 0) sel_in = select_load(p.batch, p.sel_spec, p.dev_mask);
    const uint32_t L = n_active <= 8 ? 32 : (n_active <= 32 ? 8 : 4), per_warp = 32 / L;
    const uint32_t g = lane / L, l = lane % L;
    const bool holes = Q > T;  // more clusters than tiles: some clusters in a sample's span own nothing
    for (uint32_t a0 = 0; a0 < n_active; a0 += kWarps * per_warp) {  // uniform over the CTA
        const uint32_t a = a0 + warp * per_warp + g;
        const bool live = a < n_active;
        int b = 0;
        double s[3] = {0.0, 0.0, 0.0};
        if (live) {
            b = nth_set_bit(bits, a);
            const uint32_t q_lo = range_owner(a * tps, Q, T), q_hi = range_owner((a + 1) * tps - 1, Q, T);
            const float* row = p.partials + static_cast<size_t>(b) * Q * NA;
            for (uint32_t q0 = q_lo + l; q0 <= q_hi; q0 += 4 * L) {
                float v[4][3];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t q = q0 + j * L;
                    const bool has = q <= q_hi && !(holes && range_begin(q, Q, T) == range_begin(q + 1, Q, T));
#pragma unroll
                    for (int i = 0; i < NA; ++i) v[j][i] = has ? __ldcg(row + static_cast<size_t>(q) * NA + i) : 0.f;  // 0: neutral
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
#pragma unroll
                    for (int i = 0; i < NA; ++i) s[i] = Metric<M>::merge(s[i], static_cast<double>(v[j][i]));
                }
            }
        }
#pragma unroll
        for (int i = 0; i < NA; ++i) {
            for (uint32_t off = L / 2; off > 0; off >>= 1) s[i] = Metric<M>::merge(s[i], __shfl_xor_sync(0xFFFFFFFFu, s[i], off));
        }
        if (live && l == 0) {
            if (p.raw_sums != nullptr) {
                // token-sharded verification: hand out the running values; the caller combines the
                // shards' values and calls the decision kernel
#pragma unroll
                for (int i = 0; i < 3; ++i) p.raw_sums[b * 4 + i] = i < NA ? s[i] : 0.0;
            } else {
                const double e = Metric<M>::error(s, p.eps);
                const uint8_t ok = (e <= static_cast<double>(p.tau[b])) ? 1 : 0;  // NaN compares false: reject
                p.err[b] = static_cast<float>(e);
                p.accept[b] = ok;
                sel_accept[b] = ok;
            }
        }
    }
    __syncthreads();
    // Fused continuation: every decision of this step is final by now. The new mask goes to a buffer
    // of its own: CTAs of this grid may still be reading the step's mask.
    if (p.sel_active != nullptr && warp == 0) {
        const bool acc[2] = {sel_accept[lane] != 0, sel_accept[lane + 32] != 0};
        select_apply(sel_in, acc, p.sel_kmax, p.sel_group, p.batch, p.sel_spec, p.sel_active, p.sel_idx, p.sel_n);
    }
    if (threadIdx.x == 0) *p.ticket = 0;  // ready for the next launch on this stream
}

// Decision from combined running values (token-sharded verification): sums[b][0..2] as the verify
// kernel hands them out, added (l-infinity: maximised) over the shards by the caller.
template <int M>
__device__ __forceinline__ double error_from(const double* s, double eps) {
    const double v[3] = {s[0], s[1], s[2]};
    return Metric<M>::error(v, eps);
}

__global__ void __launch_bounds__(SPECA_MAX_BATCH) decide_kernel(int metric, const double* __restrict__ sums, int batch,
                                                                  DecideParams q, const uint8_t* __restrict__ mask,
                                                                  float* __restrict__ err, uint8_t* __restrict__ accept) {
    const int b = threadIdx.x;
    if (b >= batch || (mask != nullptr && mask[b] == 0)) return;
    const double* s = sums + b * 4;
    double e;
    switch (metric) {
        case SPECA_METRIC_L1: e = error_from<SPECA_METRIC_L1>(s, q.eps); break;
        case SPECA_METRIC_LINF: e = error_from<SPECA_METRIC_LINF>(s, q.eps); break;
        case SPECA_METRIC_COSINE: e = error_from<SPECA_METRIC_COSINE>(s, q.eps); break;
        default: e = error_from<SPECA_METRIC_L2>(s, q.eps); break;
    }
    err[b] = static_cast<float>(e);
    accept[b] = (e <= static_cast<double>(q.tau[b])) ? 1 : 0;
}

cudaError_t launch_decide(int metric, const double* sums, int batch, const DecideParams& q, const uint8_t* mask,
                          float* err, uint8_t* accept, cudaStream_t stream) {
    decide_kernel<<<1, SPECA_MAX_BATCH, 0, stream>>>(metric, sums, batch, q, mask, err, accept);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// select / activate: B <= 64 samples, one small CTA
// ------------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(32) select_kernel(const uint8_t* accept, int32_t k_max, int32_t group, int32_t batch,
                                                     int32_t* spec_count, uint8_t* active, int32_t* idx_out,
                                                     int32_t* n_out) {
    // in place: a lane reads its own samples' mask bytes before the ballots and writes them after
    select_in_warp(accept, k_max, group, batch, spec_count, active, active, idx_out, n_out);
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

template <int DT, bool UPDATE, int PATH>
static const void* stream_kernel_for(int v) {
    constexpr Shape s0 = shape_for(PATH, UPDATE, 0, DT), s1 = shape_for(PATH, UPDATE, 1, DT),
                    s2 = shape_for(PATH, UPDATE, 2, DT), s3 = shape_for(PATH, UPDATE, 3, DT),
                    s4 = shape_for(PATH, UPDATE, 4, DT);
    static_assert(shape_tile_bytes(s0) == shape_tile_bytes(s2) && shape_tile_bytes(s1) == shape_tile_bytes(s2) &&
                      shape_tile_bytes(s3) == shape_tile_bytes(s2) && shape_tile_bytes(s4) == shape_tile_bytes(s2),
                  "all orders of a path share one tile size (one tile table)");
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&stream_kernel<DT, 0, UPDATE, s0.w, s0.nt, s0.u, s0.chunks, s0.minb>);
        case 1: return reinterpret_cast<const void*>(&stream_kernel<DT, 1, UPDATE, s1.w, s1.nt, s1.u, s1.chunks, s1.minb>);
        case 2: return reinterpret_cast<const void*>(&stream_kernel<DT, 2, UPDATE, s2.w, s2.nt, s2.u, s2.chunks, s2.minb>);
        case 3: return reinterpret_cast<const void*>(&stream_kernel<DT, 3, UPDATE, s3.w, s3.nt, s3.u, s3.chunks, s3.minb>);
        default: return reinterpret_cast<const void*>(&stream_kernel<DT, 4, UPDATE, s4.w, s4.nt, s4.u, s4.chunks, s4.minb>);
    }
}

static const void* stream_kernel_for(int dtype, bool update, int path, int v) {
    if (path == SPECA_PATH_WIDE) {
        if (update)
            return dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, true, SPECA_PATH_WIDE>(v)
                                       : stream_kernel_for<SPECA_F32, true, SPECA_PATH_WIDE>(v);
        return dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, false, SPECA_PATH_WIDE>(v)
                                   : stream_kernel_for<SPECA_F32, false, SPECA_PATH_WIDE>(v);
    }
    if (update)
        return dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, true, SPECA_PATH_DIRECT>(v)
                                   : stream_kernel_for<SPECA_F32, true, SPECA_PATH_DIRECT>(v);
    return dtype == SPECA_BF16 ? stream_kernel_for<SPECA_BF16, false, SPECA_PATH_DIRECT>(v)
                               : stream_kernel_for<SPECA_F32, false, SPECA_PATH_DIRECT>(v);
}

template <int DT, int M>
static const void* verify_kernel_for(int v) {
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&verify_kernel<DT, 0, M>);
        case 1: return reinterpret_cast<const void*>(&verify_kernel<DT, 1, M>);
        case 2: return reinterpret_cast<const void*>(&verify_kernel<DT, 2, M>);
        case 3: return reinterpret_cast<const void*>(&verify_kernel<DT, 3, M>);
        default: return reinterpret_cast<const void*>(&verify_kernel<DT, 4, M>);
    }
}

template <int DT>
static const void* verify_kernel_for(int metric, int v) {
    switch (metric) {
        case SPECA_METRIC_L1: return verify_kernel_for<DT, SPECA_METRIC_L1>(v);
        case SPECA_METRIC_LINF: return verify_kernel_for<DT, SPECA_METRIC_LINF>(v);
        case SPECA_METRIC_COSINE: return verify_kernel_for<DT, SPECA_METRIC_COSINE>(v);
        default: return verify_kernel_for<DT, SPECA_METRIC_L2>(v);
    }
}

static int max_order(const int8_t* order) {
    int v = 0;
    for (int b = 0; b < SPECA_MAX_BATCH; ++b) v = order[b] > v ? order[b] : v;
    return v;
}

template <int DT, bool UPDATE>
static const void* bulk_kernel_for(int v) {
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&stream_bulk_kernel<DT, 0, UPDATE>);
        case 1: return reinterpret_cast<const void*>(&stream_bulk_kernel<DT, 1, UPDATE>);
        case 2: return reinterpret_cast<const void*>(&stream_bulk_kernel<DT, 2, UPDATE>);
        case 3: return reinterpret_cast<const void*>(&stream_bulk_kernel<DT, 3, UPDATE>);
        default: return reinterpret_cast<const void*>(&stream_bulk_kernel<DT, 4, UPDATE>);
    }
}

static const void* bulk_kernel_for(int dtype, bool update, int v) {
    if (update) return dtype == SPECA_BF16 ? bulk_kernel_for<SPECA_BF16, true>(v) : bulk_kernel_for<SPECA_F32, true>(v);
    return dtype == SPECA_BF16 ? bulk_kernel_for<SPECA_BF16, false>(v) : bulk_kernel_for<SPECA_F32, false>(v);
}

static int clamp_order(int v) { return v < 0 ? 0 : (v > SPECA_MAX_ORDER ? SPECA_MAX_ORDER : v); }

uint32_t stream_tile_bytes(int path, bool update) {
    if (path == SPECA_PATH_BULK) return kBulkTileBytes;
    return shape_tile_bytes(shape_for(path, update, 2, SPECA_BF16));  // the same for every order and dtype
}

int stream_ctas_per_sm(int path, bool update, int dtype, int order) {
    if (path == SPECA_PATH_BULK) {
        const void* fn = bulk_kernel_for(dtype, update, clamp_order(order));
        const int smem = static_cast<int>(bulk_smem_bytes(clamp_order(order)));
        int n = 0;
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, kBulkThreads, smem) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        return n;
    }
    return shape_for(path, update, order, dtype).minb;
}

static cudaError_t launch_stream(const StreamParams& p, int dtype, bool update, int path, int grid,
                                 cudaStream_t stream) {
    if (path == SPECA_PATH_BULK) {
        const int v = max_order(p.order);
        const void* fn = bulk_kernel_for(dtype, update, v);
        const size_t smem = bulk_smem_bytes(v);
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
        void* args[1] = {const_cast<StreamParams*>(&p)};
        return cudaLaunchKernel(fn, dim3(grid), dim3(kBulkThreads), args, smem, stream);
    }
    if (path != SPECA_PATH_DIRECT && path != SPECA_PATH_WIDE) return cudaErrorNotSupported;
    const int v = max_order(p.order);
    const void* fn = stream_kernel_for(dtype, update, path, v);
    void* args[1] = {const_cast<StreamParams*>(&p)};
    return cudaLaunchKernel(fn, dim3(grid), dim3(shape_for(path, update, v, dtype).nt), args, 0, stream);
}

cudaError_t launch_update(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream) {
    return launch_stream(p, dtype, true, path, grid, stream);
}

cudaError_t launch_forecast(const StreamParams& p, int dtype, int path, int grid, cudaStream_t stream) {
    return launch_stream(p, dtype, false, path, grid, stream);
}

// Launch shapes of the fused kernel per order (2v + 3 streams, v + 2 of them stores), 32 KB tiles like
// the update's so that the two share a tile table. Swept on a B200 on 20 FLUX-sized entries (bf16 / fp32,
// GB/s over the 2v + 3 words): unlike the plain update this mix wants two vectors per thread and one
// 256-thread CTA per SM (order 2: 6310 / 6270 against 4680 / 6340 with the update's 128 x 1 x 3 CTAs/SM
// shape, 5010 / 6010 with 256 x 1 x 2); only order 0 (one load, two stores) prefers one vector
// (5720 / 5930 against 5440 / 5600).
#ifndef SPECA_SHAPES_FUSED
#define SPECA_SHAPES_FUSED \
    {32, 256, 1, 4, 2}, {32, 256, 2, 2, 1}, {32, 256, 2, 2, 1}, {32, 256, 2, 2, 1}, { 32, 256, 2, 2, 1 }
#endif
// Raw-feature caches: order + 1 loads and two stores per element. Measured on 20 FLUX-shaped entries
// (bf16 / fp32, GB/s over order + 3 words): orders 0 and 1 want many small CTAs (6030 / 6260 and 6330 /
// 6250 against 5200 / 5450 and 5640 / 5930 with the table layout's shape), order 2 one vector per thread
// (6610 / 6550 against 6230 / 6560), orders 3 and 4 the table layout's shape (6600-6990).
#ifndef SPECA_SHAPES_FUSED_HISTORY
#define SPECA_SHAPES_FUSED_HISTORY \
    {32, 128, 2, 4, 3}, {32, 128, 2, 4, 3}, {32, 512, 1, 2, 1}, {32, 256, 2, 2, 1}, { 32, 256, 2, 2, 1 }
#endif
// One exception by storage type, measured like the others: order 1 on bf16 tables runs at 6300 GB/s with
// one vector per thread against 5990 with two, while fp32 drops to 4520 with one (6320 with two).
#ifndef SPECA_SHAPE_FUSED1_BF16
#define SPECA_SHAPE_FUSED1_BF16 { 32, 256, 1, 4, 2 }
#endif
// With three or more targets per pass the stores dominate whatever the order and the layout, and the
// two-vector shape wins everywhere it was measured (bf16, 20 FLUX-shaped entries, K = 3 / 5 / 8: raw features,
// order 2, 627 / 795 / 1105 us against 648 / 865 / 1179 with the one-target shape; order 1 with K = 4, 623
// against 683 us, and 754 against 786 us on tables).
#ifndef SPECA_SHAPE_FUSED_MANY
#define SPECA_SHAPE_FUSED_MANY { 32, 256, 2, 2, 1 }
#endif
constexpr int kFusedManyTargets = 3;
__host__ __device__ constexpr Shape fused_shape(int v, bool hist, int dtype, bool many) {
    constexpr Shape fs[SPECA_MAX_ORDER + 1] = {SPECA_SHAPES_FUSED};
    constexpr Shape fh[SPECA_MAX_ORDER + 1] = {SPECA_SHAPES_FUSED_HISTORY};
    const int i = v < 0 ? 0 : (v > SPECA_MAX_ORDER ? SPECA_MAX_ORDER : v);
    if (many && i >= 1) return Shape SPECA_SHAPE_FUSED_MANY;
    if (!hist && i == 1 && dtype == SPECA_BF16) return Shape SPECA_SHAPE_FUSED1_BF16;
    return hist ? fh[i] : fs[i];
}
constexpr bool fused_shapes_fit_the_update_tiles() {
    for (int v = 0; v <= SPECA_MAX_ORDER; ++v)
        for (int h = 0; h < 4; ++h)
            for (int dt = 0; dt < 2; ++dt)
                if (shape_tile_bytes(fused_shape(v, (h & 1) != 0, dt, (h & 2) != 0)) !=
                    shape_tile_bytes(shape_for(SPECA_PATH_WIDE, true, v, dt)))
                    return false;
    return true;
}
static_assert(fused_shapes_fit_the_update_tiles(), "the fused kernel walks the update's tile table");

template <int DT, bool HIST, bool MANY>
static const void* fused_kernel_for(int v) {
    constexpr Shape s0 = fused_shape(0, HIST, DT, MANY), s1 = fused_shape(1, HIST, DT, MANY), s2 = fused_shape(2, HIST, DT, MANY),
                    s3 = fused_shape(3, HIST, DT, MANY), s4 = fused_shape(4, HIST, DT, MANY);
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&update_forecast_kernel<DT, 0, s0.w, s0.nt, s0.u, s0.chunks, s0.minb, HIST>);
        case 1: return reinterpret_cast<const void*>(&update_forecast_kernel<DT, 1, s1.w, s1.nt, s1.u, s1.chunks, s1.minb, HIST>);
        case 2: return reinterpret_cast<const void*>(&update_forecast_kernel<DT, 2, s2.w, s2.nt, s2.u, s2.chunks, s2.minb, HIST>);
        case 3: return reinterpret_cast<const void*>(&update_forecast_kernel<DT, 3, s3.w, s3.nt, s3.u, s3.chunks, s3.minb, HIST>);
        default: return reinterpret_cast<const void*>(&update_forecast_kernel<DT, 4, s4.w, s4.nt, s4.u, s4.chunks, s4.minb, HIST>);
    }
}
template <int DT, bool HIST>
static const void* fused_kernel_for(int v, bool many) {
    return many ? fused_kernel_for<DT, HIST, true>(v) : fused_kernel_for<DT, HIST, false>(v);
}

int fused_ctas_per_sm(int order, bool raw_features, int dtype, int n_targets) {
    return fused_shape(order, raw_features, dtype, n_targets >= kFusedManyTargets).minb;
}

// The kernel is compiled for the highest order any sample has in either half of the launch.
cudaError_t launch_update_forecast(const FusedParams& p, int dtype, int grid, cudaStream_t stream) {
    int v = max_order(p.up.order);
    const int vf = max_order(p.fc_order);
    v = vf > v ? vf : v;
    const bool hist = p.up.weighted != 0, many = p.n_targets >= kFusedManyTargets;
    const void* fn;
    if (hist)
        fn = dtype == SPECA_BF16 ? fused_kernel_for<SPECA_BF16, true>(v, many) : fused_kernel_for<SPECA_F32, true>(v, many);
    else
        fn = dtype == SPECA_BF16 ? fused_kernel_for<SPECA_BF16, false>(v, many) : fused_kernel_for<SPECA_F32, false>(v, many);
    void* args[1] = {const_cast<FusedParams*>(&p)};
    return cudaLaunchKernel(fn, dim3(grid), dim3(fused_shape(v, hist, dtype, many).nt), args, 0, stream);
}

template <int DT, int KCLASS>
static const void* multi_kernel_for(int v) {
    constexpr Shape s = multi_shape(KCLASS);
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&forecast_multi_kernel<DT, 0, s.w, s.nt, s.u, s.chunks, s.minb>);
        case 1: return reinterpret_cast<const void*>(&forecast_multi_kernel<DT, 1, s.w, s.nt, s.u, s.chunks, s.minb>);
        case 2: return reinterpret_cast<const void*>(&forecast_multi_kernel<DT, 2, s.w, s.nt, s.u, s.chunks, s.minb>);
        case 3: return reinterpret_cast<const void*>(&forecast_multi_kernel<DT, 3, s.w, s.nt, s.u, s.chunks, s.minb>);
        default: return reinterpret_cast<const void*>(&forecast_multi_kernel<DT, 4, s.w, s.nt, s.u, s.chunks, s.minb>);
    }
}

uint32_t multi_tile_bytes() { return shape_tile_bytes(multi_shape(1)); }
int multi_ctas_per_sm(int n_targets) { return multi_shape(n_targets).minb; }

cudaError_t launch_forecast_multi(const MultiParams& p, int dtype, int batch, int grid, cudaStream_t stream) {
    const int v = max_order(p.order);
    const void* fn;
    if (p.n_targets <= 5)
        fn = dtype == SPECA_BF16 ? multi_kernel_for<SPECA_BF16, 1>(v) : multi_kernel_for<SPECA_F32, 1>(v);
    else
        fn = dtype == SPECA_BF16 ? multi_kernel_for<SPECA_BF16, 8>(v) : multi_kernel_for<SPECA_F32, 8>(v);
    void* args[2] = {const_cast<MultiParams*>(&p), &batch};
    return cudaLaunchKernel(fn, dim3(grid), dim3(multi_shape(p.n_targets).nt), args, 0, stream);
}

template <int DT>
static const void* sum_kernel_for(int v) {
    switch (v) {
        case 0: return reinterpret_cast<const void*>(&forecast_sum_kernel<DT, 0>);
        case 1: return reinterpret_cast<const void*>(&forecast_sum_kernel<DT, 1>);
        case 2: return reinterpret_cast<const void*>(&forecast_sum_kernel<DT, 2>);
        case 3: return reinterpret_cast<const void*>(&forecast_sum_kernel<DT, 3>);
        default: return reinterpret_cast<const void*>(&forecast_sum_kernel<DT, 4>);
    }
}

uint32_t sum_tile_bytes() { return kSumTileBytes; }
int sum_ctas_per_sm() { return kSumMinBlocks; }

cudaError_t launch_forecast_sum(const SumParams& p, int dtype, int grid, cudaStream_t stream) {
    const int v = max_order(p.order);
    const void* fn = dtype == SPECA_BF16 ? sum_kernel_for<SPECA_BF16>(v) : sum_kernel_for<SPECA_F32>(v);
    void* args[1] = {const_cast<SumParams*>(&p)};
    return cudaLaunchKernel(fn, dim3(grid), dim3(kSumThreads), args, 0, stream);
}

static void verify_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int grid, int cluster,
                          cudaStream_t stream) {
    *cfg = {};
    cfg->gridDim = dim3(grid);
    cfg->blockDim = dim3(kThreads);
    cfg->dynamicSmemBytes = 0;
    cfg->stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
}

cudaError_t launch_verify(const VerifyParams& p, int dtype, int grid, int cluster, cudaStream_t stream) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    const int v = max_order(p.order);
    verify_config(&cfg, attr, grid, cluster, stream);
    const void* fn = dtype == SPECA_BF16 ? verify_kernel_for<SPECA_BF16>(p.metric, v)
                                         : verify_kernel_for<SPECA_F32>(p.metric, v);
    void* args[1] = {const_cast<VerifyParams*>(&p)};
    return cudaLaunchKernelExC(&cfg, fn, args);
}

// Clusters of `cluster` CTAs of the verify kernel that can be resident at once on the current
// device. A cluster needs all its CTAs in one GPC, so this is less than SMs x CTAs/SM / cluster
// when GPC sizes are not multiples of the cluster size; a grid sized above it would run its last
// clusters as a second wave.
int max_resident_verify_clusters(int dtype, int order, int cluster) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    verify_config(&cfg, attr, cluster, cluster, nullptr);
    const void* fn = dtype == SPECA_BF16 ? verify_kernel_for<SPECA_BF16>(SPECA_METRIC_L2, order)
                                         : verify_kernel_for<SPECA_F32>(SPECA_METRIC_L2, order);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        n = 1;
    }
    return n;
}

cudaError_t launch_select(const uint8_t* accept, int32_t k_max, int32_t group, int32_t batch, int32_t* spec_count,
                          uint8_t* active, int32_t* idx, int32_t* n_active, cudaStream_t stream) {
    select_kernel<<<1, 32, 0, stream>>>(accept, k_max, group, batch, spec_count, active, idx, n_active);
    return cudaGetLastError();
}

cudaError_t launch_activate(uint64_t mask_bits, int32_t batch, int32_t* spec_count, uint8_t* active,
                            cudaStream_t stream) {
    activate_kernel<<<1, SPECA_MAX_BATCH, 0, stream>>>(mask_bits, batch, spec_count, active);
    return cudaGetLastError();
}

}  // namespace speca
