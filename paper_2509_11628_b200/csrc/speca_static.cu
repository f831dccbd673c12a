// speca_verify_pred_static: Eq. 4 and the accept rule on a forecast the caller already holds, for
// callers that have no device memory to give the library and cannot allocate any.
//
// The verification kernel needs a little global scratch for its cross-CTA reduction (one pair of
// partial sums per (cluster, sample), an arrival counter) and a descriptor per sample. A cache
// handle keeps those in the caller's arena. Here they live in one file-scope __device__ array that
// is part of the loaded library image on every GPU, so the call path contains no cudaMalloc,
// cudaFree or other allocating routine.
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <mutex>

#include "speca_internal.h"

namespace speca {
namespace {

constexpr int kStaticMaxClusters = SPECA_STATIC_MAX_CLUSTERS;
constexpr size_t kSegBytes = sizeof(SegDesc) * SPECA_MAX_BATCH;                                   // 2 KB
constexpr size_t kPartialBytes = sizeof(float) * 2 * SPECA_MAX_BATCH * size_t(kStaticMaxClusters);  // 64 KB
constexpr size_t kTicketBytes = 256;
constexpr size_t kScratchBytes = kSegBytes + kPartialBytes + kTicketBytes;
static_assert(kScratchBytes == SPECA_STATIC_SCRATCH_BYTES, "header and library disagree on the scratch size");

// The scratch itself. In host code this name is only a handle for the runtime's symbol table; the
// device address comes from cudaGetSymbolAddress (scratch_on_device below).
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices];  // per device, filled on first use

// Device address of g_static_scratch on `device`, which must be the current device.
cudaError_t scratch_on_device(int device, unsigned char** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[device] == nullptr) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

// Sample b of a dense [B, n_elems] tensor is one "table" with a single plane: its row.
// Also clears the arrival counter, which must be zero when the verification kernel starts.
__global__ void __launch_bounds__(SPECA_MAX_BATCH) dense_rows_kernel(SegDesc* segs, uint32_t* ticket, uint32_t n_elems,
                                                                      uint32_t elem_bytes, int32_t batch) {
    const int b = threadIdx.x;
    if (b < batch) {
        SegDesc s;
        s.plane0_off = static_cast<uint64_t>(b) * n_elems * elem_bytes;
        s.plane_stride = 0;
        s.io_off = s.plane0_off;
        s.n_elems = n_elems;
        s.entry = 0;
        s.sample = static_cast<uint16_t>(b);
        segs[b] = s;
    }
    if (b == 0) *ticket = 0;
}

}  // namespace
}  // namespace speca

using namespace speca;

extern "C" speca_status_t speca_verify_pred_static(const void* pred, const void* fresh, int64_t n_elems, int32_t batch,
                                                   int32_t dtype, const float* tau, float eps,
                                                   const uint8_t* dev_active_mask, float* dev_err, uint8_t* dev_accept,
                                                   int32_t device, void* stream) {
    if (pred == nullptr || fresh == nullptr || tau == nullptr || dev_err == nullptr || dev_accept == nullptr)
        return SPECA_ERR_INVALID_ARG;
    if (dtype != SPECA_F32 && dtype != SPECA_BF16) return SPECA_ERR_INVALID_ARG;
    if (batch < 1 || batch > SPECA_STATIC_MAX_BATCH) return SPECA_ERR_SHAPE;
    if (n_elems < 1 || n_elems > SPECA_STATIC_MAX_ELEMS) return SPECA_ERR_SHAPE;
    if (device < 0 || device >= kMaxDevices) return SPECA_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (std::isnan(tau[b])) return SPECA_ERR_INVALID_ARG;
    const size_t esz = dtype == SPECA_BF16 ? 2 : 4;
    // every row of both tensors must start on a 16-byte boundary: the kernel reads 16-byte vectors
    if (reinterpret_cast<uintptr_t>(pred) % 16 != 0 || reinterpret_cast<uintptr_t>(fresh) % 16 != 0 ||
        reinterpret_cast<uintptr_t>(dev_err) % sizeof(float) != 0)
        return SPECA_ERR_ALIGNMENT;
    if (batch > 1 && (static_cast<uint64_t>(n_elems) * esz) % 16 != 0) return SPECA_ERR_ALIGNMENT;

    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) return SPECA_ERR_CUDA;
    if (device >= n_dev) return SPECA_ERR_INVALID_ARG;
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (major != 10) return SPECA_ERR_UNSUPPORTED;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SPECA_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return SPECA_ERR_CUDA;

    speca_status_t st = SPECA_OK;
    do {
        if (cudaPeekAtLastError() != cudaSuccess) {
            st = SPECA_ERR_CUDA;
            break;
        }
        unsigned char* scratch = nullptr;
        if (scratch_on_device(device, &scratch) != cudaSuccess) {
            st = SPECA_ERR_CUDA;
            break;
        }
        SegDesc* segs = reinterpret_cast<SegDesc*>(scratch);
        float* partials = reinterpret_cast<float*>(scratch + kSegBytes);
        uint32_t* ticket = reinterpret_cast<uint32_t*>(scratch + kSegBytes + kPartialBytes);
        cudaStream_t s = static_cast<cudaStream_t>(stream);

        dense_rows_kernel<<<1, SPECA_MAX_BATCH, 0, s>>>(segs, ticket, static_cast<uint32_t>(n_elems),
                                                         static_cast<uint32_t>(esz), batch);
        if (cudaGetLastError() != cudaSuccess) {
            st = SPECA_ERR_CUDA;
            break;
        }

        VerifyParams p;
        std::memset(&p, 0, sizeof p);
        for (int b = 0; b < SPECA_MAX_BATCH; ++b) p.order[b] = -1;
        for (int b = 0; b < batch; ++b) {
            p.order[b] = 0;  // the "table" is the forecast itself: nothing to extrapolate
            p.tau[b] = tau[b];
        }
        const int cluster = 4;
        const uint32_t te = verify_tile_elems(dtype, 0);
        p.segs = segs;
        p.arena = const_cast<char*>(static_cast<const char*>(pred));
        p.dev_mask = dev_active_mask;
        p.fresh = static_cast<const char*>(fresh);
        p.out_pred = nullptr;
        p.err = dev_err;
        p.accept = dev_accept;
        p.partials = partials;
        p.ticket = ticket;
        p.n_elems = static_cast<uint32_t>(n_elems);
        p.tiles_per_sample = (p.n_elems + te - 1) / te;
        p.units_per_sample = (p.tiles_per_sample + cluster - 1) / cluster;
        p.batch = batch;
        p.eps = eps > 0.f ? static_cast<double>(eps) : 1e-8;
        int n_clusters = max_resident_verify_clusters(dtype, 0, cluster);
        if (n_clusters > kStaticMaxClusters) n_clusters = kStaticMaxClusters;
        int grid = n_clusters * cluster;
        const uint64_t units = static_cast<uint64_t>(p.units_per_sample) * batch;
        if (units * cluster < static_cast<uint64_t>(grid)) grid = static_cast<int>(units) * cluster;
        if (launch_verify(p, dtype, grid, cluster, s) != cudaSuccess) st = SPECA_ERR_CUDA;
    } while (false);

    if (prev != device) cudaSetDevice(prev);
    return st;
}
