// speca_verify_pred_static: Eq. 4 and the accept rule on a forecast the caller already holds, for
// callers that have no device memory to give the library and cannot allocate any.
//
// The verification kernel needs a little global scratch for its cross-CTA reduction (one pair of
// partial sums per (cluster, sample), an arrival counter). A cache handle keeps those in
// the caller's arena. Here they live in one file-scope __device__ array that is part of the loaded
// library image on every GPU, so the call path contains no cudaMalloc, cudaFree or other allocating
// routine.
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <mutex>

#include "speca_internal.h"

namespace speca {
namespace {

constexpr int kStaticMaxClusters = SPECA_STATIC_MAX_CLUSTERS;
constexpr size_t kPartialBytes = sizeof(float) * 2 * SPECA_MAX_BATCH * size_t(kStaticMaxClusters);  // 64 KB
constexpr size_t kCounterBytes = 512;  // the arrival counter, padded
constexpr size_t kScratchBytes = kPartialBytes + kCounterBytes;
static_assert(kVerifyTickets * sizeof(uint32_t) <= kCounterBytes, "the counters fit their slot");
static_assert(kScratchBytes == SPECA_STATIC_SCRATCH_BYTES, "header and library disagree on the scratch size");

// The scratch itself. In host code this name is only a handle for the runtime's symbol table; the
// device address comes from cudaGetSymbolAddress (scratch_on_device below).
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
constexpr int kCluster = SPECA_VERIFY_CLUSTER;
std::mutex g_mu;
// per device, filled on the first call there: the scratch array's device address, and how many
// clusters of the verification kernel are resident at once (per storage type)
unsigned char* g_scratch_addr[kMaxDevices];
int g_resident_clusters[kMaxDevices][2];

// Device address of g_static_scratch on `device` and the resident cluster count for `dtype`; `device`
// must be the current device. Both are looked up once per device (and storage type) and remembered.
cudaError_t device_setup(int device, int dtype, unsigned char** scratch, int* n_clusters) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[device] == nullptr) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = static_cast<unsigned char*>(p);
    }
    const int k = dtype == SPECA_BF16 ? 1 : 0;
    if (g_resident_clusters[device][k] == 0) {
        int n = max_resident_verify_clusters(dtype, 0, kCluster);
        g_resident_clusters[device][k] = n > kStaticMaxClusters ? kStaticMaxClusters : n;
    }
    *scratch = g_scratch_addr[device];
    *n_clusters = g_resident_clusters[device][k];
    return cudaSuccess;
}

// The arrival counter must be zero when the verification kernel starts. The kernel leaves it at
// zero itself; this clears whatever an interrupted earlier call may have left.
__global__ void __launch_bounds__(32) clear_counters_kernel(uint32_t* counters) {
    if (threadIdx.x < kVerifyTickets) counters[threadIdx.x] = 0;
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
        if (cudaGetLastError() != cudaSuccess) {  // an earlier error on this thread: reported once, not kept
            st = SPECA_ERR_CUDA;
            break;
        }
        unsigned char* scratch = nullptr;
        int n_clusters = 0;
        if (device_setup(device, dtype, &scratch, &n_clusters) != cudaSuccess) {
            (void)cudaGetLastError();  // a failed lookup is not left behind for later calls to trip over
            st = SPECA_ERR_CUDA;
            break;
        }
        float* partials = reinterpret_cast<float*>(scratch);
        uint32_t* counters = reinterpret_cast<uint32_t*>(scratch + kPartialBytes);
        cudaStream_t s = static_cast<cudaStream_t>(stream);

        clear_counters_kernel<<<1, 32, 0, s>>>(counters);
        if (cudaGetLastError() != cudaSuccess) {  // also clears it
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
        const uint32_t te = verify_tile_elems(dtype, 0);
        // sample b of the dense [B, n_elems] forecast is a one-plane table: its row
        p.plane0_off = 0;
        p.sample_pitch = static_cast<uint64_t>(n_elems) * esz;
        p.plane_stride = 0;
        p.io_pitch = p.sample_pitch;
        p.arena = const_cast<char*>(static_cast<const char*>(pred));
        p.dev_mask = dev_active_mask;
        p.fresh = static_cast<const char*>(fresh);
        p.out_pred = nullptr;
        p.err = dev_err;
        p.accept = dev_accept;
        p.partials = partials;
        p.ticket = counters;
        p.n_elems = static_cast<uint32_t>(n_elems);
        p.tiles_per_sample = (p.n_elems + te - 1) / te;
        p.units_per_sample = (p.tiles_per_sample + kCluster - 1) / kCluster;
        p.batch = batch;
        p.eps = eps > 0.f ? static_cast<double>(eps) : 1e-8;
        int grid = n_clusters * kCluster;
        const uint64_t units = static_cast<uint64_t>(p.units_per_sample) * batch;
        if (units * kCluster < static_cast<uint64_t>(grid)) grid = static_cast<int>(units) * kCluster;
        if (launch_verify(p, dtype, grid, kCluster, s) != cudaSuccess) {
            (void)cudaGetLastError();
            st = SPECA_ERR_CUDA;
        }
    } while (false);

    if (prev != device) cudaSetDevice(prev);
    return st;
}
