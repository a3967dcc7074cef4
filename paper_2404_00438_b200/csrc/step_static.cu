// dlion_step_static: one two-stage optimizer step that allocates nothing.
//
// Some callers may not allocate device memory at the point where they step the
// optimizer: code that runs while a caching allocator has handed every byte of
// the device to someone else, a step issued from a callback or a real-time loop
// where cudaMalloc's implicit device synchronisation is not acceptable, or a
// plug-in that is only allowed to use the buffers it was given.  The regular
// path needs two pieces of device memory besides the caller's tensors: the
// context's tile table (allocated by dlion_init) and the 1-bit wire buffer
// between the two kernels.  Here the wire buffer is a fixed array that is part
// of the library image and the parameters are a flat vector, which needs no
// table, so the call needs neither dlion_init nor a caller-supplied wire buffer.
//
// The price: the array has a fixed size, every GPU on which the library's
// device code gets loaded holds it until the process exits, and all calls on a
// device share it.  The FIRST call on a device is a set-up call: it makes the
// CUDA runtime load this library's device code (which is when the array is
// reserved) and looks up the array's address.  Make it at start-up, before
// another allocator takes the remaining memory and before any stream capture;
// only the calls after it allocate nothing.
#include <mutex>

#include "dlion_common.cuh"
#include "host_checks.h"

namespace {

constexpr unsigned long long kMaxCoordWorkers = DLION_STATIC_MAX_COORD_WORKERS;   // N * d_pad limit
constexpr size_t kWireWords = kMaxCoordWorkers / 32;              // 16 MiB of sign bits

// Scratch shared by every dlion_step_static call on this device.  In host code
// this name is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) uint32_t g_static_scratch[kWireWords];

constexpr int kMaxDevices = 64;
struct PerDevice {
    uint32_t* scratch = nullptr;     // device address of g_static_scratch on that device
    int sm_count = 0;
};
PerDevice g_dev[kMaxDevices];
std::mutex g_dev_mutex;

// First call on a device: resolve the array's device address (with that device
// current) and read the SM count.  Neither call allocates.
cudaError_t setup_device(int dev, PerDevice* out) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (g_dev[dev].scratch == nullptr) {
        uint32_t* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch);
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_dev[dev].sm_count = sms;
        g_dev[dev].scratch = ptr;
    }
    *out = g_dev[dev];
    return cudaSuccess;
}

using dlion::aligned16;
using dlion::nonneg_finite;
using dlion::unit_interval;

}  // namespace

extern "C" dlion_status dlion_step_static(uint64_t d, uint32_t n_workers, float beta1, float beta2,
                                          float lr, float weight_decay, dlion_mode mode,
                                          dlion_gdtype gdtype, const void* grads, float* m, float* x,
                                          void* cuda_stream) {
    if (d == 0 || grads == nullptr || m == nullptr || x == nullptr) return DLION_EINVAL;
    if (n_workers == 0 || n_workers > DLION_MAX_WORKERS) return DLION_EINVAL;
    if (!unit_interval(beta1) || !unit_interval(beta2)) return DLION_EINVAL;
    if (!nonneg_finite(lr) || !nonneg_finite(weight_decay)) return DLION_EINVAL;
    if (mode != DLION_MAJORITY && mode != DLION_AVERAGE && mode != DLION_MAJORITY_TERNARY) return DLION_EINVAL;
    if (gdtype != DLION_GRAD_F32 && gdtype != DLION_GRAD_BF16) return DLION_EINVAL;
    if (d > kMaxCoordWorkers) return DLION_EINVAL;
    const unsigned long long d_pad = (d + DLION_ALIGN - 1) / DLION_ALIGN * DLION_ALIGN;
    if (d_pad * n_workers > kMaxCoordWorkers) return DLION_EINVAL;          // beyond the fixed scratch
    if (!aligned16(grads) || !aligned16(m) || !aligned16(x)) return DLION_EALIGN;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DLION_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return DLION_ESTATE;
    PerDevice pd;
    if (setup_device(dev, &pd) != cudaSuccess) return DLION_ECUDA;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    uint32_t* wire = pd.scratch;
    const unsigned long long ntiles = (d + dlion::kTile - 1) / dlion::kTile;

    // The wire buffer keeps the previous call's bits: the worker-side kernel
    // overwrites every word that holds a parameter and the server-side kernel reads
    // no other word, so nothing has to be cleared.
    dlion::WorkerParams wp{};
    wp.g = grads;
    wp.m = m;
    wp.packed = wire;
    wp.tiles = nullptr;
    wp.flat_d = d;
    wp.n_workers = n_workers;
    wp.ntiles = ntiles;
    wp.d_pad = d_pad;
    wp.k.b1 = beta1;
    wp.k.om1 = 1.0f - beta1;
    wp.k.b2 = beta2;
    wp.k.om2 = 1.0f - beta2;
    wp.betas = nullptr;
    wp.worker0 = 0;
    wp.m_bf16 = 0;
    if (dlion::launch_worker_step(wp, gdtype == DLION_GRAD_BF16, pd.sm_count, s) != cudaSuccess) {
        return DLION_ECUDA;
    }

    dlion::AggParams ap{};
    ap.packed = wire;
    ap.x = x;
    ap.delta_bits = nullptr;
    ap.count = nullptr;
    ap.count16 = nullptr;
    ap.tiles = nullptr;
    ap.flat_d = d;
    ap.n_workers = n_workers;
    ap.ntiles = ntiles;
    ap.w_stride = d_pad / 32;
    ap.lr = lr;
    ap.wd = weight_decay;
    ap.ternary = mode == DLION_MAJORITY_TERNARY ? 1 : 0;
    ap.average = (mode == DLION_AVERAGE || ap.ternary) ? 1 : 0;
    if (dlion::launch_aggregate_apply(ap, pd.sm_count, s) != cudaSuccess) return DLION_ECUDA;
    return DLION_OK;
}
