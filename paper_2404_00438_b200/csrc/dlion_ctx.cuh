// The host-side context behind the opaque dlion_ctx of include/dlion.h.
#pragma once

#include <vector>

#include "dlion_common.cuh"

struct dlion_ctx {
    std::vector<dlion_segment> segs;
    dlion::TileRow* tiles_dev = nullptr;     // one row per tile
    uint32_t nseg = 0;
    unsigned long long ntiles = 0;
    uint64_t d = 0;            // parameters
    uint64_t d_pad = 0;
    uint32_t n_workers = 0;
    float beta1 = 0, beta2 = 0, lr = 0, wd = 0;
    dlion_mode mode = DLION_MAJORITY;
    dlion_gdtype gdtype = DLION_GRAD_F32;
    dlion_sdtype sdtype = DLION_STATE_F32;
    std::vector<dlion::Betas> betas;         // per-worker rows (empty until one is set)
    dlion::Betas* betas_dev = nullptr;
    // per-tensor tables (dlion_bind_tensors): one device block, g rows first,
    // then m rows ([n_workers][nseg] each), then the x row ([nseg]); null until bound
    long long* tables_dev = nullptr;         // byte offsets from tables_dev itself (see WorkerParams)
    std::vector<long long> tables_host;
    bool bound_g = false, bound_m = false, bound_x = false;
    // scatter mode (dlion_bind_scatter): byte offsets of the per-slice receive buffers from scatter_dev itself
    long long* scatter_dev = nullptr;
    uint32_t scatter_n = 0, scatter_slot = 0;
    uint64_t scatter_slice_words = 0;
    int device = -1;
    int sm_count = 0;
    uint64_t launches = 0;
    cudaStream_t copy_stream = nullptr;      // host-gradient pipeline (created on first use)
    cudaEvent_t copied[2] = {nullptr, nullptr};
    cudaEvent_t consumed[2] = {nullptr, nullptr};
    cudaEvent_t entry = nullptr;
};

namespace dlion {

// Launch parameters with everything filled in from the context except the caller's
// pointers (shared by the arena entry points and the per-tensor ones).
WorkerParams worker_params(const dlion_ctx* c, int worker);
AggParams agg_params(const dlion_ctx* c);
WireParams wire_params(const dlion_ctx* c, uint64_t slice_words);
dlion_status device_ok(const dlion_ctx* c);     // DLION_ESTATE unless the context's device is current
// The three-valued tie rule's message, Delta + 1 in {0, 1, 2} as two planes, is exactly an
// Averaging message of a 2-worker problem ((2c - 2) / 2 = c - 1): the apply kernels decode
// it as such.
inline void decode_ternary_as_two_workers(WireParams& p) {
    if (p.ternary) {
        p.average = 1;
        p.n_workers = 2;
        p.kplanes = 2;
    }
}

}  // namespace dlion
