// C ABI of the library (include/dlion.h): argument checks, the context, and the
// launches.  Everything that touches parameters runs in the kernels; this file
// only validates, fills launch parameters and enqueues.
#include <cmath>
#include <cstdlib>
#include <new>
#include <vector>

#include "dlion_ctx.cuh"
#include "host_checks.h"

namespace {

using dlion::aligned;
using dlion::nonneg_finite;
using dlion::unit_interval;

dlion::Betas common_betas(const dlion_ctx* c) {
    dlion::Betas k;
    k.b1 = c->beta1;
    k.om1 = 1.0f - c->beta1;        // formed in binary32, as the contract says
    k.b2 = c->beta2;
    k.om2 = 1.0f - c->beta2;
    return k;
}

}  // namespace

namespace dlion {

dlion_status device_ok(const dlion_ctx* c) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DLION_ECUDA;
    return dev == c->device ? DLION_OK : DLION_ESTATE;
}

WorkerParams worker_params(const dlion_ctx* ctx, int worker) {
    WorkerParams p{};
    p.nseg = ctx->nseg;
    p.tiles = ctx->tiles_dev;
    p.flat_d = 0;
    p.n_workers = worker < 0 ? ctx->n_workers : 1u;
    p.ntiles = ctx->ntiles;
    p.d_pad = ctx->d_pad;
    p.k = common_betas(ctx);
    p.betas = ctx->betas_dev;
    p.worker0 = worker < 0 ? 0u : static_cast<uint32_t>(worker);
    p.m_bf16 = ctx->sdtype == DLION_STATE_BF16 ? 1 : 0;
    return p;
}

AggParams agg_params(const dlion_ctx* ctx) {
    AggParams p{};
    p.tiles = ctx->tiles_dev;
    p.flat_d = 0;
    p.n_workers = ctx->n_workers;
    p.ntiles = ctx->ntiles;
    p.w_stride = ctx->d_pad / 32;
    p.lr = ctx->lr;
    p.wd = ctx->wd;
    // the three-valued tie rule runs on the Averaging kernels with a table of signs
    p.ternary = ctx->mode == DLION_MAJORITY_TERNARY ? 1 : 0;
    p.average = (ctx->mode == DLION_AVERAGE || p.ternary) ? 1 : 0;
    return p;
}

WireParams wire_params(const dlion_ctx* ctx, uint64_t slice_words) {
    WireParams p{};
    p.tiles = ctx->tiles_dev;
    p.flat_d = 0;
    p.n_workers = ctx->n_workers;
    p.ntiles = ctx->ntiles;
    p.w_stride = ctx->d_pad / 32;
    p.plane_stride = slice_words != 0 ? slice_words : ctx->d_pad / 32;
    p.slice_words = slice_words;
    p.kplanes = dlion_delta_planes(ctx);
    p.lr = ctx->lr;
    p.wd = ctx->wd;
    p.average = ctx->mode == DLION_AVERAGE ? 1 : 0;
    p.ternary = ctx->mode == DLION_MAJORITY_TERNARY ? 1 : 0;
    return p;
}

}  // namespace dlion

using dlion::device_ok;

extern "C" {

dlion_status dlion_check_layout(const dlion_segment* segs, uint32_t nseg, uint64_t d_pad) {
    if (segs == nullptr || nseg == 0 || d_pad == 0) return DLION_EINVAL;
    if (d_pad % DLION_ALIGN != 0) return DLION_EALIGN;
    uint64_t prev_end = 0;
    for (uint32_t s = 0; s < nseg; ++s) {
        if (segs[s].elem_offset % DLION_ALIGN != 0) return DLION_EALIGN;
        if (segs[s].elem_offset < prev_end) return DLION_EINVAL;            // overlap or not ascending
        if (segs[s].numel > d_pad || segs[s].elem_offset > d_pad - segs[s].numel) return DLION_EINVAL;
        prev_end = segs[s].elem_offset + segs[s].numel;
    }
    return DLION_OK;
}

dlion_status dlion_init(dlion_ctx** out, const dlion_segment* segs, uint32_t nseg, uint64_t d_pad,
                        uint32_t n_workers, float beta1, float beta2, float lr, float weight_decay,
                        dlion_mode mode, dlion_gdtype gdtype) {
    if (out == nullptr) return DLION_EINVAL;
    const dlion_status lay = dlion_check_layout(segs, nseg, d_pad);
    if (lay != DLION_OK) return lay;
    if (n_workers == 0 || n_workers > DLION_MAX_WORKERS) return DLION_EINVAL;
    if (!unit_interval(beta1) || !unit_interval(beta2)) return DLION_EINVAL;
    if (!nonneg_finite(lr) || !nonneg_finite(weight_decay)) return DLION_EINVAL;
    if (mode != DLION_MAJORITY && mode != DLION_AVERAGE && mode != DLION_MAJORITY_TERNARY) return DLION_EINVAL;
    if (gdtype != DLION_GRAD_F32 && gdtype != DLION_GRAD_BF16) return DLION_EINVAL;

    dlion_ctx* c = new (std::nothrow) dlion_ctx;
    if (c == nullptr) return DLION_ENOMEM;
    try {
        c->segs.assign(segs, segs + nseg);
    } catch (...) {
        delete c;
        return DLION_ENOMEM;
    }
    unsigned long long tiles = 0;
    for (uint32_t s = 0; s < nseg; ++s) {
        tiles += (segs[s].numel + dlion::kTile - 1) / dlion::kTile;
        c->d += segs[s].numel;
    }
    c->nseg = nseg;
    c->ntiles = tiles;
    c->d_pad = d_pad;
    c->n_workers = n_workers;
    c->beta1 = beta1;
    c->beta2 = beta2;
    c->lr = lr;
    c->wd = weight_decay;
    c->mode = mode;
    c->gdtype = gdtype;

    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e != cudaSuccess) {
        delete c;
        return DLION_ECUDA;
    }
    if (tiles != 0) {
        std::vector<dlion::TileRow> trows;
        try {
            trows.reserve(tiles);
        } catch (...) {
            delete c;
            return DLION_ENOMEM;
        }
        for (uint32_t s = 0; s < nseg; ++s) {
            for (uint64_t off = 0; off < segs[s].numel; off += dlion::kTile) {
                dlion::TileRow r;
                r.base = segs[s].elem_offset + off;
                r.valid = static_cast<uint32_t>(segs[s].numel - off < dlion::kTile ? segs[s].numel - off : dlion::kTile);
                r.tensor = s;
                trows.push_back(r);
            }
        }
        e = cudaMalloc(reinterpret_cast<void**>(&c->tiles_dev), sizeof(dlion::TileRow) * tiles);
        if (e == cudaSuccess) {
            e = cudaMemcpy(c->tiles_dev, trows.data(), sizeof(dlion::TileRow) * tiles, cudaMemcpyHostToDevice);
        }
        if (e != cudaSuccess) {
            if (c->tiles_dev != nullptr) cudaFree(c->tiles_dev);
            delete c;
            return e == cudaErrorMemoryAllocation ? DLION_ENOMEM : DLION_ECUDA;
        }
    }
    *out = c;
    return DLION_OK;
}

dlion_status dlion_set_lr(dlion_ctx* ctx, float lr) {
    if (ctx == nullptr || !nonneg_finite(lr)) return DLION_EINVAL;
    ctx->lr = lr;
    return DLION_OK;
}

dlion_status dlion_set_momentum_dtype(dlion_ctx* ctx, dlion_sdtype sdtype) {
    if (ctx == nullptr || (sdtype != DLION_STATE_F32 && sdtype != DLION_STATE_BF16)) return DLION_EINVAL;
    ctx->sdtype = sdtype;
    return DLION_OK;
}

dlion_status dlion_set_worker_betas(dlion_ctx* ctx, int worker, float beta1, float beta2) {
    if (ctx == nullptr || worker < 0 || worker >= static_cast<int>(ctx->n_workers)) return DLION_EINVAL;
    if (!unit_interval(beta1) || !unit_interval(beta2)) return DLION_EINVAL;
    const dlion_status ds = device_ok(ctx);
    if (ds != DLION_OK) return ds;
    if (ctx->betas.empty()) {
        try {
            ctx->betas.assign(ctx->n_workers, common_betas(ctx));
        } catch (...) {
            return DLION_ENOMEM;
        }
        const cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->betas_dev),
                                         sizeof(dlion::Betas) * ctx->n_workers);
        if (e != cudaSuccess) {
            ctx->betas.clear();
            ctx->betas_dev = nullptr;
            return e == cudaErrorMemoryAllocation ? DLION_ENOMEM : DLION_ECUDA;
        }
    }
    dlion::Betas k;
    k.b1 = beta1;
    k.om1 = 1.0f - beta1;
    k.b2 = beta2;
    k.om2 = 1.0f - beta2;
    ctx->betas[worker] = k;
    if (cudaMemcpy(ctx->betas_dev, ctx->betas.data(), sizeof(dlion::Betas) * ctx->n_workers,
                   cudaMemcpyHostToDevice) != cudaSuccess) {
        return DLION_ECUDA;
    }
    return DLION_OK;
}

dlion_status dlion_worker_step(dlion_ctx* ctx, int worker, const void* grads, void* m,
                               uint32_t* packed, void* cuda_stream) {
    if (ctx == nullptr || grads == nullptr || m == nullptr || packed == nullptr) return DLION_EINVAL;
    if (worker < -1 || worker >= static_cast<int>(ctx->n_workers)) return DLION_EINVAL;
    if (!aligned(grads, 16) || !aligned(m, 16) || !aligned(packed, 16)) return DLION_EALIGN;
    const dlion_status ds = device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::WorkerParams p = dlion::worker_params(ctx, worker);
    p.g = grads;
    p.m = m;
    p.packed = packed;
    const cudaError_t e = dlion::launch_worker_step(p, ctx->gdtype == DLION_GRAD_BF16, ctx->sm_count,
                                                    static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

namespace {
dlion_status aggregate_apply_any(dlion_ctx* ctx, const uint32_t* packed, float* x, uint32_t* delta_bits_out,
                                 uint8_t* count_out, uint16_t* count16_out, void* cuda_stream);
}

dlion_status dlion_aggregate_apply(dlion_ctx* ctx, const uint32_t* packed, float* x,
                                   uint32_t* delta_bits_out, uint8_t* count_out, void* cuda_stream) {
    return aggregate_apply_any(ctx, packed, x, delta_bits_out, count_out, nullptr, cuda_stream);
}

dlion_status dlion_aggregate_apply_counts16(dlion_ctx* ctx, const uint32_t* packed, float* x,
                                            uint32_t* delta_bits_out, uint16_t* count16_out,
                                            void* cuda_stream) {
    if (count16_out == nullptr) return DLION_EINVAL;
    return aggregate_apply_any(ctx, packed, x, delta_bits_out, nullptr, count16_out, cuda_stream);
}

}  // extern "C"

namespace {
dlion_status aggregate_apply_any(dlion_ctx* ctx, const uint32_t* packed, float* x, uint32_t* delta_bits_out,
                                 uint8_t* count_out, uint16_t* count16_out, void* cuda_stream) {
    if (ctx == nullptr || packed == nullptr || x == nullptr) return DLION_EINVAL;
    if (count_out != nullptr && ctx->n_workers > DLION_MAX_WORKERS_BYTE_COUNTS) return DLION_EINVAL;
    if (!aligned(packed, 16) || !aligned(x, 16) || !aligned(delta_bits_out, 16) || !aligned(count_out, 4) ||
        !aligned(count16_out, 8)) {
        return DLION_EALIGN;
    }
    const dlion_status ds = device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::AggParams p = dlion::agg_params(ctx);
    p.packed = packed;
    p.x = x;
    p.delta_bits = delta_bits_out;
    p.count = count_out;
    p.count16 = count16_out;
    const cudaError_t e = dlion::launch_aggregate_apply(p, ctx->sm_count, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}
}  // namespace

extern "C" {

dlion_status dlion_step_fused(dlion_ctx* ctx, const void* grads, void* m, float* x,
                              uint32_t* packed_out, void* cuda_stream) {
    if (ctx == nullptr || grads == nullptr || m == nullptr || x == nullptr) return DLION_EINVAL;
    if (ctx->n_workers > DLION_MAX_WORKERS_BYTE_COUNTS) return DLION_EINVAL;       // byte-wide vote counters
    if (!aligned(grads, 16) || !aligned(m, 16) || !aligned(x, 16) || !aligned(packed_out, 16)) {
        return DLION_EALIGN;
    }
    const dlion_status ds = device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::FusedParams p;
    p.g = grads;
    p.m = m;
    p.x = x;
    p.packed = packed_out;
    p.tiles = ctx->tiles_dev;
    p.flat_d = 0;
    p.n_workers = ctx->n_workers;
    p.ntiles = ctx->ntiles;
    p.d_pad = ctx->d_pad;
    p.k = common_betas(ctx);
    p.betas = ctx->betas_dev;
    p.m_bf16 = ctx->sdtype == DLION_STATE_BF16 ? 1 : 0;
    p.lr = ctx->lr;
    p.wd = ctx->wd;
    p.ternary = ctx->mode == DLION_MAJORITY_TERNARY ? 1 : 0;
    p.average = (ctx->mode == DLION_AVERAGE || p.ternary) ? 1 : 0;      // ternary: the table variant, with signs in the table
    const cudaError_t e = dlion::launch_step_fused(p, ctx->gdtype == DLION_GRAD_BF16, ctx->sm_count,
                                                   static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

dlion_status dlion_step_global(dlion_ctx* ctx, const void* grads, float* m, float* x,
                               uint32_t* delta_bits_out, void* cuda_stream) {
    if (ctx == nullptr || grads == nullptr || m == nullptr || x == nullptr) return DLION_EINVAL;
    if (ctx->sdtype != DLION_STATE_F32 || !ctx->betas.empty()) return DLION_EINVAL;   // one beta pair, fp32 momentum
    if (!aligned(grads, 16) || !aligned(m, 16) || !aligned(x, 16) || !aligned(delta_bits_out, 16)) {
        return DLION_EALIGN;
    }
    const dlion_status ds = device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::GlobalParams p;
    p.g = grads;
    p.m = m;
    p.x = x;
    p.delta_bits = delta_bits_out;
    p.tiles = ctx->tiles_dev;
    p.flat_d = 0;
    p.n_workers = ctx->n_workers;
    p.ntiles = ctx->ntiles;
    p.d_pad = ctx->d_pad;
    p.k = common_betas(ctx);
    p.lr = ctx->lr;
    p.wd = ctx->wd;
    const cudaError_t e = dlion::launch_step_global(p, ctx->gdtype == DLION_GRAD_BF16,
                                                    static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

}  // extern "C"
