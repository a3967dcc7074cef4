// Host-gradient step, analytic wire volume, and context teardown (include/dlion.h).
#include "dlion_ctx.cuh"
#include "host_checks.h"

namespace {

using dlion::aligned16;

void drop_pipeline(dlion_ctx* c) {
    for (int k = 0; k < 2; ++k) {
        if (c->copied[k] != nullptr) cudaEventDestroy(c->copied[k]);
        if (c->consumed[k] != nullptr) cudaEventDestroy(c->consumed[k]);
        c->copied[k] = nullptr;
        c->consumed[k] = nullptr;
    }
    if (c->entry != nullptr) cudaEventDestroy(c->entry);
    c->entry = nullptr;
    if (c->copy_stream != nullptr) cudaStreamDestroy(c->copy_stream);
    c->copy_stream = nullptr;
}

// Streams and events of the copy pipeline; created once, on first use.  All or
// nothing: a partial failure destroys what was created, so a later call starts
// over instead of running with missing events.
cudaError_t ensure_pipeline(dlion_ctx* c) {
    if (c->copy_stream != nullptr) return cudaSuccess;
    cudaError_t e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) c->copy_stream = nullptr;
    for (int k = 0; k < 2 && e == cudaSuccess; ++k) {
        e = cudaEventCreateWithFlags(&c->copied[k], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->consumed[k], cudaEventDisableTiming);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->entry, cudaEventDisableTiming);
    if (e != cudaSuccess) drop_pipeline(c);
    return e;
}

}  // namespace

extern "C" {

dlion_status dlion_step_host(dlion_ctx* ctx, const void* host_grads, void* m, float* x,
                             uint32_t* packed, void* staging, void* delta_wire_dev,
                             void* host_delta_out, void* cuda_stream) {
    if (ctx == nullptr || host_grads == nullptr || m == nullptr || x == nullptr || packed == nullptr ||
        staging == nullptr) {
        return DLION_EINVAL;
    }
    if (host_delta_out != nullptr && delta_wire_dev == nullptr) return DLION_EINVAL;
    if (!aligned16(m) || !aligned16(x) || !aligned16(packed) || !aligned16(staging) ||
        !aligned16(delta_wire_dev)) {
        return DLION_EALIGN;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DLION_ECUDA;
    if (dev != ctx->device) return DLION_ESTATE;
    if (ensure_pipeline(ctx) != cudaSuccess) return DLION_ECUDA;

    cudaStream_t main = static_cast<cudaStream_t>(cuda_stream);
    const size_t gsz = ctx->gdtype == DLION_GRAD_BF16 ? 2 : 4;
    const size_t msz = ctx->sdtype == DLION_STATE_BF16 ? 2 : 4;
    const size_t slice = static_cast<size_t>(ctx->d_pad) * gsz;        // one worker's gradients
    const size_t words = static_cast<size_t>(ctx->d_pad / 32);
    const char* hsrc = static_cast<const char*>(host_grads);
    char* stage = static_cast<char*>(staging);

    // the copy stream may not start before the work already queued on main
    // (a previous step may still be reading the staging slices)
    if (cudaEventRecord(ctx->entry, main) != cudaSuccess) return DLION_ECUDA;
    if (cudaStreamWaitEvent(ctx->copy_stream, ctx->entry, 0) != cudaSuccess) return DLION_ECUDA;

    for (uint32_t i = 0; i < ctx->n_workers; ++i) {
        const int b = static_cast<int>(i & 1u);
        if (i >= 2 && cudaStreamWaitEvent(ctx->copy_stream, ctx->consumed[b], 0) != cudaSuccess) return DLION_ECUDA;
        if (cudaMemcpyAsync(stage + b * slice, hsrc + i * slice, slice, cudaMemcpyHostToDevice,
                            ctx->copy_stream) != cudaSuccess) return DLION_ECUDA;
        if (cudaEventRecord(ctx->copied[b], ctx->copy_stream) != cudaSuccess) return DLION_ECUDA;
        if (cudaStreamWaitEvent(main, ctx->copied[b], 0) != cudaSuccess) return DLION_ECUDA;
        const dlion_status st = dlion_worker_step(ctx, static_cast<int>(i), stage + b * slice,
                                                  static_cast<char*>(m) + static_cast<size_t>(i) * ctx->d_pad * msz,
                                                  packed + static_cast<size_t>(i) * words, main);
        if (st != DLION_OK) return st;
        if (cudaEventRecord(ctx->consumed[b], main) != cudaSuccess) return DLION_ECUDA;
    }
    // Server side.  The broadcast message, when asked for, is in the format of
    // dlion_aggregate: one plane of Delta bits (Majority Vote) or the K count planes
    // (Averaging; vote and update are then two launches with the message in between).
    const bool avg = ctx->mode != DLION_MAJORITY;          // more than one plane: vote and apply are two launches
    uint32_t* wire = static_cast<uint32_t*>(delta_wire_dev);
    dlion_status st;
    if (avg && wire != nullptr) {
        st = dlion_aggregate(ctx, packed, wire, main);
        if (st == DLION_OK) st = dlion_apply_delta(ctx, wire, x, main);
    } else {
        st = dlion_aggregate_apply(ctx, packed, x, wire, nullptr, main);
    }
    if (st != DLION_OK) return st;
    if (host_delta_out != nullptr) {
        const size_t bytes = static_cast<size_t>(dlion_delta_planes(ctx)) * words * 4;
        if (cudaMemcpyAsync(host_delta_out, wire, bytes, cudaMemcpyDeviceToHost, main) != cudaSuccess) {
            return DLION_ECUDA;
        }
    }
    return DLION_OK;
}

uint32_t dlion_delta_planes(const dlion_ctx* ctx) {
    if (ctx == nullptr) return 0;
    if (ctx->mode == DLION_MAJORITY_TERNARY) return 2u;       // three values of Delta: two bits
    return ctx->mode == DLION_AVERAGE ? dlion::planes_for(ctx->n_workers) : 1u;
}

dlion_status dlion_aggregate(dlion_ctx* ctx, const uint32_t* packed, uint32_t* delta_wire, void* cuda_stream) {
    if (ctx == nullptr || packed == nullptr || delta_wire == nullptr) return DLION_EINVAL;
    if (!aligned16(packed) || !aligned16(delta_wire)) return DLION_EALIGN;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DLION_ECUDA;
    if (dev != ctx->device) return DLION_ESTATE;
    dlion::WireParams p = dlion::wire_params(ctx, 0);
    p.packed = packed;
    p.wire_out = delta_wire;
    if (dlion::launch_wire(p, false, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

dlion_status dlion_apply_delta(dlion_ctx* ctx, const uint32_t* delta_wire, float* x, void* cuda_stream) {
    return dlion_apply_delta_sliced(ctx, delta_wire, 0, x, cuda_stream);
}

dlion_status dlion_apply_delta_sliced(dlion_ctx* ctx, const uint32_t* delta_wire, uint64_t slice_words,
                                      float* x, void* cuda_stream) {
    if (ctx == nullptr || delta_wire == nullptr || x == nullptr) return DLION_EINVAL;
    if (slice_words != 0 && (ctx->d_pad / 32) % slice_words != 0) return DLION_EINVAL;   // whole slices only
    if (!aligned16(delta_wire) || !aligned16(x)) return DLION_EALIGN;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DLION_ECUDA;
    if (dev != ctx->device) return DLION_ESTATE;
    dlion::WireParams p = dlion::wire_params(ctx, slice_words);
    dlion::decode_ternary_as_two_workers(p);
    p.wire_in = delta_wire;
    p.x = x;
    if (dlion::launch_wire(p, true, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

uint64_t dlion_wire_bytes(const dlion_ctx* ctx, int direction) {
    if (ctx == nullptr) return 0;
    const uint64_t d = ctx->d;
    uint64_t bits;
    if (direction == 0) {
        bits = static_cast<uint64_t>(ctx->n_workers) * d;
    } else if (direction == 1) {
        uint32_t per = 1;
        if (ctx->mode == DLION_MAJORITY_TERNARY) {
            per = 2;
        } else if (ctx->mode == DLION_AVERAGE) {
            per = 0;
            while ((1ull << per) < static_cast<uint64_t>(ctx->n_workers) + 1) ++per;   // N+1 values
        }
        bits = d * per;
    } else if (direction == 2) {
        bits = 32 * d;
    } else {
        return 0;
    }
    return (bits + 7) / 8;
}

uint64_t dlion_launch_count(const dlion_ctx* ctx) { return ctx == nullptr ? 0 : ctx->launches; }

const char* dlion_status_str(dlion_status s) {
    switch (s) {
        case DLION_OK: return "ok";
        case DLION_EINVAL: return "invalid argument";
        case DLION_EALIGN: return "misaligned pointer or offset";
        case DLION_ENOMEM: return "out of memory";
        case DLION_ECUDA: return "CUDA error";
        case DLION_ESTATE: return "wrong device or unusable context";
    }
    return "unknown status";
}

void dlion_destroy(dlion_ctx* ctx) {
    if (ctx == nullptr) return;
    if (ctx->tiles_dev != nullptr) cudaFree(ctx->tiles_dev);
    if (ctx->betas_dev != nullptr) cudaFree(ctx->betas_dev);
    if (ctx->tables_dev != nullptr) cudaFree(ctx->tables_dev);
    if (ctx->scatter_dev != nullptr) cudaFree(ctx->scatter_dev);
    drop_pipeline(ctx);
    delete ctx;
}

}  // extern "C"
