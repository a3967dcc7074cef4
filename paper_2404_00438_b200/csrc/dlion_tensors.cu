// The indirect modes of the two-stage path (include/dlion.h).
//
// Per-tensor mode: parameters, gradients and
// momenta that live in separately allocated tensors -- a framework's parameter list --
// are stepped where they are, through pointer tables, instead of being copied into flat
// arenas.  The kernels are the arena kernels; only the base address of each stream is
// looked up per tensor.
#include <cstring>

#include "dlion_ctx.cuh"
#include "host_checks.h"

namespace {

using dlion::aligned16;

// Table entry for a tensor: the distance in bytes from `base` to the tensor's storage,
// minus the byte offset of its first coordinate in the arena numbering (see WorkerParams).
// Plain integer arithmetic: the biased value is only ever used with an index that brings
// it back inside the tensor.
long long entry(const void* tensor, const void* base, uint64_t elem_offset, size_t elem_size) {
    return static_cast<long long>(reinterpret_cast<uintptr_t>(tensor) - reinterpret_cast<uintptr_t>(base) -
                                  static_cast<uintptr_t>(elem_offset) * elem_size);
}

}  // namespace

extern "C" {

dlion_status dlion_bind_tensors(dlion_ctx* ctx, const void* const* grads, void* const* m, float* const* x,
                                void* cuda_stream) {
    if (ctx == nullptr || (grads == nullptr && m == nullptr && x == nullptr)) return DLION_EINVAL;
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    const size_t nseg = ctx->nseg, N = ctx->n_workers;
    const size_t gsz = ctx->gdtype == DLION_GRAD_BF16 ? 2 : 4;
    const size_t msz = ctx->sdtype == DLION_STATE_BF16 ? 2 : 4;
    // every pointer is checked before anything changes
    for (size_t k = 0; k < nseg; ++k) {
        const bool holds = ctx->segs[k].numel != 0;
        for (size_t i = 0; i < N; ++i) {
            if (grads != nullptr && ((holds && grads[i * nseg + k] == nullptr))) return DLION_EINVAL;
            if (m != nullptr && ((holds && m[i * nseg + k] == nullptr))) return DLION_EINVAL;
            if (grads != nullptr && !aligned16(grads[i * nseg + k])) return DLION_EALIGN;
            if (m != nullptr && !aligned16(m[i * nseg + k])) return DLION_EALIGN;
        }
        if (x != nullptr && holds && x[k] == nullptr) return DLION_EINVAL;
        if (x != nullptr && !aligned16(x[k])) return DLION_EALIGN;
    }
    const size_t total = (2 * N + 1) * nseg;
    if (ctx->tables_dev == nullptr) {
        try {
            ctx->tables_host.assign(total, 0);
        } catch (...) {
            return DLION_ENOMEM;
        }
        const cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->tables_dev), total * sizeof(long long));
        if (e != cudaSuccess) {
            ctx->tables_dev = nullptr;
            ctx->tables_host.clear();
            return e == cudaErrorMemoryAllocation ? DLION_ENOMEM : DLION_ECUDA;
        }
    }
    long long* h = ctx->tables_host.data();
    const void* base = ctx->tables_dev;             // the pointer the kernels are given beside each table
    for (size_t k = 0; k < nseg; ++k) {
        const uint64_t off = ctx->segs[k].elem_offset;
        for (size_t i = 0; i < N; ++i) {
            if (grads != nullptr) h[i * nseg + k] = entry(grads[i * nseg + k], base, off, gsz);
            if (m != nullptr) h[(N + i) * nseg + k] = entry(m[i * nseg + k], base, off, msz);
        }
        if (x != nullptr) h[2 * N * nseg + k] = entry(x[k], base, off, sizeof(float));
    }
    // pageable source: the runtime has taken its copy of the table when this returns,
    // and the copy itself is ordered on the stream before the steps that follow
    if (cudaMemcpyAsync(ctx->tables_dev, h, total * sizeof(long long), cudaMemcpyHostToDevice,
                        static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        return DLION_ECUDA;
    }
    ctx->bound_g = ctx->bound_g || grads != nullptr;
    ctx->bound_m = ctx->bound_m || m != nullptr;
    ctx->bound_x = ctx->bound_x || x != nullptr;
    return DLION_OK;
}

dlion_status dlion_worker_step_tensors(dlion_ctx* ctx, int worker, uint32_t* packed, void* cuda_stream) {
    if (ctx == nullptr || packed == nullptr) return DLION_EINVAL;
    if (worker < -1 || worker >= static_cast<int>(ctx->n_workers)) return DLION_EINVAL;
    if (!ctx->bound_g || !ctx->bound_m) return DLION_ESTATE;
    if (!aligned16(packed)) return DLION_EALIGN;
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::WorkerParams p = dlion::worker_params(ctx, worker);
    const size_t rows = static_cast<size_t>(ctx->n_workers) * ctx->nseg;
    p.g = ctx->tables_dev;
    p.m = ctx->tables_dev;
    p.g_off = ctx->tables_dev;
    p.m_off = ctx->tables_dev + rows;
    p.packed = packed;
    if (dlion::launch_worker_step(p, ctx->gdtype == DLION_GRAD_BF16, ctx->sm_count,
                                  static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        return DLION_ECUDA;
    }
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

dlion_status dlion_aggregate_apply_tensors(dlion_ctx* ctx, const uint32_t* packed, uint32_t* delta_bits_out,
                                           void* cuda_stream) {
    if (ctx == nullptr || packed == nullptr) return DLION_EINVAL;
    if (!ctx->bound_x) return DLION_ESTATE;
    if (!aligned16(packed) || !aligned16(delta_bits_out)) return DLION_EALIGN;
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::AggParams p = dlion::agg_params(ctx);
    p.packed = packed;
    p.delta_bits = delta_bits_out;
    p.x = reinterpret_cast<float*>(ctx->tables_dev);
    p.x_off = ctx->tables_dev + 2 * static_cast<size_t>(ctx->n_workers) * ctx->nseg;
    if (dlion::launch_aggregate_apply(p, ctx->sm_count, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        return DLION_ECUDA;
    }
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

dlion_status dlion_apply_delta_tensors(dlion_ctx* ctx, const uint32_t* delta_wire, uint64_t slice_words,
                                       void* cuda_stream) {
    if (ctx == nullptr || delta_wire == nullptr) return DLION_EINVAL;
    if (slice_words != 0 && (ctx->d_pad / 32) % slice_words != 0) return DLION_EINVAL;
    if (!ctx->bound_x) return DLION_ESTATE;
    if (!aligned16(delta_wire)) return DLION_EALIGN;
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::WireParams p = dlion::wire_params(ctx, slice_words);
    dlion::decode_ternary_as_two_workers(p);
    p.wire_in = delta_wire;
    p.x = reinterpret_cast<float*>(ctx->tables_dev);
    p.x_off = ctx->tables_dev + 2 * static_cast<size_t>(ctx->n_workers) * ctx->nseg;
    if (dlion::launch_wire(p, true, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return DLION_ECUDA;
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

// ---- scatter mode: the send of the worker = GPU exchange fused into the worker-side kernel.
// Instead of one contiguous wire buffer, a worker's sign words are stored straight into
// one receive buffer per coordinate slice -- on a multi-GPU job the buffers of the ranks
// that vote on those slices, mapped into this process (plain stores to peer memory, no
// multicast, no loads from a peer) -- so the all-to-all needs no pass of its own.

dlion_status dlion_bind_scatter(dlion_ctx* ctx, uint32_t* const* dst, uint32_t n_dst, uint64_t slice_words,
                                uint32_t slot, uint32_t rows) {
    if (ctx == nullptr || dst == nullptr || n_dst == 0 || slice_words == 0 || slot >= rows) return DLION_EINVAL;
    if (static_cast<uint64_t>(n_dst) * slice_words != ctx->d_pad / 32) return DLION_EINVAL;   // the slices partition the arena
    for (uint32_t r = 0; r < n_dst; ++r) {
        if (dst[r] == nullptr) return DLION_EINVAL;
        if (!aligned16(dst[r])) return DLION_EALIGN;
    }
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    if (ctx->scatter_dev != nullptr && ctx->scatter_n != n_dst) {
        cudaFree(ctx->scatter_dev);
        ctx->scatter_dev = nullptr;
    }
    if (ctx->scatter_dev == nullptr) {
        const cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&ctx->scatter_dev), n_dst * sizeof(long long));
        if (e != cudaSuccess) {
            ctx->scatter_dev = nullptr;
            return e == cudaErrorMemoryAllocation ? DLION_ENOMEM : DLION_ECUDA;
        }
    }
    std::vector<long long> off;
    try {
        off.resize(n_dst);
    } catch (...) {
        return DLION_ENOMEM;
    }
    for (uint32_t r = 0; r < n_dst; ++r) off[r] = entry(dst[r], ctx->scatter_dev, 0, 1);
    // synchronous: bound once, outside the step loop
    if (cudaMemcpy(ctx->scatter_dev, off.data(), n_dst * sizeof(long long), cudaMemcpyHostToDevice) != cudaSuccess) {
        return DLION_ECUDA;
    }
    ctx->scatter_n = n_dst;
    ctx->scatter_slice_words = slice_words;
    ctx->scatter_slot = slot;
    return DLION_OK;
}

dlion_status dlion_worker_step_scatter(dlion_ctx* ctx, int worker, const void* grads, void* m, void* cuda_stream) {
    if (ctx == nullptr || grads == nullptr || m == nullptr) return DLION_EINVAL;
    if (worker < 0 || worker >= static_cast<int>(ctx->n_workers)) return DLION_EINVAL;    // one worker per call
    if (ctx->scatter_dev == nullptr) return DLION_ESTATE;
    if (!aligned16(grads) || !aligned16(m)) return DLION_EALIGN;
    const dlion_status ds = dlion::device_ok(ctx);
    if (ds != DLION_OK) return ds;
    dlion::WorkerParams p = dlion::worker_params(ctx, worker);
    p.g = grads;
    p.m = m;
    p.packed = reinterpret_cast<uint32_t*>(ctx->scatter_dev);      // the base the offsets count from
    p.dst_off = ctx->scatter_dev;
    p.slice_words = ctx->scatter_slice_words;
    p.slot = ctx->scatter_slot;
    if (dlion::launch_worker_step(p, ctx->gdtype == DLION_GRAD_BF16, ctx->sm_count,
                                  static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
        return DLION_ECUDA;
    }
    if (ctx->ntiles != 0) ctx->launches += 1;
    return DLION_OK;
}

}  // extern "C"
