// Global Lion, the full-precision scheme Distributed Lion is compared against
// (arXiv 2404.00438: appendix "Global Lion Convergence", the scheme labelled
// Global Lion; Section 5.1 "G-Lion"; Table 1 row "Global Lion/AdamW"), as one
// launch over all N workers.  Per coordinate:
//     mt_i  = beta1 m_i + (1-beta1) g_i                     (old m_i)
//     m_i  <- beta2 m_i + (1-beta2) g_i
//     G     = (1/N) sum_i mt_i       binary32, summed in worker order, one division
//     x    <- x - lr ( sign(G) + lambda x )
// What would cross the wire here is the fp32 blend of every worker (32 d bits each
// way, Table 1), which is exactly what Distributed Lion avoids; on one GPU the
// sum never leaves the registers.  It exists as the measured denominator of the
// comparison: same inputs, same state traffic (N (G + 8) + 8 bytes per
// coordinate), one sign instead of N.
//
// Same tile and lane mapping as the fused Distributed-Lion step: a thread keeps
// 16 coordinates for all workers, one fp32 accumulator each, and the worker loop
// is software-pipelined (worker i+1 in flight while worker i is consumed).
#include "worker_regs.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 256;             // 8 warps x 512 coordinates = one tile

__device__ __forceinline__ float blend_and_update(float g, float& m, const Betas& k) {
    const float mt = __fadd_rn(__fmul_rn(k.b1, m), __fmul_rn(k.om1, g));
    m = __fadd_rn(__fmul_rn(k.b2, m), __fmul_rn(k.om2, g));
    return mt;
}

__device__ __forceinline__ float sign_of_mean(float total, float nf) {
    return __fdiv_rn(total, nf) >= 0.0f ? 1.0f : -1.0f;
}

template <bool BF16>
__device__ __forceinline__ void consume(const GlobalParams& p, WorkerRegs<BF16, false>& r, bool first,
                                        unsigned long long at, float4 (&acc)[kChunksPerWarp]) {
#pragma unroll
    for (int u = 0; u < kChunksPerWarp; ++u) {
        const float4 g = r.grad(u);
        float4 t;
        t.x = blend_and_update(g.x, r.m[u].x, p.k);
        t.y = blend_and_update(g.y, r.m[u].y, p.k);
        t.z = blend_and_update(g.z, r.m[u].z, p.k);
        t.w = blend_and_update(g.w, r.m[u].w, p.k);
        store_state4<false>(p.m, at + u * kChunk, r.m[u]);
        if (first) {
            acc[u] = t;                                            // the sum starts from worker 0's blend
        } else {
            acc[u].x = __fadd_rn(acc[u].x, t.x);
            acc[u].y = __fadd_rn(acc[u].y, t.y);
            acc[u].z = __fadd_rn(acc[u].z, t.z);
            acc[u].w = __fadd_rn(acc[u].w, t.w);
        }
    }
}

// Last tile of a segment: every access guarded, one chunk at a time.
template <bool BF16>
__device__ __noinline__ void ragged_tile(const GlobalParams& p, const TileRef t, uint32_t in_tile,
                                         unsigned long long e0, uint32_t lane, float nf) {
#pragma unroll 1
    for (int u = 0; u < kChunksPerWarp; ++u) {
        const uint32_t c0 = in_tile + u * kChunk;
        if (c0 >= t.valid) break;                                  // warp-uniform
        const uint32_t j0 = c0 + lane * 4;
        const uint32_t mine_n = j0 >= t.valid ? 0u : (t.valid - j0 >= 4u ? 4u : t.valid - j0);
        float total[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        for (uint32_t i = 0; i < p.n_workers; ++i) {
            const unsigned long long e = i * p.d_pad + e0 + u * kChunk;
            for (uint32_t q = 0; q < mine_n; ++q) {
                const float g = load_grad1<BF16>(p.g, e + q);
                float m = static_cast<const float*>(p.m)[e + q];
                const float mt = blend_and_update(g, m, p.k);
                static_cast<float*>(p.m)[e + q] = m;
                total[q] = i == 0 ? mt : __fadd_rn(total[q], mt);
            }
        }
        uint32_t nib = 0;
        for (uint32_t q = 0; q < mine_n; ++q) {
            const unsigned long long e = e0 + u * kChunk + q;
            const float delta = sign_of_mean(total[q], nf);
            nib |= (delta > 0.0f ? 1u : 0u) << q;
            p.x[e] = apply_coord(p.x[e], delta, p.lr, p.wd);
        }
        if (p.delta_bits != nullptr) {                             // block-uniform
            const uint32_t w = gather_word(nib, lane);
            if ((lane & 7u) == 0 && c0 + (lane >> 3) * 32 < t.valid) {
                p.delta_bits[(t.base + c0) / 32 + (lane >> 3)] = w;
            }
        }
    }
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads, 2)
step_global_kernel(const __grid_constant__ GlobalParams p) {
    const uint32_t n = p.n_workers;
    const float nf = static_cast<float>(n);
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        const uint32_t in_tile = warp * (kChunksPerWarp * kChunk);
        if (in_tile >= t.valid) continue;                          // warp-uniform
        const unsigned long long e0 = t.base + in_tile + lane * 4;  // my first coordinate (chunk 0)
        if (t.valid != kTile) {
            ragged_tile<BF16>(p, t, in_tile, e0, lane, nf);
            continue;
        }
        float4 acc[kChunksPerWarp];
        WorkerRegs<BF16, false> a, b;
        a.load(p.g, p.m, e0);
        uint32_t i = 0;
        for (; i + 2 <= n; i += 2) {
            b.load(p.g, p.m, (i + 1) * p.d_pad + e0);
            consume<BF16>(p, a, i == 0, i * p.d_pad + e0, acc);
            if (i + 2 < n) a.load(p.g, p.m, (i + 2) * p.d_pad + e0);
            consume<BF16>(p, b, false, (i + 1) * p.d_pad + e0, acc);
        }
        // x is fetched while the last worker is consumed (two workers' registers plus
        // the accumulators leave no room to hold it through the loop)
        float4 xv[kChunksPerWarp];
#pragma unroll
        for (int u = 0; u < kChunksPerWarp; ++u) {
            xv[u] = *(reinterpret_cast<const float4*>(p.x + e0 + u * kChunk));
        }
        if (i < n) consume<BF16>(p, a, i == 0, i * p.d_pad + e0, acc);
        uint32_t mine = 0;
#pragma unroll
        for (int u = 0; u < kChunksPerWarp; ++u) {
            const float d0 = sign_of_mean(acc[u].x, nf), d1 = sign_of_mean(acc[u].y, nf);
            const float d2 = sign_of_mean(acc[u].z, nf), d3 = sign_of_mean(acc[u].w, nf);
            float4 v = xv[u];
            v.x = apply_coord(v.x, d0, p.lr, p.wd);
            v.y = apply_coord(v.y, d1, p.lr, p.wd);
            v.z = apply_coord(v.z, d2, p.lr, p.wd);
            v.w = apply_coord(v.w, d3, p.lr, p.wd);
            *reinterpret_cast<float4*>(p.x + e0 + u * kChunk) = v;
            if (p.delta_bits != nullptr) {                         // block-uniform
                const uint32_t nib = (d0 > 0.0f ? 1u : 0u) | (d1 > 0.0f ? 2u : 0u) | (d2 > 0.0f ? 4u : 0u) |
                                     (d3 > 0.0f ? 8u : 0u);
                const uint32_t w = gather_word(nib, lane);
                if ((lane & 7u) == static_cast<uint32_t>(u)) mine = w;
            }
        }
        if (p.delta_bits != nullptr && (lane & 7u) < kChunksPerWarp) {
            p.delta_bits[(t.base + in_tile) / 32 + 4u * (lane & 7u) + (lane >> 3)] = mine;
        }
    }
}

}  // namespace

cudaError_t launch_step_global(const GlobalParams& p, bool bf16, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    if (bf16) step_global_kernel<true><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    else step_global_kernel<false><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace dlion
