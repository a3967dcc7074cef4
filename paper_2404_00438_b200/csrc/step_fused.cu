// One whole iteration of Algorithm 1 (arXiv 2404.00438) in a single launch:
// worker side for all N workers, the vote, and x <- x - lr (Delta + lambda x)
// (Section 3.2).  A thread keeps the same 16 coordinates for every worker, so
// the vote never leaves its registers: four byte-wide counters per 32-bit
// register, one register per 128-coordinate chunk.  The 1-bit wire buffer is
// written only when the caller asks for it.
//
// Same tile and lane mapping as the worker-side kernel (warp = 512 consecutive
// coordinates, lane l of a chunk = coordinates 4l..4l+3).  The
// worker loop is software-pipelined: worker i+1's loads are issued before worker
// i is consumed.  HBM traffic per
// coordinate: N (G + 8) + 8 B, G = gradient bytes (+ N/8 B with the wire buffer):
// the 2 N/8 B round trip of the two-stage path is gone.
#include "worker_regs.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 256;             // 8 warps x 512 coordinates = one tile

template <bool AVG>
__device__ __forceinline__ float delta_of(uint32_t count, uint32_t thr, const float* avg_table) {
    if constexpr (AVG) return avg_table[count];
    return count >= thr ? 1.0f : -1.0f;
}

// Worker-side update of my coordinates for one worker: momenta stored, votes
// added to cnt (one byte per coordinate), wire words written if requested.
template <bool BF16, bool MB16>
__device__ __forceinline__ void consume(const FusedParams& p, WorkerRegs<BF16, MB16>& r, uint32_t worker,
                                        unsigned long long at, uint32_t* wire_words, uint32_t lane,
                                        uint32_t (&cnt)[kChunksPerWarp]) {
    const Betas k = betas_of(p.betas, p.k, worker);
    uint32_t mine = 0;
#pragma unroll
    for (int u = 0; u < kChunksPerWarp; ++u) {
        const float4 g = r.grad(u);
        uint32_t nib = lion_coord(g.x, r.m[u].x, k);
        nib |= lion_coord(g.y, r.m[u].y, k) << 1;
        nib |= lion_coord(g.z, r.m[u].z, k) << 2;
        nib |= lion_coord(g.w, r.m[u].w, k) << 3;
        store_state4<MB16>(p.m, at + u * kChunk, r.m[u]);
        cnt[u] += spread_nibble(nib);
        if (wire_words != nullptr) {                              // block-uniform
            const uint32_t w = gather_word(nib, lane);
            if ((lane & 7u) == static_cast<uint32_t>(u)) mine = w;
        }
    }
    if (wire_words != nullptr && (lane & 7u) < kChunksPerWarp) {
        wire_words[4u * (lane & 7u) + (lane >> 3)] = mine;
    }
}

// Last tile of a segment: every access guarded, one chunk at a time.
template <bool BF16, bool AVG, bool MB16>
__device__ __noinline__ void ragged_tile(const FusedParams& p, const TileRef t, uint32_t in_tile,
                                         unsigned long long e0, uint32_t lane, uint32_t thr,
                                         const float* avg_table) {
    const uint32_t n = p.n_workers;
    const unsigned long long w_stride = p.d_pad / 32;
#pragma unroll 1
    for (int u = 0; u < kChunksPerWarp; ++u) {
        const uint32_t c0 = in_tile + u * kChunk;
        if (c0 >= t.valid) break;                           // warp-uniform
        const uint32_t j0 = c0 + lane * 4;
        const uint32_t mine_n = j0 >= t.valid ? 0u : (t.valid - j0 >= 4u ? 4u : t.valid - j0);
        uint32_t c4 = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const unsigned long long e = i * p.d_pad + e0 + u * kChunk;
            const Betas k = betas_of(p.betas, p.k, i);
            uint32_t nib = 0;
            for (uint32_t q = 0; q < mine_n; ++q) {
                const float g = load_grad1<BF16>(p.g, e + q);
                float m = load_state1<MB16>(p.m, e + q);
                nib |= lion_coord(g, m, k) << q;
                store_state1<MB16>(p.m, e + q, m);
            }
            c4 += spread_nibble(nib);
            if (p.packed != nullptr) {
                const uint32_t w = gather_word(nib, lane);
                if ((lane & 7u) == 0 && c0 + (lane >> 3) * 32 < t.valid) {
                    p.packed[i * w_stride + (t.base + c0) / 32 + (lane >> 3)] = w;
                }
            }
        }
        for (uint32_t q = 0; q < mine_n; ++q) {
            const unsigned long long e = e0 + u * kChunk + q;
            p.x[e] = apply_coord(p.x[e], delta_of<AVG>((c4 >> (8 * q)) & 0xFFu, thr, avg_table), p.lr, p.wd);
        }
    }
}

template <bool BF16, bool AVG, bool MB16>
__global__ void __launch_bounds__(kThreads, 2)
step_fused_kernel(const __grid_constant__ FusedParams p) {
    __shared__ float avg_table[256];
    const uint32_t n = p.n_workers;
    if constexpr (AVG) {
        for (uint32_t c = threadIdx.x; c <= n; c += kThreads) {
            const int sum = 2 * static_cast<int>(c) - static_cast<int>(n);
            // Averaging's quotient; or, for the three-valued tie rule, the sign of the sum with sign(0) = 0
            avg_table[c] = p.ternary ? (sum > 0 ? 1.0f : (sum < 0 ? -1.0f : 0.0f))
                                     : __fdiv_rn(static_cast<float>(sum), static_cast<float>(n));
        }
        __syncthreads();
    }
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t thr = (n + 1u) >> 1;
    const unsigned long long w_stride = p.d_pad / 32;

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        const uint32_t in_tile = warp * (kChunksPerWarp * kChunk);
        if (in_tile >= t.valid) continue;                          // warp-uniform
        const unsigned long long e0 = t.base + in_tile + lane * 4;  // my first coordinate (chunk 0)

        if (t.valid == kTile) {
            // ---- full tile: while worker i is consumed, worker i+1 is already in flight
            uint32_t cnt[kChunksPerWarp];
#pragma unroll
            for (int u = 0; u < kChunksPerWarp; ++u) cnt[u] = 0;
            float4 xv[kChunksPerWarp];
#pragma unroll
            for (int u = 0; u < kChunksPerWarp; ++u) {
                xv[u] = *(reinterpret_cast<const float4*>(p.x + e0 + u * kChunk));
            }
            uint32_t* wire = p.packed == nullptr ? nullptr : p.packed + (t.base + in_tile) / 32;
            WorkerRegs<BF16, MB16> a, b;
            a.load(p.g, p.m, e0);
            uint32_t i = 0;
            for (; i + 2 <= n; i += 2) {
                b.load(p.g, p.m, (i + 1) * p.d_pad + e0);
                consume<BF16, MB16>(p, a, i, i * p.d_pad + e0, wire == nullptr ? nullptr : wire + i * w_stride, lane, cnt);
                if (i + 2 < n) a.load(p.g, p.m, (i + 2) * p.d_pad + e0);
                consume<BF16, MB16>(p, b, i + 1, (i + 1) * p.d_pad + e0, wire == nullptr ? nullptr : wire + (i + 1) * w_stride,
                              lane, cnt);
            }
            if (i < n) consume<BF16, MB16>(p, a, i, i * p.d_pad + e0, wire == nullptr ? nullptr : wire + i * w_stride, lane, cnt);
#pragma unroll
            for (int u = 0; u < kChunksPerWarp; ++u) {
                float4 v = xv[u];
                v.x = apply_coord(v.x, delta_of<AVG>(cnt[u] & 0xFFu, thr, avg_table), p.lr, p.wd);
                v.y = apply_coord(v.y, delta_of<AVG>((cnt[u] >> 8) & 0xFFu, thr, avg_table), p.lr, p.wd);
                v.z = apply_coord(v.z, delta_of<AVG>((cnt[u] >> 16) & 0xFFu, thr, avg_table), p.lr, p.wd);
                v.w = apply_coord(v.w, delta_of<AVG>(cnt[u] >> 24, thr, avg_table), p.lr, p.wd);
                *reinterpret_cast<float4*>(p.x + e0 + u * kChunk) = v;
            }
        } else {
            ragged_tile<BF16, AVG, MB16>(p, t, in_tile, e0, lane, thr, avg_table);
        }
    }
}

template <bool BF16, bool MB16>
cudaError_t launch(const FusedParams& p, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    if (p.average) {
        step_fused_kernel<BF16, true, MB16><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    } else {
        step_fused_kernel<BF16, false, MB16><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_step_fused(const FusedParams& p, bool bf16, int sm_count, cudaStream_t s) {
    (void)sm_count;
    if (p.m_bf16) return bf16 ? launch<true, true>(p, s) : launch<false, true>(p, s);
    return bf16 ? launch<true, false>(p, s) : launch<false, false>(p, s);
}

}  // namespace dlion
