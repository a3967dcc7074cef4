// One whole iteration of Algorithm 1 (arXiv 2404.00438) in a single launch:
// worker side for all N workers, the vote, and x <- x - lr (Delta + lambda x)
// (Section 3.2).  A thread keeps the same 16 coordinates for every worker, so
// the vote never leaves its registers: four byte-wide counters per 32-bit
// register, one register per 128-coordinate chunk.  The 1-bit wire buffer is
// written only when the caller asks for it.
//
// Same tile and lane mapping as the worker-side kernel (warp = 512 consecutive
// coordinates, lane l of a chunk = coordinates 4l..4l+3).  HBM traffic per
// coordinate: N (G + 8) + 8 B, G = gradient bytes (+ N/8 B with the wire buffer):
// the 2 N/8 B round trip of the two-stage path is gone.
#include "dlion_common.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 256;
constexpr int kChunksPerWarp = 4;

__device__ __forceinline__ float delta_of(uint32_t count, uint32_t n, uint32_t thr, int average,
                                          const float* avg_table) {
    if (average) return avg_table[count];
    return count >= thr ? 1.0f : -1.0f;
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads)
step_fused_kernel(const FusedParams p) {
    __shared__ float avg_table[256];
    const uint32_t n = p.n_workers;
    if (p.average) {
        for (uint32_t c = threadIdx.x; c <= n; c += kThreads) {
            avg_table[c] = __fdiv_rn(static_cast<float>(2 * static_cast<int>(c) - static_cast<int>(n)),
                                     static_cast<float>(n));
        }
        __syncthreads();
    }
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t thr = (n + 1u) >> 1;
    const unsigned long long w_stride = p.d_pad / 32;

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.segs, p.nseg, tile);
        const uint32_t in_tile = warp * (kChunksPerWarp * kChunk);
        if (in_tile >= t.valid) continue;                          // warp-uniform
        const unsigned long long e0 = t.base + in_tile + lane * 4;  // my first coordinate (chunk 0)
        uint32_t cnt[kChunksPerWarp] = {0, 0, 0, 0};

        if (t.valid == kTile) {
            float4 xv[kChunksPerWarp];
#pragma unroll
            for (int u = 0; u < kChunksPerWarp; ++u) {
                xv[u] = __ldcs(reinterpret_cast<const float4*>(p.x + e0 + u * kChunk));
            }
#pragma unroll 2
            for (uint32_t i = 0; i < n; ++i) {
                const unsigned long long wb = i * p.d_pad + e0;
                float4 g[kChunksPerWarp], m[kChunksPerWarp];
#pragma unroll
                for (int u = 0; u < kChunksPerWarp; ++u) {
                    g[u] = load_grad4<BF16>(p.g, wb + u * kChunk);
                    m[u] = __ldcs(reinterpret_cast<const float4*>(p.m + wb + u * kChunk));
                }
                uint32_t mine = 0;
#pragma unroll
                for (int u = 0; u < kChunksPerWarp; ++u) {
                    uint32_t nib = lion_coord(g[u].x, m[u].x, p.k);
                    nib |= lion_coord(g[u].y, m[u].y, p.k) << 1;
                    nib |= lion_coord(g[u].z, m[u].z, p.k) << 2;
                    nib |= lion_coord(g[u].w, m[u].w, p.k) << 3;
                    __stcs(reinterpret_cast<float4*>(p.m + wb + u * kChunk), m[u]);
                    cnt[u] += spread_nibble(nib);
                    if (p.packed != nullptr) {
                        const uint32_t w = gather_word(nib, lane);
                        if ((lane & 7u) == static_cast<uint32_t>(u)) mine = w;
                    }
                }
                if (p.packed != nullptr && (lane & 7u) < kChunksPerWarp) {
                    p.packed[i * w_stride + (t.base + in_tile) / 32 + 4u * (lane & 7u) + (lane >> 3)] = mine;
                }
            }
#pragma unroll
            for (int u = 0; u < kChunksPerWarp; ++u) {
                float4 v = xv[u];
                v.x = apply_coord(v.x, delta_of(cnt[u] & 0xFFu, n, thr, p.average, avg_table), p.lr, p.wd);
                v.y = apply_coord(v.y, delta_of((cnt[u] >> 8) & 0xFFu, n, thr, p.average, avg_table), p.lr, p.wd);
                v.z = apply_coord(v.z, delta_of((cnt[u] >> 16) & 0xFFu, n, thr, p.average, avg_table), p.lr, p.wd);
                v.w = apply_coord(v.w, delta_of(cnt[u] >> 24, n, thr, p.average, avg_table), p.lr, p.wd);
                __stcs(reinterpret_cast<float4*>(p.x + e0 + u * kChunk), v);
            }
        } else {
            // last tile of a segment: guarded, one chunk at a time
#pragma unroll 1
            for (int u = 0; u < kChunksPerWarp; ++u) {
                const uint32_t c0 = in_tile + u * kChunk;
                if (c0 >= t.valid) break;                           // warp-uniform
                const uint32_t j0 = c0 + lane * 4;
                const uint32_t mine_n = j0 >= t.valid ? 0u : (t.valid - j0 >= 4u ? 4u : t.valid - j0);
                uint32_t c4 = 0;
                for (uint32_t i = 0; i < n; ++i) {
                    const unsigned long long e = i * p.d_pad + e0 + u * kChunk;
                    uint32_t nib = 0;
                    for (uint32_t q = 0; q < mine_n; ++q) {
                        const float g = load_grad1<BF16>(p.g, e + q);
                        float m = p.m[e + q];
                        nib |= lion_coord(g, m, p.k) << q;
                        p.m[e + q] = m;
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
                    p.x[e] = apply_coord(p.x[e], delta_of((c4 >> (8 * q)) & 0xFFu, n, thr, p.average, avg_table),
                                         p.lr, p.wd);
                }
            }
        }
    }
}

template <bool BF16>
cudaError_t launch(const FusedParams& p, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    step_fused_kernel<BF16><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_step_fused(const FusedParams& p, bool bf16, int sm_count, cudaStream_t s) {
    (void)sm_count;
    return bf16 ? launch<true>(p, s) : launch<false>(p, s);
}

}  // namespace dlion
