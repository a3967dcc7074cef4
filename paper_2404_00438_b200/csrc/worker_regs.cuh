// One worker's gradients and momenta of a thread's 16 coordinates, as the one-launch
// kernels (the fused Distributed-Lion step and the Global-Lion comparison step) keep
// them in registers: warp = 512 consecutive coordinates as four 128-coordinate
// chunks, lane l of a chunk = coordinates 4l..4l+3.
#pragma once

#include "dlion_common.cuh"

namespace dlion {

constexpr int kChunksPerWarp = 4;

template <bool BF16>
struct RawGrad4 { float4 v; };            // four gradients as stored
template <>
struct RawGrad4<true> { uint2 v; };

template <bool BF16, bool MB16>
struct WorkerRegs {
    RawGrad4<BF16> g[kChunksPerWarp];
    float4 m[kChunksPerWarp];
    // at = arena index of this worker's copy of my first coordinate
    __device__ __forceinline__ void load(const void* grads, const void* mom, unsigned long long at) {
#pragma unroll
        for (int u = 0; u < kChunksPerWarp; ++u) {
            if constexpr (BF16) {
                g[u].v = *(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(grads) + at + u * kChunk));
            } else {
                g[u].v = *(reinterpret_cast<const float4*>(static_cast<const float*>(grads) + at + u * kChunk));
            }
            m[u] = load_state4<MB16>(mom, at + u * kChunk);
        }
    }
    __device__ __forceinline__ float4 grad(int u) const {
        if constexpr (BF16) {
            return make_float4(bf16_lo(g[u].v.x), bf16_hi(g[u].v.x), bf16_lo(g[u].v.y), bf16_hi(g[u].v.y));
        } else {
            return g[u].v;
        }
    }
};

}  // namespace dlion
