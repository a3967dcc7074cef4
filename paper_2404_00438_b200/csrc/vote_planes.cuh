// Bit-plane vote counting shared by the server-side kernels: lane l of a warp owns
// one 32-coordinate word position; plane p holds bit p of the 32 vote counts.
#pragma once

#include "dlion_common.cuh"

namespace dlion {

constexpr uint32_t kWarpSpan = 1024;
constexpr int kMaxPlanes = 8;             // N <= 255

__device__ __forceinline__ void csa(uint32_t& sum, uint32_t& carry, uint32_t a, uint32_t b, uint32_t c) {
    sum = a ^ b ^ c;
    carry = (a & b) | (a & c) | (b & c);
}

// counts += w << P0 : add word w into planes P0.. (ripple, stops at PLANES)
template <int PLANES, int P0>
__device__ __forceinline__ void ripple_add(uint32_t (&pl)[kMaxPlanes], uint32_t w) {
#pragma unroll
    for (int p = P0; p < PLANES; ++p) {
        const uint32_t carry = pl[p] & w;
        pl[p] ^= w;
        w = carry;
    }
}

// counts += w[0] + ... + w[7] through a carry-save tree: 7 full adders, then the
// weight-8 carry ripples into the upper planes.
template <int PLANES>
__device__ __forceinline__ void add8(uint32_t (&pl)[kMaxPlanes], const uint32_t* w) {
    uint32_t t0, t1, t2, t3, f0, f1, e;
    csa(pl[0], t0, pl[0], w[0], w[1]);
    csa(pl[0], t1, pl[0], w[2], w[3]);
    csa(pl[1], f0, pl[1], t0, t1);
    csa(pl[0], t2, pl[0], w[4], w[5]);
    csa(pl[0], t3, pl[0], w[6], w[7]);
    csa(pl[1], f1, pl[1], t2, t3);
    csa(pl[2], e, pl[2], f0, f1);
    ripple_add<PLANES, 3>(pl, e);
}

// Adds the n workers' words of one word position (col, col + w_stride, ...).
// Whole groups of 16 workers (32 once N >= 64) are fetched with all their loads
// issued before the adders run; what is left (fewer than 16) goes in ONE more batch of 8 or 16 guarded
// loads, slots past the last worker adding zero.  So N <= 16 costs one round trip
// to memory and every further 16 workers one more.
// live = false reads nothing at all (the word position holds no parameter).
template <int PLANES>
__device__ __forceinline__ void count_votes(uint32_t (&pl)[kMaxPlanes], const uint32_t* __restrict__ col,
                                            unsigned long long w_stride, uint32_t n, bool live) {
#pragma unroll
    for (int p = 0; p < kMaxPlanes; ++p) pl[p] = 0;
    if (!live) return;
    uint32_t i = 0;
    if constexpr (PLANES >= 7) {
        // N >= 64: the votes outweigh x; 32 words per round trip (the kernel then
        // runs with a larger register budget and fewer blocks per SM)
        for (; i + 32 <= n; i += 32) {
            uint32_t w[32];
#pragma unroll
            for (int q = 0; q < 32; ++q) w[q] = __ldg(col + (i + q) * w_stride);
            add8<PLANES>(pl, w);
            add8<PLANES>(pl, w + 8);
            add8<PLANES>(pl, w + 16);
            add8<PLANES>(pl, w + 24);
        }
    }
    if constexpr (PLANES >= 5) {
        for (; i + 16 <= n; i += 16) {
            uint32_t w[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) w[q] = __ldg(col + (i + q) * w_stride);
            add8<PLANES>(pl, w);
            add8<PLANES>(pl, w + 8);
        }
    }
    const uint32_t rest = n - i;
    if (PLANES >= 4 && rest > 8) {
        uint32_t w[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) w[q] = (i + q < n) ? __ldg(col + (i + q) * w_stride) : 0u;
        add8<PLANES>(pl, w);
        add8<PLANES>(pl, w + 8);
    } else if (rest > 0) {
        uint32_t w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) w[q] = (i + q < n) ? __ldg(col + (i + q) * w_stride) : 0u;
        add8<PLANES>(pl, w);
    }
}

// Bit j set where count_j >= thr (bitwise magnitude comparison, MSB first).
template <int PLANES>
__device__ __forceinline__ uint32_t planes_ge(const uint32_t (&pl)[kMaxPlanes], uint32_t thr) {
    uint32_t gt = 0, eq = kFull;
#pragma unroll
    for (int p = PLANES - 1; p >= 0; --p) {
        const uint32_t tb = ((thr >> p) & 1u) ? kFull : 0u;
        gt |= eq & pl[p] & ~tb;
        eq &= ~(pl[p] ^ tb);
    }
    return gt | eq;
}

// Delta of my four coordinates in chunk c, and (when counts are needed) their
// four vote counts, one per byte.  All 32 lanes must call this together.
template <int PLANES, bool COUNTS>
__device__ __forceinline__ void my_votes(const uint32_t (&pl)[kMaxPlanes], uint32_t dword, int c, uint32_t lane,
                                         uint32_t& dn, uint32_t& cnt4) {
    const uint32_t src = 4u * c + (lane >> 3);           // lane that owns my word
    const uint32_t sh = 4u * (lane & 7u);
    dn = (__shfl_sync(kFull, dword, src) >> sh) & 0xFu;
    cnt4 = 0;
    if constexpr (COUNTS) {
#pragma unroll
        for (int q = 0; q < PLANES; ++q) {
            cnt4 += spread_nibble((__shfl_sync(kFull, pl[q], src) >> sh) & 0xFu) << q;
        }
    }
}

template <bool AVG>
__device__ __forceinline__ float delta_value(uint32_t dn, uint32_t cnt4, int q, const float* avg_table) {
    if constexpr (AVG) return avg_table[(cnt4 >> (8 * q)) & 0xFFu];
    return ((dn >> q) & 1u) ? 1.0f : -1.0f;
}

}  // namespace dlion
