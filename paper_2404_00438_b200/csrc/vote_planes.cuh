// Bit-plane vote counting shared by the server-side kernels: lane l of a warp owns
// one 32-coordinate word position; plane p holds bit p of the 32 vote counts.
#pragma once

#include "dlion_common.cuh"

namespace dlion {

constexpr uint32_t kWarpSpan = 1024;
constexpr int kMaxPlanes = 16;            // N <= 65535

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

// Votes of my four coordinates in chunk c: the Delta bits (dn, bit q = coordinate q)
// and, when counts are needed, the four vote counts.  Up to 8 planes the counts are
// packed one per byte in lo; beyond (N > 255) two 16-bit counts each in lo and hi.
struct Votes4 {
    uint32_t dn, lo, hi;
};

// All 32 lanes must call this together.
template <int PLANES, bool COUNTS>
__device__ __forceinline__ Votes4 my_votes(const uint32_t (&pl)[kMaxPlanes], uint32_t dword, int c, uint32_t lane) {
    const uint32_t src = 4u * c + (lane >> 3);           // lane that owns my word
    const uint32_t sh = 4u * (lane & 7u);
    Votes4 v;
    v.dn = (__shfl_sync(kFull, dword, src) >> sh) & 0xFu;
    v.lo = 0;
    v.hi = 0;
    if constexpr (COUNTS) {
#pragma unroll
        for (int q = 0; q < PLANES; ++q) {
            const uint32_t nib = (__shfl_sync(kFull, pl[q], src) >> sh) & 0xFu;
            if constexpr (PLANES <= 8) {
                v.lo += spread_nibble(nib) << q;
            } else {
                v.lo += ((nib & 1u) | ((nib & 2u) << 15)) << q;
                v.hi += (((nib >> 2) & 1u) | ((nib & 8u) << 13)) << q;
            }
        }
    }
    return v;
}

template <int PLANES>
__device__ __forceinline__ uint32_t count_of(const Votes4& v, int q) {
    if constexpr (PLANES <= 8) return (v.lo >> (8 * q)) & 0xFFu;
    return ((q < 2 ? v.lo : v.hi) >> (16 * (q & 1))) & 0xFFFFu;
}

// Delta of coordinate q.  Averaging: from the per-warp table while the counts fit
// it (N <= 255), else the correctly rounded quotient directly.
template <int PLANES, bool AVG>
__device__ __forceinline__ float delta_value(const Votes4& v, int q, const float* avg_table, uint32_t n) {
    if constexpr (AVG) {
        const uint32_t c = count_of<PLANES>(v, q);
        if constexpr (PLANES <= 8) return avg_table[c];
        return __fdiv_rn(static_cast<float>(2 * static_cast<int>(c) - static_cast<int>(n)), static_cast<float>(n));
    }
    return ((v.dn >> q) & 1u) ? 1.0f : -1.0f;
}

// Fills a warp's private table of Averaging's Delta for every count (N <= 255 only).
template <int PLANES>
__device__ __forceinline__ void fill_avg_table(float* avg_table, uint32_t n, uint32_t lane) {
    if constexpr (PLANES <= 8) {
        for (uint32_t c = lane; c <= n; c += 32) {
            avg_table[c] = __fdiv_rn(static_cast<float>(2 * static_cast<int>(c) - static_cast<int>(n)),
                                     static_cast<float>(n));
        }
        __syncwarp();
    }
}

}  // namespace dlion
