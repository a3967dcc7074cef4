// Bit-plane vote counting shared by the server-side kernels: lane l of a warp owns
// one 32-coordinate word position; plane p holds bit p of the 32 vote counts.
#pragma once

#include <type_traits>

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

// ---- from bit planes to per-coordinate counts -------------------------------
//
// The lane that owns a word holds its 32 vote counts as bit planes; the lanes that
// update x need them per coordinate.  The owner turns planes 0..7 into bytes with
// three rounds of word-wide delta swaps (an 8x8 bit-matrix transpose of each
// byte column: about 60 logic ops for all 32 coordinates, fewer when upper planes
// are known to be zero) and publishes them in shared memory; a consumer then needs
// one 16-byte load and one byte permute per coordinate.
//
// After the transpose, register c holds in byte k the count of coordinate 8k + c.

__device__ __forceinline__ void delta_swap(uint32_t& a, uint32_t& b, uint32_t mask, int s) {
    const uint32_t t = ((a >> s) ^ b) & mask;      // a's upper field <-> b's lower field
    b ^= t;
    a ^= t << s;
}

template <int PLANES, int P0>
__device__ __forceinline__ void planes_to_bytes(const uint32_t (&pl)[kMaxPlanes], uint32_t (&r)[8]) {
#pragma unroll
    for (int p = 0; p < 8; ++p) r[p] = (P0 + p < PLANES) ? pl[P0 + p] : 0u;
#pragma unroll
    for (int p = 0; p < 4; ++p) delta_swap(r[p], r[p + 4], 0x0F0F0F0Fu, 4);
#pragma unroll
    for (int p = 0; p < 8; ++p) {
        if ((p & 2) == 0) delta_swap(r[p], r[p + 2], 0x33333333u, 2);
    }
#pragma unroll
    for (int p = 0; p < 8; p += 2) delta_swap(r[p], r[p + 1], 0x55555555u, 1);
}

// One warp's hand-off area.  half[h][o] = registers 4h..4h+3 of owner lane o; the
// spare 33rd slot shifts the second half by four banks, so the two halves a
// quarter-warp reads together never collide.
struct CountSlots {
    uint4 half[2][33];
};

template <bool WIDE>
struct CountArea {                                  // N > 255: bits 8..15 of every count too
    CountSlots lo, hi;
};
template <>
struct CountArea<false> {
    CountSlots lo;
};

// Owner side: all 32 lanes call this together, once per tile, after the vote.
template <int PLANES>
__device__ __forceinline__ void publish_counts(const uint32_t (&pl)[kMaxPlanes], CountArea<(PLANES > 8)>* area,
                                               uint32_t lane) {
    __syncwarp();                                   // the previous tile's readers are done
    uint32_t r[8];
    planes_to_bytes<PLANES, 0>(pl, r);
    area->lo.half[0][lane] = make_uint4(r[0], r[1], r[2], r[3]);
    area->lo.half[1][lane] = make_uint4(r[4], r[5], r[6], r[7]);
    if constexpr (PLANES > 8) {
        planes_to_bytes<PLANES, 8>(pl, r);
        area->hi.half[0][lane] = make_uint4(r[0], r[1], r[2], r[3]);
        area->hi.half[1][lane] = make_uint4(r[4], r[5], r[6], r[7]);
    }
    __syncwarp();
}

// Consumer side: the vote counts of my four coordinates in chunk c (coordinates
// 128c + 4*lane .. +3 of the warp's 1024): they sit in word 4c + lane/8, at in-word
// positions 4*(lane%8) + q, i.e. registers 4*(lane%2) + q, byte (lane%8)/2.
struct Counts4 {
    uint32_t c[4];
};

template <int PLANES>
__device__ __forceinline__ Counts4 my_counts(const CountArea<(PLANES > 8)>* area, int c, uint32_t lane) {
    const uint32_t owner = 4u * c + (lane >> 3);
    const uint32_t sel = 0x4440u | ((lane & 7u) >> 1);            // byte k of the first operand, then zeros
    const uint4 v = area->lo.half[lane & 1u][owner];
    Counts4 k;
    k.c[0] = __byte_perm(v.x, 0u, sel);
    k.c[1] = __byte_perm(v.y, 0u, sel);
    k.c[2] = __byte_perm(v.z, 0u, sel);
    k.c[3] = __byte_perm(v.w, 0u, sel);
    if constexpr (PLANES > 8) {
        const uint4 h = area->hi.half[lane & 1u][owner];
        k.c[0] |= __byte_perm(h.x, 0u, sel) << 8;
        k.c[1] |= __byte_perm(h.y, 0u, sel) << 8;
        k.c[2] |= __byte_perm(h.z, 0u, sel) << 8;
        k.c[3] |= __byte_perm(h.w, 0u, sel) << 8;
    }
    return k;
}

// The Delta bits of my four coordinates in chunk c, from the owner's Delta word
// (Majority Vote when no counts are needed).  All 32 lanes must call this together.
__device__ __forceinline__ uint32_t my_delta_bits(uint32_t dword, int c, uint32_t lane) {
    return (__shfl_sync(kFull, dword, 4u * c + (lane >> 3)) >> (4u * (lane & 7u))) & 0xFu;
}

// Delta as a function of the vote count P where it is tabulated or computed from P:
// Averaging's correctly rounded quotient (2P - N) / N, or -- the optional three-valued
// tie rule, which runs on the Averaging kernels with this other table -- the sign of
// 2P - N with sign(0) = 0.
__device__ __forceinline__ float delta_value(uint32_t count, uint32_t n, bool ternary) {
    const int s = 2 * static_cast<int>(count) - static_cast<int>(n);
    if (ternary) return s > 0 ? 1.0f : (s < 0 ? -1.0f : 0.0f);
    return __fdiv_rn(static_cast<float>(s), static_cast<float>(n));
}

// Delta of a coordinate from its vote count P.  Majority Vote: +1 iff P >= ceil(N/2).
// Averaging (and the three-valued tie rule): from the per-warp table while the counts fit
// it (N <= 255), else computed directly.
template <int PLANES, bool AVG>
__device__ __forceinline__ float delta_of_count(uint32_t count, uint32_t thr, const float* avg_table, uint32_t n,
                                                bool ternary) {
    if constexpr (AVG) {
        if constexpr (PLANES <= 8) return avg_table[count];
        return delta_value(count, n, ternary);
    }
    return count >= thr ? 1.0f : -1.0f;
}

// Fills a warp's private table of Averaging's Delta for every count (N <= 255 only).
template <int PLANES>
__device__ __forceinline__ void fill_avg_table(float* avg_table, uint32_t n, uint32_t lane, bool ternary) {
    if constexpr (PLANES <= 8) {
        for (uint32_t c = lane; c <= n; c += 32) {
            avg_table[c] = delta_value(c, n, ternary);
        }
        __syncwarp();
    }
}

// Plane capacities the kernels are compiled for: the exact plane count up to 8
// (N <= 255, where the count matters for speed), then 12 and 16.  A capacity
// above the needed count only adds zero planes.  coarse = true (the per-tensor
// variants, to keep their number down): capacities 4, 8 and 16 only.
template <typename F>
inline cudaError_t dispatch_planes(uint32_t n_workers, bool coarse, F&& f) {
    const uint32_t need = planes_for(n_workers);
    if (coarse) {
        if (need <= 4) return f(std::integral_constant<int, 4>{}, std::true_type{});
        if (need <= 8) return f(std::integral_constant<int, 8>{}, std::true_type{});
        return f(std::integral_constant<int, 16>{}, std::true_type{});
    }
    switch (need) {
        case 1: return f(std::integral_constant<int, 1>{}, std::false_type{});
        case 2: return f(std::integral_constant<int, 2>{}, std::false_type{});
        case 3: return f(std::integral_constant<int, 3>{}, std::false_type{});
        case 4: return f(std::integral_constant<int, 4>{}, std::false_type{});
        case 5: return f(std::integral_constant<int, 5>{}, std::false_type{});
        case 6: return f(std::integral_constant<int, 6>{}, std::false_type{});
        case 7: return f(std::integral_constant<int, 7>{}, std::false_type{});
        case 8: return f(std::integral_constant<int, 8>{}, std::false_type{});
        case 9: case 10: case 11: case 12: return f(std::integral_constant<int, 12>{}, std::false_type{});
        default: return f(std::integral_constant<int, 16>{}, std::false_type{});
    }
}

// The base of x for a tile: the arena, or (TABLE) tensor t.tensor's storage through the
// per-tensor offset table.
template <bool TABLE>
__device__ __forceinline__ float* x_base(float* x, const long long* x_off, const TileRef& t) {
    if constexpr (TABLE) return reinterpret_cast<float*>(reinterpret_cast<char*>(x) + x_off[t.tensor]);
    return x;
}

}  // namespace dlion
