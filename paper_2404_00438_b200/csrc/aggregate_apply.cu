// Server side of Algorithm 1 fused with the parameter update of Section 3.2
// (arXiv 2404.00438): per coordinate j,
//     P = #{ i : delta_i[j] = +1 },  S = 2P - N
//     Delta = sign(S)   (Majority Vote; S = 0 counts as +1)
//     Delta = S / N     (Averaging)
//     x[j] <- x[j] - lr (Delta + lambda x[j])
//
// The votes are counted without ever unpacking them: lane l of a warp owns one
// 32-coordinate word position and adds the N workers' words into bit-plane
// counters (plane p holds bit p of all 32 counts).  Groups of eight words go
// through a carry-save adder tree (7 full adders of two 3-input logic ops each),
// so the cost is about 3 logic ops per word and stays far below the memory time
// even at N = 128.  Majority Vote then needs one bitwise comparison of the planes
// with ceil(N/2), which yields the Delta word directly.  For the update the warp
// walks its 1024 coordinates in eight 128-coordinate chunks (lane l: coordinates
// 4l..4l+3, one 16-byte access) and fetches the needed plane bits from the owning
// lane with a shuffle.
//
// HBM traffic per coordinate: N/8 B of votes + 4 B read + 4 B write of x
// (+ 1/8 B Delta bits, + 1 B count when requested).
#include "dlion_common.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 128;             // 4 warps x 1024 coordinates = one tile
constexpr int kMinBlocks = 6;             // register budget: 6 blocks (24 warps) per SM
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
// Whole groups of 16 workers are fetched with 16 loads issued before the adders
// run; what is left (fewer than 16) goes in ONE more batch of 8 or 16 guarded
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

// Last tile of a segment: every access guarded against the segment's end.
template <int PLANES, bool AVG, bool COUNTS>
__device__ __noinline__ void ragged_tile(const AggParams& p, const TileRef t, uint32_t warp, uint32_t lane,
                                         uint32_t thr, const float* avg_table) {
    const uint32_t w0 = warp * kWarpSpan;
    if (w0 >= t.valid) return;                                  // warp-uniform
    const uint32_t my0 = w0 + lane * 32;                        // first coordinate of my word
    const uint32_t nbits = my0 >= t.valid ? 0u : (t.valid - my0 >= 32u ? 32u : t.valid - my0);
    const uint32_t vmask = nbits == 32u ? kFull : ((1u << nbits) - 1u);
    const unsigned long long word_idx = (t.base + my0) / 32;
    uint32_t pl[kMaxPlanes];
    count_votes<PLANES>(pl, p.packed + word_idx, p.w_stride, p.n_workers, nbits != 0);
    const uint32_t dword = planes_ge<PLANES>(pl, thr) & vmask;
    if (p.delta_bits != nullptr && nbits != 0) p.delta_bits[word_idx] = dword;
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        uint32_t dn, cnt4;
        my_votes<PLANES, COUNTS>(pl, dword, c, lane, dn, cnt4);
        const uint32_t j0 = w0 + c * kChunk + lane * 4;
        const unsigned long long e = t.base + j0;
        for (uint32_t q = 0; q < 4 && j0 + q < t.valid; ++q) {
            p.x[e + q] = apply_coord(p.x[e + q], delta_value<AVG>(dn, cnt4, q, avg_table), p.lr, p.wd);
            if (p.count != nullptr) p.count[e + q] = static_cast<uint8_t>((cnt4 >> (8 * q)) & 0xFFu);
        }
    }
}

// AVG: Averaging (else Majority Vote).  COUNTS: per-coordinate counts are needed
// (Averaging, or count_out requested).
template <int PLANES, bool AVG, bool COUNTS>
__global__ void __launch_bounds__(kThreads, kMinBlocks)
aggregate_apply_kernel(const __grid_constant__ AggParams p) {
    // Delta of Averaging for every count P, one private copy per warp: it is
    // filled after the tile's first loads are in flight and needs no block barrier.
    __shared__ float avg_tables[AVG ? kThreads / 32 : 1][AVG ? 256 : 1];
    const uint32_t n = p.n_workers;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t thr = (n + 1u) >> 1;   // 2P >= N  <=>  P >= ceil(N/2)
    float* avg_table = avg_tables[AVG ? warp : 0];
    bool have_table = !AVG;
    auto fill_table = [&]() {
        for (uint32_t c = lane; c <= n; c += 32) {
            avg_table[c] = __fdiv_rn(static_cast<float>(2 * static_cast<int>(c) - static_cast<int>(n)),
                                     static_cast<float>(n));
        }
        __syncwarp();
        have_table = true;
    };

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.segs, p.nseg, tile);
        if (t.valid != kTile) {
            if (!have_table) fill_table();
            ragged_tile<PLANES, AVG, COUNTS>(p, t, warp, lane, thr, avg_table);
            continue;
        }
        // ---- full tile: x loads first (they do not depend on the votes), then
        // ---- the votes, all in flight together
        const unsigned long long xe = t.base + warp * kWarpSpan + lane * 4;
        const unsigned long long word_idx = (t.base + warp * kWarpSpan) / 32 + lane;
        float4 xv[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) xv[c] = __ldcs(reinterpret_cast<const float4*>(p.x + xe + c * kChunk));
        if (!have_table) fill_table();
        uint32_t pl[kMaxPlanes];
        count_votes<PLANES>(pl, p.packed + word_idx, p.w_stride, n, true);
        const uint32_t dword = planes_ge<PLANES>(pl, thr);
        if (p.delta_bits != nullptr) p.delta_bits[word_idx] = dword;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            uint32_t dn, cnt4;
            my_votes<PLANES, COUNTS>(pl, dword, c, lane, dn, cnt4);
            float4 v = xv[c];
            v.x = apply_coord(v.x, delta_value<AVG>(dn, cnt4, 0, avg_table), p.lr, p.wd);
            v.y = apply_coord(v.y, delta_value<AVG>(dn, cnt4, 1, avg_table), p.lr, p.wd);
            v.z = apply_coord(v.z, delta_value<AVG>(dn, cnt4, 2, avg_table), p.lr, p.wd);
            v.w = apply_coord(v.w, delta_value<AVG>(dn, cnt4, 3, avg_table), p.lr, p.wd);
            __stcs(reinterpret_cast<float4*>(p.x + xe + c * kChunk), v);
            if constexpr (COUNTS) {
                if (p.count != nullptr) *reinterpret_cast<uint32_t*>(p.count + xe + c * kChunk) = cnt4;
            }
        }
    }
}

template <int PLANES, bool AVG, bool COUNTS>
cudaError_t launch3(const AggParams& p, cudaStream_t s) {
    aggregate_apply_kernel<PLANES, AVG, COUNTS><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <int PLANES>
cudaError_t launch(const AggParams& p, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    if (p.average) return launch3<PLANES, true, true>(p, s);
    if (p.count != nullptr) return launch3<PLANES, false, true>(p, s);
    return launch3<PLANES, false, false>(p, s);
}

}  // namespace

cudaError_t launch_aggregate_apply(const AggParams& p, int sm_count, cudaStream_t s) {
    (void)sm_count;
    const uint32_t n = p.n_workers;       // planes = bit length of N
    if (n < 2) return launch<1>(p, s);
    if (n < 4) return launch<2>(p, s);
    if (n < 8) return launch<3>(p, s);
    if (n < 16) return launch<4>(p, s);
    if (n < 32) return launch<5>(p, s);
    if (n < 64) return launch<6>(p, s);
    if (n < 128) return launch<7>(p, s);
    return launch<8>(p, s);
}

}  // namespace dlion
