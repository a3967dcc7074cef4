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

template <int PLANES>
__device__ __forceinline__ void count_votes(uint32_t (&pl)[kMaxPlanes], const uint32_t* __restrict__ col,
                                            unsigned long long w_stride, uint32_t n, bool live) {
#pragma unroll
    for (int p = 0; p < kMaxPlanes; ++p) pl[p] = 0;
    uint32_t i = 0;
    if constexpr (PLANES >= 4) {
        for (; i + 8 <= n; i += 8) {
            uint32_t w[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) w[q] = live ? __ldg(col + (i + q) * w_stride) : 0u;
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
    }
    for (; i + 4 <= n; i += 4) {
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) w[q] = live ? __ldg(col + (i + q) * w_stride) : 0u;
#pragma unroll
        for (int q = 0; q < 4; ++q) ripple_add<PLANES, 0>(pl, w[q]);
    }
    for (; i < n; ++i) ripple_add<PLANES, 0>(pl, live ? __ldg(col + i * w_stride) : 0u);
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

template <int PLANES>
__global__ void __launch_bounds__(kThreads)
aggregate_apply_kernel(const AggParams p) {
    __shared__ float avg_table[256];      // Delta of Averaging for every count P
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
    const uint32_t thr = (n + 1u) >> 1;   // 2P >= N  <=>  P >= ceil(N/2)
    const bool need_counts = p.average || p.count != nullptr;

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.segs, p.nseg, tile);
        const uint32_t w0 = warp * kWarpSpan;                   // first coordinate of this warp
        if (w0 >= t.valid) continue;                            // warp-uniform
        const uint32_t my0 = w0 + lane * 32;                    // first coordinate of my word
        const uint32_t nbits = my0 >= t.valid ? 0u : (t.valid - my0 >= 32u ? 32u : t.valid - my0);
        const uint32_t vmask = nbits == 32u ? kFull : ((1u << nbits) - 1u);
        const unsigned long long word_idx = (t.base + my0) / 32;

        // issue the x loads of full chunks early; they do not depend on the votes
        const unsigned long long xe = t.base + w0 + lane * 4;
        float4 xv[8];
        const bool full_warp = w0 + kWarpSpan <= t.valid;
        if (full_warp) {
#pragma unroll
            for (int c = 0; c < 8; ++c) xv[c] = __ldcs(reinterpret_cast<const float4*>(p.x + xe + c * kChunk));
        }

        uint32_t pl[kMaxPlanes];
        count_votes<PLANES>(pl, p.packed + word_idx, p.w_stride, n, nbits != 0);
        const uint32_t dword = planes_ge<PLANES>(pl, thr) & vmask;
        if (p.delta_bits != nullptr && nbits != 0) p.delta_bits[word_idx] = dword;

#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t src = 4u * c + (lane >> 3);           // lane that owns my word
            const uint32_t sh = 4u * (lane & 7u);
            const uint32_t dn = (__shfl_sync(kFull, dword, src) >> sh) & 0xFu;
            uint32_t cnt4 = 0;                                   // four counts, one per byte
            if (need_counts) {
#pragma unroll
                for (int q = 0; q < PLANES; ++q) {
                    const uint32_t pn = (__shfl_sync(kFull, pl[q], src) >> sh) & 0xFu;
                    cnt4 += spread_nibble(pn) << q;
                }
            }
            const uint32_t j0 = w0 + c * kChunk + lane * 4;      // my first coordinate in the tile
            if (j0 >= t.valid) continue;                         // after the shuffles: all lanes took part
            float d[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                d[q] = p.average ? avg_table[(cnt4 >> (8 * q)) & 0xFFu]
                                 : (((dn >> q) & 1u) ? 1.0f : -1.0f);
            }
            const unsigned long long e = xe + c * kChunk;
            if (j0 + 4 <= t.valid) {
                float4 v = full_warp ? xv[c] : __ldcs(reinterpret_cast<const float4*>(p.x + e));
                v.x = apply_coord(v.x, d[0], p.lr, p.wd);
                v.y = apply_coord(v.y, d[1], p.lr, p.wd);
                v.z = apply_coord(v.z, d[2], p.lr, p.wd);
                v.w = apply_coord(v.w, d[3], p.lr, p.wd);
                __stcs(reinterpret_cast<float4*>(p.x + e), v);
                if (p.count != nullptr) *reinterpret_cast<uint32_t*>(p.count + e) = cnt4;
            } else {
                for (uint32_t q = 0; q < 4 && j0 + q < t.valid; ++q) {
                    p.x[e + q] = apply_coord(p.x[e + q], d[q], p.lr, p.wd);
                    if (p.count != nullptr) p.count[e + q] = static_cast<uint8_t>((cnt4 >> (8 * q)) & 0xFFu);
                }
            }
        }
    }
}

template <int PLANES>
cudaError_t launch(const AggParams& p, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    aggregate_apply_kernel<PLANES><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    return cudaGetLastError();
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
