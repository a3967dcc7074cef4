// The two halves of the server round trip of Algorithm 1 (arXiv 2404.00438) as
// separate kernels, for deployments where the vote and the update run in
// different places:
//
//   aggregate_kernel    server side: from the N binary vectors, the message that
//                       is broadcast.  Majority Vote: d bits (bit = 1 iff
//                       Delta = +1).  Averaging: the integer P in {0..N} per
//                       coordinate (Section 3.2, "Communication Cost") as
//                       K = ceil(log2(N+1)) bit planes of d bits each, plane p
//                       holding bit p of every P -- exactly the K*d bits of
//                       Table 1, and exactly the counters the vote already keeps.
//   apply_delta_kernel  worker side, first line of the loop body of Algorithm 1:
//                       x <- x - eps (Delta + lambda x), Delta decoded from that
//                       message.
//
// Run one after the other they give what aggregate_apply_kernel gives in one pass.
// Traffic per coordinate: aggregate N/8 + K/8 B; apply 8 + K/8 B.
#include "vote_planes.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 128;             // 4 warps x 1024 coordinates = one tile
constexpr int kWarps = kThreads / 32;

// TERNARY (Majority Vote only): the three-valued tie rule's two-plane message.  A template
// parameter: as a run-time test it cost the plain Majority-Vote vote 3 %.
template <int PLANES, bool AVG, bool TERNARY>
__device__ __forceinline__ void aggregate_body(const WireParams& p) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t thr = (p.n_workers + 1u) >> 1;
    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        const uint32_t my0 = warp * kWarpSpan + lane * 32;          // first coordinate of my word
        if (my0 >= t.valid) continue;                               // my word holds no parameter
        const uint32_t nbits = t.valid - my0 >= 32u ? 32u : t.valid - my0;
        const uint32_t vmask = nbits == 32u ? kFull : ((1u << nbits) - 1u);
        const unsigned long long word_idx = (t.base + my0) / 32;
        uint32_t pl[kMaxPlanes];
        count_votes<PLANES>(pl, p.packed + word_idx, p.w_stride, p.n_workers, true);
        if constexpr (AVG) {
#pragma unroll
            for (int q = 0; q < PLANES; ++q) {
                if (q < static_cast<int>(p.kplanes)) p.wire_out[q * p.plane_stride + word_idx] = pl[q] & vmask;
            }
        } else if constexpr (TERNARY) {
            // the three-valued rule: Delta + 1 in {0, 1, 2} as two planes (bit 0 = tie, bit 1 = S > 0)
            const uint32_t ge = planes_ge<PLANES>(pl, thr);
            const uint32_t tie = (p.n_workers & 1u) ? 0u : (ge & ~planes_ge<PLANES>(pl, thr + 1u));
            p.wire_out[word_idx] = tie & vmask;
            p.wire_out[p.plane_stride + word_idx] = ge & ~tie & vmask;
        } else {
            p.wire_out[word_idx] = planes_ge<PLANES>(pl, thr) & vmask;
        }
    }
}

// Blocks per SM, measured on the 1.3 B-parameter workload (N = 16, vote + apply pair):
// Averaging 2.41 ms as the compiler allocates unprompted -> 2.25 ms with 10 blocks here and
// 7 in the apply kernel; Majority Vote is fastest unprompted (34 registers, 12 blocks), and
// N >= 64 was not re-measured: both keep the compiler's own allocation.
template <int PLANES, bool AVG, bool TERNARY>
__global__ void __launch_bounds__(kThreads)
aggregate_kernel(const __grid_constant__ WireParams p) {
    aggregate_body<PLANES, AVG, TERNARY>(p);
}

template <int PLANES>
__global__ void __launch_bounds__(kThreads, 10)
aggregate_kernel_averaging(const __grid_constant__ WireParams p) {
    aggregate_body<PLANES, true, false>(p);
}

template <int PLANES, bool AVG, bool TABLE>
__global__ void __launch_bounds__(kThreads, AVG ? 7 : 6)
apply_delta_kernel(const __grid_constant__ WireParams p) {
    __shared__ float avg_tables[(AVG && PLANES <= 8) ? kWarps : 1][(AVG && PLANES <= 8) ? 256 : 1];
    __shared__ CountArea<(PLANES > 8)> areas[AVG ? kWarps : 1];
    const uint32_t n = p.n_workers;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    float* avg_table = avg_tables[(AVG && PLANES <= 8) ? warp : 0];
    CountArea<(PLANES > 8)>* area = &areas[AVG ? warp : 0];
    bool have_table = !AVG;

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        const uint32_t w0 = warp * kWarpSpan;
        if (w0 >= t.valid) continue;                                // warp-uniform
        const bool full = w0 + kWarpSpan <= t.valid;
        const unsigned long long xe = t.base + w0 + lane * 4;
        const unsigned long long word_idx = (t.base + w0) / 32 + lane;
        const bool live = w0 + lane * 32 < t.valid;                 // my word holds a parameter

        float* const xs = x_base<TABLE>(p.x, p.x_off, t);   // one arena, or tensor t.tensor's storage
        float4 xv[8];
        if (full) {
#pragma unroll
            for (int c = 0; c < 8; ++c) xv[c] = *(reinterpret_cast<const float4*>(xs + xe + c * kChunk));
        }
        // where my word of plane 0 sits: planes contiguous over all coordinates, or the
        // all-gather order [slice][plane][slice_words] (plane_stride = slice_words then)
        unsigned long long at = word_idx;
        if (p.slice_words != 0) {
            const unsigned long long r = word_idx / p.slice_words;
            at = r * p.slice_words * p.kplanes + (word_idx - r * p.slice_words);
        }
        uint32_t dword = 0;
        if constexpr (AVG) {
            uint32_t pl[kMaxPlanes];
#pragma unroll
            for (int q = 0; q < kMaxPlanes; ++q) {
                pl[q] = (q < PLANES && q < static_cast<int>(p.kplanes) && live)
                            ? __ldg(p.wire_in + q * p.plane_stride + at) : 0u;
            }
            if (!have_table) {
                fill_avg_table<PLANES>(avg_table, n, lane, false);
                have_table = true;
            }
            publish_counts<PLANES>(pl, area, lane);
        } else {
            dword = live ? __ldg(p.wire_in + at) : 0u;
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float d[4];
            if constexpr (AVG) {
                const Counts4 k = my_counts<PLANES>(area, c, lane);
#pragma unroll
                for (int q = 0; q < 4; ++q) d[q] = delta_of_count<PLANES, true>(k.c[q], 0u, avg_table, n, false);
            } else {
                const uint32_t dn = my_delta_bits(dword, c, lane);
#pragma unroll
                for (int q = 0; q < 4; ++q) d[q] = ((dn >> q) & 1u) ? 1.0f : -1.0f;
            }
            const uint32_t j0 = w0 + c * kChunk + lane * 4;
            if (j0 >= t.valid) continue;                            // after the shuffles: all lanes took part
            const unsigned long long e = xe + c * kChunk;
            if (full) {
                float4 v = xv[c];
                v.x = apply_coord(v.x, d[0], p.lr, p.wd);
                v.y = apply_coord(v.y, d[1], p.lr, p.wd);
                v.z = apply_coord(v.z, d[2], p.lr, p.wd);
                v.w = apply_coord(v.w, d[3], p.lr, p.wd);
                *reinterpret_cast<float4*>(xs + e) = v;
            } else {
                for (uint32_t q = 0; q < 4 && j0 + q < t.valid; ++q) {
                    xs[e + q] = apply_coord(xs[e + q], d[q], p.lr, p.wd);
                }
            }
        }
    }
}

template <int PLANES, bool TABLE>
cudaError_t launch(const WireParams& p, bool apply, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    const unsigned grid = grid_for(p.ntiles);
    if (apply) {
        if (p.average) apply_delta_kernel<PLANES, true, TABLE><<<grid, kThreads, 0, s>>>(p);
        else apply_delta_kernel<1, false, TABLE><<<grid, kThreads, 0, s>>>(p);
    } else if constexpr (!TABLE) {                       // the vote touches no parameter tensor
        if (p.ternary) aggregate_kernel<PLANES, false, true><<<grid, kThreads, 0, s>>>(p);
        else if (!p.average) aggregate_kernel<PLANES, false, false><<<grid, kThreads, 0, s>>>(p);
        else if constexpr (PLANES < 7) aggregate_kernel_averaging<PLANES><<<grid, kThreads, 0, s>>>(p);
        else aggregate_kernel<PLANES, true, false><<<grid, kThreads, 0, s>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace

uint32_t planes_for(uint32_t n_workers) {      // bit length of N = ceil(log2(N+1))
    uint32_t k = 0;
    while ((1u << k) < n_workers + 1u) ++k;
    return k;
}

cudaError_t launch_wire(const WireParams& p, bool apply, cudaStream_t s) {
    return dispatch_planes(p.n_workers, apply && p.x_off != nullptr, [&](auto planes, auto table) {
        return launch<decltype(planes)::value, decltype(table)::value>(p, apply, s);
    });
}

}  // namespace dlion
