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
// 4l..4l+3, one 16-byte access).  Majority Vote fetches its four Delta bits from
// the owning lane with one shuffle per chunk.  Averaging needs the counts
// themselves: the owning lane transposes its planes into one byte per coordinate
// (word-wide delta swaps) and hands them over through shared memory, so a
// consumer pays one 16-byte shared load per chunk and one byte permute plus one
// table lookup per coordinate.
//
// HBM traffic per coordinate: N/8 B of votes + 4 B read + 4 B write of x
// (+ 1/8 B Delta bits, + 1 B count when requested).
#include "vote_planes.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 128;             // 4 warps x 1024 coordinates = one tile
constexpr int kWarps = kThreads / 32;
// Blocks per SM (register budget), measured: 7 up to N = 63 (Averaging at N = 16 on the
// 1.3 B-parameter workload: 1.96 ms at 6 blocks, 1.89 ms at 7, 2.02 ms at 8, which
// spills); 5 once N >= 64, where 32 vote words are fetched per round trip (flat 100 M
// vector, Averaging, N = 64 / 128: 5.9 / 6.15 TB/s at 4 blocks, 6.5 / 6.6 at 5, 6.2 at 6).
constexpr int kMinBlocks = 7;
constexpr int kMinBlocksManyWorkers = 5;

__device__ __forceinline__ uint32_t pack_counts(const Counts4& k) {          // N <= 255: one byte each
    return k.c[0] | (k.c[1] << 8) | (k.c[2] << 16) | (k.c[3] << 24);
}

// Last tile of a segment: every access guarded against the segment's end.
template <int PLANES, bool AVG, bool COUNTS, bool TABLE>
__device__ __noinline__ void ragged_tile(const AggParams& p, const TileRef t, uint32_t warp, uint32_t lane,
                                         uint32_t thr, const float* avg_table, CountArea<(PLANES > 8)>* area) {
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
    if constexpr (COUNTS) publish_counts<PLANES>(pl, area, lane);
    float* const xs = x_base<TABLE>(p.x, p.x_off, t);
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        Counts4 k;
        uint32_t dn = 0;
        if constexpr (COUNTS) k = my_counts<PLANES>(area, c, lane);
        else dn = my_delta_bits(dword, c, lane);
        const uint32_t j0 = w0 + c * kChunk + lane * 4;
        const unsigned long long e = t.base + j0;
        for (uint32_t q = 0; q < 4 && j0 + q < t.valid; ++q) {
            float delta;
            if constexpr (COUNTS) delta = delta_of_count<PLANES, AVG>(k.c[q], thr, avg_table, p.n_workers, p.ternary != 0);
            else delta = ((dn >> q) & 1u) ? 1.0f : -1.0f;
            xs[e + q] = apply_coord(xs[e + q], delta, p.lr, p.wd);
            if constexpr (COUNTS) {
                if (p.count != nullptr) p.count[e + q] = static_cast<uint8_t>(k.c[q]);
                if (p.count16 != nullptr) p.count16[e + q] = static_cast<uint16_t>(k.c[q]);
            }
        }
    }
}

// AVG: Averaging (else Majority Vote).  COUNTS: per-coordinate counts are needed
// (Averaging, or count_out requested).  TABLE: x is a list of separate tensors (a
// template parameter, not a run-time test: with the test compiled in, the Averaging
// kernel measured 7 % slower in arena mode too).
template <int PLANES, bool AVG, bool COUNTS, bool TABLE>
__global__ void __launch_bounds__(kThreads, PLANES >= 7 ? kMinBlocksManyWorkers : kMinBlocks)
aggregate_apply_kernel(const __grid_constant__ AggParams p) {
    // Delta of Averaging for every count P, one private copy per warp: it is
    // filled after the tile's first loads are in flight and needs no block barrier.
    __shared__ float avg_tables[(AVG && PLANES <= 8) ? kWarps : 1][(AVG && PLANES <= 8) ? 256 : 1];
    __shared__ CountArea<(PLANES > 8)> areas[COUNTS ? kWarps : 1];
    const uint32_t n = p.n_workers;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t thr = (n + 1u) >> 1;   // 2P >= N  <=>  P >= ceil(N/2)
    float* avg_table = avg_tables[(AVG && PLANES <= 8) ? warp : 0];
    CountArea<(PLANES > 8)>* area = &areas[COUNTS ? warp : 0];
    bool have_table = !AVG;
    auto fill_table = [&]() {
        fill_avg_table<PLANES>(avg_table, n, lane, p.ternary != 0);
        have_table = true;
    };

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        if (t.valid != kTile) {
            if (!have_table) fill_table();
            ragged_tile<PLANES, AVG, COUNTS, TABLE>(p, t, warp, lane, thr, avg_table, area);
            continue;
        }
        // ---- full tile: x loads first (they do not depend on the votes), then
        // ---- the votes, all in flight together
        const unsigned long long xe = t.base + warp * kWarpSpan + lane * 4;
        const unsigned long long word_idx = (t.base + warp * kWarpSpan) / 32 + lane;
        float* const xs = x_base<TABLE>(p.x, p.x_off, t);   // separate tensors, or one arena
        float4 xv[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) xv[c] = *(reinterpret_cast<const float4*>(xs + xe + c * kChunk));
        if (!have_table) fill_table();
        uint32_t pl[kMaxPlanes];
        count_votes<PLANES>(pl, p.packed + word_idx, p.w_stride, n, true);
        uint32_t dword = 0;
        if (!COUNTS || p.delta_bits != nullptr) dword = planes_ge<PLANES>(pl, thr);
        if (p.delta_bits != nullptr) p.delta_bits[word_idx] = dword;
        if constexpr (COUNTS) publish_counts<PLANES>(pl, area, lane);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float d0, d1, d2, d3;
            if constexpr (COUNTS) {
                const Counts4 k = my_counts<PLANES>(area, c, lane);
                d0 = delta_of_count<PLANES, AVG>(k.c[0], thr, avg_table, n, p.ternary != 0);
                d1 = delta_of_count<PLANES, AVG>(k.c[1], thr, avg_table, n, p.ternary != 0);
                d2 = delta_of_count<PLANES, AVG>(k.c[2], thr, avg_table, n, p.ternary != 0);
                d3 = delta_of_count<PLANES, AVG>(k.c[3], thr, avg_table, n, p.ternary != 0);
                if (p.count != nullptr) *reinterpret_cast<uint32_t*>(p.count + xe + c * kChunk) = pack_counts(k);   // N <= 255 here
                if (p.count16 != nullptr) {
                    *reinterpret_cast<uint2*>(p.count16 + xe + c * kChunk) =
                        make_uint2(k.c[0] | (k.c[1] << 16), k.c[2] | (k.c[3] << 16));
                }
            } else {
                const uint32_t dn = my_delta_bits(dword, c, lane);
                d0 = (dn & 1u) ? 1.0f : -1.0f;
                d1 = (dn & 2u) ? 1.0f : -1.0f;
                d2 = (dn & 4u) ? 1.0f : -1.0f;
                d3 = (dn & 8u) ? 1.0f : -1.0f;
            }
            float4 v = xv[c];
            v.x = apply_coord(v.x, d0, p.lr, p.wd);
            v.y = apply_coord(v.y, d1, p.lr, p.wd);
            v.z = apply_coord(v.z, d2, p.lr, p.wd);
            v.w = apply_coord(v.w, d3, p.lr, p.wd);
            *reinterpret_cast<float4*>(xs + xe + c * kChunk) = v;
        }
    }
}

template <int PLANES, bool AVG, bool COUNTS, bool TABLE>
cudaError_t launch3(const AggParams& p, cudaStream_t s) {
    aggregate_apply_kernel<PLANES, AVG, COUNTS, TABLE><<<grid_for(p.ntiles), kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <int PLANES, bool TABLE>
cudaError_t launch(const AggParams& p, cudaStream_t s) {
    if (p.ntiles == 0) return cudaSuccess;
    if (p.average) return launch3<PLANES, true, true, TABLE>(p, s);
    if (p.count != nullptr || p.count16 != nullptr) return launch3<PLANES, false, true, TABLE>(p, s);
    return launch3<PLANES, false, false, TABLE>(p, s);
}

}  // namespace

cudaError_t launch_aggregate_apply(const AggParams& p, int sm_count, cudaStream_t s) {
    (void)sm_count;
    return dispatch_planes(p.n_workers, p.x_off != nullptr, [&](auto planes, auto table) {
        return launch<decltype(planes)::value, decltype(table)::value>(p, s);
    });
}

}  // namespace dlion
