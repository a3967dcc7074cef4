// Worker side of Algorithm 1 (arXiv 2404.00438): for every worker i and
// coordinate j,
//     delta_i[j] = sign(beta1 m_i[j] + (1-beta1) g_i[j])      (old m_i)
//     m_i[j]    <- beta2 m_i[j] + (1-beta2) g_i[j]
// with delta_i packed 32 signs per word into the 1-bit wire buffer
// (Section 3.2, "Communication Cost": each worker sends d bits).
//
// A pure streaming kernel, bound by HBM: per coordinate and worker it reads the
// gradient (2 or 4 B) and the momentum (4 B), writes the momentum (4 B) and 1/8 B
// of signs.  Work item = (worker, tile of 4096 coordinates), one thread block per
// item, dispatched by the hardware in item order: the blocks in flight then form
// a compact window that sweeps the arenas front to back, which measured 12 %
// faster on B200 than a persistent grid striding over the items (6.9 vs 6.2
// TB/s), and the same as a persistent grid drawing items from an atomic
// counter.  Inside a tile each of the block's four warps owns 1024 consecutive
// coordinates as eight 128-coordinate chunks; lane l of a chunk holds coordinates
// 4l..4l+3, so every load and store instruction of a warp is one contiguous run
// (16 B per lane for fp32, 8 B per lane for bf16 gradients).  Eight lanes'
// nibbles are merged into a word by three xor-shuffles, and the warp's 32 words
// leave as one 128-byte run, one word per lane.  A thread thus carries 32
// coordinates: the per-block work that does not scale with coordinates (tile
// lookup, 64-bit index arithmetic, beta row) is paid once per 32, not per 16 --
// against 256-thread blocks with 16 coordinates per thread this measured +0.3 to
// +1.4 % for the DRAM-bound variants and +10 % for the bf16/bf16 variant below.
#include "dlion_common.cuh"

namespace dlion {
namespace {

constexpr int kThreads = 128;            // 4 warps x 1024 coordinates = one tile
constexpr int kChunksPerWarp = 8;        // 128-coordinate chunks per warp
constexpr int kWideChunks = 4;           // 256-coordinate chunks per warp (bf16/bf16 path)

// TABLE: gradients and momenta are separate tensors reached through per-tensor offset
// tables (one extra 8-byte load per stream and block) instead of two flat arenas.
// Occupancy, measured on the 1.3 B-parameter workload: with fp32 momentum the kernel is
// bound by DRAM and fastest with the register allocation the compiler picks unprompted
// (80-96 registers, 5 blocks per SM; forced to more blocks it spills and loses up to
// 50 %); with bf16 gradients AND bf16 momentum it moves 40 % fewer bytes per coordinate,
// leans on instruction issue, and is fastest at 10 blocks per SM (48 registers; 18.5 ms
// against 19.1 at 9 and 8 blocks and 20.7 at 11 and 12, which spill).
// Where sign word `wi` (arena word index) of worker `worker` is written: the wire arena,
// or (SCATTER) row slot + worker of the receive buffer of the coordinate slice it falls in.
template <bool SCATTER>
__device__ __forceinline__ uint32_t* word_at(const WorkerParams& p, unsigned long long worker,
                                             unsigned long long w_stride, unsigned long long wi) {
    if constexpr (SCATTER) {
        const unsigned long long r = wi / p.slice_words;
        uint32_t* buf = reinterpret_cast<uint32_t*>(reinterpret_cast<char*>(p.packed) + p.dst_off[r]);
        return buf + (p.slot + worker) * p.slice_words + (wi - r * p.slice_words);
    } else {
        return p.packed + worker * w_stride + wi;
    }
}

// MODE 0: flat arenas.  MODE 1: per-tensor tables for g and m.  MODE 2: flat g and m, sign
// words scattered to per-slice receive buffers (the send of the exchange fused in).
template <bool BF16, bool MB16, int MODE>
__device__ __forceinline__ void worker_step_body(const WorkerParams& p) {
    constexpr bool TABLE = MODE == 1;
    constexpr bool SCATTER = MODE == 2;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp = threadIdx.x >> 5;
    const unsigned long long w_stride = p.d_pad / 32;
    const unsigned long long worker = blockIdx.y;                  // grid: x = tile (fastest), y = worker

    for (unsigned long long tile = blockIdx.x; tile < p.ntiles; tile += gridDim.x) {
        const TileRef t = find_tile(p.tiles, p.flat_d, tile);
        unsigned long long wbase = worker * p.d_pad;               // element offset of this worker
        const void* gsrc = p.g;
        void* mdst = p.m;
        if constexpr (TABLE) {
            const unsigned long long row = (p.worker0 + worker) * p.nseg + t.tensor;
            gsrc = static_cast<const char*>(p.g) + p.g_off[row];
            mdst = static_cast<char*>(p.m) + p.m_off[row];
            wbase = 0;
        }
        const Betas k = betas_of(p.betas, p.k, p.worker0 + worker);
        const uint32_t in_tile = warp * (kChunksPerWarp * kChunk); // first coordinate of this warp
        const unsigned long long word0 = (t.base + in_tile) / 32;  // arena index of this warp's first sign word

        if (t.valid == kTile) {
            // ---- full tile: vector path, all loads issued before any use ----
            if constexpr (BF16 && MB16) {
                // both streams are bf16: lane l of a 256-coordinate chunk holds coordinates
                // 8l..8l+7 (one 16-byte access each for g and m), its eight signs are a byte,
                // and four lanes' bytes make a word (two xor-shuffles); the products come
                // from the packed multiply (this variant is bound by instruction issue:
                // 20.7 -> 20.0 ms on the 1.3 B-parameter workload; the DRAM-bound fp32-momentum
                // variants measured 6 % SLOWER with it and keep the scalar form)
                const unsigned long long e0 = wbase + t.base + in_tile + lane * 8;
                const uint16_t* gp = static_cast<const uint16_t*>(gsrc) + e0;
                uint16_t* mp = static_cast<uint16_t*>(mdst) + e0;
                uint4 gv[kWideChunks], mv[kWideChunks];
#pragma unroll
                for (int u = 0; u < kWideChunks; ++u) {
                    gv[u] = *reinterpret_cast<const uint4*>(gp + u * 2 * kChunk);
                    mv[u] = *reinterpret_cast<const uint4*>(mp + u * 2 * kChunk);
                }
                uint32_t mine = 0;
#pragma unroll
                for (int u = 0; u < kWideChunks; ++u) {
                    const uint32_t gw[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
                    const uint32_t mw[4] = {mv[u].x, mv[u].y, mv[u].z, mv[u].w};
                    uint32_t out[4], byte = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float2 m2 = make_float2(bf16_lo(mw[q]), bf16_hi(mw[q]));
                        byte |= lion_pair(make_float2(bf16_lo(gw[q]), bf16_hi(gw[q])), m2, k) << (2 * q);
                        out[q] = pack_bf16x2_rne(m2.x, m2.y);
                    }
                    *reinterpret_cast<uint4*>(mp + u * 2 * kChunk) = make_uint4(out[0], out[1], out[2], out[3]);
                    uint32_t w = byte << (8u * (lane & 3u));
                    w |= __shfl_xor_sync(kFull, w, 1);
                    w |= __shfl_xor_sync(kFull, w, 2);
                    if ((lane & 3u) == static_cast<uint32_t>(u)) mine = w;
                }
                // lane l holds word l/4 of chunk l%4: word index 8*(l%4) + l/4
                *word_at<SCATTER>(p, worker, w_stride, word0 + 8u * (lane & 3u) + (lane >> 2)) = mine;
            } else {
                const unsigned long long e0 = wbase + t.base + in_tile + lane * 4;
                float4 g[kChunksPerWarp], m[kChunksPerWarp];
#pragma unroll
                for (int u = 0; u < kChunksPerWarp; ++u) {
                    g[u] = load_grad4<BF16>(gsrc, e0 + u * kChunk);
                    m[u] = load_state4<MB16>(mdst, e0 + u * kChunk);
                }
                uint32_t mine = 0;
#pragma unroll
                for (int u = 0; u < kChunksPerWarp; ++u) {
                    uint32_t nib = lion_coord(g[u].x, m[u].x, k);
                    nib |= lion_coord(g[u].y, m[u].y, k) << 1;
                    nib |= lion_coord(g[u].z, m[u].z, k) << 2;
                    nib |= lion_coord(g[u].w, m[u].w, k) << 3;
                    store_state4<MB16>(mdst, e0 + u * kChunk, m[u]);
                    const uint32_t w = gather_word(nib, lane);
                    if ((lane & 7u) == static_cast<uint32_t>(u)) mine = w;
                }
                // lane l holds the word of chunk l%8, group l/8: word index 4*(l%8) + l/8
                *word_at<SCATTER>(p, worker, w_stride, word0 + 4u * (lane & 7u) + (lane >> 3)) = mine;
            }
        } else {
            // ---- last tile of a segment: per-coordinate guards -------------
#pragma unroll 1
            for (int u = 0; u < kChunksPerWarp; ++u) {
                const uint32_t c0 = in_tile + u * kChunk;           // chunk start within the tile
                if (c0 >= t.valid) break;                            // warp-uniform
                const uint32_t j0 = c0 + lane * 4;
                const unsigned long long e = wbase + t.base + j0;
                uint32_t nib = 0;
                if (j0 + 4 <= t.valid) {
                    float4 g = load_grad4<BF16>(gsrc, e);
                    float4 m = load_state4<MB16>(mdst, e);
                    nib = lion_coord(g.x, m.x, k);
                    nib |= lion_coord(g.y, m.y, k) << 1;
                    nib |= lion_coord(g.z, m.z, k) << 2;
                    nib |= lion_coord(g.w, m.w, k) << 3;
                    store_state4<MB16>(mdst, e, m);
                } else {
                    for (uint32_t q = 0; q < 4 && j0 + q < t.valid; ++q) {
                        const float g = load_grad1<BF16>(gsrc, e + q);
                        float m = load_state1<MB16>(mdst, e + q);
                        nib |= lion_coord(g, m, k) << q;
                        store_state1<MB16>(mdst, e + q, m);
                    }
                }
                const uint32_t w = gather_word(nib, lane);
                // only words that hold at least one parameter are written
                if ((lane & 7u) == 0 && c0 + (lane >> 3) * 32 < t.valid) {
                    *word_at<SCATTER>(p, worker, w_stride, word0 + 4u * u + (lane >> 3)) = w;
                }
            }
        }
    }
}

// (Parameters are taken by value on purpose: marking them __grid_constant__ measured 6 % slower here.)
template <bool BF16, bool MB16, int MODE>
__global__ void __launch_bounds__(kThreads)
worker_step_kernel(const WorkerParams p) {
    worker_step_body<BF16, MB16, MODE>(p);
}

// bf16 gradients and bf16 momentum: 10 blocks per SM (see above)
template <int MODE>
__global__ void __launch_bounds__(kThreads, 10)
worker_step_kernel_bf16(const WorkerParams p) {
    worker_step_body<true, true, MODE>(p);
}

template <bool BF16, bool MB16, int MODE>
cudaError_t launch_mode(const WorkerParams& p, const dim3 grid, cudaStream_t s) {
    if constexpr (BF16 && MB16) worker_step_kernel_bf16<MODE><<<grid, kThreads, 0, s>>>(p);
    else worker_step_kernel<BF16, MB16, MODE><<<grid, kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <bool BF16, bool MB16>
cudaError_t launch(const WorkerParams& p, cudaStream_t s) {
    if (p.ntiles == 0 || p.n_workers == 0) return cudaSuccess;
    const dim3 grid(grid_for(p.ntiles), p.n_workers);               // blocks are dispatched x first: worker-major item order
    if (p.g_off != nullptr) return launch_mode<BF16, MB16, 1>(p, grid, s);
    if (p.dst_off != nullptr) return launch_mode<BF16, MB16, 2>(p, grid, s);
    return launch_mode<BF16, MB16, 0>(p, grid, s);
}

}  // namespace

cudaError_t launch_worker_step(const WorkerParams& p, bool bf16, int sm_count, cudaStream_t s) {
    (void)sm_count;
    if (p.m_bf16) return bf16 ? launch<true, true>(p, s) : launch<false, true>(p, s);
    return bf16 ? launch<true, false>(p, s) : launch<false, false>(p, s);
}

}  // namespace dlion
