// Shared declarations of the CUDA library: device-side segment table, the tile
// lookup every kernel uses, and the pinned floating-point steps.
//
// Arithmetic contract (see include/dlion.h): binary32, one rounding per
// operation, no fused multiply-add.  The _rn intrinsics below are never
// contracted by the compiler, whatever -fmad says.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dlion.h"

namespace dlion {

constexpr uint32_t kTile = 4096;        // coordinates per work item (all kernels)
constexpr uint32_t kChunk = 128;        // coordinates one warp covers per vector access
constexpr uint32_t kFull = 0xFFFFFFFFu;

struct TileRef {
    unsigned long long base;   // arena index of the tile's first coordinate
    uint32_t valid;            // parameters in the tile, 1..kTile
    uint32_t tensor;           // index of the segment (tensor) the tile belongs to
};

// One row per tile (built by dlion_init): a block finds its tile with a single
// 16-byte load.  A tile never spans two segments.
struct TileRow {
    unsigned long long base;   // arena index of the tile's first coordinate
    uint32_t valid;            // parameters in the tile, 1..kTile
    uint32_t tensor;           // segment index
};

// Tile lookup.  With a table: one load.  Without one the parameters are a flat
// vector of flat_d coordinates starting at arena index 0 (the fixed-scratch step,
// which owns no table): plain arithmetic.
// (Kept out of line on purpose: inlined into the worker-side kernel it changed the
// register allocation of the whole kernel from 48 to 64 registers, one block less
// per SM, and the c5 step from 30 to 34 ms.)
static __device__ __noinline__ TileRef flat_tile(unsigned long long flat_d, unsigned long long tile) {
    TileRef t;
    t.base = tile * kTile;
    const unsigned long long left = flat_d - t.base;
    t.valid = left < kTile ? static_cast<uint32_t>(left) : kTile;
    t.tensor = 0;
    return t;
}

__device__ __forceinline__ TileRef find_tile(const TileRow* __restrict__ tiles, unsigned long long flat_d,
                                             unsigned long long tile) {
    TileRef t;
    if (tiles != nullptr) {
        const uint4 r = __ldg(reinterpret_cast<const uint4*>(tiles + tile));
        t.base = static_cast<unsigned long long>(r.x) | (static_cast<unsigned long long>(r.y) << 32);
        t.valid = r.z;
        t.tensor = r.w;
        return t;
    }
    return flat_tile(flat_d, tile);
}

// Algorithm 1, worker side, one coordinate: returns the sign bit of
// beta1*m + (1-beta1)*g and replaces m by beta2*m + (1-beta2)*g (old m in both).
struct Betas { float b1, om1, b2, om2; };

__device__ __forceinline__ uint32_t lion_coord(float g, float& m, const Betas& k) {
    const float c = __fadd_rn(__fmul_rn(k.b1, m), __fmul_rn(k.om1, g));
    m = __fadd_rn(__fmul_rn(k.b2, m), __fmul_rn(k.om2, g));
    return c >= 0.0f ? 1u : 0u;
}

// The same for two coordinates at once: the four products come from the packed
// binary32 multiply of sm_100 (mul.rn.f32x2: each element rounded to nearest exactly
// like the scalar multiply, half the issue slots), the sums from scalar adds.
// (The packed ADD must not be used here: fed by a packed multiply, the assembler
// contracts the pair into a packed fused multiply-add even with contraction
// switched off -- measured on B200, every mismatch against the scalar form was
// explained by one fused rounding -- and a fused blend decides other signs.
// __fadd_rn is never contracted.)  Returns the two sign bits, coordinate 0 in bit 0.
__device__ __forceinline__ uint32_t lion_pair(float2 g, float2& m, const Betas& k) {
    const float2 p1 = __fmul2_rn(make_float2(k.b1, k.b1), m), q1 = __fmul2_rn(make_float2(k.om1, k.om1), g);
    const float2 p2 = __fmul2_rn(make_float2(k.b2, k.b2), m), q2 = __fmul2_rn(make_float2(k.om2, k.om2), g);
    const float c0 = __fadd_rn(p1.x, q1.x), c1 = __fadd_rn(p1.y, q1.y);
    m = make_float2(__fadd_rn(p2.x, q2.x), __fadd_rn(p2.y, q2.y));
    return (c0 >= 0.0f ? 1u : 0u) | (c1 >= 0.0f ? 2u : 0u);
}

// Section 3.2, last equation: x - lr*(Delta + lambda*x).
__device__ __forceinline__ float apply_coord(float x, float delta, float lr, float wd) {
    return __fsub_rn(x, __fmul_rn(lr, __fadd_rn(delta, __fmul_rn(wd, x))));
}

__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xFFFF0000u); }

// Four consecutive gradients as floats, from fp32 or bf16 storage.  (Plain loads and
// stores throughout: evict-first streaming hints measured 3 % slower on B200.)
template <bool BF16>
__device__ __forceinline__ float4 load_grad4(const void* g, unsigned long long idx) {
    if constexpr (BF16) {
        const uint2 v = *(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(g) + idx));
        return make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    } else {
        return *(reinterpret_cast<const float4*>(static_cast<const float*>(g) + idx));
    }
}

template <bool BF16>
__device__ __forceinline__ float load_grad1(const void* g, unsigned long long idx) {
    if constexpr (BF16) {
        return __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(g)[idx]) << 16);
    } else {
        return static_cast<const float*>(g)[idx];
    }
}

// Momentum storage: fp32, or bf16 (widened exactly on load; on store the binary32
// result is rounded to nearest, ties to even, by the hardware conversion; NaN stays
// NaN).  Two values per conversion: lo goes to the low half of the word.
__device__ __forceinline__ uint32_t pack_bf16x2_rne(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t f32_to_bf16_rne(float f) { return pack_bf16x2_rne(f, 0.0f) & 0xFFFFu; }

template <bool MB16>
__device__ __forceinline__ float4 load_state4(const void* m, unsigned long long idx) {
    if constexpr (MB16) {
        const uint2 v = *(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(m) + idx));
        return make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    } else {
        return *(reinterpret_cast<const float4*>(static_cast<const float*>(m) + idx));
    }
}

template <bool MB16>
__device__ __forceinline__ void store_state4(void* m, unsigned long long idx, const float4& v) {
    if constexpr (MB16) {
        uint2 o;
        o.x = pack_bf16x2_rne(v.x, v.y);
        o.y = pack_bf16x2_rne(v.z, v.w);
        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(m) + idx) = o;
    } else {
        *reinterpret_cast<float4*>(static_cast<float*>(m) + idx) = v;
    }
}

template <bool MB16>
__device__ __forceinline__ float load_state1(const void* m, unsigned long long idx) {
    if constexpr (MB16) {
        return __uint_as_float(static_cast<uint32_t>(static_cast<const uint16_t*>(m)[idx]) << 16);
    } else {
        return static_cast<const float*>(m)[idx];
    }
}

template <bool MB16>
__device__ __forceinline__ void store_state1(void* m, unsigned long long idx, float v) {
    if constexpr (MB16) static_cast<uint16_t*>(m)[idx] = static_cast<uint16_t>(f32_to_bf16_rne(v));
    else static_cast<float*>(m)[idx] = v;
}

// Worker i's coefficients: its row of the per-worker table when one is set
// (Algorithm 1 lets every worker choose its own beta1, beta2), else the common ones.
__device__ __forceinline__ Betas betas_of(const Betas* __restrict__ table, const Betas& common,
                                          unsigned long long worker) {
    if (table == nullptr) return common;
    const float4 r = __ldg(reinterpret_cast<const float4*>(table + worker));
    Betas k;
    k.b1 = r.x; k.om1 = r.y; k.b2 = r.z; k.om2 = r.w;
    return k;
}

// Lane l of each group of 8 lanes holds a nibble (signs of coordinates 4l..4l+3
// of a 32-coordinate word).  Returns the assembled word in all 8 lanes.
__device__ __forceinline__ uint32_t gather_word(uint32_t nibble, uint32_t lane) {
    uint32_t v = nibble << (4u * (lane & 7u));
    v |= __shfl_xor_sync(kFull, v, 1);
    v |= __shfl_xor_sync(kFull, v, 2);
    v |= __shfl_xor_sync(kFull, v, 4);
    return v;
}

// Bit k of a nibble -> byte k of a word (no carries: the four shifted copies do not overlap).
__device__ __forceinline__ uint32_t spread_nibble(uint32_t nibble) {
    return (nibble * 0x00204081u) & 0x01010101u;
}

// ---- launch parameters ----------------------------------------------------
// Per-tensor tables (dlion_bind_tensors): entry k of a table is the BYTE OFFSET, from the
// base pointer passed beside the table, of tensor k's storage minus the byte offset of
// its first coordinate in the arena numbering -- so that base + table[k] +
// arena_index * element_size is the element's address and the kernels index exactly as
// they do into one flat arena.  (Offsets from a kernel-argument pointer rather than raw
// addresses: the compiler then knows the accesses are to global memory and keeps
// reordering them freely around the shared-memory traffic of the vote; with addresses
// loaded from a table the Averaging kernel measured 11 % slower, arena mode included.)
struct WorkerParams {
    const void* g;
    void* m;                         // float, or bf16 when m_bf16
    const long long* g_off;          // [n_workers_total][nseg] offsets from g, or null: g is an arena
    const long long* m_off;          // likewise for the momentum, from m
    uint32_t nseg;
    // scatter mode (dlion_worker_step_scatter): the sign words of coordinate slice r go to
    // the buffer at byte offset dst_off[r] from packed, row `slot` of [rows][slice_words]
    const long long* dst_off;        // [n_dst] offsets from packed, or null: packed is the [N][d_pad/32] arena
    unsigned long long slice_words;
    uint32_t slot;
    uint32_t* packed;
    const TileRow* tiles;            // per-tile rows (device), or null: flat vector of flat_d coordinates
    unsigned long long flat_d;
    uint32_t n_workers;              // workers this launch covers (1 for a single-worker call)
    unsigned long long ntiles;       // tiles per worker
    unsigned long long d_pad;        // elements between consecutive workers in g and m
    Betas k;
    const Betas* betas;              // per-worker table (device), or null
    uint32_t worker0;                // id of the first worker this launch covers
    int m_bf16;
};

struct AggParams {
    const uint32_t* packed;
    float* x;
    const long long* x_off;          // [nseg] offsets from x, or null: x is an arena
    uint32_t* delta_bits;            // nullable
    uint8_t* count;                  // nullable: vote counts, one byte each (N <= 255)
    uint16_t* count16;               // nullable: vote counts, 16 bits each (any N)
    const TileRow* tiles;            // per-tile rows (device), or null: flat vector of flat_d coordinates
    unsigned long long flat_d;
    uint32_t n_workers;
    unsigned long long ntiles;
    unsigned long long w_stride;     // words between consecutive workers in packed
    float lr, wd;
    int average;                     // 0 = majority vote, 1 = averaging (or, with ternary, the same kernel with a sign table)
    int ternary;                     // Majority Vote with Delta = 0 on an even-N tie
};

struct FusedParams {
    const void* g;
    void* m;                         // float, or bf16 when m_bf16
    float* x;
    uint32_t* packed;                // nullable
    const TileRow* tiles;            // per-tile rows (device), or null: flat vector of flat_d coordinates
    unsigned long long flat_d;
    uint32_t n_workers;
    unsigned long long ntiles;
    unsigned long long d_pad;
    Betas k;
    const Betas* betas;              // per-worker table (device), or null
    int m_bf16;
    float lr, wd;
    int average;
    int ternary;                     // see AggParams
};

struct GlobalParams {                // Global-Lion comparison step
    const void* g;
    float* m;
    float* x;
    uint32_t* delta_bits;            // nullable
    const TileRow* tiles;
    unsigned long long flat_d;
    uint32_t n_workers;
    unsigned long long ntiles;
    unsigned long long d_pad;
    Betas k;
    float lr, wd;
};

struct WireParams {                  // server-only aggregate / worker-side apply
    const uint32_t* packed;          // aggregate: the N binary vectors
    uint32_t* wire_out;              // aggregate: the broadcast message
    const uint32_t* wire_in;         // apply: the broadcast message
    float* x;                        // apply: parameters
    const long long* x_off;          // apply: [nseg] offsets from x, or null: x is an arena
    const TileRow* tiles;            // per-tile rows (device), or null: flat vector of flat_d coordinates
    unsigned long long flat_d;
    uint32_t n_workers;
    unsigned long long ntiles;
    unsigned long long w_stride;     // words between consecutive binary vectors in packed
    unsigned long long plane_stride; // words between consecutive planes of the message
    uint32_t kplanes;                // planes in the message: 1, or ceil(log2(N+1)) for Averaging
    unsigned long long slice_words;  // apply: 0, or the message is [slice][plane][slice_words] (all-gather order)
    float lr, wd;
    int average;
    int ternary;                     // aggregate: write the two planes of Delta + 1 instead of the Delta bit
};

// One thread block per work item, in item order (the kernels still stride, so a
// count beyond the largest grid is covered too).
inline unsigned grid_for(unsigned long long n_items) {
    return n_items > 0x7FFFFFFFull ? 0x7FFFFFFFu : static_cast<unsigned>(n_items);
}

// Host-side launchers (one per .cu file).
cudaError_t launch_worker_step(const WorkerParams& p, bool bf16, int sm_count, cudaStream_t s);   // table mode when p.g_off
cudaError_t launch_aggregate_apply(const AggParams& p, int sm_count, cudaStream_t s);
cudaError_t launch_step_fused(const FusedParams& p, bool bf16, int sm_count, cudaStream_t s);
cudaError_t launch_wire(const WireParams& p, bool apply, cudaStream_t s);
cudaError_t launch_step_global(const GlobalParams& p, bool bf16, cudaStream_t s);
uint32_t planes_for(uint32_t n_workers);   // ceil(log2(N+1))

}  // namespace dlion
