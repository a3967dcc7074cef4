// Distributed Lion -- CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what one
// Distributed-Lion optimizer step computes.  It exists so that the CUDA library
// can be checked against it.  It shares no code, header, table or helper with
// the CUDA path and must never be called from the product path.
//
// What it follows (arXiv 2404.00438):
//   * worker side  -- Algorithm 1 "Worker-side", and the pair of equations in
//                     Section 3.2 that define m_{i,t+1} and delta_{i,t};
//   * server side  -- Algorithm 1 "Server-side", and the aggregate(S_t)
//                     equation of Section 3.2 (Averaging / Majority Vote);
//   * apply        -- x_{i,t+1} = x_{i,t} - eps (Delta_t + lambda x_{i,t}),
//                     last equation of Section 3.2;
//   * wire format  -- Section 3.2 "Communication Cost" and Table 1: delta_i is a
//                     binary vector of d bits; Delta is binary (Majority Vote) or
//                     an integer in {0..N} (Averaging);
//   * Global Lion  -- the full-precision comparison scheme of the appendix
//                     ("Global Lion Convergence") and Section 5.1.
//
// The method is exact arithmetic on given inputs, so the oracle is the
// definition written out coordinate by coordinate.  The paper does not fix the
// floating-point format, the evaluation order, sign(0) or the even-N tie; the
// readings used here are:
//   R1  all arithmetic in IEEE binary32, one rounding per operation, no fused
//       multiply-add (build with -ffp-contract=off):
//           c   = fl( fl(beta1*m) + fl((1-beta1)*g) )
//           m'  = fl( fl(beta2*m) + fl((1-beta2)*g) )
//           x'  = fl( x - fl( eps * fl( Delta + fl(lambda*x) ) ) )
//       with (1-beta) itself computed once in binary32.  bf16 gradients are
//       widened exactly (bits << 16).
//   R2  sgn(v) = +1 if v >= 0 else -1.  Both zeros give +1; NaN gives -1.  The
//       wire carries one bit per coordinate, so sign has to be two-valued.
//   R3  the same rule decides an even-N tie: S = 0 gives Delta = +1.
//   R4  "S_t in {0..N}" is read as the count P of +1 votes; S = 2P - N.
//   R5  delta_{i,t} uses the OLD momentum m_{i,t} (both equations carry the
//       subscript t on their right-hand sides).
//   R6  Averaging: Delta = (float)(2P-N) / (float)N, IEEE division.
//   R3' (optional, mode DLION_ORACLE_MAJORITY_TERNARY) the other reading of an
//       even-N tie: the three-valued sign the appendix's lemma works with,
//       sign(0) = 0, so S = 0 gives Delta = 0 and the step is pure weight decay
//       there.  Delta then has three values and takes two bits on the wire,
//       sent as the integer Delta + 1 in {0, 1, 2} (two planes, like a count).
//
// Parity status: every function below is pinned by tests/test_oracle_pins.py
// (special cases N=1, identical workers, beta=0, beta1=beta2, brute-force vote
// sums, closed forms for x and m in double precision, the Phase-I contraction of
// Theorem "Phase I", a hand-derived worked example under tests/golden/).  The
// one thing those cannot pin is reading R1 itself (the rounding order): the
// paper is silent on it -- "parity unpinned" for the last-bit rounding order
// only; the double-precision pins bound it to within an ulp per operation.
//
// Layout (the same conventions the C-ABI of the CUDA library documents, restated
// here independently): arenas are worker-major, g[N][d_pad], m[N][d_pad],
// packed[N][d_pad/32]; bit b of word w is coordinate 32*w+b; bit 1 means +1.
// A segment table {elem_offset, numel} names the coordinates that are real
// parameters; everything else is padding: never read as a parameter, never
// written, and its packed bits are 0.

#include <cstddef>
#include <cstdint>
#include <cstring>

extern "C" {

struct dlion_oracle_segment {
    uint64_t elem_offset;
    uint64_t numel;
};

enum { DLION_ORACLE_MAJORITY = 0, DLION_ORACLE_AVERAGE = 1, DLION_ORACLE_MAJORITY_TERNARY = 2 };

static bool known_mode(int mode) {
    return mode == DLION_ORACLE_MAJORITY || mode == DLION_ORACLE_AVERAGE || mode == DLION_ORACLE_MAJORITY_TERNARY;
}
enum { DLION_ORACLE_GRAD_F32 = 0, DLION_ORACLE_GRAD_BF16 = 1 };
enum { DLION_ORACLE_STATE_F32 = 0, DLION_ORACLE_STATE_BF16 = 1 };

}  // extern "C"

namespace {

inline float widen_bf16(uint16_t h) {
    uint32_t u = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

inline float load_grad(const void* g, int gdtype, size_t idx) {
    if (gdtype == DLION_ORACLE_GRAD_BF16) {
        return widen_bf16(static_cast<const uint16_t*>(g)[idx]);
    }
    return static_cast<const float*>(g)[idx];
}

// Momentum kept in bf16 (optional): widened exactly on load; on store the binary32
// result is rounded to the nearest bf16, ties to the even mantissa (IEEE
// round-to-nearest-even on the upper 16 bits).  NaN stays NaN (quiet bit set).
inline uint16_t round_to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, sizeof u);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return static_cast<uint16_t>((u >> 16) | 0x0040u);
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

inline float load_state(const void* m, int mdtype, size_t idx) {
    if (mdtype == DLION_ORACLE_STATE_BF16) return widen_bf16(static_cast<const uint16_t*>(m)[idx]);
    return static_cast<const float*>(m)[idx];
}

inline void store_state(void* m, int mdtype, size_t idx, float v) {
    if (mdtype == DLION_ORACLE_STATE_BF16) static_cast<uint16_t*>(m)[idx] = round_to_bf16(v);
    else static_cast<float*>(m)[idx] = v;
}

// R2: two-valued sign as a bit.
inline uint32_t sign_bit(float v) { return (v >= 0.0f) ? 1u : 0u; }

}  // namespace

extern "C" {

// Worker side of Algorithm 1 for all N workers (or for one worker when the
// caller passes N = 1 and that worker's slices).
//   g       [N][d_pad]  gradients g_{i,t}, f32 or bf16            (read)
//   m       [N][d_pad]  momenta m_{i,t} -> m_{i,t+1}, f32         (in place)
//   packed  [N][d_pad/32] delta_{i,t}, one bit per coordinate     (written:
//           words that hold at least one parameter; others untouched)
// Returns 0, or -1 on a malformed argument.
// General form.  Algorithm 1 lets every worker set its own beta1, beta2 (footnote
// to its inputs): beta1s[i], beta2s[i] are worker i's.  mdtype selects fp32 or
// bf16 storage of the momentum (arithmetic is binary32 either way).
int dlion_oracle_worker_step_ex(const dlion_oracle_segment* segs, uint32_t nseg,
                                uint64_t d_pad, uint32_t n_workers, int gdtype, int mdtype,
                                const void* g, void* m, uint32_t* packed,
                                const float* beta1s, const float* beta2s, int nthreads) {
    if (!segs || !g || !m || !packed || !beta1s || !beta2s || d_pad % 32 != 0 || n_workers == 0) return -1;
    const uint64_t W = d_pad / 32;
    (void)nthreads;
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t lo = segs[s].elem_offset;
        const uint64_t hi = lo + segs[s].numel;
        if (hi > d_pad || lo % 32 != 0) return -1;      // no word is shared by two segments
        if (hi == lo) continue;
        const int64_t w_lo = static_cast<int64_t>(lo / 32);
        const int64_t w_hi = static_cast<int64_t>((hi + 31) / 32);
#pragma omp parallel for collapse(2) schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
        for (uint32_t i = 0; i < n_workers; ++i) {
            for (int64_t w = w_lo; w < w_hi; ++w) {
                uint32_t word = 0;
                for (uint32_t b = 0; b < 32; ++b) {
                    const uint64_t j = static_cast<uint64_t>(w) * 32 + b;
                    if (j < lo || j >= hi) continue;            // padding bit stays 0
                    const size_t idx = static_cast<size_t>(i) * d_pad + j;
                    const float beta1 = beta1s[i], beta2 = beta2s[i];
                    const float om1 = 1.0f - beta1;             // R1: (1-beta) in binary32
                    const float om2 = 1.0f - beta2;
                    const float gf = load_grad(g, gdtype, idx);
                    const float mo = load_state(m, mdtype, idx);  // R5: old momentum
                    const float a1 = beta1 * mo;
                    const float b1 = om1 * gf;
                    const float c = a1 + b1;                    // Alg. 1, delta line
                    word |= sign_bit(c) << b;
                    const float a2 = beta2 * mo;
                    const float b2 = om2 * gf;
                    store_state(m, mdtype, idx, a2 + b2);       // Alg. 1, momentum line
                }
                packed[static_cast<size_t>(i) * W + static_cast<size_t>(w)] = word;
            }
        }
    }
    return 0;
}

// The common case: one (beta1, beta2) for all workers, fp32 momentum.
int dlion_oracle_worker_step(const dlion_oracle_segment* segs, uint32_t nseg,
                             uint64_t d_pad, uint32_t n_workers, int gdtype,
                             const void* g, float* m, uint32_t* packed,
                             float beta1, float beta2, int nthreads) {
    if (n_workers == 0 || n_workers > 65536) return -1;
    float* b1 = new float[n_workers];
    float* b2 = new float[n_workers];
    for (uint32_t i = 0; i < n_workers; ++i) { b1[i] = beta1; b2[i] = beta2; }
    const int rc = dlion_oracle_worker_step_ex(segs, nseg, d_pad, n_workers, gdtype, DLION_ORACLE_STATE_F32,
                                               g, m, packed, b1, b2, nthreads);
    delete[] b1;
    delete[] b2;
    return rc;
}

// Server side of Algorithm 1 followed by the parameter update of Section 3.2.
//   packed     [N][d_pad/32]  the N binary vectors delta_{i,t}         (read)
//   x          [d_pad]        parameters x_t -> x_{t+1}, f32           (in place)
//   delta_bits [d_pad/32]     optional: Delta_t as bits (Majority Vote; for
//                             Averaging it is sgn of the sum), padding bits 0
//   count      [d_pad]        optional: P = number of +1 votes, u8 (N <= 255)
// Returns 0, or -1 on a malformed argument.
int dlion_oracle_aggregate_apply(const dlion_oracle_segment* segs, uint32_t nseg,
                                 uint64_t d_pad, uint32_t n_workers, int mode,
                                 const uint32_t* packed, float* x,
                                 uint32_t* delta_bits, uint8_t* count,
                                 float lr, float weight_decay, int nthreads) {
    if (!segs || !packed || !x || d_pad % 32 != 0 || n_workers == 0) return -1;
    if (count && n_workers > 255) return -1;
    if (!known_mode(mode)) return -1;
    const uint64_t W = d_pad / 32;
    const int32_t N = static_cast<int32_t>(n_workers);
    (void)nthreads;
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t lo = segs[s].elem_offset;
        const uint64_t hi = lo + segs[s].numel;
        if (hi > d_pad || lo % 32 != 0) return -1;
        if (hi == lo) continue;
        const int64_t w_lo = static_cast<int64_t>(lo / 32);
        const int64_t w_hi = static_cast<int64_t>((hi + 31) / 32);
#pragma omp parallel for schedule(static) num_threads(nthreads > 0 ? nthreads : 1)
        for (int64_t w = w_lo; w < w_hi; ++w) {
            uint32_t dword = 0;
            for (uint32_t b = 0; b < 32; ++b) {
                const uint64_t j = static_cast<uint64_t>(w) * 32 + b;
                if (j < lo || j >= hi) continue;
                int32_t P = 0;                                   // R4: +1 votes
                for (int32_t i = 0; i < N; ++i) {
                    P += static_cast<int32_t>((packed[static_cast<size_t>(i) * W + static_cast<size_t>(w)] >> b) & 1u);
                }
                const int32_t S = 2 * P - N;                     // S_t = sum_i delta_i
                float Delta;
                if (mode == DLION_ORACLE_AVERAGE) {
                    Delta = static_cast<float>(S) / static_cast<float>(N);   // R6
                } else if (mode == DLION_ORACLE_MAJORITY_TERNARY) {
                    Delta = (S > 0) ? 1.0f : ((S < 0) ? -1.0f : 0.0f);       // R3': sign(0) = 0
                } else {
                    Delta = (S >= 0) ? 1.0f : -1.0f;             // R2, R3
                }
                if (S >= 0) dword |= 1u << b;
                if (count) count[j] = static_cast<uint8_t>(P);
                const float xo = x[j];
                const float t1 = weight_decay * xo;
                const float t2 = Delta + t1;
                const float t3 = lr * t2;
                x[j] = xo - t3;                                  // Section 3.2, last eq.
            }
            if (delta_bits) delta_bits[w] = dword;
        }
    }
    return 0;
}

// Number of bit planes of the server->worker message: 1 for Majority Vote (Delta
// is binary); for Averaging the integer P in {0..N} takes ceil(log2(N+1)) bits
// (Section 3.2 "Communication Cost"; the paper rounds this to log N).
uint32_t dlion_oracle_delta_planes(uint32_t n_workers, int mode) {
    if (mode == DLION_ORACLE_MAJORITY) return 1;
    if (mode == DLION_ORACLE_MAJORITY_TERNARY) return 2;        // three values: two bits
    uint32_t bits = 0;
    while ((1ull << bits) < static_cast<uint64_t>(n_workers) + 1ull) ++bits;
    return bits;
}

// Analytic communication volume per step in BITS (Table 1 and Section 3.2
// "Communication Cost"), for d parameters and N workers.
//   direction 0: all workers -> server, N * d (one bit per parameter per worker)
//   direction 1: server -> one worker, d for Majority Vote; for Averaging an
//                integer in {0..N} per parameter, which takes ceil(log2(N+1))
//                bits (the paper rounds this to log N)
uint64_t dlion_oracle_wire_bits(uint64_t d, uint32_t n_workers, int mode, int direction) {
    if (direction == 0) return static_cast<uint64_t>(n_workers) * d;
    return d * dlion_oracle_delta_planes(n_workers, mode);
}

// Server side of Algorithm 1 alone: from the N binary vectors, the message that
// is broadcast to the workers.
//   Majority Vote: delta_wire[d_pad/32], bit j = 1 iff Delta_j = +1 (S_j >= 0, R2/R3).
//   Averaging:     K = ceil(log2(N+1)) planes, plane p at delta_wire + p*(d_pad/32):
//                  bit j of plane p = bit p of P_j (the integer in {0..N}, R4).
// Words that hold no parameter are left untouched; padding bits of written words are 0.
int dlion_oracle_aggregate(const dlion_oracle_segment* segs, uint32_t nseg, uint64_t d_pad,
                           uint32_t n_workers, int mode, const uint32_t* packed,
                           uint32_t* delta_wire) {
    if (!segs || !packed || !delta_wire || d_pad % 32 != 0 || n_workers == 0) return -1;
    if (!known_mode(mode)) return -1;
    const uint64_t W = d_pad / 32;
    const uint32_t K = dlion_oracle_delta_planes(n_workers, mode);
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t lo = segs[s].elem_offset;
        const uint64_t hi = lo + segs[s].numel;
        if (hi > d_pad || lo % 32 != 0) return -1;
        for (uint64_t w = lo / 32; w < (hi + 31) / 32; ++w) {
            for (uint32_t p = 0; p < K; ++p) delta_wire[p * W + w] = 0;
            for (uint32_t b = 0; b < 32; ++b) {
                const uint64_t j = w * 32 + b;
                if (j < lo || j >= hi) continue;
                uint32_t P = 0;
                for (uint32_t i = 0; i < n_workers; ++i) P += (packed[i * W + w] >> b) & 1u;
                if (mode == DLION_ORACLE_MAJORITY) {
                    if (2 * static_cast<int64_t>(P) - static_cast<int64_t>(n_workers) >= 0) delta_wire[w] |= 1u << b;
                } else if (mode == DLION_ORACLE_MAJORITY_TERNARY) {
                    const int64_t S3 = 2 * static_cast<int64_t>(P) - static_cast<int64_t>(n_workers);
                    const uint32_t code = (S3 > 0) ? 2u : ((S3 < 0) ? 0u : 1u);    // Delta + 1
                    delta_wire[w] |= (code & 1u) << b;
                    delta_wire[W + w] |= (code >> 1) << b;
                } else {
                    for (uint32_t p = 0; p < K; ++p) delta_wire[p * W + w] |= ((P >> p) & 1u) << b;
                }
            }
        }
    }
    return 0;
}

// The integer the server holds for each coordinate (Section 3.2: the sum of the
// binary vectors, read as the number of +1 votes, R4) written out as 16-bit
// values, for worker counts that do not fit the byte output of
// dlion_oracle_aggregate_apply.  count16[d_pad]; padding is left untouched.
int dlion_oracle_vote_counts16(const dlion_oracle_segment* segs, uint32_t nseg, uint64_t d_pad,
                               uint32_t n_workers, const uint32_t* packed, uint16_t* count16) {
    if (!segs || !packed || !count16 || d_pad % 32 != 0 || n_workers == 0 || n_workers > 65535) return -1;
    const uint64_t words = d_pad / 32;
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t first = segs[s].elem_offset;
        const uint64_t last = first + segs[s].numel;
        if (last > d_pad) return -1;
        for (uint64_t j = first; j < last; ++j) {
            uint32_t votes = 0;
            for (uint32_t worker = 0; worker < n_workers; ++worker) {
                votes += (packed[worker * words + j / 32] >> (j % 32)) & 1u;
            }
            count16[j] = static_cast<uint16_t>(votes);
        }
    }
    return 0;
}

// Worker side, first line of Algorithm 1's loop body: every worker applies the
// broadcast Delta, x <- x - eps (Delta + lambda x), decoding it from the wire
// format written by dlion_oracle_aggregate.
int dlion_oracle_apply_delta(const dlion_oracle_segment* segs, uint32_t nseg, uint64_t d_pad,
                             uint32_t n_workers, int mode, const uint32_t* delta_wire, float* x,
                             float lr, float weight_decay) {
    if (!segs || !delta_wire || !x || d_pad % 32 != 0 || n_workers == 0) return -1;
    if (!known_mode(mode)) return -1;
    const uint64_t W = d_pad / 32;
    const uint32_t K = dlion_oracle_delta_planes(n_workers, mode);
    const int32_t N = static_cast<int32_t>(n_workers);
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t lo = segs[s].elem_offset;
        const uint64_t hi = lo + segs[s].numel;
        if (hi > d_pad || lo % 32 != 0) return -1;
        for (uint64_t j = lo; j < hi; ++j) {
            float Delta;
            if (mode == DLION_ORACLE_MAJORITY) {
                Delta = ((delta_wire[j / 32] >> (j % 32)) & 1u) ? 1.0f : -1.0f;
            } else if (mode == DLION_ORACLE_MAJORITY_TERNARY) {
                const uint32_t low = (delta_wire[j / 32] >> (j % 32)) & 1u;
                const uint32_t high = (delta_wire[W + j / 32] >> (j % 32)) & 1u;
                Delta = static_cast<float>(static_cast<int32_t>(low + 2u * high) - 1);    // code - 1
            } else {
                int32_t P = 0;
                for (uint32_t p = 0; p < K; ++p) P |= static_cast<int32_t>((delta_wire[p * W + j / 32] >> (j % 32)) & 1u) << p;
                Delta = static_cast<float>(2 * P - N) / static_cast<float>(N);
            }
            const float xo = x[j];
            const float u1 = weight_decay * xo;
            const float u2 = Delta + u1;
            const float u3 = lr * u2;
            x[j] = xo - u3;
        }
    }
    return 0;
}

// Global Lion, the full-precision scheme the paper compares against (Appendix,
// "Global Lion Convergence", the scheme labelled Global Lion; Section 5.1 "G-Lion";
// Table 1 row "Global Lion/AdamW": 32 d bits each way).  Per coordinate:
//     mt_i  = beta1 m_i + (1-beta1) g_i                    (old m_i)
//     m_i  <- beta2 m_i + (1-beta2) g_i
//     G     = (1/N) sum_i mt_i
//     x    <- x - eps ( sign(G) + lambda x )
// Readings: R1 (binary32, one rounding per operation, no FMA) with the sum taken
// in worker order i = 0, 1, ..., N-1 starting from mt_0, then ONE division by
// (float)N; R2 for the sign (G >= 0 gives +1); every worker keeps its own m_i as
// the appendix scheme writes it (Section 5.1's "Lion on the averaged gradients" is
// the same sequence in exact arithmetic when all m_i start equal).
//   delta_bits [d_pad/32]  optional: bit = 1 iff sign(G) = +1, padding bits 0
// Returns 0, or -1 on a malformed argument.
int dlion_oracle_global_step(const dlion_oracle_segment* segs, uint32_t nseg, uint64_t d_pad,
                             uint32_t n_workers, int gdtype, const void* g, float* m, float* x,
                             uint32_t* delta_bits, float beta1, float beta2, float lr,
                             float weight_decay) {
    if (!segs || !g || !m || !x || d_pad % 32 != 0 || n_workers == 0) return -1;
    const float w1 = 1.0f - beta1;                               // R1: (1-beta) in binary32
    const float w2 = 1.0f - beta2;
    const float Nf = static_cast<float>(n_workers);
    for (uint32_t s = 0; s < nseg; ++s) {
        const uint64_t lo = segs[s].elem_offset;
        const uint64_t hi = lo + segs[s].numel;
        if (hi > d_pad || lo % 32 != 0) return -1;
        for (uint64_t w = lo / 32; w < (hi + 31) / 32; ++w) {
            uint32_t dword = 0;
            for (uint32_t b = 0; b < 32; ++b) {
                const uint64_t j = w * 32 + b;
                if (j < lo || j >= hi) continue;
                float total = 0.0f;
                for (uint32_t i = 0; i < n_workers; ++i) {
                    const size_t idx = static_cast<size_t>(i) * d_pad + j;
                    const float gf = load_grad(g, gdtype, idx);
                    const float mo = m[idx];
                    const float p1 = beta1 * mo;
                    const float q1 = w1 * gf;
                    const float mt = p1 + q1;                    // the blend each worker would send
                    total = (i == 0) ? mt : total + mt;          // fp32 sum in worker order
                    const float p2 = beta2 * mo;
                    const float q2 = w2 * gf;
                    m[idx] = p2 + q2;
                }
                const float G = total / Nf;
                const float Delta = (G >= 0.0f) ? 1.0f : -1.0f;
                if (G >= 0.0f) dword |= 1u << b;
                const float xo = x[j];
                const float v1 = weight_decay * xo;
                const float v2 = Delta + v1;
                const float v3 = lr * v2;
                x[j] = xo - v3;
            }
            if (delta_bits) delta_bits[w] = dword;
        }
    }
    return 0;
}

// 1 when this build honours the nthreads argument (OpenMP), else 0.
int dlion_oracle_has_openmp(void) {
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}

}  // extern "C"
