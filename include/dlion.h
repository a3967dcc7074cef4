/*
 * dlion.h -- C ABI of the Distributed-Lion optimizer step for NVIDIA B200 (sm_100a).
 *
 * One optimizer step of Distributed Lion (arXiv 2404.00438, Algorithm 1 and
 * Section 3.2) over d parameters with N data-parallel workers, the N workers
 * held as N state slices on one GPU:
 *
 *   worker i :  delta_i = sign(beta1 m_i + (1-beta1) g_i)      (old m_i)
 *               m_i    <- beta2 m_i + (1-beta2) g_i
 *               delta_i is packed 32 signs per uint32: the 1-bit wire buffer
 *   server   :  S = sum_i delta_i ;  Delta = sign(S)  (Majority Vote)
 *                                    Delta = S / N    (Averaging)
 *   apply    :  x <- x - lr (Delta + lambda x)
 *
 * Conventions (the paper leaves them open; they are fixed here once):
 *   - all arithmetic is IEEE binary32, one rounding per operation, no fused
 *     multiply-add:  c = fl(fl(beta1*m) + fl((1-beta1)*g)), likewise m', and
 *     x' = fl(x - fl(lr*fl(Delta + fl(lambda*x)))); (1-beta) is formed in binary32;
 *     bf16 gradients are widened exactly;
 *   - sign(v) = +1 when v >= 0 (either zero), -1 otherwise (NaN gives -1);
 *   - an even-N tie (S = 0) gives Delta = +1 under Majority Vote (Delta = 0 under the
 *     optional DLION_MAJORITY_TERNARY rule);
 *   - the server's integer is P = number of +1 votes in {0..N}; S = 2P - N;
 *   - Averaging uses the correctly rounded quotient (float)(2P-N) / (float)N.
 *
 * Memory layout. Every buffer is DEVICE memory owned by the caller, unless a
 * parameter says "host".  Arenas are flat and worker-major:
 *     grads  [N][d_pad]     float or bf16 (dlion_gdtype)
 *     m      [N][d_pad]     float (or bf16, see dlion_set_momentum_dtype)
 *     packed [N][d_pad/32]  uint32; bit b of word w is coordinate 32*w+b; 1 = "+1"
 *     x      [d_pad]        float (all workers hold the same x, so one copy)
 * A segment table names the coordinates that are parameters: segment k covers
 * [elem_offset, elem_offset+numel).  elem_offset and d_pad are multiples of
 * DLION_ALIGN (128) elements, segments are ascending and do not overlap.
 * Coordinates outside every segment are padding: never read as parameters, never
 * written; packed words that hold no parameter are never written, and padding
 * bits inside a written word are 0.  Base pointers must be 16-byte aligned
 * (count_out: 4-byte).
 *
 * Calls that launch work are asynchronous on the given CUDA stream (a
 * cudaStream_t passed as void*; NULL = the default stream) and never
 * synchronise.  The context's device must be current.  A context is not
 * thread-safe: serialise calls on one context.  Nothing here throws,
 * aborts or traps: every failure is a status code.  No CPU fallback exists.
 */
#ifndef DLION_H_
#define DLION_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DLION_ALIGN 128u        /* elements: alignment of segment starts and of d_pad */
#define DLION_MAX_WORKERS 65535u /* up to 16 bit planes of votes */
#define DLION_MAX_WORKERS_BYTE_COUNTS 255u /* count_out of dlion_aggregate_apply (one byte per count) */
#define DLION_STATIC_MAX_COORD_WORKERS 134217728ull /* dlion_step_static: limit on N * d_pad */

typedef struct dlion_ctx dlion_ctx; /* opaque; host-side object */

typedef enum {
    DLION_OK = 0,
    DLION_EINVAL = 1, /* null pointer, value out of range, malformed segment table */
    DLION_EALIGN = 2, /* a pointer or offset violates the alignment rules above */
    DLION_ENOMEM = 3, /* host or device allocation failed */
    DLION_ECUDA = 4,  /* a CUDA runtime call or a kernel launch reported an error */
    DLION_ESTATE = 5  /* wrong device current, or context unusable */
} dlion_status;

/* Aggregation rule (Section 3.2).  DLION_MAJORITY_TERNARY is the optional other reading of
 * an even-N tie: the three-valued sign of the appendix's lemma, sign(0) = 0, so S = 0 gives
 * Delta = 0 and that coordinate's step is pure weight decay; with an odd N it is
 * DLION_MAJORITY.  Delta then has three values: the server->worker message is two planes
 * holding Delta + 1 in {0, 1, 2} (plane 0 = bit 0 = "tie", plane 1 = bit 1 = "S > 0"),
 * dlion_delta_planes is 2, and dlion_wire_bytes(ctx, 1) counts 2 d bits.  delta_bits_out of
 * dlion_aggregate_apply stays bit = (S >= 0). */
typedef enum { DLION_MAJORITY = 0, DLION_AVERAGE = 1, DLION_MAJORITY_TERNARY = 2 } dlion_mode;
typedef enum { DLION_GRAD_F32 = 0, DLION_GRAD_BF16 = 1 } dlion_gdtype;
typedef enum { DLION_STATE_F32 = 0, DLION_STATE_BF16 = 1 } dlion_sdtype;

typedef struct {
    uint64_t elem_offset; /* first coordinate, in elements, multiple of DLION_ALIGN */
    uint64_t numel;       /* number of parameters (0 allowed) */
} dlion_segment;

/* Host-only check of a segment table against the layout rules above.
 * Returns DLION_OK, DLION_EINVAL (null, nseg = 0, overlap, out of d_pad) or
 * DLION_EALIGN (offset or d_pad not a multiple of DLION_ALIGN).  Touches no GPU. */
dlion_status dlion_check_layout(const dlion_segment* segs, uint32_t nseg, uint64_t d_pad);

/* Algorithm 1 "Inputs": N, beta1, beta2 in [0,1], learning rate eps >= 0, weight
 * decay lambda >= 0, and the aggregation rule (Section 3.2).  Validates, then
 * copies the segment table and a 16-byte row per 4096-coordinate tile to the
 * current device (the only device memory the library owns: 0.1 % of x's size).  *out is set only on DLION_OK.
 * nseg = 1 with elem_offset = 0 describes a flat vector of d = numel. */
dlion_status dlion_init(dlion_ctx** out, const dlion_segment* segs, uint32_t nseg,
                        uint64_t d_pad, uint32_t n_workers, float beta1, float beta2,
                        float lr, float weight_decay, dlion_mode mode, dlion_gdtype gdtype);

/* Learning-rate schedules (the paper's CIFAR runs use a cosine schedule,
 * Section 5.1): sets eps for the following steps.  lr >= 0 and finite. */
dlion_status dlion_set_lr(dlion_ctx* ctx, float lr);

/* Storage type of the momentum arenas (default fp32).  With DLION_STATE_BF16 the
 * m buffers hold bf16: values are widened exactly on load, all arithmetic stays
 * binary32, and the new momentum is rounded to the nearest bf16, ties to even,
 * when stored (NaN stays NaN, payload unspecified).  Halves the optimizer state of every worker.
 * Call before the first step; x stays fp32.  dlion_step_static is fp32 only. */
dlion_status dlion_set_momentum_dtype(dlion_ctx* ctx, dlion_sdtype sdtype);

/* Algorithm 1 allows every worker its own beta1, beta2 (footnote to its inputs):
 * sets worker's pair, both in [0,1]; the others keep the values of dlion_init.
 * beta1 = beta2 makes that worker a Signum worker, beta1 = beta2 = 0 a signSGD
 * worker (Section 5.1 uses both as D-SIGNUM / D-SignSGD).  Allocates the
 * per-worker table on first use and copies it synchronously: call it outside
 * the step loop. */
dlion_status dlion_set_worker_betas(dlion_ctx* ctx, int worker, float beta1, float beta2);

/* Worker side of Algorithm 1 (the two worker-side assignments; same equations
 * in Section 3.2).  worker = -1: all N workers, pointers are the [N][...]
 * arenas.  worker = i in [0,N): that worker only, pointers are ITS slices
 * (grads[d_pad], m[d_pad], packed[d_pad/32]).
 *   grads   in     gradients g_{i,t}
 *   m       in/out momentum (float, or bf16 after dlion_set_momentum_dtype), updated in place
 *   packed  out    delta_{i,t}, 1 bit per coordinate (Table 1: d bits per worker) */
dlion_status dlion_worker_step(dlion_ctx* ctx, int worker, const void* grads, void* m,
                               uint32_t* packed, void* cuda_stream);

/* Server side of Algorithm 1 (aggregate(S_t), Section 3.2) fused with the
 * parameter update x <- x - eps (Delta + lambda x) (last equation of Section 3.2).
 *   packed          in     [N][d_pad/32], the N binary vectors
 *   x               in/out parameters, updated in place
 *   delta_bits_out  out, nullable  [d_pad/32]: bit = (S >= 0), i.e. Delta of
 *                   Majority Vote, the d-bit server->worker message of Table 1
 *   count_out       out, nullable  [d_pad] bytes: P, the integer in {0..N} that
 *                   Averaging sends back (Section 3.2 "Communication Cost");
 *                   N <= 255 only (DLION_EINVAL otherwise; dlion_aggregate has
 *                   the bit-plane form for any N) */
dlion_status dlion_aggregate_apply(dlion_ctx* ctx, const uint32_t* packed, float* x,
                                   uint32_t* delta_bits_out, uint8_t* count_out,
                                   void* cuda_stream);

/* dlion_aggregate_apply with the vote counts written as 16-bit values, for any N up to
 * DLION_MAX_WORKERS (the byte output stops at 255): the same vote and the same update.
 *   count16_out  out, required  [d_pad] uint16: P, the integer in {0..N} the server holds
 *                (Section 3.2 "Communication Cost"); 8-byte aligned; padding untouched */
dlion_status dlion_aggregate_apply_counts16(dlion_ctx* ctx, const uint32_t* packed, float* x,
                                            uint32_t* delta_bits_out, uint16_t* count16_out,
                                            void* cuda_stream);

/* Server side of Algorithm 1 ALONE (no parameter update): from the N binary
 * vectors, the message the server broadcasts (Section 3.2, "Communication
 * Cost"; Table 1, server->worker column).
 *   packed      in   [N][d_pad/32]
 *   delta_wire  out  dlion_delta_planes(ctx) planes of d_pad/32 words, plane p at
 *               delta_wire + p*(d_pad/32).  Majority Vote: one plane, bit = 1 iff
 *               Delta = +1.  Averaging: K = ceil(log2(N+1)) planes, bit j of plane
 *               p = bit p of P_j, the integer in {0..N} the paper describes; K*d
 *               bits in all.  Words that hold no parameter are not written;
 *               padding bits of written words are 0. */
dlion_status dlion_aggregate(dlion_ctx* ctx, const uint32_t* packed, uint32_t* delta_wire,
                             void* cuda_stream);

/* Worker side, first line of the loop body of Algorithm 1: every worker applies
 * the broadcast update, x <- x - eps (Delta + lambda x), with Delta decoded from
 * the message written by dlion_aggregate (Averaging: Delta = (2P-N)/N).
 * dlion_aggregate + dlion_apply_delta give exactly what dlion_aggregate_apply gives.
 *   delta_wire  in      as written by dlion_aggregate
 *   x           in/out  parameters */
dlion_status dlion_apply_delta(dlion_ctx* ctx, const uint32_t* delta_wire, float* x,
                               void* cuda_stream);

/* dlion_apply_delta for a message assembled by an all-gather.  When the server's work
 * is spread over S ranks (rank r votes on coordinate slice r and sends its part of the
 * message to everyone -- the 1-bit analogue of reduce-scatter + all-gather of the
 * exchange in Algorithm 1), the parts arrive slice after slice:
 *   delta_wire  in  [S][K][slice_words]: for slice r, its K = dlion_delta_planes(ctx)
 *               planes of slice_words words each (arena words r*slice_words ..), i.e.
 *               word j of plane p of slice r at delta_wire[(r*K + p)*slice_words + j]
 *   slice_words     words per slice; must divide d_pad/32 (DLION_EINVAL otherwise);
 *                   0 means the plane-major layout of dlion_apply_delta
 * Same update, same results; the parts are read where the collective put them. */
dlion_status dlion_apply_delta_sliced(dlion_ctx* ctx, const uint32_t* delta_wire, uint64_t slice_words,
                                      float* x, void* cuda_stream);

/* Number of d-bit planes of the server->worker message: 1 for Majority Vote,
 * ceil(log2(N+1)) for Averaging (the paper's "log(N) bits" per parameter), 2 for
 * DLION_MAJORITY_TERNARY.
 * 0 for a null context. */
uint32_t dlion_delta_planes(const dlion_ctx* ctx);

/* The whole of one Algorithm-1 iteration in ONE launch: a thread block holds a
 * tile of coordinates for all N workers, votes in registers and applies x.
 * Same results as dlion_worker_step(-1) followed by dlion_aggregate_apply.
 * N <= 255 (votes are counted in bytes); DLION_EINVAL beyond.
 *   packed_out  out, nullable: the wire buffer, if the caller still wants it. */
dlion_status dlion_step_fused(dlion_ctx* ctx, const void* grads, void* m, float* x,
                              uint32_t* packed_out, void* cuda_stream);

/* Global Lion, the full-precision scheme the paper compares Distributed Lion with
 * (appendix "Global Lion Convergence", the scheme labelled Global Lion; Section 5.1
 * "G-Lion"; Table 1 row "Global Lion/AdamW", 32 d bits each way), in one launch:
 *     mt_i = beta1 m_i + (1-beta1) g_i  (old m_i);   m_i <- beta2 m_i + (1-beta2) g_i
 *     x   <- x - eps ( sign( (1/N) sum_i mt_i ) + lambda x )
 * Arithmetic as in the conventions above: the sum is taken in binary32 in worker
 * order starting from mt_0, divided once by (float)N, and sign(v) = +1 for v >= 0.
 * It is here as the measured denominator of the comparison (time per step, and
 * dlion_wire_bytes(ctx, 2) for what it would send); the mode of the context is
 * not used.  fp32 momentum and one (beta1, beta2) for all workers only:
 * DLION_EINVAL after dlion_set_momentum_dtype(bf16) or dlion_set_worker_betas.
 *   grads [N][d_pad] in; m [N][d_pad] in/out; x [d_pad] in/out
 *   delta_bits_out  out, nullable  [d_pad/32]: bit = 1 iff the sign is +1 */
dlion_status dlion_step_global(dlion_ctx* ctx, const void* grads, float* m, float* x,
                               uint32_t* delta_bits_out, void* cuda_stream);

/* ---- Per-tensor mode -------------------------------------------------------------
 * Algorithm 1 steps a parameter vector x in R^d; in a training framework that vector is
 * a LIST of separately allocated tensors, with one gradient tensor each.  These calls
 * step such a list where it lies, without copying it into flat arenas: segment k of the
 * context's table is tensor k (its elem_offset only numbers its coordinates: the sign
 * words, Delta bits and the broadcast message stay flat buffers in that numbering).
 *
 * dlion_bind_tensors registers the tensors' device addresses:
 *   grads  host array [N][nseg] of device pointers: worker i's gradient of tensor k at
 *          grads[i*nseg + k]  (element type as dlion_init's gdtype)
 *   m      host array [N][nseg]: worker i's momentum of tensor k (float, or bf16 after
 *          dlion_set_momentum_dtype; set that first)
 *   x      host array [nseg]: the parameters (float)
 * A null ARRAY keeps that table as it was bound before (gradients usually move from
 * step to step, parameters and momenta do not); at least one must be given.  Every
 * tensor must hold its segment's numel elements and start on a 16-byte boundary
 * (DLION_EALIGN otherwise; a null tensor pointer is accepted only for numel = 0, else
 * DLION_EINVAL); nothing is changed when a pointer is rejected.  The tables are copied
 * into device memory the context owns (allocated on the first call, (2N+1)*nseg
 * pointers), asynchronously on cuda_stream, in order with the steps issued after it on
 * the same stream; the host arrays may be reused as soon as the call returns.
 * Coordinates between one tensor's end and the next segment's start do not exist in
 * this mode; nothing is read or written outside the tensors. */
dlion_status dlion_bind_tensors(dlion_ctx* ctx, const void* const* grads, void* const* m,
                                float* const* x, void* cuda_stream);

/* dlion_worker_step on the bound gradient and momentum tensors (worker = -1: all N;
 * worker = i: that worker's tensors only, packed then being ITS [d_pad/32] slice).
 * DLION_ESTATE until gradients and momenta have been bound. */
dlion_status dlion_worker_step_tensors(dlion_ctx* ctx, int worker, uint32_t* packed, void* cuda_stream);

/* dlion_aggregate_apply on the bound parameter tensors (packed [N][d_pad/32] as there;
 * delta_bits_out nullable).  DLION_ESTATE until parameters have been bound. */
dlion_status dlion_aggregate_apply_tensors(dlion_ctx* ctx, const uint32_t* packed,
                                           uint32_t* delta_bits_out, void* cuda_stream);

/* dlion_apply_delta_sliced (slice_words = 0: dlion_apply_delta) on the bound parameter
 * tensors.  DLION_ESTATE until parameters have been bound. */
dlion_status dlion_apply_delta_tensors(dlion_ctx* ctx, const uint32_t* delta_wire, uint64_t slice_words,
                                       void* cuda_stream);

/* ---- Scatter mode: the worker -> server send fused into the worker-side kernel -------
 * In Algorithm 1 every worker "sends delta_{i,t} to the server".  When the server's work
 * is spread over S ranks (rank r votes on coordinate slice r), worker i's d bits are cut
 * into S slices and slice r must reach rank r: an all-to-all.  In this mode the
 * worker-side kernel stores each sign word straight into the receive buffer of the
 * slice it belongs to, so that exchange needs no pass of its own.  On a multi-GPU job
 * the buffers are the peers' memory mapped into this process: the kernel only ever
 * STORES to them (plain stores; no loads from a peer, no multicast); the caller orders
 * the vote after every worker's kernel (a barrier) as it would after an all-to-all.
 *
 * dlion_bind_scatter (once, outside the step loop; copies synchronously):
 *   dst          host array [n_dst] of device pointers: dst[r] = receive buffer of slice r,
 *                uint32 [rows][slice_words], 16-byte aligned
 *   slice_words  words per slice; n_dst * slice_words must equal d_pad/32
 *   slot, rows   this worker's row in every receive buffer (slot < rows)
 * dlion_worker_step_scatter(worker = i): dlion_worker_step for ONE worker (grads and m are
 * its slices), sign word w of the arena numbering going to
 * dst[w / slice_words][slot * slice_words + w % slice_words].  Words that hold no
 * parameter are not written, as in the arena form.  DLION_ESTATE until bound. */
dlion_status dlion_bind_scatter(dlion_ctx* ctx, uint32_t* const* dst, uint32_t n_dst, uint64_t slice_words,
                                uint32_t slot, uint32_t rows);
dlion_status dlion_worker_step_scatter(dlion_ctx* ctx, int worker, const void* grads, void* m,
                                       void* cuda_stream);

/* One whole step with the gradients in HOST memory (pinned memory makes the
 * copies asynchronous).  Worker i's gradients are copied to the device while
 * worker i-1's are being consumed by the worker-side kernel; after the last
 * worker the server-side kernel runs and, if asked, Delta is copied back.
 *   host_grads      in, host   [N][d_pad] gradients
 *   m, x, packed    device     as above (packed is used as the wire buffer)
 *   staging         device     2 * d_pad gradient elements (two slices)
 *   delta_wire_dev  device, nullable  the broadcast message in the format of
 *                   dlion_aggregate: dlion_delta_planes(ctx) planes of d_pad/32 words
 *                   (one plane of Delta bits for Majority Vote, the K count planes
 *                   for Averaging; any N)
 *   host_delta_out  out, host, nullable: copy of delta_wire_dev (planes * d_pad/8
 *                   bytes); needs delta_wire_dev.  Complete when cuda_stream's work is.
 * Every argument is checked before anything is enqueued: a rejected call leaves
 * m, packed and x untouched.
 * Uses one internal copy stream ordered against cuda_stream by events. */
dlion_status dlion_step_host(dlion_ctx* ctx, const void* host_grads, void* m, float* x,
                             uint32_t* packed, void* staging, void* delta_wire_dev,
                             void* host_delta_out, void* cuda_stream);

/* (No counterpart in the paper: an entry point for callers that cannot allocate.)
 * One two-stage step -- the worker-side kernel for all N workers, then the
 * server-side kernel -- on a flat vector of d parameters, without dlion_init and
 * without a caller-supplied wire buffer.  It is meant for callers that must not
 * call cudaMalloc where they step the optimizer: a host whose allocator already
 * owns all device memory, a latency-critical loop that cannot take cudaMalloc's
 * device-wide synchronisation, or a plug-in restricted to the buffers it is
 * handed.  The 1-bit wire buffer is a fixed 16 MiB array inside the library image
 * (held, until the process exits, by every GPU on which the library's device
 * code has been loaded), and a flat vector needs no tile table.
 * The FIRST call on a device is a set-up call: the CUDA runtime loads the
 * library's device code then (which is when the array is reserved, and can fail
 * with DLION_ECUDA if the device is already full) and the array's device address
 * is looked up, with that device current.  Make it at start-up, before another
 * allocator takes the remaining memory and before any stream capture begins.
 * Every later call allocates nothing, on host or device.
 *   d, n_workers   the problem; d_pad = d rounded up to DLION_ALIGN, and
 *                  n_workers * d_pad <= DLION_STATIC_MAX_COORD_WORKERS, else
 *                  DLION_EINVAL ("does not fit the fixed scratch")
 *   grads [N][d_pad], m [N][d_pad] (in/out), x [d_pad] (in/out): device, 16-byte
 *                  aligned, as for dlion_worker_step(-1) / dlion_aggregate_apply
 * Results are those of dlion_worker_step(-1) + dlion_aggregate_apply with the
 * same hyper-parameters (fp32 momentum, one beta pair).  All calls on a device
 * share the array and it keeps the last call's bits: every word the step reads is
 * rewritten first, so nothing needs clearing, but two calls that overlap on the
 * GPU (different streams, no ordering) race on it and give undefined results. */
dlion_status dlion_step_static(uint64_t d, uint32_t n_workers, float beta1, float beta2,
                               float lr, float weight_decay, dlion_mode mode,
                               dlion_gdtype gdtype, const void* grads, float* m, float* x,
                               void* cuda_stream);

/* Analytic communication volume per step in bytes (Table 1; Section 3.2
 * "Communication Cost"), d = number of parameters:
 *   direction 0, all workers -> server:  N * d / 8
 *   direction 1, server -> one worker:   d / 8 (Majority Vote), or
 *                                        d * ceil(log2(N+1)) / 8 (Averaging)
 *   direction 2: what one worker moves each way when fp32 gradients are
 *                exchanged instead (Table 1, "Global Lion/AdamW": 32 d bits)
 * Rounded up to whole bytes.  Returns 0 for a null context or bad direction. */
uint64_t dlion_wire_bytes(const dlion_ctx* ctx, int direction);

/* Number of kernels this context has launched so far. */
uint64_t dlion_launch_count(const dlion_ctx* ctx);

/* Static, human-readable name of a status code. */
const char* dlion_status_str(dlion_status s);

/* Frees the context and its device table.  Pending work must have completed. */
void dlion_destroy(dlion_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* DLION_H_ */
