/*
 * hgrn2.h -- C ABI of the B200 (sm_100a) HGRN2 recurrence library.
 *
 * The library computes, per independent (batch, head) unit, the outer-product
 * state-expanded gated linear recurrence of the paper's Eq. 3 (multi-head variant,
 * Section 3.2), written with the state transposed (rows = gate dimension k,
 * columns = input dimension v):
 *
 *     S_t = Diag(f_t) S_{t-1} + (1 - f_t)^T i_t          S_t in R^{dk x dv}
 *     y_t = o_t S_t                                       (the updated state feeds y_t)
 *
 * i.e. linear attention with q = o, k = 1 - f, v = i and a per-key-dimension decay f
 * (Table 4).  Eq. 3 carries no 1/sqrt(d) scale and none is applied.
 *
 * Conventions common to every call
 *   - All data pointers are DEVICE pointers, 16-byte aligned, to dense row-major
 *     tensors; the library never allocates, frees or copies host memory, never
 *     synchronises, and enqueues work only on `cuda_stream` (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream).  The caller owns every buffer and
 *     must keep it alive until the stream has passed the call.
 *   - Sequence tensors are [B][H][N][d] with d innermost; o and f have d = dk, i, y
 *     and dy have d = dv.  Their element type is desc->io (float or bf16).
 *   - State tensors S0, SN, dS0, dSN, S are [B][H][dk][dv] float32, dv innermost.
 *   - f must lie in [0, 1]; the whole closed interval is supported by every call.  The
 *     tensor-core kernels rescale their operands by in-chunk cumulative decay, which they can
 *     represent only while the decay across each half of a 64-token chunk stays above 2^-100
 *     per key dimension (a gate that averages above ~0.12 over 32 steps).  A (batch, head) unit
 *     that leaves this range is detected on the device and redone, inside the same call, by
 *     pairwise-safe fp32 routines (exact, but two orders of magnitude slower for that unit);
 *     hgrn2_exact_path_units reports how many units a call handled that way.  d_f divides by
 *     f (f below 2^-100 is taken as 2^-100 there), so it loses accuracy as f -> 0.
 *   - Errors detected on the host (bad sizes, NULL or misaligned pointers, unsupported
 *     shapes, too small a workspace) are returned at once and nothing is launched.
 *     A failed launch returns HGRN2_ERR_CUDA.  Device-side problems (a bounded wait
 *     that ran out) are written to the status word at the start of `ws` and reported
 *     by hgrn2_poll after the caller has synchronised the stream.  Nothing aborts,
 *     traps or throws.
 *   - When B * H * N = 0 the sequence tensors have no elements and their pointers may be
 *     NULL; with N = 0 the calls copy S0 to SN (and dSN to dS0).
 *   - Supported shapes: dk, dv in {16, 32, 64, 128}; any B, H, N >= 1 (N = 0 is
 *     accepted and does nothing).  bf16 I/O with dk = dv = 128 runs on the tcgen05
 *     tensor-core kernels; everything else, and anything with
 *     HGRN2_FLAG_FORCE_ALU, runs on the fp32 CUDA-core kernels.
 */
#ifndef HGRN2_H_
#define HGRN2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HGRN2_OK = 0,
    HGRN2_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, negative size, bad enum */
    HGRN2_ERR_UNSUPPORTED = 2,   /* shape / dtype / chunk the kernels do not cover            */
    HGRN2_ERR_ALIGNMENT   = 3,   /* a pointer is not 16-byte aligned                          */
    HGRN2_ERR_WORKSPACE   = 4,   /* workspace missing                                         */
    HGRN2_ERR_CUDA        = 5,   /* a CUDA runtime call or launch failed                      */
    HGRN2_ERR_TIMEOUT     = 6,   /* device side: a bounded wait expired (status word)         */
    HGRN2_ERR_DOMAIN      = 7    /* device side: input outside the supported domain           */
} hgrn2_status;

typedef enum { HGRN2_F32 = 0, HGRN2_BF16 = 1 } hgrn2_dtype;

/* desc->flags */
#define HGRN2_FLAG_FORCE_ALU 1u  /* use the fp32 CUDA-core kernels even where tensor-core ones exist */
/* Debugging aid: every CTA of the tensor-core kernels starts as if its first device-side wait had just run out
 * of its 2 s (the abort flag that such a wait raises is raised from the start; the timer comparison itself is
 * not involved).  The call then takes the kernels' time-out exit - waits return at once, the load lanes stop
 * asking for tiles, what is in flight is allowed to land, tensor memory is released, the kernel returns - and
 * leaves HGRN2_ERR_TIMEOUT in the status word and unspecified values in its outputs (all writes stay inside
 * the caller's buffers).  Used to test that exit. */
#define HGRN2_FLAG_DEBUG_EXPIRE_WAITS 0x80000000u

/* Problem description shared by all calls.  `chunk` is the chunk length C of the
 * chunkwise-parallel form (an implementation parameter: results agree for every
 * supported value up to rounding); 0 selects the default. */
typedef struct hgrn2_desc {
    int32_t  B, H, N, dk, dv;
    int32_t  io;      /* hgrn2_dtype of o, f, i, y, dy, d_o, d_f, d_i */
    int32_t  chunk;
    uint32_t flags;
} hgrn2_desc;

/* Bytes of the `saved` buffer that hgrn2_fwd fills for hgrn2_bwd: the state at the
 * start of every chunk (derived from Eq. 3 by unrolling C steps) and, on the tensor-core
 * path, the two per-chunk decay totals of every key dimension.  On that path the layout is private
 * to the library and, for few long sequences that are not a whole number of chunks (which run as
 * segments), a little larger than one state per chunk: the size then depends on the current device,
 * and forward and backward of one buffer must run on devices with the same SM count.  0 on a bad desc. */
size_t hgrn2_saved_bytes(const hgrn2_desc *desc);

/* Bytes of the workspace `ws` every call takes: a 256-byte status block, room for the
 * saved data that hgrn2_bwd re-creates when it is given saved = NULL and, on the tensor-core
 * path, scratch for running each sequence as several segments when the batch has too few
 * (batch, head) units to fill the GPU (the size therefore depends on the current device) and
 * one dk x dv float matrix per unit for units redone on the exact path.  0 on a bad desc. */
size_t hgrn2_workspace_bytes(const hgrn2_desc *desc);

/* Forward over a whole sequence (Eq. 3 unrolled chunk by chunk; training and prefill).
 *   o, f [B][H][N][dk], i [B][H][N][dv]  in   (desc->io)
 *   S0   [B][H][dk][dv] float32          in,  NULL = zero initial state
 *   y    [B][H][N][dv]                   out  (desc->io)
 *   SN   [B][H][dk][dv] float32          out, NULL = not wanted
 *   saved  hgrn2_saved_bytes(desc) bytes out, NULL = inference (nothing kept for backward)
 *   ws     hgrn2_workspace_bytes(desc) bytes, scratch; its first word is the status word,
 *          which every call resets to HGRN2_OK on the stream before any of its work can report into it
 *          (a small asynchronous clear, or the first kernel of the call itself). */
hgrn2_status hgrn2_fwd(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                       const float *S0, void *y, float *SN, void *saved, void *ws,
                       void *cuda_stream);

/* Backward of hgrn2_fwd: the vector-Jacobian product for L = <dy, y> + <dSN, S_N>
 * (the paper delegates training to prior work and prints no backward; this is the
 * reverse-mode derivative of Eq. 3, run chunk by chunk in reverse).
 *   o, f, i, S0   as given to hgrn2_fwd
 *   dy  [B][H][N][dv] in;  dSN [B][H][dk][dv] float32 in, NULL = zero
 *   saved  the buffer hgrn2_fwd filled with the same desc, or NULL: the chunk states
 *          are then re-created inside `ws`
 *   d_o, d_f [B][H][N][dk], d_i [B][H][N][dv] out (desc->io).  d_f folds both paths of
 *          f: the decay and the tied input gate k = 1 - f.
 *   dS0 [B][H][dk][dv] float32 out, NULL = not wanted */
hgrn2_status hgrn2_bwd(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                       const float *S0, const void *dy, const float *dSN, const void *saved,
                       void *d_o, void *d_f, void *d_i, float *dS0, void *ws,
                       void *cuda_stream);

/* Variable-length (packed) batches.  Eq. 3 runs over each sequence separately - the state is reset to the
 * sequence's own initial state at every boundary - and a recurrent model's cost is linear in the tokens actually
 * present (Section 1: linear-time inference with a constant-size state), so ragged batches are passed packed
 * instead of padded to a common length:
 *   desc->B = number of sequences, desc->N = T, the total number of token rows per head, desc->H heads;
 *   o, f [H][T][dk], i, y, dy [H][T][dv] and the gradients likewise (desc->io), device memory, 16-byte aligned;
 *   cu_seqlens  int32[B + 1] in DEVICE memory, 4-byte aligned: sequence b occupies rows [cu[b], cu[b+1]) of every
 *               head; cu[0] = 0, non-decreasing, cu[B] <= T.  Empty sequences are allowed (their state passes
 *               through).  The offsets are read on the device only; malformed ones make the affected units write
 *               nothing and, on the tensor-core path, put HGRN2_ERR_INVALID_ARG into the status word.
 *   S0, SN, dSN, dS0 [B][H][dk][dv] float32: one state per (sequence, head), NULL as in hgrn2_fwd / hgrn2_bwd;
 *   saved  hgrn2_saved_bytes_varlen(desc) bytes (NULL as in hgrn2_fwd / hgrn2_bwd);
 *   ws     hgrn2_workspace_bytes_varlen(desc) bytes.
 * Everything else - ownership, streams, errors, the closed interval for f - is as for hgrn2_fwd / hgrn2_bwd.
 * One CTA serves one (sequence, head) unit, dispatched in index order: with more units than SMs, put long
 * sequences first.  With few units (no more than half the SMs; T > 512) every sequence runs as up to eight segments,
 * cut on the device; the two size queries then depend on the current device, and the boundary states SN and
 * dS0 come from the chaining of the segments' summaries (same tolerance, other rounding than hgrn2_fwd). */
size_t hgrn2_saved_bytes_varlen(const hgrn2_desc *desc);
size_t hgrn2_workspace_bytes_varlen(const hgrn2_desc *desc);
hgrn2_status hgrn2_fwd_varlen(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              const int32_t *cu_seqlens, const float *S0, void *y, float *SN,
                              void *saved, void *ws, void *cuda_stream);
hgrn2_status hgrn2_bwd_varlen(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              const int32_t *cu_seqlens, const float *S0, const void *dy,
                              const float *dSN, const void *saved, void *d_o, void *d_f, void *d_i,
                              float *dS0, void *ws, void *cuda_stream);

/* The layer's gate activations fused in front of the recurrence.  Eq. 1 forms the gates from dense projections,
 * o = sigmoid(.), i = SiLU(.), and Eq. 2 gives the forget gate a per-channel lower bound beta in [0, 1):
 *
 *     o = sigmoid(zo),      f = beta + (1 - beta) * sigmoid(zf),      i = silu(zi)
 *
 * These calls take the pre-activations and return y (forward) and the gradients with respect to the
 * pre-activations and to beta (backward), so the three gate tensors and their three gradients never make a round
 * trip through a framework's element-wise kernels, and f is never rounded to the I/O type (a bf16 f near 1 would
 * distort every decay product by 2^-9 / (1 - f)).
 *   zo, zf [B][H][N][dk], zi [B][H][N][dv]   in  (desc->io), device memory, 16-byte aligned
 *   beta   [H][dk] float32                   in, device memory, 16-byte aligned, values in [0, 1)
 *   S0, y, SN, dy, dSN, dS0                  as in hgrn2_fwd / hgrn2_bwd
 *   d_zo, d_zf [B][H][N][dk], d_zi [B][H][N][dv] out (desc->io)
 *   d_beta [H][dk] float32                   out, NULL = not wanted (summed over batch and time in a fixed order)
 *   saved  hgrn2_saved_bytes_gated(desc) bytes out of the forward / into the backward, NULL as in hgrn2_fwd /
 *          hgrn2_bwd (inference; re-created inside the workspace)
 *   ws     hgrn2_workspace_bytes_gated(desc) bytes
 * On the fp32 kernels the activations are applied in the load stage and their derivatives in the store stage.
 * On the tensor-core kernels (bf16, dk = dv = 128) one element-wise kernel in front writes o, i and the gate as
 * bf16 (kept in `saved`) - the gate as the smaller of f and 1 - f with a sign that says which, so that it is
 * resolved to 2^-9 of min(f, 1 - f) at both ends of [0, 1] - the recurrence kernels decode that, and one
 * element-wise kernel behind applies the chain rule in place and sums d_beta.
 * Ownership, streams and errors as for hgrn2_fwd / hgrn2_bwd. */
size_t hgrn2_saved_bytes_gated(const hgrn2_desc *desc);
size_t hgrn2_workspace_bytes_gated(const hgrn2_desc *desc);
hgrn2_status hgrn2_fwd_gated(const hgrn2_desc *desc, const void *zo, const void *zf, const void *zi,
                             const float *beta, const float *S0, void *y, float *SN, void *saved,
                             void *ws, void *cuda_stream);
hgrn2_status hgrn2_bwd_gated(const hgrn2_desc *desc, const void *zo, const void *zf, const void *zi,
                             const float *beta, const float *S0, const void *dy, const float *dSN,
                             const void *saved, void *d_zo, void *d_zf, void *d_zi, float *d_beta,
                             float *dS0, void *ws, void *cuda_stream);

/* Sequence (context) parallelism: a sequence cut into R consecutive spans, one per GPU.  Eq. 3 is linear in the
 * state and the state has constant size (Section 1), so one exchange of d_k + d_k d_v floats per unit and rank is
 * all the spans need of each other (the library itself never communicates; the caller all-gathers):
 *   1. hgrn2_span_summary_fwd on the rank's own span: S_loc = the span's end state from a ZERO start state,
 *      lam = the product of f over the span, per key dimension.  desc->N = tokens of the span.
 *        f [B][H][N][dk], i [B][H][N][dv] in (desc->io); S_loc [B][H][dk][dv], lam [B][H][dk] float32 out
 *   2. all-gather S_loc and lam into X_all [R][B][H][dk][dv], lam_all [R][B][H][dk] (the caller's collective)
 *   3. hgrn2_span_compose(desc, 0, r, 0, X_all, lam_all, S0, S_start): this rank's start state,
 *        S <- Diag(lam[r']) S + X[r']  for r' = 0 .. r-1, from init = the sequence's S0 (NULL = zero);
 *      with (0, R) it gives the sequence's final state
 *   4. hgrn2_fwd on the span with S0 = S_start.
 * Backward, mirrored: hgrn2_span_summary_bwd gives G_loc = the span's state gradient at its START from a zero
 * gradient at its end (o, f [..][dk], dy [..][dv] in); after the all-gather
 * hgrn2_span_compose(desc, r + 1, R, 1, G_all, lam_all, dSN, dS_end) folds r' = R-1 .. r+1 downwards from the
 * sequence's dS_N (NULL = zero), and hgrn2_bwd runs on the span with S0 = S_start, dSN = dS_end; with (0, R, 1)
 * the fold gives the sequence's dS_0.
 * r0 <= r' < r1 selects the spans folded; reverse = 0 ascending, 1 descending; an empty range copies init (or
 * writes zero).  ws: at least 256 bytes (status block).  Shapes and errors as for hgrn2_fwd; the summaries run on
 * the tensor cores for bf16, dk = dv = 128 and N a multiple of 64, on plain fp32 loops otherwise. */
hgrn2_status hgrn2_span_summary_fwd(const hgrn2_desc *desc, const void *f, const void *i, float *S_loc,
                                    float *lam, void *ws, void *cuda_stream);
hgrn2_status hgrn2_span_summary_bwd(const hgrn2_desc *desc, const void *o, const void *f, const void *dy,
                                    float *G_loc, float *lam, void *ws, void *cuda_stream);
hgrn2_status hgrn2_span_compose(const hgrn2_desc *desc, int32_t r0, int32_t r1, int32_t reverse,
                                const float *X_all, const float *lam_all, const float *init, float *out,
                                void *cuda_stream);

/* Largest chunk-state scratch, in bytes, that hgrn2_bwd_static_scratch can serve. */
#define HGRN2_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)

/* Backward pass that allocates nothing and asks the caller for no scratch.  (The paper has no
 * counterpart: this entry point exists for integration reasons only.)
 *
 * It is meant for callers that cannot obtain device memory at the point of the call: code that runs
 * inside a serving process whose memory pool already owns all of the GPU's memory, plug-ins that
 * are handed tensors but no allocator, and latency-critical loops where cudaMalloc / cudaFree are
 * off limits because they may synchronise the whole device.  Such a caller has neither a `saved`
 * buffer from the forward pass nor a workspace, so this variant of hgrn2_bwd re-creates the
 * chunk-start states in a fixed array of HGRN2_STATIC_SCRATCH_BYTES (+ a 256-byte status block)
 * that is compiled into the library; every GPU that loads the library holds that array until the
 * process exits.  The call itself performs no cudaMalloc, cudaFree or other allocating call.
 *
 * Arguments are those of hgrn2_bwd without `saved` and `ws`; results are those of hgrn2_bwd.
 *   status_out  device pointer to at least 8 bytes, 16-byte aligned, or NULL.  The device-side
 *               status word of the call is copied there on the stream, for hgrn2_poll.
 * Limits and caveats
 *   - hgrn2_workspace_bytes(desc) - 256 must not exceed HGRN2_STATIC_SCRATCH_BYTES (bf16 d = 128:
 *     B*H*(33 KB * ceil(N/64) + 64 KB) <= 32 MiB); larger problems return HGRN2_ERR_WORKSPACE and nothing
 *     is launched.  Use hgrn2_bwd with a caller-owned workspace for those.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in
 *     it.  Each call clears the status block and overwrites every state it later reads, so stale
 *     contents are never consumed; but two calls that can overlap on the GPU (different streams,
 *     or different host threads without ordering) race on the array and must be serialised by
 *     the caller.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress,
 *     with that device current).  Make that first call outside any stream capture.  With CUDA's
 *     lazy module loading this is also the moment the driver sets the array's memory aside, so
 *     make it early - a warm-up call per device at start-up, e.g. with N = 0 - while the device
 *     still has 32 MiB free: once a pool owns all memory the lookup fails with HGRN2_ERR_CUDA.
 * Errors: as hgrn2_bwd, plus HGRN2_ERR_WORKSPACE as above and HGRN2_ERR_CUDA if the address
 * lookup fails. */
hgrn2_status hgrn2_bwd_static_scratch(const hgrn2_desc *desc, const void *o, const void *f,
                                      const void *i, const float *S0, const void *dy,
                                      const float *dSN, void *d_o, void *d_f, void *d_i,
                                      float *dS0, void *status_out, void *cuda_stream);

/* One decode step for every unit (Eq. 3 once; constant-size state, Section 1).
 *   o, f [B][H][dk], i [B][H][dv] in (desc->io); desc->N is ignored
 *   S    [B][H][dk][dv] float32, updated in place
 *   y    [B][H][dv] out (desc->io), computed from the updated state */
hgrn2_status hgrn2_step(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                        float *S, void *y, void *cuda_stream);

/* desc->N successive decode steps in one launch (Eq. 3 applied N times; multi-token or speculative decoding):
 * the state of a unit is read once, stays on chip across the tokens and is written once, so the state traffic
 * per token falls N-fold (constant-size state, Section 1).  Results equal N calls of hgrn2_step bit for bit.
 *   o, f [B][H][N][dk], i [B][H][N][dv] in (desc->io), device memory, 16-byte aligned, caller-owned
 *   S    [B][H][dk][dv] float32, updated in place to the state after the last token
 *   y    [B][H][N][dv] out (desc->io), y_t computed from the state after token t
 * Supported: dk = dv in {64, 128}; anything else returns HGRN2_ERR_UNSUPPORTED.  N = 0 is a no-op.
 * Errors: HGRN2_ERR_INVALID_ARG (null pointer, bad descriptor), HGRN2_ERR_ALIGNMENT, HGRN2_ERR_CUDA (launch). */
hgrn2_status hgrn2_step_multi(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              float *S, void *y, void *cuda_stream);

/* Reads the device status word of `ws` (a device pointer) with a blocking copy.  Call it
 * after synchronising the stream the work ran on.  Returns HGRN2_OK, HGRN2_ERR_TIMEOUT,
 * HGRN2_ERR_DOMAIN, or HGRN2_ERR_CUDA if the copy itself failed. */
hgrn2_status hgrn2_poll(const void *ws);

/* Number of (batch, head) unit passes that the last tensor-core call using `ws` (a device pointer) redid on
 * the exact fp32 path because the unit's decay left the range described at the top of this file (Eq. 3 holds
 * on all of [0, 1]; the rescaled-operand form of the chunkwise products does not).  A backward that re-creates
 * its states (saved = NULL) counts a unit once for each of its two passes; few long sequences whose length is
 * not a whole number of 64-token chunks run as segments, each of which is redone and counted on its own.
 * Blocking copy: synchronise the
 * stream first.  0 on the fp32 kernels; -1 if `ws` is NULL or the copy failed. */
int32_t hgrn2_exact_path_units(const void *ws);

/* Static, human-readable name of a status code. */
const char *hgrn2_status_string(hgrn2_status s);

/* Chunk length the library will use for this desc (resolves chunk = 0); 0 on a bad desc. */
int32_t hgrn2_chunk(const hgrn2_desc *desc);

/* Name of the kernel family that serves this desc: "alu" or "tcgen05"; "" on a bad desc. */
const char *hgrn2_path(const hgrn2_desc *desc);

#ifdef __cplusplus
}
#endif
#endif /* HGRN2_H_ */
