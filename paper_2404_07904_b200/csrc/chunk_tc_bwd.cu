// Chunkwise HGRN2 backward on the Blackwell tensor cores (tcgen05 + TMEM + TMA), bf16 I/O, fp32
// state gradient, d_k = d_v = 128, chunk length C = 64 (frame and notation: tc_chunk.cuh).
//
// Reverse sweep over the chunks with the state gradient resident in tensor memory.  In the mid frame,
// with dS'' = Diag(E) dS_out and S' the saved forward state of the chunk:
//
//   A  = tril(Qs Ks^T)          dA = tril(dY V^T)
//   dQs^T       = Ks^T dA^T + S' dY^T            (accumulator [key dim][t])
//   dKs_intra^T = Qs^T dA                        (accumulator [key dim][s])
//   dKs_inter^T = dS'' V^T                       (accumulator [key dim][s])
//   dV^T        = dY^T A + dS''^T Ks^T           (accumulator [value dim][s])
//   dS'         = dS'' + Qs^T dY,   dS_in = Diag(Pm) dS'
//   a = Qs*dQs - Ks*dKs_intra,  e = Ks*dKs_inter,  R_k = sum_v dS''[k,v] S'[k,v]
//   dg_t = sum_{j>=t} a_j + sum_{s<t} e_s + R            (gradient w.r.t. log f_t)
//   d_o = dQs * exp(b_t - b_m),  dk = (dKs_intra + dKs_inter) * exp(b_m - b_s),  d_f = dg / f - dk
//
// Every accumulator that feeds an output puts one key (or value) dimension in each TMEM lane, so the
// thread that owns the lane sees a whole column of the chunk: the scans along time stay in registers
// and each output store of a warp covers 64 contiguous bytes of one token row.
//
// Warp roles (hand-offs are mbarriers, every wait is bounded; loops stay rolled to keep the
// instruction footprint of the concurrently running roles small):
//   T   4 warps: raw o, f tiles -> Qs, Ks in place, one chunk ahead (two TMA stages); paced so that it does not
//       run alongside the output walk two chunks back;
//   E1  4 warps: rescale the dS accumulator and publish its bf16 copy dS'' (the chain between chunks), R;
//   E3  8 warps: d_o and d_f from dQs^T, dKs_intra^T, dKs_inter^T.  A thread owns (key dim, half of the chunk)
//       and walks its 32 steps outwards from the middle, carrying the decay product and one running sum;
//       what is still missing then is one constant per key dimension (R plus the two halves' sums), so the
//       almost finished d_f and 1/f are parked in the TMEM columns just read, and once all eight warps are
//       through each thread completes its own 32 rows.  It works from a second, unswizzled copy of raw o and f
//       and recomputes Qs, Ks with the transform's roundings, so the operand stage is free as soon as the
//       chunk's products are done;
//   O   4 warps: the causal masks of A and dA into operand slabs (32 rows per warp), and d_i from dV^T;
//   L   1 warp: TMA loads (o, f, dy stage; v; saved S'; raw o, f), each refilled when its last reader is done;
//   MX, MY1, MY2  1 warp each: tcgen05.mma issue of the groups below (one lane issuing all 56
//       products of a chunk is itself a bottleneck: its instruction stream is long and serial).
// Per chunk the tensor pipe runs, each group as soon as what it overwrites has been read out
//   X  (MX) : dS' += Qs^T dY | A | dA      (overlaps the outputs of the previous chunk)
//   Y1a (MY1): dV^T = dS''^T Ks^T           (needs the previous chunk's d_i out: early)
//   Y1b (MY1): dKs_inter^T                  (needs the previous chunk's output walk finished)
//   Y2a (MY2): dV^T += dY^T A               (needs tril(A), and Y1a complete)
//   Y2b (MY2): dQs^T | dKs_intra^T          (needs tril(dA), S', and the previous chunk's parked values consumed)
// Event stamps of one CTA put the chunk period at: output walk (3.7 k cycles) -> completion of d_f (1.3 k) ->
// Y2b (1.1 k) -> next walk; with a single Y1 group behind the walk and the masks and the completion pass in the
// other roles' hands the same stamps showed a second, equally long chain through Y1 and Y2.
//
// Tensor-memory plan (512 columns, no spare): dS [0,128); A [128,192) in lanes 0..63 and dA [192,256) in
// lanes 64..127 (products of the stacked operand (Qs; dY), M = 128); dQs^T [256,320); dKs_intra^T [320,384);
// dKs_inter^T [384,448); dV^T [448,512).
#include "chunk_alu.cuh"
#include "tc_chunk.cuh"

namespace hgrn2 {

namespace {

using namespace tc;

constexpr int kTWarps = 4, kE1Warps = 4, kE3Warps = 8, kOWarps = 4;
constexpr int kE1Threads = kE1Warps * 32, kE3Threads = kE3Warps * 32, kOThreads = kOWarps * 32;
constexpr int kWarpE1 = kTWarps, kWarpE3 = kWarpE1 + kE1Warps, kWarpO = kWarpE3 + kE3Warps;
constexpr int kWarpLoad = kWarpO + kOWarps, kWarpMmaX = kWarpLoad + 1, kWarpMmaY1 = kWarpLoad + 2,
              kWarpMmaY2 = kWarpLoad + 3;
constexpr int kThreads = (kWarpMmaY2 + 1) * 32;

constexpr int kStages = 2;
constexpr uint32_t kStageBytes = 3 * kTile;                       // q, dy, f: free again when the chunk's products are done
// Stage layout: [q slab 0][dy slab 0][q slab 1][dy slab 1][f slab 0][f slab 1].  With the slabs of q and dy
// interleaved, (Qs; dY) also reads as ONE 128-row K-major operand whose slabs are 16 KB apart.
constexpr uint32_t kSS = 2 * kSlab;                               // distance between the two slabs of the q and dy tiles
constexpr uint32_t kOffQ = 0, kOffG = kSlab, kOffK = 2 * kTile;
constexpr uint32_t kOffV = kStages * kStageBytes;                 // v: one buffer, free when X and Y1 of the chunk are done
constexpr uint32_t kOffS = kOffV + kTile;                         // S' (bf16, from the forward)
constexpr uint32_t kOffDS = kOffS + kStateTile;                   // bf16 copy of dS''
constexpr uint32_t kOffP = kOffDS + kStateTile;                   // bf16 tril(A)
constexpr uint32_t kOffDP = kOffP + kSlab;                        // bf16 tril(dA)
constexpr uint32_t kOffRawO = kOffDP + kSlab;                     // raw o and f of the chunk, plain [64][128] bf16, for
constexpr uint32_t kOffRawF = kOffRawO + kTile;                   // the output warps (the stage holds Qs, Ks by then)
constexpr uint32_t kOffR = kOffRawF + kTile;                      // float rr[2][128]
constexpr uint32_t kOffX = kOffR + 2 * 128 * 4;                   // float xa[128], xe[128]
constexpr uint32_t kOffCtl = kOffX + 2 * 128 * 4;
constexpr uint32_t kSmemBytes = kOffCtl + 256;                    // no slack: the base must be 1024-byte aligned

constexpr uint32_t kColDS = 0, kColA = 128, kColDA = 192, kColDQ = 256, kColDKi = 320, kColDKx = 384, kColDV = 448;

struct Ctl {
    uint64_t full[kStages];       // TMA (o, f, dy tiles) -> T, M
    uint64_t vfull;               // TMA (v tile) -> M
    uint64_t rawfull;             // TMA (second, unswizzled copy of o and f) -> E3
    uint64_t raw_read;            // E3 -> L: the raw copies have been read for the last time
    uint64_t t_done[kStages];     // T -> M, E1
    uint64_t sfull;               // TMA (saved S') -> E1, M
    uint64_t m_done;              // E1 -> M: dS'' is in TMEM and in shared memory
    uint64_t barX;                // tcgen05.commit -> E1, O, L: dS' update, A, dA complete
    uint64_t pd_ready;            // O -> M: tril(A), tril(dA) are in shared memory
    uint64_t barY1a;              // tcgen05.commit -> MY2: dV^T = dS''^T Ks^T complete
    uint64_t barY1;               // tcgen05.commit -> E1, L, MY2: both products of dS'' complete (its copy and v no longer read)
    uint64_t barY2;               // tcgen05.commit -> E3, O, L: every product of the chunk complete
    uint64_t r_ready[2];          // E1 -> E3, L: R of the chunk is in shared memory, S' no longer read by threads
                                  // (two barriers: the slower of the two waiters must not be lapped)
    uint64_t acc_free1;           // E3 -> M: dKs_inter^T has been read out
    uint64_t acc_freeV;           // O -> M: dV^T has been read out
    uint64_t parked;              // E3 -> E3: every thread's parked values and the halves' sums are in place
    uint64_t acc_free2;           // E3 -> M: dQs^T and dKs_intra^T columns are free again
    uint64_t drain;               // tcgen05.commit (MX, MY1, MY2, after their loops): every product issued has completed
    int abort_flag;               // set by the first wait that runs out: every later wait returns at once
    uint32_t tmem_base;
    int o_done;                   // E3 -> T: output walks finished so far, counted per warp (pacing only)
    int exact_flag;               // E1: a decay of this CTA's tokens left the range of the rescaled operands
    int l_stage, l_v, l_state, l_raw;   // L: fills asked for so far, per buffer, for the abort epilogue
};
static_assert(sizeof(Ctl) <= 256, "control block");
static_assert(kSmemBytes <= 232448, "shared memory budget");

constexpr int kExactC = 32;       // chunk length of the exact fp32 routines at d = 128 (their shared-memory budget)
static_assert(alu::bwd_smem_floats(kD, kD, kExactC) * sizeof(float) <= kSmemBytes, "exact path fits the CTA's shared memory");

// d_o and the nearly finished d_f of one thread: key dimension k, local times [32 * kUp, 32 * kUp + 32),
// walked outwards from the middle of the chunk in blocks of four rows (a short loop body: the role shares its
// scheduler's instruction stream with four others).  Returns this half's sums of a and e.
// do_g points at element (row 0 of the chunk, column k) of d_o in global memory.  oraw, fraw: the chunk's raw
// o and f as plain [64][128] bf16 tiles (rows beyond the end of the sequence hold zeros, or in a packed batch
// the next sequence's tokens: they are patched to the neutral f = 1, o = 0).  Qs and Ks are recomputed from
// them with the transform's own roundings, so the operand stage does not have to be held until the outputs
// are done.  The role is bound by its instruction count: per element one reciprocal (1/f is the ratio of two
// consecutive products), fused packed multiply-adds, and a single running sum.
template <bool kUp, bool kRagged, bool kEnc>
__device__ __forceinline__ void phase_main(uint32_t tmem_lane, const __nv_bfloat16 *oraw, const __nv_bfloat16 *fraw,
                                           int k, __nv_bfloat16 *do_g, int n_valid, float &asum, float &esum)
{
    float cp = 1.f, ci = 1.f;       // running product of f between the middle and the current row, and its reciprocal
    float W = 0.f;                  // running sum of a - e over the rows visited so far
    float2 Gp = make_float2(0.f, 0.f);   // sum of a over the rows visited so far, even and odd rows apart
#pragma unroll 1
    for (int b = 0; b < 8; ++b) {
        const int t0 = kUp ? 32 + 4 * b : 28 - 4 * b;          // lowest row of the block (a multiple of 4)
        uint32_t x[4], y[4], z[4];
        tmem_ld4(tmem_lane + kColDQ + t0, x);
        tmem_ld4(tmem_lane + kColDKi + t0, y);
        tmem_ld4(tmem_lane + kColDKx + t0, z);
        uint32_t fw[4], qw[4];         // raw bf16 bits
        float fv[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = t0 + j;
            fw[j] = reinterpret_cast<const unsigned short *>(fraw)[t * kD + k];
            qw[j] = reinterpret_cast<const unsigned short *>(oraw)[t * kD + k];
            if (kRagged && t >= n_valid) { fw[j] = kEnc ? 0x8000u : 0x3F80u; qw[j] = 0u; }
            if (kEnc) {                       // fw[j] becomes the bf16 bits of k, as the transform formed them
                float kv;
                gate_decode(fw[j], fv[j], kv);
                fw[j] = pack_bf16(kv, 0.f) & 0xFFFFu;        // rounded to bf16 exactly as the transform rounds it
            } else {
                fv[j] = __uint_as_float(fw[j] << 16);
            }
        }
        tmem_wait_ld();
        // Scale factors along the walk (sequential in the running product) and 1/f.  No floor here: a product
        // that would need one has put the unit on the exact path already (the totals the state warps test are
        // never larger than any product formed here), and what this pass writes for such a unit is overwritten.
        // 1/f is the ratio of two consecutive products, so one reciprocal per element serves both.
        float sq[4], sk[4], rf[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = kUp ? i : 3 - i;                      // visiting order: away from the middle
            const float c0 = cp, i0 = ci;
            cp *= fv[j];
            ci = rcp_fast(cp);
            sq[j] = kUp ? cp : i0;
            sk[j] = kUp ? ci : c0;
            rf[j] = kEnc ? rcp_fast(fmaxf(fv[j], kFDivMinK)) : c0 * ci;
        }
        // element-wise part, two rows per instruction (packed fp32)
        float w[4], dk[4];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const int j = 2 * p;
            const float2 X = make_float2(__uint_as_float(x[j]), __uint_as_float(x[j + 1]));
            const float2 Y = make_float2(__uint_as_float(y[j]), __uint_as_float(y[j + 1]));
            const float2 Z = make_float2(__uint_as_float(z[j]), __uint_as_float(z[j + 1]));
            // Qs and -Ks of the two rows exactly as the transform warps rounded them for the products: the terms
            // of a cancel in pairs along the chunk only if both sides use the same operand values
            const uint32_t sqp = pack_bf16(sq[j], sq[j + 1]), skp = pack_bf16(sk[j], sk[j + 1]);
            const uint32_t qsp = mul_bf16x2(qw[j] | (qw[j + 1] << 16), sqp);
            const uint32_t ksn = kEnc ? mul_bf16x2(fw[j] | (fw[j + 1] << 16), skp ^ 0x80008000u)
                                      : fma_bf16x2(fw[j] | (fw[j + 1] << 16), skp, skp ^ 0x80008000u);
            const float2 QS = make_float2(bf16_lo(qsp), bf16_hi(qsp)), KSn = make_float2(bf16_lo(ksn), bf16_hi(ksn));
            const float2 dox = mul2(X, make_float2(sq[j], sq[j + 1]));
            const float2 a2 = fma2(KSn, Y, mul2(QS, X));
            const float2 w2 = fma2(KSn, Z, a2);                 // a - e
            Gp = add2(Gp, a2);
            const float2 dk2 = mul2(add2(Y, Z), make_float2(sk[j], sk[j + 1]));
            if (!kRagged || t0 + j < n_valid) do_g[(size_t)(t0 + j) * kD] = __float2bfloat16_rn(dox.x);
            if (!kRagged || t0 + j + 1 < n_valid) do_g[(size_t)(t0 + j + 1) * kD] = __float2bfloat16_rn(dox.y);
            w[j] = w2.x; w[j + 1] = w2.y;
            dk[j] = dk2.x; dk[j + 1] = dk2.y;
        }
        // With K = R + (sum of a over the second half) + (sum of e over the first half), which the final pass
        // adds, dg_t = K - sum_{32 <= s < t} (a_s - e_s) after the middle and K + sum_{t <= j < 32} (a_j - e_j)
        // before it: one running sum along the walk
        float u[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = kUp ? i : 3 - i;
            if (kUp) {
                u[j] = fmaf(-W, rf[j], -dk[j]);
                W += w[j];
            } else {
                W += w[j];
                u[j] = fmaf(W, rf[j], -dk[j]);
            }
        }
        // park u and 1/f in the columns just read
        tmem_st4(tmem_lane + kColDQ + t0, u);
        tmem_st4(tmem_lane + kColDKi + t0, rf);
    }
    asum = Gp.x + Gp.y;
    esum = asum - W;
}

// kRagged: N is not a whole number of chunks (the tail chunk is padded with neutral tokens); when false,
// every per-row validity test below folds away.
// kMultiCta: a unit runs as several CTAs (segments) of this launch (see the forward kernel).
// kEnc: the f tensor holds the signed gate encoding (see transform_half); d_f stays the gradient with respect to f.
template <bool kRagged, bool kMultiCta, bool kEnc>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_f,
              const __grid_constant__ CUtensorMap map_i, const __grid_constant__ CUtensorMap map_dy,
              const __grid_constant__ CUtensorMap map_saved, const __grid_constant__ CUtensorMap map_o_raw,
              const __grid_constant__ CUtensorMap map_f_raw, const float *__restrict__ totals,
              const float *__restrict__ dSN, __nv_bfloat16 *__restrict__ d_o, __nv_bfloat16 *__restrict__ d_f,
              __nv_bfloat16 *__restrict__ d_i, float *__restrict__ dS0, int N_all, int NC_all, StatusBlock *status,
              int clear_status, const ExactArgs ex, const PackedArgs pk, int start_aborted)
{
    // the first kernel of a call zeroes the status word; the only early report, the alignment check below, is the
    // same in every CTA, so CTA 0 repeats it after its own clear
    if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) {
        status->code = 0;
        status->where = 0;
        status->exact_units = 0;
    }
    extern __shared__ __align__(1024) uint8_t smem[];
    if (smem_u32(smem) & 1023u) {          // every byte is spoken for: the swizzled tiles need the base aligned
        if (threadIdx.x == 0) report_error(status, HGRN2_ERR_CUDA, 3);
        return;
    }
    uint8_t *sbuf = smem + kOffS;
    uint8_t *dsbuf = smem + kOffDS;
    uint8_t *pbuf = smem + kOffP;
    uint8_t *dpbuf = smem + kOffDP;
    const __nv_bfloat16 *oraw = reinterpret_cast<const __nv_bfloat16 *>(smem + kOffRawO);
    const __nv_bfloat16 *fraw = reinterpret_cast<const __nv_bfloat16 *>(smem + kOffRawF);
    uint8_t *vbuf = smem + kOffV;
    float *rr = reinterpret_cast<float *>(smem + kOffR);
    float *xa = reinterpret_cast<float *>(smem + kOffX);
    float *xe = xa + 128;
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + kOffCtl);
    volatile int *abort_flag = &ctl->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int u = blockIdx.x;
    // This CTA's sequence: rows [row0, row0 + N) of plane zu of the [planes][rows][128] tensors, NC chunks, chunk-start
    // state c in slot slot0 + c.  Packed batches (ragged instantiations only) read theirs from the offsets array.
    int row0 = 0, zu = u, N = N_all, NC = NC_all;
    size_t slot0 = (size_t)u * NC_all;
    if constexpr (kRagged) {
        if (pk.cu != nullptr) {
            const int b = u / pk.H;
            zu = u - b * pk.H;
            row0 = __ldg(pk.cu + b);
            N = __ldg(pk.cu + b + 1) - row0;
            NC = (N + kC - 1) / kC;
            slot0 = (size_t)zu * pk.slots_per_head + row0 / kC + b;
            if (row0 < 0 || N < 0 || row0 + N > N_all) {          // malformed offsets: report, touch nothing
                if (tid == 0) report_error(status, HGRN2_ERR_INVALID_ARG, 4);
                return;
            }
            if (N <= 0) {                // empty sequence: the state gradient passes through
                if (dS0 != nullptr)
                    for (int x = tid; x < kD * kD; x += kThreads)
                        dS0[(size_t)u * kD * kD + x] = dSN ? dSN[(size_t)u * kD * kD + x] : 0.f;
                return;
            }
        }
    }
    const size_t grow0 = (size_t)zu * N_all + row0;                 // first row of the sequence in the [planes * rows][128] view

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->t_done[s], kTransformThreads);
        }
        mbar_init(&ctl->vfull, 1);
        mbar_init(&ctl->rawfull, 1);
        mbar_init(&ctl->raw_read, kE3Threads);
        mbar_init(&ctl->sfull, 1);
        mbar_init(&ctl->m_done, kE1Threads);
        mbar_init(&ctl->barX, 1);
        mbar_init(&ctl->pd_ready, kOThreads);
        mbar_init(&ctl->barY1a, 1);
        mbar_init(&ctl->barY1, 1);
        mbar_init(&ctl->barY2, 1);
        mbar_init(&ctl->r_ready[0], kE1Threads);
        mbar_init(&ctl->r_ready[1], kE1Threads);
        mbar_init(&ctl->acc_free1, kE3Threads);
        mbar_init(&ctl->acc_freeV, kOThreads);
        mbar_init(&ctl->parked, kE3Threads);
        mbar_init(&ctl->acc_free2, kE3Threads);
        mbar_init(&ctl->drain, 3);
        ctl->abort_flag = start_aborted;
        ctl->o_done = 0;
        ctl->exact_flag = 0;
        ctl->l_stage = ctl->l_v = ctl->l_state = ctl->l_raw = 0;
        fence_barrier_init();
        tma_prefetch_desc(&map_o);
        tma_prefetch_desc(&map_f);
        tma_prefetch_desc(&map_i);
        tma_prefetch_desc(&map_dy);
        tma_prefetch_desc(&map_saved);
        tma_prefetch_desc(&map_o_raw);
        tma_prefetch_desc(&map_f_raw);
    }
    if (warp == 0) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    const int sub = warp & 3;                                        // TMEM lane quarter of this warp
    const uint32_t lane_base = static_cast<uint32_t>(32 * sub) << 16;
    const int krow = 32 * sub + lane;                                // TMEM lane of this thread

    // it = 0, 1, ... counts processed chunks; chunk index c = NC - 1 - it
    if (warp < kTWarps) {
        // ================= T: transform =================
        PT_DECL
        for (int it = 0; it < NC; ++it) {
            const int s = it % kStages, c = NC - 1 - it;
            uint8_t *qbuf = smem + s * kStageBytes;
            mbar_wait(&ctl->full[s], (it / kStages) & 1, abort_flag);
            // Pacing, not a data dependence: the transform of chunk `it` starts only when the output walk of chunk
            // it - 2 is over (its completion pass may still run).  The tiles are there well before, but run earlier
            // the transform shares the issue slots with that walk, the longest stretch of the per-chunk loop
            // (event stamps: waiting for the completion pass as well made this the longest chain of the kernel;
            // no pacing at all measured the same as this).
            if (it >= 2) {
                if (lane == 0) count_wait(&ctl->o_done, kE3Warps * (it - 1), abort_flag);   // one poller per warp
                __syncwarp();
            }
            PT_MARK(0)
            PT_STAMP(status, 1, tid == 0 && it == 16) PT_STAMP(status, 20, tid == 0 && it == 18)
            const int n_valid = kRagged ? N - c * kC : kC;
            // Pm and E of the chunk are not kept: the backward takes them from what the forward saved
            if (n_valid >= kC) {
                transform_stream<true, kEnc, kSS, kSlab>(qbuf + kOffQ, qbuf + kOffK, nullptr, nullptr, nullptr, nullptr, kC, tid);
            } else {
                transform_stream<false, kEnc, kSS, kSlab>(qbuf + kOffQ, qbuf + kOffK, nullptr, nullptr, nullptr, nullptr, n_valid, tid);
            }
            fence_proxy_async_smem();
            mbar_arrive(&ctl->t_done[s]);
            PT_MARK(1)
            PT_STAMP(status, 2, tid == 0 && it == 16)
        }
        PT_DUMP(status, 0, 2, tid == 0)
    } else if (warp < kWarpE3) {
        // ================= E1: state-gradient warps =================
        // Pm, E of every chunk come from the forward's saved totals, so this chain does not wait for T
        float pm_prev = 1.f;
        const float *tot_u = totals + slot0 * 2 * kD + krow;
        float pm_c = __ldg(tot_u + (size_t)(NC - 1) * 2 * kD), ee_c = __ldg(tot_u + (size_t)(NC - 1) * 2 * kD + kD);
        PT_DECL
        for (int it = 0; it < NC; ++it) {
            // ---- dS'' = (Pm_prev E) dS' (the accumulator, or dSN first) -> TMEM, bf16 copy -> dsbuf
            PT_MARK(0)
            // a total on the floor: the decay across that half chunk is more than the rescaled operands can carry
            if (fminf(pm_c, ee_c) <= kProdFloor) ctl->exact_flag = 1;
            const float pm_old = pm_prev, ee_old = ee_c;
            const float factor = pm_prev * ee_c;
            pm_prev = pm_c;
            if (it + 1 < NC) {
                pm_c = __ldg(tot_u + (size_t)(NC - 2 - it) * 2 * kD);
                ee_c = __ldg(tot_u + (size_t)(NC - 2 - it) * 2 * kD + kD);
            }
            if (it > 0) {
                mbar_wait(&ctl->barX, (it - 1) & 1, abort_flag);   // dS' of the previous chunk is complete
                mbar_wait(&ctl->barY1, (it - 1) & 1, abort_flag);    // its dS'' copy is no longer read
                tc_fence_after_sync();
            }
            PT_MARK(1)
            PT_STAMP(status, 5, tid == kWarpE1 * 32 && it == 16)
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                uint32_t r[32];
                if (it == 0) {
                    if (dSN) {
                        const float4 *src = reinterpret_cast<const float4 *>(dSN + ((size_t)u * kD + krow) * kD + 32 * part);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 v4 = __ldg(src + j);
                            r[4 * j + 0] = __float_as_uint(v4.x); r[4 * j + 1] = __float_as_uint(v4.y);
                            r[4 * j + 2] = __float_as_uint(v4.z); r[4 * j + 3] = __float_as_uint(v4.w);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                    }
                } else {
                    tmem_ld32(tmem + lane_base + kColDS + 32 * part, r);
                    tmem_wait_ld();
                }
                if (factor >= kFactorSafe) {
#pragma unroll
                    for (int j = 0; j < 32; j += 2) scale2(r[j], r[j + 1], factor);
                } else {                         // see the forward kernel: the two decays one after the other
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * pm_old * ee_old);
                }
                tmem_st32(tmem + lane_base + kColDS + 32 * part, r);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<uint4 *>(dsbuf + (part >> 1) * kStateSlab + slab_chunk_off(krow, 4 * (part & 1) + j)) =
                        pack8(r + 8 * j);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            fence_proxy_async_smem();
            mbar_arrive(&ctl->m_done);
            PT_MARK(2)
            PT_STAMP(status, 6, tid == kWarpE1 * 32 && it == 16)

            // ---- R_k = sum_v dS''[k,v] S'[k,v] from the two bf16 copies
            mbar_wait(&ctl->sfull, it & 1, abort_flag);
            PT_MARK(3)
            float2 racc2 = make_float2(0.f, 0.f);
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
#pragma unroll 2
                for (int j = 0; j < 8; ++j) {
                    const uint32_t off = h * kStateSlab + slab_chunk_off(krow, j);
                    const uint4 dw = *reinterpret_cast<const uint4 *>(dsbuf + off);
                    const uint4 sw = *reinterpret_cast<const uint4 *>(sbuf + off);
                    racc2 = fma2(make_float2(bf16_lo(dw.x), bf16_hi(dw.x)), make_float2(bf16_lo(sw.x), bf16_hi(sw.x)), racc2);
                    racc2 = fma2(make_float2(bf16_lo(dw.y), bf16_hi(dw.y)), make_float2(bf16_lo(sw.y), bf16_hi(sw.y)), racc2);
                    racc2 = fma2(make_float2(bf16_lo(dw.z), bf16_hi(dw.z)), make_float2(bf16_lo(sw.z), bf16_hi(sw.z)), racc2);
                    racc2 = fma2(make_float2(bf16_lo(dw.w), bf16_hi(dw.w)), make_float2(bf16_lo(sw.w), bf16_hi(sw.w)), racc2);
                }
            }
            const float racc = racc2.x + racc2.y;
            rr[(it & 1) * 128 + krow] = racc;
            mbar_arrive(&ctl->r_ready[it & 1]);
            PT_MARK(4)
            PT_STAMP(status, 9, tid == kWarpE1 * 32 && it == 16)
        }
        PT_DUMP(status, 2, 5, tid == kWarpE1 * 32)

        // dS_0 = Diag(Pm of chunk 0) dS'
        mbar_wait(&ctl->barY2, (NC - 1) & 1, abort_flag);
        tc_fence_after_sync();
        if (dS0) {
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + kColDS + 32 * part, r);
                tmem_wait_ld();
                float4 *dst = reinterpret_cast<float4 *>(dS0 + ((size_t)u * kD + krow) * kD + 32 * part);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__uint_as_float(r[4 * j + 0]) * pm_prev, __uint_as_float(r[4 * j + 1]) * pm_prev,
                                         __uint_as_float(r[4 * j + 2]) * pm_prev, __uint_as_float(r[4 * j + 3]) * pm_prev);
            }
        }
    } else if (warp < kWarpO) {
        // ================= E3: d_o and d_f =================
        const int half = (warp - kWarpE3) >> 2;                      // half of the chunk: local times [32 * half, +32)
        const uint32_t tl = tmem + lane_base;
        PT_DECL
        for (int it = 0; it < NC; ++it) {
            const int c = NC - 1 - it;
            const int n_valid = kRagged ? min(kC, N - c * kC) : kC;
            const size_t crow0 = grow0 + (size_t)c * kC;
            // ---- outputs
            mbar_wait(&ctl->rawfull, it & 1, abort_flag);
            mbar_wait(&ctl->barY2, it & 1, abort_flag);
            PT_MARK(2)
            tc_fence_after_sync();
            float asum, esum;
            PT_STAMP(status, 14, tid == kWarpE3 * 32 && it == 16)
            if (half) phase_main<true, kRagged, kEnc>(tl, oraw, fraw, krow, d_o + crow0 * kD + krow, n_valid, asum, esum);
            else      phase_main<false, kRagged, kEnc>(tl, oraw, fraw, krow, d_o + crow0 * kD + krow, n_valid, asum, esum);
            mbar_arrive(&ctl->raw_read);
            if (half) xa[krow] = asum; else xe[krow] = esum;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&ctl->acc_free1);
            mbar_arrive(&ctl->parked);
            __syncwarp();
            if (lane == 0) atomicAdd(&ctl->o_done, 1);
            PT_MARK(3)
            PT_STAMP(status, 15, tid == kWarpE3 * 32 && it == 16)
            // ---- d_f completed from the parked values, each thread its own 32 rows, once both halves' sums and R
            // of the chunk are there
            mbar_wait(&ctl->r_ready[it & 1], (it >> 1) & 1, abort_flag);
            mbar_wait(&ctl->parked, it & 1, abort_flag);
            tc_fence_after_sync();
            {
                const float K = rr[(it & 1) * 128 + krow] + xa[krow] + xe[krow];
                __nv_bfloat16 *df_g = d_f + crow0 * kD + krow;
                // the thread's 64 parked values in two reads (the pass is on the chunk's critical chain)
                uint32_t uu[32], rf[32];
                tmem_ld32(tl + kColDQ + 32 * half, uu);
                tmem_ld32(tl + kColDKi + 32 * half, rf);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (!kRagged || 32 * half + j < n_valid)
                        df_g[(size_t)(32 * half + j) * kD] =
                            __float2bfloat16_rn(fmaf(K, __uint_as_float(rf[j]), __uint_as_float(uu[j])));
            }
            tc_fence_before_sync();
            mbar_arrive(&ctl->acc_free2);
            PT_MARK(4)
        }
        PT_DUMP(status, 7, 5, tid == kWarpE3 * 32)
    } else if (warp < kWarpLoad) {
        // ================= O: causal masks, d_i =================
        const uint32_t tl = tmem + lane_base;
        PT_DECL
        for (int it = 0; it < NC; ++it) {
            const int c = NC - 1 - it;
            const int n_valid = kRagged ? min(kC, N - c * kC) : kC;
            const size_t crow0 = grow0 + (size_t)c * kC;
            // ---- tril(A), tril(dA) -> operand slabs: rows of A sit in lanes 0..63, rows of dA in lanes 64..127, a
            // warp converts its 32 rows.  The previous chunk's products have read the slabs: this role waited for
            // them before that chunk's d_i.
            mbar_wait(&ctl->barX, it & 1, abort_flag);
            tc_fence_after_sync();
#pragma unroll 1
            for (int hh = 0; hh < 2; ++hh)
                tril_row_block(tl + (sub < 2 ? kColA : kColDA) + 32 * hh, sub < 2 ? pbuf : dpbuf, krow & 63, hh);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&ctl->pd_ready);
            mbar_wait(&ctl->barY2, it & 1, abort_flag);
            PT_MARK(0)
            PT_STAMP(status, 16, tid == kWarpO * 32 && it == 16)
            tc_fence_after_sync();
            // d_i = dV: lane = value dimension, columns = local times
#pragma unroll 1
            for (int b = 0; b < 8; ++b) {
                uint32_t r[8];
                tmem_ld8(tl + kColDV + 8 * b, r);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (8 * b + j < n_valid)
                        d_i[(crow0 + 8 * b + j) * kD + krow] = __float2bfloat16_rn(__uint_as_float(r[j]));
            }
            tc_fence_before_sync();
            mbar_arrive(&ctl->acc_freeV);
            PT_MARK(1)
            PT_STAMP(status, 17, tid == kWarpO * 32 && it == 16)
        }
        PT_DUMP(status, 11, 4, tid == kWarpO * 32)
    } else if (warp == kWarpLoad) {
        // ================= L: TMA loads =================
        if (lane == 0) {
            int n_stage = 0, n_v = 0, n_state = 0, n_raw = 0;       // fills asked for so far, per buffer
            auto issue_stage = [&](int it) {
                n_stage = it + 1;
                const int s = it % kStages, c = NC - 1 - it;
                uint8_t *st = smem + s * kStageBytes;
                mbar_arrive_expect_tx(&ctl->full[s], kStageBytes);
                for (int b = 0; b < 2; ++b) {
                    tma_load_3d(st + kOffQ + b * kSS, &map_o, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                    tma_load_3d(st + kOffK + b * kSlab, &map_f, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                }
                for (int b = 0; b < 2; ++b)
                    tma_load_3d(st + kOffG + b * kSS, &map_dy, &ctl->full[s], 64 * b, row0 + c * kC, zu);
            };
            auto issue_v = [&](int it) {
                n_v = it + 1;
                const int c = NC - 1 - it;
                mbar_arrive_expect_tx(&ctl->vfull, kTile);
                for (int b = 0; b < 2; ++b) tma_load_3d(vbuf + b * kSlab, &map_i, &ctl->vfull, 64 * b, row0 + c * kC, zu);
            };
            auto issue_raw = [&](int it) {
                n_raw = it + 1;
                const int c = NC - 1 - it;
                mbar_arrive_expect_tx(&ctl->rawfull, 2 * kTile);
                tma_load_3d(smem + kOffRawO, &map_o_raw, &ctl->rawfull, 0, row0 + c * kC, zu);
                tma_load_3d(smem + kOffRawF, &map_f_raw, &ctl->rawfull, 0, row0 + c * kC, zu);
            };
            auto issue_state = [&](int it) {
                n_state = it + 1;
                const int c = NC - 1 - it;
                mbar_arrive_expect_tx(&ctl->sfull, kStateTile);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d(sbuf + b * kStateSlab, &map_saved, &ctl->sfull, 64 * b, 0, (int)(slot0 + c));
            };
            issue_stage(0);
            issue_v(0);
            issue_state(0);
            issue_raw(0);
            if (NC > 1) issue_stage(1);
            // Every buffer is refilled as soon as its last reader of chunk `it` is done; the waits below are in
            // the order in which those readers finish.
            // A barrier must never be armed twice within one phase.  Normally a buffer's previous fill has long been
            // consumed when its readers report; on the time-out exit those waits return at once, so before every
            // refill the previous fill is waited for explicitly (one poll that succeeds at once in normal running).
            for (int it = 0; it + 1 < NC; ++it) {
                mbar_wait(&ctl->barX, it & 1, abort_flag);           // dA = dY V^T ...
                mbar_wait(&ctl->barY1, it & 1, abort_flag);          // ... and dKs_inter^T = dS'' V^T have read v
                mbar_wait_drain(&ctl->vfull, it & 1, 20000000ull);
                issue_v(it + 1);
                mbar_wait(&ctl->r_ready[it & 1], (it >> 1) & 1, abort_flag);   // R has read S' ...
                mbar_wait(&ctl->barY2, it & 1, abort_flag);          // ... and so have the chunk's products;
                mbar_wait_drain(&ctl->sfull, it & 1, 20000000ull);
                issue_state(it + 1);
                if (it + 2 < NC) {                                   // o, f, dy of the stage are free as well
                    mbar_wait_drain(&ctl->full[it % kStages], (it / kStages) & 1, 20000000ull);
                    issue_stage(it + 2);
                }
                PT_STAMP(status, 0, it == 14) PT_STAMP(status, 21, it == 16) PT_STAMP(status, 22, it == 15)
                mbar_wait(&ctl->raw_read, it & 1, abort_flag);       // the output warps are done with raw o, f
                mbar_wait_drain(&ctl->rawfull, it & 1, 20000000ull);
                issue_raw(it + 1);
            }
            ctl->l_stage = n_stage; ctl->l_v = n_v; ctl->l_state = n_state; ctl->l_raw = n_raw;
        }
    } else if (lane == 0) {
        // ================= MX, MY1, MY2: MMA issue =================
        constexpr uint32_t idDS = idesc_bf16(128, 128, 1, 1);     // Qs^T (MN-major) x dY (MN-major)
        constexpr uint32_t idKK = idesc_bf16(128, 64, 0, 0);      // dS'' x V^T, S' x dY^T (all K-major)
        constexpr uint32_t idMK = idesc_bf16(128, 64, 1, 0);      // dS''^T (MN) x Ks^T (K);  Ks^T (MN) x dP^T (K)
        constexpr uint32_t idMM = idesc_bf16(128, 64, 1, 1);      // Qs^T (MN) x dP (MN);  dY^T (MN) x P (MN)
        // descriptors once; K steps and stage changes only add to the 14-bit start-address field
        const uint32_t sm0 = smem_u32(smem);
        const uint64_t dqk0 = smem_desc_sw128(sm0 + kOffQ, 16, 1024), dqm0 = smem_desc_sw128(sm0 + kOffQ, kSS, 1024);
        const uint64_t dfk0 = smem_desc_sw128(sm0 + kOffK, 16, 1024), dfm0 = smem_desc_sw128(sm0 + kOffK, kSlab, 1024);
        const uint64_t dvk = smem_desc_sw128(smem_u32(vbuf), 16, 1024);
        const uint64_t dgk0 = smem_desc_sw128(sm0 + kOffG, 16, 1024), dgm0 = smem_desc_sw128(sm0 + kOffG, kSS, 1024);
        const uint64_t dsk = smem_desc_sw128(smem_u32(sbuf), 16, 1024);
        const uint64_t ddsk = smem_desc_sw128(smem_u32(dsbuf), 16, 1024), ddsm = smem_desc_sw128(smem_u32(dsbuf), kStateSlab, 1024);
        const uint64_t dpm = smem_desc_sw128(smem_u32(pbuf), kSlab, 1024);
        const uint64_t ddpk = smem_desc_sw128(smem_u32(dpbuf), 16, 1024), ddpm = smem_desc_sw128(smem_u32(dpbuf), kSlab, 1024);
        auto kmaj = [](int kk) { return (uint64_t)(((kk >> 2) * kSlab + (kk & 3) * 32) >> 4); };          // [64][128] tile
        auto kmaj_i = [](int kk) { return (uint64_t)(((kk >> 2) * kSS + (kk & 3) * 32) >> 4); };          // interleaved q / dy tile
        auto kmaj_s = [](int kk) { return (uint64_t)(((kk >> 2) * kStateSlab + (kk & 3) * 32) >> 4); };   // [128][128] tile
        PT_DECL
        if (warp == kWarpMmaX) {
            for (int it = 0; it < NC; ++it) {
                const int s = it % kStages;
                const uint64_t so = (uint64_t)s * (kStageBytes >> 4);
                const uint64_t dqk = dqk0 + so, dqm = dqm0 + so, dfk = dfk0 + so, dgm = dgm0 + so;
                mbar_wait(&ctl->full[s], (it / kStages) & 1, abort_flag);
                mbar_wait(&ctl->t_done[s], (it / kStages) & 1, abort_flag);
                PT_MARK(0)
                mbar_wait(&ctl->m_done, it & 1, abort_flag);          // dS'' in TMEM
                if (it > 0) mbar_wait(&ctl->pd_ready, (it - 1) & 1, abort_flag);   // A, dA of the previous chunk read out
                mbar_wait(&ctl->vfull, it & 1, abort_flag);
                PT_MARK(1)
                PT_STAMP(status, 3, it == 16)
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dS' = dS'' + Qs^T dY
                    mma_bf16_ss(tmem + kColDS, dqm + (uint64_t)(kk * 128), dgm + (uint64_t)(kk * 128), idDS, 1);
                {
                    // (Qs; dY) as one 128-row operand: (Qs; dY) Ks^T has A in lanes 0..63 and (Qs; dY) V^T has dA
                    // in lanes 64..127 (the other halves are not used), so every lane carries a row to mask
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_bf16_ss(tmem + kColA, dqk + kmaj_i(kk), dfk + kmaj(kk), idKK, kk > 0);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_bf16_ss(tmem + kColDA, dqk + kmaj_i(kk), dvk + kmaj(kk), idKK, kk > 0);
                    mma_commit(&ctl->barX);
                }
                PT_MARK(2)
                PT_STAMP(status, 4, it == 16)
            }
            PT_DUMP(status, 15, 3, true)
        } else if (warp == kWarpMmaY1) {
            for (int it = 0; it < NC; ++it) {
                const int s = it % kStages;
                const uint64_t so = (uint64_t)s * (kStageBytes >> 4);
                const uint64_t dfk = dfk0 + so;
                mbar_wait(&ctl->full[s], (it / kStages) & 1, abort_flag);
                mbar_wait(&ctl->t_done[s], (it / kStages) & 1, abort_flag);
                mbar_wait(&ctl->m_done, it & 1, abort_flag);          // bf16 dS'' in shared memory
                PT_MARK(0)
                // dV^T first: its accumulator is free as soon as d_i of the previous chunk is out, long before the
                // output warps have finished with dKs_inter^T
                if (it > 0) mbar_wait(&ctl->acc_freeV, (it - 1) & 1, abort_flag);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)              // dV^T = dS''^T Ks^T
                    mma_bf16_ss(tmem + kColDV, ddsm + (uint64_t)(kk * 128), dfk + kmaj(kk), idMK, kk > 0);
                mma_commit(&ctl->barY1a);
                mbar_wait(&ctl->vfull, it & 1, abort_flag);
                if (it > 0) mbar_wait(&ctl->acc_free1, (it - 1) & 1, abort_flag);
                PT_MARK(1)
                PT_STAMP(status, 10, it == 16)
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)              // dKs_inter^T = dS'' V^T
                    mma_bf16_ss(tmem + kColDKx, ddsk + kmaj_s(kk), dvk + kmaj(kk), idKK, kk > 0);
                mma_commit(&ctl->barY1);
                PT_MARK(2)
            }
            PT_DUMP(status, 18, 3, true)
        } else {
            for (int it = 0; it < NC; ++it) {
                const int s = it % kStages;
                const uint64_t so = (uint64_t)s * (kStageBytes >> 4);
                const uint64_t dqm = dqm0 + so, dfm = dfm0 + so, dgk = dgk0 + so, dgm = dgm0 + so;
                mbar_wait(&ctl->pd_ready, it & 1, abort_flag);   // tril(A), tril(dA); implies X and T of the chunk
                mbar_wait(&ctl->barY1a, it & 1, abort_flag);          // dV^T += ... must follow dV^T = ...
                PT_MARK(0)
                PT_STAMP(status, 11, it == 16)
                tc_fence_after_sync();
                // dV^T first: it does not touch the columns that still hold the previous chunk's parked values
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dV^T += dY^T A
                    mma_bf16_ss(tmem + kColDV, dgm + (uint64_t)(kk * 128), dpm + (uint64_t)(kk * 128), idMM, 1);
                mbar_wait(&ctl->sfull, it & 1, abort_flag);
                if (it > 0) mbar_wait(&ctl->acc_free2, (it - 1) & 1, abort_flag);
                PT_MARK(1)
                PT_STAMP(status, 12, it == 16)
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dQs^T = Ks^T dA^T
                    mma_bf16_ss(tmem + kColDQ, dfm + (uint64_t)(kk * 128), ddpk + (uint64_t)(kk * 2), idMK, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)              //        + S' dY^T
                    mma_bf16_ss(tmem + kColDQ, dsk + kmaj_s(kk), dgk + kmaj_i(kk), idKK, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dKs_intra^T = Qs^T dA
                    mma_bf16_ss(tmem + kColDKi, dqm + (uint64_t)(kk * 128), ddpm + (uint64_t)(kk * 128), idMM, kk > 0);
                // barY2 stands for every product of the chunk: dKs_inter^T is another lane's, so wait for it first
                // (it was issued when the output warps finished the previous chunk, well before this point)
                mbar_wait(&ctl->barY1, it & 1, abort_flag);
                mma_commit(&ctl->barY2);
                PT_MARK(2)
                PT_STAMP(status, 13, it == 16)
            }
            PT_DUMP(status, 21, 3, true)
        }
        mma_commit(&ctl->drain);          // each of the three issuing lanes, after its loop
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        // Nothing may be in flight when the CTA gives up its tensor and shared memory.  The three issuing lanes
        // committed once more after their loops: that barrier completes when every product they issued has.
        mbar_wait_drain(&ctl->drain, 0, 20000000ull);
        if (*abort_flag) {
            report_error(status, HGRN2_ERR_TIMEOUT, 2);
            // tiles asked for but never consumed may still be on their way into this CTA's shared memory
            const int ns = ctl->l_stage, nv = ctl->l_v, nst = ctl->l_state, nr = ctl->l_raw;
            for (int s = 0; s < kStages; ++s)
                if (ns > s) mbar_wait_drain(&ctl->full[s], ((ns - 1 - s) / kStages) & 1, 20000000ull);
            if (nv > 0) mbar_wait_drain(&ctl->vfull, (nv - 1) & 1, 20000000ull);
            if (nst > 0) mbar_wait_drain(&ctl->sfull, (nst - 1) & 1, 20000000ull);
            if (nr > 0) mbar_wait_drain(&ctl->rawfull, (nr - 1) & 1, 20000000ull);
        }
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);

    // ---- exact path (see the forward kernel): the unit is redone from its inputs and its saved chunk states by the
    // pairwise-safe fp32 routine; with several CTAs per unit the last one to finish does it.
    if (ex.o == nullptr) return;
    const int unit = kMultiCta ? u / ex.G : u;
    if constexpr (kMultiCta) {
        if (tid == 0) {
            if (ctl->exact_flag) atomicOr(&ex.unit_flag[unit], 1);
            __threadfence();
            int go = 0;
            if (atomicAdd(&ex.unit_count[unit], 1) == ex.G - 1) {
                __threadfence();
                go = atomicOr(&ex.unit_flag[unit], 0);
            }
            ctl->exact_flag = go;
        }
        __syncthreads();
    }
    if (!ctl->exact_flag || *abort_flag) return;
    __syncthreads();                                               // every thread has read the flag: smem is reused now
    if (tid == 0) atomicAdd(&status->exact_units, 1);
    const bool packed = kRagged && pk.cu != nullptr;
    const int n_unit = packed ? N : ex.N;                          // tokens of the whole unit
    const size_t seq = packed ? grow0 * kD : (size_t)unit * ex.N * kD, st = (size_t)unit * kD * kD;
    const size_t slot_u = packed ? slot0 : (size_t)unit * ((ex.N + kC - 1) / kC);
    alu::bwd_unit<__nv_bfloat16, __nv_bfloat16, kEnc ? alu::kGateEnc : alu::kGateIsF>(
        reinterpret_cast<float *>(smem), ex.o + seq, ex.f + seq, ex.i + seq, ex.dy + seq, ex.dSN ? ex.dSN + st : nullptr,
        ex.states + slot_u * kD * kD, kC / kExactC, ex.scratch + st, ex.d_o + seq, ex.d_f + seq,
        ex.d_i + seq, ex.dS0 ? ex.dS0 + st : nullptr, n_unit, kD, kD, kExactC, (n_unit + kExactC - 1) / kExactC);
}

}  // namespace

// ---- sequences split into segments (see chunk_tc_fwd.cu) ----------------------------------------------
// Chains the segments in reverse: dS_end[r] = gradient w.r.t. the state at the end of segment r.
// seg_major: see seg_combine_kernel.
__global__ void seg_combine_bwd_kernel(const float *__restrict__ dSN, const float *__restrict__ G_loc,
                                       const float *__restrict__ lam, float *__restrict__ dS_end,
                                       float *__restrict__ dS0, int G, int *__restrict__ unit_flag,
                                       int *__restrict__ unit_count, int units, int seg_major, size_t U, int H)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // element of [U][128][128]
    if (e < (size_t)units) {             // exact-path bookkeeping of the full pass that follows starts at zero
        unit_flag[e] = 0;
        unit_count[e] = 0;
    }
    const size_t u = e / (kD * kD);
    const int k = (int)((e / kD) % kD);
    const size_t kv = e % (kD * kD);
    float D = dSN ? dSN[e] : 0.f;
    for (int r = G - 1; r >= 0; --r) {
        const size_t ur = seg_index(seg_major, u, r, G, U, H);
        dS_end[ur * kD * kD + kv] = D;
        D = fmaf(lam[ur * kD + k], D, G_loc[ur * kD * kD + kv]);
    }
    if (dS0) dS0[e] = D;
}


static ExactArgs exact_args(const SeqArgs &a, int N_unit, int G, int *unit_flag, int *unit_count)
{
    ExactArgs ex;
    ex.o = static_cast<const __nv_bfloat16 *>(a.o);
    ex.f = static_cast<const __nv_bfloat16 *>(a.f);
    ex.i = static_cast<const __nv_bfloat16 *>(a.i);
    ex.dy = static_cast<const __nv_bfloat16 *>(a.dy);
    ex.dSN = a.dSN;
    ex.d_o = static_cast<__nv_bfloat16 *>(a.d_o);
    ex.d_f = static_cast<__nv_bfloat16 *>(a.d_f);
    ex.d_i = static_cast<__nv_bfloat16 *>(a.d_i);
    ex.dS0 = a.dS0;
    ex.states = reinterpret_cast<__nv_bfloat16 *>(a.states);
    ex.scratch = a.exact_scratch;
    ex.N = N_unit;
    ex.G = G;
    ex.unit_flag = unit_flag;
    ex.unit_count = unit_count;
    return ex;
}

PackedArgs tc_packed_args(const SeqArgs &a, int G);

// U CTAs; ordinary layout: U planes of N rows; packed batch (pk.cu set): pk.H planes of N rows shared by the U units.
static cudaError_t launch_bwd_once(const SeqArgs &a, uint64_t U, int N, int NC, const float *dSN, float *dS0,
                                   bool clear, const ExactArgs &ex, const PackedArgs &pk = PackedArgs{})
{
    CUtensorMap mo, mf, mi, mg, ms, mor, mfr;
    const uint64_t planes = pk.cu ? (uint64_t)pk.H : U;
    const uint64_t slots = pk.cu ? (uint64_t)pk.H * pk.slots_per_head : U * NC;
    if (!make_map(&mo, a.o, planes, N, kC) || !make_map(&mf, a.f, planes, N, kC) || !make_map(&mi, a.i, planes, N, kC) ||
        !make_map(&mg, a.dy, planes, N, kC) || !make_map(&ms, a.states, slots, kD, kD) ||
        !make_map_plain(&mor, a.o, planes, N, kC) || !make_map_plain(&mfr, a.f, planes, N, kC))
        return cudaErrorInvalidValue;
    const bool ragged = N % kC != 0 || pk.cu != nullptr;
    if (ex.o != nullptr && ex.G > 1 && ragged) return cudaErrorInvalidValue;      // segments are whole chunks
    auto kernel = a.gate_enc ? (ragged ? tc_bwd_kernel<true, false, true>
                                   : (ex.o != nullptr && ex.G > 1 ? tc_bwd_kernel<false, true, true>
                                                                   : tc_bwd_kernel<false, false, true>))
                         : (ragged ? tc_bwd_kernel<true, false, false>
                                   : (ex.o != nullptr && ex.G > 1 ? tc_bwd_kernel<false, true, false>
                                                                   : tc_bwd_kernel<false, false, false>));
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), kSmemBytes);
    if (err != cudaSuccess) return err;
    kernel<<<(unsigned)U, kThreads, kSmemBytes, a.stream>>>(
        mo, mf, mi, mg, ms, mor, mfr,
        a.totals, dSN, static_cast<__nv_bfloat16 *>(a.d_o),
        static_cast<__nv_bfloat16 *>(a.d_f), static_cast<__nv_bfloat16 *>(a.d_i), dS0, N, NC, a.status, clear ? 1 : 0, ex, pk, a.start_aborted);
    return cudaGetLastError();
}

cudaError_t launch_tc_bwd(const SeqArgs &a0)
{
    const uint64_t U = (uint64_t)a0.B * a0.H;
    SeqArgs a = a0;
    if (a.cu) {
        // packed batch: one CTA per (sequence, head), every CTA reads its own rows from the offsets array
        const int G = a.seg_scratch ? tc_packed_segments(U, a.N) : 1;
        PackedArgs pk = tc_packed_args(a, G);
        a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) +
                                             (size_t)pk.H * pk.slots_per_head * kSavedStateBytes);
        if (G <= 1)
            return launch_bwd_once(a, U, a.N, 0, a.dSN, a.dS0, a.clear_status, exact_args(a, a.N, 1, nullptr, nullptr),
                                   pk);
        // few units: every sequence as G segments (see launch_tc_fwd)
        const uint64_t CT = U * G;
        char *base = static_cast<char *>(a.seg_scratch);
        int *cu_seg = reinterpret_cast<int *>(base);
        float *G_loc = reinterpret_cast<float *>(base + tc_packed_offsets_bytes(a.B, G));
        float *dS_end = G_loc + CT * kD * kD;
        float *lam = dS_end + CT * kD * kD;
        launch_seg_offsets_packed(a.cu, a.B, G, cu_seg, a.stream);
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        pk.cu = cu_seg;
        err = launch_tc_state_bwd(a.o, a.f, a.dy, (uint64_t)a.H, a.N, G_loc, lam, a.gate_enc, a.status, a.clear_status,
                                  a.start_aborted, a.stream, cu_seg, a.B * G);
        if (err != cudaSuccess) return err;
        seg_combine_bwd_kernel<<<(unsigned)(U * kD * kD / 256), 256, 0, a.stream>>>(a.dSN, G_loc, lam, dS_end, a.dS0, G,
                                                                                   nullptr, nullptr, 0, 2, (size_t)U, a.H);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        SeqArgs t = a;
        t.dSN = dS_end;
        t.dS0 = nullptr;
        return launch_bwd_once(t, CT, a.N, 0, dS_end, nullptr, false, exact_args(t, a.N, 1, nullptr, nullptr), pk);
    }
    const RSegPlan rp = a.seg_scratch ? tc_rseg_plan(U, a.N, a.NC) : RSegPlan{U, 0, 1, 0};
    if (rp.tail_units) {
        // ragged segments (see launch_tc_fwd): state-gradient summaries per segment, chained in reverse, then the
        // full pass per segment through the packed-batch geometry
        const int G = rp.G;
        const uint64_t Ut = rp.tail_units, CT = Ut * G;
        const size_t spp = (size_t)(a.N / kC + G + 1);
        a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) +
                                             ((size_t)rp.main_units * a.NC + (size_t)Ut * spp) * kSavedStateBytes);
        cudaError_t err = cudaSuccess;
        bool clear = a.clear_status;
        if (rp.main_units) {
            const SeqArgs m = tc_slice_units(a, 0, rp.main_units);
            err = launch_bwd_once(m, rp.main_units, a.N, a.NC, m.dSN, m.dS0, clear, exact_args(m, a.N, 1, nullptr, nullptr));
            if (err != cudaSuccess) return err;
            clear = false;
        }
        SeqArgs t = tc_slice_units(a, rp.main_units, Ut);
        char *base = static_cast<char *>(a.seg_scratch);
        int *cu = reinterpret_cast<int *>(base);
        float *G_loc = reinterpret_cast<float *>(base + kRSegOffsetsBytes);
        float *dS_end = G_loc + CT * kD * kD;
        float *lam = dS_end + CT * kD * kD;
        launch_seg_offsets(cu, G, rp.Lc * kC, a.N, a.stream);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        PackedArgs pk;
        pk.cu = cu;
        pk.H = (int)Ut;
        pk.slots_per_head = (int)spp;
        err = launch_tc_state_bwd(t.o, t.f, t.dy, Ut, a.N, G_loc, lam, a.gate_enc, a.status, clear, a.start_aborted,
                                  a.stream, cu, G);
        if (err != cudaSuccess) return err;
        seg_combine_bwd_kernel<<<(unsigned)(Ut * kD * kD / 256), 256, 0, a.stream>>>(t.dSN, G_loc, lam, dS_end, t.dS0, G,
                                                                                    nullptr, nullptr, 0, 1, (size_t)Ut, 1);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        t.dSN = dS_end;
        t.dS0 = nullptr;
        return launch_bwd_once(t, CT, a.N, 0, dS_end, nullptr, false, exact_args(t, a.N, 1, nullptr, nullptr), pk);
    }
    a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) + U * a.NC * kSavedStateBytes);
    const SegPlan plan = a.seg_scratch ? tc_seg_plan(U, a.N, a.NC) : SegPlan{U, 0, 1};
    cudaError_t err = cudaSuccess;
    bool clear = a.clear_status;                                  // for the first kernel launched only
    if (plan.main_units) {
        const SeqArgs m = tc_slice_units(a, 0, plan.main_units);
        err = launch_bwd_once(m, plan.main_units, a.N, a.NC, m.dSN, m.dS0, clear,
                              exact_args(m, a.N, 1, nullptr, nullptr));
        if (err != cudaSuccess) return err;
        clear = false;
    }
    if (plan.tail_units) {
        const SeqArgs t = tc_slice_units(a, plan.main_units, plan.tail_units);
        const uint64_t Ut = plan.tail_units;
        const int G = plan.G;
        // scratch: G_local [Ut*G][128][128], dS_end [Ut*G][128][128], Lambda [Ut*G][128]
        float *G_loc = static_cast<float *>(a.seg_scratch);
        float *dS_end = G_loc + Ut * G * kD * kD;
        float *lam = dS_end + Ut * G * kD * kD;
        int *unit_flag = reinterpret_cast<int *>(lam + Ut * G * kD), *unit_count = unit_flag + Ut;
        // state-gradient contributions of the segments (chunk_tc_state.cu): they hold for every f
        err = launch_tc_state_bwd(t.o, t.f, t.dy, Ut * G, a.N / G, G_loc, lam, a.gate_enc, a.status, clear, a.start_aborted, a.stream);
        if (err != cudaSuccess) return err;
        seg_combine_bwd_kernel<<<(unsigned)(Ut * kD * kD / 256), 256, 0, a.stream>>>(t.dSN, G_loc, lam, dS_end, t.dS0, G,
                                                                                    unit_flag, unit_count, (int)Ut, 0, (size_t)Ut, 1);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        err = launch_bwd_once(t, Ut * G, a.N / G, a.NC / G, dS_end, nullptr, false,
                              exact_args(t, a.N, G, unit_flag, unit_count));
    }
    return err;
}

}  // namespace hgrn2
