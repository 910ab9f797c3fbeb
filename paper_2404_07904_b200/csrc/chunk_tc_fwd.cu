// Chunkwise HGRN2 forward on the Blackwell tensor cores (tcgen05 + TMEM + TMA), bf16 I/O, fp32
// state, d_k = d_v = 128, chunk length C = 64.  One CTA per (batch, head) unit walks the chunks in
// order with the running state resident in tensor memory (frame and formulas: tc_chunk.cuh).
//
// Warp roles (none of them ever waits on a CTA-wide barrier inside the chunk loop; every stretch of
// work between two hand-offs is latency-bound, so the roles are many and narrow rather than few and
// wide, and their loops stay rolled to keep the instruction footprint small):
//   T   transform warps (4 per group): raw o, f tiles -> Qs, Ks in place, running ahead of the rest
//       by up to two chunks (three TMA stages);
//   E1  8 state warps: rescale the accumulator once per chunk (the critical chain) and publish its
//       bf16 copy S' for Y = Qs S' and for the saved-state store;
//   E2  4 output warps: causal mask of A into an operand slab, Y into a staging tile;
//   L   1 warp: TMA loads of o, f, i;
//   MS  1 warp: tcgen05.mma issue of A = Qs Ks^T and of the state update S' += Ks^T V, then the TMA store of
//       S' (the saved chunk state) straight from the operand copy;
//   MY  1 warp: tcgen05.mma issue of Y = Qs S', Y += tril(A) V;
//   ST  1 warp: TMA stores of the Y tiles.
// Hand-offs are mbarriers; every wait is bounded (tc_common.cuh).
//
// Tensor-memory plan (512 columns): S' at [0,128) (lane = key dim, column = value dim); Y, double
// buffered, at [128,384) and A, double buffered, at [384,512) in the M = 64 accumulator layout
// (row r -> lane 32 * (r / 16) + r % 16).
#include "chunk_alu.cuh"
#include "tc_chunk.cuh"

namespace hgrn2 {

namespace {

using namespace tc;

constexpr int kTGroups = 1, kTWarps = 4 * kTGroups;
constexpr int kE1Warps = 8, kE2Warps = 4;
constexpr int kE1Threads = kE1Warps * 32, kE2Threads = kE2Warps * 32;
constexpr int kWarpE1 = kTWarps, kWarpE2 = kWarpE1 + kE1Warps;
constexpr int kWarpLoad = kWarpE2 + kE2Warps, kWarpMmaS = kWarpLoad + 1, kWarpMmaY = kWarpLoad + 2,
              kWarpStore = kWarpLoad + 3;
constexpr int kThreads = (kWarpStore + 1) * 32;
static_assert(kWarpE1 % 4 == 0 && kWarpE2 % 4 == 0, "epilogue warps must start on a TMEM lane-quarter boundary");

constexpr int kStages = 3;
constexpr uint32_t kStageBytes = 3 * kTile;                       // q, f, v
constexpr uint32_t kOffS = kStages * kStageBytes;                 // bf16 copy of S'
constexpr uint32_t kOffP = kOffS + kStateTile;                    // bf16 tril(A): two slabs (double buffer)
constexpr uint32_t kOffY = kOffP + 2 * kSlab;                     // Y staging tile for the TMA store
constexpr uint32_t kOffPm = kOffY + kTile;                        // float pm[4][128]
constexpr uint32_t kOffE = kOffPm + 4 * 128 * 4;                  // float ee[4][128]
constexpr uint32_t kOffCtl = kOffE + 4 * 128 * 4;
constexpr uint32_t kSmemBytes = kOffCtl + 320 + 1024;             // + alignment slack

constexpr uint32_t kColS = 0, kColY = 128, kColA = 384;

struct Ctl {
    uint64_t fullqf[kStages];    // TMA (o, f tiles) -> T
    uint64_t full[kStages];      // TMA (i tile) -> MS, MY
    uint64_t emptyqf[kStages];   // tcgen05.commit (MS and MY) -> L: every MMA reading Qs, Ks of the stage has completed
    uint64_t emptyv[kStages];    // tcgen05.commit (MS and MY) -> L: every MMA reading V of the stage has completed
    uint64_t t_done[kStages];    // T -> MS, MY, E1 (Pm, E of the chunk)
    uint64_t m_tmem;             // E1 -> MS: the accumulator holds S' of the chunk
    uint64_t m_done;             // E1 -> MY: the bf16 copy of S' is in shared memory
    uint64_t barS;               // tcgen05.commit -> E1: state update complete
    uint64_t barS2;              // tcgen05.commit (MY) + MS -> E1: Y = Qs S' complete, S' stored: copy reusable
    uint64_t barA[2];            // tcgen05.commit -> E2: A is complete
    uint64_t p_ready[2];         // E2 -> MY: tril(A) is in shared memory
    uint64_t barY[2];            // tcgen05.commit -> E2: Y is complete
    uint64_t y_tfree[2];         // E2 -> MY: the Y accumulator has been read out
    uint64_t y_staged;           // E2 -> ST
    uint64_t y_sfree;            // ST -> E2: the staging tile may be overwritten
    uint64_t drain;              // tcgen05.commit (MS and MY, after their loops): every product issued has completed
    int abort_flag;              // set by the first wait that runs out: every later wait returns at once
    uint32_t tmem_base;
    int exact_flag;              // E1: a decay of this CTA's tokens left the range of the rescaled operands
    int l_qf, l_v;               // L: chunks whose o, f tiles (i tile) have been asked for, for the abort epilogue
};
static_assert(sizeof(Ctl) <= 320, "control block");
static_assert(kSmemBytes <= 232448, "shared memory budget");

constexpr int kExactC = 32;      // chunk length of the exact fp32 routines at d = 128 (their shared-memory budget)
static_assert(alu::fwd_smem_floats(kD, kD, kExactC) * sizeof(float) <= kSmemBytes - 1024, "exact path fits the CTA's shared memory");

// kRagged: N is not a whole number of chunks (the tail chunk is padded with neutral tokens).
// kMultiCta: a unit runs as several CTAs (segments) of this launch; the bookkeeping that lets the last of them
// take the unit's exact path is compiled in only then (its mere presence costs the one-CTA-per-unit launch 3 %).
// kEnc: the f tensor holds k = 1 - f (see transform_half).
template <bool kRagged, bool kMultiCta, bool kEnc>
__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_f,
              const __grid_constant__ CUtensorMap map_i, const __grid_constant__ CUtensorMap map_y,
              const __grid_constant__ CUtensorMap map_saved, const float *__restrict__ S0, float *__restrict__ SN,
              float *__restrict__ totals, int want_y, int want_saved, int N_all, int NC_all,
              StatusBlock *status, int clear_status, const ExactArgs ex, const PackedArgs pk,
              int start_aborted)
{
    // the first kernel of a call zeroes the status word (errors are reported seconds later, after a wait ran out)
    if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) {
        status->code = 0;
        status->where = 0;
        status->exact_units = 0;
    }
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sbuf = smem + kOffS;
    uint8_t *pbuf = smem + kOffP;
    uint8_t *ybuf = smem + kOffY;
    float *pm = reinterpret_cast<float *>(smem + kOffPm);
    float *ee = reinterpret_cast<float *>(smem + kOffE);
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
            if (N <= 0) {                // empty sequence: the state passes through
                if (SN != nullptr)
                    for (int x = tid; x < kD * kD; x += kThreads)
                        SN[(size_t)u * kD * kD + x] = S0 ? S0[(size_t)u * kD * kD + x] : 0.f;
                return;
            }
        }
    }

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->fullqf[s], 1);
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->emptyqf[s], 2);
            mbar_init(&ctl->emptyv[s], 2);
            mbar_init(&ctl->t_done[s], kTransformThreads);
        }
        mbar_init(&ctl->m_tmem, kE1Threads);
        mbar_init(&ctl->m_done, kE1Threads);
        mbar_init(&ctl->barS, 1);
        mbar_init(&ctl->barS2, 2);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&ctl->barA[b], 1);
            mbar_init(&ctl->p_ready[b], kE2Threads);
            mbar_init(&ctl->barY[b], 1);
            mbar_init(&ctl->y_tfree[b], kE2Threads);
        }
        mbar_init(&ctl->y_staged, kE2Threads);
        mbar_init(&ctl->y_sfree, 1);
        mbar_init(&ctl->drain, 2);
        ctl->abort_flag = start_aborted;
        ctl->exact_flag = 0;
        ctl->l_qf = 0;
        ctl->l_v = 0;
        fence_barrier_init();
        tma_prefetch_desc(&map_o);
        tma_prefetch_desc(&map_f);
        tma_prefetch_desc(&map_i);
        tma_prefetch_desc(&map_y);
        tma_prefetch_desc(&map_saved);
    }
    if (warp == 0) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    const int sub = warp & 3;                                        // TMEM lane quarter of this warp
    const uint32_t lane_base = static_cast<uint32_t>(32 * sub) << 16;

    if (warp < kTWarps) {
        // ================= T: transform =================
        PT_DECL
        const int tt = tid & (kTransformThreads - 1);
        for (int c = warp >> 2; c < NC; c += kTGroups) {
            const int s = c % kStages;
            uint8_t *qbuf = smem + s * kStageBytes;
            mbar_wait(&ctl->fullqf[s], (c / kStages) & 1, abort_flag);
            PT_MARK(0)
            const int n_valid = kRagged ? N - c * kC : kC;
            float *tg = totals ? totals + (slot0 + c) * 2 * kD : nullptr;       // Pm, E of the chunk for the backward
            if (n_valid >= kC) {
                transform_stream<true, kEnc>(qbuf, qbuf + kTile, pm + (c & 3) * 128, ee + (c & 3) * 128, tg, tg ? tg + kD : nullptr,
                                       kC, tt);
            } else {
                transform_stream<false, kEnc>(qbuf, qbuf + kTile, pm + (c & 3) * 128, ee + (c & 3) * 128, tg, tg ? tg + kD : nullptr,
                                        n_valid, tt);
            }
            fence_proxy_async_smem();
            mbar_arrive(&ctl->t_done[s]);
            PT_MARK(1)
        }
        PT_DUMP(status, 0, 2, tid == 0)
    } else if (warp < kWarpE2) {
        // ================= E1: state warps =================
        const int half = (warp - kWarpE1) >> 2;                      // column half [64 * half, 64 * half + 64)
        const int krow = 32 * sub + lane;
        const int v0 = 64 * half;
        float e_prev = 1.f;
        PT_DECL
        for (int c = 0; c < NC; ++c) {
            // S' = (E_prev Pm) S'' (S'' = the accumulator, or S0 for the first chunk) back into TMEM
            mbar_wait(&ctl->t_done[c % kStages], (c / kStages) & 1, abort_flag);
            PT_MARK(0)
            const float pm_c = pm[(c & 3) * 128 + krow];
            const float e_old = e_prev;
            const float factor = e_prev * pm_c;
            e_prev = ee[(c & 3) * 128 + krow];
            // a total on the floor: the decay across that half chunk is more than the rescaled operands can carry
            if (fminf(pm_c, e_prev) <= kProdFloor) ctl->exact_flag = 1;
            uint32_t r[64];
            if (c == 0) {
                if (S0) {
                    const float4 *src = reinterpret_cast<const float4 *>(S0 + ((size_t)u * kD + krow) * kD + v0);
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float4 x = __ldg(src + j);
                        r[4 * j + 0] = __float_as_uint(x.x); r[4 * j + 1] = __float_as_uint(x.y);
                        r[4 * j + 2] = __float_as_uint(x.z); r[4 * j + 3] = __float_as_uint(x.w);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 64; ++j) r[j] = 0u;
                }
            } else {
                mbar_wait(&ctl->barS, (c - 1) & 1, abort_flag);
                PT_MARK(1)
                tc_fence_after_sync();
                tmem_ld32(tmem + lane_base + kColS + v0, *reinterpret_cast<uint32_t(*)[32]>(r));
                tmem_ld32(tmem + lane_base + kColS + v0 + 32, *reinterpret_cast<uint32_t(*)[32]>(r + 32));
                tmem_wait_ld();
            }
            // Each of the two decays is above the floor, but their product can leave fp32's range although the
            // accumulator, which sits in the previous chunk's frame, is as large as that decay is small: then the
            // two are applied one after the other (key dimensions whose decay over those 64 tokens is below
            // 2^-120: rare, so a branch around the single multiply).
            if (factor >= kFactorSafe) {
#pragma unroll
                for (int j = 0; j < 64; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * factor);
            } else {
#pragma unroll
                for (int j = 0; j < 64; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * e_old * pm_c);
            }
            tmem_st32(tmem + lane_base + kColS + v0, *reinterpret_cast<uint32_t(*)[32]>(r));
            tmem_st32(tmem + lane_base + kColS + v0 + 32, *reinterpret_cast<uint32_t(*)[32]>(r + 32));
            uint4 sw[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) sw[j] = pack8(r + 8 * j);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&ctl->m_tmem);
            PT_MARK(2)
            // its bf16 copy, once Y = Qs S' of the previous chunk no longer reads the old one
            if (c >= 1) mbar_wait(&ctl->barS2, (c - 1) & 1, abort_flag);
            PT_MARK(3)
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4 *>(sbuf + half * kStateSlab + slab_chunk_off(krow, j)) = sw[j];
            fence_proxy_async_smem();
            mbar_arrive(&ctl->m_done);
            PT_MARK(4)
        }
        PT_DUMP(status, 2, 5, tid == kWarpE1 * 32)


        // S_N = Diag(E_last) S''
        mbar_wait(&ctl->barS, (NC - 1) & 1, abort_flag);
        tc_fence_after_sync();
        if (SN) {
            uint32_t r[32];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                tmem_ld32(tmem + lane_base + kColS + v0 + 32 * part, r);
                tmem_wait_ld();
                float4 *dst = reinterpret_cast<float4 *>(SN + ((size_t)u * kD + krow) * kD + v0 + 32 * part);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__uint_as_float(r[4 * j + 0]) * e_prev, __uint_as_float(r[4 * j + 1]) * e_prev,
                                         __uint_as_float(r[4 * j + 2]) * e_prev, __uint_as_float(r[4 * j + 3]) * e_prev);
            }
        }
    } else if (warp < kWarpLoad) {
        // ================= E2: output warps =================
        if (want_y) {
            const int t = 16 * sub + lane;                           // accumulator row of lanes 0..15
            PT_DECL
            // iteration c: tril(A(c)) -> operand slab | Y(c-1) -> staging tile
            for (int c = 0; c <= NC; ++c) {
                if (c < NC) {
                    const int b = c & 1;
                    mbar_wait(&ctl->barA[b], (c >> 1) & 1, abort_flag);
                    PT_MARK(0)
                    tc_fence_after_sync();
                    tril_to_slab(tmem + lane_base + kColA + 64 * b, pbuf + b * kSlab, sub, 0, lane);
                    tril_to_slab(tmem + lane_base + kColA + 64 * b + 32, pbuf + b * kSlab, sub, 1, lane);
                    fence_proxy_async_smem();
                    tc_fence_before_sync();
                    mbar_arrive(&ctl->p_ready[b]);
                    PT_MARK(1)
                }
                if (c >= 1) {
                    const int b = (c - 1) & 1;
                    mbar_wait(&ctl->barY[b], ((c - 1) >> 1) & 1, abort_flag);
                    PT_MARK(2)
                    tc_fence_after_sync();
                    if (c >= 2) mbar_wait(&ctl->y_sfree, (c - 2) & 1, abort_flag);
                    PT_MARK(3)
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        uint32_t r[64];
                        const uint32_t ta = tmem + lane_base + kColY + 128 * b + 64 * h;
                        tmem_ld32(ta, *reinterpret_cast<uint32_t(*)[32]>(r));
                        tmem_ld32(ta + 32, *reinterpret_cast<uint32_t(*)[32]>(r + 32));
                        tmem_wait_ld();
                        if (lane < 16) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<uint4 *>(ybuf + h * kSlab + slab_chunk_off(t, j)) = pack8(r + 8 * j);
                        }
                    }
                    tc_fence_before_sync();
                    mbar_arrive(&ctl->y_tfree[b]);
                    fence_proxy_async_smem();
                    mbar_arrive(&ctl->y_staged);
                    PT_MARK(4)
                }
            }
            PT_DUMP(status, 7, 5, tid == kWarpE2 * 32)
        }
    } else if (warp == kWarpLoad) {
        // ================= L: TMA loads =================
        if (lane == 0) {
            int n_qf = 0, n_v = 0;                                   // chunks whose tiles have been asked for
            for (int c = 0; c < NC; ++c) {
                const int s = c % kStages;
                uint8_t *st = smem + s * kStageBytes;
                // o and f have barriers of their own in both directions: the transform, which paces the kernel,
                // needs only them, and their tiles are free as soon as Y = Qs S' of the chunk three back is done,
                // well before its last product Y += P V has read V
                // A barrier must never be armed twice within one phase.  Normally the stage's previous fill has long
                // been consumed when its empty barrier completes; on the time-out exit that wait returns at once, so
                // the previous fill is waited for explicitly (one poll that succeeds at once in normal running;
                // stopping this lane on the wait's return value instead cost 8 %).
                if (c >= kStages) {
                    mbar_wait(&ctl->emptyqf[s], ((c / kStages) - 1) & 1, abort_flag);
                    mbar_wait_drain(&ctl->fullqf[s], ((c / kStages) - 1) & 1, 20000000ull);
                }
                // the next chunk's o, f tiles are asked into L2 now: their load can be issued only when their stage
                // frees, one chunk from now, and then finds them there (measured on the fwd + bwd step: -1 %; two
                // chunks ahead, or including the v tile, gave nothing)
                if (c + 1 < NC)
                    for (int b = 0; b < 2; ++b) {
                        tma_prefetch_3d(&map_o, 64 * b, row0 + (c + 1) * kC, zu);
                        tma_prefetch_3d(&map_f, 64 * b, row0 + (c + 1) * kC, zu);
                    }
                mbar_arrive_expect_tx(&ctl->fullqf[s], 2 * kTile);
                for (int b = 0; b < 2; ++b) {
                    tma_load_3d(st + b * kSlab, &map_o, &ctl->fullqf[s], 64 * b, row0 + c * kC, zu);
                    tma_load_3d(st + kTile + b * kSlab, &map_f, &ctl->fullqf[s], 64 * b, row0 + c * kC, zu);
                }
                n_qf = c + 1;
                if (c >= kStages) {
                    mbar_wait(&ctl->emptyv[s], ((c / kStages) - 1) & 1, abort_flag);
                    mbar_wait_drain(&ctl->full[s], ((c / kStages) - 1) & 1, 20000000ull);
                }
                mbar_arrive_expect_tx(&ctl->full[s], kTile);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d(st + 2 * kTile + b * kSlab, &map_i, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                n_v = c + 1;
            }
            ctl->l_qf = n_qf;
            ctl->l_v = n_v;
        }
    } else if (warp == kWarpMmaS) {
        // ================= MS: state update =================
        if (lane == 0) {
            constexpr uint32_t idescS = idesc_bf16(128, 128, 1, 1);    // Ks^T (MN-major) x V (MN-major)
            // Descriptors are formed once; a K step or a stage change only adds to the 14-bit
            // start-address field (addresses are in 16-byte units and stay below 2^14).
            const uint64_t dfm0 = smem_desc_sw128(smem_u32(smem) + kTile, kSlab, 1024);      // Ks, MN-major
            const uint64_t dvm0 = smem_desc_sw128(smem_u32(smem) + 2 * kTile, kSlab, 1024);  // V, MN-major
            constexpr uint32_t idescA = idesc_bf16(64, 64, 0, 0);      // Qs (K-major) x Ks (K-major)
            const uint64_t dq0 = smem_desc_sw128(smem_u32(smem), 16, 1024);                  // Qs, K-major
            const uint64_t dfk0 = smem_desc_sw128(smem_u32(smem) + kTile, 16, 1024);         // Ks, K-major
            auto kmaj = [](int kk) { return (uint64_t)(((kk >> 2) * kSlab + (kk & 3) * 32) >> 4); };
            PT_DECL
            for (int c = 0; c < NC; ++c) {
                const int s = c % kStages;
                const uint64_t so = (uint64_t)s * (kStageBytes >> 4);
                mbar_wait(&ctl->full[s], (c / kStages) & 1, abort_flag);
                mbar_wait(&ctl->t_done[s], (c / kStages) & 1, abort_flag);
                PT_MARK(0)
                // A = Qs Ks^T is issued here, not by the lane of the other output products: this lane has nothing
                // to do until the state is rescaled, and every tcgen05.mma also costs the issuing lane's scheduler
                // (shared with a transform warp) issue time, so the products are spread over two schedulers
                if (want_y) {
                    const int b = c & 1;
                    if (c >= 2) {                                    // tril(A) of chunk c - 2 has left this buffer
                        mbar_wait(&ctl->p_ready[b], ((c - 2) >> 1) & 1, abort_flag);
                        tc_fence_after_sync();
                    }
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        mma_bf16_ss(tmem + kColA + 64 * b, dq0 + so + kmaj(kk), dfk0 + so + kmaj(kk), idescA, kk > 0);
                    mma_commit(&ctl->barA[b]);
                }
                mbar_wait(&ctl->m_tmem, c & 1, abort_flag);
                PT_MARK(1)
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // S' += Ks^T V
                    mma_bf16_ss(tmem + kColS, dfm0 + so + (uint64_t)(kk * 128), dvm0 + so + (uint64_t)(kk * 128),
                                idescS, 1);
                mma_commit(&ctl->barS);
                mma_commit(&ctl->emptyqf[s]);
                mma_commit(&ctl->emptyv[s]);
                PT_MARK(2)
                // the saved chunk state, straight from the operand copy of S' (this lane is idle until the next
                // chunk's state is ready; in the lane that issues the outputs' products the wait for the store
                // to have read 32 KB would hold those up)
                mbar_wait(&ctl->m_done, c & 1, abort_flag);
                if (want_saved) {
                    tma_store_3d(&map_saved, sbuf, 0, 0, (int)(slot0 + c));
                    tma_store_3d(&map_saved, sbuf + kStateSlab, 64, 0, (int)(slot0 + c));
                    tma_store_commit();
                    tma_store_wait_read();
                }
                mbar_arrive(&ctl->barS2);                   // second arrival: the tcgen05.commit of Y = Qs S'
            }
            PT_DUMP(status, 12, 3, true)
            if (want_saved) tma_store_wait_all();
            mma_commit(&ctl->drain);
        }
    } else if (warp == kWarpMmaY) {
        // ================= MY: outputs (+ saved-state stores) =================
        if (lane == 0) {
            constexpr uint32_t idescY = idesc_bf16(64, 128, 0, 1);     // Qs or P (K-major) x S' or V (MN-major)
            const uint64_t dq0 = smem_desc_sw128(smem_u32(smem), 16, 1024);                  // Qs, K-major
            const uint64_t dvm0 = smem_desc_sw128(smem_u32(smem) + 2 * kTile, kSlab, 1024);  // V, MN-major
            const uint64_t dsm = smem_desc_sw128(smem_u32(sbuf), kStateSlab, 1024);          // S', MN-major
            const uint64_t dp0 = smem_desc_sw128(smem_u32(pbuf), 16, 1024);                  // tril(A), K-major
            auto kmaj = [](int kk) { return (uint64_t)(((kk >> 2) * kSlab + (kk & 3) * 32) >> 4); };
            PT_DECL
            for (int c = 0; c < NC; ++c) {
                const int s = c % kStages, b = c & 1;
                const uint64_t so = (uint64_t)s * (kStageBytes >> 4);
                const uint64_t dq = dq0 + so, dvm = dvm0 + so;
                const uint64_t dp = dp0 + (uint64_t)b * (kSlab >> 4);
                const uint32_t ty = tmem + kColY + 128 * b;
                mbar_wait(&ctl->full[s], (c / kStages) & 1, abort_flag);
                mbar_wait(&ctl->t_done[s], (c / kStages) & 1, abort_flag);
                PT_MARK(0)
                mbar_wait(&ctl->m_done, c & 1, abort_flag);
                PT_MARK(1)
                if (want_y) {
                    if (c >= 2) {
                        mbar_wait(&ctl->y_tfree[b], ((c - 2) >> 1) & 1, abort_flag);
                        tc_fence_after_sync();
                    }
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)          // Y = Qs S'
                        mma_bf16_ss(ty, dq + kmaj(kk), dsm + (uint64_t)(kk * 128), idescY, kk > 0);
                }
                PT_MARK(2)
                mma_commit(&ctl->barS2);
                mma_commit(&ctl->emptyqf[s]);               // A and Y = Qs S' were the last readers of Qs, Ks here
                if (want_y) {
                    mbar_wait(&ctl->p_ready[b], (c >> 1) & 1, abort_flag);
                    PT_MARK(3)
                    tc_fence_after_sync();
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)          // Y += P V
                        mma_bf16_ss(ty, dp + (uint64_t)(kk * 2), dvm + (uint64_t)(kk * 128), idescY, 1);
                    mma_commit(&ctl->barY[b]);
                }
                mma_commit(&ctl->emptyv[s]);
                PT_MARK(4)
            }
            PT_DUMP(status, 15, 5, true)
            mma_commit(&ctl->drain);
        }
    } else {
        // ================= ST: Y stores =================
        if constexpr (!kRagged) {
            if (lane == 0 && want_y) {
                for (int c = 0; c < NC; ++c) {
                    mbar_wait(&ctl->y_staged, c & 1, abort_flag);
                    tma_store_3d(&map_y, ybuf, 0, c * kC, u);
                    tma_store_3d(&map_y, ybuf + kSlab, 64, c * kC, u);
                    tma_store_commit();
                    tma_store_wait_read();
                    mbar_arrive(&ctl->y_sfree);
                }
                tma_store_wait_all();
            }
        } else if (want_y) {
            // In a packed batch the rows after a sequence's last token belong to the next sequence (a tile store
            // would overwrite them; past the end of an ordinary tensor it simply drops them), so the partial last
            // chunk of a packed sequence is stored row by row, by the whole warp.
            for (int c = 0; c < NC; ++c) {
                mbar_wait(&ctl->y_staged, c & 1, abort_flag);
                const int n_valid = min(kC, N - c * kC);
                if (pk.cu == nullptr || n_valid == kC) {
                    if (lane == 0) {
                        tma_store_3d(&map_y, ybuf, 0, row0 + c * kC, zu);
                        tma_store_3d(&map_y, ybuf + kSlab, 64, row0 + c * kC, zu);
                        tma_store_commit();
                        tma_store_wait_read();
                    }
                } else {
                    uint4 *dst = reinterpret_cast<uint4 *>(ex.y + ((size_t)zu * N_all + row0 + (size_t)c * kC) * kD);
                    for (int x = lane; x < n_valid * 16; x += 32) {          // 16-byte pieces: row, slab, chunk
                        const int r = x >> 4, h = (x >> 3) & 1, j = x & 7;
                        dst[(size_t)r * 16 + h * 8 + j] = *reinterpret_cast<const uint4 *>(ybuf + h * kSlab + slab_chunk_off(r, j));
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->y_sfree);
            }
            if (lane == 0) tma_store_wait_all();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        // Nothing may be in flight when the CTA gives up its tensor and shared memory.  The two issuing lanes
        // committed once more after their loops: that barrier completes when every product they issued has.
        mbar_wait_drain(&ctl->drain, 0, 20000000ull);
        if (*abort_flag) {
            report_error(status, HGRN2_ERR_TIMEOUT, 1);
            // tiles asked for but never consumed may still be on their way into this CTA's shared memory
            for (int s = 0; s < kStages; ++s) {
                const int nq = ctl->l_qf, nv = ctl->l_v;
                if (nq > s) mbar_wait_drain(&ctl->fullqf[s], (((nq - 1 - s) / kStages)) & 1, 20000000ull);
                if (nv > s) mbar_wait_drain(&ctl->full[s], (((nv - 1 - s) / kStages)) & 1, 20000000ull);
            }
        }
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);

    // ---- exact path: the sweep met a decay its operands cannot represent, so the unit is redone, from its inputs,
    // by the pairwise-safe fp32 routine (every output of the unit is overwritten).  With several CTAs per unit
    // (segments) the last one to finish does it, once every other has written its part.
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
    const size_t seq = packed ? ((size_t)zu * N_all + row0) * kD : (size_t)unit * ex.N * kD, st = (size_t)unit * kD * kD;
    const size_t slot_u = packed ? slot0 : (size_t)unit * ((ex.N + kC - 1) / kC);
    alu::fwd_unit<__nv_bfloat16, __nv_bfloat16, kEnc ? alu::kGateEnc : alu::kGateIsF>(
        reinterpret_cast<float *>(smem), ex.o + seq, ex.f + seq, ex.i + seq, ex.S0 ? ex.S0 + st : nullptr,
        ex.y ? ex.y + seq : nullptr, ex.SN ? ex.SN + st : nullptr,
        ex.states ? ex.states + slot_u * kD * kD : nullptr, kC / kExactC, n_unit, kD, kD, kExactC,
        (n_unit + kExactC - 1) / kExactC);
}

}  // namespace

bool tc_supported(const hgrn2_desc *d)
{
    return d->io == HGRN2_BF16 && d->dk == kD && d->dv == kD;
}
int  tc_default_chunk() { return kC; }
bool tc_chunk_supported(int C) { return C == kC; }

size_t tc_saved_bytes(const hgrn2_desc *d, int C)
{
    const size_t NC = ((size_t)d->N + C - 1) / C;
    const uint64_t U = (uint64_t)d->B * d->H;
    const RSegPlan rp = tc_rseg_plan(U, d->N, (int)NC);
    // ragged segments use the packed batch's slot numbering: N / C + (segments) + 1 slots per unit
    const size_t slots = rp.tail_units ? (size_t)rp.main_units * NC + (size_t)rp.tail_units * ((size_t)d->N / C + rp.G + 1)
                                       : (size_t)U * NC;
    return slots * (kSavedStateBytes + kSavedTotalsBytes);
}

// ---- sequences split into segments ----------------------------------------------------------------------
// One CTA per unit leaves most SMs idle when there are few units (a 16K-token batch of two sequences has
// 32).  The recurrence is linear in the state, so a sequence can be cut into G segments that run as separate
// CTAs: (1) every segment runs state-only from a zero state (chunk_tc_state.cu), giving its local end state and
// its total decay Lambda = prod f; (2) a small kernel chains them, S_start[r+1] = Diag(Lambda[r]) S_start[r] + S_local[r];
// (3) every segment runs in full from its S_start.  Token (r, t) of unit u is token t of "unit" u * G + r of a
// [U * G][N / G][128] view of the same memory, so the kernel itself does not know about segments.
// seg_major = 0: segment r of unit u sits at index u * G + r; 1: at r * U + u (the packed-batch order of the
// ragged segments); 2: unit u = (sequence b, head h) of a packed batch with H heads, its segment r at
// (b * G + r) * H + h.
__global__ void seg_combine_kernel(const float *__restrict__ S0, const float *__restrict__ S_loc,
                                   const float *__restrict__ lam, float *__restrict__ S_start, float *__restrict__ SN,
                                   int G, int *__restrict__ unit_flag, int *__restrict__ unit_count, int units,
                                   int seg_major, size_t U, int H)
{
    const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // element of [U][128][128]
    if (e < (size_t)units) {             // exact-path bookkeeping of the full pass that follows starts at zero
        unit_flag[e] = 0;
        unit_count[e] = 0;
    }
    const size_t u = e / (kD * kD);
    const int k = (int)((e / kD) % kD);
    const size_t kv = e % (kD * kD);
    float S = S0 ? S0[e] : 0.f;
    for (int r = 0; r < G; ++r) {
        const size_t ur = seg_index(seg_major, u, r, G, U, H);
        S_start[ur * kD * kD + kv] = S;
        S = fmaf(lam[ur * kD + k], S, S_loc[ur * kD * kD + kv]);
    }
    if (SN) SN[e] = S;
}

int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

// Number of segments per sequence (1 = do not split): as many as fill the SMs, at most 8, dividing the chunk
// count, each at least 8 chunks long; for sequences made of whole chunks (others: tc_rseg_plan).
int segments_for(uint64_t U, int N, int NC)
{
    if (U == 0 || N % kC != 0) return 1;
    int G = (int)(sm_count() / (int)U);
    if (G > 8) G = 8;
    while (G >= 2 && (NC % G != 0 || NC / G < 8)) --G;
    return G >= 2 ? G : 1;
}

// Sequences that are not whole chunks: segments of Lc chunks (at least 8), the last one shorter, for all units
// when they are few and for the units beyond the last full wave otherwise (the rule of tc_seg_plan).
RSegPlan tc_rseg_plan(uint64_t U, int N, int NC)
{
    RSegPlan p{U, 0, 1, 0};
    const uint64_t sms = (uint64_t)sm_count();
    if (U == 0 || sms == 0 || N % kC == 0) return p;
    uint64_t split = U, whole = 0;
    if (U > sms) {
        split = U % sms;
        whole = U - split;
        if (split == 0 || 2 * split > sms) return p;
    }
    int G0 = (int)(sms / split);
    if (G0 > 8) G0 = 8;
    if (G0 < 2) return p;
    int Lc = (NC + G0 - 1) / G0;
    if (Lc < 8) Lc = 8;
    const int G = (NC + Lc - 1) / Lc;
    if (G < 2) return p;
    return RSegPlan{whole, split, G, Lc};
}

// cu[r] = first row of segment r (r = 0 .. G), segments of L rows, the last one ends at N
__global__ void seg_offsets_kernel(int *__restrict__ cu, int G, int L, int N)
{
    const int r = threadIdx.x;
    if (r <= G) cu[r] = min(r * L, N);
}

void launch_seg_offsets(int *cu, int G, int L, int N, cudaStream_t stream)
{
    seg_offsets_kernel<<<1, 32, 0, stream>>>(cu, G, L, N);
}

// Packed batch: sequence b = rows [cu[b], cu[b + 1]) becomes G segments of Lc = max(8, ceil(chunks / G)) chunks
// each (the last one shorter, those beyond the sequence's end empty); segment b * G + r starts at cu_seg[b * G + r]
// and ends where the next one starts.  Malformed offsets give segments of negative length, which every kernel
// that reads them reports and skips.
__global__ void seg_offsets_packed_kernel(const int *__restrict__ cu, int B, int G, int *__restrict__ cu_seg)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x > B * G) return;
    if (x == B * G) {
        cu_seg[x] = cu[B];
        return;
    }
    const int b = x / G, r = x - b * G;
    const int start = cu[b], n = cu[b + 1] - start;
    const int nc = (n + kC - 1) / kC;
    int Lc = (nc + G - 1) / G;
    if (Lc < 8) Lc = 8;
    cu_seg[x] = start + (n <= 0 ? (r == 0 ? 0 : n) : min(r * Lc * kC, n));
}

void launch_seg_offsets_packed(const int *cu, int B, int G, int *cu_seg, cudaStream_t stream)
{
    const int n = B * G + 1;
    seg_offsets_packed_kernel<<<(n + 127) / 128, 128, 0, stream>>>(cu, B, G, cu_seg);
}

// Segments per sequence of a packed batch of T rows per head: as many as fill the SMs when the units alone fill at
// most half of them; none when no sequence can be longer than one segment (8 chunks).
int tc_packed_segments(uint64_t U, int T)
{
    const int sms = sm_count();
    if (U == 0 || sms == 0 || 2 * U > (uint64_t)sms || T <= 8 * kC) return 1;
    const int G = sms / (int)U;
    return G > 8 ? 8 : G;
}

size_t tc_packed_offsets_bytes(int B, int G) { return (((size_t)B * G + 1) * sizeof(int) + 255) & ~(size_t)255; }

// Few units (no more than SMs): all of them are split.  More units than SMs: the units beyond the last full
// wave of CTAs would keep a few SMs busy for a whole sequence while the rest idle, so those - when they are at
// most half a wave - are split as well and run after the full waves.
SegPlan tc_seg_plan(uint64_t U, int N, int NC)
{
    SegPlan p{U, 0, 1};
    const uint64_t sms = (uint64_t)sm_count();
    if (U == 0 || sms == 0) return p;
    if (U <= sms) {
        const int G = segments_for(U, N, NC);
        if (G > 1) p = SegPlan{0, U, G};
        return p;
    }
    const uint64_t r = U % sms;
    if (r > 0 && 2 * r <= sms) {
        const int G = segments_for(r, N, NC);
        if (G > 1) p = SegPlan{U - r, r, G};
    }
    return p;
}

// The same call restricted to units [u0, u0 + n): every per-unit pointer advanced (bf16 sequence tensors,
// fp32 states; a.totals must be set).  The result has B = n, H = 1.
SeqArgs tc_slice_units(const SeqArgs &a, uint64_t u0, uint64_t n)
{
    SeqArgs s = a;
    s.B = (int)n;
    s.H = 1;
    const size_t seq = (size_t)u0 * a.N * kD * 2, st = (size_t)u0 * kD * kD;
    auto adv = [](const void *p, size_t bytes) { return p ? static_cast<const char *>(p) + bytes : nullptr; };
    s.o = adv(a.o, seq); s.f = adv(a.f, seq); s.i = adv(a.i, seq); s.dy = adv(a.dy, seq);
    s.y = const_cast<char *>(static_cast<const char *>(adv(a.y, seq)));
    s.d_o = const_cast<char *>(static_cast<const char *>(adv(a.d_o, seq)));
    s.d_f = const_cast<char *>(static_cast<const char *>(adv(a.d_f, seq)));
    s.d_i = const_cast<char *>(static_cast<const char *>(adv(a.d_i, seq)));
    s.S0 = a.S0 ? a.S0 + st : nullptr;
    s.SN = a.SN ? a.SN + st : nullptr;
    s.dSN = a.dSN ? a.dSN + st : nullptr;
    s.dS0 = a.dS0 ? a.dS0 + st : nullptr;
    s.exact_scratch = a.exact_scratch ? a.exact_scratch + st : nullptr;
    if (a.states) {
        s.states = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) + (size_t)u0 * a.NC * kSavedStateBytes);
        s.totals = a.totals + (size_t)u0 * a.NC * 2 * kD;
    }
    return s;
}

// Per-unit flag and counter of the exact path when a unit runs as several CTAs, after the segment scratch proper.
static size_t seg_flag_bytes(uint64_t units) { return ((size_t)units * 2 * sizeof(int) + 15) & ~(size_t)15; }

size_t tc_segment_scratch_bytes(const hgrn2_desc *d, int C)
{
    const uint64_t U = (uint64_t)d->B * d->H;
    const int NC = (d->N + C - 1) / C;
    const RSegPlan rp = tc_rseg_plan(U, d->N, NC);
    if (rp.tail_units) return kRSegOffsetsBytes + (size_t)rp.tail_units * rp.G * (2 * kD * kD + kD) * sizeof(float);
    const SegPlan p = tc_seg_plan(U, d->N, NC);
    return p.tail_units ? (size_t)p.tail_units * p.G * (2 * kD * kD + kD) * sizeof(float) + seg_flag_bytes(p.tail_units) : 0;
}

// One float matrix per unit for the exact path of the backward (chunk_alu.cuh, bwd_unit).
size_t tc_exact_scratch_bytes(const hgrn2_desc *d, bool packed)
{
    const uint64_t U = (uint64_t)d->B * d->H;
    // sequences run as segments of their own geometry: one matrix per segment
    if (packed) return (size_t)U * tc_packed_segments(U, d->N) * kD * kD * sizeof(float);
    const RSegPlan rp = tc_rseg_plan(U, d->N, (d->N + kC - 1) / kC);
    return ((size_t)rp.main_units + (size_t)rp.tail_units * rp.G) * kD * kD * sizeof(float);
}

static ExactArgs exact_args(const SeqArgs &a, int N_unit, int G, int *unit_flag, int *unit_count)
{
    ExactArgs ex;
    ex.o = static_cast<const __nv_bfloat16 *>(a.o);
    ex.f = static_cast<const __nv_bfloat16 *>(a.f);
    ex.i = static_cast<const __nv_bfloat16 *>(a.i);
    ex.S0 = a.S0;
    ex.y = static_cast<__nv_bfloat16 *>(a.y);
    ex.SN = a.SN;
    ex.states = reinterpret_cast<__nv_bfloat16 *>(a.states);
    ex.N = N_unit;
    ex.G = G;
    ex.unit_flag = unit_flag;
    ex.unit_count = unit_count;
    return ex;
}

// U CTAs; ordinary layout: U planes of N rows; packed batch (pk.cu set): pk.H planes of N rows shared by the U units.
static cudaError_t launch_fwd_once(const SeqArgs &a, uint64_t U, int N, int NC, const float *S0, float *SN,
                                   bool want_y, bool want_saved, bool clear, const ExactArgs &ex,
                                   const PackedArgs &pk = PackedArgs{})
{
    CUtensorMap mo, mf, mi, my, ms;
    const uint64_t planes = pk.cu ? (uint64_t)pk.H : U;
    const uint64_t slots = pk.cu ? (uint64_t)pk.H * pk.slots_per_head : U * NC;
    // tensor maps need a valid base even for outputs that are not wanted: point those at an input
    const void *ybase = want_y ? a.y : a.i;
    const void *sbase = want_saved ? static_cast<const void *>(a.states) : a.i;
    const uint64_t srows = want_saved ? (uint64_t)kD : (uint64_t)N;
    const uint64_t sunits = want_saved ? slots : planes;
    if (!make_map(&mo, a.o, planes, N, kC) || !make_map(&mf, a.f, planes, N, kC) || !make_map(&mi, a.i, planes, N, kC) ||
        !make_map(&my, ybase, planes, N, kC) || !make_map(&ms, sbase, sunits, srows, want_saved ? kD : kC))
        return cudaErrorInvalidValue;
    const bool ragged = N % kC != 0 || pk.cu != nullptr;
    if (ex.o != nullptr && ex.G > 1 && ragged) return cudaErrorInvalidValue;      // segments are whole chunks
    auto kernel = a.gate_enc ? (ragged ? tc_fwd_kernel<true, false, true>
                                   : (ex.o != nullptr && ex.G > 1 ? tc_fwd_kernel<false, true, true>
                                                                   : tc_fwd_kernel<false, false, true>))
                         : (ragged ? tc_fwd_kernel<true, false, false>
                                   : (ex.o != nullptr && ex.G > 1 ? tc_fwd_kernel<false, true, false>
                                                                   : tc_fwd_kernel<false, false, false>));
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), kSmemBytes);
    if (err != cudaSuccess) return err;
    float *totals = want_saved ? a.totals : nullptr;
    kernel<<<(unsigned)U, kThreads, kSmemBytes, a.stream>>>(mo, mf, mi, my, ms, S0, SN, totals, want_y,
                                                                   want_saved, N, NC, a.status, clear ? 1 : 0, ex, pk,
                                                                   a.start_aborted);
    return cudaGetLastError();
}

// G segments per sequence: B * G pseudo-sequences share the slot numbering
PackedArgs tc_packed_args(const SeqArgs &a, int G)
{
    PackedArgs pk;
    pk.cu = a.cu;
    pk.H = a.H;
    pk.slots_per_head = a.N / kC + a.B * G + 1;
    return pk;
}

size_t tc_saved_bytes_packed(const hgrn2_desc *d)
{
    const int G = tc_packed_segments((uint64_t)d->B * d->H, d->N);
    return (size_t)d->H * ((size_t)d->N / kC + (size_t)d->B * G + 1) * (kSavedStateBytes + kSavedTotalsBytes);
}

// offsets of the segments | S_local, S_start (or G_local, dS_end) [B * G * H][128][128] | Lambda [B * G * H][128]
size_t tc_segment_scratch_bytes_packed(const hgrn2_desc *d)
{
    const int G = tc_packed_segments((uint64_t)d->B * d->H, d->N);
    if (G <= 1) return 0;
    return tc_packed_offsets_bytes(d->B, G) + (size_t)d->B * G * d->H * (2 * kD * kD + kD) * sizeof(float);
}

cudaError_t launch_tc_fwd(const SeqArgs &a0)
{
    const uint64_t U = (uint64_t)a0.B * a0.H;
    SeqArgs a = a0;
    if (a.cu) {
        // packed batch: one CTA per (sequence, head), every CTA reads its own rows from the offsets array
        const int G = a.seg_scratch ? tc_packed_segments(U, a.N) : 1;
        PackedArgs pk = tc_packed_args(a, G);
        if (a.states)
            a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) +
                                                 (size_t)pk.H * pk.slots_per_head * kSavedStateBytes);
        if (G <= 1)
            return launch_fwd_once(a, U, a.N, 0, a.S0, a.SN, a.y != nullptr, a.states != nullptr, a.clear_status,
                                   exact_args(a, a.N, 1, nullptr, nullptr), pk);
        // few units: every sequence as G segments (state-only pass, chaining, full pass: see below), the segments'
        // offsets derived from the batch's on the device
        const uint64_t CT = U * G;
        char *base = static_cast<char *>(a.seg_scratch);
        int *cu_seg = reinterpret_cast<int *>(base);
        float *S_loc = reinterpret_cast<float *>(base + tc_packed_offsets_bytes(a.B, G));
        float *S_start = S_loc + CT * kD * kD;
        float *lam = S_start + CT * kD * kD;
        launch_seg_offsets_packed(a.cu, a.B, G, cu_seg, a.stream);
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        pk.cu = cu_seg;
        err = launch_tc_state_fwd(a.f, a.i, (uint64_t)a.H, a.N, S_loc, lam, a.gate_enc, a.status, a.clear_status,
                                  a.start_aborted, a.stream, cu_seg, a.B * G);
        if (err != cudaSuccess) return err;
        seg_combine_kernel<<<(unsigned)(U * kD * kD / 256), 256, 0, a.stream>>>(a.S0, S_loc, lam, S_start, a.SN, G,
                                                                               nullptr, nullptr, 0, 2, (size_t)U, a.H);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        SeqArgs t = a;
        t.S0 = S_start;
        t.SN = nullptr;
        return launch_fwd_once(t, CT, a.N, 0, S_start, nullptr, a.y != nullptr, a.states != nullptr, false,
                               exact_args(t, a.N, 1, nullptr, nullptr), pk);
    }
    const bool want_y = a.y != nullptr, want_saved = a.states != nullptr;
    const RSegPlan rp = a.seg_scratch ? tc_rseg_plan(U, a.N, a.NC) : RSegPlan{U, 0, 1, 0};
    if (rp.tail_units) {
        // ragged segments: the three steps of the whole-chunk segments below, with per-CTA rows from an offsets
        // array (the packed-batch geometry: "sequence" r of "head" u = segment r of unit u); every segment CTA
        // takes its own exact path from its start state, which the state-only pass gives for every f.  Saved
        // states: the whole units' slots first, then the split units' in the packed slot numbering.
        const int G = rp.G;
        const uint64_t Ut = rp.tail_units, CT = Ut * G;
        const size_t spp = (size_t)(a.N / kC + G + 1);
        if (a.states)
            a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) +
                                                 ((size_t)rp.main_units * a.NC + (size_t)Ut * spp) * kSavedStateBytes);
        cudaError_t err = cudaSuccess;
        bool clear = a.clear_status;
        if (rp.main_units) {
            const SeqArgs m = tc_slice_units(a, 0, rp.main_units);
            err = launch_fwd_once(m, rp.main_units, a.N, a.NC, m.S0, m.SN, want_y, want_saved, clear,
                                  exact_args(m, a.N, 1, nullptr, nullptr));
            if (err != cudaSuccess) return err;
            clear = false;
        }
        SeqArgs t = tc_slice_units(a, rp.main_units, Ut);
        char *base = static_cast<char *>(a.seg_scratch);
        int *cu = reinterpret_cast<int *>(base);
        float *S_loc = reinterpret_cast<float *>(base + kRSegOffsetsBytes);
        float *S_start = S_loc + CT * kD * kD;
        float *lam = S_start + CT * kD * kD;
        launch_seg_offsets(cu, G, rp.Lc * kC, a.N, a.stream);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        PackedArgs pk;
        pk.cu = cu;
        pk.H = (int)Ut;
        pk.slots_per_head = (int)spp;
        err = launch_tc_state_fwd(t.f, t.i, Ut, a.N, S_loc, lam, a.gate_enc, a.status, clear, a.start_aborted,
                                  a.stream, cu, G);
        if (err != cudaSuccess) return err;
        seg_combine_kernel<<<(unsigned)(Ut * kD * kD / 256), 256, 0, a.stream>>>(t.S0, S_loc, lam, S_start, t.SN, G,
                                                                                nullptr, nullptr, 0, 1, (size_t)Ut, 1);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        t.S0 = S_start;
        t.SN = nullptr;
        return launch_fwd_once(t, CT, a.N, 0, S_start, nullptr, want_y, want_saved, false,
                               exact_args(t, a.N, 1, nullptr, nullptr), pk);
    }
    if (a.states) a.totals = reinterpret_cast<float *>(reinterpret_cast<char *>(a.states) + U * a.NC * kSavedStateBytes);
    const SegPlan plan = a.seg_scratch ? tc_seg_plan(U, a.N, a.NC) : SegPlan{U, 0, 1};
    cudaError_t err = cudaSuccess;
    bool clear = a.clear_status;                                  // for the first kernel launched only
    if (plan.main_units) {
        const SeqArgs m = tc_slice_units(a, 0, plan.main_units);
        err = launch_fwd_once(m, plan.main_units, a.N, a.NC, m.S0, m.SN, want_y, want_saved, clear,
                              exact_args(m, a.N, 1, nullptr, nullptr));
        if (err != cudaSuccess) return err;
        clear = false;
    }
    if (plan.tail_units) {
        const SeqArgs t = tc_slice_units(a, plan.main_units, plan.tail_units);
        const uint64_t Ut = plan.tail_units;
        const int G = plan.G;
        // scratch: S_local [Ut*G][128][128], S_start [Ut*G][128][128], Lambda [Ut*G][128]
        float *S_loc = static_cast<float *>(a.seg_scratch);
        float *S_start = S_loc + Ut * G * kD * kD;
        float *lam = S_start + Ut * G * kD * kD;
        int *unit_flag = reinterpret_cast<int *>(lam + Ut * G * kD), *unit_count = unit_flag + Ut;
        // the state-only pass (chunk_tc_state.cu) holds for every f: it needs no exact path of its own
        err = launch_tc_state_fwd(t.f, t.i, Ut * G, a.N / G, S_loc, lam, a.gate_enc, a.status, clear, a.start_aborted, a.stream);
        if (err != cudaSuccess) return err;
        seg_combine_kernel<<<(unsigned)(Ut * kD * kD / 256), 256, 0, a.stream>>>(t.S0, S_loc, lam, S_start, t.SN, G,
                                                                                unit_flag, unit_count, (int)Ut, 0, (size_t)Ut, 1);
        if ((err = cudaGetLastError()) != cudaSuccess) return err;
        err = launch_fwd_once(t, Ut * G, a.N / G, a.NC / G, S_start, nullptr, want_y, want_saved, false,
                              exact_args(t, a.N, G, unit_flag, unit_count));
    }
    return err;
}

}  // namespace hgrn2
