// State-only passes over sequence segments on the Blackwell tensor cores (tcgen05 + TMEM + TMA), bf16 I/O,
// d_k = d_v = 128, chunk length C = 64.
//
// When sequences are split into segments (chunk_tc_fwd.cu), every segment first needs what it contributes to the
// state chain on its own, from a zero boundary state:
//
//   forward :  S_loc = sum_s  (k_s * prod_{s < r <= end} f_r)^T  v_s          (state at the segment's end)
//   backward:  G_loc = sum_t  (q_t * prod_{start <= r <= t} f_r)^T dy_t       (state gradient at its start)
//
// (Eq. 3 unrolled over the segment, and its transpose; k = 1 - f, q = o, v = i.)  Both are one contraction
// X^T W over all tokens of the segment with X = x * c, c a running product of f that only ever shrinks: every
// factor is <= 1, so nothing needs a reference frame, a floor or a reciprocal, an underflowing factor is a
// contribution that has really vanished, and the accumulator is never rescaled: the per-chunk hand-off between the
// state warps and the tensor pipe, which paces the full kernels, does not exist here.  The forward pass walks the
// chunks from the last to the first (suffix products), the backward pass from the first to the last (prefix
// products).  Either pass also leaves the segment's total decay Lambda = prod f.
//
// Warp roles: T 4 warps (x, f tiles -> X in place; thread = column pair x half chunk: it first multiplies up
// its half's f, exchanges that with the other half through shared memory, then walks its rows), L 1 warp (TMA
// loads, four stages), M 1 warp (tcgen05.mma issue, 4 K-steps per chunk into one 128 x 128 fp32 accumulator);
// at the end the T warps move the accumulator to global memory.  Every wait is bounded (tc_common.cuh).
//
// kRagged instantiations: the segment need not be a whole number of chunks (rows past its end act as the
// neutral token f = 1, q = 0), and a CTA may take its rows from an offsets array: CTA u = b * planes + h then
// covers rows [cu[b], cu[b + 1]) of plane h of the [planes][rows][128] tensors (sequences cut into segments of
// unequal length, chunk_tc_fwd.cu).
#include "tc_chunk.cuh"

namespace hgrn2 {

namespace {

using namespace tc;

constexpr int kTWarps = 4;
constexpr int kWarpLoad = kTWarps, kWarpMma = kTWarps + 1;
constexpr int kThreads = (kWarpMma + 1) * 32;
constexpr int kStages = 4;

template <bool kBwd> struct Geo {
    // stage layout: forward [f][v]; backward [o][f][dy].  X overwrites f (forward: X = k c) or o (backward: X = q c).
    static constexpr uint32_t kOffX = 0;
    static constexpr uint32_t kOffF = kBwd ? kTile : 0;
    static constexpr uint32_t kOffW = kBwd ? 2 * kTile : kTile;
    static constexpr uint32_t kStageBytes = kBwd ? 3 * kTile : 2 * kTile;
    static constexpr uint32_t kOffHp = kStages * kStageBytes;            // float hp[2][2][128]: half products, double buffered
    static constexpr uint32_t kOffCtl = kOffHp + 2 * 2 * 128 * 4;
    static constexpr uint32_t kSmemBytes = kOffCtl + 256 + 1024;         // + alignment slack
};

struct Ctl {
    uint64_t full[kStages];      // TMA -> T
    uint64_t t_done[kStages];    // T -> M
    uint64_t empty[kStages];     // tcgen05.commit -> L: the chunk's products have read the stage
    uint64_t acc_done;           // tcgen05.commit -> T: every product has completed
    uint32_t tmem_base;
    int abort_flag;
    int l_issued;                // L: chunks asked for so far, for the abort epilogue
};
static_assert(sizeof(Ctl) <= 256, "control block");

// kEnc: the f tensor holds the signed gate encoding (see transform_half in tc_chunk.cuh).
template <bool kBwd, bool kEnc, bool kRagged>
__global__ void __launch_bounds__(kThreads, 1)
tc_state_kernel(const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_f,
                const __grid_constant__ CUtensorMap map_w, float *__restrict__ out, float *__restrict__ lam, int N_all,
                int NC_all, const int *__restrict__ cu, int planes, StatusBlock *status, int clear_status,
                int start_aborted)
{
    using G = Geo<kBwd>;
    if (clear_status && blockIdx.x == 0 && threadIdx.x == 0) {
        status->code = 0;
        status->where = 0;
        status->exact_units = 0;
    }
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float *hp = reinterpret_cast<float *>(smem + G::kOffHp);
    Ctl *ctl = reinterpret_cast<Ctl *>(smem + G::kOffCtl);
    volatile int *abort_flag = &ctl->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int u = blockIdx.x;
    // this CTA's segment: rows [row0, row0 + N) of plane zu, NC chunks
    int row0 = 0, zu = u, N = N_all, NC = NC_all;
    if constexpr (kRagged) {
        if (cu != nullptr) {
            const int b = u / planes;
            zu = u - b * planes;
            row0 = __ldg(cu + b);
            N = __ldg(cu + b + 1) - row0;
            if (row0 < 0 || N < 0 || row0 + N > N_all) {          // malformed offsets: report, touch nothing
                if (tid == 0) report_error(status, HGRN2_ERR_INVALID_ARG, 6);
                return;
            }
        }
        NC = (N + kC - 1) / kC;
        if (N <= 0) {                    // an empty segment contributes nothing and does not decay
            for (int x = tid; x < kD * kD; x += kThreads) out[(size_t)u * kD * kD + x] = 0.f;
            if (lam != nullptr && tid < kD) lam[(size_t)u * kD + tid] = 1.f;
            return;
        }
    }

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->t_done[s], kTransformThreads);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->acc_done, 1);
        ctl->abort_flag = start_aborted;
        ctl->l_issued = 0;
        fence_barrier_init();
        if (kBwd) tma_prefetch_desc(&map_o);
        tma_prefetch_desc(&map_f);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 0) tmem_alloc(&ctl->tmem_base, 128);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;

    // n = 0, 1, ... counts processed chunks; the forward pass visits chunk NC - 1 - n, the backward pass chunk n
    if (warp < kTWarps) {
        // ================= T: X = x * (running product of f), in place =================
        const int p = tid & 63, half = tid >> 6;
        const int col = 2 * p;
        const int jch = (col & 63) >> 3;
        const uint32_t base = (col >> 6) * kSlab + (col & 7) * 2;
        uint32_t xo[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) xo[jj] = base + ((jch ^ jj) << 4);
        float P0 = 1.f, P1 = 1.f;                 // product of f over the chunks already visited, this column pair
        for (int n = 0; n < NC; ++n) {
            const int s = n % kStages;
            uint8_t *xbuf = smem + s * G::kStageBytes + G::kOffX;
            const uint8_t *fbuf = smem + s * G::kStageBytes + G::kOffF;
            mbar_wait(&ctl->full[s], (n / kStages) & 1, abort_flag);
            const int n_valid = kRagged ? N - (kBwd ? n : NC - 1 - n) * kC : kC;     // rows of the chunk inside the segment
            // this half's f (32 rows of the column pair) and its product
            uint32_t fw[32];
            float h0 = 1.f, h1 = 1.f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int r = 32 * half + j;
                fw[j] = *reinterpret_cast<const uint32_t *>(fbuf + xo[r & 7] + r * 128);
                if (kRagged && r >= n_valid) fw[j] = kEnc ? 0x80008000u : 0x3F803F80u;      // f = 1, k = 0
                float f0, f1, k0, k1;
                if (kEnc) {
                    gate_decode(fw[j], f0, k0);
                    gate_decode(fw[j] >> 16, f1, k1);
                } else {
                    f0 = bf16_lo(fw[j]);
                    f1 = bf16_hi(fw[j]);
                }
                h0 *= f0;
                h1 *= f1;
            }
            float *hb = hp + (n & 1) * 256;
            *reinterpret_cast<float2 *>(hb + half * 128 + col) = make_float2(h0, h1);
            asm volatile("bar.sync 1, 128;" ::: "memory");           // the 128 transform threads only
            const float2 ho = *reinterpret_cast<const float2 *>(hb + (half ^ 1) * 128 + col);
            // the half visited second starts behind the other half's rows
            const bool second = kBwd ? (half == 1) : (half == 0);
            float a0 = second ? P0 * ho.x : P0, a1 = second ? P1 * ho.y : P1;
            P0 *= h0 * ho.x;
            P1 *= h1 * ho.y;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int j = kBwd ? i : 31 - i;                      // forward pass: rows from the end backwards
                const int r = 32 * half + j;
                const uint32_t off = xo[r & 7] + r * 128;
                float f0, f1, k0 = 0.f, k1 = 0.f;
                if (kEnc) {
                    gate_decode(fw[j], f0, k0);
                    gate_decode(fw[j] >> 16, f1, k1);
                } else {
                    f0 = bf16_lo(fw[j]);
                    f1 = bf16_hi(fw[j]);
                }
                if (kBwd) {                                           // c includes row r: X = q * prod_{<= r} f
                    a0 *= f0;
                    a1 *= f1;
                    uint32_t qw = *reinterpret_cast<const uint32_t *>(xbuf + off);
                    if (kRagged && r >= n_valid) qw = 0u;
                    *reinterpret_cast<uint32_t *>(xbuf + off) = mul_bf16x2(qw, pack_bf16(a0, a1));
                } else {                                              // c excludes row r: X = (1 - f) * prod_{> r} f
                    const uint32_t cp = pack_bf16(a0, a1);
                    *reinterpret_cast<uint32_t *>(xbuf + off) = kEnc ? mul_bf16x2(pack_bf16(k0, k1), cp) : fma_bf16x2(fw[j], cp ^ 0x80008000u, cp);
                    a0 *= f0;
                    a1 *= f1;
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(&ctl->t_done[s]);
        }
        if (lam != nullptr && half == 0)
            *reinterpret_cast<float2 *>(lam + (size_t)u * kD + col) = make_float2(P0, P1);

        // the accumulator, one row per thread (TMEM lane = key dimension = 32 * (warp % 4) + lane)
        mbar_wait(&ctl->acc_done, 0, abort_flag);
        tc_fence_after_sync();
        const int krow = 32 * (warp & 3) + lane;
        const uint32_t tl = tmem + (static_cast<uint32_t>(32 * (warp & 3)) << 16);
#pragma unroll 1
        for (int part = 0; part < 4; ++part) {
            uint32_t r[32];
            tmem_ld32(tl + 32 * part, r);
            tmem_wait_ld();
            float4 *dst = reinterpret_cast<float4 *>(out + ((size_t)u * kD + krow) * kD + 32 * part);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                dst[j] = make_float4(__uint_as_float(r[4 * j + 0]), __uint_as_float(r[4 * j + 1]),
                                     __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
        }
    } else if (warp == kWarpLoad) {
        // ================= L: TMA loads =================
        if (lane == 0) {
            int issued = 0;
            for (int n = 0; n < NC; ++n) {
                const int s = n % kStages, c = kBwd ? n : NC - 1 - n;
                uint8_t *st = smem + s * G::kStageBytes;
                if (n >= kStages) {
                    mbar_wait(&ctl->empty[s], ((n / kStages) - 1) & 1, abort_flag);
                    // never arm a barrier twice within one phase (the wait above returns at once on the time-out exit)
                    mbar_wait_drain(&ctl->full[s], ((n / kStages) - 1) & 1, 20000000ull);
                }
                mbar_arrive_expect_tx(&ctl->full[s], G::kStageBytes);
                for (int b = 0; b < 2; ++b) {
                    if (kBwd) tma_load_3d(st + G::kOffX + b * kSlab, &map_o, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                    tma_load_3d(st + G::kOffF + b * kSlab, &map_f, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                    tma_load_3d(st + G::kOffW + b * kSlab, &map_w, &ctl->full[s], 64 * b, row0 + c * kC, zu);
                }
                issued = n + 1;
            }
            ctl->l_issued = issued;
        }
    } else {
        // ================= M: accumulate X^T W =================
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, 128, 1, 1);           // X^T (MN-major) x W (MN-major)
            const uint64_t dx0 = smem_desc_sw128(smem_u32(smem) + G::kOffX, kSlab, 1024);
            const uint64_t dw0 = smem_desc_sw128(smem_u32(smem) + G::kOffW, kSlab, 1024);
            for (int n = 0; n < NC; ++n) {
                const int s = n % kStages;
                const uint64_t so = (uint64_t)s * (G::kStageBytes >> 4);
                mbar_wait(&ctl->t_done[s], (n / kStages) & 1, abort_flag);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_bf16_ss(tmem, dx0 + so + (uint64_t)(kk * 128), dw0 + so + (uint64_t)(kk * 128), idesc,
                                (n > 0 || kk > 0) ? 1u : 0u);
                mma_commit(&ctl->empty[s]);
            }
            mma_commit(&ctl->acc_done);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag) {
        report_error(status, HGRN2_ERR_TIMEOUT, 5);
        // the accumulator's last commit, then tiles asked for but never consumed
        mbar_wait_drain(&ctl->acc_done, 0, 20000000ull);
        const int ni = ctl->l_issued;
        for (int s = 0; s < kStages; ++s)
            if (ni > s) mbar_wait_drain(&ctl->full[s], ((ni - 1 - s) / kStages) & 1, 20000000ull);
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 128);
}

template <bool kBwd, bool kEnc, bool kRagged>
cudaError_t launch_state_t(const void *o, const void *f, const void *w, uint64_t planes, int N, uint64_t ctas, const int *cu,
                           float *out, float *lam, StatusBlock *status, bool clear, int start_aborted, cudaStream_t stream)
{
    using G = Geo<kBwd>;
    CUtensorMap mo, mf, mw;
    if (!make_map(&mo, kBwd ? o : f, planes, N, kC) || !make_map(&mf, f, planes, N, kC) || !make_map(&mw, w, planes, N, kC))
        return cudaErrorInvalidValue;
    auto kernel = tc_state_kernel<kBwd, kEnc, kRagged>;
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), G::kSmemBytes);
    if (err != cudaSuccess) return err;
    kernel<<<(unsigned)ctas, kThreads, G::kSmemBytes, stream>>>(mo, mf, mw, out, lam, N, N / kC, cu, (int)planes, status,
                                                             clear ? 1 : 0, start_aborted);
    return cudaGetLastError();
}

// planes x N rows; without offsets one CTA per plane, with offsets nseq CTAs per plane (see the kernel)
template <bool kBwd>
cudaError_t launch_state(const void *o, const void *f, const void *w, uint64_t planes, int N, const int *cu, int nseq,
                         float *out, float *lam, bool gate_enc, StatusBlock *status, bool clear, int start_aborted,
                         cudaStream_t stream)
{
    const bool ragged = cu != nullptr || N % kC != 0;
    const uint64_t ctas = cu ? planes * (uint64_t)nseq : planes;
    if (ctas == 0 || N <= 0) return cudaSuccess;
    if (ctas > 0x7fffffffull) return cudaErrorInvalidConfiguration;
    if (gate_enc)
        return ragged ? launch_state_t<kBwd, true, true>(o, f, w, planes, N, ctas, cu, out, lam, status, clear, start_aborted, stream)
                      : launch_state_t<kBwd, true, false>(o, f, w, planes, N, ctas, cu, out, lam, status, clear, start_aborted, stream);
    return ragged ? launch_state_t<kBwd, false, true>(o, f, w, planes, N, ctas, cu, out, lam, status, clear, start_aborted, stream)
                  : launch_state_t<kBwd, false, false>(o, f, w, planes, N, ctas, cu, out, lam, status, clear, start_aborted, stream);
}

}  // namespace

// Forward: S_loc [.][128][128] and Lambda [.][128] from f and i.  Without `cu`: one segment per plane, the N rows
// of each of the U planes.  With `cu` (device, nseq + 1 offsets): segment b * U + h = rows [cu[b], cu[b + 1]) of plane h.
cudaError_t launch_tc_state_fwd(const void *f, const void *i, uint64_t U, int N, float *S_loc, float *lam, bool gate_enc,
                                StatusBlock *status, bool clear, int start_aborted, cudaStream_t stream, const int *cu,
                                int nseq)
{
    return launch_state<false>(nullptr, f, i, U, N, cu, nseq, S_loc, lam, gate_enc, status, clear, start_aborted, stream);
}

// Backward: G_loc and Lambda of the same segments from o, f and dy.
cudaError_t launch_tc_state_bwd(const void *o, const void *f, const void *dy, uint64_t U, int N, float *G_loc,
                                float *lam, bool gate_enc, StatusBlock *status, bool clear, int start_aborted,
                                cudaStream_t stream, const int *cu, int nseq)
{
    return launch_state<true>(o, f, dy, U, N, cu, nseq, G_loc, lam, gate_enc, status, clear, start_aborted, stream);
}

}  // namespace hgrn2
