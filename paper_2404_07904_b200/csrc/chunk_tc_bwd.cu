// Chunkwise HGRN2 backward on the Blackwell tensor cores (tcgen05 + TMEM + TMA), bf16 I/O, fp32
// state gradient, d_k = d_v = 128, chunk length C = 64 (frame and formulas: tc_chunk.cuh).
#include "tc_chunk.cuh"

namespace hgrn2 {

namespace {

using namespace tc;

constexpr int kWorkers = 256;                   // warps 0..7: transforms, TMEM epilogues, outputs
constexpr int kThreads = kWorkers + 32;         // warp 8: TMA loads and tcgen05.mma issue (one lane)

__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// In-place rescaling of the raw o and f tiles of one chunk into Qs and Ks (see the file header).
// Thread layout: 64 column pairs x 4 row quarters; quarter q owns rows 16q..16q+15.  Quarter totals
// go through `tot`; Pm and E of the chunk are left in `pm` and `ee`.  Called by all 256 workers.
__device__ __forceinline__ void transform_chunk(uint8_t *qbuf, uint8_t *fbuf, float *tot, float *pm, float *ee,
                                                int n_valid, int tid)
{
    const int quarter = tid >> 6, p = tid & 63;
    const int col = 2 * p;
    const int jch = (col & 63) >> 3;
    const uint32_t base = (col >> 6) * kSlab + quarter * 16 * 128 + (col & 7) * 2;
    uint32_t xo[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) xo[jj] = base + ((jch ^ jj) << 4);   // row 16q + j has (row & 7) == (j & 7)
    uint32_t qw[16];
    float f0[16], f1[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint32_t off = xo[j & 7] + j * 128;
        uint32_t fw = *reinterpret_cast<const uint32_t *>(fbuf + off);
        qw[j] = *reinterpret_cast<const uint32_t *>(qbuf + off);
        if (quarter * 16 + j >= n_valid) {       // neutral padding token: f = 1, o = 0
            fw = 0x3F803F80u;
            qw[j] = 0u;
        }
        f0[j] = bf16_lo(fw);
        f1[j] = bf16_hi(fw);
    }
    // m0[j], m1[j]: product of f over the rows between row j and the middle of the chunk
    // (quarters 0, 1: rows j+1 .. 31; quarters 2, 3: rows 32 .. j), restricted to this quarter.
    float m0[16], m1[16];
    float t0, t1;
    if (quarter < 2) {
        float a0 = 1.f, a1 = 1.f;
#pragma unroll
        for (int j = 15; j >= 0; --j) {
            m0[j] = a0; m1[j] = a1;
            a0 *= f0[j]; a1 *= f1[j];
        }
        t0 = a0; t1 = a1;
    } else {
        float a0 = 1.f, a1 = 1.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            a0 *= f0[j]; a1 *= f1[j];
            m0[j] = a0; m1[j] = a1;
        }
        t0 = a0; t1 = a1;
    }
    *reinterpret_cast<float2 *>(tot + quarter * 128 + col) = make_float2(t0, t1);
    worker_sync();
    float o0 = 1.f, o1 = 1.f;
    if (quarter == 0) { const float2 x = *reinterpret_cast<const float2 *>(tot + 128 + col); o0 = x.x; o1 = x.y; }
    if (quarter == 3) { const float2 x = *reinterpret_cast<const float2 *>(tot + 256 + col); o0 = x.x; o1 = x.y; }
    if (quarter == 0)
        *reinterpret_cast<float2 *>(pm + col) = make_float2(fmaxf(t0 * o0, kProdFloor), fmaxf(t1 * o1, kProdFloor));
    if (quarter == 3)
        *reinterpret_cast<float2 *>(ee + col) = make_float2(fmaxf(t0 * o0, kProdFloor), fmaxf(t1 * o1, kProdFloor));
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint32_t off = xo[j & 7] + j * 128;
        const float mm0 = fmaxf(m0[j] * o0, kProdFloor), mm1 = fmaxf(m1[j] * o1, kProdFloor);
        const float i0 = rcp_fast(mm0), i1 = rcp_fast(mm1);
        const float sq0 = quarter < 2 ? i0 : mm0, sq1 = quarter < 2 ? i1 : mm1;
        const float sk0 = quarter < 2 ? mm0 : i0, sk1 = quarter < 2 ? mm1 : i1;
        const float q0 = bf16_lo(qw[j]), q1 = bf16_hi(qw[j]);
        *reinterpret_cast<uint32_t *>(qbuf + off) = pack_bf16(q0 * sq0, q1 * sq1);
        *reinterpret_cast<uint32_t *>(fbuf + off) = pack_bf16((1.f - f0[j]) * sk0, (1.f - f1[j]) * sk1);
    }
}

// One 64 x 128 fp32 accumulator (M = 64 layout) to a bf16 [token][128] global tensor.
__device__ __forceinline__ void rows_to_global(uint32_t taddr_half, __nv_bfloat16 *dst_row0, int sub, int half,
                                               int lane, int n_valid)
{
    uint32_t r[32];
    const int t = 16 * sub + lane;
#pragma unroll
    for (int part = 0; part < 2; ++part) {
        tmem_ld32(taddr_half + 32 * part, r);
        tmem_wait_ld();
        if (lane < 16 && t < n_valid) {
            uint4 *dst = reinterpret_cast<uint4 *>(dst_row0 + (size_t)t * kD + 64 * half + 32 * part);
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j] = pack8(r + 8 * j);
        }
    }
}

// ---- backward ---------------------------------------------------------------------------------------
// Reverse sweep over the chunks with the state gradient resident in tensor memory.  In the mid frame
// (file header), with dS'' = Diag(E) dS_out and S' the saved forward state of the chunk:
//
//   A  = tril(Qs Ks^T)          dA = tril(dY V^T)
//   dQs^T       = Ks^T dA^T + S' dY^T            (accumulator [key dim][t]: lane = key dim)
//   dKs_intra^T = Qs^T dA                        (accumulator [key dim][s])
//   dKs_inter^T = dS'' V^T                       (accumulator [key dim][s])
//   dV          = A^T dY + Ks dS''               (accumulator [s][value dim])
//   dS'         = dS'' + Qs^T dY,   dS_in = Diag(Pm) dS'
//   a = Qs*dQs - Ks*dKs_intra,  e = Ks*dKs_inter,  R_k = sum_v dS''[k,v] S'[k,v]
//   dg_t = sum_{j>=t} a_j + sum_{s<t} e_s + R            (gradient w.r.t. log f_t; no cancellation
//                                                         between the inter-chunk terms)
//   d_o = dQs * exp(b_t - b_m),  dk = (dKs_intra + dKs_inter) * exp(b_m - b_s),  d_f = dg / f - dk
//
// The three key-dimension-major accumulators put one key dimension in each TMEM lane, so the thread
// that owns the lane sees a whole column of the chunk and the scans along time stay in registers.
// Tensor-memory plan: dS [0,128); A [128,192) and dA [192,256) first, then dQs^T and dKs_intra^T in
// the same columns; dKs_inter^T [256,320); dV [320,448).
//
// Worker schedule per processed chunk `it` (chunk index c = NC-1-it):
//   P/dP epilogue(it) | transform(it+1) | dV epilogue(it), d_o/d_f phase(it) | dS maintenance(it+1)
// so the second group of MMAs overlaps the next transform.  The raw-tile stage is released to TMA as
// soon as the d_o/d_f phase has read Qs and Ks from it.
constexpr int kBwdStages = 2;
constexpr uint32_t kBwdStageBytes = 4 * kTile;                        // q, f, v, dy
constexpr uint32_t kBwdOffS = kBwdStages * kBwdStageBytes;            // S' (bf16, from the forward)
constexpr uint32_t kBwdOffDS = kBwdOffS + kStateTile;                 // bf16 copy of dS''
constexpr uint32_t kBwdOffP = kBwdOffDS + kStateTile;                 // bf16 tril(A)
constexpr uint32_t kBwdOffDP = kBwdOffP + kSlab;                      // bf16 tril(dA)
constexpr uint32_t kBwdOffTot = kBwdOffDP + kSlab;                    // float tot[4][128]
constexpr uint32_t kBwdOffPm = kBwdOffTot + 4 * 128 * 4;
constexpr uint32_t kBwdOffE = kBwdOffPm + 128 * 4;
constexpr uint32_t kBwdOffR = kBwdOffE + 128 * 4;                     // float rpart[2][128]
constexpr uint32_t kBwdOffX = kBwdOffR + 2 * 128 * 4;                 // float xa[128], xe[128]
constexpr uint32_t kBwdOffBar = kBwdOffX + 2 * 128 * 4;
constexpr uint32_t kBwdSmemBytes = kBwdOffBar + 256 + 1024;

constexpr uint32_t kColDS = 0, kColA2 = 128, kColDA = 192, kColDQ = 128, kColDKi = 192, kColDKx = 256, kColDV = 320;

struct BwdCtl {
    uint64_t full[kBwdStages];     // TMA (raw tiles) -> workers
    uint64_t sfull;                // TMA (saved S') -> workers
    uint64_t g1_ready;             // workers -> issuer: Qs, Ks, dS'' ready: first MMA group may go
    uint64_t pd_ready;             // workers -> issuer: tril(A), tril(dA) in shared memory: second group may go
    uint64_t f_done;               // workers -> issuer: the chunk's stage has been read for the last time
    uint64_t bar1, bar2;           // tcgen05.commit -> workers
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap map_o, const __grid_constant__ CUtensorMap map_f,
              const __grid_constant__ CUtensorMap map_i, const __grid_constant__ CUtensorMap map_dy,
              const __grid_constant__ CUtensorMap map_saved, const __nv_bfloat16 *__restrict__ f_gmem,
              const float *__restrict__ dSN, __nv_bfloat16 *__restrict__ d_o, __nv_bfloat16 *__restrict__ d_f,
              __nv_bfloat16 *__restrict__ d_i, float *__restrict__ dS0, int N, int NC, StatusBlock *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sbuf = smem + kBwdOffS;
    uint8_t *dsbuf = smem + kBwdOffDS;
    uint8_t *pbuf = smem + kBwdOffP;
    uint8_t *dpbuf = smem + kBwdOffDP;
    float *tot = reinterpret_cast<float *>(smem + kBwdOffTot);
    float *pm = reinterpret_cast<float *>(smem + kBwdOffPm);
    float *ee = reinterpret_cast<float *>(smem + kBwdOffE);
    float *rpart = reinterpret_cast<float *>(smem + kBwdOffR);
    float *xa = reinterpret_cast<float *>(smem + kBwdOffX);
    float *xe = xa + 128;
    BwdCtl *ctl = reinterpret_cast<BwdCtl *>(smem + kBwdOffBar);
    volatile int *abort_flag = &ctl->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int u = blockIdx.x;

    if (tid == 0) {
        for (int s = 0; s < kBwdStages; ++s) mbar_init(&ctl->full[s], 1);
        mbar_init(&ctl->sfull, 1);
        mbar_init(&ctl->g1_ready, kWorkers);
        mbar_init(&ctl->pd_ready, kWorkers);
        mbar_init(&ctl->f_done, kWorkers);
        mbar_init(&ctl->bar1, 1);
        mbar_init(&ctl->bar2, 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&map_o);
        tma_prefetch_desc(&map_f);
        tma_prefetch_desc(&map_i);
        tma_prefetch_desc(&map_dy);
        tma_prefetch_desc(&map_saved);
    }
    if (warp == 0) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 8) {
        // ================= issuer =================
        if (lane == 0) {
            constexpr uint32_t idA = idesc_bf16(64, 64, 0, 0);        // Qs x Ks^T, dY x V^T
            constexpr uint32_t idKX = idesc_bf16(128, 64, 0, 0);      // dS'' (K-major) x V (K-major); S' x dY
            constexpr uint32_t idDV2 = idesc_bf16(64, 128, 0, 1);     // Ks (K-major) x dS'' (MN-major)
            constexpr uint32_t idDS = idesc_bf16(128, 128, 1, 1);     // Qs^T (MN-major) x dY (MN-major)
            constexpr uint32_t idDQ1 = idesc_bf16(128, 64, 1, 0);     // Ks^T (MN-major) x dA^T (dP K-major)
            constexpr uint32_t idDKi = idesc_bf16(128, 64, 1, 1);     // Qs^T (MN-major) x dA (dP MN-major)
            constexpr uint32_t idDV1 = idesc_bf16(64, 128, 1, 1);     // P^T (MN-major) x dY (MN-major)
            // it = 0, 1, ... counts processed chunks; chunk index c = NC - 1 - it
            auto issue_loads = [&](int it) {
                const int s = it % kBwdStages, c = NC - 1 - it;
                uint8_t *st = smem + s * kBwdStageBytes;
                mbar_arrive_expect_tx(&ctl->full[s], kBwdStageBytes);
                for (int b = 0; b < 2; ++b) {
                    tma_load_3d(st + b * kSlab, &map_o, &ctl->full[s], 64 * b, c * kC, u);
                    tma_load_3d(st + kTile + b * kSlab, &map_f, &ctl->full[s], 64 * b, c * kC, u);
                    tma_load_3d(st + 2 * kTile + b * kSlab, &map_i, &ctl->full[s], 64 * b, c * kC, u);
                    tma_load_3d(st + 3 * kTile + b * kSlab, &map_dy, &ctl->full[s], 64 * b, c * kC, u);
                }
            };
            auto issue_state_load = [&](int it) {
                const int c = NC - 1 - it;
                mbar_arrive_expect_tx(&ctl->sfull, kStateTile);
                for (int b = 0; b < 2; ++b)
                    tma_load_3d(sbuf + b * kStateSlab, &map_saved, &ctl->sfull, 64 * b, 0, u * NC + c);
            };
            for (int it = 0; it < kBwdStages && it < NC; ++it) issue_loads(it);
            issue_state_load(0);
            const uint32_t sa = smem_u32(sbuf), dsa = smem_u32(dsbuf), pa = smem_u32(pbuf), dpa = smem_u32(dpbuf);
            for (int it = 0; it < NC; ++it) {
                const uint32_t qa = smem_u32(smem + (it % kBwdStages) * kBwdStageBytes);
                const uint32_t fa = qa + kTile, va = qa + 2 * kTile, ga = qa + 3 * kTile;
                mbar_wait(&ctl->g1_ready, it & 1, abort_flag);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            // A = Qs Ks^T
                    const uint32_t koff = (kk >> 2) * kSlab + (kk & 3) * 32;
                    mma_bf16_ss(tmem + kColA2, smem_desc_sw128(qa + koff, 16, 1024),
                                smem_desc_sw128(fa + koff, 16, 1024), idA, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            // dA = dY V^T
                    const uint32_t koff = (kk >> 2) * kSlab + (kk & 3) * 32;
                    mma_bf16_ss(tmem + kColDA, smem_desc_sw128(ga + koff, 16, 1024),
                                smem_desc_sw128(va + koff, 16, 1024), idA, kk > 0);
                }
                mma_commit(&ctl->bar1);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            // dKs_inter^T = dS'' V^T
                    const uint32_t ko_s = (kk >> 2) * kStateSlab + (kk & 3) * 32;
                    const uint32_t koff = (kk >> 2) * kSlab + (kk & 3) * 32;
                    mma_bf16_ss(tmem + kColDKx, smem_desc_sw128(dsa + ko_s, 16, 1024),
                                smem_desc_sw128(va + koff, 16, 1024), idKX, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            // dV = Ks dS''
                    const uint32_t koff = (kk >> 2) * kSlab + (kk & 3) * 32;
                    mma_bf16_ss(tmem + kColDV, smem_desc_sw128(fa + koff, 16, 1024),
                                smem_desc_sw128(dsa + kk * 2048, kStateSlab, 1024), idDV2, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dS' = dS'' + Qs^T dY
                    mma_bf16_ss(tmem + kColDS, smem_desc_sw128(qa + kk * 2048, kSlab, 1024),
                                smem_desc_sw128(ga + kk * 2048, kSlab, 1024), idDS, 1);
                mbar_wait(&ctl->pd_ready, it & 1, abort_flag);
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dQs^T = Ks^T dA^T
                    mma_bf16_ss(tmem + kColDQ, smem_desc_sw128(fa + kk * 2048, kSlab, 1024),
                                smem_desc_sw128(dpa + kk * 32, 16, 1024), idDQ1, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            //        + S' dY^T
                    const uint32_t ko_s = (kk >> 2) * kStateSlab + (kk & 3) * 32;
                    const uint32_t koff = (kk >> 2) * kSlab + (kk & 3) * 32;
                    mma_bf16_ss(tmem + kColDQ, smem_desc_sw128(sa + ko_s, 16, 1024),
                                smem_desc_sw128(ga + koff, 16, 1024), idKX, 1);
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dKs_intra^T = Qs^T dA
                    mma_bf16_ss(tmem + kColDKi, smem_desc_sw128(qa + kk * 2048, kSlab, 1024),
                                smem_desc_sw128(dpa + kk * 2048, kSlab, 1024), idDKi, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)              // dV += P^T dY
                    mma_bf16_ss(tmem + kColDV, smem_desc_sw128(pa + kk * 2048, kSlab, 1024),
                                smem_desc_sw128(ga + kk * 2048, kSlab, 1024), idDV1, 1);
                mma_commit(&ctl->bar2);
                // S' of this chunk is dead once the second group is complete: fetch the next one
                mbar_wait(&ctl->bar2, it & 1, abort_flag);
                if (it + 1 < NC) issue_state_load(it + 1);
                // the raw-tile stage is dead once the workers have read Qs and Ks for d_o / d_f
                mbar_wait(&ctl->f_done, it & 1, abort_flag);
                if (it + kBwdStages < NC) issue_loads(it + kBwdStages);
            }
        }
    } else {
        // ================= workers =================
        const int sub = warp & 3, half = warp >> 2;
        const uint32_t lane_base = static_cast<uint32_t>(32 * sub) << 16;
        const int krow = 32 * sub + lane;
        float pm_prev = 1.f;

        // dS'' = (Pm_prev E) dS' (the accumulator, or dSN first), bf16 copy, partial sums of R
        auto maintain = [&](bool first) {
            const float factor = pm_prev * ee[krow];
            pm_prev = pm[krow];
            float racc = 0.f;
            uint32_t r[32];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const int v0 = 64 * half + 32 * part;
                if (first) {
                    if (dSN) {
                        const float4 *src = reinterpret_cast<const float4 *>(dSN + ((size_t)u * kD + krow) * kD + v0);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float4 x = __ldg(src + j);
                            r[4 * j + 0] = __float_as_uint(x.x); r[4 * j + 1] = __float_as_uint(x.y);
                            r[4 * j + 2] = __float_as_uint(x.z); r[4 * j + 3] = __float_as_uint(x.w);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                    }
                } else {
                    tmem_ld32(tmem + lane_base + kColDS + v0, r);
                    tmem_wait_ld();
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * factor);
                tmem_st32(tmem + lane_base + kColDS + v0, r);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t off = half * kStateSlab + slab_chunk_off(krow, 4 * part + j);
                    const uint4 sw = *reinterpret_cast<const uint4 *>(sbuf + off);
                    racc = fmaf(__uint_as_float(r[8 * j + 0]), bf16_lo(sw.x), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 1]), bf16_hi(sw.x), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 2]), bf16_lo(sw.y), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 3]), bf16_hi(sw.y), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 4]), bf16_lo(sw.z), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 5]), bf16_hi(sw.z), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 6]), bf16_lo(sw.w), racc);
                    racc = fmaf(__uint_as_float(r[8 * j + 7]), bf16_hi(sw.w), racc);
                    *reinterpret_cast<uint4 *>(dsbuf + off) = pack8(r + 8 * j);
                }
            }
            rpart[half * 128 + krow] = racc;
            tmem_wait_st();
            tc_fence_before_sync();
            fence_proxy_async_smem();
            mbar_arrive(&ctl->g1_ready);
        };

        mbar_wait(&ctl->full[0], 0, abort_flag);
        transform_chunk(smem, smem + kTile, tot, pm, ee, min(kC, N - (NC - 1) * kC), tid);
        worker_sync();
        mbar_wait(&ctl->sfull, 0, abort_flag);
        maintain(true);
        PT_DECL

        for (int it = 0; it < NC; ++it) {
            const int c = NC - 1 - it;
            uint8_t *qbuf = smem + (it % kBwdStages) * kBwdStageBytes;
            uint8_t *fbuf = qbuf + kTile;
            const int n_valid = min(kC, N - c * kC);

            // tril(A), tril(dA) -> shared memory
            mbar_wait(&ctl->bar1, it & 1, abort_flag);
            tc_fence_after_sync();
            PT_MARK(0)
            tril_to_slab(tmem + lane_base + kColA2 + 32 * half, pbuf, sub, half, lane);
            tril_to_slab(tmem + lane_base + kColDA + 32 * half, dpbuf, sub, half, lane);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&ctl->pd_ready);
            PT_MARK(1)

            // next chunk's operands while the second MMA group runs
            if (it + 1 < NC) {
                const int s1 = (it + 1) % kBwdStages;
                uint8_t *qn = smem + s1 * kBwdStageBytes;
                mbar_wait(&ctl->full[s1], ((it + 1) / kBwdStages) & 1, abort_flag);
                PT_MARK(2)
                transform_chunk(qn, qn + kTile, tot, pm, ee, min(kC, N - (c - 1) * kC), tid);
                worker_sync();
                PT_MARK(3)
            }

            mbar_wait(&ctl->bar2, it & 1, abort_flag);
            tc_fence_after_sync();
            PT_MARK(4)

            // d_i = dV
            rows_to_global(tmem + lane_base + kColDV + 64 * half, d_i + ((size_t)u * N + (size_t)c * kC) * kD, sub,
                           half, lane, n_valid);
            PT_MARK(5)

            // d_o and d_f: thread (krow, half) owns key dimension krow and local times 32*half .. 32*half+31
            {
                const int tb = 32 * half;
                const size_t gbase = ((size_t)u * N + (size_t)c * kC + tb) * kD + krow;
                const int kch = (krow & 63) >> 3;
                const uint32_t kbase = (krow >> 6) * kSlab + tb * 128 + (krow & 7) * 2;
                uint32_t xo[8];
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) xo[jj] = kbase + ((kch ^ jj) << 4);    // (tb + j) & 7 == j & 7
                float fv[32], m[32];
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    fv[j] = (tb + j < n_valid) ? __bfloat162float(f_gmem[gbase + (size_t)j * kD]) : 1.f;
                if (half == 0) {
                    float acc = 1.f;
#pragma unroll
                    for (int j = 31; j >= 0; --j) { m[j] = fmaxf(acc, kProdFloor); acc *= fv[j]; }
                } else {
                    float acc = 1.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) { acc *= fv[j]; m[j] = fmaxf(acc, kProdFloor); }
                }
                float a[32], dks[32], ev[32];
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + kColDQ + tb, r);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float qs = __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(qbuf + xo[j & 7] + j * 128));
                    const float x = __uint_as_float(r[j]);
                    a[j] = qs * x;
                    const float mi = rcp_fast(m[j]);
                    const float sq = half == 0 ? mi : m[j];
                    m[j] = half == 0 ? m[j] : mi;            // from here on m holds exp(b_m - b_s)
                    if (tb + j < n_valid) d_o[gbase + (size_t)j * kD] = __float2bfloat16_rn(x * sq);
                }
                tmem_ld32(tmem + lane_base + kColDKi + tb, r);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float ks = __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(fbuf + xo[j & 7] + j * 128));
                    const float x = __uint_as_float(r[j]);
                    a[j] = fmaf(-ks, x, a[j]);
                    dks[j] = x;
                    ev[j] = ks;
                }
                mbar_arrive(&ctl->f_done);          // last read of this chunk's stage
                tmem_ld32(tmem + lane_base + kColDKx + tb, r);
                tmem_wait_ld();
                float asum = 0.f, esum = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float x = __uint_as_float(r[j]);
                    dks[j] = (dks[j] + x) * m[j];
                    ev[j] *= x;
                    asum += a[j];
                    esum += ev[j];
                }
                if (half == 1) xa[krow] = asum;       // each written by exactly one of the two threads of a key dim
                if (half == 0) xe[krow] = esum;
                const float R = rpart[krow] + rpart[128 + krow];
                PT_MARK(6)
                worker_sync();
                PT_MARK(7)
                float pre = (half == 1) ? xe[krow] : 0.f;
                float suf = (half == 0) ? xa[krow] : 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {        // exclusive prefix sums of e
                    const float e = ev[j];
                    ev[j] = pre;
                    pre += e;
                }
#pragma unroll
                for (int j = 31; j >= 0; --j) {
                    suf += a[j];
                    const float dg = R + suf + ev[j];
                    if (tb + j < n_valid)
                        d_f[gbase + (size_t)j * kD] =
                            __float2bfloat16_rn(fmaf(dg, rcp_fast(fmaxf(fv[j], kProdFloor)), -dks[j]));
                }
            }
            tc_fence_before_sync();
            PT_MARK(8)

            if (it + 1 < NC) {
                mbar_wait(&ctl->sfull, (it + 1) & 1, abort_flag);
                PT_MARK(9)
                maintain(false);
                PT_MARK(10)
            }
        }
        PT_DUMP(status, 0, 12, tid == 0)

        // dS_0 = Diag(Pm of chunk 0) dS'
        if (dS0) {
            tc_fence_after_sync();
            uint32_t r[32];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const int v0 = 64 * half + 32 * part;
                tmem_ld32(tmem + lane_base + kColDS + v0, r);
                tmem_wait_ld();
                float4 *dst = reinterpret_cast<float4 *>(dS0 + ((size_t)u * kD + krow) * kD + v0);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    dst[j] = make_float4(__uint_as_float(r[4 * j + 0]) * pm_prev, __uint_as_float(r[4 * j + 1]) * pm_prev,
                                         __uint_as_float(r[4 * j + 2]) * pm_prev, __uint_as_float(r[4 * j + 3]) * pm_prev);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag) report_error(status, HGRN2_ERR_TIMEOUT, 2);
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t launch_tc_bwd(const SeqArgs &a)
{
    const uint64_t U = (uint64_t)a.B * a.H;
    CUtensorMap mo, mf, mi, mg, ms;
    if (!make_map(&mo, a.o, U, a.N, kC) || !make_map(&mf, a.f, U, a.N, kC) || !make_map(&mi, a.i, U, a.N, kC) ||
        !make_map(&mg, a.dy, U, a.N, kC) || !make_map(&ms, a.states, U * a.NC, kD, kD))
        return cudaErrorInvalidValue;
    cudaError_t err = cudaFuncSetAttribute(tc_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBwdSmemBytes);
    if (err != cudaSuccess) return err;
    tc_bwd_kernel<<<(unsigned)U, kThreads, kBwdSmemBytes, a.stream>>>(
        mo, mf, mi, mg, ms, static_cast<const __nv_bfloat16 *>(a.f), a.dSN, static_cast<__nv_bfloat16 *>(a.d_o),
        static_cast<__nv_bfloat16 *>(a.d_f), static_cast<__nv_bfloat16 *>(a.d_i), a.dS0, a.N, a.NC, a.status);
    return cudaGetLastError();
}

}  // namespace hgrn2
