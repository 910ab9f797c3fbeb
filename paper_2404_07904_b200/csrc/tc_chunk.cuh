// Pieces shared by the tensor-core forward and backward kernels: tile geometry, the in-place
// operand transform of one chunk, accumulator-to-operand conversions and the TMA tensor maps.
//
// Mid-chunk reference frame.  Within a chunk of C = 64 steps let b_j = sum_{r<=j} log f_r (per key
// dimension) and let m be the middle of the chunk (after local row 31).  Only two rescaled operands
// are formed:
//
//     Qs_t = q_t * exp(b_t - b_m)          Ks_s = k_s * exp(b_m - b_s)          (q = o, k = 1 - f)
//
// so that Qs_t . Ks_s = q_t k_s exp(b_t - b_s) for every pair, and with Pm = exp(b_m),
// E = exp(b_C - b_m) (per key dimension):
//
//     A  = tril(Qs Ks^T)                       S' = Diag(Pm) S_in      (state in the mid frame)
//     Y  = A V + Qs S'                         S_out = Diag(E) (S' + Ks^T V)
//
// The factors exp(b_t - b_m) are in-chunk cumulative PRODUCTS of f taken outward from the middle
// (the linear-space image of the log-space cumulative sum): rows after m multiply by prod f, rows
// before m divide by it.  The two factors of a pair can be represented only while the decay across each
// half of the chunk stays above 2^-100 per key dimension.  The totals Pm and E are floored there; a half whose
// total sits on the floor has left the range, which the state warps of both kernels see when they pick the
// totals up: they raise the CTA's exact-path flag and the kernels then redo the whole unit with the
// pairwise-safe fp32 routines of chunk_alu.cuh, which hold on all of [0, 1].  The running products inside a
// half are NOT floored (every one of them is at least as large as the half's total, so inside the range none
// needs it, and two instructions per element pair in the role that paces the forward are worth 5 % of it):
// outside the range they may reach zero and the operands Inf or NaN, which stay inside that unit's own
// accumulators and outputs, all of which the exact path then rewrites.
#pragma once

#include "tc_common.cuh"

namespace hgrn2 {
namespace tc {

constexpr int kC = 64;                          // chunk length
constexpr int kD = 128;                         // d_k = d_v
constexpr uint32_t kSlab = kC * 128;            // bytes of one slab of a [64][128] bf16 tile
constexpr uint32_t kTile = 2 * kSlab;           // one [64][128] bf16 tile
constexpr uint32_t kStateSlab = kD * 128;       // bytes of one slab of a [128][128] bf16 state copy
constexpr uint32_t kStateTile = 2 * kStateSlab;
constexpr float kProdFloor = 7.888609052210118e-31f;   // 2^-100
constexpr float kFactorSafe = 7.52316384526264e-37f;    // 2^-120: below it the product of two decay totals is applied in two steps
constexpr uint32_t kTmemCols = 512;
constexpr int kTransformThreads = 128;          // threads that run transform_stream together
// Saved-for-backward buffer of the tensor-core path, per (unit, chunk): the bf16 state S' in the mid
// frame ([128][128]), then, after all states, the decay totals Pm[128], E[128] (float) of every chunk.
constexpr size_t kSavedStateBytes = (size_t)kD * kD * 2;
constexpr size_t kSavedTotalsBytes = 2 * kD * sizeof(float);

// Optional per-role cycle counters of CTA 0 (development aid; compiled out unless HGRN2_PHASE_TIMING
// is defined).  Totals land in the padding words of the status block.
#ifdef HGRN2_PHASE_TIMING
#define PT_DECL long long pt_t0 = clock64(); long long pt_acc[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
#define PT_MARK(i) { const long long pt_t = clock64(); pt_acc[i] += pt_t - pt_t0; pt_t0 = pt_t; }
#define PT_DUMP(st, base, n, cond) if ((cond) && blockIdx.x == 0 && (st) != nullptr) { for (int pt_i = 0; pt_i < (n); ++pt_i) (st)->pad[(base) + pt_i] = (int)(pt_acc[pt_i] >> 4); }
#define PT_STAMP(st, idx, cond) if (blockIdx.x == 0 && (cond) && (st) != nullptr) (st)->pad[30 + (idx)] = (int)(clock64() & 0x3fffffff);
#else
#define PT_STAMP(st, idx, cond)
#define PT_DECL
#define PT_MARK(i)
#define PT_DUMP(st, base, n, cond)
#endif

// Signed gate encoding (kEnc): bits of one bf16 value in the low half of w -> f and k = 1 - f.  Sign clear: the
// magnitude is f; sign set: the magnitude is k (so the neutral token f = 1, k = 0 is 0x8000).
__device__ __forceinline__ void gate_decode(uint32_t w, float &f, float &k)
{
    const float m = __uint_as_float((w & 0x7FFFu) << 16);
    const bool is_k = (w & 0x8000u) != 0u;
    f = is_k ? 1.0f - m : m;
    k = is_k ? m : 1.0f - m;
}

__device__ __forceinline__ float rcp_fast(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ uint4 pack8(const uint32_t *r)
{
    uint4 w;
    w.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
    w.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
    w.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
    w.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
    return w;
}

// In-place rescaling of the raw o and f tiles of one chunk into Qs and Ks (see the file header).
// Run by 128 threads with no synchronisation among them: thread = one column pair x one half of the
// chunk.  The half before the middle walks its rows downwards from row 31, the half after it walks
// upwards from row 32, each carrying the running product of f, so only a few rows are live.  Rows are
// handled in batches of eight, and the loads of the next batch are issued before the stores of the
// current one (the tiles are rewritten in place, so the compiler would otherwise serialise every
// load behind the previous row's stores).  Pm (product over rows 0..31) and E (product over rows
// 32..63) of the chunk are left in pm[128] and ee[128] (shared memory) and / or pm_g[128], ee_g[128]
// (global memory); either pair may be null.  Rows at or beyond n_valid are the neutral token
// f = 1, o = 0.  kEnc: the gate tile holds the SMALLER of f and k = 1 - f, with the sign bit set when it is k
// (gate_decode below).  The gated entry points hand the kernels that: bf16 then resolves the gate to 2^-9 of
// min(f, 1 - f) at both ends of [0, 1], whereas a bf16 f close to 1 would distort every decay product.
template <bool kFull, bool kUp, uint32_t kQSlabStride, uint32_t kFSlabStride, bool kEnc>
__device__ __forceinline__ void transform_half(uint8_t *qbuf, uint8_t *fbuf, float *tot, float *tot_g, int n_valid,
                                               int p)
{
    const int col = 2 * p;
    const int jch = (col & 63) >> 3;
    const uint32_t base = (col >> 6) * kQSlabStride + (col & 7) * 2;
    if (kFSlabStride != kQSlabStride && (col >> 6)) fbuf -= kQSlabStride - kFSlabStride;   // offsets below are the q tile's
    uint32_t xo[8];
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) xo[jj] = base + ((jch ^ jj) << 4);
    auto row_of = [](int i) { return kUp ? 32 + i : 31 - i; };     // i-th row visited
    uint32_t fw[8], qw[8], fn[8], qn[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int r = row_of(j);
        const uint32_t off = xo[r & 7] + r * 128;
        fn[j] = *reinterpret_cast<const uint32_t *>(fbuf + off);
        qn[j] = *reinterpret_cast<const uint32_t *>(qbuf + off);
    }
    float a0 = 1.f, a1 = 1.f;
#pragma unroll 1
    for (int b = 0; b < 4; ++b) {      // kept rolled: the body is long and every transform warp streams through it
#pragma unroll
        for (int j = 0; j < 8; ++j) { fw[j] = fn[j]; qw[j] = qn[j]; }
        if (b < 3) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int r = row_of(8 * (b + 1) + j);
                const uint32_t off = xo[r & 7] + r * 128;
                fn[j] = *reinterpret_cast<const uint32_t *>(fbuf + off);
                qn[j] = *reinterpret_cast<const uint32_t *>(qbuf + off);
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int r = row_of(8 * b + j);
            const uint32_t off = xo[r & 7] + r * 128;
            if (!kFull && r >= n_valid) { fw[j] = kEnc ? 0x80008000u : 0x3F803F80u; qw[j] = 0u; }
            float f0, f1, k0 = 0.f, k1 = 0.f;
            if (kEnc) {
                gate_decode(fw[j], f0, k0);
                gate_decode(fw[j] >> 16, f1, k1);
            } else {
                f0 = bf16_lo(fw[j]);
                f1 = bf16_hi(fw[j]);
            }
            if (kUp) { a0 *= f0; a1 *= f1; }
            const float i0 = rcp_fast(a0), i1 = rcp_fast(a1);            // no floor: see the file header
            const float sq0 = kUp ? a0 : i0, sq1 = kUp ? a1 : i1;
            const float sk0 = kUp ? i0 : a0, sk1 = kUp ? i1 : a1;
            if (!kUp) { a0 *= f0; a1 *= f1; }
            // packed bf16 arithmetic: the scale factors are rounded to bf16 first, then one bf16x2 multiply
            // (resp. fused multiply-add for k = 1 - f) produces the operand pair
            const uint32_t sqp = pack_bf16(sq0, sq1), skp = pack_bf16(sk0, sk1);
            *reinterpret_cast<uint32_t *>(qbuf + off) = mul_bf16x2(qw[j], sqp);
            *reinterpret_cast<uint32_t *>(fbuf + off) = kEnc ? mul_bf16x2(pack_bf16(k0, k1), skp)
                                                             : fma_bf16x2(fw[j], skp ^ 0x80008000u, skp);
        }
    }
    // the products only shrink along the walk, so the last one tells whether the half stayed inside the range
    const float2 t2 = make_float2(fmaxf(a0, kProdFloor), fmaxf(a1, kProdFloor));
    if (tot) *reinterpret_cast<float2 *>(tot + col) = t2;
    if (tot_g) *reinterpret_cast<float2 *>(tot_g + col) = t2;
}

// kQSlabStride, kFSlabStride: distance in bytes between the two 64-column slabs of the q tile and of the f tile.
template <bool kFull, bool kEnc, uint32_t kQSlabStride = kSlab, uint32_t kFSlabStride = kSlab>
__device__ __forceinline__ void transform_stream(uint8_t *qbuf, uint8_t *fbuf, float *pm, float *ee, float *pm_g,
                                                 float *ee_g, int n_valid, int tid)
{
    if (tid >> 6) transform_half<kFull, true, kQSlabStride, kFSlabStride, kEnc>(qbuf, fbuf, ee, ee_g, n_valid, tid & 63);
    else          transform_half<kFull, false, kQSlabStride, kFSlabStride, kEnc>(qbuf, fbuf, pm, pm_g, n_valid, tid & 63);
}

// Causal mask + bf16 of 32 columns (32 * half ...) of one 64 x 64 fp32 accumulator in the M = 64
// layout (row r -> lane 32 * (r / 16) + r % 16) into a K-major slab.  `sub` = TMEM lane quarter.
__device__ __forceinline__ void tril_to_slab(uint32_t taddr, uint8_t *dstbuf, int sub, int half, int lane)
{
    uint32_t r[32];
    tmem_ld32(taddr, r);
    tmem_wait_ld();
    if (lane < 16) {
        const int t = 16 * sub + lane;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int s0 = 32 * half + 8 * j;
            uint32_t x[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) x[q] = (s0 + q <= t) ? r[8 * j + q] : 0u;
            *reinterpret_cast<uint4 *>(dstbuf + slab_chunk_off(t, 4 * half + j)) = pack8(x);
        }
    }
}

// Causal mask + bf16 of columns [32 * half, +32) of row t of a 64 x 64 fp32 accumulator whose rows sit one per
// TMEM lane (taddr = this thread's lane, first of the 32 columns) into a K-major slab.  The 32 threads of the
// warp hold 32 consecutive rows; a block that lies wholly above the diagonal is zero and is not read.
__device__ __forceinline__ void tril_row_block(uint32_t taddr, uint8_t *dstbuf, int t, int half)
{
    if (32 * half > (t | 31)) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4 *>(dstbuf + slab_chunk_off(t, 4 * half + j)) = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    uint32_t r[32];
    tmem_ld32(taddr, r);
    tmem_wait_ld();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int s0 = 32 * half + 8 * j;
        uint32_t x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) x[q] = (s0 + q <= t) ? r[8 * j + q] : 0u;
        *reinterpret_cast<uint4 *>(dstbuf + slab_chunk_off(t, 4 * half + j)) = pack8(x);
    }
}

// Where segment r of unit u sits among the segment summaries (chunk_tc_fwd.cu, sequences split into segments):
// order 0: u * G + r; order 1: r * U + u (ragged segments of an ordinary batch); order 2: unit u = (sequence b,
// head h) of a packed batch with H heads, its segment r at (b * G + r) * H + h.
__device__ __forceinline__ size_t seg_index(int order, size_t u, int r, int G, size_t U, int H)
{
    if (order == 1) return (size_t)r * U + u;
    if (order == 2) return ((u / H) * G + r) * H + u % H;
    return u * G + r;
}

// ---- host side: tensor maps ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [U][rows][128] bf16 tensor, tiles of [box_rows][64] with the 128-byte swizzle; rows beyond `rows`
// read as zero and are dropped on stores.
inline bool make_map(CUtensorMap *m, const void *base, uint64_t U, uint64_t rows, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {128, rows, U};
    cuuint64_t strides[2] = {256, rows * 256};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same tensor as whole-width tiles of [box_rows][128] without swizzle (rows of 256 bytes, in order).
inline bool make_map_plain(CUtensorMap *m, const void *base, uint64_t U, uint64_t rows, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {128, rows, U};
    cuuint64_t strides[2] = {256, rows * 256};
    cuuint32_t box[3] = {128, box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc
}  // namespace hgrn2
