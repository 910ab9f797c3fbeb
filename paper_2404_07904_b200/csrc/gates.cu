// Gate activations in front of the recurrence (Eq. 1 and Eq. 2 of the paper):
//
//     o = sigmoid(zo),     f = beta + (1 - beta) * sigmoid(zf),     i = silu(zi)
//
// with zo, zf, zi the layer's pre-activations and beta the layer's per-channel lower bound of the forget gate.
//
// fp32 kernels: the activations are applied as the tiles are loaded and their derivatives as the gradients are
// stored (chunk_alu.cuh, kGatePre), all in fp32.
//
// Tensor-core kernels: they take bf16 operand tiles through TMA, and a bf16 f close to 1 would carry a relative
// error of 2^-9 / (1 - f) into every decay product (a bf16 k = 1 - f close to 1 would do the same to d_f and
// d_beta at hard-forget gates).  So one element-wise kernel in front writes o, i and the SMALLER of f and
// k = (1 - beta)(1 - sigmoid(zf)), negated when it is k - bf16 then resolves the gate to 2^-9 of min(f, k) - and
// the kernels decode it (tc_chunk.cuh, gate_decode; the other of the two is 1 minus it, exact in fp32); one
// element-wise kernel behind turns the gradients
// with respect to o, f, i into those with respect to zo, zf, zi, in place, and sums the gradient with respect to
// beta.  Both are single passes over their tensors with 16-byte accesses.
#include "chunk_alu.cuh"

namespace hgrn2 {

namespace {

constexpr int kGD = 128;                 // the tensor-core path: d_k = d_v = 128

__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
// sigmoid with the fast exponential and reciprocal (a few ulp: far inside what the bf16 results keep)
__device__ __forceinline__ float sigmoid_fast(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ uint32_t bf_pack(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// zo, zf, zi [U][N][128] bf16 -> o, signed gate encoding, i [U][N][128] bf16; one thread per 8 consecutive elements of a row.
__global__ void __launch_bounds__(256)
gate_fwd_kernel(const uint4 *__restrict__ zo, const uint4 *__restrict__ zf, const uint4 *__restrict__ zi,
                const float *__restrict__ beta, uint4 *__restrict__ o, uint4 *__restrict__ k, uint4 *__restrict__ i,
                long long nvec, int N, int H)
{
    for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < nvec; x += (long long)gridDim.x * blockDim.x) {
        const int c8 = (int)(x & 15) * 8;
        const int h = (int)((x >> 4) / N % H);
        const float *bh = beta + (size_t)h * kGD + c8;
        const uint4 a = zo[x], b = zf[x], c = zi[x];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w}, cw[4] = {c.x, c.y, c.z, c.w};
        uint32_t ow[4], kw[4], iw[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float z0 = bf_lo(cw[j]), z1 = bf_hi(cw[j]);
            ow[j] = bf_pack(sigmoid_fast(bf_lo(aw[j])), sigmoid_fast(bf_hi(aw[j])));
            const float k0 = (1.0f - bh[2 * j]) * (1.0f - sigmoid_fast(bf_lo(bw[j])));
            const float k1 = (1.0f - bh[2 * j + 1]) * (1.0f - sigmoid_fast(bf_hi(bw[j])));
            kw[j] = bf_pack(k0 <= 0.5f ? -k0 : 1.0f - k0, k1 <= 0.5f ? -k1 : 1.0f - k1);   // the smaller of f and k; negative = k
            iw[j] = bf_pack(z0 * sigmoid_fast(z0), z1 * sigmoid_fast(z1));
        }
        o[x] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
        k[x] = make_uint4(kw[0], kw[1], kw[2], kw[3]);
        i[x] = make_uint4(iw[0], iw[1], iw[2], iw[3]);
    }
}

// In place: d_o, d_f, d_i [U][N][128] bf16 -> d_zo, d_zf, d_zi, and this block's share of d_beta.
// Grid (U, P): block (u, p) owns the rows [p * rows_per, (p + 1) * rows_per) of unit u; thread = (row lane of 16,
// column group of 8).  partial [U * P][128].
__global__ void __launch_bounds__(256)
gate_bwd_kernel(const uint4 *__restrict__ zo, const uint4 *__restrict__ zf, const uint4 *__restrict__ zi,
                const float *__restrict__ beta, uint4 *__restrict__ g_o, uint4 *__restrict__ g_f, uint4 *__restrict__ g_i,
                float *__restrict__ partial, int N, int H, int rows_per)
{
    __shared__ float red[16][kGD + 4];
    const int u = blockIdx.x, p = blockIdx.y;
    const int cg = threadIdx.x & 15, rl = threadIdx.x >> 4;
    const int h = u % H;
    float bh[8], db[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { bh[j] = beta[(size_t)h * kGD + cg * 8 + j]; db[j] = 0.f; }
    const int r1 = min(N, (p + 1) * rows_per);
    // The gradients are rewritten in place, so the compiler must keep every load behind the previous row's
    // stores: the next row's six loads are therefore issued by hand before the current row is worked on.
    uint4 na, nb, nc, nda, ndb, ndc;
    int r = p * rows_per + rl;
    if (r < r1) {
        const size_t x = ((size_t)u * N + r) * 16 + cg;
        na = zo[x]; nb = zf[x]; nc = zi[x]; nda = g_o[x]; ndb = g_f[x]; ndc = g_i[x];
    }
    for (; r < r1; r += 16) {
        const size_t x = ((size_t)u * N + r) * 16 + cg;
        const uint4 a = na, b = nb, c = nc, da = nda, dbv = ndb, dc = ndc;
        if (r + 16 < r1) {
            const size_t xn = x + 16 * 16;
            na = zo[xn]; nb = zf[xn]; nc = zi[xn]; nda = g_o[xn]; ndb = g_f[xn]; ndc = g_i[xn];
        }
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w}, cw[4] = {c.x, c.y, c.z, c.w};
        const uint32_t dao[4] = {da.x, da.y, da.z, da.w}, dbf[4] = {dbv.x, dbv.y, dbv.z, dbv.w}, dci[4] = {dc.x, dc.y, dc.z, dc.w};
        uint32_t ro[4], rf[4], ri[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float res[6];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float zov = e ? bf_hi(aw[j]) : bf_lo(aw[j]), zfv = e ? bf_hi(bw[j]) : bf_lo(bw[j]);
                const float ziv = e ? bf_hi(cw[j]) : bf_lo(cw[j]);
                const float dov = e ? bf_hi(dao[j]) : bf_lo(dao[j]), dfv = e ? bf_hi(dbf[j]) : bf_lo(dbf[j]);
                const float div = e ? bf_hi(dci[j]) : bf_lo(dci[j]);
                const float so = sigmoid_fast(zov), g = sigmoid_fast(zfv), si = sigmoid_fast(ziv);
                res[e] = dov * so * (1.0f - so);
                res[2 + e] = dfv * (1.0f - bh[2 * j + e]) * g * (1.0f - g);
                res[4 + e] = div * si * (1.0f + ziv * (1.0f - si));
                db[2 * j + e] += dfv * (1.0f - g);
            }
            ro[j] = bf_pack(res[0], res[1]);
            rf[j] = bf_pack(res[2], res[3]);
            ri[j] = bf_pack(res[4], res[5]);
        }
        g_o[x] = make_uint4(ro[0], ro[1], ro[2], ro[3]);
        g_f[x] = make_uint4(rf[0], rf[1], rf[2], rf[3]);
        g_i[x] = make_uint4(ri[0], ri[1], ri[2], ri[3]);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) red[rl][cg * 8 + j] = db[j];
    __syncthreads();
    if (threadIdx.x < kGD) {
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < 16; ++q) s += red[q][threadIdx.x];      // fixed order: run-to-run identical
        partial[((size_t)u * gridDim.y + p) * kGD + threadIdx.x] = s;
    }
}

// d_beta[h][k] = sum over the batch and the row slices of partial[(b * H + h) * P + p][k], in a fixed order.
__global__ void gate_reduce_beta_kernel(const float *__restrict__ partial, float *__restrict__ d_beta, int B, int H, int P,
                                        int dk)
{
    const int h = blockIdx.x, k = threadIdx.x;
    if (k >= dk) return;
    float s = 0.f;
    for (int b = 0; b < B; ++b)
        for (int p = 0; p < P; ++p) s += partial[(((size_t)b * H + h) * P + p) * dk + k];
    d_beta[(size_t)h * dk + k] = s;
}

// ---- fp32 kernels with the activations applied in the load stage ---------------------------------------------
constexpr int kAluThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_fwd_gated_kernel(const T *__restrict__ zo, const T *__restrict__ zf, const T *__restrict__ zi,
                     const float *__restrict__ beta, const float *__restrict__ S0, T *__restrict__ y,
                     float *__restrict__ SN, float *__restrict__ states, int N, int H, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    alu::fwd_unit<T, float, alu::kGatePre>(smem, zo + u * N * dk, zf + u * N * dk, zi + u * N * dv,
                                           S0 ? S0 + u * ss : nullptr, y ? y + u * N * dv : nullptr,
                                           SN ? SN + u * ss : nullptr, states ? states + u * NC * ss : nullptr, 1, N, dk,
                                           dv, C, NC, beta + (u % H) * dk);
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_bwd_gated_kernel(const T *__restrict__ zo, const T *__restrict__ zf, const T *__restrict__ zi,
                     const float *__restrict__ beta, const T *__restrict__ dy, const float *__restrict__ dSN,
                     const float *__restrict__ states, T *__restrict__ d_zo, T *__restrict__ d_zf, T *__restrict__ d_zi,
                     float *__restrict__ dS0, float *__restrict__ partial, int N, int H, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    alu::bwd_unit<T, float, alu::kGatePre>(smem, zo + u * N * dk, zf + u * N * dk, zi + u * N * dv, dy + u * N * dv,
                                           dSN ? dSN + u * ss : nullptr, states + u * NC * ss, 1, nullptr,
                                           d_zo + u * N * dk, d_zf + u * N * dk, d_zi + u * N * dv,
                                           dS0 ? dS0 + u * ss : nullptr, N, dk, dv, C, NC, beta + (u % H) * dk,
                                           partial + u * dk);
}

template <typename T>
cudaError_t alu_gated_fwd_t(const SeqArgs &a, const float *beta)
{
    const size_t smem = alu::fwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(alu_fwd_gated_kernel<T>), smem);
    if (err != cudaSuccess) return err;
    alu_fwd_gated_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), beta, a.S0,
        static_cast<T *>(a.y), a.SN, a.states, a.N, a.H, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

template <typename T>
cudaError_t alu_gated_bwd_t(const SeqArgs &a, const float *beta, float *partial)
{
    const size_t smem = alu::bwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(alu_bwd_gated_kernel<T>), smem);
    if (err != cudaSuccess) return err;
    alu_bwd_gated_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), beta,
        static_cast<const T *>(a.dy), a.dSN, a.states, static_cast<T *>(a.d_o), static_cast<T *>(a.d_f),
        static_cast<T *>(a.d_i), a.dS0, partial, a.N, a.H, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

}  // namespace

// Row slices per unit of the element-wise backward: enough blocks to fill the GPU several times over.
int gate_bwd_slices(long long U, int N)
{
    long long P = (8 * 592 + U - 1) / (U > 0 ? U : 1);
    const long long most = (N + 63) / 64;
    if (P > most) P = most;
    return (int)(P < 1 ? 1 : P);
}

// a.o, a.f, a.i hold the pre-activations; o_out, k_out, i_out receive o, the signed gate encoding, i (bf16, d = 128).
cudaError_t launch_gate_fwd(const SeqArgs &a, const float *beta, void *o_out, void *k_out, void *i_out)
{
    const long long nvec = (long long)a.B * a.H * a.N * (kGD / 8);
    if (nvec == 0) return cudaSuccess;
    const long long want = (nvec + 255) / 256;
    const unsigned grid = (unsigned)(want < 148 * 16 ? want : 148 * 16);
    gate_fwd_kernel<<<grid, 256, 0, a.stream>>>(static_cast<const uint4 *>(a.o), static_cast<const uint4 *>(a.f),
                                                static_cast<const uint4 *>(a.i), beta, static_cast<uint4 *>(o_out),
                                                static_cast<uint4 *>(k_out), static_cast<uint4 *>(i_out), nvec, a.N, a.H);
    return cudaGetLastError();
}

// a.o, a.f, a.i hold the pre-activations; a.d_o, a.d_f, a.d_i hold d_o, d_f, d_i and receive d_zo, d_zf, d_zi.
cudaError_t launch_gate_bwd(const SeqArgs &a, const float *beta, float *partial, float *d_beta)
{
    const long long U = (long long)a.B * a.H;
    if (U == 0 || a.N == 0) return cudaSuccess;
    const int P = gate_bwd_slices(U, a.N);
    const int rows_per = (a.N + P - 1) / P;
    gate_bwd_kernel<<<dim3((unsigned)U, (unsigned)P), 256, 0, a.stream>>>(
        static_cast<const uint4 *>(a.o), static_cast<const uint4 *>(a.f), static_cast<const uint4 *>(a.i), beta,
        static_cast<uint4 *>(a.d_o), static_cast<uint4 *>(a.d_f), static_cast<uint4 *>(a.d_i), partial, a.N, a.H, rows_per);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess || d_beta == nullptr) return err;
    gate_reduce_beta_kernel<<<a.H, 128, 0, a.stream>>>(partial, d_beta, a.B, a.H, P, kGD);
    return cudaGetLastError();
}

cudaError_t launch_alu_fwd_gated(const SeqArgs &a, const float *beta)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    if ((long long)a.B * a.H > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    return a.io == HGRN2_BF16 ? alu_gated_fwd_t<__nv_bfloat16>(a, beta) : alu_gated_fwd_t<float>(a, beta);
}

cudaError_t launch_alu_bwd_gated(const SeqArgs &a, const float *beta, float *partial, float *d_beta)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    if ((long long)a.B * a.H > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    cudaError_t err = a.io == HGRN2_BF16 ? alu_gated_bwd_t<__nv_bfloat16>(a, beta, partial)
                                         : alu_gated_bwd_t<float>(a, beta, partial);
    if (err != cudaSuccess || d_beta == nullptr) return err;
    gate_reduce_beta_kernel<<<a.H, 128, 0, a.stream>>>(partial, d_beta, a.B, a.H, 1, a.dk);
    return cudaGetLastError();
}

}  // namespace hgrn2
