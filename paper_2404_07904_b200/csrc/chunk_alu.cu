// Chunkwise forward and backward of the HGRN2 recurrence on fp32 CUDA cores.
//
// This is the path for float32 I/O (a single-pass bf16/tf32 tensor-core product cannot hold
// a 1e-4 error bound) and for every shape the tensor-core kernels do not cover.  One CTA per
// (batch, head) unit walks the chunks in order (forward) or in reverse (backward) with the
// running state S (forward) or state gradient dS (backward) resident in shared memory.
//
// Chunk-local form, derived from Eq. 3 by unrolling C steps.  Per chunk, q = o, k = 1 - f,
// v = i, b_j = sum_{r<=j} log f_r (inclusive, per key dimension), Lam_j = exp(b_j):
//
//   A[t,s]  = sum_k q_tk k_sk exp(b_tk - b_sk)            (s <= t; every exponent is <= 0)
//   Y       = A V + (q * Lam) S_in
//   S_out   = Diag(Lam_C) S_in + (k * Lam_C/Lam)^T V
//   dA      = tril(dY V^T)
//   dq_tk   = sum_{s<=t} dA[t,s] k_sk exp(b_tk-b_sk) + Lam_tk (dY S_in^T)_tk
//   dk_sk   = sum_{t>=s} dA[t,s] q_tk exp(b_tk-b_sk)  [intra]  + (Lam_C/Lam_s)_k (V dS_out^T)_sk  [inter]
//   dV      = A^T dY + (k * Lam_C/Lam) dS_out
//   dS_in   = Diag(Lam_C) dS_out + (q * Lam)^T dY
//   dg_jk   = sum_{j'>=j} (q dq - k dk_intra)_{j'k} + sum_{s<j} (k dk_inter)_{sk}
//             + Lam_Ck sum_v dS_out[k,v] S_in[k,v]                   (gradient w.r.t. log f_j)
//   d_o = dq,  d_i = dV,  d_f = dg / f - dk        (decay path and the tied gate k = 1 - f)
//
// Decay factors are always formed pairwise as exp(b_t - b_s) with t >= s, so nothing can
// overflow whatever f is.  A ragged last chunk is padded with neutral tokens (f = 1, o = i =
// dy = 0), which leave S and dS untouched.
#include "common.cuh"

namespace hgrn2 {

namespace {

constexpr int kAluThreads = 256;

__host__ __device__ inline size_t alu_fwd_smem_floats(int dk, int dv, int C)
{
    const size_t ldk = dk + 1, ldv = dv + 1;
    return 3 * (size_t)C * ldk + (size_t)C * ldv + (size_t)C * (C + 1) + (size_t)dk * dv;
}
__host__ __device__ inline size_t alu_bwd_smem_floats(int dk, int dv, int C)
{
    const size_t ldk = dk + 1, ldv = dv + 1;
    return 6 * (size_t)C * ldk + 2 * (size_t)C * ldv + 2 * (size_t)C * (C + 1) + (size_t)dk * ldv;
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_fwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const float *__restrict__ S0, T *__restrict__ y, float *__restrict__ SN,
               float *__restrict__ states, int N, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const int ldk = dk + 1, ldv = dv + 1, ldA = C + 1;
    float *q = smem;                 // [C][ldk]   o, later o * Lam
    float *k = q + C * ldk;          // [C][ldk]   1 - f, later (1 - f) * Lam_C / Lam
    float *b = k + C * ldk;          // [C][ldk]   log f, then its inclusive running sum
    float *v = b + C * ldk;          // [C][ldv]
    float *A = v + C * ldv;          // [C][ldA]
    float *S = A + C * ldA;          // [dk][dv]

    const int tid = threadIdx.x, nt = blockDim.x;
    const long long u = blockIdx.x;
    const T *ou = o + u * (long long)N * dk, *fu = f + u * (long long)N * dk;
    const T *iu = i + u * (long long)N * dv;
    const int ss = dk * dv;

    for (int x = tid; x < ss; x += nt) S[x] = S0 ? S0[u * ss + x] : 0.f;
    __syncthreads();

    for (int c = 0; c < NC; ++c) {
        const int t0 = c * C;
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk, tok = t0 + t;
            float qv = 0.f, fv = 1.f;
            if (tok < N) {
                qv = load_f(ou + (long long)tok * dk + kx);
                fv = load_f(fu + (long long)tok * dk + kx);
            }
            q[t * ldk + kx] = qv;
            k[t * ldk + kx] = 1.0f - fv;
            b[t * ldk + kx] = logf(fmaxf(fv, kFMin));
        }
        for (int x = tid; x < C * dv; x += nt) {
            const int t = x / dv, vx = x - t * dv, tok = t0 + t;
            v[t * ldv + vx] = tok < N ? load_f(iu + (long long)tok * dv + vx) : 0.f;
        }
        if (states) {
            float *dst = states + (u * NC + c) * (long long)ss;
            for (int x = tid; x < ss; x += nt) dst[x] = S[x];
        }
        __syncthreads();
        for (int kx = tid; kx < dk; kx += nt) {
            float run = 0.f;
            for (int t = 0; t < C; ++t) {
                run += b[t * ldk + kx];
                b[t * ldk + kx] = run;
            }
        }
        __syncthreads();
        if (y) {
            for (int x = tid; x < C * C; x += nt) {
                const int t = x / C, s = x - t * C;
                float acc = 0.f;
                if (s <= t) {
                    const float *qt = q + t * ldk, *ks = k + s * ldk, *bt = b + t * ldk, *bs = b + s * ldk;
                    for (int kx = 0; kx < dk; ++kx)
                        acc = fmaf(qt[kx] * ks[kx], expf(bt[kx] - bs[kx]), acc);
                }
                A[t * ldA + s] = acc;
            }
            __syncthreads();
        }
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk;
            const float bv = b[t * ldk + kx], bC = b[(C - 1) * ldk + kx];
            q[t * ldk + kx] *= expf(bv);
            k[t * ldk + kx] *= expf(bC - bv);
        }
        __syncthreads();
        if (y) {
            T *yu = y + u * (long long)N * dv;
            for (int x = tid; x < C * dv; x += nt) {
                const int t = x / dv, vx = x - t * dv, tok = t0 + t;
                if (tok >= N) continue;
                float acc = 0.f;
                const float *At = A + t * ldA, *qt = q + t * ldk;
                for (int s = 0; s <= t; ++s) acc = fmaf(At[s], v[s * ldv + vx], acc);
                for (int kx = 0; kx < dk; ++kx) acc = fmaf(qt[kx], S[kx * dv + vx], acc);
                store_f(yu + (long long)tok * dv + vx, acc);
            }
            __syncthreads();
        }
        for (int x = tid; x < ss; x += nt) {
            const int kx = x / dv, vx = x - kx * dv;
            float acc = expf(b[(C - 1) * ldk + kx]) * S[x];
            for (int s = 0; s < C; ++s) acc = fmaf(k[s * ldk + kx], v[s * ldv + vx], acc);
            S[x] = acc;
        }
        __syncthreads();
    }
    if (SN)
        for (int x = tid; x < ss; x += nt) SN[u * ss + x] = S[x];
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_bwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const T *__restrict__ dy, const float *__restrict__ dSN,
               const float *__restrict__ states, T *__restrict__ d_o, T *__restrict__ d_f,
               T *__restrict__ d_i, float *__restrict__ dS0, int N, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const int ldk = dk + 1, ldv = dv + 1, ldA = C + 1;
    float *q   = smem;               // [C][ldk]  o, later o * Lam
    float *k   = q + C * ldk;        // [C][ldk]  1 - f, later (1 - f) * Lam_C / Lam
    float *b   = k + C * ldk;        // [C][ldk]  running sum of log f
    float *dq  = b + C * ldk;        // [C][ldk]  dq, later q dq - k dk_intra
    float *dkk = dq + C * ldk;       // [C][ldk]  dk (intra + inter)
    float *e   = dkk + C * ldk;      // [C][ldk]  k * dk_inter, later its exclusive prefix sum
    float *v   = e + C * ldk;        // [C][ldv]
    float *g   = v + C * ldv;        // [C][ldv]  dy
    float *A   = g + C * ldv;        // [C][ldA]
    float *dA  = A + C * ldA;        // [C][ldA]
    float *dS  = dA + C * ldA;       // [dk][ldv]

    const int tid = threadIdx.x, nt = blockDim.x;
    const long long u = blockIdx.x;
    const T *ou = o + u * (long long)N * dk, *fu = f + u * (long long)N * dk;
    const T *iu = i + u * (long long)N * dv, *gu = dy + u * (long long)N * dv;
    T *dou = d_o + u * (long long)N * dk, *dfu = d_f + u * (long long)N * dk;
    T *diu = d_i + u * (long long)N * dv;
    const int ss = dk * dv;

    for (int x = tid; x < ss; x += nt) {
        const int kx = x / dv, vx = x - kx * dv;
        dS[kx * ldv + vx] = dSN ? dSN[u * ss + x] : 0.f;
    }
    __syncthreads();

    for (int c = NC - 1; c >= 0; --c) {
        const int t0 = c * C;
        const float *Sin = states + (u * NC + c) * (long long)ss;
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk, tok = t0 + t;
            float qv = 0.f, fv = 1.f;
            if (tok < N) {
                qv = load_f(ou + (long long)tok * dk + kx);
                fv = load_f(fu + (long long)tok * dk + kx);
            }
            q[t * ldk + kx] = qv;
            k[t * ldk + kx] = 1.0f - fv;
            b[t * ldk + kx] = logf(fmaxf(fv, kFMin));
        }
        for (int x = tid; x < C * dv; x += nt) {
            const int t = x / dv, vx = x - t * dv, tok = t0 + t;
            float vv = 0.f, gv = 0.f;
            if (tok < N) {
                vv = load_f(iu + (long long)tok * dv + vx);
                gv = load_f(gu + (long long)tok * dv + vx);
            }
            v[t * ldv + vx] = vv;
            g[t * ldv + vx] = gv;
        }
        __syncthreads();
        for (int kx = tid; kx < dk; kx += nt) {
            float run = 0.f;
            for (int t = 0; t < C; ++t) {
                run += b[t * ldk + kx];
                b[t * ldk + kx] = run;
            }
        }
        __syncthreads();
        // A and dA (lower triangles, diagonal kept)
        for (int x = tid; x < C * C; x += nt) {
            const int t = x / C, s = x - t * C;
            float acc = 0.f, dacc = 0.f;
            if (s <= t) {
                const float *qt = q + t * ldk, *ks = k + s * ldk, *bt = b + t * ldk, *bs = b + s * ldk;
                for (int kx = 0; kx < dk; ++kx)
                    acc = fmaf(qt[kx] * ks[kx], expf(bt[kx] - bs[kx]), acc);
                const float *gt = g + t * ldv, *vs = v + s * ldv;
                for (int vx = 0; vx < dv; ++vx) dacc = fmaf(gt[vx], vs[vx], dacc);
            }
            A[t * ldA + s] = acc;
            dA[t * ldA + s] = dacc;
        }
        __syncthreads();
        // dq, dk, e
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk;
            const float bt = b[t * ldk + kx], bC = b[(C - 1) * ldk + kx];
            float accq = 0.f;
            for (int s = 0; s <= t; ++s)
                accq = fmaf(dA[t * ldA + s] * k[s * ldk + kx], expf(bt - b[s * ldk + kx]), accq);
            float acck = 0.f;
            for (int r = t; r < C; ++r)
                acck = fmaf(dA[r * ldA + t] * q[r * ldk + kx], expf(b[r * ldk + kx] - bt), acck);
            float iq = 0.f, ik = 0.f;
            const float *Srow = Sin + (long long)kx * dv, *dSrow = dS + kx * ldv;
            const float *gt = g + t * ldv, *vt = v + t * ldv;
            for (int vx = 0; vx < dv; ++vx) {
                iq = fmaf(gt[vx], __ldg(Srow + vx), iq);
                ik = fmaf(vt[vx], dSrow[vx], ik);
            }
            ik *= expf(bC - bt);
            dq[t * ldk + kx]  = accq + expf(bt) * iq;
            dkk[t * ldk + kx] = acck + ik;
            e[t * ldk + kx]   = k[t * ldk + kx] * ik;
        }
        __syncthreads();
        // d_o out; dq <- q dq - k dk_intra; q <- q Lam; k <- k Lam_C / Lam
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk, tok = t0 + t;
            const int p = t * ldk + kx;
            const float qv = q[p], kv = k[p], bv = b[p], bC = b[(C - 1) * ldk + kx];
            const float dqv = dq[p];
            if (tok < N) store_f(dou + (long long)tok * dk + kx, dqv);
            dq[p] = qv * dqv - kv * dkk[p] + e[p];
            q[p] = qv * expf(bv);
            k[p] = kv * expf(bC - bv);
        }
        __syncthreads();
        // d_i
        for (int x = tid; x < C * dv; x += nt) {
            const int s = x / dv, vx = x - s * dv, tok = t0 + s;
            if (tok >= N) continue;
            float acc = 0.f;
            for (int t = s; t < C; ++t) acc = fmaf(A[t * ldA + s], g[t * ldv + vx], acc);
            const float *ks = k + s * ldk;
            for (int kx = 0; kx < dk; ++kx) acc = fmaf(ks[kx], dS[kx * ldv + vx], acc);
            store_f(diu + (long long)tok * dv + vx, acc);
        }
        // d_f: one thread per key dimension scans the chunk
        for (int kx = tid; kx < dk; kx += nt) {
            float R = 0.f;
            const float *Srow = Sin + (long long)kx * dv, *dSrow = dS + kx * ldv;
            for (int vx = 0; vx < dv; ++vx) R = fmaf(dSrow[vx], __ldg(Srow + vx), R);
            const float base = expf(b[(C - 1) * ldk + kx]) * R;
            float pre = 0.f;
            for (int t = 0; t < C; ++t) {
                const float ev = e[t * ldk + kx];
                e[t * ldk + kx] = pre;
                pre += ev;
            }
            float suf = 0.f;
            for (int t = C - 1; t >= 0; --t) {
                suf += dq[t * ldk + kx];
                const int tok = t0 + t;
                if (tok < N) {
                    const float fv = load_f(fu + (long long)tok * dk + kx);
                    const float dg = base + e[t * ldk + kx] + suf;
                    store_f(dfu + (long long)tok * dk + kx, dg / fmaxf(fv, kFMin) - dkk[t * ldk + kx]);
                }
            }
        }
        __syncthreads();
        // dS_in = Lam_C dS_out + (q Lam)^T dY
        for (int x = tid; x < ss; x += nt) {
            const int kx = x / dv, vx = x - kx * dv;
            float acc = expf(b[(C - 1) * ldk + kx]) * dS[kx * ldv + vx];
            for (int t = 0; t < C; ++t) acc = fmaf(q[t * ldk + kx], g[t * ldv + vx], acc);
            dS[kx * ldv + vx] = acc;
        }
        __syncthreads();
    }
    if (dS0)
        for (int x = tid; x < ss; x += nt) {
            const int kx = x / dv, vx = x - kx * dv;
            dS0[u * ss + x] = dS[kx * ldv + vx];
        }
}

constexpr size_t kMaxSmem = 227 * 1024;

template <typename T>
cudaError_t launch_fwd_t(const SeqArgs &a)
{
    const size_t smem = alu_fwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = cudaFuncSetAttribute(alu_fwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    alu_fwd_kernel<T><<<a.B * a.H, kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), a.S0,
        static_cast<T *>(a.y), a.SN, a.states, a.N, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bwd_t(const SeqArgs &a)
{
    const size_t smem = alu_bwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = cudaFuncSetAttribute(alu_bwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    alu_bwd_kernel<T><<<a.B * a.H, kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i),
        static_cast<const T *>(a.dy), a.dSN, a.states, static_cast<T *>(a.d_o), static_cast<T *>(a.d_f),
        static_cast<T *>(a.d_i), a.dS0, a.N, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

}  // namespace

bool alu_chunk_supported(int dk, int dv, int C)
{
    if (C != 16 && C != 32 && C != 64) return false;
    return alu_bwd_smem_floats(dk, dv, C) * sizeof(float) <= kMaxSmem &&
           alu_fwd_smem_floats(dk, dv, C) * sizeof(float) <= kMaxSmem;
}

int alu_default_chunk(int dk, int dv)
{
    for (int C = 64; C >= 16; C /= 2)
        if (alu_chunk_supported(dk, dv, C)) return C;
    return 0;
}

cudaError_t launch_alu_fwd(const SeqArgs &a)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    return a.io == HGRN2_BF16 ? launch_fwd_t<__nv_bfloat16>(a) : launch_fwd_t<float>(a);
}

cudaError_t launch_alu_bwd(const SeqArgs &a)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    return a.io == HGRN2_BF16 ? launch_bwd_t<__nv_bfloat16>(a) : launch_bwd_t<float>(a);
}

}  // namespace hgrn2
