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
//
// The per-unit bodies live in this header as device functions: the kernels of chunk_alu.cu call them for
// every unit, and the tensor-core kernels call them for the units whose decay leaves the range their
// rescaled operands can represent (the "exact path": there the chunk-start states are kept as bf16 for every
// second chunk, in the slots of the tensor-core path's saved data, and the others are re-created on the fly).
#pragma once

#include "common.cuh"

namespace hgrn2 {
namespace alu {

// What the three input tensors hold.  kGateIsF: o, f, i themselves.  kGateEnc: o, the signed gate encoding
// (the smaller of f and k = 1 - f, negative when it is k; what the tensor-core path of the gated entry points is
// handed), i.  kGatePre: the pre-activations zo, zf, zi of Eq. 1 / Eq. 2, turned into
// o = sigmoid(zo), f = beta + (1 - beta) sigmoid(zf), i = silu(zi) as they are loaded (fp32, so f is never rounded to
// the I/O type), and the backward returns the gradients with respect to the pre-activations and to beta.
enum GateMode { kGateIsF = 0, kGateEnc = 1, kGatePre = 2 };

__device__ __forceinline__ float sigmoid_f(float x) { return 1.0f / (1.0f + expf(-x)); }

// Gate values of one (token, key dimension) from what the tensors hold: q, f and k = 1 - f.
template <int kMode>
__device__ __forceinline__ void gate_values(float qraw, float fraw, float beta, float &qv, float &fv, float &kv)
{
    if (kMode == kGateIsF) { qv = qraw; fv = fraw; kv = 1.0f - fraw; }
    else if (kMode == kGateEnc) {
        qv = qraw;
        const float m = fabsf(fraw);
        if (signbit(fraw)) { kv = m; fv = 1.0f - m; } else { fv = m; kv = 1.0f - m; }
    }
    else {
        const float g = sigmoid_f(fraw);
        qv = sigmoid_f(qraw);
        kv = (1.0f - beta) * (1.0f - g);
        fv = 1.0f - kv;
    }
}
template <int kMode> __device__ __forceinline__ float value_of(float vraw)
{
    return kMode == kGatePre ? vraw * sigmoid_f(vraw) : vraw;
}

__host__ __device__ constexpr size_t fwd_smem_floats(int dk, int dv, int C)
{
    const size_t ldk = dk + 1, ldv = dv + 1;
    return 3 * (size_t)C * ldk + (size_t)C * ldv + (size_t)C * (C + 1) + (size_t)dk * dv;
}
__host__ __device__ constexpr size_t bwd_smem_floats(int dk, int dv, int C)
{
    const size_t ldk = dk + 1, ldv = dv + 1;
    return 6 * (size_t)C * ldk + 2 * (size_t)C * ldv + 2 * (size_t)C * (C + 1) + (size_t)dk * ldv;
}

// Forward of one unit, run by every thread of the CTA.  All pointers are the unit's own (token 0, element 0).
// ST = element type of the kept chunk-start states; the state of chunk c goes to slot c / every when
// c % every == 0 (every = 1: all chunks).  yu, SNu, states_u may be null.
// beta_h: this head's lower bounds [dk] (kGatePre only).
template <typename T, typename ST, int kMode = kGateIsF>
__device__ void fwd_unit(float *smem, const T *__restrict__ ou, const T *__restrict__ fu, const T *__restrict__ iu,
                         const float *__restrict__ S0u, T *__restrict__ yu, float *__restrict__ SNu,
                         ST *__restrict__ states_u, int every, int N, int dk, int dv, int C, int NC,
                         const float *__restrict__ beta_h = nullptr)
{
    const int ldk = dk + 1, ldv = dv + 1, ldA = C + 1;
    float *q = smem;                 // [C][ldk]   o, later o * Lam
    float *k = q + C * ldk;          // [C][ldk]   1 - f, later (1 - f) * Lam_C / Lam
    float *b = k + C * ldk;          // [C][ldk]   log f, then its inclusive running sum
    float *v = b + C * ldk;          // [C][ldv]
    float *A = v + C * ldv;          // [C][ldA]
    float *S = A + C * ldA;          // [dk][dv]

    const int tid = threadIdx.x, nt = blockDim.x;
    const int ss = dk * dv;

    for (int x = tid; x < ss; x += nt) S[x] = S0u ? S0u[x] : 0.f;
    __syncthreads();

    for (int c = 0; c < NC; ++c) {
        const int t0 = c * C;
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk, tok = t0 + t;
            float qv = 0.f, fv = 1.f, kv = 0.f;
            if (tok < N)
                gate_values<kMode>(load_f(ou + (long long)tok * dk + kx), load_f(fu + (long long)tok * dk + kx),
                                   kMode == kGatePre ? beta_h[kx] : 0.f, qv, fv, kv);
            q[t * ldk + kx] = qv;
            k[t * ldk + kx] = kv;
            b[t * ldk + kx] = logf(fmaxf(fv, kFMin));
        }
        for (int x = tid; x < C * dv; x += nt) {
            const int t = x / dv, vx = x - t * dv, tok = t0 + t;
            v[t * ldv + vx] = tok < N ? value_of<kMode>(load_f(iu + (long long)tok * dv + vx)) : 0.f;
        }
        if (states_u && c % every == 0) {
            ST *dst = states_u + (long long)(c / every) * ss;
            for (int x = tid; x < ss; x += nt) store_f(dst + x, S[x]);
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
        if (yu) {
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
        if (yu) {
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
    if (SNu)
        for (int x = tid; x < ss; x += nt) SNu[x] = S[x];
}

// Backward of one unit.  states_u holds the chunk-start state of chunk c in slot c / every for c % every == 0;
// with every = 2 the state of an odd chunk is re-created from the slot of the chunk before it and that chunk's
// tokens into `scratch` ([dk][dv] floats in global memory, this unit's own).  dSNu, dS0u may be null.
// kGatePre: beta_h = this head's lower bounds [dk]; dou, dfu, diu receive the gradients with respect to zo, zf, zi
// and dbeta_u[dk] (nullable) this unit's share of the gradient with respect to beta.
template <typename T, typename ST, int kMode = kGateIsF>
__device__ void bwd_unit(float *smem, const T *__restrict__ ou, const T *__restrict__ fu, const T *__restrict__ iu,
                         const T *__restrict__ gu, const float *__restrict__ dSNu, const ST *states_u, int every,
                         float *scratch, T *__restrict__ dou, T *__restrict__ dfu, T *__restrict__ diu,
                         float *__restrict__ dS0u, int N, int dk, int dv, int C, int NC,
                         const float *__restrict__ beta_h = nullptr, float *__restrict__ dbeta_u = nullptr)
{
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
    const int ss = dk * dv;

    for (int x = tid; x < ss; x += nt) {
        const int kx = x / dv, vx = x - kx * dv;
        dS[kx * ldv + vx] = dSNu ? dSNu[x] : 0.f;
    }
    __syncthreads();

    float dbeta_acc = 0.f;           // kGatePre: a thread owns one key dimension in the d_f scan (dk <= blockDim.x)
    for (int c = NC - 1; c >= 0; --c) {
        const int t0 = c * C;
        const ST *slot = states_u + (long long)(c / every) * ss;
        const bool recreate = c % every != 0;
        if (recreate) {
            // S at the start of chunk c = Diag(Lam_C) S_slot + (k * Lam_C / Lam)^T V over the (whole) chunk c - 1
            const int p0 = (c - 1) * C;
            for (int x = tid; x < C * dk; x += nt) {
                const int t = x / dk, kx = x - t * dk;
                float qv, fv, kv;
                gate_values<kMode>(0.f, load_f(fu + (long long)(p0 + t) * dk + kx), kMode == kGatePre ? beta_h[kx] : 0.f,
                                   qv, fv, kv);
                k[t * ldk + kx] = kv;
                b[t * ldk + kx] = logf(fmaxf(fv, kFMin));
            }
            for (int x = tid; x < C * dv; x += nt) {
                const int t = x / dv, vx = x - t * dv;
                v[t * ldv + vx] = value_of<kMode>(load_f(iu + (long long)(p0 + t) * dv + vx));
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
            for (int x = tid; x < C * dk; x += nt) {
                const int t = x / dk, kx = x - t * dk;
                k[t * ldk + kx] *= expf(b[(C - 1) * ldk + kx] - b[t * ldk + kx]);
            }
            __syncthreads();
            for (int x = tid; x < ss; x += nt) {
                const int kx = x / dv, vx = x - kx * dv;
                float acc = expf(b[(C - 1) * ldk + kx]) * load_f(slot + x);
                for (int s = 0; s < C; ++s) acc = fmaf(k[s * ldk + kx], v[s * ldv + vx], acc);
                scratch[x] = acc;
            }
            __syncthreads();
        }
        auto S_in = [&](int idx) -> float { return recreate ? scratch[idx] : load_f(slot + idx); };
        for (int x = tid; x < C * dk; x += nt) {
            const int t = x / dk, kx = x - t * dk, tok = t0 + t;
            float qv = 0.f, fv = 1.f, kv = 0.f;
            if (tok < N)
                gate_values<kMode>(load_f(ou + (long long)tok * dk + kx), load_f(fu + (long long)tok * dk + kx),
                                   kMode == kGatePre ? beta_h[kx] : 0.f, qv, fv, kv);
            q[t * ldk + kx] = qv;
            k[t * ldk + kx] = kv;
            b[t * ldk + kx] = logf(fmaxf(fv, kFMin));
        }
        for (int x = tid; x < C * dv; x += nt) {
            const int t = x / dv, vx = x - t * dv, tok = t0 + t;
            float vv = 0.f, gv = 0.f;
            if (tok < N) {
                vv = value_of<kMode>(load_f(iu + (long long)tok * dv + vx));
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
            const float *dSrow = dS + kx * ldv;
            const float *gt = g + t * ldv, *vt = v + t * ldv;
            for (int vx = 0; vx < dv; ++vx) {
                iq = fmaf(gt[vx], S_in(kx * dv + vx), iq);
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
            if (tok < N) store_f(dou + (long long)tok * dk + kx, kMode == kGatePre ? dqv * qv * (1.0f - qv) : dqv);
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
            if (kMode == kGatePre) {                  // d silu(z) / dz = s (1 + z (1 - s)), s = sigmoid(z)
                const float z = load_f(iu + (long long)tok * dv + vx), sg = sigmoid_f(z);
                acc *= sg * (1.0f + z * (1.0f - sg));
            }
            store_f(diu + (long long)tok * dv + vx, acc);
        }
        // d_f: one thread per key dimension scans the chunk
        for (int kx = tid; kx < dk; kx += nt) {
            float R = 0.f;
            const float *dSrow = dS + kx * ldv;
            for (int vx = 0; vx < dv; ++vx) R = fmaf(dSrow[vx], S_in(kx * dv + vx), R);
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
                    const float fraw = load_f(fu + (long long)tok * dk + kx);
                    float qv, fv, kv;
                    gate_values<kMode>(0.f, fraw, kMode == kGatePre ? beta_h[kx] : 0.f, qv, fv, kv);
                    const float dg = base + e[t * ldk + kx] + suf;
                    float dfv = dg / fmaxf(fv, kMode == kGateEnc ? kFDivMinK : kFMin) - dkk[t * ldk + kx];
                    if (kMode == kGatePre) {          // f = beta + (1 - beta) g:  df/dzf = (1 - beta) g (1 - g),  df/dbeta = 1 - g
                        const float g = sigmoid_f(fraw);
                        dbeta_acc += dfv * (1.0f - g);
                        dfv *= (1.0f - beta_h[kx]) * g * (1.0f - g);
                    }
                    store_f(dfu + (long long)tok * dk + kx, dfv);
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
    if (dS0u)
        for (int x = tid; x < ss; x += nt) {
            const int kx = x / dv, vx = x - kx * dv;
            dS0u[x] = dS[kx * ldv + vx];
        }
    if (kMode == kGatePre && dbeta_u != nullptr && tid < dk) dbeta_u[tid] = dbeta_acc;
}

}  // namespace alu
}  // namespace hgrn2
