// Single-token decode step (Eq. 3 applied once), bandwidth-bound.
//
// One CTA of 256 threads per (batch, head) unit streams that unit's dk x dv float32 state
// through registers exactly once:  S[k][v] <- f[k] S[k][v] + (1 - f[k]) i[v],  and reduces
// y[v] = sum_k o[k] S_new[k][v] on the way.  A thread owns one float4 column group and the
// rows k = rg, rg + RG, ...; all of a batch's 16-byte loads are issued before the first
// dependent instruction so that many are in flight per thread.  No atomics: the cross-row
// reduction goes through shared memory in a fixed order, so results are run-to-run identical.
#include "common.cuh"

namespace hgrn2 {

namespace {

constexpr int kStepThreads = 256;
constexpr int kBatch = 8;   // rows a thread loads before it starts computing

template <typename T, int DV>
__global__ void __launch_bounds__(kStepThreads)
step_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
            float *__restrict__ S, T *__restrict__ y, int dk, long long units)
{
    constexpr int C4 = DV / 4;                 // float4 column groups per row
    constexpr int RG = kStepThreads / C4;      // rows covered per pass
    __shared__ float s_o[128], s_f[128], s_i[DV];
    __shared__ float4 s_red[RG][C4];

    const int tid = threadIdx.x;
    const int c4 = tid % C4;
    const int rg = tid / C4;

    for (long long u = blockIdx.x; u < units; u += gridDim.x) {
        if (tid < dk) {
            s_o[tid] = load_f(o + u * dk + tid);
            s_f[tid] = load_f(f + u * dk + tid);
        }
        if (tid < DV) s_i[tid] = load_f(i + u * DV + tid);
        __syncthreads();

        const float4 iv = make_float4(s_i[c4 * 4 + 0], s_i[c4 * 4 + 1], s_i[c4 * 4 + 2], s_i[c4 * 4 + 3]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 *Su = reinterpret_cast<float4 *>(S + u * (long long)dk * DV) + c4;

        for (int k0 = rg; k0 < dk; k0 += RG * kBatch) {
            float4 s[kBatch];
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int k = k0 + j * RG;
                if (k < dk) s[j] = __ldcs(Su + (long long)k * C4);
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                const int k = k0 + j * RG;
                if (k < dk) {
                    const float fk = s_f[k], kk = 1.0f - fk, ok = s_o[k];
                    s[j].x = fmaf(fk, s[j].x, kk * iv.x);
                    s[j].y = fmaf(fk, s[j].y, kk * iv.y);
                    s[j].z = fmaf(fk, s[j].z, kk * iv.z);
                    s[j].w = fmaf(fk, s[j].w, kk * iv.w);
                    __stcs(Su + (long long)k * C4, s[j]);
                    acc.x = fmaf(ok, s[j].x, acc.x);
                    acc.y = fmaf(ok, s[j].y, acc.y);
                    acc.z = fmaf(ok, s[j].z, acc.z);
                    acc.w = fmaf(ok, s[j].w, acc.w);
                }
            }
        }
        s_red[rg][c4] = acc;
        __syncthreads();
        if (tid < DV) {
            const float *red = reinterpret_cast<const float *>(&s_red[0][0]);
            float t = 0.f;
#pragma unroll 4
            for (int r = 0; r < RG; ++r) t += red[r * DV + tid];
            store_f(y + u * DV + tid, t);
        }
        __syncthreads();
    }
}

// Packed fp32 arithmetic (sm_100): one instruction per two results, each rounded exactly like the scalar op,
// so the results below stay bit-identical to step_kernel's.
__device__ __forceinline__ float2 mul_x2(float2 a, float2 b)
{
    float2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(reinterpret_cast<unsigned long long &>(d))
        : "l"(reinterpret_cast<unsigned long long &>(a)), "l"(reinterpret_cast<unsigned long long &>(b)));
    return d;
}
__device__ __forceinline__ float2 fma_x2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(reinterpret_cast<unsigned long long &>(d))
        : "l"(reinterpret_cast<unsigned long long &>(a)), "l"(reinterpret_cast<unsigned long long &>(b)),
          "l"(reinterpret_cast<unsigned long long &>(c)));
    return d;
}

// Several successive tokens in one launch (multi-token / speculative decode): the unit's state is read once,
// kept in registers while Eq. 3 is applied Tn times, and written once, so the state traffic per token falls
// Tn-fold.  d_k = d_v = D.  Thread layout, arithmetic and summation order are those of step_kernel, so the
// results are bit-identical to Tn single steps.  Sequence tensors are [unit][token][D].
template <typename T, int D>
__global__ void __launch_bounds__(kStepThreads)
step_multi_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
                  float *__restrict__ S, T *__restrict__ y, int Tn, long long units)
{
    constexpr int C4 = D / 4;                  // float4 column groups per row
    constexpr int RG = kStepThreads / C4;      // rows covered per pass
    constexpr int R = D / RG;                  // rows (float4 registers) per thread
    constexpr int TB = 8;                      // tokens whose gates are staged together (one global round trip)
    __shared__ float s_o[TB * D], s_f[TB * D], s_i[TB * D];
    __shared__ float4 s_red[2][RG][C4];

    const int tid = threadIdx.x;
    const int c4 = tid % C4;
    const int rg = tid / C4;

    for (long long u = blockIdx.x; u < units; u += gridDim.x) {
        float4 *Su = reinterpret_cast<float4 *>(S + u * (long long)D * D) + c4;
        float4 s[R];
#pragma unroll
        for (int j = 0; j < R; ++j) s[j] = __ldcs(Su + (long long)(rg + j * RG) * C4);

        for (int t0 = 0; t0 < Tn; t0 += TB) {
            const int nb = min(TB, Tn - t0);
            const long long row0 = (u * Tn + t0) * D;
            for (int idx = tid; idx < nb * D; idx += kStepThreads) {
                s_o[idx] = load_f(o + row0 + idx);
                s_f[idx] = load_f(f + row0 + idx);
                s_i[idx] = load_f(i + row0 + idx);
            }
            __syncthreads();
            for (int tt = 0; tt < nb; ++tt) {
                const float *so = s_o + tt * D, *sf = s_f + tt * D, *si = s_i + tt * D;
                const float2 iv0 = make_float2(si[c4 * 4 + 0], si[c4 * 4 + 1]), iv1 = make_float2(si[c4 * 4 + 2], si[c4 * 4 + 3]);
                float2 a0 = make_float2(0.f, 0.f), a1 = make_float2(0.f, 0.f);
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    const int k = rg + j * RG;
                    const float fk = sf[k], kk = 1.0f - fk, ok = so[k];
                    const float2 f2 = make_float2(fk, fk), k2 = make_float2(kk, kk), o2 = make_float2(ok, ok);
                    float2 lo = make_float2(s[j].x, s[j].y), hi = make_float2(s[j].z, s[j].w);
                    lo = fma_x2(f2, lo, mul_x2(k2, iv0));
                    hi = fma_x2(f2, hi, mul_x2(k2, iv1));
                    a0 = fma_x2(o2, lo, a0);
                    a1 = fma_x2(o2, hi, a1);
                    s[j] = make_float4(lo.x, lo.y, hi.x, hi.y);
                }
                const float4 acc = make_float4(a0.x, a0.y, a1.x, a1.y);
                // partial sums alternate between two buffers, so one barrier per token is enough: a buffer is
                // rewritten two tokens later, after a barrier that its readers reach only when they are done
                s_red[tt & 1][rg][c4] = acc;
                __syncthreads();
                if (tid < D) {
                    const float *red = reinterpret_cast<const float *>(&s_red[tt & 1][0][0]);
                    float sum = 0.f;
#pragma unroll 4
                    for (int r = 0; r < RG; ++r) sum += red[r * D + tid];
                    store_f(y + row0 + tt * D + tid, sum);
                }
            }
            // the gates of the next block overwrite s_o, s_f, s_i, all of whose reads precede the last barrier;
            // its first token writes s_red[0] only after the block's staging barrier
        }
#pragma unroll
        for (int j = 0; j < R; ++j) __stcs(Su + (long long)(rg + j * RG) * C4, s[j]);
        __syncthreads();
    }
}

template <typename T, int D>
cudaError_t launch_step_multi_t(const StepArgs &a)
{
    const long long units = (long long)a.B * a.H;
    if (units == 0 || a.T == 0) return cudaSuccess;
    const long long grid = units < (1ll << 30) ? units : (1ll << 30);
    step_multi_kernel<T, D><<<(unsigned)grid, kStepThreads, 0, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), a.S,
        static_cast<T *>(a.y), a.T, units);
    return cudaGetLastError();
}

template <typename T, int DV>
cudaError_t launch_step_t(const StepArgs &a)
{
    const long long units = (long long)a.B * a.H;
    if (units == 0) return cudaSuccess;
    const long long grid = units < (1ll << 30) ? units : (1ll << 30);
    step_kernel<T, DV><<<(unsigned)grid, kStepThreads, 0, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), a.S,
        static_cast<T *>(a.y), a.dk, units);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_step_dv(const StepArgs &a)
{
    switch (a.dv) {
        case 16:  return launch_step_t<T, 16>(a);
        case 32:  return launch_step_t<T, 32>(a);
        case 64:  return launch_step_t<T, 64>(a);
        case 128: return launch_step_t<T, 128>(a);
        default:  return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_step(const StepArgs &a)
{
    return a.io == HGRN2_BF16 ? launch_step_dv<__nv_bfloat16>(a) : launch_step_dv<float>(a);
}

bool step_multi_supported(int dk, int dv) { return dk == dv && (dk == 64 || dk == 128); }

cudaError_t launch_step_multi(const StepArgs &a)
{
    if (!step_multi_supported(a.dk, a.dv)) return cudaErrorInvalidValue;
    if (a.io == HGRN2_BF16)
        return a.dk == 128 ? launch_step_multi_t<__nv_bfloat16, 128>(a) : launch_step_multi_t<__nv_bfloat16, 64>(a);
    return a.dk == 128 ? launch_step_multi_t<float, 128>(a) : launch_step_multi_t<float, 64>(a);
}

}  // namespace hgrn2
