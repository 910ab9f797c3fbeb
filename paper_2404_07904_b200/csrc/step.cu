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

}  // namespace hgrn2
