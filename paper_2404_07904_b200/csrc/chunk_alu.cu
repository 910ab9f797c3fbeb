// Chunkwise forward and backward of the HGRN2 recurrence on fp32 CUDA cores.
//
// This is the path for float32 I/O (a single-pass bf16/tf32 tensor-core product cannot hold
// a 1e-4 error bound) and for every shape the tensor-core kernels do not cover.  One CTA per
// (batch, head) unit walks the chunks in order (forward) or in reverse (backward) with the
// running state S (forward) or state gradient dS (backward) resident in shared memory.
//
// The per-unit bodies (and the chunk-local formulas they follow) are in chunk_alu.cuh.
#include "chunk_alu.cuh"

namespace hgrn2 {

namespace {

constexpr int kAluThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_fwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const float *__restrict__ S0, T *__restrict__ y, float *__restrict__ SN,
               float *__restrict__ states, int N, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    alu::fwd_unit<T, float>(smem, o + u * N * dk, f + u * N * dk, i + u * N * dv, S0 ? S0 + u * ss : nullptr,
                            y ? y + u * N * dv : nullptr, SN ? SN + u * ss : nullptr,
                            states ? states + u * NC * ss : nullptr, 1, N, dk, dv, C, NC);
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_bwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const T *__restrict__ dy, const float *__restrict__ dSN,
               const float *__restrict__ states, T *__restrict__ d_o, T *__restrict__ d_f,
               T *__restrict__ d_i, float *__restrict__ dS0, int N, int dk, int dv, int C, int NC)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    alu::bwd_unit<T, float>(smem, o + u * N * dk, f + u * N * dk, i + u * N * dv, dy + u * N * dv,
                            dSN ? dSN + u * ss : nullptr, states + u * NC * ss, 1, nullptr, d_o + u * N * dk,
                            d_f + u * N * dk, d_i + u * N * dv, dS0 ? dS0 + u * ss : nullptr, N, dk, dv, C, NC);
}

constexpr size_t kMaxSmem = 227 * 1024;

template <typename T>
cudaError_t launch_fwd_t(const SeqArgs &a)
{
    const size_t smem = alu::fwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = cudaFuncSetAttribute(alu_fwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    alu_fwd_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), a.S0,
        static_cast<T *>(a.y), a.SN, a.states, a.N, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bwd_t(const SeqArgs &a)
{
    const size_t smem = alu::bwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = cudaFuncSetAttribute(alu_bwd_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    alu_bwd_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i),
        static_cast<const T *>(a.dy), a.dSN, a.states, static_cast<T *>(a.d_o), static_cast<T *>(a.d_f),
        static_cast<T *>(a.d_i), a.dS0, a.N, a.dk, a.dv, a.C, a.NC);
    return cudaGetLastError();
}

}  // namespace

bool alu_chunk_supported(int dk, int dv, int C)
{
    if (C != 16 && C != 32 && C != 64) return false;
    return alu::bwd_smem_floats(dk, dv, C) * sizeof(float) <= kMaxSmem &&
           alu::fwd_smem_floats(dk, dv, C) * sizeof(float) <= kMaxSmem;
}

int alu_default_chunk(int dk, int dv)
{
    for (int C = 64; C >= 16; C /= 2)
        if (alu_chunk_supported(dk, dv, C)) return C;
    return 0;
}

// one CTA per unit: the unit count must fit the grid's x dimension
static bool grid_ok(const SeqArgs &a) { return (long long)a.B * a.H <= 0x7fffffffLL; }

cudaError_t launch_alu_fwd(const SeqArgs &a)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    if (!grid_ok(a)) return cudaErrorInvalidConfiguration;
    return a.io == HGRN2_BF16 ? launch_fwd_t<__nv_bfloat16>(a) : launch_fwd_t<float>(a);
}

cudaError_t launch_alu_bwd(const SeqArgs &a)
{
    if ((long long)a.B * a.H == 0 || a.N == 0) return cudaSuccess;
    if (!grid_ok(a)) return cudaErrorInvalidConfiguration;
    return a.io == HGRN2_BF16 ? launch_bwd_t<__nv_bfloat16>(a) : launch_bwd_t<float>(a);
}

}  // namespace hgrn2
