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

// Where unit u lives: first token row in the [rows][d] view, tokens, chunks, first chunk-state slot.  Ordinary
// layout: unit u owns rows [u N, u N + N).  Packed batch (cu set; unit = sequence b, head h; N rows per head):
// rows [h N + cu[b], h N + cu[b + 1]), state slots from h (N / C + B + 1) + cu[b] / C + b.
struct Geom { long long row; int n; int nc; long long slot; };
__device__ inline Geom unit_geom(long long u, int N, int C, int NC, const int *cu, int H)
{
    if (cu == nullptr) return Geom{u * N, N, NC, u * NC};
    const int B = gridDim.x / H;
    const int b = (int)(u / H), h = (int)(u - (long long)b * H);
    const int start = cu[b];
    int n = cu[b + 1] - start;
    if (start < 0 || n < 0 || start + n > N) n = 0;          // malformed offsets: touch nothing
    return Geom{(long long)h * N + start, n, (n + C - 1) / C, (long long)h * (N / C + B + 1) + start / C + b};
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_fwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const float *__restrict__ S0, T *__restrict__ y, float *__restrict__ SN,
               float *__restrict__ states, int N, int dk, int dv, int C, int NC, const int *__restrict__ cu, int H)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    const Geom g = unit_geom(u, N, C, NC, cu, H);
    alu::fwd_unit<T, float>(smem, o + g.row * dk, f + g.row * dk, i + g.row * dv, S0 ? S0 + u * ss : nullptr,
                            y ? y + g.row * dv : nullptr, SN ? SN + u * ss : nullptr,
                            states ? states + g.slot * ss : nullptr, 1, g.n, dk, dv, C, g.nc);
}

template <typename T>
__global__ void __launch_bounds__(kAluThreads)
alu_bwd_kernel(const T *__restrict__ o, const T *__restrict__ f, const T *__restrict__ i,
               const T *__restrict__ dy, const float *__restrict__ dSN,
               const float *__restrict__ states, T *__restrict__ d_o, T *__restrict__ d_f,
               T *__restrict__ d_i, float *__restrict__ dS0, int N, int dk, int dv, int C, int NC,
               const int *__restrict__ cu, int H)
{
    extern __shared__ float smem[];
    const long long u = blockIdx.x, ss = (long long)dk * dv;
    const Geom g = unit_geom(u, N, C, NC, cu, H);
    alu::bwd_unit<T, float>(smem, o + g.row * dk, f + g.row * dk, i + g.row * dv, dy + g.row * dv,
                            dSN ? dSN + u * ss : nullptr, states + g.slot * ss, 1, nullptr, d_o + g.row * dk,
                            d_f + g.row * dk, d_i + g.row * dv, dS0 ? dS0 + u * ss : nullptr, g.n, dk, dv, C, g.nc);
}

constexpr size_t kMaxSmem = 227 * 1024;

template <typename T>
cudaError_t launch_fwd_t(const SeqArgs &a)
{
    const size_t smem = alu::fwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(alu_fwd_kernel<T>), smem);
    if (err != cudaSuccess) return err;
    alu_fwd_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i), a.S0,
        static_cast<T *>(a.y), a.SN, a.states, a.N, a.dk, a.dv, a.C, a.NC, a.cu, a.H);
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bwd_t(const SeqArgs &a)
{
    const size_t smem = alu::bwd_smem_floats(a.dk, a.dv, a.C) * sizeof(float);
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(alu_bwd_kernel<T>), smem);
    if (err != cudaSuccess) return err;
    alu_bwd_kernel<T><<<(unsigned)((long long)a.B * a.H), kAluThreads, smem, a.stream>>>(
        static_cast<const T *>(a.o), static_cast<const T *>(a.f), static_cast<const T *>(a.i),
        static_cast<const T *>(a.dy), a.dSN, a.states, static_cast<T *>(a.d_o), static_cast<T *>(a.d_f),
        static_cast<T *>(a.d_i), a.dS0, a.N, a.dk, a.dv, a.C, a.NC, a.cu, a.H);
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
