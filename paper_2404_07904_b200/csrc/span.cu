// Sequence (context) parallelism: what one span of a sequence contributes to the state chain, and how the
// contributions of all spans compose.
//
// Eq. 3 is linear in the state, so a sequence cut into R consecutive spans (one per GPU) needs one exchange: every
// rank summarises its span from a zero boundary state,
//
//   forward :  S_loc = sum_s (k_s prod_{s < r <= end} f_r)^T v_s ,   Lambda = prod f          (per key dimension)
//   backward:  G_loc = sum_t (q_t prod_{start <= r <= t} f_r)^T dy_t , the same Lambda
//
// the ranks all-gather (Lambda, S_loc) - d_k + d_k d_v floats per unit and rank - and each composes its own
// boundary state locally:  S_start[r] = fold_{r' < r}  S <- Diag(Lambda[r']) S + S_loc[r']  (from the sequence's S_0),
// and for the gradient  dS_end[r] = fold_{r' > r}  D <- Diag(Lambda[r']) D + G_loc[r']  (from dS_N).  The span itself
// then runs through hgrn2_fwd / hgrn2_bwd with that boundary state.  On the tensor-core shapes the summaries are
// the state-only kernel of chunk_tc_state.cu; everything else uses the plain loops below.
#include "common.cuh"

namespace hgrn2 {

namespace {

// One CTA per unit, state in shared memory, tokens in order.  kBwd = false: S <- Diag(f_t) S + k_t^T v_t.
// kBwd = true: c <- c f_t, G <- G + (c q_t)^T dy_t.  x = o (backward only), w = i or dy.
template <typename T, bool kBwd>
__global__ void __launch_bounds__(256)
span_summary_kernel(const T *__restrict__ x, const T *__restrict__ f, const T *__restrict__ w, float *__restrict__ out,
                    float *__restrict__ lam, int N, int dk, int dv)
{
    extern __shared__ float sm[];
    float *S = sm;                  // [dk][dv]
    float *a = S + dk * dv;         // [dk]  forward: f_t; backward: c_t q_t
    float *b = a + dk;              // [dk]  forward: k_t; backward: running product c
    float *wv = b + dk;             // [dv]
    const long long u = blockIdx.x;
    const int tid = threadIdx.x, nt = blockDim.x, ss = dk * dv;
    for (int e = tid; e < ss; e += nt) S[e] = 0.f;
    for (int k = tid; k < dk; k += nt) b[k] = 1.f;
    float prod = 1.f;               // forward: Lambda of key dimension tid
    __syncthreads();
    for (int t = 0; t < N; ++t) {
        for (int k = tid; k < dk; k += nt) {
            const float fv = load_f(f + (u * N + t) * dk + k);
            if (kBwd) {
                b[k] *= fv;
                a[k] = b[k] * load_f(x + (u * N + t) * dk + k);
            } else {
                a[k] = fv;
                b[k] = 1.0f - fv;
                prod *= fv;
            }
        }
        for (int v = tid; v < dv; v += nt) wv[v] = load_f(w + (u * N + t) * dv + v);
        __syncthreads();
        for (int e = tid; e < ss; e += nt) {
            const int k = e / dv, v = e - k * dv;
            S[e] = kBwd ? fmaf(a[k], wv[v], S[e]) : fmaf(a[k], S[e], b[k] * wv[v]);
        }
        __syncthreads();
    }
    for (int e = tid; e < ss; e += nt) out[u * ss + e] = S[e];
    if (lam != nullptr)
        for (int k = tid; k < dk; k += nt) lam[u * dk + k] = kBwd ? b[k] : prod;
}

// S_out = fold of (Lambda[r'], X[r']) over r' in [r0, r1) ascending (reverse = 0) or descending (reverse = 1),
// starting from `init` (nullable = zero).  X_all [R][U][dk][dv], lam_all [R][U][dk].
__global__ void span_compose_kernel(const float *__restrict__ X_all, const float *__restrict__ lam_all,
                                    const float *__restrict__ init, float *__restrict__ out, long long U, int dk, int dv,
                                    int r0, int r1, int reverse)
{
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long ss = (long long)dk * dv;
    if (e >= U * ss) return;
    const long long u = e / ss;
    const int k = (int)((e % ss) / dv);
    float S = init ? init[e] : 0.f;
    for (int j = 0; j < r1 - r0; ++j) {
        const int r = reverse ? r1 - 1 - j : r0 + j;
        S = fmaf(lam_all[((long long)r * U + u) * dk + k], S, X_all[(long long)r * U * ss + e]);
    }
    out[e] = S;
}

template <typename T, bool kBwd>
cudaError_t launch_summary_t(const void *x, const void *f, const void *w, long long U, int N, int dk, int dv, float *out,
                             float *lam, cudaStream_t stream)
{
    const size_t smem = ((size_t)dk * dv + 2 * dk + dv) * sizeof(float);
    cudaError_t err = ensure_dynamic_smem(reinterpret_cast<const void *>(span_summary_kernel<T, kBwd>), smem);
    if (err != cudaSuccess) return err;
    span_summary_kernel<T, kBwd><<<(unsigned)U, 256, smem, stream>>>(static_cast<const T *>(x), static_cast<const T *>(f),
                                                                   static_cast<const T *>(w), out, lam, N, dk, dv);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_span_summary(bool bwd, int io, const void *x, const void *f, const void *w, long long U, int N, int dk,
                                int dv, float *out, float *lam, cudaStream_t stream)
{
    if (U == 0) return cudaSuccess;
    if (U > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (io == HGRN2_BF16)
        return bwd ? launch_summary_t<__nv_bfloat16, true>(x, f, w, U, N, dk, dv, out, lam, stream)
                   : launch_summary_t<__nv_bfloat16, false>(x, f, w, U, N, dk, dv, out, lam, stream);
    return bwd ? launch_summary_t<float, true>(x, f, w, U, N, dk, dv, out, lam, stream)
               : launch_summary_t<float, false>(x, f, w, U, N, dk, dv, out, lam, stream);
}

cudaError_t launch_span_compose(const float *X_all, const float *lam_all, const float *init, float *out, long long U,
                                int dk, int dv, int r0, int r1, int reverse, cudaStream_t stream)
{
    const long long n = U * dk * dv;
    if (n == 0) return cudaSuccess;
    span_compose_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(X_all, lam_all, init, out, U, dk, dv, r0, r1,
                                                                         reverse);
    return cudaGetLastError();
}

}  // namespace hgrn2
