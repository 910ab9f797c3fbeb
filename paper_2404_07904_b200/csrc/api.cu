// C ABI of the HGRN2 library: argument checks and dispatch.  Every step of the path runs in
// the kernels of this directory; nothing here computes on the host.
#include <stddef.h>
#include <string.h>

#include "common.cuh"

using namespace hgrn2;

namespace hgrn2 {
// tensor-core family (chunk_tc_fwd.cu, chunk_tc_bwd.cu)
bool        tc_supported(const hgrn2_desc *d);
int         tc_default_chunk();
bool        tc_chunk_supported(int C);
size_t      tc_saved_bytes(const hgrn2_desc *d, int C);
size_t      tc_segment_scratch_bytes(const hgrn2_desc *d, int C);
size_t      tc_exact_scratch_bytes(const hgrn2_desc *d, bool packed);
size_t      tc_segment_scratch_bytes_packed(const hgrn2_desc *d);
size_t      tc_saved_bytes_packed(const hgrn2_desc *d);
// span summaries for sequence parallelism (span.cu)
cudaError_t launch_span_summary(bool bwd, int io, const void *x, const void *f, const void *w, long long U, int N, int dk,
                                int dv, float *out, float *lam, cudaStream_t stream);
cudaError_t launch_span_compose(const float *X_all, const float *lam_all, const float *init, float *out, long long U,
                                int dk, int dv, int r0, int r1, int reverse, cudaStream_t stream);
// gate activations (gates.cu)
int         gate_bwd_slices(long long U, int N);
cudaError_t launch_gate_fwd(const SeqArgs &a, const float *beta, void *o_out, void *k_out, void *i_out);
cudaError_t launch_gate_bwd(const SeqArgs &a, const float *beta, float *partial, float *d_beta);
cudaError_t launch_alu_fwd_gated(const SeqArgs &a, const float *beta);
cudaError_t launch_alu_bwd_gated(const SeqArgs &a, const float *beta, float *partial, float *d_beta);
cudaError_t launch_tc_fwd(const SeqArgs &a);
cudaError_t launch_tc_bwd(const SeqArgs &a);
}  // namespace hgrn2

namespace {

bool dim_ok(int d) { return d == 16 || d == 32 || d == 64 || d == 128; }

bool desc_ok(const hgrn2_desc *d)
{
    if (!d) return false;
    if (d->B < 0 || d->H < 0 || d->N < 0) return false;
    if (d->io != HGRN2_F32 && d->io != HGRN2_BF16) return false;
    if (d->chunk < 0) return false;
    return true;
}

bool use_tc(const hgrn2_desc *d)
{
    return !(d->flags & HGRN2_FLAG_FORCE_ALU) && tc_supported(d);
}

// 0 = unsupported
int resolve_chunk(const hgrn2_desc *d)
{
    if (!desc_ok(d) || !dim_ok(d->dk) || !dim_ok(d->dv)) return 0;
    if (use_tc(d)) {
        if (d->chunk == 0) return tc_default_chunk();
        return tc_chunk_supported(d->chunk) ? d->chunk : 0;
    }
    if (d->chunk == 0) return alu_default_chunk(d->dk, d->dv);
    return alu_chunk_supported(d->dk, d->dv, d->chunk) ? d->chunk : 0;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

hgrn2_status check_ptrs(const void *const *req, int nreq, const void *const *opt, int nopt)
{
    for (int j = 0; j < nreq; ++j)
        if (!req[j]) return HGRN2_ERR_INVALID_ARG;
    for (int j = 0; j < nreq; ++j)
        if (!aligned16(req[j])) return HGRN2_ERR_ALIGNMENT;
    for (int j = 0; j < nopt; ++j)
        if (opt[j] && !aligned16(opt[j])) return HGRN2_ERR_ALIGNMENT;
    return HGRN2_OK;
}

size_t state_bytes(const hgrn2_desc *d) { return (size_t)d->B * d->H * d->dk * d->dv * sizeof(float); }

// packed = a variable-length batch: d->B sequences share d->N token rows per head (state slots: see PackedArgs)
size_t saved_bytes_for(const hgrn2_desc *d, int C, bool packed = false)
{
    if (use_tc(d)) return packed ? tc_saved_bytes_packed(d) : tc_saved_bytes(d, C);
    const size_t NC = ((size_t)d->N + C - 1) / C;
    const size_t slots = packed ? (size_t)d->H * ((size_t)d->N / C + d->B + 1) : (size_t)d->B * d->H * NC;
    return slots * d->dk * d->dv * sizeof(float);
}

size_t workspace_bytes_for(const hgrn2_desc *d, int C, bool packed)
{
    return sizeof(StatusBlock) + saved_bytes_for(d, C, packed) +
           (use_tc(d) ? (packed ? tc_segment_scratch_bytes_packed(d) : tc_segment_scratch_bytes(d, C)) +
                            tc_exact_scratch_bytes(d, packed)
                      : 0);
}

void fill_args(SeqArgs &a, const hgrn2_desc *d, int C, void *stream, void *ws, const int32_t *cu = nullptr)
{
    memset(&a, 0, sizeof(a));
    a.cu = cu;
    a.start_aborted = (d->flags & HGRN2_FLAG_DEBUG_EXPIRE_WAITS) ? 1 : 0;
    // workspace layout: status block | room for re-created saved data | tensor-core path: segment scratch, then one
    // float matrix per unit for units redone on the exact path
    a.seg_scratch = nullptr;
    a.exact_scratch = nullptr;
    if (use_tc(d)) {
        char *p = static_cast<char *>(ws) + sizeof(StatusBlock) + saved_bytes_for(d, C, cu != nullptr);
        const size_t seg = cu ? tc_segment_scratch_bytes_packed(d) : tc_segment_scratch_bytes(d, C);
        if (seg != 0) a.seg_scratch = p;
        a.exact_scratch = reinterpret_cast<float *>(p + seg);
    }
    a.B = d->B; a.H = d->H; a.N = d->N; a.dk = d->dk; a.dv = d->dv; a.C = C;
    a.NC = (d->N + C - 1) / C;
    a.io = d->io;
    a.stream = static_cast<cudaStream_t>(stream);
}

}  // namespace

extern "C" {

int32_t hgrn2_chunk(const hgrn2_desc *desc) { return resolve_chunk(desc); }

const char *hgrn2_path(const hgrn2_desc *desc)
{
    if (resolve_chunk(desc) == 0) return "";
    return use_tc(desc) ? "tcgen05" : "alu";
}

size_t hgrn2_saved_bytes(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    if (C == 0) return 0;
    return saved_bytes_for(desc, C);
}

size_t hgrn2_workspace_bytes(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    if (C == 0) return 0;
    return workspace_bytes_for(desc, C, false);
}

size_t hgrn2_saved_bytes_varlen(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    if (C == 0) return 0;
    return saved_bytes_for(desc, C, true);
}

size_t hgrn2_workspace_bytes_varlen(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    if (C == 0) return 0;
    return workspace_bytes_for(desc, C, true);
}

const char *hgrn2_status_string(hgrn2_status s)
{
    switch (s) {
        case HGRN2_OK:              return "ok";
        case HGRN2_ERR_INVALID_ARG: return "invalid argument";
        case HGRN2_ERR_UNSUPPORTED: return "unsupported shape, dtype or chunk";
        case HGRN2_ERR_ALIGNMENT:   return "pointer not 16-byte aligned";
        case HGRN2_ERR_WORKSPACE:   return "workspace missing";
        case HGRN2_ERR_CUDA:        return "CUDA runtime error";
        case HGRN2_ERR_TIMEOUT:     return "device-side wait timed out";
        case HGRN2_ERR_DOMAIN:      return "input outside the supported domain";
    }
    return "unknown status";
}

}  // extern "C"

namespace {

// cu == nullptr: [B][H][N][d] tensors; otherwise a packed batch of desc->B sequences in [H][N][d] tensors
hgrn2_status fwd_impl(const hgrn2_desc *desc, const void *o, const void *f, const void *i, const int32_t *cu,
                      const float *S0, void *y, float *SN, void *saved, void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const bool empty = (size_t)desc->B * desc->H * desc->N == 0;   // sequence tensors have no elements
    const void *req[] = {ws, o, f, i, y};
    const void *opt[] = {S0, SN, saved, o, f, i, y};
    hgrn2_status st = check_ptrs(req, empty ? 1 : 5, opt, empty ? 7 : 3);
    if (st != HGRN2_OK) return st;

    SeqArgs a;
    fill_args(a, desc, C, cuda_stream, ws, cu);
    a.o = o; a.f = f; a.i = i; a.S0 = S0; a.y = y; a.SN = SN;
    a.states = static_cast<float *>(saved);
    a.status = static_cast<StatusBlock *>(ws);
    // The status word starts every call at zero.  On the tensor-core path the first kernel of the call does that
    // itself (a separate clear between two kernels of a stream costs a microsecond of idle GPU each time);
    // everywhere else, and when no kernel will run, it is a small asynchronous memset.
    a.clear_status = use_tc(desc) && !empty;
    if (!a.clear_status && cudaMemsetAsync(ws, 0, sizeof(StatusBlock), a.stream) != cudaSuccess) return HGRN2_ERR_CUDA;
    if ((size_t)desc->B * desc->H == 0) return HGRN2_OK;
    if (desc->N == 0) {
        if (SN) {
            cudaError_t e = S0 ? cudaMemcpyAsync(SN, S0, state_bytes(desc), cudaMemcpyDeviceToDevice, a.stream)
                               : cudaMemsetAsync(SN, 0, state_bytes(desc), a.stream);
            if (e != cudaSuccess) return HGRN2_ERR_CUDA;
        }
        return HGRN2_OK;
    }
    cudaError_t e = use_tc(desc) ? launch_tc_fwd(a) : launch_alu_fwd(a);
    return e == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status bwd_impl(const hgrn2_desc *desc, const void *o, const void *f, const void *i, const int32_t *cu,
                      const float *S0, const void *dy, const float *dSN, const void *saved,
                      void *d_o, void *d_f, void *d_i, float *dS0, void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const bool empty = (size_t)desc->B * desc->H * desc->N == 0;
    const void *req[] = {ws, o, f, i, dy, d_o, d_f, d_i};
    const void *opt[] = {S0, dSN, saved, dS0, o, f, i, dy, d_o, d_f, d_i};
    hgrn2_status st = check_ptrs(req, empty ? 1 : 8, opt, empty ? 11 : 4);
    if (st != HGRN2_OK) return st;

    SeqArgs a;
    fill_args(a, desc, C, cuda_stream, ws, cu);
    a.o = o; a.f = f; a.i = i; a.S0 = S0; a.dy = dy; a.dSN = dSN;
    a.d_o = d_o; a.d_f = d_f; a.d_i = d_i; a.dS0 = dS0;
    a.status = static_cast<StatusBlock *>(ws);
    a.clear_status = use_tc(desc) && !empty;                     // see hgrn2_fwd
    if (!a.clear_status && cudaMemsetAsync(ws, 0, sizeof(StatusBlock), a.stream) != cudaSuccess) return HGRN2_ERR_CUDA;
    if ((size_t)desc->B * desc->H == 0) return HGRN2_OK;
    if (desc->N == 0) {
        if (dS0) {
            cudaError_t e = dSN ? cudaMemcpyAsync(dS0, dSN, state_bytes(desc), cudaMemcpyDeviceToDevice, a.stream)
                                : cudaMemsetAsync(dS0, 0, state_bytes(desc), a.stream);
            if (e != cudaSuccess) return HGRN2_ERR_CUDA;
        }
        return HGRN2_OK;
    }
    const bool tc = use_tc(desc);
    if (saved) {
        a.states = const_cast<float *>(static_cast<const float *>(saved));
    } else {
        // re-create the chunk-start states inside the workspace with a states-only forward
        SeqArgs r = a;
        r.y = nullptr; r.SN = nullptr;
        r.states = reinterpret_cast<float *>(static_cast<char *>(ws) + sizeof(StatusBlock));
        cudaError_t e = tc ? launch_tc_fwd(r) : launch_alu_fwd(r);
        if (e != cudaSuccess) return HGRN2_ERR_CUDA;
        a.states = r.states;
        a.clear_status = false;                                  // the forward's first kernel has done it
    }
    cudaError_t e = tc ? launch_tc_bwd(a) : launch_alu_bwd(a);
    return e == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

}  // namespace

extern "C" {

hgrn2_status hgrn2_fwd(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                       const float *S0, void *y, float *SN, void *saved, void *ws, void *cuda_stream)
{
    return fwd_impl(desc, o, f, i, nullptr, S0, y, SN, saved, ws, cuda_stream);
}

hgrn2_status hgrn2_bwd(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                       const float *S0, const void *dy, const float *dSN, const void *saved,
                       void *d_o, void *d_f, void *d_i, float *dS0, void *ws, void *cuda_stream)
{
    return bwd_impl(desc, o, f, i, nullptr, S0, dy, dSN, saved, d_o, d_f, d_i, dS0, ws, cuda_stream);
}

}  // extern "C"

namespace {

// Gated entry points.  Tensor-core path: `saved` = [o | encoded gate | i] (bf16, what the element-wise kernel in front wrote)
// followed by the ordinary saved data; the workspace = status block | room for all of that when saved is NULL |
// segment scratch | exact-path scratch | partial sums of d_beta.  fp32 path: the ordinary saved data and workspace
// plus one row of partial sums per unit.
size_t gate_tensor_bytes(const hgrn2_desc *d) { return (size_t)d->B * d->H * d->N * d->dk * 2; }

size_t saved_bytes_gated(const hgrn2_desc *d, int C)
{
    return (use_tc(d) ? 3 * gate_tensor_bytes(d) : 0) + saved_bytes_for(d, C);
}

size_t beta_partial_bytes(const hgrn2_desc *d)
{
    const long long U = (long long)d->B * d->H;
    const int P = use_tc(d) ? gate_bwd_slices(U, d->N) : 1;
    return (((size_t)U * P * d->dk * sizeof(float)) + 255) & ~(size_t)255;
}

size_t workspace_bytes_gated(const hgrn2_desc *d, int C)
{
    return sizeof(StatusBlock) + saved_bytes_gated(d, C) +
           (use_tc(d) ? tc_segment_scratch_bytes(d, C) + tc_exact_scratch_bytes(d, false) : 0) + beta_partial_bytes(d);
}

// Pointers into the workspace behind the saved-data room.
void gated_ws_layout(SeqArgs &a, const hgrn2_desc *d, int C, void *ws, float **partial)
{
    char *p = static_cast<char *>(ws) + sizeof(StatusBlock) + saved_bytes_gated(d, C);
    a.seg_scratch = nullptr;
    a.exact_scratch = nullptr;
    if (use_tc(d)) {
        const size_t seg = tc_segment_scratch_bytes(d, C);
        if (seg != 0) a.seg_scratch = p;
        a.exact_scratch = reinterpret_cast<float *>(p + seg);
        p += seg + tc_exact_scratch_bytes(d, false);
    }
    *partial = reinterpret_cast<float *>(p);
}

}  // namespace

extern "C" {

size_t hgrn2_saved_bytes_gated(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    return C == 0 ? 0 : saved_bytes_gated(desc, C);
}

size_t hgrn2_workspace_bytes_gated(const hgrn2_desc *desc)
{
    const int C = resolve_chunk(desc);
    return C == 0 ? 0 : workspace_bytes_gated(desc, C);
}

hgrn2_status hgrn2_fwd_gated(const hgrn2_desc *desc, const void *zo, const void *zf, const void *zi, const float *beta,
                             const float *S0, void *y, float *SN, void *saved, void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const bool empty = (size_t)desc->B * desc->H * desc->N == 0;
    const void *req[] = {ws, zo, zf, zi, y, beta};
    const void *opt[] = {S0, SN, saved, zo, zf, zi, y, beta};
    hgrn2_status st = check_ptrs(req, empty ? 1 : 6, opt, empty ? 8 : 3);
    if (st != HGRN2_OK) return st;

    SeqArgs a;
    fill_args(a, desc, C, cuda_stream, ws);
    float *partial = nullptr;
    gated_ws_layout(a, desc, C, ws, &partial);
    a.o = zo; a.f = zf; a.i = zi; a.S0 = S0; a.y = y; a.SN = SN;
    a.status = static_cast<StatusBlock *>(ws);
    const bool tc = use_tc(desc);
    a.clear_status = tc && !empty;
    if (!a.clear_status && cudaMemsetAsync(ws, 0, sizeof(StatusBlock), a.stream) != cudaSuccess) return HGRN2_ERR_CUDA;
    if ((size_t)desc->B * desc->H == 0) return HGRN2_OK;
    if (desc->N == 0) {
        if (SN) {
            cudaError_t e = S0 ? cudaMemcpyAsync(SN, S0, state_bytes(desc), cudaMemcpyDeviceToDevice, a.stream)
                               : cudaMemsetAsync(SN, 0, state_bytes(desc), a.stream);
            if (e != cudaSuccess) return HGRN2_ERR_CUDA;
        }
        return HGRN2_OK;
    }
    if (!tc) {
        a.states = static_cast<float *>(saved);
        return launch_alu_fwd_gated(a, beta) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
    }
    // the gates go to the head of `saved` (kept for the backward) or, for inference, of the workspace's room for it
    char *gates = saved ? static_cast<char *>(saved) : static_cast<char *>(ws) + sizeof(StatusBlock);
    const size_t gb = gate_tensor_bytes(desc);
    if (launch_gate_fwd(a, beta, gates, gates + gb, gates + 2 * gb) != cudaSuccess) return HGRN2_ERR_CUDA;
    a.o = gates; a.f = gates + gb; a.i = gates + 2 * gb;
    a.gate_enc = true;
    a.states = saved ? reinterpret_cast<float *>(gates + 3 * gb) : nullptr;
    return launch_tc_fwd(a) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_bwd_gated(const hgrn2_desc *desc, const void *zo, const void *zf, const void *zi, const float *beta,
                             const float *S0, const void *dy, const float *dSN, const void *saved, void *d_zo,
                             void *d_zf, void *d_zi, float *d_beta, float *dS0, void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const bool empty = (size_t)desc->B * desc->H * desc->N == 0;
    const void *req[] = {ws, zo, zf, zi, dy, d_zo, d_zf, d_zi, beta};
    const void *opt[] = {S0, dSN, saved, dS0, d_beta, zo, zf, zi, dy, d_zo, d_zf, d_zi, beta};
    hgrn2_status st = check_ptrs(req, empty ? 1 : 9, opt, empty ? 13 : 5);
    if (st != HGRN2_OK) return st;

    SeqArgs a;
    fill_args(a, desc, C, cuda_stream, ws);
    float *partial = nullptr;
    gated_ws_layout(a, desc, C, ws, &partial);
    a.o = zo; a.f = zf; a.i = zi; a.S0 = S0; a.dy = dy; a.dSN = dSN;
    a.d_o = d_zo; a.d_f = d_zf; a.d_i = d_zi; a.dS0 = dS0;
    a.status = static_cast<StatusBlock *>(ws);
    const bool tc = use_tc(desc);
    a.clear_status = tc && !empty;
    if (!a.clear_status && cudaMemsetAsync(ws, 0, sizeof(StatusBlock), a.stream) != cudaSuccess) return HGRN2_ERR_CUDA;
    const size_t beta_bytes = (size_t)desc->H * desc->dk * sizeof(float);
    if (empty) {                                 // no token: nothing depends on beta; the state gradient passes through
        if (d_beta && cudaMemsetAsync(d_beta, 0, beta_bytes, a.stream) != cudaSuccess) return HGRN2_ERR_CUDA;
        if ((size_t)desc->B * desc->H != 0 && dS0) {
            cudaError_t e = dSN ? cudaMemcpyAsync(dS0, dSN, state_bytes(desc), cudaMemcpyDeviceToDevice, a.stream)
                                : cudaMemsetAsync(dS0, 0, state_bytes(desc), a.stream);
            if (e != cudaSuccess) return HGRN2_ERR_CUDA;
        }
        return HGRN2_OK;
    }
    if (!tc) {
        if (saved) {
            a.states = const_cast<float *>(static_cast<const float *>(saved));
        } else {
            SeqArgs r = a;
            r.y = nullptr; r.SN = nullptr;
            r.states = reinterpret_cast<float *>(static_cast<char *>(ws) + sizeof(StatusBlock));
            if (launch_alu_fwd_gated(r, beta) != cudaSuccess) return HGRN2_ERR_CUDA;
            a.states = r.states;
        }
        return launch_alu_bwd_gated(a, beta, partial, d_beta) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
    }
    const size_t gb = gate_tensor_bytes(desc);
    char *gates;
    SeqArgs k = a;                               // the recurrence proper, on o, the encoded gate, i
    k.gate_enc = true;
    if (saved) {
        gates = const_cast<char *>(static_cast<const char *>(saved));
    } else {
        gates = static_cast<char *>(ws) + sizeof(StatusBlock);
        if (launch_gate_fwd(a, beta, gates, gates + gb, gates + 2 * gb) != cudaSuccess) return HGRN2_ERR_CUDA;
        SeqArgs r = k;
        r.o = gates; r.f = gates + gb; r.i = gates + 2 * gb;
        r.y = nullptr; r.SN = nullptr;
        r.states = reinterpret_cast<float *>(gates + 3 * gb);
        if (launch_tc_fwd(r) != cudaSuccess) return HGRN2_ERR_CUDA;
        k.clear_status = false;
    }
    k.o = gates; k.f = gates + gb; k.i = gates + 2 * gb;
    k.states = reinterpret_cast<float *>(gates + 3 * gb);
    if (launch_tc_bwd(k) != cudaSuccess) return HGRN2_ERR_CUDA;
    // d_o, d_f, d_i sit in the output buffers: chain rule through the activations, in place, and d_beta
    return launch_gate_bwd(a, beta, partial, d_beta) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_span_summary_fwd(const hgrn2_desc *desc, const void *f, const void *i, float *S_loc, float *lam,
                                    void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const long long U = (long long)desc->B * desc->H;
    const bool empty = U * desc->N == 0;
    const void *req[] = {ws, S_loc, lam, f, i};
    const void *opt[] = {f, i};
    hgrn2_status st = check_ptrs(req, U == 0 ? 1 : (empty ? 3 : 5), opt, 2);
    if (st != HGRN2_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (U == 0) return cudaMemsetAsync(ws, 0, sizeof(StatusBlock), stream) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
    cudaError_t e;
    if (use_tc(desc) && desc->N > 0) {
        e = launch_tc_state_fwd(f, i, (uint64_t)U, desc->N, S_loc, lam, false, static_cast<StatusBlock *>(ws), true,
                                (desc->flags & HGRN2_FLAG_DEBUG_EXPIRE_WAITS) ? 1 : 0, stream);
    } else {
        if (cudaMemsetAsync(ws, 0, sizeof(StatusBlock), stream) != cudaSuccess) return HGRN2_ERR_CUDA;
        e = launch_span_summary(false, desc->io, nullptr, f, i, U, desc->N, desc->dk, desc->dv, S_loc, lam, stream);
    }
    return e == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_span_summary_bwd(const hgrn2_desc *desc, const void *o, const void *f, const void *dy, float *G_loc,
                                    float *lam, void *ws, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    const int C = resolve_chunk(desc);
    if (C == 0) return HGRN2_ERR_UNSUPPORTED;
    if (!ws) return HGRN2_ERR_WORKSPACE;
    const long long U = (long long)desc->B * desc->H;
    const bool empty = U * desc->N == 0;
    const void *req[] = {ws, G_loc, lam, o, f, dy};
    const void *opt[] = {o, f, dy};
    hgrn2_status st = check_ptrs(req, U == 0 ? 1 : (empty ? 3 : 6), opt, 3);
    if (st != HGRN2_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (U == 0) return cudaMemsetAsync(ws, 0, sizeof(StatusBlock), stream) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
    cudaError_t e;
    if (use_tc(desc) && desc->N > 0) {
        e = launch_tc_state_bwd(o, f, dy, (uint64_t)U, desc->N, G_loc, lam, false, static_cast<StatusBlock *>(ws), true,
                                (desc->flags & HGRN2_FLAG_DEBUG_EXPIRE_WAITS) ? 1 : 0, stream);
    } else {
        if (cudaMemsetAsync(ws, 0, sizeof(StatusBlock), stream) != cudaSuccess) return HGRN2_ERR_CUDA;
        e = launch_span_summary(true, desc->io, o, f, dy, U, desc->N, desc->dk, desc->dv, G_loc, lam, stream);
    }
    return e == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_span_compose(const hgrn2_desc *desc, int32_t r0, int32_t r1, int32_t reverse, const float *X_all,
                                const float *lam_all, const float *init, float *out, void *cuda_stream)
{
    if (!desc_ok(desc) || r0 < 0 || r1 < r0) return HGRN2_ERR_INVALID_ARG;
    if (!dim_ok(desc->dk) || !dim_ok(desc->dv)) return HGRN2_ERR_UNSUPPORTED;
    const long long U = (long long)desc->B * desc->H;
    if (U == 0) return HGRN2_OK;
    const void *req[] = {out, X_all, lam_all};
    const void *opt[] = {init};
    hgrn2_status st = check_ptrs(req, r1 > r0 ? 3 : 1, opt, 1);
    if (st != HGRN2_OK) return st;
    cudaError_t e = launch_span_compose(X_all, lam_all, init, out, U, desc->dk, desc->dv, r0, r1, reverse ? 1 : 0,
                                        static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_fwd_varlen(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              const int32_t *cu_seqlens, const float *S0, void *y, float *SN, void *saved, void *ws,
                              void *cuda_stream)
{
    if (!cu_seqlens) return HGRN2_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u) return HGRN2_ERR_ALIGNMENT;
    return fwd_impl(desc, o, f, i, cu_seqlens, S0, y, SN, saved, ws, cuda_stream);
}

hgrn2_status hgrn2_bwd_varlen(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              const int32_t *cu_seqlens, const float *S0, const void *dy, const float *dSN,
                              const void *saved, void *d_o, void *d_f, void *d_i, float *dS0, void *ws,
                              void *cuda_stream)
{
    if (!cu_seqlens) return HGRN2_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u) return HGRN2_ERR_ALIGNMENT;
    return bwd_impl(desc, o, f, i, cu_seqlens, S0, dy, dSN, saved, d_o, d_f, d_i, dS0, ws, cuda_stream);
}

hgrn2_status hgrn2_step(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                        float *S, void *y, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    if (!dim_ok(desc->dk) || !dim_ok(desc->dv)) return HGRN2_ERR_UNSUPPORTED;
    if ((size_t)desc->B * desc->H == 0) return HGRN2_OK;         // no unit: nothing to update, pointers may be NULL
    const void *req[] = {o, f, i, S, y};
    hgrn2_status st = check_ptrs(req, 5, nullptr, 0);
    if (st != HGRN2_OK) return st;
    StepArgs a;
    a.B = desc->B; a.H = desc->H; a.dk = desc->dk; a.dv = desc->dv; a.io = desc->io;
    a.o = o; a.f = f; a.i = i; a.S = S; a.y = y;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_step(a) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_step_multi(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                              float *S, void *y, void *cuda_stream)
{
    if (!desc_ok(desc)) return HGRN2_ERR_INVALID_ARG;
    if (!step_multi_supported(desc->dk, desc->dv)) return HGRN2_ERR_UNSUPPORTED;
    const bool empty = (size_t)desc->B * desc->H * desc->N == 0;
    if (empty) return HGRN2_OK;                                  // no token: the state stays as it is
    const void *req[] = {o, f, i, S, y};
    hgrn2_status st = check_ptrs(req, 5, nullptr, 0);
    if (st != HGRN2_OK) return st;
    StepArgs a;
    a.B = desc->B; a.H = desc->H; a.dk = desc->dk; a.dv = desc->dv; a.io = desc->io; a.T = desc->N;
    a.o = o; a.f = f; a.i = i; a.S = S; a.y = y;
    a.stream = static_cast<cudaStream_t>(cuda_stream);
    return launch_step_multi(a) == cudaSuccess ? HGRN2_OK : HGRN2_ERR_CUDA;
}

hgrn2_status hgrn2_poll(const void *ws)
{
    if (!ws) return HGRN2_ERR_INVALID_ARG;
    int32_t code = 0;
    if (cudaMemcpy(&code, ws, sizeof(code), cudaMemcpyDeviceToHost) != cudaSuccess) return HGRN2_ERR_CUDA;
    if (code < 0 || code > HGRN2_ERR_DOMAIN) return HGRN2_ERR_CUDA;
    return static_cast<hgrn2_status>(code);
}

int32_t hgrn2_exact_path_units(const void *ws)
{
    if (!ws) return -1;
    int32_t n = 0;
    if (cudaMemcpy(&n, static_cast<const char *>(ws) + offsetof(StatusBlock, exact_units), sizeof(n),
                   cudaMemcpyDeviceToHost) != cudaSuccess)
        return -1;
    return n;
}

}  // extern "C"
