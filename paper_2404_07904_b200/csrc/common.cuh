// Shared device/host helpers of the HGRN2 library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "hgrn2.h"

namespace hgrn2 {

// Smallest forget-gate value the chunked kernels distinguish from zero: below it the
// in-chunk cumulative decay is formed as if f were this value.
constexpr float kFMin = 7.888609052210118e-31f;   // 2^-100
// d_f divides the decay gradient (a sum that cancels down to ~f times its terms) by f.  With the gated entry
// points' encoded gate, f is whatever the sigmoid gave, down to exactly 0; the divisor is kept above 2^-20 there:
// below it the quotient would be the sum's rounding noise times up to 2^100.
constexpr float kFDivMinK = 9.5367431640625e-7f;  // 2^-20

// Layout of the 256-byte status block at the start of every workspace.
struct StatusBlock {
    int32_t code;      // hgrn2_status, 0 = ok; first error wins
    int32_t where;     // kernel-specific location tag of the first error
    int32_t exact_units;   // tensor-core path: units the call redid on the exact fp32 path (decay out of range)
    int32_t pad[61];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");

template <typename T> __device__ __forceinline__ float load_f(const T *p);
template <> __device__ __forceinline__ float load_f<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float load_f<__nv_bfloat16>(const __nv_bfloat16 *p)
{
    return __bfloat162float(*p);
}

template <typename T> __device__ __forceinline__ void store_f(T *p, float x);
template <> __device__ __forceinline__ void store_f<float>(float *p, float x) { *p = x; }
template <> __device__ __forceinline__ void store_f<__nv_bfloat16>(__nv_bfloat16 *p, float x)
{
    *p = __float2bfloat16_rn(x);
}

__device__ __forceinline__ void report_error(StatusBlock *sb, int code, int where)
{
    if (sb != nullptr && atomicCAS(&sb->code, 0, code) == 0) sb->where = where;
}

// A kernel's dynamic shared-memory limit has to be raised once per device before its first launch with more than
// 48 KB; later calls find the (kernel, device) pair here and skip the runtime call.
inline cudaError_t ensure_dynamic_smem(const void *kernel, size_t bytes)
{
    struct Entry { const void *kernel; int device; size_t bytes; };
    static std::mutex mu;
    static std::vector<Entry> done;
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry &e : done)
        if (e.kernel == kernel && e.device == dev) {
            if (e.bytes >= bytes) return cudaSuccess;
            err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (err == cudaSuccess) e.bytes = bytes;
            return err;
        }
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (err == cudaSuccess) done.push_back(Entry{kernel, dev, bytes});
    return err;
}

// ---- internal launchers (defined in the .cu files, called from api.cu) ----------------------

struct SeqArgs {
    int B, H, N, dk, dv, C, NC;
    int io;                       // hgrn2_dtype
    const void *o, *f, *i;        // inputs
    const float *S0;              // nullable
    void *y;                      // fwd out (nullable: states only)
    float *SN;                    // nullable
    float *states;                // [B*H][NC][dk][dv] chunk-start states: fwd writes (nullable), bwd reads
    const void *dy;               // bwd
    const float *dSN;             // nullable
    void *d_o, *d_f, *d_i;        // bwd out
    float *dS0;                   // nullable
    StatusBlock *status;
    void *seg_scratch;            // tensor-core path: scratch for sequences split into segments (nullable)
    float *exact_scratch = nullptr;   // tensor-core backward: [B*H][dk][dv] floats for units redone on the exact path
    float *totals = nullptr;      // tensor-core path: per-chunk decay totals inside the saved data (set by its launchers)
    bool clear_status = false;    // tensor-core path: the first kernel of the call zeroes the status word itself
    int start_aborted = 0;        // tensor-core path, debugging: every CTA starts as if its first wait had run out
    bool gate_enc = false;         // the f tensor holds the signed gate encoding (gated entry points)
    const int *cu = nullptr;      // packed batch: device array of B + 1 row offsets (B = sequences, N = total rows per head)
    cudaStream_t stream;
};

struct StepArgs {
    int B, H, dk, dv, io;
    int T = 1;             // tokens per launch (launch_step_multi)
    const void *o, *f, *i;
    float *S;
    void *y;
    cudaStream_t stream;
};

// Tensor-core path: what a CTA needs to redo a whole unit on the exact fp32 path (chunk_alu.cuh) after its
// sweep has found a decay that the rescaled operands cannot represent.  Plain pointers to unit 0 of the launch
// (the kernels proper work through tensor maps); o == nullptr switches the exact path off.
struct ExactArgs {
    const __nv_bfloat16 *o = nullptr, *f = nullptr, *i = nullptr, *dy = nullptr;
    const float *S0 = nullptr, *dSN = nullptr;
    __nv_bfloat16 *y = nullptr, *d_o = nullptr, *d_f = nullptr, *d_i = nullptr;
    float *SN = nullptr, *dS0 = nullptr;
    __nv_bfloat16 *states = nullptr;    // saved chunk states: [unit][chunk of 64][128][128] bf16
    float *scratch = nullptr;           // backward: [unit][128][128] floats
    int N = 0;                          // tokens of a whole unit (rows per head of a packed batch)
    int G = 1;                          // CTAs (segments) per unit in this launch
    int *unit_flag = nullptr;           // G > 1: per unit, set by any segment that left the range
    int *unit_count = nullptr;          // G > 1: per unit, segments finished so far
};

// Packed (variable-length) batches: the sequence tensors are [H][T][d] and sequence b occupies the token rows
// [cu[b], cu[b + 1]) of every head; unit u = b * H + h.  cu == nullptr: the ordinary [B][H][N][d] layout.
// Chunk-start states of a packed batch live in slots: sequence b owns slots floor(cu[b] / C) + b ... of its head
// (never overlapping the next sequence's), slots_per_head = floor(T / C) + B + 1.
struct PackedArgs {
    const int *cu = nullptr;
    int H = 0;
    int slots_per_head = 0;
};

// Tensor-core path, few or left-over units: which units run whole and which are split into G segments each.
struct SegPlan {
    uint64_t main_units;   // units [0, main_units) run as one CTA each
    uint64_t tail_units;   // units [main_units, main_units + tail_units) are split into G segments each
    int G;
};
SegPlan     tc_seg_plan(uint64_t U, int N, int NC);
// Sequences that are NOT whole chunks, few or left-over units (as SegPlan): those units' sequences are cut into G
// segments of Lc chunks (the last one shorter), which run through the packed-batch geometry (per-CTA rows from an
// offsets array).
struct RSegPlan {
    uint64_t main_units;   // units [0, main_units) run as one CTA each
    uint64_t tail_units;   // units [main_units, main_units + tail_units) run as G segments each (0: nothing is split)
    int G;
    int Lc;
};
RSegPlan    tc_rseg_plan(uint64_t U, int N, int NC);
constexpr size_t kRSegOffsetsBytes = 256;      // the offsets array of the ragged segments, in front of their scratch
void        launch_seg_offsets(int *cu, int G, int L, int N, cudaStream_t stream);
// Packed batch on few units: every sequence is cut into the same number G of segments (short sequences leave
// some of theirs empty); the lengths are known on the device only, so the offsets of the B * G segments are
// written there.  G = 1: not split.
int         tc_packed_segments(uint64_t U, int T);
size_t      tc_packed_offsets_bytes(int B, int G);
void        launch_seg_offsets_packed(const int *cu, int B, int G, int *cu_seg, cudaStream_t stream);
SeqArgs     tc_slice_units(const SeqArgs &a, uint64_t u0, uint64_t n);

cudaError_t launch_tc_state_fwd(const void *f, const void *i, uint64_t U, int N, float *S_loc, float *lam, bool gate_enc,
                                StatusBlock *status, bool clear, int start_aborted, cudaStream_t stream,
                                const int *cu = nullptr, int nseq = 1);
cudaError_t launch_tc_state_bwd(const void *o, const void *f, const void *dy, uint64_t U, int N, float *G_loc,
                                float *lam, bool gate_enc, StatusBlock *status, bool clear, int start_aborted,
                                cudaStream_t stream, const int *cu = nullptr, int nseq = 1);
cudaError_t launch_step(const StepArgs &a);
bool        step_multi_supported(int dk, int dv);
cudaError_t launch_step_multi(const StepArgs &a);
int         alu_default_chunk(int dk, int dv);
bool        alu_chunk_supported(int dk, int dv, int C);
cudaError_t launch_alu_fwd(const SeqArgs &a);
cudaError_t launch_alu_bwd(const SeqArgs &a);

}  // namespace hgrn2
