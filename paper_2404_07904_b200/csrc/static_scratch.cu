// Backward pass for callers that cannot allocate device memory: the chunk-state scratch that
// hgrn2_bwd otherwise takes from the caller's workspace lives in a fixed array inside this library.
#include <mutex>

#include "common.cuh"

namespace {

// Scratch shared by every call of hgrn2_bwd_static_scratch on a device: a 256-byte status block
// followed by the re-created chunk-start states.  Each GPU that loads the library holds one copy
// until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[HGRN2_STATIC_SCRATCH_BYTES + 256];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code the array's name is only a handle; the address kernels can use has to be asked for,
// once per device, with that device current.
void *scratch_for_current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
        g_scratch_addr[dev] = p;
    }
    return g_scratch_addr[dev];
}

}  // namespace

extern "C" hgrn2_status hgrn2_bwd_static_scratch(const hgrn2_desc *desc, const void *o, const void *f, const void *i,
                                                 const float *S0, const void *dy, const float *dSN, void *d_o,
                                                 void *d_f, void *d_i, float *dS0, void *status_out,
                                                 void *cuda_stream)
{
    if (!desc) return HGRN2_ERR_INVALID_ARG;
    const size_t need = hgrn2_workspace_bytes(desc);            // status block + chunk states; 0 = bad desc
    if (need == 0) {
        const bool fields_ok = desc->B >= 0 && desc->H >= 0 && desc->N >= 0 && desc->chunk >= 0 &&
                               (desc->io == HGRN2_F32 || desc->io == HGRN2_BF16);
        return fields_ok ? HGRN2_ERR_UNSUPPORTED : HGRN2_ERR_INVALID_ARG;
    }
    if (need > sizeof(g_static_scratch)) return HGRN2_ERR_WORKSPACE;   // problem too large for the built-in scratch
    if (status_out && (reinterpret_cast<uintptr_t>(status_out) & 15u)) return HGRN2_ERR_ALIGNMENT;
    void *scratch = scratch_for_current_device();
    if (!scratch) return HGRN2_ERR_CUDA;
    // saved = NULL: the states are re-created inside the scratch; the call clears the status block first.
    hgrn2_status st = hgrn2_bwd(desc, o, f, i, S0, dy, dSN, nullptr, d_o, d_f, d_i, dS0, scratch, cuda_stream);
    if (st != HGRN2_OK) return st;
    if (status_out &&
        cudaMemcpyAsync(status_out, scratch, 8, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)) !=
            cudaSuccess)
        return HGRN2_ERR_CUDA;
    return HGRN2_OK;
}
