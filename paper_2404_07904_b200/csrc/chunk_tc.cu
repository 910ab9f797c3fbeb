// tcgen05 tensor-core family: placeholder until the kernels land (nothing is served from here yet).
#include "common.cuh"

namespace hgrn2 {
bool        tc_supported(const hgrn2_desc *) { return false; }
int         tc_default_chunk() { return 64; }
bool        tc_chunk_supported(int C) { return C == 64; }
size_t      tc_saved_bytes(const hgrn2_desc *, int) { return 0; }
cudaError_t launch_tc_fwd(const SeqArgs &) { return cudaErrorNotSupported; }
cudaError_t launch_tc_bwd(const SeqArgs &) { return cudaErrorNotSupported; }
}  // namespace hgrn2
