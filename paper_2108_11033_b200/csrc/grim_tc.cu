// Tensor-core (tcgen05) path for bf16 handles at large N.  Placeholder until the kernel lands:
// reports the path as unavailable so that callers stay on the CUDA-core kernels.
#include "grim_internal.h"

namespace grim {
bool tc_path_supported(const grim_bcr*, const SpmmArgs&) { return false; }
grim_status_t launch_spmm_tc(const grim_bcr*, const SpmmArgs&, cudaStream_t) { return GRIM_ERR_UNSUPPORTED; }
}  // namespace grim
