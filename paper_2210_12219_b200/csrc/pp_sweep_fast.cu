// Register-tiled sweep kernel for 16-bit ranks (placeholder: not built yet).
#include "pp_internal.cuh"

namespace pp {

bool fast_sweep_supported(const Dev &) { return false; }

cudaError_t launch_sweep_fast(const Dev &, int, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace pp
