// LM-head projection (placeholder until the tensor-core kernel lands): reports "not supported".
#include "polyspec_kernels.cuh"

namespace polyspec {

size_t lmhead_workspace_bytes(int, int, int) { return 0; }

cudaError_t launch_lmhead(const void*, const void*, int, int, int, float*, int32_t*, cudaStream_t)
{
    return cudaErrorNotSupported;
}

}  // namespace polyspec
