// tcgen05 tensor-core kernel of the expanded layer (placeholder until the kernel lands).
#include "pipe_common.cuh"
namespace pipe {
pipe_status forward_tcgen05(const ForwardArgs&, cudaStream_t) { return PIPE_ERR_UNSUPPORTED; }
}  // namespace pipe
