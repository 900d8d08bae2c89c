// Small-token weight-streaming kernel of the expanded layer (placeholder until the kernel lands).
#include "pipe_common.cuh"
namespace pipe {
pipe_status forward_stream(const ForwardArgs&, cudaStream_t) { return PIPE_ERR_UNSUPPORTED; }
}  // namespace pipe
