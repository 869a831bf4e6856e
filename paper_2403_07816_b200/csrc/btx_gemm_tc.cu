#include "btx_common.cuh"
namespace btx {
btx_status launch_expert_forward_bf16(const Plan&, const void*, const void*, const void*, const Buffers&, int, cudaStream_t) { return BTX_ERR_UNSUPPORTED; }
btx_status launch_expert_backward_bf16(const Plan&, const void*, const void*, const void*, const Buffers&, float*, float*, float*, int, cudaStream_t) { return BTX_ERR_UNSUPPORTED; }
}
