// placeholder until the tensor-core kernel lands: reports "unsupported"
#include "common.cuh"
namespace hyq {
size_t attn_tc_workspace_bytes(const hyq_attn_args&) { return 0; }
int launch_attn_tc(const hyq_attn_args&, float, cudaStream_t) { return HYQ_ERR_UNSUPPORTED; }
}  // namespace hyq
