// ds_attn_pruned, tensor-core path (placeholder until the tcgen05 kernel lands).
#include "ds_common.cuh"

namespace ds {
bool attn_tc_supported(const ds_attn_params &) { return false; }
size_t attn_tc_workspace_bytes(const ds_attn_params &) { return 0; }
int launch_attn_tc(const ds_attn_params &, cudaStream_t) { return DS_ERR_UNSUPPORTED; }
}  // namespace ds
