// placeholder until the tensor-core kernel lands
#include "attn_common.cuh"
namespace sv {
bool attn_tc_supported(const sv_attn_params &) { return false; }
size_t attn_tc_workspace_bytes(int32_t, int32_t, int32_t, int32_t, int32_t, int32_t) { return 0; }
sv_status launch_attn_tc(const sv_attn_params &, void *, size_t, cudaStream_t) { return SV_EUNSUPPORTED; }
}
