// Stage 1b on tensor cores (placeholder until the tcgen05 kernel lands: reports "not supported",
// so every call takes the CUDA-core kernel).
#include "tsd_common.cuh"
namespace tsd {
bool attention_tc_supported(const AttnArgs&) { return false; }
size_t attention_tc_workspace_bytes(const tsd_layout&) { return 0; }
int launch_attention_tc(const AttnArgs&) { return TSD_ERR_UNSUPPORTED; }
}  // namespace tsd
