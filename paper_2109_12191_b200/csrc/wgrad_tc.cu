// placeholder until the tcgen05 kernel lands: nothing is eligible, so every layer takes the CUDA-core path
#include "wgrad_tc.cuh"
namespace dp {
bool tc_eligible(int, const ConvGeom &, int) { return false; }
int tc_norm_slots(int, const ConvGeom &, int) { return 0; }
size_t tc_workspace_bytes(int, const ConvGeom &, int) { return 0; }
dp_status launch_conv_tc(int, int, const void *, const void *, const ConvGeom &, float *, float *, int, const float *,
                         float *, void *, int *, cudaStream_t) { return DP_ERR_UNSUPPORTED; }
}  // namespace dp
