// placeholder until the tcgen05 backward lands
#include "pskv_common.cuh"
namespace pskv {
bool tc_bwd_supported(const Dims &) { return false; }
size_t tc_bwd_workspace_bytes(const Dims &) { return 0; }
cudaError_t launch_tc_bwd(const BwdArgs &, void *, unsigned int *, cudaStream_t) { return cudaErrorNotSupported; }
}
