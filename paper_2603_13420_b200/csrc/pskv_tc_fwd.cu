// placeholder until the tcgen05 forward lands
#include "pskv_common.cuh"
namespace pskv {
bool tc_fwd_supported(const Dims &) { return false; }
size_t tc_fwd_workspace_bytes(const Dims &) { return 0; }
cudaError_t launch_tc_fwd(const FwdArgs &, void *, unsigned int *, cudaStream_t) { return cudaErrorNotSupported; }
}
