// placeholder until the tcgen05 window kernel lands
#include "common.cuh"
namespace gf {
bool tc_window_supported(int, int, int, int) { return false; }
cudaError_t launch_window_tc(const void*, const void*, const void*, void*, int, int, int, int, int, float, int,
                             int, int, WsHeader*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace gf
