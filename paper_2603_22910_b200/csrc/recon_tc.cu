// placeholder until the tcgen05 kernel lands
#include "recon_tc.h"
namespace echokv {
bool tc_shape_supported(int, int, int, int, int) { return false; }
cudaError_t tc_encode_pool_maps(TcLayerMaps*, const void*, const void*, int, uint64_t, int) { return cudaErrorNotSupported; }
cudaError_t tc_encode_weight_maps(TcLayerMaps*, const void*, const void*, int, int) { return cudaErrorNotSupported; }
cudaError_t launch_recon_tc(const AttnArgs&, const ReconArgs&, const TcLayerMaps&, const TcLayerMaps&, int, cudaStream_t) { return cudaErrorNotSupported; }
}
