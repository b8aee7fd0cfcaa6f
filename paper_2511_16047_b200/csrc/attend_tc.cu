// placeholder until the tcgen05 kernel lands
#include "kernels.cuh"
namespace amskv {
bool tc_supported(int32_t) { return false; }
bool tc_encode_kv_maps(const LayerRegion&, int64_t, int32_t, void*, void*) { return false; }
cudaError_t launch_attend_tc(const Strided&, const Strided&, const LayerRegion&, const void*, const void*,
                             const RangeList&, int32_t, int32_t, int32_t, int32_t, float, int*, int, cudaStream_t)
{
    return cudaErrorNotSupported;
}
}  // namespace amskv
