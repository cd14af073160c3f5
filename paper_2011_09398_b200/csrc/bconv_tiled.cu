#include "common.cuh"
namespace lce {
lce_status launch_bconv_tiled(const ConvGeom &, const uint32_t *, const uint32_t *, const float *, const float *,
                              const int32_t *, void *, cudaStream_t)
{
    return LCE_ERR_UNSUPPORTED;
}
}  // namespace lce
