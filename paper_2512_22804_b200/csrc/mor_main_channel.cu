// Instantiations of the fused main kernel: per-channel blocks (the row amax spans tiles: always taken from the pre-pass).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_channel(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    return v.scan || v.three ? cudaErrorInvalidValue : launch_main_ks<KIND_CHANNEL, false>(v, p, partials, s);
}

}  // namespace mor
