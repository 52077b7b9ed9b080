// Instantiations of the fused main kernel: the per-tensor partition (the block amax is the tensor amax: always from the pre-pass).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_tensor(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    return v.scan || v.three ? cudaErrorInvalidValue : launch_main_ks<KIND_TENSOR, false>(v, p, partials, s);
}

}  // namespace mor
