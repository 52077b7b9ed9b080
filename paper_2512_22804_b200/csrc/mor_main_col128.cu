// Instantiations of the fused main kernel: 128x1 sub-column blocks (the main kernel always scans: the pre-pass leaves no column keys).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_col128(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    return v.scan ? launch_main_ks<KIND_COL128, true>(v, p, partials, s) : cudaErrorInvalidValue;
}

}  // namespace mor
