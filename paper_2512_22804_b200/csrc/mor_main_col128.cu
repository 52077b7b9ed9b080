// Instantiations of the fused main kernel: 128x1 sub-column blocks.
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_col128(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    return v.scan ? launch_main_ks<KIND_COL128, true>(v, p, partials, s) : launch_main_ks<KIND_COL128, false>(v, p, partials, s);
}

}  // namespace mor
