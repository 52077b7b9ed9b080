// Instantiations of the fused main kernel: per-channel blocks along the columns (one block per column; the column's
// amax spans tile rows, so it is always taken from the pre-pass; codes are stored transposed).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_colch(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    return v.scan || v.three ? cudaErrorInvalidValue : launch_main_ks<KIND_COLCH, false>(v, p, partials, s);
}

}  // namespace mor
