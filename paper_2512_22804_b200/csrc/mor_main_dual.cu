// Instantiations of the fused main kernel: rows and columns of the same tensors from one read (codes are always stored, no BF16 outputs; every thread counts its non-zeros).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_dual(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    if (!v.store) return cudaErrorInvalidValue;     // (pairs that want a BF16 output are never formed; statistics are always on here)
    if (v.scan) {
        return v.three ? launch_main_t<KIND_DUAL, true, true, true, true, false>(p, partials, s)
             : v.yard  ? launch_main_t<KIND_DUAL, true, false, true, true, false>(p, partials, s)
                       : launch_main_t<KIND_DUAL, false, false, true, true, false>(p, partials, s);
    }
    return v.three ? launch_main_t<KIND_DUAL, true, true, true, false, false>(p, partials, s)
         : v.yard  ? launch_main_t<KIND_DUAL, true, false, true, false, false>(p, partials, s)
                   : launch_main_t<KIND_DUAL, false, false, true, false, false>(p, partials, s);
}

}  // namespace mor
