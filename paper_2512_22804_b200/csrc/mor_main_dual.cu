// Instantiations of the fused main kernel: rows and columns of the same tensors from one read (codes are always stored, no BF16 outputs).
#include "mor_main.cuh"

namespace mor {

cudaError_t launch_main_dual(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    if (!v.store) return cudaErrorInvalidValue;     // (pairs that want a BF16 output are never formed)
    if (v.scan) {
        return v.three ? launch_main_t<KIND_DUAL, true, true, true, true, false>(p, partials, s)
             : v.yard  ? launch_main_t<KIND_DUAL, true, false, true, true, false>(p, partials, s)
                       : launch_main_t<KIND_DUAL, false, false, true, true, false>(p, partials, s);
    }
    if (v.three) return launch_main_t<KIND_DUAL, true, true, true, false, false>(p, partials, s);
    // two formats with keys of both directions from the pre-pass: the plain instantiation takes prepared scales and
    // counts nothing per block; with block statistics or a decision that needs per-block counts, the general one
    if (v.extra) return v.yard ? launch_main_t<KIND_DUAL, true, false, true, false, true>(p, partials, s)
                               : launch_main_t<KIND_DUAL, false, false, true, false, true>(p, partials, s);
    return v.yard ? launch_main_t<KIND_DUAL, true, false, true, false, false>(p, partials, s)
                  : launch_main_t<KIND_DUAL, false, false, true, false, false>(p, partials, s);
}

}  // namespace mor
