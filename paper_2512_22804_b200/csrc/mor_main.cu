// Dispatch of the fused main kernel by partition kind; the kernel itself is in mor_main.cuh and is
// instantiated kind by kind in the mor_main_*.cu files (separate files so that they compile side by side).
#include "mor_internal.h"

namespace mor {

cudaError_t launch_main_tensor(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_row128(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_blk128(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_blk64(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_col128(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_channel(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_dual(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_main_colch(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);

cudaError_t launch_main(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
    if (p.total_tiles == 0) return cudaSuccess;
    switch (v.kind) {
        case KIND_TENSOR: return launch_main_tensor(v, p, partials, s);
        case KIND_ROW128: return launch_main_row128(v, p, partials, s);
        case KIND_BLK128: return launch_main_blk128(v, p, partials, s);
        case KIND_BLK64: return launch_main_blk64(v, p, partials, s);
        case KIND_COL128: return launch_main_col128(v, p, partials, s);
        case KIND_CHANNEL: return launch_main_channel(v, p, partials, s);
        case KIND_DUAL: return launch_main_dual(v, p, partials, s);
        case KIND_COLCH: return launch_main_colch(v, p, partials, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mor
