// Internal contract between the host entry points (mor_api.cu) and the kernels
// (mor_kernels.cu).  Not part of the C boundary.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "mor.h"

namespace mor {

// A tile is 128 segments of 128 contiguous BF16 elements (32 KiB), handled by one CTA of
// 256 threads, two threads per segment.  What a segment is depends on the partition:
//   KIND_TENSOR / KIND_ROW128  consecutive 128-element pieces of the rows, row-major
//   KIND_BLK128                the 128 rows of one 128x128 block
constexpr int kSegsPerTile = 128;
constexpr int kSegElems = 128;
constexpr int kThreads = 256;
constexpr int kMaxBatch = 20;   // tensors per launch; the records travel as kernel parameters

enum Kind : int { KIND_TENSOR = 0, KIND_ROW128 = 1, KIND_BLK128 = 2 };

// Per-tile partial results, reduced in tile order by the finalise kernel.
struct Partial {
    double   sum43, sum52;        // relative-error sums of the tile (E4M3, E5M2)
    uint32_t nnz, nonfinite;
    uint32_t n_e4m3, n_e5m2, n_bf16;
    uint32_t min_nz_bits;         // min |x| over non-zeros as BF16 bits, 0xFFFF if none (three-way only)
};
static_assert(sizeof(Partial) == 40, "Partial layout");

struct TensorRec {
    const uint16_t* x;
    uint8_t* codes;
    uint8_t* scale_e8m0;
    uint8_t* sel;
    float* scale_f32;
    uint16_t* fallback;
    mor_block_stats_t* block_stats;
    mor_tensor_stats_t* tensor_stats;
    const float* amax;            // group amax on the device (workspace slot or the caller's)
    float* amax_slot;             // workspace: tensor amax written by the pre-pass (when it runs)
    uint32_t* nonfinite_slot;     // workspace: element count of NaN/inf found by the amax pre-pass
    int64_t rows, cols, ld, codes_ld;
    uint32_t nbc;                 // segments per row = ceil(cols / 128)
    uint32_t nbr;                 // KIND_BLK128: block rows = ceil(rows / 128)
    uint32_t n_units;             // KIND_BLK128: blocks; otherwise segments = rows * nbc
    uint32_t n_tiles;
    uint32_t tile_begin;          // index of the tensor's first Partial
    int32_t criterion, scale_mode, n_formats;
    uint32_t flags;
    float threshold;
};

struct BatchParams {
    int n;
    uint32_t tile_end[kMaxBatch]; // exclusive prefix of tiles within this launch
    TensorRec t[kMaxBatch];
};

struct MainVariant {
    int kind;        // Kind
    bool yard;       // evaluate E5M2 as well (Eq. 3, or statistics asked for)
    bool three;      // three-way recipe: keep E5M2 codes and the non-zero minimum (Eq. 4)
    bool store;      // write codes (false for mor_select_stats)
};

cudaError_t launch_amax(const BatchParams& p, uint32_t total_tiles, cudaStream_t s);
cudaError_t launch_main(const MainVariant& v, const BatchParams& p, Partial* partials,
                        uint32_t total_tiles, cudaStream_t s);
cudaError_t launch_finalise(const BatchParams& p, const Partial* partials, int kind, cudaStream_t s);
cudaError_t launch_copy_amax(const BatchParams& p, float* out, cudaStream_t s);

}  // namespace mor
