// Internal contract between the host entry points (mor_api.cu) and the kernels
// (mor_kernels.cu: amax pre-pass and finalise; mor_main.cu: the fused main kernel).
// Not part of the C boundary.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "mor.h"

// Test hook, exported but not part of mor.h: the next launches of the main kernel leave out the TMA load of tile
// `tile` (numbered within each launch) and give up waiting after `wait_cycles` clock cycles; every such call then
// reports MOR_ERR_TIMEOUT in mor_tensor_stats_t.status.  tile = 0xFFFFFFFF switches the hook off again.
extern "C" MOR_API void mor_test_skip_tile_load(uint32_t tile, long long wait_cycles);
// The same for the amax pre-pass (tiles numbered within each of its launches).
extern "C" MOR_API void mor_test_skip_prepass_tile_load(uint32_t tile, long long wait_cycles);

namespace mor {

// The main kernel works on tiles of 128 rows x 128 columns (32 KiB of BF16), whatever the
// partition: a tile is one 128x128 block, or four 64x64 blocks, or 128 one-row blocks of 128
// elements, or a piece of the single block of the per-tensor partition.  Tiles are numbered row-major over the tile
// grid [ceil(rows/128), ceil(cols/128)].  The amax pre-pass uses the same tiles.
constexpr int kTileRows = 128;
constexpr int kTileCols = 128;
constexpr int kSegsPerTile = 128;
constexpr int kSegElems = 128;
constexpr int kThreads = 256;          // amax and finalise kernels; compute threads of the main kernel
constexpr int kMainThreads = 320;      // 8 compute warps + load warp + store warp
constexpr int kRowKeyStride = kTileRows + 4;   // 128 block keys + the count of finite non-zero elements of the tile (+ padding to 16 bytes)
constexpr int kTileKeyStride = 8;              // up to 4 block keys + the count (+ padding)
constexpr int kMaxBatch = 16;          // tensors per launch; records and tensor maps travel as kernel parameters

enum Kind : int { KIND_TENSOR = 0, KIND_ROW128 = 1, KIND_BLK128 = 2, KIND_BLK64 = 3, KIND_CHANNEL = 4, KIND_COL128 = 5,
                  // main kernel only: 1x128 blocks and 128x1 blocks of the same tensor from one read of each tile; the
                  // launch's records come in pairs (rows, columns) that share their tiles
                  KIND_DUAL = 6,
                  // per-channel along the columns: one block per column; computed like 128x1 blocks (column pieces,
                  // transposed codes) with the column's scale taken from keys that span all tile rows
                  KIND_COLCH = 7 };

// Per-tile partial results, reduced in tile order by the finalise kernel.
struct Partial {
    double   sum43, sum52;        // relative-error sums of the tile (E4M3, E5M2)
    uint32_t nnz, nonfinite;
    uint32_t n_e4m3, n_e5m2, n_bf16;
    uint32_t min_nz_bits;         // min |x| over non-zeros as BF16 bits minus one, 0xFFFF if none
};
static_assert(sizeof(Partial) == 40, "Partial layout");

struct TensorRec {
    const uint16_t* x;
    uint8_t* codes;
    uint8_t* scale_e8m0;
    uint8_t* sel;
    float* scale_f32;
    uint16_t* fallback;
    uint16_t* fake_quant;
    mor_block_stats_t* block_stats;
    mor_tensor_stats_t* tensor_stats;
    uint32_t* hist;               // optional 12-bin histogram of the tensor-level error (Section 4.1.3)
    const float* amax;            // group amax on the device (workspace slot or the caller's)
    float* amax_slot;             // workspace: tensor amax written by the pre-pass (when it runs)
    const uint32_t* device_status;// workspace: non-zero when a bounded device-side wait expired
    uint32_t* keys;               // workspace: block keys written by the pre-pass (nullptr: none)
    uint32_t* col_keys;           // workspace: per tile one key per column piece (kRowKeyStride words per tile, the tile's
                                  // non-zero count after the 128 keys), wanted from the pre-pass.  Blocks along the
                                  // columns: the same area as `keys`; the rows' record of a rows-and-columns pair: the
                                  // key area of the columns' record; nullptr: none
    uint32_t* row_keys;           // KIND_CHANNEL: one key per row (the row's amax over all its tiles), padded to 128 rows;
                                  // KIND_COLCH: one key per column, padded to 128 columns
    float4* row_part;             // KIND_CHANNEL / KIND_COLCH with a per-line decision or per-line statistics: per tile and row (column) of the tile
                                  // {sum of E4M3 terms, sum of E5M2 terms, bits(non-zeros | non-finites << 16), unused},
                                  // written by the main kernel, added up along each row by mor_row_decide_kernel
    uint32_t key_stride;          // words per tile in `keys`: kRowKeyStride (one key per row piece, then the tile's
                                  // non-zero count) or kTileKeyStride (one key per tile, or one per 64x64 quadrant in the
                                  // order top-left, top-right, bottom-left, bottom-right; word 4: the tile's non-zero count)
    int64_t rows, cols, ld, codes_ld;
    uint32_t nbc;                 // tile columns = ceil(cols / 128)
    uint32_t nbr;                 // tile rows = ceil(rows / 128)
    uint32_t nbc_blk;             // KIND_BLK64: block columns = ceil(cols / 64)
    int32_t kind;                 // Kind
    uint32_t n_units;             // blocks of the partition (KIND_TENSOR: row pieces, used by the pre-pass)
    uint32_t n_tiles;
    uint32_t tile_begin;          // index of the tensor's first Partial
    int32_t criterion, scale_mode, n_formats;
    uint32_t flags;
    float threshold;
};

// Internal bit of TensorRec::flags (the public MOR_FLAG_* bits are the low ones): the amax pre-pass ran for this
// tensor, so its amax slot is final and the main kernel need not gather the tensor amax.
constexpr uint32_t kFlagAmaxFinal = 0x80000000u;

struct BatchParams {
    int n;
    uint32_t tile_end[kMaxBatch]; // exclusive prefix of tiles within this launch
    TensorRec t[kMaxBatch];
};

// Parameters of the main kernel: the records plus one TMA descriptor per tensor for the BF16
// input (box 128 x 128 elements) and one for the code output (box 128 x 128 bytes).
struct alignas(64) MainParams {
    CUtensorMap in_map[kMaxBatch];
    CUtensorMap out_map[kMaxBatch];
    BatchParams b;
    uint32_t total_tiles;
    uint32_t* device_status;
    long long wait_cycles;        // a wait on an mbarrier gives up after this many clock cycles (kDefaultWaitCycles: about 0.2 s)
    uint32_t test_skip_tile;      // test hook: the load of this tile of the launch is never started (0xFFFFFFFF: none)
};

constexpr long long kDefaultWaitCycles = 400000000ll;

static_assert(sizeof(MainParams) <= 32764, "kernel parameters are limited to 32764 bytes");

struct MainVariant {
    int kind;        // Kind
    bool yard;       // evaluate E5M2 as well (Eq. 3, or statistics asked for)
    bool three;      // three-way recipe: keep E5M2 codes and the non-zero minimum (Eq. 4)
    bool store;      // write codes (false for mor_select_stats)
    bool scan;       // the kernel scans the data for amax / smallest non-zero itself (no keys from the pre-pass)
    bool extra;      // some tensor of the launch wants more than codes, scales, selection and the tensor summary: a BF16
                     // copy of rejected blocks, the fake-quantised output, block statistics, or a decision that needs the
                     // per-block count of non-zeros (Eq. 1-2 per block; the literal minimum of Eq. 4)
};

// Programmatic dependent launch: a kernel launched with launch_dependent() may become resident while the
// kernel before it in the stream is still draining; it runs its prologue and then blocks in pdl_wait() until that
// kernel has completed and its writes are visible.  A kernel lets its successor in early with pdl_trigger()
// (called by every CTA at its start, so the successor's CTAs only take what finishing CTAs free).  Every CTA of
// a kernel launched this way passes pdl_wait(), so completion of a kernel implies completion of all before it.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}
#endif

cudaError_t launch_amax(const MainParams& p, bool rows_only, cudaStream_t s);   // records, input tensor maps, tile count, status word, wait limit
cudaError_t launch_row_keys(const BatchParams& p, cudaStream_t s);      // per-channel: keys of whole rows / whole columns
cudaError_t launch_row_decide(const BatchParams& p, Partial* partials, int kind, cudaStream_t s);
cudaError_t launch_main(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s);
cudaError_t launch_finalise(const BatchParams& p, const Partial* partials, int kind, cudaStream_t s);

}  // namespace mor
