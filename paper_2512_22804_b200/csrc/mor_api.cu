// Host side of the C boundary: argument checks, workspace layout, grouping of tensors by
// partition kind and launch sequence.  No device code lives here.
#include <cmath>
#include <atomic>
#include <cstring>
#include <vector>

#include "mor_internal.h"

namespace mor {
namespace {

constexpr size_t kAlign = 256;
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct Shape {
    int kind;
    uint32_t nbc, nbr, n_units, n_tiles;
    uint64_t key_words;      // words of block keys the pre-pass writes for the main kernel
    uint64_t n_blocks;
};

// Partition geometry of one descriptor; MOR_OK or the reason it cannot run.
mor_status_t shape_of(const mor_tensor_desc_t& d, Shape& s)
{
    if (d.rows < 0 || d.cols < 0) return MOR_ERR_INVALID_ARG;
    if (d.block_rows == 0 && d.block_cols == 0) s.kind = KIND_TENSOR;
    else if (d.block_rows == 1 && d.block_cols == 128) s.kind = KIND_ROW128;
    else if (d.block_rows == 128 && d.block_cols == 128) s.kind = KIND_BLK128;
    else if (d.block_rows == 64 && d.block_cols == 64) s.kind = KIND_BLK64;
    else if (d.block_rows == 1 && d.block_cols == 0) s.kind = KIND_CHANNEL;
    else if (d.block_rows == 128 && d.block_cols == 1) s.kind = KIND_COL128;
    else if (d.block_rows == 0 && d.block_cols == 1) s.kind = KIND_COLCH;
    else return MOR_ERR_UNSUPPORTED;
    const bool empty = d.rows == 0 || d.cols == 0;
    const uint64_t nbc = empty ? 0 : (uint64_t)(d.cols + 127) / 128;
    const uint64_t nbr = empty ? 0 : (uint64_t)(d.rows + 127) / 128;
    const uint64_t segs = empty ? 0 : (uint64_t)d.rows * nbc;
    if (segs >= (1ull << 31) || nbc >= (1ull << 24)) return MOR_ERR_UNSUPPORTED;
    s.nbc = (uint32_t)nbc;
    s.nbr = (uint32_t)nbr;
    s.n_tiles = (uint32_t)(nbr * nbc);       // the main kernel works on 128 x 128 tiles whatever the partition
    if (s.kind == KIND_BLK128) {
        s.n_units = s.n_tiles;
        s.n_blocks = s.n_units;
    } else if (s.kind == KIND_BLK64) {
        const uint64_t nb = empty ? 0 : ((uint64_t)(d.rows + 63) / 64) * ((uint64_t)(d.cols + 63) / 64);
        if (nb >= (1ull << 31)) return MOR_ERR_UNSUPPORTED;
        s.n_units = (uint32_t)nb;
        s.n_blocks = nb;
    } else if (s.kind == KIND_COL128) {
        const uint64_t nb = empty ? 0 : nbr * (uint64_t)d.cols;
        if (nb >= (1ull << 31)) return MOR_ERR_UNSUPPORTED;
        s.n_units = (uint32_t)nb;
        s.n_blocks = nb;
    } else if (s.kind == KIND_CHANNEL) {
        s.n_units = empty ? 0u : (uint32_t)d.rows;
        s.n_blocks = s.n_units;
    } else if (s.kind == KIND_COLCH) {
        if (d.cols >= (1ll << 31)) return MOR_ERR_UNSUPPORTED;
        s.n_units = empty ? 0u : (uint32_t)d.cols;
        s.n_blocks = s.n_units;
    } else {
        s.n_units = (uint32_t)segs;
        s.n_blocks = s.kind == KIND_TENSOR ? (empty ? 0 : 1) : segs;
    }
    const bool line_keys = s.kind == KIND_ROW128 || s.kind == KIND_COL128 || s.kind == KIND_CHANNEL || s.kind == KIND_COLCH;
    s.key_words = (uint64_t)s.n_tiles * (line_keys ? (uint64_t)kRowKeyStride : (uint64_t)kTileKeyStride);
    if (s.kind == KIND_COLCH) s.key_words += (uint64_t)s.nbc * kTileCols + (uint64_t)s.n_tiles * kTileCols * 4;   // as for rows, below
    if (s.kind == KIND_CHANNEL) s.key_words += (uint64_t)s.nbr * kTileRows      // + one key per row
                                             + (uint64_t)s.n_tiles * kTileRows * 4; // + per tile and row the partial sums of a per-row decision
    return MOR_OK;
}

mor_status_t check_desc(const mor_tensor_desc_t& d, Shape& s)
{
    mor_status_t st = shape_of(d, s);
    if (st != MOR_OK) return st;
    if (d.ld < d.cols) return MOR_ERR_INVALID_ARG;
    if (d.ld % 8 != 0) return MOR_ERR_ALIGNMENT;
    const bool empty = d.rows == 0 || d.cols == 0;
    if (!empty && d.x == nullptr) return MOR_ERR_INVALID_ARG;
    if (!aligned(d.x, 16)) return MOR_ERR_ALIGNMENT;
    if (d.n_formats == 2) {
        if (d.formats[0] != MOR_FMT_E4M3 || d.formats[1] != MOR_FMT_BF16) return MOR_ERR_UNSUPPORTED;
    } else if (d.n_formats == 3) {
        if (d.formats[0] != MOR_FMT_E4M3 || d.formats[1] != MOR_FMT_E5M2 || d.formats[2] != MOR_FMT_BF16)
            return MOR_ERR_UNSUPPORTED;
        // the paper defines the E5M2 metric (Eq. 4) only after the Eq. 3 test, per block;
        // a per-tensor block would need its codes rewritten after the last tile
        if (d.criterion != MOR_CRIT_BLOCK_VS_E5M2 || s.kind == KIND_TENSOR) return MOR_ERR_UNSUPPORTED;
    } else {
        return MOR_ERR_INVALID_ARG;
    }
    if (d.criterion < MOR_CRIT_TENSOR_MEAN_REL || d.criterion > MOR_CRIT_BLOCK_MEAN_REL) return MOR_ERR_INVALID_ARG;
    // per-channel blocks span many tiles: their decision (tensor-level as in Section 4.1, or per row by Eq. 3 or by
    // Eq. 1-2 on the row) is taken after the main kernel, when the codes are written; a row that chose E5M2 would need
    // its codes rewritten, so three formats are not offered here
    if ((s.kind == KIND_CHANNEL || s.kind == KIND_COLCH) && d.n_formats != 2) return MOR_ERR_UNSUPPORTED;
    if (d.scale_mode < MOR_SCALE_GAM || d.scale_mode > MOR_SCALE_FP32_AMAX) return MOR_ERR_INVALID_ARG;
    if (!(d.threshold >= 0.0f) || std::isinf(d.threshold)) return MOR_ERR_INVALID_ARG;
    if (d.flags & ~(uint32_t)(MOR_FLAG_STRICT_TIES | MOR_FLAG_RANGE_MIN_INCLUDES_ZERO)) return MOR_ERR_INVALID_ARG;
    if (d.group_amax && !aligned(d.group_amax, 4)) return MOR_ERR_ALIGNMENT;
    return MOR_OK;
}

mor_status_t check_out(const mor_tensor_desc_t& d, const Shape& s, const mor_outputs_t& o, bool store)
{
    if (o.tensor_stats == nullptr) return MOR_ERR_INVALID_ARG;
    if (o.error_histogram && !aligned(o.error_histogram, 4)) return MOR_ERR_ALIGNMENT;
    if (!aligned(o.tensor_stats, 8) || !aligned(o.block_stats, 4) || !aligned(o.scale_f32, 4)) return MOR_ERR_ALIGNMENT;
    // a per-row decision of the per-channel partition is known only after the main kernel: no BF16 outputs that depend on it
    if ((s.kind == KIND_CHANNEL || s.kind == KIND_COLCH) && d.criterion != MOR_CRIT_TENSOR_MEAN_REL &&
        (o.bf16_fallback != nullptr || o.fake_quant != nullptr))
        return MOR_ERR_UNSUPPORTED;
    const bool empty = d.rows == 0 || d.cols == 0;
    if (store) {
        if (!empty && o.codes == nullptr) return MOR_ERR_INVALID_ARG;
        // sub-column blocks leave their codes transposed: [cols, codes_ld] with the rows along the contiguous dimension
        const bool transposed = s.kind == KIND_COL128 || s.kind == KIND_COLCH;
        if (o.codes_ld < (int64_t)round_up((size_t)(transposed ? d.rows : d.cols), 16)) return MOR_ERR_INVALID_ARG;
        if (o.codes_ld % 16 != 0 || !aligned(o.codes, 16)) return MOR_ERR_ALIGNMENT;
        if (d.scale_mode == MOR_SCALE_FP32_AMAX && o.scale_f32 == nullptr && s.n_blocks) return MOR_ERR_INVALID_ARG;
        if (o.fake_quant && !aligned(o.fake_quant, 16)) return MOR_ERR_ALIGNMENT;
        if (o.bf16_fallback) {
            if (s.kind == KIND_TENSOR || d.criterion == MOR_CRIT_TENSOR_MEAN_REL) return MOR_ERR_UNSUPPORTED;
            if (!aligned(o.bf16_fallback, 16)) return MOR_ERR_ALIGNMENT;
        }
    }
    return MOR_OK;
}

// ---- TMA descriptors (cuTensorMapEncodeTiled, reached through the runtime so that the library
// does not link against the driver library)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static std::atomic<EncodeTiledFn> cached{nullptr};   // host threads may race here: every one stores the same address
    EncodeTiledFn fn = cached.load(std::memory_order_acquire);
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess) {
            fn = reinterpret_cast<EncodeTiledFn>(p);
            cached.store(fn, std::memory_order_release);
        }
    }
    return fn;
}

// One descriptor for the BF16 input [rows, cols] with row pitch ld (box 128 x 128 elements; elements
// past the edge read as zero) and one for the codes [rows, cols] bytes with row pitch codes_ld (box
// 128 x 128 bytes; the part of a box past the edge is not written).
bool encode_maps(const mor_tensor_desc_t& d, const mor_outputs_t& o, bool store, CUtensorMap& in_map, CUtensorMap& out_map)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (enc == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d.cols, (cuuint64_t)d.rows};
    const cuuint32_t box[2] = {(cuuint32_t)kTileCols, (cuuint32_t)kTileRows};
    const cuuint32_t estr[2] = {1, 1};
    const cuuint64_t in_stride[1] = {(cuuint64_t)d.ld * 2};
    if (enc(&in_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d.x), dims, in_stride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (store) {
        const cuuint64_t out_stride[1] = {(cuuint64_t)o.codes_ld};
        const cuuint64_t dims_t[2] = {(cuuint64_t)d.rows, (cuuint64_t)d.cols};      // transposed codes of sub-column blocks
        const bool transposed = d.block_cols == 1 && (d.block_rows == 128 || d.block_rows == 0);
        if (enc(&out_map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, o.codes, transposed ? dims_t : dims, out_stride, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    return true;
}

std::atomic<uint32_t> g_test_skip_tile{0xFFFFFFFFu};
std::atomic<long long> g_test_wait_cycles{kDefaultWaitCycles};
std::atomic<uint32_t> g_test_skip_pre_tile{0xFFFFFFFFu};
std::atomic<long long> g_test_pre_wait_cycles{kDefaultWaitCycles};

struct Layout {
    size_t amax_off, status_off, partial_off, keys_off, total;
};

Layout layout_of(int n, uint64_t tiles, uint64_t key_words)
{
    Layout l;
    l.amax_off = 0;
    l.status_off = (size_t)n * sizeof(float);
    l.partial_off = round_up(l.status_off + sizeof(uint32_t), kAlign);
    l.keys_off = l.partial_off + round_up((size_t)tiles * sizeof(Partial), kAlign);
    l.total = l.keys_off + round_up((size_t)key_words * sizeof(uint32_t), kAlign);
    return l;
}

struct Item {
    const mor_tensor_desc_t* d;
    mor_outputs_t o;
    Shape s;
    MainVariant v;
    uint32_t tile_begin;
    uint64_t key_begin;      // first word of the tensor's keys
    bool prepass;            // the amax pre-pass runs for this tensor (and leaves keys)
    bool has_keys;           // the main kernel finds keys for this tensor (its own pre-pass, or that of the rows' item of its pair)
    long long col_key_begin; // rows' item of a pair: first word of the columns' item's keys, which its pre-pass fills too (-1: none)
    int dual;                // 1, 2: first (1x128 blocks) and second (128x1 blocks) item of a pair on the same tensor
                             // that the main kernel serves from one read of each tile; 0: not part of a pair
    int index;
};

void fill_rec(const Item& it, unsigned char* ws, const Layout& l, TensorRec& r)
{
    const mor_tensor_desc_t& d = *it.d;
    r.x = static_cast<const uint16_t*>(d.x);
    r.codes = it.o.codes;
    r.scale_e8m0 = it.o.scale_e8m0;
    r.sel = it.o.sel;
    r.scale_f32 = it.o.scale_f32;
    r.fallback = static_cast<uint16_t*>(it.o.bf16_fallback);
    r.fake_quant = static_cast<uint16_t*>(it.o.fake_quant);
    r.block_stats = it.o.block_stats;
    r.tensor_stats = it.o.tensor_stats;
    r.hist = it.o.error_histogram;
    r.amax_slot = reinterpret_cast<float*>(ws + l.amax_off) + it.index;
    r.amax = d.group_amax ? d.group_amax : r.amax_slot;
    r.device_status = reinterpret_cast<const uint32_t*>(ws + l.status_off);
    r.keys = it.has_keys ? reinterpret_cast<uint32_t*>(ws + l.keys_off) + it.key_begin : nullptr;
    r.col_keys = (it.s.kind == KIND_COL128 || it.s.kind == KIND_COLCH) ? r.keys
               : (it.prepass && it.col_key_begin >= 0) ? reinterpret_cast<uint32_t*>(ws + l.keys_off) + it.col_key_begin : nullptr;
    const bool lines = it.s.kind == KIND_CHANNEL || it.s.kind == KIND_COLCH;     // blocks are whole rows / whole columns
    r.key_stride = (it.s.kind == KIND_ROW128 || it.s.kind == KIND_COL128 || lines) ? (uint32_t)kRowKeyStride : (uint32_t)kTileKeyStride;
    r.row_keys = (it.prepass && lines) ? r.keys + (size_t)it.s.n_tiles * kRowKeyStride : nullptr;
    const bool per_row = lines && (d.criterion != MOR_CRIT_TENSOR_MEAN_REL || it.o.block_stats != nullptr);
    r.row_part = per_row && r.row_keys ? reinterpret_cast<float4*>(r.row_keys + (size_t)(it.s.kind == KIND_COLCH ? it.s.nbc : it.s.nbr) * kTileRows) : nullptr;
    r.rows = d.rows; r.cols = d.cols; r.ld = d.ld; r.codes_ld = it.o.codes_ld;
    r.nbc = it.s.nbc; r.nbr = it.s.nbr; r.n_units = it.s.n_units; r.n_tiles = it.s.n_tiles;
    r.nbc_blk = (uint32_t)((d.cols + 63) / 64); r.kind = it.s.kind;
    r.tile_begin = it.tile_begin;
    r.criterion = d.criterion; r.scale_mode = d.scale_mode; r.n_formats = d.n_formats;
    r.flags = d.flags | (it.prepass ? kFlagAmaxFinal : 0u); r.threshold = d.threshold;
}

inline bool same_variant(const MainVariant& a, const MainVariant& b)
{
    return a.kind == b.kind && a.yard == b.yard && a.three == b.three && a.store == b.store && a.scan == b.scan &&
           a.extra == b.extra;
}

// The launch sequence shared by every entry point.
mor_status_t run(std::vector<Item>& items, void* workspace, size_t workspace_bytes, cudaStream_t stream,
                 const mor_stage_events_t* ev = nullptr)
{
    auto record = [&](void* e) -> bool {
        return e == nullptr || cudaEventRecord(static_cast<cudaEvent_t>(e), stream) == cudaSuccess;
    };
    const int n = (int)items.size();
    uint64_t tiles = 0;
    uint64_t key_words = 0;
    for (Item& it : items) {
        it.tile_begin = (uint32_t)tiles; tiles += it.s.n_tiles;
        it.key_begin = key_words; key_words += it.s.key_words;
    }
    if (tiles >= (1ull << 31)) return MOR_ERR_UNSUPPORTED;
    // Two neighbouring items that ask for the same tensor under the same recipe, once with 1x128 blocks and once
    // with 128x1 blocks (the operand layouts of the forward and the backward GEMM), are served by one main
    // kernel that reads every tile once.  Nothing in the results depends on it.
    for (int i = 0; i + 1 < n; ++i) {
        Item& a = items[i];
        Item& b = items[i + 1];
        if (a.dual || b.dual || a.s.kind != KIND_ROW128 || b.s.kind != KIND_COL128 || a.s.n_tiles == 0) continue;
        const mor_tensor_desc_t& da = *a.d;
        const mor_tensor_desc_t& db = *b.d;
        const bool same = da.x == db.x && da.rows == db.rows && da.cols == db.cols && da.ld == db.ld &&
                          da.n_formats == db.n_formats && da.criterion == db.criterion && da.threshold == db.threshold &&
                          da.scale_mode == db.scale_mode && da.flags == db.flags && da.group_amax == db.group_amax;
        const bool plain = a.v.store && b.v.store && a.o.bf16_fallback == nullptr && a.o.fake_quant == nullptr &&
                           a.v.yard == b.v.yard && a.v.three == b.v.three;
        if (!same || !plain) continue;
        a.dual = 1; b.dual = 2;
        b.prepass = false;                 // one pre-pass, the rows' item's, leaves the keys of both and the tensor amax
        b.has_keys = a.prepass;
        a.col_key_begin = (long long)b.key_begin;
        a.v.kind = b.v.kind = KIND_DUAL;
        b.v.scan = a.v.scan;
        a.v.extra = b.v.extra = a.v.extra || b.v.extra;    // (one launch serves both items)
    }
    const Layout l = layout_of(n, tiles, key_words);
    if (workspace == nullptr || workspace_bytes < l.total) return MOR_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign)) return MOR_ERR_ALIGNMENT;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    Partial* partials = reinterpret_cast<Partial*>(ws + l.partial_off);
    // every TMA descriptor is encoded before anything is enqueued: a call that fails here has launched nothing.
    // The encoder is a driver entry point and wants a current context; a host thread that has made no runtime
    // call yet has none, so the thread's device is made current first (a no-op for every later call).
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaSetDevice(dev) != cudaSuccess) return MOR_ERR_CUDA;
    }
    std::vector<CUtensorMap> in_maps((size_t)n), out_maps((size_t)n);
    for (int i = 0; i < n; ++i) {
        if (items[i].s.n_tiles == 0) continue;
        if (!encode_maps(*items[i].d, items[i].o, items[i].v.store, in_maps[i], out_maps[i])) return MOR_ERR_CUDA;
    }

    // 1. Algorithm 1, group amax, for the tensors whose caller did not supply it
    if (ev && !record(ev->amax_begin)) return MOR_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, l.partial_off, stream) != cudaSuccess) return MOR_ERR_CUDA;
    {
        MainParams pre;
        pre.device_status = reinterpret_cast<uint32_t*>(ws + l.status_off);
        pre.test_skip_tile = g_test_skip_pre_tile.load(std::memory_order_relaxed);
        pre.wait_cycles = g_test_pre_wait_cycles.load(std::memory_order_relaxed);
        BatchParams& bp = pre.b;
        bp.n = 0;
        uint32_t t_end = 0;
        bool rows_only = false;       // the launch being filled holds tensors that want row keys and nothing else
        auto flush = [&]() -> bool {
            if (bp.n == 0) return true;
            pre.total_tiles = t_end;
            bool ok = launch_amax(pre, rows_only, stream) == cudaSuccess;
            bool channel = false;
            for (int k = 0; k < bp.n; ++k) channel = channel || bp.t[k].kind == KIND_CHANNEL || bp.t[k].kind == KIND_COLCH;
            if (ok && channel) ok = launch_row_keys(bp, stream) == cudaSuccess;
            bp.n = 0; t_end = 0;
            return ok;
        };
        // two rounds: the tensors that want row keys alone go through the pre-pass instantiation made for them
        for (int round = 0; round < 2; ++round) {
            rows_only = round == 0;
            for (int i = 0; i < n; ++i) {
                const Item& it = items[i];
                // a supplied group amax only fixes the shared mantissa; the per-tensor partition still
                // needs its block amax, which is the tensor amax, from the data (Algorithm 1)
                if (!it.prepass) continue;
                const bool wants_rows_only = (it.s.kind == KIND_ROW128 || it.s.kind == KIND_CHANNEL) && it.col_key_begin < 0;
                if (wants_rows_only != rows_only) continue;
                TensorRec& r = bp.t[bp.n];
                fill_rec(it, ws, l, r);
                pre.in_map[bp.n] = in_maps[i];
                t_end += r.n_tiles;
                bp.tile_end[bp.n++] = t_end;
                if (bp.n == kMaxBatch && !flush()) return MOR_ERR_CUDA;
            }
            if (!flush()) return MOR_ERR_CUDA;
        }
    }

    // 2. main kernels, one launch per (variant, chunk of tensors); 3. their finalise kernels
    struct Chunk { BatchParams bp; int kind; };
    std::vector<Chunk> chunks;
    if (ev && !record(ev->main_begin)) return MOR_ERR_CUDA;
    std::vector<char> done(n, 0);
    MainParams mp;
    mp.device_status = reinterpret_cast<uint32_t*>(ws + l.status_off);
    mp.test_skip_tile = g_test_skip_tile.load(std::memory_order_relaxed);
    mp.wait_cycles = g_test_wait_cycles.load(std::memory_order_relaxed);
    for (int i = 0; i < n; ++i) {
        if (done[i]) continue;
        const MainVariant v = items[i].v;
        BatchParams& bp = mp.b;
        bp.n = 0;
        uint32_t t_end = 0;
        auto flush = [&]() -> bool {
            if (bp.n == 0) return true;
            mp.total_tiles = t_end;
            const bool ok = launch_main(v, mp, partials, stream) == cudaSuccess;
            chunks.push_back(Chunk{bp, v.kind});
            bp.n = 0; t_end = 0;
            return ok;
        };
        for (int j = i; j < n; ++j) {
            if (done[j] || !same_variant(items[j].v, v)) continue;
            done[j] = 1;
            if (items[j].s.n_tiles == 0) {
                // an empty tensor has no tiles; its summary is still written by the finalise kernel
                fill_rec(items[j], ws, l, bp.t[bp.n]);
                bp.tile_end[bp.n++] = t_end;
            } else {
                fill_rec(items[j], ws, l, bp.t[bp.n]);
                mp.in_map[bp.n] = in_maps[j];
                mp.out_map[bp.n] = out_maps[j];
                if (items[j].dual == 2) {
                    // the columns' record shares the tiles and the group amax of the rows' record before it
                    if (items[j].d->group_amax == nullptr) bp.t[bp.n].amax = bp.t[bp.n - 1].amax_slot;
                } else {
                    t_end += items[j].s.n_tiles;
                }
                bp.tile_end[bp.n++] = t_end;
            }
            if (bp.n == kMaxBatch && !flush()) return MOR_ERR_CUDA;
        }
        if (!flush()) return MOR_ERR_CUDA;
    }
    if (ev && !record(ev->main_end)) return MOR_ERR_CUDA;
    for (Chunk& c : chunks) {
        if (c.kind == KIND_CHANNEL || c.kind == KIND_COLCH) {
            bool per_row = false;
            for (int k = 0; k < c.bp.n; ++k) per_row = per_row || c.bp.t[k].row_part != nullptr;
            if (per_row && launch_row_decide(c.bp, partials, c.kind, stream) != cudaSuccess) return MOR_ERR_CUDA;
        }
        if (c.kind != KIND_DUAL) {
            if (launch_finalise(c.bp, partials, c.kind, stream) != cudaSuccess) return MOR_ERR_CUDA;
            continue;
        }
        // a launch of pairs: the rows' records and the columns' records are summarised as what they are
        for (int dir = 0; dir < 2; ++dir) {
            BatchParams half;
            half.n = 0;
            for (int k = dir; k < c.bp.n; k += 2) { half.t[half.n] = c.bp.t[k]; half.tile_end[half.n] = 0; ++half.n; }
            if (launch_finalise(half, partials, dir ? KIND_COL128 : KIND_ROW128, stream) != cudaSuccess) return MOR_ERR_CUDA;
        }
    }
    if (ev && !record(ev->finalise_end)) return MOR_ERR_CUDA;
    return MOR_OK;
}

mor_status_t make_item(const mor_tensor_desc_t* d, const mor_outputs_t& o, bool store, int index, Item& it)
{
    if (d == nullptr) return MOR_ERR_INVALID_ARG;
    mor_status_t st = check_desc(*d, it.s);
    if (st != MOR_OK) return st;
    st = check_out(*d, it.s, o, store);
    if (st != MOR_OK) return st;
    it.d = d;
    it.o = o;
    it.index = index;
    it.v.kind = it.s.kind;
    it.v.three = d->n_formats == 3;
    it.v.yard = it.v.three || d->criterion == MOR_CRIT_BLOCK_VS_E5M2 || o.block_stats != nullptr;
    it.v.store = store;
    it.v.extra = (store && (o.bf16_fallback != nullptr || o.fake_quant != nullptr)) || o.block_stats != nullptr ||
                 ((it.s.kind == KIND_CHANNEL || it.s.kind == KIND_COLCH) && d->criterion != MOR_CRIT_TENSOR_MEAN_REL) ||
                 d->criterion == MOR_CRIT_BLOCK_MEAN_REL || (d->flags & MOR_FLAG_RANGE_MIN_INCLUDES_ZERO) != 0;
    // a supplied group amax only fixes the shared mantissa, so the pre-pass can be skipped -- except for
    // the per-tensor partition, whose block amax is the tensor amax and has to come from the data
    // Nor is it needed where the scale has no shared mantissa (E8M0 and FP32-amax modes): those need the block
    // amax only, which the main kernel finds in the tile it has just read, so the tensor is read once.
    const bool whole_rows = it.s.kind == KIND_TENSOR || it.s.kind == KIND_CHANNEL || it.s.kind == KIND_COLCH;
    it.prepass = it.s.n_tiles != 0 && (whole_rows || (d->group_amax == nullptr && d->scale_mode == MOR_SCALE_GAM));
    it.v.scan = !it.prepass;
    it.has_keys = it.prepass;
    it.col_key_begin = -1;
    it.dual = 0;
    return MOR_OK;
}

}  // namespace
}  // namespace mor

using namespace mor;

extern "C" {

size_t mor_workspace_bytes(const mor_tensor_desc_t* host_descs, int n)
{
    if (host_descs == nullptr || n <= 0) return 0;
    uint64_t tiles = 0, key_words = 0;
    for (int i = 0; i < n; ++i) {
        Shape s;
        if (shape_of(host_descs[i], s) != MOR_OK) return 0;
        tiles += s.n_tiles;
        key_words += s.key_words;
    }
    return layout_of(n, tiles, key_words).total;
}

mor_status_t mor_analyze_quantize_batched_ex(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs,
                                             int n, void* workspace, size_t workspace_bytes, void* cuda_stream,
                                             const mor_stage_events_t* host_events)
{
    if (host_descs == nullptr || host_outs == nullptr || n < 0) return MOR_ERR_INVALID_ARG;
    if (n == 0) return MOR_OK;
    std::vector<Item> items((size_t)n);
    for (int i = 0; i < n; ++i) {
        mor_status_t st = make_item(&host_descs[i], host_outs[i], true, i, items[i]);
        if (st != MOR_OK) return st;
    }
    return run(items, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream), host_events);
}

mor_status_t mor_analyze_quantize_batched(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs,
                                          int n, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    return mor_analyze_quantize_batched_ex(host_descs, host_outs, n, workspace, workspace_bytes, cuda_stream, nullptr);
}

mor_status_t mor_analyze_quantize(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    return mor_analyze_quantize_batched(host_desc, host_out, 1, workspace, workspace_bytes, cuda_stream);
}

mor_status_t mor_select_stats(const mor_tensor_desc_t* host_desc, mor_block_stats_t* block_stats,
                              mor_tensor_stats_t* tensor_stats, uint8_t* sel, uint8_t* scale_e8m0,
                              void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    mor_outputs_t o;
    std::memset(&o, 0, sizeof(o));
    o.block_stats = block_stats;
    o.tensor_stats = tensor_stats;
    o.sel = sel;
    o.scale_e8m0 = scale_e8m0;
    std::vector<Item> items(1);
    mor_status_t st = make_item(host_desc, o, false, 0, items[0]);
    if (st != MOR_OK) return st;
    return run(items, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

mor_status_t mor_select_stats_batched(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs, int n,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (host_descs == nullptr || host_outs == nullptr || n < 0) return MOR_ERR_INVALID_ARG;
    if (n == 0) return MOR_OK;
    std::vector<Item> items((size_t)n);
    for (int i = 0; i < n; ++i) {
        mor_outputs_t o = host_outs[i];
        o.codes = nullptr; o.codes_ld = 0; o.bf16_fallback = nullptr; o.fake_quant = nullptr;
        mor_status_t st = make_item(&host_descs[i], o, false, i, items[i]);
        if (st != MOR_OK) return st;
    }
    return run(items, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

mor_status_t mor_group_amax(const mor_tensor_desc_t* host_descs, int n, float* amax_out,
                            void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    if (host_descs == nullptr || n < 0 || (n > 0 && amax_out == nullptr)) return MOR_ERR_INVALID_ARG;
    if (n == 0) return MOR_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const Layout l = layout_of(n, 0, 0);
    if (workspace == nullptr || workspace_bytes < l.total) return MOR_ERR_WORKSPACE;
    if (!aligned(workspace, kAlign) || !aligned(amax_out, 4)) return MOR_ERR_ALIGNMENT;
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    // only the geometry matters here (pointer, shape, pitch, alignment); every descriptor is checked before
    // anything is enqueued
    std::vector<Shape> shapes((size_t)n);
    for (int i = 0; i < n; ++i) {
        const mor_tensor_desc_t& d = host_descs[i];
        const mor_status_t st = shape_of(d, shapes[i]);
        if (st != MOR_OK) return st;
        if (d.ld < d.cols) return MOR_ERR_INVALID_ARG;
        if (d.ld % 8 != 0 || !aligned(d.x, 16)) return MOR_ERR_ALIGNMENT;
        if (d.rows != 0 && d.cols != 0 && d.x == nullptr) return MOR_ERR_INVALID_ARG;
    }
    // the pre-pass reads its tiles with TMA: every descriptor is encoded before anything is enqueued (the encoder
    // wants a current context, see run())
    {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaSetDevice(dev) != cudaSuccess) return MOR_ERR_CUDA;
    }
    std::vector<CUtensorMap> in_maps((size_t)n);
    {
        mor_outputs_t none;
        std::memset(&none, 0, sizeof(none));
        CUtensorMap unused;
        for (int i = 0; i < n; ++i)
            if (shapes[i].n_tiles && !encode_maps(host_descs[i], none, false, in_maps[i], unused)) return MOR_ERR_CUDA;
    }
    if (cudaMemsetAsync(ws, 0, l.partial_off, stream) != cudaSuccess) return MOR_ERR_CUDA;
    MainParams pre;
    pre.device_status = reinterpret_cast<uint32_t*>(ws + l.status_off);
    pre.test_skip_tile = 0xFFFFFFFFu;
    pre.wait_cycles = kDefaultWaitCycles;
    BatchParams& bp = pre.b;
    bp.n = 0;
    uint32_t t_end = 0;
    for (int i = 0; i < n; ++i) {
        Item it;
        mor_tensor_desc_t d = host_descs[i];
        d.group_amax = nullptr;
        it.s = shapes[i];
        std::memset(&it.o, 0, sizeof(it.o));
        it.d = &d; it.index = i; it.tile_begin = 0; it.key_begin = 0; it.prepass = false; it.has_keys = false; it.col_key_begin = -1;   // no keys wanted
        if (it.s.n_tiles) {
            TensorRec& r = bp.t[bp.n];
            fill_rec(it, ws, l, r);
            pre.in_map[bp.n] = in_maps[i];
            t_end += r.n_tiles;
            bp.tile_end[bp.n++] = t_end;
        }
        if (bp.n == kMaxBatch || (i == n - 1 && bp.n)) {
            pre.total_tiles = t_end;
            if (launch_amax(pre, false, stream) != cudaSuccess) return MOR_ERR_CUDA;
            bp.n = 0; t_end = 0;
        }
    }
    if (cudaMemcpyAsync(amax_out, ws + l.amax_off, (size_t)n * sizeof(float), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return MOR_ERR_CUDA;
    return MOR_OK;
}

// ---- host-memory variant: staging layout [x | codes | scale | sel | scale_f32 | block_stats | tensor_stats | workspace]

namespace {
struct Staging {
    size_t x, codes, scale, sel, sf32, bstats, tstats, ws, ws_bytes, total;
};
bool staging_of(const mor_tensor_desc_t& d, int64_t codes_ld, Staging& g)
{
    Shape s;
    if (shape_of(d, s) != MOR_OK) return false;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes ? bytes : 1, kAlign); return o; };
    g.x = take((size_t)d.rows * (size_t)d.ld * 2);
    g.codes = take((size_t)d.rows * (size_t)codes_ld);
    g.scale = take((size_t)s.n_blocks);
    g.sel = take((size_t)s.n_blocks);
    g.sf32 = take((size_t)s.n_blocks * 4);
    g.bstats = take((size_t)s.n_blocks * sizeof(mor_block_stats_t));
    g.tstats = take(sizeof(mor_tensor_stats_t));
    g.ws_bytes = layout_of(1, s.n_tiles, s.key_words).total;
    g.ws = take(g.ws_bytes);
    g.total = off;
    return true;
}
}  // namespace

size_t mor_host_staging_bytes(const mor_tensor_desc_t* host_desc)
{
    if (host_desc == nullptr || host_desc->cols < 0 || host_desc->rows < 0) return 0;
    Staging g;
    if (!staging_of(*host_desc, (int64_t)round_up((size_t)host_desc->cols, 16), g)) return 0;
    return g.total;
}

mor_status_t mor_analyze_quantize_host(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                       void* device_staging, size_t staging_bytes, void* cuda_stream)
{
    if (host_desc == nullptr || host_out == nullptr) return MOR_ERR_INVALID_ARG;
    if (host_desc->group_amax != nullptr) return MOR_ERR_INVALID_ARG;
    if (host_out->bf16_fallback != nullptr) return MOR_ERR_UNSUPPORTED;   // the fallback is the caller's own host tensor
    if (host_out->fake_quant != nullptr) return MOR_ERR_UNSUPPORTED;
    if (host_out->error_histogram != nullptr) return MOR_ERR_UNSUPPORTED;  // a device array that outlives the call
    if (host_desc->block_cols == 1) return MOR_ERR_UNSUPPORTED;   // column blocks leave transposed codes: device entry points only
    if (host_desc->rows < 0 || host_desc->cols < 0 || host_desc->ld < host_desc->cols) return MOR_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int64_t dev_codes_ld = (int64_t)round_up((size_t)host_desc->cols, 16);
    if (host_out->codes_ld < host_desc->cols) return MOR_ERR_INVALID_ARG;
    Staging g;
    if (!staging_of(*host_desc, dev_codes_ld, g)) return MOR_ERR_UNSUPPORTED;
    if (device_staging == nullptr || staging_bytes < g.total) return MOR_ERR_WORKSPACE;
    if (!aligned(device_staging, kAlign)) return MOR_ERR_ALIGNMENT;
    unsigned char* base = static_cast<unsigned char*>(device_staging);

    mor_tensor_desc_t d = *host_desc;
    d.x = base + g.x;
    mor_outputs_t o;
    std::memset(&o, 0, sizeof(o));
    o.codes = base + g.codes;
    o.codes_ld = dev_codes_ld;
    o.scale_e8m0 = base + g.scale;
    o.sel = base + g.sel;
    o.scale_f32 = reinterpret_cast<float*>(base + g.sf32);
    o.block_stats = host_out->block_stats ? reinterpret_cast<mor_block_stats_t*>(base + g.bstats) : nullptr;
    o.tensor_stats = reinterpret_cast<mor_tensor_stats_t*>(base + g.tstats);

    std::vector<Item> items(1);
    mor_status_t st = make_item(&d, o, true, 0, items[0]);
    if (st != MOR_OK) return st;
    if (host_out->tensor_stats == nullptr) return MOR_ERR_INVALID_ARG;
    const Shape& s = items[0].s;
    const size_t xbytes = (size_t)d.rows * (size_t)d.ld * 2;
    if (xbytes && host_desc->x == nullptr) return MOR_ERR_INVALID_ARG;
    if (xbytes && cudaMemcpyAsync(base + g.x, host_desc->x, xbytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return MOR_ERR_CUDA;
    st = run(items, base + g.ws, g.ws_bytes, stream);
    if (st != MOR_OK) return st;
    bool ok = true;
    if (host_out->codes && d.rows && d.cols)
        ok = ok && cudaMemcpy2DAsync(host_out->codes, (size_t)host_out->codes_ld, o.codes, (size_t)dev_codes_ld,
                                     (size_t)d.cols, (size_t)d.rows, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_out->scale_e8m0 && s.n_blocks)
        ok = ok && cudaMemcpyAsync(host_out->scale_e8m0, o.scale_e8m0, (size_t)s.n_blocks, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_out->sel && s.n_blocks)
        ok = ok && cudaMemcpyAsync(host_out->sel, o.sel, (size_t)s.n_blocks, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_out->scale_f32 && s.n_blocks)
        ok = ok && cudaMemcpyAsync(host_out->scale_f32, o.scale_f32, (size_t)s.n_blocks * 4, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (host_out->block_stats && s.n_blocks)
        ok = ok && cudaMemcpyAsync(host_out->block_stats, o.block_stats, (size_t)s.n_blocks * sizeof(mor_block_stats_t),
                                   cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(host_out->tensor_stats, o.tensor_stats, sizeof(mor_tensor_stats_t), cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    return ok ? MOR_OK : MOR_ERR_CUDA;
}

void mor_test_skip_tile_load(uint32_t tile, long long wait_cycles)
{
    g_test_skip_tile.store(tile, std::memory_order_relaxed);
    g_test_wait_cycles.store(tile == 0xFFFFFFFFu || wait_cycles <= 0 ? kDefaultWaitCycles : wait_cycles, std::memory_order_relaxed);
}

void mor_test_skip_prepass_tile_load(uint32_t tile, long long wait_cycles)
{
    g_test_skip_pre_tile.store(tile, std::memory_order_relaxed);
    g_test_pre_wait_cycles.store(tile == 0xFFFFFFFFu || wait_cycles <= 0 ? kDefaultWaitCycles : wait_cycles, std::memory_order_relaxed);
}

const char* mor_status_string(mor_status_t status)
{
    switch (status) {
        case MOR_OK: return "ok";
        case MOR_ERR_INVALID_ARG: return "invalid argument";
        case MOR_ERR_UNSUPPORTED: return "unsupported recipe or block shape";
        case MOR_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
        case MOR_ERR_WORKSPACE: return "workspace missing or too small";
        case MOR_ERR_CUDA: return "CUDA runtime error";
        case MOR_ERR_TIMEOUT: return "device-side wait expired";
        case MOR_ERR_STATIC_SCRATCH: return "tensor needs more scratch than the built-in array holds";
    }
    return "unknown status";
}

int mor_version(void) { return 100; }

}  // extern "C"
