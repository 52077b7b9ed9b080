// The fused main kernel of the MoR analyse-and-quantise pass for sm_100a (device code and launcher template;
// included by the mor_main_*.cu files, each of which instantiates the kernel for one partition kind).
//
// Per 128 x 128 tile: block amax and GAM scale (Algorithm 1), cast to E4M3 and E5M2,
// relative-error sums (Eq. 1-3), range statistics (Eq. 4), per-block decision (Algorithm 2),
// codes, scale bytes, selection bytes and a per-tile partial for the tensor-wide aggregate.
//
// Structure: persistent CTAs (two per SM), ten warps each.
//   load warp      sleeps on a hardware barrier until the compute warps have copied a stage of the
//                  two-stage ring of 32 KiB buffers to registers, then one thread starts the TMA
//                  tile load (cp.async.bulk.tensor.2d, zero fill past the tensor's edge) of the
//                  tile that uses the stage next; an mbarrier per stage tells when it has landed;
//   compute warps  8 warps.  A thread takes its 64 elements of the tile from the stage (two threads per tile row; with
//                  128x128 blocks one 16-byte chunk of eight rows; with column blocks four columns over 16 rows,
//                  or a column piece gathered by 16-bit loads), takes the block's scale as the load warp prepared
//                  it from the key that the amax pre-pass left (or scans its elements for amax and smallest
//                  non-zero where the caller supplied the group amax and no pre-pass ran), converts and
//                  accumulates the error terms, and writes its codes to a 16 KiB staging buffer.  Without BF16
//                  outputs it streams: 16 registers of data at a time, straight from the stage;
//   store warp     sleeps on a hardware barrier until the staging buffer is complete, issues the
//                  TMA tile store of the codes (clipped at the tensor's edge by the hardware, to 16-byte pieces of a row),
//                  adds up the threads' sums in a fixed order, and writes the tile's partial and the blocks'
//                  decisions and metadata (with the optional outputs, or three formats in line blocks, the
//                  compute threads decide).
// The load warp and the store warp keep what they need of a tensor's record in registers: reading the kernel's
// parameter space once per tile with a computed index is slow enough to make them the pipeline's bottleneck.
// Every wait on an mbarrier is bounded; a wait that runs out sets a status word that the
// finalise kernel copies into mor_tensor_stats_t.status.  From then on the CTA's threads skip
// the work and the waits but keep every barrier arrival, so that nobody is left waiting.
//
// Arithmetic that must be exact: amax (integer compare of BF16 bit patterns), the scale (IEEE
// binary32 division, looked up by the 7 mantissa bits of the BF16 amax from a table that each
// CTA fills with that same division), the scaled value (one IEEE binary32 multiply) and the FP8
// codes (cvt.rn.satfinite).  The error ratio uses an approximate reciprocal; it only feeds
// sums that are compared with a tolerance.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <float.h>
#include <stddef.h>

#include <atomic>
#include <mutex>

#include "mor_internal.h"
#include "mor_ptx.cuh"

namespace mor {
namespace {

constexpr int kStages = 2;
constexpr int kInBytes = kTileRows * kTileCols * 2;      // 32768
constexpr int kOutBytes = kTileRows * kTileCols;         // 16384
constexpr int kComputeWarps = kThreads / 32;             // 8
constexpr int kLoadWarp = kComputeWarps;                 // warp 8; warp 9 is the store warp
constexpr int kBarCompute = 1;                           // hardware barrier of the compute threads
constexpr int kBarOutFull = 2;                           // + staging buffer index: compute threads arrive, store warp waits
constexpr int kBarStageFree = 4;                         // + stage index: compute threads arrive, load warp waits
constexpr uint32_t kBf16Inf = 0x7F80u;
constexpr uint32_t kSelNone = 3u;                        // entry of a tile row outside the tensor

// What the load warp tells the other warps about the tile in a stage.
struct __align__(16) TileMeta {
    int32_t ti;            // tensor index within the launch
    int32_t vrows, vcols;  // rows / columns of the tile inside the tensor (1..128)
    uint32_t blk_base;     // ROW128: index of the block of the tile's first row
    uint32_t local;        // tile index within the tensor
    int32_t row0, col0;    // first row / column of the tile
    uint32_t nnz;          // finite non-zero elements of the tile, counted by the pre-pass (prepared tiles only)
};

// What a compute thread hands to the store warp: its (ROW128: its block's) sums and counts.
struct __align__(16) Entry {
    float e43, e52;
    uint32_t nnz_nonf;     // non-zeros | non-finites << 16
    uint32_t sel_min;      // selection (kSelNone: not a block) | (smallest non-zero bits - 1) << 16
};

struct Control {
    unsigned long long full[kStages];                   // input ring: the tile has landed
    unsigned long long out_empty[2];                    // code staging + entries have been consumed
    unsigned long long dec_full[2];                     // BLK128: the block's decision, when compute threads need it
    unsigned long long codes_full[2];                   // BLK128, three formats: codes in place after the decision
    TileMeta meta[kStages];
    alignas(16) uint32_t keys[kStages][kRowKeyStride];             // block keys of the tile from the pre-pass (arrive with the tile)
    alignas(16) uint32_t prep[kStages][kTileRows];              // by the load warp, from the keys: scale bits of the row's block (entry = row),
                                                         // of the quadrant (entry q) or of the tile (entry 0); bit 31: careful path
    Entry entry[2][kThreads];
    // 128x128 and 64x64 blocks (a tile holds one block, or four: index q = 2 * (row >= 64) + (column >= 64))
    uint32_t wmax[2][2][2 * kComputeWarps];              // per tile parity, per pass: warp (and column half) amax | inverted min
    uint32_t tile_scale[2][4][2];                        // scale bits (E4M3, E5M2) of the tile's blocks
    uint32_t tile_key[2][4];                             // amax bits << 16 | 0xFFFF - (min - 1)
    uint32_t dec_sel[2][4];
    alignas(16) float wsum[2][3][kComputeWarps];         // 128x128 blocks, three formats: per warp the E4M3 sum, the E5M2 sum, NaN/inf count (as bits)
    uint32_t rtab[128];                                  // bits of fl32(448 / (1 + m/128))
    // blocks along the columns with prepared scales (compute_cols_fast): what the store warp needs per tile besides
    // the entries -- per column the scale bits (bit 31: the column piece holds NaN or inf), per warp the count of
    // NaN/inf elements, and the tile's count of finite non-zeros from the pre-pass
    alignas(16) uint32_t prep2[kStages][kTileCols];      // rows and columns from one read: the columns' prepared scales (prep holds the rows')
    alignas(16) uint32_t colscale[2][kTileCols];
    uint32_t colflag[kStages];                           // by the load warp: some column of the tile needs the careful path
    uint32_t colnonf[2][kComputeWarps];
    uint32_t colnnz[2];
    uint32_t issued;                                     // tile loads issued so far by this CTA
    volatile uint32_t abort;
};

constexpr int kSmemBytes = 1024 + kStages * kInBytes + 2 * kOutBytes + (int)sizeof(Control);
static_assert(2 * (kSmemBytes + 1024) <= 228 * 1024, "two CTAs per SM must fit in shared memory");
static_assert(offsetof(Control, keys) % 16 == 0 && offsetof(Control, prep) % 16 == 0 && offsetof(Control, entry) % 16 == 0 &&
              offsetof(Control, prep2) % 16 == 0 && offsetof(Control, colscale) % 16 == 0 && offsetof(Control, wmax) % 16 == 0 &&
              offsetof(Control, meta) % 16 == 0, "16-byte shared-memory accesses");

// (PTX helpers for mbarriers, TMA copies and shared-memory accesses: mor_ptx.cuh)

// barrier over the compute threads that also ORs a predicate
__device__ __forceinline__ bool compute_bar_or(bool v)
{
    uint32_t r;
    asm volatile("{ .reg .pred p, q; setp.ne.u32 p, %1, 0; barrier.cta.red.or.pred q, %2, %3, p; selp.u32 %0, 1, 0, q; }"
                 : "=r"(r) : "r"((uint32_t)v), "n"(kBarCompute), "n"(kThreads) : "memory");
    return r != 0;
}
// Producer / consumer hand-off on hardware barriers: the 256 compute threads announce, the 32
// threads of the load warp (a stage is free) or of the store warp (a staging buffer is complete)
// sleep until all have.  A thread asleep on a hardware barrier takes no issue slots.
__device__ __forceinline__ void stage_free_arrive(uint32_t s)
{
    asm volatile("barrier.cta.arrive %0, %1;" ::"r"(kBarStageFree + s), "n"(kThreads + 32) : "memory");
}
__device__ __forceinline__ void stage_free_sync(uint32_t s)
{
    asm volatile("barrier.cta.sync %0, %1;" ::"r"(kBarStageFree + s), "n"(kThreads + 32) : "memory");
}
__device__ __forceinline__ void out_full_arrive(uint32_t b)
{
    asm volatile("barrier.cta.arrive %0, %1;" ::"r"(kBarOutFull + b), "n"(kThreads + 32) : "memory");
}
__device__ __forceinline__ void out_full_sync(uint32_t b)
{
    asm volatile("barrier.cta.sync %0, %1;" ::"r"(kBarOutFull + b), "n"(kThreads + 32) : "memory");
}

// {hi, lo} -> two FP8 codes, `lo` in the low byte (round to nearest even, saturate to the largest finite)
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t cvt_e5m2x2(float hi, float lo)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// two FP8 codes -> f16x2 (exact: every E4M3 and E5M2 value is a binary16 number)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t c)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(static_cast<uint16_t>(c)));
    return r;
}
__device__ __forceinline__ uint32_t e5m2x2_to_f16x2(uint32_t c)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(r) : "h"(static_cast<uint16_t>(c)));
    return r;
}
// Four scaled values -> their four E4M3 codes in one word (y0 in the low byte: memory order) and the codes'
// values as two f16x2 words.  One statement, so that the 16-bit halves never pass through 32-bit variables
// (which would cost a mask each).  The pairs are joined first and decoded from the joined word: decoding a
// pair straight from its conversion, before the join, gave wrong values with this compiler (checked on the
// device against this form).
__device__ __forceinline__ void cast4_e4m3(float y0, float y1, float y2, float y3, uint32_t& codes, uint32_t& q01, uint32_t& q23)
{
    asm("{ .reg .b16 l, h;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 l, %4, %3;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 h, %6, %5;\n\t"
        "mov.b32 %0, {l, h};\n\t"
        "cvt.rn.f16x2.e4m3x2 %1, l;\n\t"
        "cvt.rn.f16x2.e4m3x2 %2, h; }"
        : "=r"(codes), "=r"(q01), "=r"(q23) : "f"(y0), "f"(y1), "f"(y2), "f"(y3));
}
__device__ __forceinline__ void cast4_e5m2(float y0, float y1, float y2, float y3, uint32_t& codes, uint32_t& q01, uint32_t& q23)
{
    asm("{ .reg .b16 l, h;\n\t"
        "cvt.rn.satfinite.e5m2x2.f32 l, %4, %3;\n\t"
        "cvt.rn.satfinite.e5m2x2.f32 h, %6, %5;\n\t"
        "mov.b32 %0, {l, h};\n\t"
        "cvt.rn.f16x2.e5m2x2 %1, l;\n\t"
        "cvt.rn.f16x2.e5m2x2 %2, h; }"
        : "=r"(codes), "=r"(q01), "=r"(q23) : "f"(y0), "f"(y1), "f"(y2), "f"(y3));
}
// (q.lo - ylo, q.hi - yhi) with q binary16 and y binary32, each one binary32 operation; exact
// here because q is the FP8 neighbour of y
__device__ __forceinline__ void diff_f16x2_f32(uint32_t q, float ylo, float yhi, float& dlo, float& dhi)
{
    asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; sub.f32.f16 %0, l, %3; sub.f32.f16 %1, h, %4; }"
        : "=f"(dlo), "=f"(dhi) : "r"(q), "f"(ylo), "f"(yhi));
}
// the two BF16 halves of a word as binary32, by the mixed-precision subtract x - 0 (keeps -0)
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi)
{
    asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; sub.f32.bf16 %0, l, %3; sub.f32.bf16 %1, h, %3; }"
        : "=f"(lo), "=f"(hi) : "r"(w), "f"(0.0f));
}
__device__ __forceinline__ float rcp_ftz(float a)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}
__device__ __forceinline__ float rcp_approx(float a)
{
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// two IEEE binary32 multiplies / fused multiply-adds in one instruction (each lane rounds to nearest even)
__device__ __forceinline__ unsigned long long mul_f32x2(unsigned long long a, unsigned long long b)
{
    unsigned long long r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c)
{
    unsigned long long r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// ------------------------------------------------------------------ Algorithm 1 ----

// Algorithm 1's binary32 scaling factor 448 / amax by one IEEE division; a quotient above the largest
// finite binary32 is replaced by it
__device__ __forceinline__ uint32_t ideal_scale_bits_div(float amax)
{
    return __float_as_uint(fminf(__fdiv_rn(448.0f, amax), FLT_MAX));
}

// The same for an amax that is a finite non-zero BF16 value, given as its 15 magnitude bits:
// 448 / (2^e * (1 + m/128)) = (448 / (1 + m/128)) * 2^-e, and scaling by a power of two is exact
// as long as the result stays a normal binary32 (it always does at the small end; at the large end,
// and for subnormal amax, the exponent test finds the overflow).
__device__ __forceinline__ uint32_t ideal_scale_bits_tab(uint32_t a, const uint32_t* rtab)
{
    const int32_t e = (int32_t)(a >> 7);
    const uint32_t t = rtab[a & 127u];
    const int32_t ef = (int32_t)(t >> 23) + 127 - e;
    return ef > 254 ? 0x7F7FFFFFu : t + (uint32_t)((127 - e) * (1 << 23));
}

// Algorithm 1, group part: mantissa of 448 / g_amax (0 for an all-zero tensor, and for the
// scale modes that have no shared mantissa)
__device__ __forceinline__ uint32_t group_mantissa(float g_amax, int scale_mode)
{
    if (scale_mode != MOR_SCALE_GAM || !(g_amax > 0.0f)) return 0u;
    return ideal_scale_bits_div(g_amax) & 0x7FFFFFu;
}

// Algorithm 1, block part: exponent of 448 / b_amax, lowered by one when the group mantissa
// exceeds the block's; the scale is the shared mantissa joined to that exponent.  The E5M2
// scale is 7 binades higher (57344 = 448 * 2^7), capped at exponent field 254.
__device__ __forceinline__ void block_scale(uint32_t amax_bits, uint32_t m_g, int scale_mode, const uint32_t* rtab,
                                            uint32_t& s4_bits, uint32_t& s5_bits)
{
    uint32_t e = 127u, m = (scale_mode == MOR_SCALE_FP32_AMAX) ? 0u : m_g;
    if (amax_bits != 0u) {
        const uint32_t sb = ideal_scale_bits_tab(amax_bits, rtab);
        const uint32_t m_b = sb & 0x7FFFFFu;
        e = sb >> 23;
        if (scale_mode == MOR_SCALE_FP32_AMAX) m = m_b;
        else if (m_g > m_b) e -= 1u;
    }
    const uint32_t e5 = min(e + 7u, 254u);
    s4_bits = (e << 23) | m;
    s5_bits = (e5 << 23) | m;
}

__device__ __forceinline__ float minnz_value(uint32_t minm1_bits)
{
    return minm1_bits == 0xFFFFu ? __uint_as_float(0x7F800000u) : __uint_as_float((minm1_bits + 1u) << 16);
}

// ------------------------------------------------------------------ scan ----

// Block statistics of a thread's 64 elements in one pass over packed BF16 pairs, returned as
// one word: amax bits << 16 | 0xFFFF - (smallest non-zero bits - 1), so that both combine with
// a packed 16-bit maximum.
//   amax  per-halfword max of the |x| bit patterns.  NaN and inf compare above every finite
//         pattern, which is how a non-finite input is noticed.
//   min   per-halfword min of (|x| bits - 1) mod 2^16: zeros wrap to 0xFFFF and drop out.
__device__ __forceinline__ uint32_t scan_words(const uint32_t (&w)[32])
{
    uint32_t mx[2] = {0u, 0u}, mn[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
        const uint32_t a0 = w[i] & 0x7FFF7FFFu, a1 = w[i + 1] & 0x7FFF7FFFu, a2 = w[i + 2] & 0x7FFF7FFFu, a3 = w[i + 3] & 0x7FFF7FFFu;
        mx[0] = __vimax3_u16x2(mx[0], a0, a1);
        mx[1] = __vimax3_u16x2(mx[1], a2, a3);
        mn[0] = __viaddmin_u16x2(a0, 0xFFFFFFFFu, mn[0]);
        mn[1] = __viaddmin_u16x2(a1, 0xFFFFFFFFu, mn[1]);
        mn[2] = __viaddmin_u16x2(a2, 0xFFFFFFFFu, mn[2]);
        mn[3] = __viaddmin_u16x2(a3, 0xFFFFFFFFu, mn[3]);
    }
    const uint32_t mxx = __vimax3_u16x2(mx[0], mx[1], mx[1]);
    const uint32_t mnn = __vimin3_u16x2(__vimin3_u16x2(mn[0], mn[1], mn[2]), mn[3], mn[3]);
    const uint32_t amax = max(mxx & 0xFFFFu, mxx >> 16), minm1 = min(mnn & 0xFFFFu, mnn >> 16);
    return (amax << 16) | (0xFFFFu - minm1);
}

// the same over finite elements only (used once a non-finite element has been seen).  A real
// call, with the words passed by value in registers: inlined, the compiler turns this rare path
// into predicated instructions that every tile would pay for.
__device__ __forceinline__ void scan_finite4(uint4 v, uint32_t& m, uint32_t& n)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
        if (lo < kBf16Inf) { m = max(m, lo); n = min(n, (lo - 1u) & 0xFFFFu); }
        if (hi < kBf16Inf) { m = max(m, hi); n = min(n, (hi - 1u) & 0xFFFFu); }
    }
}
__device__ __noinline__ uint32_t scan_finite_call(uint4 a, uint4 b, uint4 c, uint4 d, uint4 e, uint4 f, uint4 g, uint4 h)
{
    uint32_t m = 0u, n = 0xFFFFu;
    scan_finite4(a, m, n); scan_finite4(b, m, n); scan_finite4(c, m, n); scan_finite4(d, m, n);
    scan_finite4(e, m, n); scan_finite4(f, m, n); scan_finite4(g, m, n); scan_finite4(h, m, n);
    return (m << 16) | (0xFFFFu - n);
}
__device__ __forceinline__ uint32_t scan_words_finite(const uint32_t (&w)[32])
{
#define MOR_W4(j) make_uint4(w[4 * (j)], w[4 * (j) + 1], w[4 * (j) + 2], w[4 * (j) + 3])
    return scan_finite_call(MOR_W4(0), MOR_W4(1), MOR_W4(2), MOR_W4(3), MOR_W4(4), MOR_W4(5), MOR_W4(6), MOR_W4(7));
#undef MOR_W4
}

__device__ __forceinline__ uint32_t key_max(uint32_t a, uint32_t b) { return __vimax3_u16x2(a, b, b); }

// Where a streaming thread finds the j-th of its eight 16-byte chunks of the stage, and where the chunk's eight codes
// go in the staging buffer.  Swizzled (a thread owns half a tile row: the chunks of its 128 bytes in an order that
// keeps the lanes of a load or store phase on distinct banks) or LINEAR (partitions whose blocks are not made of
// rows -- a thread then owns chunk tid & 15 of rows (tid >> 4) + 16 j, the lanes of a phase read neighbouring
// chunks of one row, and every address is its base plus a constant).
template <bool LINEAR> __device__ __forceinline__ uint32_t in_chunk(uint32_t a, int j) { return LINEAR ? a + (uint32_t)(j * 16 * 256) : a ^ (uint32_t)(j << 4); }
template <bool LINEAR> __device__ __forceinline__ uint32_t out_chunk(uint32_t a, int j) { return LINEAR ? a + (uint32_t)(j * 16 * 128) : a ^ (uint32_t)(j << 3); }

// The same two scans for a thread that has not copied its elements to registers: the eight 16-byte chunks are read
// from the stage (the conversion reads them a second time afterwards).
template <bool LINEAR = false>
__device__ __forceinline__ uint32_t scan_stage(uint32_t a)
{
    uint32_t mx[2] = {0u, 0u}, mn[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 v = lds128(in_chunk<LINEAR>(a, j));
        const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
        mx[0] = __vimax3_u16x2(mx[0], a0, a1);
        mx[1] = __vimax3_u16x2(mx[1], a2, a3);
        mn[0] = __viaddmin_u16x2(a0, 0xFFFFFFFFu, mn[0]);
        mn[1] = __viaddmin_u16x2(a1, 0xFFFFFFFFu, mn[1]);
        mn[2] = __viaddmin_u16x2(a2, 0xFFFFFFFFu, mn[2]);
        mn[3] = __viaddmin_u16x2(a3, 0xFFFFFFFFu, mn[3]);
    }
    const uint32_t mxx = __vimax3_u16x2(mx[0], mx[1], mx[1]);
    const uint32_t mnn = __vimin3_u16x2(__vimin3_u16x2(mn[0], mn[1], mn[2]), mn[3], mn[3]);
    const uint32_t amax = max(mxx & 0xFFFFu, mxx >> 16), minm1 = min(mnn & 0xFFFFu, mnn >> 16);
    return (amax << 16) | (0xFFFFu - minm1);
}
template <bool LINEAR = false>
__device__ __noinline__ uint32_t scan_stage_finite(uint32_t a)
{
    uint32_t m = 0u, n = 0xFFFFu;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) scan_finite4(lds128(in_chunk<LINEAR>(a, j)), m, n);
    return (m << 16) | (0xFFFFu - n);
}

// Raise the tensor amax slot to the BF16 magnitude `bits` (non-negative binary32 patterns order like the
// values).  Atomics on one address are served one at a time, so the slot is read first: after the first
// tiles of a tensor almost every call ends there.
__device__ __forceinline__ void raise_amax(float* slot, uint32_t bits, bool active)
{
    if (!active || bits == 0u) return;
    unsigned int* p = reinterpret_cast<unsigned int*>(slot);
    if (__ldcg(p) < (bits << 16)) atomicMax(p, bits << 16);
}

// ------------------------------------------------------------------ conversion ----

// Fast path for two BF16 pairs (four neighbouring elements): four E4M3 codes, and their terms of Eq. 1-3
// for E4M3 (and, with YARD, for E5M2).   y = fl32(x * scale); c = RNE-saturating cast; q = value of c;
// term = |y - q| / |y|, formed as |y - q| * |rcp(y + 2^-126)| (the sum inside a fused
// multiply-add).  The caller guarantees that the block holds no NaN/inf and that every non-zero
// |y| is at least 2^-100, so the added constant changes a term by less than 2^-26 relative, and a
// zero element gives 0 * 2^126.  With COUNT the same reciprocal counts the non-zeros: y * rcp is 1 for a
// non-zero element (within 2^-22) and 0 for a zero.  Pair p of the quad adds into a43[p], a52[p], cnt2[p].
template <bool YARD, bool COUNT>
__device__ __forceinline__ void convert_quad_fast(uint32_t w0, uint32_t w1, unsigned long long s4x2,
                                                  unsigned long long tiny2, float (&a43)[2], float (&a52)[2],
                                                  unsigned long long (&cnt2)[2], uint32_t& c4, uint32_t& c5)
{
    float x0, x1, x2, x3;
    unpack_bf16x2(w0, x0, x1);
    unpack_bf16x2(w1, x2, x3);
    const unsigned long long xa = pack_f32x2(x0, x1), xb = pack_f32x2(x2, x3);
    const unsigned long long ya = mul_f32x2(xa, s4x2), yb = mul_f32x2(xb, s4x2);
    float y0, y1, y2, y3, u0, u1, u2, u3;
    unpack_f32x2(ya, y0, y1);
    unpack_f32x2(yb, y2, y3);
    unpack_f32x2(fma_f32x2(xa, s4x2, tiny2), u0, u1);
    unpack_f32x2(fma_f32x2(xb, s4x2, tiny2), u2, u3);
    const float r0 = rcp_ftz(u0), r1 = rcp_ftz(u1), r2 = rcp_ftz(u2), r3 = rcp_ftz(u3);
    if (COUNT) {
        cnt2[0] = fma_f32x2(ya, pack_f32x2(r0, r1), cnt2[0]);
        cnt2[1] = fma_f32x2(yb, pack_f32x2(r2, r3), cnt2[1]);
    }
    uint32_t qa, qb;
    cast4_e4m3(y0, y1, y2, y3, c4, qa, qb);
    float d0, d1, d2, d3;
    diff_f16x2_f32(qa, y0, y1, d0, d1);
    diff_f16x2_f32(qb, y2, y3, d2, d3);
    a43[0] = fmaf(fabsf(d0), fabsf(r0), a43[0]);
    a43[0] = fmaf(fabsf(d1), fabsf(r1), a43[0]);
    a43[1] = fmaf(fabsf(d2), fabsf(r2), a43[1]);
    a43[1] = fmaf(fabsf(d3), fabsf(r3), a43[1]);
    if (YARD) {
        // the E5M2 scale is the E4M3 scale times 2^7 (the caller sends blocks whose E5M2 exponent is capped to the
        // careful path), and y is a normal number or zero here, so fl32(x * scale5) = 128 y exactly
        const unsigned long long k128 = pack_f32x2(128.0f, 128.0f);
        float z0, z1, z2, z3;
        unpack_f32x2(mul_f32x2(ya, k128), z0, z1);
        unpack_f32x2(mul_f32x2(yb, k128), z2, z3);
        cast4_e5m2(z0, z1, z2, z3, c5, qa, qb);           // (the codes are kept only where the caller stashes them)
        diff_f16x2_f32(qa, z0, z1, d0, d1);
        diff_f16x2_f32(qb, z2, z3, d2, d3);
        // |z - q'| / |z| = |z - q'| * (1/|y|) / 128; the factor is applied once per block
        a52[0] = fmaf(fabsf(d0), fabsf(r0), a52[0]);
        a52[0] = fmaf(fabsf(d1), fabsf(r1), a52[0]);
        a52[1] = fmaf(fabsf(d2), fabsf(r2), a52[1]);
        a52[1] = fmaf(fabsf(d3), fabsf(r3), a52[1]);
    } else {
        c5 = 0u;
    }
}

struct CarefulAcc {
    float a43, a52;
    uint32_t nnz, nbig, nonfinite;
};

// Careful path for one BF16 pair: handles NaN/inf elements (stated reading: ignored by
// every count and sum, NaN -> 0x7F, +-inf -> +-largest finite) and non-zero elements whose
// scaled value leaves binary32's normal range (flushed by both formats: term 1, added by
// the caller from the counts nnz - nbig).
template <bool YARD>
__device__ __forceinline__ void convert_pair_careful(uint32_t w, float s4, float s5, CarefulAcc& A, uint32_t& c4, uint32_t& c5)
{
    const uint32_t blo = w << 16, bhi = w & 0xFFFF0000u;
    const uint32_t alo = blo & 0x7FFFFFFFu, ahi = bhi & 0x7FFFFFFFu;
    const float xlo = __uint_as_float(blo), xhi = __uint_as_float(bhi);
    const bool uselo = alo < 0x7F800000u, usehi = ahi < 0x7F800000u;
    A.nonfinite += (uselo ? 0u : 1u) + (usehi ? 0u : 1u);
    A.nnz += ((alo != 0u && uselo) ? 1u : 0u) + ((ahi != 0u && usehi) ? 1u : 0u);

    const float ylo = __fmul_rn(xlo, s4), yhi = __fmul_rn(xhi, s4);
    c4 = cvt_e4m3x2(yhi, ylo);
    float dlo, dhi;
    diff_f16x2_f32(e4m3x2_to_f16x2(c4), ylo, yhi, dlo, dhi);
    const float aylo = fabsf(ylo), ayhi = fabsf(yhi);
    const bool biglo = (aylo >= FLT_MIN) && uselo, bighi = (ayhi >= FLT_MIN) && usehi;
    const float rlo = rcp_approx(aylo), rhi = rcp_approx(ayhi);
    if (biglo) { A.a43 = fmaf(fabsf(dlo), rlo, A.a43); A.nbig++; }
    if (bighi) { A.a43 = fmaf(fabsf(dhi), rhi, A.a43); A.nbig++; }

    if (YARD) {
        const float zlo = __fmul_rn(xlo, s5), zhi = __fmul_rn(xhi, s5);
        c5 = cvt_e5m2x2(zhi, zlo);
        float elo, ehi;
        diff_f16x2_f32(e5m2x2_to_f16x2(c5), zlo, zhi, elo, ehi);
        if (biglo) A.a52 = fmaf(fabsf(elo), rlo, A.a52);
        if (bighi) A.a52 = fmaf(fabsf(ehi), rhi, A.a52);
    } else {
        c5 = 0;
    }
    if (!uselo) {
        const bool nan = (alo & 0x007F0000u) != 0u;
        const uint32_t sg = (blo >> 24) & 0x80u;
        c4 = (c4 & 0xFF00u) | (nan ? 0x7Fu : (sg | 0x7Eu));
        c5 = (c5 & 0xFF00u) | (nan ? 0x7Fu : (sg | 0x7Bu));
    }
    if (!usehi) {
        const bool nan = (ahi & 0x007F0000u) != 0u;
        const uint32_t sg = (bhi >> 24) & 0x80u;
        c4 = (c4 & 0x00FFu) | ((nan ? 0x7Fu : (sg | 0x7Eu)) << 8);
        c5 = (c5 & 0x00FFu) | ((nan ? 0x7Fu : (sg | 0x7Bu)) << 8);
    }
}

// Running sums of a thread over the elements of its block(s) that it has converted so far.
struct ConvAcc {
    float q43[2][2], q52[2][2];          // fast path: four chains per format
    unsigned long long cnt2[2];          // fast path: packed non-zero counts
    CarefulAcc A;                        // careful path
};
__device__ __forceinline__ void conv_init(ConvAcc& c)
{
#pragma unroll
    for (int k = 0; k < 2; ++k) { c.q43[k][0] = c.q43[k][1] = 0.0f; c.q52[k][0] = c.q52[k][1] = 0.0f; c.cnt2[k] = 0ull; }
    c.A.a43 = c.A.a52 = 0.0f;
    c.A.nnz = c.A.nbig = c.A.nonfinite = 0u;
}

// NCH chunks of 4 words (8 elements each) of a thread's 64 elements; chunk j0 + j belongs at byte offset
// ((j0 + j) ^ swz) * 8 of the thread's 64 code bytes (out_addr has the swizzle folded in).  The E4M3 codes go to
// the staging buffer; a block that ends up in E5M2 has them replaced afterwards (emit_e5m2_codes).
// With STASH the E5M2 codes are kept as well: chunk j0 + j's eight codes go to stash_addr ^ ((j0 + j) << 4), which
// is the place of the chunk's own (already consumed) input in the stage.
template <bool YARD, bool CAREFUL, bool STORE, int NCH, bool COUNT = true, bool STASH = false, bool LINEAR = false>
__device__ __forceinline__ void convert_chunks(const uint32_t (&w)[4 * NCH], uint32_t out_addr, int j0, uint32_t s4b, uint32_t s5b, ConvAcc& c,
                                               uint32_t stash_addr = 0u)
{
    const float s4 = __uint_as_float(s4b), s5 = __uint_as_float(s5b);
    const unsigned long long s4x2 = pack_f32x2(s4, s4), tiny2 = pack_f32x2(FLT_MIN, FLT_MIN);
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        if (CAREFUL) {
            uint32_t a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) convert_pair_careful<YARD>(w[4 * j + i], s4, s5, c.A, a[i], b[i]);
            if (STORE) sts64(out_chunk<LINEAR>(out_addr, j0 + j), make_uint2(__byte_perm(a[0], a[1], 0x5410), __byte_perm(a[2], a[3], 0x5410)));
            if (STASH) sts64(in_chunk<LINEAR>(stash_addr, j0 + j), make_uint2(__byte_perm(b[0], b[1], 0x5410), __byte_perm(b[2], b[3], 0x5410)));
        } else {
            uint32_t c4[2], c5[2];
#pragma unroll
            for (int k = 0; k < 2; ++k)
                convert_quad_fast<YARD, COUNT>(w[4 * j + 2 * k], w[4 * j + 2 * k + 1], s4x2, tiny2, c.q43[k], c.q52[k], c.cnt2, c4[k], c5[k]);
            if (STORE) sts64(out_chunk<LINEAR>(out_addr, j0 + j), make_uint2(c4[0], c4[1]));
            if (STASH) sts64(in_chunk<LINEAR>(stash_addr, j0 + j), make_uint2(c5[0], c5[1]));
        }
    }
}

// Results: e43 = the thread's sum of E4M3 terms, complete; e52 = its sum of E5M2 terms, complete; nnz; nonfinite.
// (Without COUNT the fast path reports no non-zeros: the caller has the tile's count from the pre-pass.)
template <bool YARD, bool CAREFUL, bool COUNT = true>
__device__ __forceinline__ void conv_finish(const ConvAcc& c, uint32_t s4b, uint32_t s5b, float& e43, float& e52, uint32_t& nnz, uint32_t& nonfinite)
{
    if (CAREFUL) {
        // scale4 / scale5 = 2^(e4 - e5)
        const float ratio = __uint_as_float((127u - ((s5b >> 23) - (s4b >> 23))) << 23);
        const float tiny = (float)(c.A.nnz - c.A.nbig);
        nnz = COUNT ? c.A.nnz : 0u;
        nonfinite = c.A.nonfinite;
        e43 = c.A.a43 + tiny;
        e52 = YARD ? c.A.a52 * ratio + tiny : 0.0f;
    } else {
        nnz = 0u;
        if (COUNT) {
            float c0, c1, c2, c3;
            unpack_f32x2(c.cnt2[0], c0, c1);
            unpack_f32x2(c.cnt2[1], c2, c3);
            nnz = (uint32_t)__float2int_rn((c0 + c1) + (c2 + c3));
        }
        nonfinite = 0u;
        e43 = (c.q43[0][0] + c.q43[0][1]) + (c.q43[1][0] + c.q43[1][1]);
        e52 = YARD ? ((c.q52[0][0] + c.q52[0][1]) + (c.q52[1][0] + c.q52[1][1])) * 0.0078125f : 0.0f;
    }
}

// A thread's 64 elements, held as 8 chunks of 4 words, in one go.
template <bool YARD, bool CAREFUL, bool STORE, bool COUNT = true>
__device__ __forceinline__ void convert_words(const uint32_t (&w)[32], uint32_t out_addr, uint32_t s4b, uint32_t s5b,
                                              float& e43, float& e52, uint32_t& nnz, uint32_t& nonfinite)
{
    ConvAcc c;
    conv_init(c);
    convert_chunks<YARD, CAREFUL, STORE, 8, COUNT>(w, out_addr, 0, s4b, s5b, c);
    conv_finish<YARD, CAREFUL, COUNT>(c, s4b, s5b, e43, e52, nnz, nonfinite);
}

// A block selected E5M2: the thread's 64 stashed E5M2 codes replace its E4M3 codes in the staging buffer.
template <bool LINEAR = false>
__device__ __forceinline__ void copy_stash(uint32_t stash_addr, uint32_t out_addr)
{
#pragma unroll
    for (int j = 0; j < 8; ++j) sts64(out_chunk<LINEAR>(out_addr, j), lds64(in_chunk<LINEAR>(stash_addr, j)));
}

// The E5M2 codes of a thread's 64 elements, for a block that selected E5M2 (such a block holds no
// NaN or inf): z = fl32(x * scale5), RNE-saturating cast, over the E4M3 codes in the staging buffer.
__device__ __forceinline__ void emit_e5m2_codes(const uint32_t (&w)[32], uint32_t out_addr, uint32_t s5b)
{
    const float s5 = __uint_as_float(s5b);
    const unsigned long long s5x2 = pack_f32x2(s5, s5);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        uint32_t c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t ww = w[4 * j + i];
            float zlo, zhi;
            unpack_f32x2(mul_f32x2(pack_f32x2(__uint_as_float(ww << 16), __uint_as_float(ww & 0xFFFF0000u)), s5x2), zlo, zhi);
            c[i] = cvt_e5m2x2(zhi, zlo);
        }
        sts64(out_addr ^ (j << 3), make_uint2(__byte_perm(c[0], c[1], 0x5410), __byte_perm(c[2], c[3], 0x5410)));
    }
}

// Algorithm 2 for one block with the per-block metrics (M_1 = Eq. 3, M_2 = Eq. 4, or
// Eq. 1-2 on the block alone).
template <typename T, typename REC>
__device__ __forceinline__ uint32_t decide_block(const REC& R, T e43, T e52, uint32_t nnz,
                                                 uint32_t nonfinite, uint32_t amax_bits, uint32_t minm1_bits,
                                                 uint32_t n_elems)
{
    if (nonfinite) return MOR_FMT_BF16;
    if (R.criterion == MOR_CRIT_BLOCK_VS_E5M2) {
        const bool ok = (R.flags & MOR_FLAG_STRICT_TIES) ? (e43 < e52) : (e43 <= e52);
        if (ok) return MOR_FMT_E4M3;
        if (R.n_formats == 3) {
            // max|b| < (57344 * 2^14) * min|b|, exact in binary32 (11 significant bits)
            float mnv = minnz_value(minm1_bits);
            if ((R.flags & MOR_FLAG_RANGE_MIN_INCLUDES_ZERO) && nnz < n_elems) mnv = 0.0f;
            const float amax = __uint_as_float(amax_bits << 16);
            if (amax < 939524096.0f * mnv) return MOR_FMT_E5M2;
        }
        return MOR_FMT_BF16;
    }
    if (R.criterion == MOR_CRIT_BLOCK_MEAN_REL) {
        const double err = nnz ? (double)e43 / (double)nnz : 0.0;
        return err < (double)R.threshold ? MOR_FMT_E4M3 : MOR_FMT_BF16;
    }
    return MOR_FMT_E4M3;   // tensor-level criterion: decided by the finalise kernel
}


// ------------------------------------------------------------------ tile bookkeeping ----

struct TileId {
    int ti;
    uint32_t local;
    int row0, col0, vrows, vcols;
};

__device__ __forceinline__ TileId locate_tile(const BatchParams& b, uint32_t tile)
{
    int ti = 0;
    uint32_t begin = 0;
#pragma unroll 1
    while (ti < b.n - 1 && tile >= b.tile_end[ti]) { begin = b.tile_end[ti]; ++ti; }
    const TensorRec& R = b.t[ti];
    TileId t;
    t.ti = ti;
    t.local = tile - begin;
    const uint32_t bi = t.local / R.nbc, bj = t.local - bi * R.nbc;
    t.row0 = (int)(bi * kTileRows);
    t.col0 = (int)(bj * kTileCols);
    const long long rr = R.rows - t.row0, cc = R.cols - t.col0;
    t.vrows = (int)(rr < kTileRows ? rr : kTileRows);
    t.vcols = (int)(cc < kTileCols ? cc : kTileCols);
    return t;
}

// The load warp and the store warp work once per tile, and what they need of the tensor's record sits in the
// kernel's parameter space, where a read with a computed index is slow and a chain of them (pointer, test, branch,
// next pointer) adds up to microseconds per tile.  They keep what they need in registers instead and reload it when
// the CTA moves on to another tensor; a CTA's tile numbers only grow, so the search for a tile's tensor goes forward
// from the last one.
struct RecFacts {
    uint8_t* sel;
    uint8_t* scale_e8m0;
    float* scale_f32;
    mor_block_stats_t* block_stats;
    uint32_t* keys;
    uint32_t* row_keys;
    long long cols;
    uint32_t tile_begin, nbc, nbc_blk, key_stride, flags;
    int32_t criterion, n_formats;
    float threshold;
    __device__ __forceinline__ void load(const TensorRec& R)
    {
        sel = R.sel; scale_e8m0 = R.scale_e8m0; scale_f32 = R.scale_f32; block_stats = R.block_stats;
        keys = R.keys; row_keys = R.row_keys; cols = R.cols;
        tile_begin = R.tile_begin; nbc = R.nbc; nbc_blk = R.nbc_blk; key_stride = R.key_stride; flags = R.flags;
        criterion = R.criterion; n_formats = R.n_formats; threshold = R.threshold;
    }
};

struct TileWalker {
    int ti;
    uint32_t begin, end, nbc;
    long long rows, cols;
    __device__ __forceinline__ TileWalker() : ti(-1), begin(0u), end(0u), nbc(1u), rows(0), cols(0) {}
    // moves to the tensor of `tile`; true when that is another tensor than before (or the first call)
    __device__ __forceinline__ bool seek(const BatchParams& b, uint32_t tile)
    {
        if (ti >= 0 && (tile < end || ti >= b.n - 1)) return false;
        if (ti < 0) { ti = 0; begin = 0u; end = b.tile_end[0]; }
#pragma unroll 1
        while (ti < b.n - 1 && tile >= end) { begin = end; ++ti; end = b.tile_end[ti]; }
        nbc = b.t[ti].nbc; rows = b.t[ti].rows; cols = b.t[ti].cols;
        return true;
    }
    __device__ __forceinline__ TileId id(uint32_t tile) const
    {
        TileId t;
        t.ti = ti;
        t.local = tile - begin;
        const uint32_t bi = t.local / nbc, bj = t.local - bi * nbc;
        t.row0 = (int)(bi * kTileRows);
        t.col0 = (int)(bj * kTileCols);
        const long long rr = rows - t.row0, cc = cols - t.col0;
        t.vrows = (int)(rr < kTileRows ? rr : kTileRows);
        t.vcols = (int)(cc < kTileCols ? cc : kTileCols);
        return t;
    }
};

// tiles blockIdx.x, blockIdx.x + gridDim.x, ... below total_tiles (the grid never exceeds the tile count)
__device__ __forceinline__ uint32_t my_tile_count(const MainParams& p)
{
    return (p.total_tiles - blockIdx.x + gridDim.x - 1u) / gridDim.x;
}

__device__ __forceinline__ void give_up(Control& C, uint32_t* device_status)
{
    C.abort = 1u;
    atomicOr(device_status, 1u);
}

__device__ __forceinline__ double shfl_xor_f64(double v, int o) { return __shfl_xor_sync(0xFFFFFFFFu, v, o); }

// ------------------------------------------------------------------ load warp ----

// The fast path needs every non-zero |x * scale| to be at least 2^-100 (see convert_quad_fast), no NaN/inf, and an
// E5M2 exponent that is not capped at 254 (the fast path takes scale5 = 128 scale4).
__device__ __forceinline__ bool needs_careful(bool nonfin, uint32_t minm1, uint32_t s4b)
{
    bool careful = nonfin || (s4b >> 23) > 247u;
    if (minm1 != 0xFFFFu) careful = careful || !(__fmul_rn(minnz_value(minm1), __uint_as_float(s4b)) >= 7.888609052210118e-31f);
    return careful;
}

// The load warp.  For the CTA's tile number `it`: lane 0 starts the TMA load into the tile's stage (the stage must be
// free) and the bulk copy of the tile's keys.  With PREP (the pre-pass left keys: nothing has to be scanned) the warp
// also turns the keys into what the compute threads need -- per row, quadrant or tile the scale of Algorithm 1 and
// whether the careful path is needed -- so that 256 threads need not each derive them.  The stage's barrier takes two
// arrivals: one with the byte count when the copies start, one when the tile's facts are in shared memory.
// One key per line (row or column) of the tile -> one prepared word per line: the scale bits of Algorithm 1 and a
// flag in bit 31.  MODE 0 (rows): the flag says that the line's warp -- lines 16 w .. 16 w + 15, i.e. this half of
// the lanes -- takes the careful path.  MODE 1 (columns, gathered by 16-bit loads): the same for the CTA as a whole
// (a warp's elements then come from many columns).  MODE 2 (columns, full-width path): the flag says that the
// column piece holds NaN or inf (its block then stays in BF16).  Returns whether any line needs the careful path.
template <int MODE>
__device__ __forceinline__ bool prepare_lines(const uint32_t* key_src, uint32_t m_g, int scale_mode, const uint32_t* rtab, uint32_t* dst, int lane)
{
    uint32_t key[4], sb[4], any[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) key[k] = key_src[lane + 32 * k];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const bool nonfin = (key[k] >> 31) != 0u;
        const uint32_t kk = key[k] & 0x7FFFFFFFu;
        uint32_t s5b;
        block_scale(kk >> 16, m_g, scale_mode, rtab, sb[k], s5b);
        any[k] = __ballot_sync(0xFFFFFFFFu, needs_careful(nonfin, 0xFFFFu - (kk & 0xFFFFu), sb[k]));
    }
    const bool all = (any[0] | any[1] | any[2] | any[3]) != 0u;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        bool flag = ((lane < 16 ? any[k] : any[k] >> 16) & 0xFFFFu) != 0u;
        if (MODE == 1) flag = all;
        if (MODE == 2) flag = (key[k] >> 31) != 0u;
        dst[lane + 32 * k] = sb[k] | (flag ? 0x80000000u : 0u);
    }
    return all;
}

// What a compute thread needs of the record to decide a block (Algorithm 2), kept in registers per tensor.
struct DecideFacts {
    int32_t criterion, n_formats;
    uint32_t flags;
    float threshold;
    __device__ __forceinline__ void load(const TensorRec& R) { criterion = R.criterion; n_formats = R.n_formats; flags = R.flags; threshold = R.threshold; }
};

// What the load warp keeps about the tensor it is on.
struct LoadState {
    TileWalker walk;
    RecFacts R;
    const uint32_t* col_keys2;      // rows and columns from one read: the keys of the columns' record
    uint32_t m_g, tensor_amax_bits;
    int scale_mode;
    __device__ __forceinline__ LoadState() : col_keys2(nullptr), m_g(0u), tensor_amax_bits(0u), scale_mode(0) {}
};

template <int KIND, bool PREP, bool COLFAST>
__device__ __forceinline__ void issue_tile_load(const MainParams& p, Control& C, unsigned char* in, uint32_t it, int lane, LoadState& L)
{
    const uint32_t tile = blockIdx.x + it * gridDim.x;
    if (tile >= p.total_tiles) return;
    const uint32_t s = it % kStages;
    if (L.walk.seek(p.b, tile)) {
        const TensorRec& T = p.b.t[L.walk.ti];
        L.R.load(T);
        if (PREP) {
            L.scale_mode = T.scale_mode;
            L.m_g = group_mantissa(*T.amax, L.scale_mode);
            if (KIND == KIND_TENSOR) L.tensor_amax_bits = __float_as_uint(*T.amax_slot) >> 16;
            if (KIND == KIND_DUAL) L.col_keys2 = p.b.t[L.walk.ti + 1].keys;
        }
    }
    const TileId t = L.walk.id(tile);
    const RecFacts& R = L.R;
    const uint32_t m_g = L.m_g, tensor_amax_bits = L.tensor_amax_bits;
    const int scale_mode = L.scale_mode;
    // (the full-width column paths need nothing but the prepared words: no copy of the keys)
    const uint32_t key_bytes = (R.keys == nullptr || COLFAST) ? 0u : ((KIND == KIND_CHANNEL || KIND == KIND_COLCH) ? (uint32_t)kTileRows * 4u : R.key_stride * 4u);
    const uint32_t* key_src = KIND == KIND_CHANNEL ? R.row_keys + t.row0 : KIND == KIND_COLCH ? R.row_keys + t.col0
                                                   : R.keys + (size_t)t.local * R.key_stride;
    // (test hook: for one chosen tile neither the copies nor their arrival are issued, so that the tile's barrier
    // never completes and the bounded waits of the other warps run out)
    if (lane == 0 && tile != p.test_skip_tile) {
        mbar_arrive_expect_tx(&C.full[s], kInBytes + key_bytes);
        tma_load_tile(in + s * kInBytes, &p.in_map[t.ti], t.col0, t.row0, &C.full[s]);
        if (key_bytes) bulk_load(&C.keys[s][0], key_src, key_bytes, &C.full[s]);
    }
    uint32_t tile_nnz = 0u;
    if (PREP) {
        tile_nnz = R.keys[(size_t)t.local * R.key_stride + (R.key_stride == (uint32_t)kRowKeyStride ? (uint32_t)kTileRows : 4u)];
        if (KIND == KIND_ROW128 || KIND == KIND_CHANNEL || KIND == KIND_DUAL) {          // one key per row of the tile
            prepare_lines<0>(key_src, m_g, scale_mode, C.rtab, &C.prep[s][0], lane);
            if (KIND == KIND_DUAL) {
                // ... and one per column, from the columns' record (same tiles, same group amax)
                const bool any = prepare_lines<2>(L.col_keys2 + (size_t)t.local * kRowKeyStride, m_g, scale_mode, C.rtab, &C.prep2[s][0], lane);
                if (lane == 0) C.colflag[s] = any ? 1u : 0u;
            }
        } else if (KIND == KIND_COL128 || KIND == KIND_COLCH) {                            // one key per column of the tile
            if (COLFAST) {
                const bool any = prepare_lines<2>(key_src, m_g, scale_mode, C.rtab, &C.prep[s][0], lane);
                if (lane == 0) C.colflag[s] = any ? 1u : 0u;
            } else {
                prepare_lines<1>(key_src, m_g, scale_mode, C.rtab, &C.prep[s][0], lane);
            }
        } else {
            // one key per tile, or one per quadrant (lanes 0..3; the other lanes repeat lane 0's work)
            const uint32_t q = KIND == KIND_BLK64 ? (uint32_t)(lane & 3) : 0u;
            const uint32_t key = key_src[q];
            const bool nonfin = (key >> 31) != 0u;
            const uint32_t kk = key & 0x7FFFFFFFu;
            uint32_t s4b, s5b;
            block_scale(KIND == KIND_TENSOR ? tensor_amax_bits : kk >> 16, m_g, scale_mode, C.rtab, s4b, s5b);
            bool careful = needs_careful(nonfin, 0xFFFFu - (kk & 0xFFFFu), s4b);
            // 64x64: a warp covers both column halves of its rows, and takes the careful path as a whole
            if (KIND == KIND_BLK64) {
                const int other = __shfl_xor_sync(0xFFFFFFFFu, (int)careful, 1);   // (every lane takes part: no short-circuit)
                careful = careful || other != 0;
            }
            if (lane < (KIND == KIND_BLK64 ? 4 : 1)) C.prep[s][lane] = s4b | (careful ? 0x80000000u : 0u);
        }
    }
    if (lane == 0) {
        TileMeta m;
        m.ti = t.ti; m.local = t.local; m.row0 = t.row0; m.col0 = t.col0; m.vrows = t.vrows; m.vcols = t.vcols;
        m.blk_base = (uint32_t)t.row0 * R.nbc + (uint32_t)(t.col0 / kTileCols);
        if (KIND == KIND_COL128) m.blk_base = (uint32_t)(t.row0 / kTileRows) * (uint32_t)R.cols + (uint32_t)t.col0;
        if (KIND == KIND_CHANNEL) m.blk_base = t.col0 == 0 ? (uint32_t)t.row0 : 0xFFFFFFFFu;   // first tile of its rows: writes the row scales
        if (KIND == KIND_COLCH) m.blk_base = t.row0 == 0 ? (uint32_t)t.col0 : 0xFFFFFFFFu;     // first tile of its columns: the column scales
        m.nnz = tile_nnz;
        C.meta[s] = m;
        C.issued = it + 1;
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&C.full[s]);             // the tile's facts are in place (release)
}

template <int KIND, bool PREP, bool COLFAST>
__device__ __forceinline__ void load_warp(const MainParams& p, Control& C, unsigned char* in, int lane)
{
    LoadState L;
    for (uint32_t it = 0; it < (uint32_t)kStages; ++it) issue_tile_load<KIND, PREP, COLFAST>(p, C, in, it, lane, L);
    const uint32_t n_it = my_tile_count(p);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        stage_free_sync(it % kStages);                  // sleeps until every compute thread has its copy
        if (!__any_sync(0xFFFFFFFFu, C.abort != 0u))
            issue_tile_load<KIND, PREP, COLFAST>(p, C, in, it + kStages, lane, L);
    }
    if (lane == 0 && C.abort) {
        // copies that may still be in flight must land (or be given up on) before the CTA goes
        const uint32_t issued = C.issued;
        for (uint32_t k = 0; k < (uint32_t)kStages && k < issued; ++k) {
            const uint32_t it = issued - 1 - k;
            mbar_wait(&C.full[it % kStages], (it / kStages) & 1u, nullptr, p.wait_cycles);
        }
    }
}

// ------------------------------------------------------------------ store warp ----

template <int KIND, bool THREE, bool STORE, bool EXTRA, bool COLFAST = false>
__device__ __forceinline__ void store_warp(const MainParams& p, Control& C, unsigned char* out, Partial* __restrict__ partials,
                                           int lane)
{
    constexpr bool kLineBlocks = KIND == KIND_ROW128 || KIND == KIND_COL128 || KIND == KIND_DUAL;   // 128 one-line blocks per tile
    constexpr int kEntries = kLineBlocks ? kTileRows : kThreads;
    // 1x128 / 128x1 blocks without the optional outputs, where the compute threads decide (three formats, or the
    // 16-bit column gather): the metadata is written here, from the entries
    constexpr bool kMetaHere = (KIND == KIND_ROW128 || KIND == KIND_COL128) && !EXTRA && !COLFAST;
    bool stores_pending = false;
    TileWalker walk;
    RecFacts F0, F1;                                     // F1: the columns' record of a rows-and-columns pair
    if (KIND == KIND_DUAL) F1 = RecFacts();
#pragma unroll 1
    for (uint32_t it = 0;; ++it) {
        // both directions from one read: two conversions per tile, rows (record ti) then columns (record ti + 1)
        const uint32_t tile = blockIdx.x + (KIND == KIND_DUAL ? it >> 1 : it) * gridDim.x;
        if (tile >= p.total_tiles) break;
        const uint32_t b = it & 1u, n = it >> 1;
        const bool columns = KIND == KIND_COL128 || KIND == KIND_COLCH || (KIND == KIND_DUAL && (it & 1u));
        if (walk.seek(p.b, tile)) {                      // (before the wait: off the critical path)
            F0.load(p.b.t[walk.ti]);
            if (KIND == KIND_DUAL) F1.load(p.b.t[walk.ti + 1]);
        }
        TileId t = walk.id(tile);
        if (KIND == KIND_DUAL && columns) t.ti += 1;
        const RecFacts R = (KIND == KIND_DUAL && columns) ? F1 : F0;     // (a copy: both stay in registers)
        constexpr bool kTileBlocks = KIND == KIND_BLK128 || KIND == KIND_BLK64;
        // the decision is handed back on every tile of a launch whose compute threads may need it (three formats:
        // E5M2 codes; EXTRA: a BF16 copy or a fake-quantised output for some tensor of the launch), whether this
        // tensor's threads wait for it or not: the barrier's phase then follows the tile count
        // (128x128 blocks, three formats, plain outputs: the compute threads have decided and the codes are final)
        constexpr bool kSelfDecided = KIND == KIND_BLK128 && THREE && STORE && !EXTRA;
        constexpr bool need_dec = kTileBlocks && (THREE || EXTRA) && !kSelfDecided;
        const bool codes_wait = STORE && kTileBlocks && THREE && !kSelfDecided;
        out_full_sync(b);                                // sleeps until every compute thread has arrived
        if (!__any_sync(0xFFFFFFFFu, C.abort != 0u)) {
            if (STORE && !codes_wait && lane == 0) {
                // the codes are complete: start the tile store at once, it runs while the sums are formed
                // (sub-column blocks: the staging tile and the code tensor are transposed)
                tma_store_tile(&p.out_map[t.ti], columns ? t.row0 : t.col0, columns ? t.col0 : t.row0, out + b * kOutBytes);
                bulk_commit();
                stores_pending = true;
            }

            if (COLFAST && KIND == KIND_ROW128) {
                // 1x128 blocks whose compute threads hand over their sums and the row's scale (entry of thread
                // 2 row + h: {E4M3 sum, E5M2 sum, non-zeros | non-finites << 16, scale bits}): this lane adds the two
                // halves of rows lane, lane + 32, ..., decides their blocks and writes their metadata.
                const uint32_t ea = smem_addr(&C.entry[b][0]) + (uint32_t)lane * 32u;
                float f43 = 0.0f, f52 = 0.0f;
                uint32_t n4 = 0, n5 = 0, nb = 0, tnnz = 0, tnonf = 0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint4 e0 = lds128(ea + (uint32_t)k * 1024u), e1 = lds128(ea + (uint32_t)k * 1024u + 16u);
                    const float e43 = __uint_as_float(e0.x) + __uint_as_float(e1.x), e52 = __uint_as_float(e0.y) + __uint_as_float(e1.y);
                    const uint32_t nz = e0.z + e1.z;
                    f43 += e43; f52 += e52; tnnz += nz & 0xFFFFu; tnonf += nz >> 16;
                    const int row = lane + 32 * k;
                    if (row < t.vrows) {
                        const uint32_t bsel = decide_block(R, e43, e52, 0u, nz >> 16, 0u, 0xFFFFu, (uint32_t)t.vcols);
                        const uint32_t blk = (uint32_t)(t.row0 + row) * R.nbc + (uint32_t)(t.col0 / kTileCols);
                        if (R.sel) R.sel[blk] = (uint8_t)bsel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(e0.w >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(e0.w);
                        n4 += bsel == MOR_FMT_E4M3; n5 += bsel == MOR_FMT_E5M2; nb += bsel == MOR_FMT_BF16;
                    }
                }
                double s43 = (double)f43, s52 = (double)f52;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) { s43 += shfl_xor_f64(s43, o); s52 += shfl_xor_f64(s52, o); }
                n4 = __reduce_add_sync(0xFFFFFFFFu, n4);
                n5 = __reduce_add_sync(0xFFFFFFFFu, n5);
                nb = __reduce_add_sync(0xFFFFFFFFu, nb);
                tnnz = __reduce_add_sync(0xFFFFFFFFu, tnnz);
                tnonf = __reduce_add_sync(0xFFFFFFFFu, tnonf);
                if (lane == 0) {
                    Partial P;
                    P.sum43 = s43; P.sum52 = s52; P.nnz = tnnz; P.nonfinite = tnonf;
                    P.n_e4m3 = n4; P.n_e5m2 = n5; P.n_bf16 = nb; P.min_nz_bits = 0xFFFFu;
                    partials[R.tile_begin + t.local] = P;
                }
            } else if (COLFAST && (KIND != KIND_DUAL || columns)) {
                // Blocks along the columns, handed over by cols_fast_tile: this lane takes columns 4 lane ..
                // 4 lane + 3; a column's sums come in four parts (row groups), added in the order of the parts.
                const uint32_t ea = smem_addr(&C.entry[b][0]) + (uint32_t)lane * 32u;
                float e43[4] = {0.0f, 0.0f, 0.0f, 0.0f}, e52[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int part = 0; part < 4; ++part) {
                    const uint4 v0 = lds128(ea + (uint32_t)part * 1024u), v1 = lds128(ea + (uint32_t)part * 1024u + 16u);
                    e43[0] += __uint_as_float(v0.x); e52[0] += __uint_as_float(v0.y); e43[1] += __uint_as_float(v0.z); e52[1] += __uint_as_float(v0.w);
                    e43[2] += __uint_as_float(v1.x); e52[2] += __uint_as_float(v1.y); e43[3] += __uint_as_float(v1.z); e52[3] += __uint_as_float(v1.w);
                }
                const uint4 sc4 = *reinterpret_cast<const uint4*>(&C.colscale[b][4 * lane]);
                const uint32_t sc[4] = {sc4.x, sc4.y, sc4.z, sc4.w};
                uint32_t n4 = 0, n5 = 0, nb = 0;
                const uint32_t blk0 = (uint32_t)(t.row0 / kTileRows) * (uint32_t)R.cols + (uint32_t)t.col0 + 4u * (uint32_t)lane;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (4 * lane + c >= t.vcols) continue;
                    const uint32_t s4b = sc[c] & 0x7FFFFFFFu;
                    if (KIND == KIND_COLCH) {
                        // per-channel: a column is one block over all tile rows; its decision is the tensor's (finalise
                        // kernel); the first tile row writes the column's scale
                        if (t.row0 == 0) {
                            const uint32_t blk = (uint32_t)t.col0 + 4u * (uint32_t)lane + (uint32_t)c;
                            if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(s4b >> 23);
                            if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(s4b);
                        }
                        continue;
                    }
                    const uint32_t bsel = decide_block(R, e43[c], e52[c], 0u, sc[c] >> 31, 0u, 0xFFFFu, (uint32_t)t.vrows);
                    if (R.sel) R.sel[blk0 + c] = (uint8_t)bsel;
                    if (R.scale_e8m0) R.scale_e8m0[blk0 + c] = (uint8_t)(s4b >> 23);
                    if (R.scale_f32) R.scale_f32[blk0 + c] = __uint_as_float(s4b);
                    n4 += bsel == MOR_FMT_E4M3; n5 += bsel == MOR_FMT_E5M2; nb += bsel == MOR_FMT_BF16;
                }
                double s43 = (double)((e43[0] + e43[1]) + (e43[2] + e43[3])), s52 = (double)((e52[0] + e52[1]) + (e52[2] + e52[3]));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) { s43 += shfl_xor_f64(s43, o); s52 += shfl_xor_f64(s52, o); }
                n4 = __reduce_add_sync(0xFFFFFFFFu, n4);
                n5 = __reduce_add_sync(0xFFFFFFFFu, n5);
                nb = __reduce_add_sync(0xFFFFFFFFu, nb);
                const uint32_t tnonf = __reduce_add_sync(0xFFFFFFFFu, lane < kComputeWarps ? C.colnonf[b][lane] : 0u);
                if (lane == 0) {
                    Partial P;
                    P.sum43 = s43; P.sum52 = s52; P.nnz = C.colnnz[b]; P.nonfinite = tnonf;
                    P.n_e4m3 = n4; P.n_e5m2 = n5; P.n_bf16 = nb; P.min_nz_bits = 0xFFFFu;
                    partials[R.tile_begin + t.local] = P;
                }
            } else {
            // the threads' sums in a fixed order: lane-strided in binary32, then a butterfly in double.
            // With 64x64 blocks a lane's entries belong to one column half (lane & 1) and to the upper
            // (k < 4) or lower rows: two sets of sums per lane, combined over the lanes of equal parity.
            constexpr int NR = KIND == KIND_BLK64 ? 2 : 1;
            float f43[NR], f52[NR];
            uint32_t nnz[NR], nonf[NR], n4 = 0, n5 = 0, nb = 0, mn = 0xFFFFu;
#pragma unroll
            for (int r = 0; r < NR; ++r) { f43[r] = 0.0f; f52[r] = 0.0f; nnz[r] = 0; nonf[r] = 0; }
#pragma unroll
            for (int k = 0; k < kEntries / 32; ++k) {
                const Entry e = C.entry[b][lane + 32 * k];
                const int r = (NR == 2 && k >= 4) ? 1 : 0;
                f43[r] += e.e43;
                f52[r] += e.e52;
                nnz[r] += e.nnz_nonf & 0xFFFFu;
                nonf[r] += e.nnz_nonf >> 16;
                if (kLineBlocks) {
                    const uint32_t sel = e.sel_min & 0xFFFFu;
                    n4 += sel == MOR_FMT_E4M3; n5 += sel == MOR_FMT_E5M2; nb += sel == MOR_FMT_BF16;
                    if (kMetaHere && sel != kSelNone) {
                        // the block's selection and scale, left by the line's first thread
                        const uint32_t line = (uint32_t)(lane + 32 * k), sb = C.colscale[b][line];
                        const uint32_t blk = KIND == KIND_COL128 ? (uint32_t)(t.row0 / kTileRows) * (uint32_t)R.cols + (uint32_t)t.col0 + line
                                                                 : ((uint32_t)t.row0 + line) * R.nbc + (uint32_t)(t.col0 / kTileCols);
                        if (R.sel) R.sel[blk] = (uint8_t)sel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(sb >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(sb);
                    }
                }
                mn = min(mn, e.sel_min >> 16);
            }
            double s43[NR], s52[NR];
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                s43[r] = (double)f43[r]; s52[r] = (double)f52[r];
#pragma unroll
                for (int o = 16; o > (NR == 2 ? 1 : 0); o >>= 1) {
                    s43[r] += shfl_xor_f64(s43[r], o); s52[r] += shfl_xor_f64(s52[r], o);
                    if (NR == 2) { nnz[r] += __shfl_xor_sync(0xFFFFFFFFu, nnz[r], o); nonf[r] += __shfl_xor_sync(0xFFFFFFFFu, nonf[r], o); }
                }
                if (NR == 1) { nnz[r] = __reduce_add_sync(0xFFFFFFFFu, nnz[r]); nonf[r] = __reduce_add_sync(0xFFFFFFFFu, nonf[r]); }
            }
            mn = __reduce_min_sync(0xFFFFFFFFu, mn);
            if (kLineBlocks) {
                n4 = __reduce_add_sync(0xFFFFFFFFu, n4);
                n5 = __reduce_add_sync(0xFFFFFFFFu, n5);
                nb = __reduce_add_sync(0xFFFFFFFFu, nb);
            }

            // tile totals (64x64: the four blocks in the order q = 0..3, taken from lanes 0 and 1)
            double t43 = s43[0], t52 = s52[0];
            uint32_t tnnz = nnz[0], tnonf = nonf[0];
            if (NR == 2) {
                const double a1 = __shfl_sync(0xFFFFFFFFu, s43[0], 1), b1 = __shfl_sync(0xFFFFFFFFu, s52[0], 1);
                const double a3 = __shfl_sync(0xFFFFFFFFu, s43[NR - 1], 1), b3 = __shfl_sync(0xFFFFFFFFu, s52[NR - 1], 1);
                t43 = ((s43[0] + a1) + s43[NR - 1]) + a3;
                t52 = ((s52[0] + b1) + s52[NR - 1]) + b3;
                tnnz = nnz[0] + nnz[NR - 1]; tnnz += __shfl_xor_sync(0xFFFFFFFFu, tnnz, 1);
                tnonf = nonf[0] + nonf[NR - 1]; tnonf += __shfl_xor_sync(0xFFFFFFFFu, tnonf, 1);
            }

            if (kTileBlocks && lane < (NR == 2 ? 2 : 1)) {
                // Algorithm 2 for the tile's block(s): lane 0 decides block(s) of the left column half, lane 1 of the right
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                    const int q = NR == 2 ? 2 * r + lane : 0;
                    const int br = NR == 2 ? 64 : 128;
                    const int vr = min(br, t.vrows - (NR == 2 ? 64 * r : 0)), vc = min(br, t.vcols - (NR == 2 ? 64 * lane : 0));
                    uint32_t bsel = kSelNone;
                    if (vr > 0 && vc > 0) {
                        const uint32_t key = C.tile_key[b][q], s4b = C.tile_scale[b][q][0], s5b = C.tile_scale[b][q][1];
                        const uint32_t amax_bits = key >> 16, minm1 = 0xFFFFu - (key & 0xFFFFu);
                        bsel = kSelfDecided ? C.dec_sel[b][0] : decide_block(R, s43[r], s52[r], nnz[r], nonf[r], amax_bits, minm1, (uint32_t)(vr * vc));
                        const uint32_t blk = NR == 2 ? (uint32_t)(t.row0 / 64 + r) * R.nbc_blk + (uint32_t)(t.col0 / 64 + lane) : t.local;
                        const uint32_t sb = (bsel == MOR_FMT_E5M2) ? s5b : s4b;
                        if (R.sel) R.sel[blk] = (uint8_t)bsel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(sb >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(sb);
                        if (R.block_stats) {
                            mor_block_stats_t bs;
                            bs.amax = __uint_as_float(amax_bits << 16);
                            bs.min_abs_nz = THREE ? minnz_value(minm1) : __uint_as_float(0x7F800000u);
                            bs.nnz = nnz[r]; bs.n_nonfinite = nonf[r];
                            bs.sum_rel_e4m3 = (float)s43[r]; bs.sum_rel_e5m2 = (float)s52[r];
                            R.block_stats[blk] = bs;
                        }
                    }
                    if (need_dec) C.dec_sel[b][q] = bsel;
                    n4 += bsel == MOR_FMT_E4M3; n5 += bsel == MOR_FMT_E5M2; nb += bsel == MOR_FMT_BF16;
                }
            }
            if (NR == 2) {
                n4 += __shfl_xor_sync(0xFFFFFFFFu, n4, 1); n5 += __shfl_xor_sync(0xFFFFFFFFu, n5, 1); nb += __shfl_xor_sync(0xFFFFFFFFu, nb, 1);
            }
            if (need_dec) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&C.dec_full[b]);      // compute threads may be waiting for the decision
            }
            if (lane == 0) {
                Partial P;
                P.sum43 = t43; P.sum52 = t52; P.nnz = tnnz; P.nonfinite = tnonf;
                P.n_e4m3 = n4; P.n_e5m2 = n5; P.n_bf16 = nb; P.min_nz_bits = mn;
                partials[R.tile_begin + t.local] = P;
            }
            }
            if (codes_wait) {
                // three formats, 128x128 blocks: the compute threads put the chosen format's codes in place
                // after the decision
                bool ok = mbar_wait(&C.codes_full[b], n & 1u, &C.abort, p.wait_cycles);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok && lane == 0) give_up(C, p.device_status);
                if (ok && lane == 0) {
                    tma_store_tile(&p.out_map[t.ti], t.col0, t.row0, out + b * kOutBytes);
                    bulk_commit();
                    stores_pending = true;
                }
            }
            if (STORE && lane == 0 && stores_pending) bulk_wait_read<0>();   // the staging buffer may be overwritten from here on
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&C.out_empty[b]);
    }
    if (lane == 0 && stores_pending) bulk_wait_all();
}

// ------------------------------------------------------------------ compute warps ----

// copy of every block that stays in BF16, straight from the registers
__device__ __forceinline__ void write_fallback(const TensorRec& R, const uint32_t (&w)[32], const TileMeta& m, int row, int h, int swz)
{
    if (row >= m.vrows) return;
    uint16_t* dst_row = R.fallback + (long long)(m.row0 + row) * R.ld + m.col0 + h * 64;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = (j ^ swz) * 8;                      // first of the chunk's 8 elements within the thread's 64
        const int left = m.vcols - (h * 64 + c);
        if (left >= 8) {
            *reinterpret_cast<uint4*>(dst_row + c) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (i < left) dst_row[c + i] = (uint16_t)(w[4 * j + (i >> 1)] >> (16 * (i & 1)));
        }
    }
}

// Fake quantisation of a thread's 64 elements (Section 4: quantise, dequantise, de-scale; BF16 out): the FP8
// value of format `fmt` divided by the scale in one binary32 division, rounded to BF16; a block that stays
// in BF16 and NaN/inf elements are copied.  Straight from the registers, like the fallback copy.
__device__ __noinline__ void fake_quant_chunk(uint4 v, uint32_t fmt, float s, uint32_t (&o)[4])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t ww = w[i];
        const float xlo = __uint_as_float(ww << 16), xhi = __uint_as_float(ww & 0xFFFF0000u);
        const float ylo = __fmul_rn(xlo, s), yhi = __fmul_rn(xhi, s);
        const uint32_t q = fmt == MOR_FMT_E5M2 ? e5m2x2_to_f16x2(cvt_e5m2x2(yhi, ylo)) : e4m3x2_to_f16x2(cvt_e4m3x2(yhi, ylo));
        const float2 qf = __half22float2(*reinterpret_cast<const __half2*>(&q));
        const float tlo = __fdiv_rn(qf.x, s), thi = __fdiv_rn(qf.y, s);
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(thi), "f"(tlo));
        if ((ww & 0x7F80u) == 0x7F80u) r = (r & 0xFFFF0000u) | (ww & 0xFFFFu);             // NaN / inf: as they are
        if ((ww & 0x7F800000u) == 0x7F800000u) r = (r & 0xFFFFu) | (ww & 0xFFFF0000u);
        o[i] = r;
    }
}
__device__ __forceinline__ void write_fake_quant(const TensorRec& R, const uint32_t (&w)[32], const TileMeta& m, int row, int h, int swz,
                                                 uint32_t fmt, uint32_t s4b, uint32_t s5b)
{
    if (row >= m.vrows) return;
    const float s = __uint_as_float(fmt == MOR_FMT_E5M2 ? s5b : s4b);
    uint16_t* dst_row = R.fake_quant + (long long)(m.row0 + row) * R.ld + m.col0 + h * 64;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        const int c = (j ^ swz) * 8;
        const int left = m.vcols - (h * 64 + c);
        if (left <= 0) continue;
        // chunk j of the registers, selected without indexing them dynamically
        uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
        for (int k = 1; k < 8; ++k)
            if (j == k) v = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
        uint32_t o[4] = {v.x, v.y, v.z, v.w};
        if (fmt != MOR_FMT_BF16) fake_quant_chunk(v, fmt, s, o);
        if (left >= 8) {
            *reinterpret_cast<uint4*>(dst_row + c) = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            for (int i = 0; i < left; ++i) dst_row[c + i] = (uint16_t)(o[i >> 1] >> (16 * (i & 1)));
        }
    }
}

// Sub-column blocks: 64 elements down a column of the row-major tile, two rows per word, chunk by chunk (a chunk
// is 8 rows): chunk j of the registers holds rows 8 (j ^ swz) .. + 7 (the order in which the code chunks are stored),
// so one address is formed per chunk and the eight 16-bit loads of a chunk use constant offsets from it.
__device__ __forceinline__ void load_column(uint32_t a, int swz, uint32_t (&w)[32])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t cb = a + ((uint32_t)(j ^ swz) << 11);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t lo, hi;
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo) : "r"(cb + (uint32_t)(2 * k * 256)));
            asm volatile("ld.shared.u16 %0, [%1];" : "=r"(hi) : "r"(cb + (uint32_t)((2 * k + 1) * 256)));
            w[4 * j + k] = __byte_perm(lo, hi, 0x5410);
        }
    }
}

// The BF16 outputs of a thread that holds a column piece (sub-column blocks): element by element down the column
// (2-byte stores; the 16 columns of a warp make 32-byte runs).  `fq`: fake quantisation with format `fmt` and scale
// `s` (BF16-selected blocks and NaN/inf elements are copied); otherwise the plain copy of a rejected block.
__device__ __noinline__ void write_column(uint16_t* dst, long long ld, const TileMeta& m, int col, int h, int swz,
                                          const uint32_t (&w)[32], bool fq, uint32_t fmt, float s)
{
    if (col >= m.vcols) return;
    uint16_t* base = dst + (long long)m.row0 * ld + m.col0 + col;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
        for (int k = 1; k < 8; ++k)
            if (j == k) v = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
        uint32_t o[4] = {v.x, v.y, v.z, v.w};
        if (fq && fmt != MOR_FMT_BF16) fake_quant_chunk(v, fmt, s, o);
        const int r0 = 64 * h + 8 * (j ^ swz);             // first of the chunk's 8 rows within the tile
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (r0 + i < m.vrows) base[(long long)(r0 + i) * ld] = (uint16_t)(o[i >> 1] >> (16 * (i & 1)));
    }
}

template <int KIND, bool YARD, bool THREE, bool STORE, bool SCAN, bool EXTRA>
__device__ __forceinline__ void compute_warps(const MainParams& p, Control& C, unsigned char* in, unsigned char* out, int tid)
{
    const int lane = tid & 31, warp = tid >> 5;
    const int row = tid >> 1, h = tid & 1;
    // Chunk order: thread (row, h) holds the 16-byte chunk c of its 128 bytes as chunk c ^ swz.  With
    // this choice the 8 threads of a 128-bit load phase and the 16 threads of a 64-bit store phase
    // touch distinct banks.
    // Sub-column blocks read 16-bit pieces down a column; all rows of a column share a bank, so there
    // the two columns that share a 32-bit word get the same order (they then read the same word) at the
    // price of a two-way conflict on the stores.
    constexpr bool kColumns = KIND == KIND_COL128 || KIND == KIND_COLCH;   // the thread holds a column piece, codes are stored transposed
    const int swz = kColumns ? ((row >> 1) & 3) ^ (h << 2) : (row & 7) ^ (h << 2);
    constexpr bool kLineBlocks = KIND == KIND_ROW128 || KIND == KIND_COL128;
    const int q = KIND == KIND_BLK64 ? ((row >> 6) << 1) | h : 0;     // which of the tile's blocks this thread's elements belong to
    // 128x128 blocks and the per-tensor block without BF16 outputs: any 64 elements of the tile will do for a thread,
    // so it takes chunk tid & 15 of rows (tid >> 4) + 16 j and every address is a base plus a constant
    constexpr bool kLinear = (KIND == KIND_BLK128 || KIND == KIND_TENSOR) && !EXTRA;
    const uint32_t in_off = kLinear ? (uint32_t)((tid >> 4) * 256 + (tid & 15) * 16) : (uint32_t)(row * 256 + h * 128 + (swz << 4));
    const uint32_t out_off = kLinear ? (uint32_t)((tid >> 4) * 128 + (tid & 15) * 8) : (uint32_t)(row * 128 + h * 64 + (swz << 3));
    const uint32_t in_base = smem_addr(in), out_base = smem_addr(out), entry_base = smem_addr(&C.entry[0][0]);

    // what changes only with the tensor, kept in registers
    int cur_ti = -1;
    uint32_t m_g = 0;            // Algorithm 1, group part
    int scale_mode = 0;
    bool has_fallback = false;
    bool has_fq = false, fq_e4m3 = false;   // fake-quantised output wanted; ... with E4M3 values whatever the block's selection
    float* amax_slot = nullptr;              // scanning variants: where to gather the tensor amax (nullptr: nowhere)
    const uint32_t meta_base = smem_addr(&C.meta[0]), keys_base = smem_addr(&C.keys[0][0]), prep_base = smem_addr(&C.prep[0][0]);
    bool dead = false;       // a wait has run out somewhere in the CTA: keep the arrivals, skip the rest
    DecideFacts D;           // line blocks: what the block's decision needs of the record, reloaded per tensor
    int d_ti = -1;
    // line blocks without the optional outputs: the store warp writes the blocks' metadata (from the entries and the
    // scale that the row's first thread leaves it); with them everything about a block is written from here
    constexpr bool kRowFast = KIND == KIND_ROW128 && !EXTRA && !THREE;
    constexpr bool kMetaInStore = kLineBlocks && !EXTRA && !kRowFast;
    // 128x128 blocks, three formats, plain outputs: the compute threads settle the block's format among themselves
    // (warp sums, one barrier, the same fixed-order total in every thread) and put the chosen codes in place before
    // they hand the tile to the store warp -- no round trip through that warp
    constexpr bool kSelfDecide = KIND == KIND_BLK128 && THREE && STORE && !EXTRA;
    const uint32_t n_it = my_tile_count(p);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        const uint32_t s = it % kStages, b = it & 1u, n2 = it >> 1;

        if (!dead) {
            bool ok = mbar_wait(&C.full[s], (it / kStages) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
        }
        TileMeta m;
        {
            const uint4 q = lds128(meta_base + s * (uint32_t)sizeof(TileMeta));
            m.ti = dead ? 0 : (int32_t)q.x; m.vrows = (int32_t)q.y; m.vcols = (int32_t)q.z; m.blk_base = q.w;
            m.local = 0; m.row0 = 0; m.col0 = 0; m.nnz = 0;
        }
        // What the thread has to find out itself.  With keys from the pre-pass (no SCAN) the load warp has prepared the
        // block's scale; the key itself (amax, smallest non-zero) is then needed only for Eq. 4 and for statistics,
        // and the non-zeros are counted per thread only where a per-block count is wanted (EXTRA) -- otherwise the
        // tile's count comes from the pre-pass and travels in thread 0's entry.
        constexpr bool kNeedKey = SCAN || THREE || EXTRA;
        constexpr bool kCount = SCAN || EXTRA;
        // Two ways through a tile.  Streaming (no BF16 output): the thread converts its 64 elements in two halves
        // straight from the stage, 16 registers of data at a time, and hands the stage back after the second half's
        // loads; where no pre-pass ran it first scans them, also from the stage.  Otherwise the 64 elements are
        // copied to registers first (the stage goes back at once) and serve the scan, the conversion and whatever
        // follows the block's decision (BF16 copy, fake quantisation).
#ifdef MOR_NO_STREAM
        constexpr bool kStream = false;
#else
        constexpr bool kStream = !EXTRA && !kColumns;
#endif
        // Three formats: the E5M2 codes of every element are kept in the thread's part of the stage until the block's
        // decision is known (a copy then puts them in place); the stage goes back after that.
        constexpr bool kStash = kStream && THREE && STORE;
        uint32_t w[32];
        if (kStream) {
        } else if (kColumns) {
            // sub-column blocks: this thread takes column `row` of the tile, rows 64 h .. 64 h + 63, two rows
            // per word, so that everything after this point works on the block as on a row piece
            const uint32_t a = in_base + s * kInBytes + (uint32_t)(h * 64 * 256 + row * 2);
            load_column(a, swz, w);
        } else {
            const uint32_t a = in_base + s * kInBytes + in_off;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint4 v = lds128(a ^ (j << 4));
                w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
            }
        }
        const TensorRec& R = p.b.t[m.ti];
        if (((kLineBlocks && !kRowFast) || kSelfDecide) && m.ti != d_ti) { d_ti = m.ti; D.load(R); }
        if ((SCAN || EXTRA) && m.ti != cur_ti) {
            cur_ti = m.ti;
            has_fallback = EXTRA && STORE && R.fallback != nullptr;
            has_fq = EXTRA && STORE && R.fake_quant != nullptr;
            fq_e4m3 = KIND == KIND_TENSOR || KIND == KIND_CHANNEL || KIND == KIND_COLCH || R.criterion == MOR_CRIT_TENSOR_MEAN_REL;
            if (SCAN) {
                scale_mode = R.scale_mode;
                if (!dead) m_g = group_mantissa(*R.amax, scale_mode);
                // no pre-pass ran and the caller gave no amax: the tensor amax that the summary reports is gathered here
                amax_slot = (!(R.flags & kFlagAmaxFinal) && R.amax == R.amax_slot) ? R.amax_slot : nullptr;
            }
        }
        if (EXTRA || (!kCount && tid == 0)) {          // the tile's position (BF16 outputs) and its non-zero count
            const uint4 q = lds128(meta_base + s * (uint32_t)sizeof(TileMeta) + 16u);
            m.local = q.x; m.row0 = (int32_t)q.y; m.col0 = (int32_t)q.z; m.nnz = q.w;
        }
        uint32_t key = 0u, prep = 0u;
        if (!SCAN) {
            // the pre-pass left the block's (1x128) or the tile's amax and smallest non-zero; the load warp made the scale
            const uint32_t e = (KIND == KIND_ROW128 || KIND == KIND_COL128 || KIND == KIND_CHANNEL || KIND == KIND_COLCH) ? (uint32_t)row * 4u : (uint32_t)q * 4u;
            if (kNeedKey) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(key) : "r"(keys_base + s * (uint32_t)(kRowKeyStride * 4) + e));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(prep) : "r"(prep_base + s * (uint32_t)(kTileRows * 4) + e));
        }
        if (!kStream) stage_free_arrive(s);             // this thread's copy of the stage is in registers

        // ---- block amax and smallest non-zero (Algorithm 1; Eq. 4) ----
        bool nonfin = false;
        if (!SCAN) {
            key &= 0x7FFFFFFFu;                         // (the flag for NaN/inf is part of the prepared word)
        } else if (kLineBlocks) {
            key = kStream ? scan_stage<kLinear>(in_base + s * kInBytes + in_off) : scan_words(w);
            key = key_max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 1));
            nonfin = __any_sync(0xFFFFFFFFu, (key >> 16) >= kBf16Inf);            // warp-uniform
            if (nonfin) {
                key = kStream ? scan_stage_finite<kLinear>(in_base + s * kInBytes + in_off) : scan_words_finite(w);
                key = key_max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 1));
            }
            // no pre-pass ran: the tensor amax that the summary reports is gathered here (non-negative binary32
            // patterns order like the values)
            if (amax_slot != nullptr) {
                const uint32_t wamax = __reduce_max_sync(0xFFFFFFFFu, key >> 16);
                raise_amax(amax_slot, wamax, lane == 0 && !dead);
            }
        } else if (KIND == KIND_BLK128 || KIND == KIND_BLK64) {
            key = kStream ? scan_stage<kLinear>(in_base + s * kInBytes + in_off) : scan_words(w);
            uint32_t tile_amax = 0u;
#pragma unroll 1
            for (int pass = 0; pass < 2; ++pass) {
                // the warps exchange their keys; with 64x64 blocks a warp has one per column half (lane parity)
                const uint32_t part = KIND == KIND_BLK64 ? (h ? 0xAAAAAAAAu : 0x55555555u) : 0xFFFFFFFFu;
                const uint32_t hi = __reduce_max_sync(part, key >> 16), lo = __reduce_max_sync(part, key & 0xFFFFu);
                if (KIND == KIND_BLK64) { if (lane < 2) C.wmax[b][pass][2 * warp + h] = (hi << 16) | lo; }
                else if (lane == 0) C.wmax[b][pass][warp] = (hi << 16) | lo;
                dead = compute_bar_or(dead);                                       // also spreads the word that a wait ran out
                uint32_t any;                                                      // the largest key of the tile: CTA-uniform
                if (KIND == KIND_BLK64) {
                    const uint4 k0 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][0]), k1 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][4]);
                    const uint4 k2 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][8]), k3 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][12]);
                    // entries 2 * warp + h: warps 0-3 hold the upper rows, 4-7 the lower
                    const uint32_t u0 = __vimax3_u16x2(k0.x, k0.z, key_max(k1.x, k1.z)), u1 = __vimax3_u16x2(k0.y, k0.w, key_max(k1.y, k1.w));
                    const uint32_t l0 = __vimax3_u16x2(k2.x, k2.z, key_max(k3.x, k3.z)), l1 = __vimax3_u16x2(k2.y, k2.w, key_max(k3.y, k3.w));
                    key = (row >> 6) ? (h ? l1 : l0) : (h ? u1 : u0);
                    any = key_max(key_max(u0, u1), key_max(l0, l1));
                } else {
                    const uint4 k0 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][0]);
                    const uint4 k1 = *reinterpret_cast<const uint4*>(&C.wmax[b][pass][4]);
                    key = key_max(key_max(__vimax3_u16x2(k0.x, k0.y, k0.z), k0.w), key_max(__vimax3_u16x2(k1.x, k1.y, k1.z), k1.w));
                    any = key;
                }
                nonfin = pass == 1 || (any >> 16) >= kBf16Inf;                     // CTA-uniform
                if (dead) { key = 0u; nonfin = false; }
                tile_amax = any >> 16;
                if (pass == 1 || !nonfin) break;
                key = kStream ? scan_stage_finite<kLinear>(in_base + s * kInBytes + in_off) : scan_words_finite(w);
            }
            // no pre-pass ran: the tensor amax that the summary reports is gathered here
            if (amax_slot != nullptr) raise_amax(amax_slot, tile_amax, tid == 0 && !dead);
        } else {
            key = kStream ? scan_stage<kLinear>(in_base + s * kInBytes + in_off) : scan_words(w);
            nonfin = __any_sync(0xFFFFFFFFu, (key >> 16) >= kBf16Inf);
            if (nonfin) key = kStream ? scan_stage_finite<kLinear>(in_base + s * kInBytes + in_off) : scan_words_finite(w);
        }
        uint32_t amax_bits = key >> 16;
        const uint32_t minm1 = 0xFFFFu - (key & 0xFFFFu);

        uint32_t s4b, s5b;
        bool careful;
        if (!SCAN) {
            // prepared by the load warp: the scale of Algorithm 1 and, warp-uniform, whether the careful path is needed
            s4b = prep & 0x7FFFFFFFu;
            s5b = (min((s4b >> 23) + 7u, 254u) << 23) | (s4b & 0x7FFFFFu);
            careful = (prep >> 31) != 0u;
        } else {
            block_scale(amax_bits, m_g, scale_mode, C.rtab, s4b, s5b);
            // minm1 covers this thread's block (1x128), this tile (128x128), this quadrant (64x64)
            careful = needs_careful(nonfin, minm1, s4b);
            if (KIND != KIND_BLK128) careful = __any_sync(0xFFFFFFFFu, careful);
        }

        // ---- staging buffer and entries of tile it - 2 must have been consumed ----
        if (n2 > 0 && !dead) {
            bool ok = mbar_wait(&C.out_empty[b], (n2 - 1) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
        }

        const uint32_t oa = out_base + b * kOutBytes + out_off;
        uint32_t sel = MOR_FMT_E4M3;
        if (!dead) {
            // ---- cast and error terms ----
            float e43, e52;
            uint32_t nnz, nonf;
            if (kStream) {
                const uint32_t a = in_base + s * kInBytes + in_off;
                ConvAcc acc;
                conv_init(acc);
                if (careful) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t wh[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 v = lds128(in_chunk<kLinear>(a, 4 * half + j));
                            wh[4 * j] = v.x; wh[4 * j + 1] = v.y; wh[4 * j + 2] = v.z; wh[4 * j + 3] = v.w;
                        }
                        if (half == 1 && !kStash) stage_free_arrive(s);
                        convert_chunks<YARD, true, STORE, 4, kCount, kStash, kLinear>(wh, oa, 4 * half, s4b, s5b, acc, a);
                    }
                    conv_finish<YARD, true, kCount>(acc, s4b, s5b, e43, e52, nnz, nonf);
                } else {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t wh[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 v = lds128(in_chunk<kLinear>(a, 4 * half + j));
                            wh[4 * j] = v.x; wh[4 * j + 1] = v.y; wh[4 * j + 2] = v.z; wh[4 * j + 3] = v.w;
                        }
                        if (half == 1 && !kStash) stage_free_arrive(s);
                        convert_chunks<YARD, false, STORE, 4, kCount, kStash, kLinear>(wh, oa, 4 * half, s4b, s5b, acc, a);
                    }
                    conv_finish<YARD, false, kCount>(acc, s4b, s5b, e43, e52, nnz, nonf);
                }
            } else if (careful) {
                convert_words<YARD, true, STORE, kCount>(w, oa, s4b, s5b, e43, e52, nnz, nonf);
            } else {
                convert_words<YARD, false, STORE, kCount>(w, oa, s4b, s5b, e43, e52, nnz, nonf);
            }
            if (!kCount && tid == 0) nnz = m.nnz;       // the tile's count from the pre-pass, handed on in this thread's entry

            if (kRowFast) {
                // the store warp adds the row's two halves, decides the block and writes its metadata
                sts128(entry_base + b * (uint32_t)sizeof(C.entry[0]) + (uint32_t)tid * 16u,
                       make_uint4(__float_as_uint(e43), __float_as_uint(e52), nnz | (nonf << 16), s4b));
            } else if (kLineBlocks) {
                // ---- block sums, decision, metadata ----
                e43 += __shfl_xor_sync(0xFFFFFFFFu, e43, 1);
                e52 += __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
                uint32_t nz = nnz | (nonf << 16);
                nz += __shfl_xor_sync(0xFFFFFFFFu, nz, 1);
                const bool valid = row < (KIND == KIND_COL128 ? m.vcols : m.vrows);
                sel = decide_block(D, e43, e52, nz & 0xFFFFu, nz >> 16, amax_bits, minm1, (uint32_t)(KIND == KIND_COL128 ? m.vrows : m.vcols));
                if (kStash) {
                    if (sel == MOR_FMT_E5M2) copy_stash<kLinear>(in_base + s * kInBytes + in_off, oa);
                    fence_async_smem();                  // the stage is written by the next TMA load: order the stash accesses before it
                    stage_free_arrive(s);
                } else if (THREE && STORE && sel == MOR_FMT_E5M2) {
                    emit_e5m2_codes(w, oa, s5b);
                }
                if (h == 0) {
                    sts128(entry_base + b * (uint32_t)sizeof(C.entry[0]) + (uint32_t)row * 16u,
                           make_uint4(__float_as_uint(e43), __float_as_uint(e52), nz, (valid ? sel : kSelNone) | (minm1 << 16)));
                    if (kMetaInStore) {
                        C.colscale[b][row] = (sel == MOR_FMT_E5M2) ? s5b : s4b;
                    } else if (valid) {
                        const uint32_t blk = m.blk_base + (uint32_t)row * (KIND == KIND_COL128 ? 1u : R.nbc);
                        const uint32_t sb = (sel == MOR_FMT_E5M2) ? s5b : s4b;
                        if (R.sel) R.sel[blk] = (uint8_t)sel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(sb >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(sb);
                        if (EXTRA && R.block_stats) {
                            mor_block_stats_t bs;
                            bs.amax = __uint_as_float(amax_bits << 16);
                            bs.min_abs_nz = THREE ? minnz_value(minm1) : __uint_as_float(0x7F800000u);
                            bs.nnz = nz & 0xFFFFu; bs.n_nonfinite = nz >> 16; bs.sum_rel_e4m3 = e43; bs.sum_rel_e5m2 = e52;
                            R.block_stats[blk] = bs;
                        }
                    }
                }
                if (KIND == KIND_COL128) {
                    if (EXTRA && has_fallback && sel == MOR_FMT_BF16) write_column(R.fallback, R.ld, m, row, h, swz, w, false, sel, 0.0f);
                    if (EXTRA && has_fq) {
                        const uint32_t f = fq_e4m3 ? (uint32_t)MOR_FMT_E4M3 : sel;
                        write_column(R.fake_quant, R.ld, m, row, h, swz, w, true, f, __uint_as_float(f == MOR_FMT_E5M2 ? s5b : s4b));
                    }
                } else {
                    if (EXTRA && has_fallback && sel == MOR_FMT_BF16) write_fallback(R, w, m, row, h, swz);
                    if (EXTRA && has_fq) write_fake_quant(R, w, m, row, h, swz, fq_e4m3 ? (uint32_t)MOR_FMT_E4M3 : sel, s4b, s5b);
                }
            } else {
                sts128(entry_base + b * (uint32_t)sizeof(C.entry[0]) + (uint32_t)tid * 16u,
                       make_uint4(__float_as_uint(e43), __float_as_uint(e52), nnz | (nonf << 16), kSelNone | (minm1 << 16)));
                if (EXTRA && (KIND == KIND_TENSOR || KIND == KIND_CHANNEL) && has_fq)
                    write_fake_quant(R, w, m, row, h, swz, (uint32_t)MOR_FMT_E4M3, s4b, s5b);
                if (EXTRA && (KIND == KIND_CHANNEL || KIND == KIND_COLCH) && R.row_part != nullptr) {
                    // per-row decision or statistics: this tile's part of the row's sums, for mor_row_decide_kernel
                    const float r43 = e43 + __shfl_xor_sync(0xFFFFFFFFu, e43, 1), r52 = e52 + __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
                    uint32_t nz = nnz | (nonf << 16);
                    nz += __shfl_xor_sync(0xFFFFFFFFu, nz, 1);
                    if (h == 0 && row < (KIND == KIND_COLCH ? m.vcols : m.vrows))
                        R.row_part[(size_t)m.local * kTileRows + row] = make_float4(r43, r52, __uint_as_float(nz), 0.0f);
                }
                if (EXTRA && KIND == KIND_COLCH && has_fq)
                    write_column(R.fake_quant, R.ld, m, row, h, swz, w, true, (uint32_t)MOR_FMT_E4M3, __uint_as_float(s4b));
                if ((KIND == KIND_CHANNEL || KIND == KIND_COLCH) && h == 0 && m.blk_base != 0xFFFFFFFFu &&
                    row < (KIND == KIND_COLCH ? m.vcols : m.vrows)) {
                    // per-channel: the row's scale, written by the tile that holds the row's first columns
                    const uint32_t blk = m.blk_base + (uint32_t)row;
                    if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(s4b >> 23);
                    if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(s4b);
                }
                if ((KIND == KIND_BLK128 && tid == 0) || (KIND == KIND_BLK64 && (row & 63) == 0)) {
                    C.tile_scale[b][q][0] = s4b; C.tile_scale[b][q][1] = s5b; C.tile_key[b][q] = key;
                }
                if (kSelfDecide) {
                    float w43 = e43, w52 = e52;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) { w43 += __shfl_xor_sync(0xFFFFFFFFu, w43, o); w52 += __shfl_xor_sync(0xFFFFFFFFu, w52, o); }
                    const uint32_t wnf = __reduce_add_sync(0xFFFFFFFFu, nonf);
                    if (lane == 0) { C.wsum[b][0][warp] = w43; C.wsum[b][1][warp] = w52; C.wsum[b][2][warp] = __uint_as_float(wnf); }
                }
            }
            if (STORE) fence_async_smem();              // the codes must be visible to the TMA store
        } else if (kStream && !(kStash && !kLineBlocks)) {
            stage_free_arrive(s);                       // given up: the arrival that the conversion would have made
        }
        if (kSelfDecide) {
            dead = compute_bar_or(dead);                // every compute thread, whatever its state; spreads the word of a wait that ran out
            if (!dead) {
                const float4 a0 = *reinterpret_cast<const float4*>(&C.wsum[b][0][0]), a1 = *reinterpret_cast<const float4*>(&C.wsum[b][0][4]);
                const float4 b0 = *reinterpret_cast<const float4*>(&C.wsum[b][1][0]), b1 = *reinterpret_cast<const float4*>(&C.wsum[b][1][4]);
                const uint4 n0 = *reinterpret_cast<const uint4*>(&C.wsum[b][2][0]), n1 = *reinterpret_cast<const uint4*>(&C.wsum[b][2][4]);
                const float t43 = ((a0.x + a0.y) + (a0.z + a0.w)) + ((a1.x + a1.y) + (a1.z + a1.w));
                const float t52 = ((b0.x + b0.y) + (b0.z + b0.w)) + ((b1.x + b1.y) + (b1.z + b1.w));
                const uint32_t tnf = (n0.x + n0.y + n0.z + n0.w) + (n1.x + n1.y + n1.z + n1.w);
                sel = decide_block(D, t43, t52, 0u, tnf, amax_bits, minm1, (uint32_t)(m.vrows * m.vcols));
                if (sel == MOR_FMT_E5M2) copy_stash<kLinear>(in_base + s * kInBytes + in_off, oa);
                fence_async_smem();                      // stash accesses before the next TMA load; codes visible to the TMA store
                if (tid == 0) C.dec_sel[b][0] = sel;     // for the store warp's metadata
            }
            stage_free_arrive(s);
        }
        out_full_arrive(b);

        if (!kSelfDecide && (KIND == KIND_BLK128 || KIND == KIND_BLK64)) {
            const bool need_dec = THREE || (EXTRA && (has_fallback || has_fq));
            if ((THREE || EXTRA) && need_dec) {
                if (!dead) {
                    bool ok = mbar_wait(&C.dec_full[b], n2 & 1u, &C.abort, p.wait_cycles);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
                }
                if (!dead) sel = C.dec_sel[b][q];
                if (THREE && STORE) {
                    if (kStash) {
                        if (!dead && sel == MOR_FMT_E5M2) copy_stash<kLinear>(in_base + s * kInBytes + in_off, oa);
                    } else if (!dead && sel == MOR_FMT_E5M2) {
                        emit_e5m2_codes(w, oa, s5b);
                    }
                    fence_async_smem();
                    if (kStash) stage_free_arrive(s);     // after the fence: the stash accesses come before the next TMA load
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&C.codes_full[b]);
                }
                if (EXTRA && has_fallback && !dead && sel == MOR_FMT_BF16) write_fallback(R, w, m, row, h, swz);
                if (EXTRA && has_fq && !dead) write_fake_quant(R, w, m, row, h, swz, fq_e4m3 ? (uint32_t)MOR_FMT_E4M3 : sel, s4b, s5b);
            }
        }
    }
}

// ------------------------------------------------------------------ blocks along the columns, prepared scales ----

// Four rows of two neighbouring columns (w[i]: the pair's word of row i), each column with its own scale (packed in
// s2): the fast conversion of convert_quad_fast with the cast pairing rows of one column, so that a column's four
// codes come out as one word in memory order of the transposed code tile.  Column c of the pair adds into a43[c],
// a52[c] and leaves its codes in c4[c] (and its E5M2 codes in c5[c]).
template <bool YARD>
__device__ __forceinline__ void convert_colpair_fast(const uint32_t (&w)[4], unsigned long long s2, unsigned long long tiny2,
                                                     float* a43, float* a52, uint32_t* c4, uint32_t* c5)
{
    unsigned long long y2[4];
    float y[4][2], r[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float x0, x1, u0, u1;
        unpack_bf16x2(w[i], x0, x1);
        const unsigned long long x2 = pack_f32x2(x0, x1);
        y2[i] = mul_f32x2(x2, s2);
        unpack_f32x2(y2[i], y[i][0], y[i][1]);
        unpack_f32x2(fma_f32x2(x2, s2, tiny2), u0, u1);
        r[i][0] = rcp_ftz(u0);
        r[i][1] = rcp_ftz(u1);
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint32_t qa, qb;
        float d0, d1, d2, d3;
        cast4_e4m3(y[0][c], y[1][c], y[2][c], y[3][c], c4[c], qa, qb);
        diff_f16x2_f32(qa, y[0][c], y[1][c], d0, d1);
        diff_f16x2_f32(qb, y[2][c], y[3][c], d2, d3);
        a43[c] = fmaf(fabsf(d0), fabsf(r[0][c]), a43[c]);
        a43[c] = fmaf(fabsf(d1), fabsf(r[1][c]), a43[c]);
        a43[c] = fmaf(fabsf(d2), fabsf(r[2][c]), a43[c]);
        a43[c] = fmaf(fabsf(d3), fabsf(r[3][c]), a43[c]);
    }
    if (YARD) {
        // (as in convert_quad_fast: the E5M2 scale is 2^7 times the E4M3 scale, so z = 128 y exactly)
        const unsigned long long k128 = pack_f32x2(128.0f, 128.0f);
        float z[4][2];
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack_f32x2(mul_f32x2(y2[i], k128), z[i][0], z[i][1]);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t qa, qb;
            float d0, d1, d2, d3;
            cast4_e5m2(z[0][c], z[1][c], z[2][c], z[3][c], c5[c], qa, qb);
            diff_f16x2_f32(qa, z[0][c], z[1][c], d0, d1);
            diff_f16x2_f32(qb, z[2][c], z[3][c], d2, d3);
            a52[c] = fmaf(fabsf(d0), fabsf(r[0][c]), a52[c]);
            a52[c] = fmaf(fabsf(d1), fabsf(r[1][c]), a52[c]);
            a52[c] = fmaf(fabsf(d2), fabsf(r[2][c]), a52[c]);
            a52[c] = fmaf(fabsf(d3), fabsf(r[3][c]), a52[c]);
        }
    } else {
        c5[0] = c5[1] = 0u;
    }
}

// Careful path for 16 rows of one column (NaN/inf, scaled values below binary32's normal range, capped E5M2
// exponent): the elements are gathered with 16-bit loads, two rows to a word, and go through
// convert_pair_careful.  `a`: shared-memory address of the column's first element.  Returns the column's sums
// and its 16 codes; adds its NaN/inf elements to `nonfinite`.
template <bool YARD>
__device__ __noinline__ void convert_col_careful(uint32_t a, uint32_t s4b, uint32_t s5b, float& e43, float& e52, uint4& codes, uint32_t& nonfinite)
{
    CarefulAcc A;
    A.a43 = A.a52 = 0.0f;
    A.nnz = A.nbig = A.nonfinite = 0u;
    uint32_t c[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        uint32_t lo, hi, c5;
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(lo) : "r"(a + (uint32_t)(2 * k * 256)));
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(hi) : "r"(a + (uint32_t)((2 * k + 1) * 256)));
        convert_pair_careful<YARD>(__byte_perm(lo, hi, 0x5410), __uint_as_float(s4b), __uint_as_float(s5b), A, c[k], c5);
    }
    codes = make_uint4(__byte_perm(c[0], c[1], 0x5410), __byte_perm(c[2], c[3], 0x5410),
                       __byte_perm(c[4], c[5], 0x5410), __byte_perm(c[6], c[7], 0x5410));
    const float ratio = __uint_as_float((127u - ((s5b >> 23) - (s4b >> 23))) << 23);   // scale4 / scale5
    const float tiny = (float)(A.nnz - A.nbig);
    e43 = A.a43 + tiny;
    e52 = YARD ? A.a52 * ratio + tiny : 0.0f;
    nonfinite += A.nonfinite;
}

// 128x1 blocks with keys from the pre-pass, plain outputs, two formats.  The tile is taken in its row-major order
// with full-width loads instead of a 16-bit gather: a thread owns four neighbouring columns (one 8-byte piece of
// each row) over 16 rows, i.e. 16 elements of four different blocks, each block with its own prepared scale.  The
// cast pairs rows of one column, so a column's 16 codes are 16 contiguous bytes of the transposed code tile.
//   thread (warp wp, lane l):  columns 4 qc .. 4 qc + 3 with qc = (l & 15) + 16 (wp & 1),
//                              rows 16 g .. 16 g + 15 with g = ((l & 7) + 2 (wp >> 1) + (l >> 4)) & 7.
// A half-warp's 8-byte loads cover 128 contiguous bytes of a row each (rows differ between lanes, their pitch is a
// multiple of all banks); the eight lanes of a 16-byte store phase have eight different g, i.e. all banks once.
// Lanes l and l ^ 16 hold the same columns: they add their sums, and lane l < 16 hands the four columns' sums to
// the store warp as part wp >> 1 of four (entry area: [part][column] {E4M3 sum, E5M2 sum}); the store warp adds
// the parts in order, decides the 128 blocks and writes their metadata (store_warp, COLFAST).
// One tile of that path.  `pw`: the four columns' prepared words; `careful`: the tile takes the careful path;
// s, b: stage and staging buffer; n2: how many tiles have used staging buffer b before.
struct ColsFastThread {
    int lane, wp, qc;
    uint32_t in_off, out_off;
    __device__ __forceinline__ ColsFastThread(int tid)
    {
        lane = tid & 31; wp = tid >> 5;
        qc = (lane & 15) + 16 * (wp & 1);
        const int g = ((lane & 7) + 2 * (wp >> 1) + (lane >> 4)) & 7;
        in_off = (uint32_t)(g * 16 * 256 + qc * 8);
        out_off = (uint32_t)(qc * 4 * 128 + g * 16);
    }
};

template <bool YARD, bool STORE>
__device__ __forceinline__ void cols_fast_tile(const MainParams& p, Control& C, const ColsFastThread& T, uint32_t in_base, uint32_t out_base,
                                               uint4 pw, bool careful, uint32_t tile_nnz, uint32_t s, uint32_t b, uint32_t n2, bool& dead)
{
    const int lane = T.lane, wp = T.wp, qc = T.qc;
    const uint32_t s4b[4] = {pw.x & 0x7FFFFFFFu, pw.y & 0x7FFFFFFFu, pw.z & 0x7FFFFFFFu, pw.w & 0x7FFFFFFFu};
    // ---- staging buffer and entries of the tile that used them before must have been consumed ----
    if (n2 > 0 && !dead) {
        bool ok = mbar_wait(&C.out_empty[b], (n2 - 1) & 1u, &C.abort, p.wait_cycles);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
    }
    const uint32_t a = in_base + s * kInBytes + T.in_off;
    const uint32_t oa = out_base + b * kOutBytes + T.out_off;
    if (!dead) {
        float e43[4] = {0.0f, 0.0f, 0.0f, 0.0f}, e52[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        uint32_t nonf = 0u;
        if (!careful) {
            const unsigned long long tiny2 = pack_f32x2(FLT_MIN, FLT_MIN);
            const unsigned long long sa = pack_f32x2(__uint_as_float(s4b[0]), __uint_as_float(s4b[1]));
            const unsigned long long sb = pack_f32x2(__uint_as_float(s4b[2]), __uint_as_float(s4b[3]));
            uint32_t cw[4][4];                       // [column][group of four rows]
#pragma unroll
            for (int grp = 0; grp < 4; ++grp) {
                uint32_t wa[4], wb[4], c4[4], c5[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint2 v = lds64(a + (uint32_t)((4 * grp + i) * 256));
                    wa[i] = v.x; wb[i] = v.y;
                }
                if (grp == 3) stage_free_arrive(s);
                convert_colpair_fast<YARD>(wa, sa, tiny2, &e43[0], &e52[0], &c4[0], &c5[0]);
                convert_colpair_fast<YARD>(wb, sb, tiny2, &e43[2], &e52[2], &c4[2], &c5[2]);
#pragma unroll
                for (int c = 0; c < 4; ++c) cw[c][grp] = c4[c];
            }
            if (STORE) {
#pragma unroll
                for (int c = 0; c < 4; ++c) sts128(oa + (uint32_t)(c * 128), make_uint4(cw[c][0], cw[c][1], cw[c][2], cw[c][3]));
            }
            if (YARD) {
#pragma unroll
                for (int c = 0; c < 4; ++c) e52[c] *= 0.0078125f;   // the factor 1/128 of the E5M2 terms, once per column
            }
        } else {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                const uint32_t sc = c == 0 ? s4b[0] : c == 1 ? s4b[1] : c == 2 ? s4b[2] : s4b[3];
                const uint32_t s5 = (min((sc >> 23) + 7u, 254u) << 23) | (sc & 0x7FFFFFu);
                float x43, x52;
                uint4 codes;
                convert_col_careful<YARD>(a + (uint32_t)(2 * c), sc, s5, x43, x52, codes, nonf);
                if (STORE) sts128(oa + (uint32_t)(c * 128), codes);
                if (c == 0) { e43[0] = x43; e52[0] = x52; }
                if (c == 1) { e43[1] = x43; e52[1] = x52; }
                if (c == 2) { e43[2] = x43; e52[2] = x52; }
                if (c == 3) { e43[3] = x43; e52[3] = x52; }
            }
            stage_free_arrive(s);
        }
        // ---- the sums of lanes l and l ^ 16 (same columns, neighbouring row groups), handed on by lane l < 16 ----
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            e43[c] += __shfl_xor_sync(0xFFFFFFFFu, e43[c], 16);
            e52[c] += __shfl_xor_sync(0xFFFFFFFFu, e52[c], 16);
        }
        nonf = __reduce_add_sync(0xFFFFFFFFu, nonf);
        if (lane < 16) {
            const uint32_t ea = smem_addr(&C.entry[b][0]) + (uint32_t)(wp >> 1) * 1024u + (uint32_t)qc * 32u;
            sts128(ea, make_uint4(__float_as_uint(e43[0]), __float_as_uint(e52[0]), __float_as_uint(e43[1]), __float_as_uint(e52[1])));
            sts128(ea + 16u, make_uint4(__float_as_uint(e43[2]), __float_as_uint(e52[2]), __float_as_uint(e43[3]), __float_as_uint(e52[3])));
            if (wp < 2) sts128(smem_addr(&C.colscale[b][0]) + (uint32_t)qc * 16u, pw);      // one thread per four columns
        }
        if (lane == 0) C.colnonf[b][wp] = nonf;
        if (wp == 0 && lane == 0) C.colnnz[b] = tile_nnz;
        if (STORE) fence_async_smem();              // the codes must be visible to the TMA store
    } else {
        stage_free_arrive(s);                       // given up: the arrival that the conversion would have made
    }
    out_full_arrive(b);
}

template <bool YARD, bool STORE>
__device__ __forceinline__ void compute_cols_fast(const MainParams& p, Control& C, unsigned char* in, unsigned char* out, int tid)
{
    const ColsFastThread T(tid);
    const uint32_t in_base = smem_addr(in), out_base = smem_addr(out);
    const uint32_t meta_base = smem_addr(&C.meta[0]), prep_base = smem_addr(&C.prep[0][0]), flag_base = smem_addr(&C.colflag[0]);
    bool dead = false;
    const uint32_t n_it = my_tile_count(p);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        const uint32_t s = it % kStages;
        if (!dead) {
            bool ok = mbar_wait(&C.full[s], (it / kStages) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { dead = true; if (T.lane == 0) give_up(C, p.device_status); }
        }
        // prepared by the load warp: the four columns' scales (bit 31: NaN or inf in the column piece), whether the
        // tile takes the careful path, and the tile's count of finite non-zeros
        const uint4 pw = lds128(prep_base + s * (uint32_t)(kTileRows * 4) + (uint32_t)T.qc * 16u);
        uint32_t careful, tile_nnz = 0u;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(careful) : "r"(flag_base + s * 4u));
        if (tid == 0) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tile_nnz) : "r"(meta_base + s * (uint32_t)sizeof(TileMeta) + 28u));
        cols_fast_tile<YARD, STORE>(p, C, T, in_base, out_base, pw, careful != 0u, tile_nnz, s, it & 1u, it >> 1, dead);
    }
}

// Rows and columns of the same tensors from one read, keys of both directions from the pre-pass, two formats, plain
// outputs.  Per tile the rows' conversion streams from the stage exactly as the 1x128 path does (prepared row
// scales), then the columns' conversion takes the stage as compute_cols_fast does (prepared column scales) and
// hands it back.  Staging buffer 0 and its entries serve the rows, buffer 1 the columns.
template <bool YARD>
__device__ __forceinline__ void compute_dual_fast(const MainParams& p, Control& C, unsigned char* in, unsigned char* out, int tid)
{
    const ColsFastThread T(tid);
    const int lane = tid & 31;
    const int row = tid >> 1, h = tid & 1;
    const int swz = (row & 7) ^ (h << 2);
    const uint32_t in_off = (uint32_t)(row * 256 + h * 128 + (swz << 4));
    const uint32_t out_off = (uint32_t)(row * 128 + h * 64 + (swz << 3));
    const uint32_t in_base = smem_addr(in), out_base = smem_addr(out), entry_base = smem_addr(&C.entry[0][0]);
    const uint32_t meta_base = smem_addr(&C.meta[0]), prep_base = smem_addr(&C.prep[0][0]), prep2_base = smem_addr(&C.prep2[0][0]);
    const uint32_t flag_base = smem_addr(&C.colflag[0]);
    bool dead = false;
    RecFacts Q;              // what the rows' decision and metadata need of their record, reloaded per tensor
    int q_ti = -1;
    const uint32_t n_it = my_tile_count(p);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        const uint32_t s = it % kStages;
        if (!dead) {
            bool ok = mbar_wait(&C.full[s], (it / kStages) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
        }
        TileMeta m;
        {
            const uint4 q0 = lds128(meta_base + s * (uint32_t)sizeof(TileMeta));
            m.ti = dead ? 0 : (int32_t)q0.x; m.vrows = (int32_t)q0.y; m.vcols = (int32_t)q0.z; m.blk_base = q0.w;
        }
        uint32_t tile_nnz = 0u;
        if (tid == 0) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tile_nnz) : "r"(meta_base + s * (uint32_t)sizeof(TileMeta) + 28u));

        // ---- rows (record ti): the streaming 1x128 path ----
        {
            if (m.ti != q_ti) { q_ti = m.ti; Q.load(p.b.t[m.ti]); }
            const RecFacts& R = Q;
            uint32_t prep;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(prep) : "r"(prep_base + s * (uint32_t)(kTileRows * 4) + (uint32_t)row * 4u));
            const uint32_t s4b = prep & 0x7FFFFFFFu;
            const uint32_t s5b = (min((s4b >> 23) + 7u, 254u) << 23) | (s4b & 0x7FFFFFu);
            const bool careful = (prep >> 31) != 0u;
            if (it > 0 && !dead) {
                bool ok = mbar_wait(&C.out_empty[0], (it - 1) & 1u, &C.abort, p.wait_cycles);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
            }
            const uint32_t oa = out_base + out_off;
            if (!dead) {
                const uint32_t a = in_base + s * kInBytes + in_off;
                float e43, e52;
                uint32_t nnz, nonf;
                ConvAcc acc;
                conv_init(acc);
                if (careful) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t wh[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 v = lds128(a ^ ((4 * half + j) << 4));
                            wh[4 * j] = v.x; wh[4 * j + 1] = v.y; wh[4 * j + 2] = v.z; wh[4 * j + 3] = v.w;
                        }
                        convert_chunks<YARD, true, true, 4, false, false>(wh, oa, 4 * half, s4b, s5b, acc, a);
                    }
                    conv_finish<YARD, true, false>(acc, s4b, s5b, e43, e52, nnz, nonf);
                } else {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t wh[16];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 v = lds128(a ^ ((4 * half + j) << 4));
                            wh[4 * j] = v.x; wh[4 * j + 1] = v.y; wh[4 * j + 2] = v.z; wh[4 * j + 3] = v.w;
                        }
                        convert_chunks<YARD, false, true, 4, false, false>(wh, oa, 4 * half, s4b, s5b, acc, a);
                    }
                    conv_finish<YARD, false, false>(acc, s4b, s5b, e43, e52, nnz, nonf);
                }
                if (tid == 0) nnz = tile_nnz;            // the tile's count from the pre-pass, handed on in this thread's entry
                e43 += __shfl_xor_sync(0xFFFFFFFFu, e43, 1);
                e52 += __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
                uint32_t nz = nnz | (nonf << 16);
                nz += __shfl_xor_sync(0xFFFFFFFFu, nz, 1);
                const bool valid = row < m.vrows;
                const uint32_t sel = decide_block(R, e43, e52, nz & 0xFFFFu, nz >> 16, 0u, 0xFFFFu, (uint32_t)m.vcols);
                if (h == 0) {
                    sts128(entry_base + (uint32_t)row * 16u,
                           make_uint4(__float_as_uint(e43), __float_as_uint(e52), nz, (valid ? sel : kSelNone) | (0xFFFFu << 16)));
                    if (valid) {
                        const uint32_t blk = m.blk_base + (uint32_t)row * R.nbc;
                        if (R.sel) R.sel[blk] = (uint8_t)sel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(s4b >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(s4b);
                    }
                }
                fence_async_smem();                      // the codes must be visible to the TMA store
            }
            out_full_arrive(0);
        }

        // ---- columns (record ti + 1): the full-width column path; the stage goes back after its loads ----
        {
            const uint4 pw = lds128(prep2_base + s * (uint32_t)(kTileCols * 4) + (uint32_t)T.qc * 16u);
            uint32_t careful;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(careful) : "r"(flag_base + s * 4u));
            cols_fast_tile<YARD, true>(p, C, T, in_base, out_base, pw, careful != 0u, tile_nnz, s, 1u, it, dead);
        }
    }
}

// ------------------------------------------------------------------ both directions from one read ----

// KIND_DUAL: the tensor is wanted with 1x128 blocks and with 128x1 blocks (the two operand layouts of the forward
// and backward GEMMs).  A tile is loaded once; the compute threads take it from the stage twice, first as rows
// (record ti, exactly the 1x128 path), then as columns (record ti + 1, exactly the 128x1 path, codes transposed),
// and hand each direction to the store warp as a tile of its own, so the two staging buffers alternate between
// the directions.  The stage is released after the second copy to registers.
template <bool YARD, bool THREE, bool SCAN>
__device__ __forceinline__ void compute_warps_dual(const MainParams& p, Control& C, unsigned char* in, unsigned char* out, int tid)
{
    const int lane = tid & 31;
    const int row = tid >> 1, h = tid & 1;
    const uint32_t in_base = smem_addr(in), out_base = smem_addr(out), entry_base = smem_addr(&C.entry[0][0]);
    const uint32_t meta_base = smem_addr(&C.meta[0]), keys_base = smem_addr(&C.keys[0][0]);
    int cur_ti = -1;
    uint32_t m_g = 0;
    int scale_mode = 0;
    bool dead = false;
    const uint32_t n_it = my_tile_count(p);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        const uint32_t s = it % kStages;
        if (!dead) {
            bool ok = mbar_wait(&C.full[s], (it / kStages) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
        }
        TileMeta m;
        {
            const uint4 q0 = lds128(meta_base + s * (uint32_t)sizeof(TileMeta));
            const uint4 q1 = lds128(meta_base + s * (uint32_t)sizeof(TileMeta) + 16u);
            m.ti = dead ? 0 : (int32_t)q0.x; m.vrows = (int32_t)q0.y; m.vcols = (int32_t)q0.z; m.blk_base = q0.w;
            m.local = q1.x; m.row0 = (int32_t)q1.y; m.col0 = (int32_t)q1.z; m.nnz = q1.w;
        }
        if (m.ti != cur_ti) {
            cur_ti = m.ti;
            scale_mode = p.b.t[m.ti].scale_mode;
            if (!dead) m_g = group_mantissa(*p.b.t[m.ti].amax, scale_mode);
        }
#pragma unroll 1
        for (int dir = 0; dir < 2; ++dir) {
            const TensorRec& R = p.b.t[m.ti + dir];
            const uint32_t b = (uint32_t)dir, n2 = it;        // conversion number 2 * it + dir
            const int swz = dir ? ((row >> 1) & 3) ^ (h << 2) : (row & 7) ^ (h << 2);
            uint32_t w[32];
            uint32_t key = 0u;
            if (dir == 0) {
                const uint32_t a = in_base + s * kInBytes + (uint32_t)(row * 256 + h * 128 + (swz << 4));
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 v = lds128(a ^ (j << 4));
                    w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
                }
                if (!SCAN) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(key) : "r"(keys_base + s * (uint32_t)(kRowKeyStride * 4) + (uint32_t)row * 4u));
            } else {
                // this thread takes column `row` of the tile, rows 64 h .. 64 h + 63, two rows per word
                const uint32_t a = in_base + s * kInBytes + (uint32_t)(h * 64 * 256 + row * 2);
                load_column(a, swz, w);
                stage_free_arrive(s);                       // both copies of the stage are in registers
            }

            // ---- block amax and smallest non-zero (Algorithm 1; Eq. 4) ----
            bool nonfin;
            if (dir == 0 && !SCAN) {
                nonfin = __any_sync(0xFFFFFFFFu, (key >> 31) != 0u);
                key &= 0x7FFFFFFFu;
            } else {
                key = scan_words(w);
                key = key_max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 1));
                nonfin = __any_sync(0xFFFFFFFFu, (key >> 16) >= kBf16Inf);
                if (nonfin) {
                    key = scan_words_finite(w);
                    key = key_max(key, __shfl_xor_sync(0xFFFFFFFFu, key, 1));
                }
                if (dir == 0) {                             // no pre-pass ran: gather the tensor amax for the summaries
                    const uint32_t wamax = __reduce_max_sync(0xFFFFFFFFu, key >> 16);
                    raise_amax(R.amax_slot, wamax, lane == 0 && !dead && R.amax == R.amax_slot);
                }
            }
            const uint32_t amax_bits = key >> 16, minm1 = 0xFFFFu - (key & 0xFFFFu);
            uint32_t s4b, s5b;
            block_scale(amax_bits, m_g, scale_mode, C.rtab, s4b, s5b);
            bool careful = nonfin;
            if (minm1 != 0xFFFFu) careful = careful || !(__fmul_rn(minnz_value(minm1), __uint_as_float(s4b)) >= 7.888609052210118e-31f);
            careful = careful || (s4b >> 23) > 247u;
            careful = __any_sync(0xFFFFFFFFu, careful);

            // ---- staging buffer and entries of the same direction of the tile before must have been consumed ----
            if (n2 > 0 && !dead) {
                bool ok = mbar_wait(&C.out_empty[b], (n2 - 1) & 1u, &C.abort, p.wait_cycles);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) { dead = true; if (lane == 0) give_up(C, p.device_status); }
            }
            const uint32_t oa = out_base + b * kOutBytes + (uint32_t)(row * 128 + h * 64 + (swz << 3));
            if (!dead) {
                float e43, e52;
                uint32_t nnz, nonf;
                if (careful) convert_words<YARD, true, true>(w, oa, s4b, s5b, e43, e52, nnz, nonf);
                else         convert_words<YARD, false, true>(w, oa, s4b, s5b, e43, e52, nnz, nonf);
                e43 += __shfl_xor_sync(0xFFFFFFFFu, e43, 1);
                e52 += __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
                uint32_t nz = nnz | (nonf << 16);
                nz += __shfl_xor_sync(0xFFFFFFFFu, nz, 1);
                const bool valid = row < (dir ? m.vcols : m.vrows);
                const uint32_t sel = decide_block(R, e43, e52, nz & 0xFFFFu, nz >> 16, amax_bits, minm1, (uint32_t)(dir ? m.vrows : m.vcols));
                if (THREE && sel == MOR_FMT_E5M2) emit_e5m2_codes(w, oa, s5b);
                if (h == 0) {
                    sts128(entry_base + b * (uint32_t)sizeof(C.entry[0]) + (uint32_t)row * 16u,
                           make_uint4(__float_as_uint(e43), __float_as_uint(e52), nz, (valid ? sel : kSelNone) | (minm1 << 16)));
                    if (valid) {
                        const uint32_t blk = dir ? (uint32_t)(m.row0 / kTileRows) * (uint32_t)R.cols + (uint32_t)m.col0 + (uint32_t)row
                                                 : m.blk_base + (uint32_t)row * R.nbc;
                        const uint32_t sb = (sel == MOR_FMT_E5M2) ? s5b : s4b;
                        if (R.sel) R.sel[blk] = (uint8_t)sel;
                        if (R.scale_e8m0) R.scale_e8m0[blk] = (uint8_t)(sb >> 23);
                        if (R.scale_f32) R.scale_f32[blk] = __uint_as_float(sb);
                        if (R.block_stats) {
                            mor_block_stats_t bs;
                            bs.amax = __uint_as_float(amax_bits << 16);
                            bs.min_abs_nz = THREE ? minnz_value(minm1) : __uint_as_float(0x7F800000u);
                            bs.nnz = nz & 0xFFFFu; bs.n_nonfinite = nz >> 16; bs.sum_rel_e4m3 = e43; bs.sum_rel_e5m2 = e52;
                            R.block_stats[blk] = bs;
                        }
                    }
                }
                fence_async_smem();                      // the codes must be visible to the TMA store
            }
            out_full_arrive(b);
        }
    }
}

// ------------------------------------------------------------------ kernel ----

template <int KIND, bool YARD, bool THREE, bool STORE, bool SCAN, bool EXTRA>
__global__ void __launch_bounds__(kMainThreads, 2)
mor_main_kernel(const __grid_constant__ MainParams p, Partial* __restrict__ partials)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    unsigned char* in = base;
    unsigned char* out = base + kStages * kInBytes;
    Control& C = *reinterpret_cast<Control*>(out + 2 * kOutBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&C.full[s], 2);   // copies started (with the byte count) + tile facts written
        for (int b = 0; b < 2; ++b) {
            mbar_init(&C.out_empty[b], 1);
            mbar_init(&C.dec_full[b], 1);
            mbar_init(&C.codes_full[b], kComputeWarps);
        }
        C.abort = 0u;
        C.issued = 0u;
        fence_mbar_init();
    }
    // fl32(448 / (1 + m/128)) for the 128 mantissas of a BF16 amax: the division of Algorithm 1,
    // done here once per CTA with the IEEE divide and looked up per block afterwards
    if (tid < 128) C.rtab[tid] = __float_as_uint(__fdiv_rn(448.0f, 1.0f + (float)tid * 0.0078125f));
    __syncthreads();
    // Up to here nothing was read that an earlier kernel of the stream writes: this CTA may have become resident
    // while the amax pre-pass was still draining.  From here on its amax and keys are needed.
    pdl_trigger();
    pdl_wait();

    // 128x1 blocks (alone, or beside the 1x128 blocks of the same tensor) and per-channel columns with keys from the
    // pre-pass, two formats, plain outputs: the full-width column path
    constexpr bool kColFast = (KIND == KIND_COL128 || KIND == KIND_DUAL || KIND == KIND_COLCH) && !SCAN && !EXTRA && !THREE;
    // ... and the 1x128 blocks of that recipe (scanning or not) leave their decisions and metadata to the store warp too
    constexpr bool kRowFast = KIND == KIND_ROW128 && !EXTRA && !THREE;
    if (warp < kComputeWarps) {
        if constexpr (KIND == KIND_DUAL && kColFast) compute_dual_fast<YARD>(p, C, in, out, tid);
        else if constexpr (KIND == KIND_DUAL) compute_warps_dual<YARD, THREE, SCAN>(p, C, in, out, tid);
        else if constexpr (kColFast) compute_cols_fast<YARD, STORE>(p, C, in, out, tid);
        else compute_warps<KIND, YARD, THREE, STORE, SCAN, EXTRA>(p, C, in, out, tid);
    }
    else if (warp == kLoadWarp) load_warp<KIND, !SCAN && (KIND != KIND_DUAL || kColFast), kColFast>(p, C, in, lane);
    else store_warp<KIND, THREE, STORE, EXTRA, kColFast || kRowFast>(p, C, out, partials, lane);
}

template <int KIND, bool YARD, bool THREE, bool STORE, bool SCAN, bool EXTRA>
cudaError_t launch_main_t(const MainParams& p, Partial* partials, cudaStream_t s)
{
    auto kfn = mor_main_kernel<KIND, YARD, THREE, STORE, SCAN, EXTRA>;
    static std::atomic<int> sm_count[64];   // per instantiation and device; 0 = not set up yet
    static std::mutex setup;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int sms = sm_count[dev].load(std::memory_order_acquire);
    if (sms == 0) {
        std::lock_guard<std::mutex> lock(setup);         // host threads may make their first call together
        e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (sms <= 0) return cudaErrorInvalidDevice;
        sm_count[dev].store(sms, std::memory_order_release);
    }
    const uint32_t resident = 2u * (uint32_t)sms;
    const uint32_t grid = p.total_tiles < resident ? p.total_tiles : resident;
    return launch_dependent(kfn, dim3(grid), dim3(kMainThreads), (size_t)kSmemBytes, s, p, partials);
}

// The instantiations of one partition kind for the recipe and output flags of `v`.
template <int KIND, bool SCAN>
cudaError_t launch_main_ks(const MainVariant& v, const MainParams& p, Partial* partials, cudaStream_t s)
{
#define MOR_LAUNCH(Y, T, S, E) launch_main_t<KIND, Y, T, S, SCAN, E>(p, partials, s)
#define MOR_LAUNCH_SE(Y, T) (v.store ? (v.extra ? MOR_LAUNCH(Y, T, true, true) : MOR_LAUNCH(Y, T, true, false)) \
                                     : (v.extra ? MOR_LAUNCH(Y, T, false, true) : MOR_LAUNCH(Y, T, false, false)))
    if (v.three) return MOR_LAUNCH_SE(true, true);
    if (v.yard) return MOR_LAUNCH_SE(true, false);
    return MOR_LAUNCH_SE(false, false);
#undef MOR_LAUNCH_SE
#undef MOR_LAUNCH
}

}  // namespace
}  // namespace mor
