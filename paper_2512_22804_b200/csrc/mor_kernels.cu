// The two small kernels around the fused main kernel (mor_main.cu).
//
//   mor_amax_kernel      Algorithm 1, first step: the largest magnitude of the group, the tensor being one group
//                        (persistent, TMA-fed); it also leaves the block keys and non-zero counts of every tile
//   mor_finalise_kernel  tensor-wide aggregate of the per-tile partials and the Eq. 2 decision
#include <cuda_bf16.h>
#include <float.h>

#include <atomic>
#include <mutex>

#include "mor_internal.h"
#include "mor_ptx.cuh"

namespace mor {
namespace {

constexpr uint32_t kBf16Inf = 0x7F80u;

struct WarpPart {
    double s43, s52;
    uint32_t nnz, nonfinite, n4, n5, nb, mn;
};

// Algorithm 1's binary32 scaling factor 448 / amax: one IEEE division; a quotient above the largest
// finite binary32 is replaced by it
__device__ __forceinline__ uint32_t ideal_scale_bits(float amax)
{
    return __float_as_uint(fminf(__fdiv_rn(448.0f, amax), FLT_MAX));
}

// Algorithm 1, group part: mantissa of 448 / g_amax (0 for an all-zero tensor, and for the
// scale modes that have no shared mantissa)
__device__ __forceinline__ uint32_t group_mantissa(float g_amax, int scale_mode)
{
    if (scale_mode != MOR_SCALE_GAM || !(g_amax > 0.0f)) return 0u;
    return ideal_scale_bits(g_amax) & 0x7FFFFFu;
}

// Algorithm 1, block part: exponent of 448 / b_amax, lowered by one when the group mantissa
// exceeds the block's; the scale is the shared mantissa joined to that exponent.  The E5M2
// scale is 7 binades higher (57344 = 448 * 2^7), capped at exponent field 254.
__device__ __forceinline__ void block_scale(float b_amax, uint32_t m_g, int scale_mode,
                                            uint32_t& s4_bits, uint32_t& s5_bits)
{
    uint32_t e = 127u, m = (scale_mode == MOR_SCALE_FP32_AMAX) ? 0u : m_g;
    if (b_amax > 0.0f) {
        const uint32_t sb = ideal_scale_bits(b_amax);
        const uint32_t m_b = sb & 0x7FFFFFu;
        e = sb >> 23;
        if (scale_mode == MOR_SCALE_FP32_AMAX) m = m_b;
        else if (m_g > m_b) e -= 1u;
    }
    const uint32_t e5 = min(e + 7u, 254u);
    s4_bits = (e << 23) | m;
    s5_bits = (e5 << 23) | m;
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float minnz_value(uint32_t minm1_bits)
{
    return minm1_bits == 0xFFFFu ? __uint_as_float(0x7F800000u) : __uint_as_float((minm1_bits + 1u) << 16);
}

// ------------------------------------------------------------------ amax pre-pass ----

// Key of 8 elements (four packed BF16 pairs): amax bits << 16 | 0xFFFF - (smallest non-zero bits - 1),
// so that keys combine with a packed 16-bit maximum.  NaN and inf compare above every finite pattern.
__device__ __forceinline__ uint32_t key_of_masked(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    const uint32_t mx = __vimax3_u16x2(__vimax3_u16x2(a0, a1, a2), a3, a3);
    uint32_t mn = __viaddmin_u16x2(a0, 0xFFFFFFFFu, 0xFFFFFFFFu);
    mn = __viaddmin_u16x2(a1, 0xFFFFFFFFu, mn);
    mn = __viaddmin_u16x2(a2, 0xFFFFFFFFu, mn);
    mn = __viaddmin_u16x2(a3, 0xFFFFFFFFu, mn);
    return (max(mx & 0xFFFFu, mx >> 16) << 16) | (0xFFFFu - min(mn & 0xFFFFu, mn >> 16));
}
__device__ __forceinline__ uint32_t key_of_chunk(uint4 v)
{
    return key_of_masked(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu, v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu);
}
// the same over finite elements only, with the count of the others (a real call: rare path)
__device__ __noinline__ uint2 key_of_chunk_finite(uint4 v)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t m = 0u, n = 0xFFFFu, nf = 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
        if (lo < kBf16Inf) { m = max(m, lo); n = min(n, (lo - 1u) & 0xFFFFu); } else nf++;
        if (hi < kBf16Inf) { m = max(m, hi); n = min(n, (hi - 1u) & 0xFFFFu); } else nf++;
    }
    return make_uint2((m << 16) | (0xFFFFu - n), nf);
}
__device__ __forceinline__ uint32_t key_max(uint32_t a, uint32_t b) { return __vimax3_u16x2(a, b, b); }

// The pre-pass works on the 128 x 128 tiles of the main kernel.  Results: the tensor's amax (Algorithm 1, first step,
// with the tensor as one group) by atomicMax and, when the tensor record has a key array, per tile the key of every
// row piece (1x128 partition: that is the block's amax and smallest non-zero), of every column piece (blocks along
// the columns), of every 64x64 quadrant or of the whole tile (other partitions), and the tile's count of finite
// non-zero elements, which let the main kernel skip its own scan.  Bit 31 of a key marks NaN/inf among its
// elements (the key itself covers the finite ones only).
// What the load warp tells the other warps about the tile in a stage (and, copied into the scratch, the tail warp).
constexpr uint32_t kModeKeys = 1u;        // the record wants keys (and the tile's count of non-zeros)
constexpr uint32_t kModePerPiece = 2u;    // ... one per row piece
constexpr uint32_t kModeColPiece = 4u;    // ... one per column piece
constexpr uint32_t kModeBlk64 = 8u;       // ... one per 64x64 quadrant
constexpr uint32_t kModeColsApart = 16u;  // the column keys have an area of their own (rows and columns from one pre-pass)
struct __align__(16) AmaxMeta {
    int32_t ti;                // tensor index within the launch
    uint32_t local;            // tile index within the tensor
    uint32_t mode;
    uint32_t key_stride;
    uint32_t* keys;
    uint32_t* col_keys;
};
static_assert(sizeof(AmaxMeta) == 32, "two 16-byte loads");

struct AmaxShared {
    AmaxMeta meta;
    uint32_t wkey[kThreads / 32], wnf[kThreads / 32], wnz[kThreads / 32];
    uint32_t qkey[kThreads / 32][4], qnf[kThreads / 32][4];                   // 64x64 blocks: per warp and quadrant
    uint32_t cm[kThreads / 32][64], cn[kThreads / 32][64], cf[kThreads / 32][16];   // blocks along the columns
};

// Hand-off between the 256 compute threads and the tail warp on hardware barriers (a thread asleep there takes no
// issue slots): "scratch b is complete" (compute threads announce, the tail warp sleeps) and "scratch b has been
// read" (the tail warp announces, compute threads wait -- normally long past).
__device__ __forceinline__ void scratch_full_arrive(uint32_t b) { asm volatile("barrier.cta.arrive %0, %1;" ::"r"(2u + b), "n"(kThreads + 32) : "memory"); }
__device__ __forceinline__ void scratch_full_sync(uint32_t b) { asm volatile("barrier.cta.sync %0, %1;" ::"r"(2u + b), "n"(kThreads + 32) : "memory"); }
__device__ __forceinline__ void scratch_free_arrive(uint32_t b) { asm volatile("barrier.cta.arrive %0, %1;" ::"r"(4u + b), "n"(kThreads + 32) : "memory"); }
__device__ __forceinline__ void scratch_free_sync(uint32_t b) { asm volatile("barrier.cta.sync %0, %1;" ::"r"(4u + b), "n"(kThreads + 32) : "memory"); }

// The work of a compute thread on one tile whose data it holds in registers: thread t has the 16-byte chunk
// (t & 15) of rows (t >> 4) + 16 j, j = 0..7 (zeros past the tensor's edge).  Keys of row pieces are complete within
// a warp and written from here; everything that spans warps (tile key, quadrant keys, column keys, counts, the
// tensor amax) is left per warp in the scratch `S` for the tail warp.  `dead`: a bounded wait has run out in this
// warp -- its data are zeros and it writes no keys, but keeps its part in the hand-off.
template <bool ROWS_ONLY>
__device__ __forceinline__ void amax_thread_part(const AmaxMeta& M, const uint4 (&v)[8], AmaxShared& S)
{
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int k = t & 15;
    const uint32_t local = M.local;
    const bool has_keys = (M.mode & kModeKeys) != 0u;
    const bool col_piece = (M.mode & kModeColPiece) != 0u;
    // Keys of row pieces alone (1x128 blocks, per-channel rows): the thread holds half a row piece (see the kernel), so
    // a piece's key is the thread's own key joined with its neighbour's.  In the general instantiation the thread
    // holds chunks of eight row pieces and the 16 lanes of a piece are joined by shuffles.
    // (ROWS_ONLY: the instantiation for launches all of whose tensors want row keys and nothing else)
    const bool row_map = ROWS_ONLY;
    const bool per_piece = !ROWS_ONLY && (M.mode & kModePerPiece) != 0u;
    uint32_t key[8], all = 0u, nf = 0u;
    // non-zero elements of the thread's 64: per 16-bit half min(|x| bits, 1), summed in both halves at once (on the
    // words already masked for the keys).  The main kernel takes the tile's count from here and need not count while
    // it converts.
    uint32_t nz2 = 0u;
    // per column of the thread's chunk (two columns to a word): the maximum and the wrapped minimum over its eight rows
    uint32_t cm[4] = {0u, 0u, 0u, 0u}, cn[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
    bool have_cols = false;
    if (col_piece && !per_piece) {
        // column keys alone: the thread's own key is folded from its columns' (no second pass over the elements)
        have_cols = true;
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            const uint32_t a[4] = {v[j].x & 0x7FFF7FFFu, v[j].y & 0x7FFF7FFFu, v[j].z & 0x7FFF7FFFu, v[j].w & 0x7FFF7FFFu};
            const uint32_t c[4] = {v[j + 1].x & 0x7FFF7FFFu, v[j + 1].y & 0x7FFF7FFFu, v[j + 1].z & 0x7FFF7FFFu, v[j + 1].w & 0x7FFF7FFFu};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                nz2 += __vimin3_u16x2(a[i], 0x00010001u, 0x00010001u) + __vimin3_u16x2(c[i], 0x00010001u, 0x00010001u);
                cm[i] = __vimax3_u16x2(cm[i], a[i], c[i]);
                cn[i] = __viaddmin_u16x2(c[i], 0xFFFFFFFFu, __viaddmin_u16x2(a[i], 0xFFFFFFFFu, cn[i]));
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) key[j] = 0u;
        const uint32_t mxx = __vimax3_u16x2(__vimax3_u16x2(cm[0], cm[1], cm[2]), cm[3], cm[3]);
        const uint32_t m2 = __vimin3_u16x2(__vimin3_u16x2(cn[0], cn[1], cn[2]), cn[3], cn[3]);
        all = (max(mxx & 0xFFFFu, mxx >> 16) << 16) | (0xFFFFu - min(m2 & 0xFFFFu, m2 >> 16));
    } else if (per_piece) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t a0 = v[j].x & 0x7FFF7FFFu, a1 = v[j].y & 0x7FFF7FFFu, a2 = v[j].z & 0x7FFF7FFFu, a3 = v[j].w & 0x7FFF7FFFu;
            const uint32_t n01 = __vimin3_u16x2(a0, 0x00010001u, 0x00010001u) + __vimin3_u16x2(a1, 0x00010001u, 0x00010001u);
            const uint32_t n23 = __vimin3_u16x2(a2, 0x00010001u, 0x00010001u) + __vimin3_u16x2(a3, 0x00010001u, 0x00010001u);
            nz2 += n01 + n23;
            key[j] = key_of_masked(a0, a1, a2, a3);
            all = key_max(all, key[j]);
        }
    } else {
        // one key for the thread's 64 elements: packed halves are folded once at the end; two independent chains of
        // every running value (even and odd chunks), so that a warp has something to issue while a result is on its way
        uint32_t mx[2] = {0u, 0u}, mn[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu}, nzc[2] = {0u, 0u};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = j & 1;
            const uint32_t a0 = v[j].x & 0x7FFF7FFFu, a1 = v[j].y & 0x7FFF7FFFu, a2 = v[j].z & 0x7FFF7FFFu, a3 = v[j].w & 0x7FFF7FFFu;
            if (has_keys) {
                const uint32_t n01 = __vimin3_u16x2(a0, 0x00010001u, 0x00010001u) + __vimin3_u16x2(a1, 0x00010001u, 0x00010001u);
                const uint32_t n23 = __vimin3_u16x2(a2, 0x00010001u, 0x00010001u) + __vimin3_u16x2(a3, 0x00010001u, 0x00010001u);
                nzc[c] += n01 + n23;
            }
            mx[c] = __vimax3_u16x2(mx[c], __vimax3_u16x2(a0, a1, a2), a3);
            mn[2 * c] = __viaddmin_u16x2(a2, 0xFFFFFFFFu, __viaddmin_u16x2(a0, 0xFFFFFFFFu, mn[2 * c]));
            mn[2 * c + 1] = __viaddmin_u16x2(a3, 0xFFFFFFFFu, __viaddmin_u16x2(a1, 0xFFFFFFFFu, mn[2 * c + 1]));
            key[j] = 0u;
        }
        nz2 = nzc[0] + nzc[1];
        const uint32_t mxx = __vimax3_u16x2(mx[0], mx[1], mx[1]);
        const uint32_t m2 = __vimin3_u16x2(__vimin3_u16x2(mn[0], mn[1], mn[2]), mn[3], mn[3]);
        all = (max(mxx & 0xFFFFu, mxx >> 16) << 16) | (0xFFFFu - min(m2 & 0xFFFFu, m2 >> 16));
    }
    uint32_t nz = (nz2 & 0xFFFFu) + (nz2 >> 16);
    // NaN or inf somewhere in the warp's data: redo the keys over finite elements and count the others
    const bool warp_nf = __any_sync(0xFFFFFFFFu, (all >> 16) >= kBf16Inf);
    uint32_t nf_piece = 0u;                                  // bit j: this thread saw NaN/inf in its chunk of piece j
    if (warp_nf) {
        all = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint2 r = key_of_chunk_finite(v[j]);
            key[j] = r.x;
            all = key_max(all, r.x);
            nf += r.y;
            nf_piece |= (r.y ? 1u : 0u) << j;
        }
    }
    if (row_map) {
        const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, all, 1);
        uint32_t f = nf ? 1u : 0u;
        f |= __shfl_xor_sync(0xFFFFFFFFu, f, 1);
        if ((t & 1) == 0) M.keys[(size_t)local * kRowKeyStride + (t >> 1)] = key_max(all, other) | (f << 31);
    }
    if (per_piece) {
        // one key per row piece: combine the 16 lanes that share the piece
        const uint32_t half = (lane & 16) ? 0xFFFF0000u : 0x0000FFFFu;
        uint32_t* kp = M.keys + (size_t)local * kRowKeyStride + (t >> 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t kk = key[j];
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) kk = key_max(kk, __shfl_xor_sync(0xFFFFFFFFu, kk, o));
            if (warp_nf) {
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, (nf_piece >> j) & 1u);
                if (b & half) kk |= 0x80000000u;
            }
            if (k == 0) kp[16 * j] = kk;
        }
    }
    if ((M.mode & kModeBlk64) != 0u) {
        // one key per 64x64 quadrant: this thread's chunk lies in column half (k >> 3); its first four rows
        // are in the upper half of the tile, the other four in the lower half
        uint32_t kq[2], nq[2] = {0u, 0u};
        if (warp_nf) {
            kq[0] = key_max(key_max(key[0], key[1]), key_max(key[2], key[3]));
            kq[1] = key_max(key_max(key[4], key[5]), key_max(key[6], key[7]));
            nq[0] = nf_piece & 0xFu; nq[1] = nf_piece >> 4;
        } else {
            kq[0] = key_max(key_max(key_of_chunk(v[0]), key_of_chunk(v[1])), key_max(key_of_chunk(v[2]), key_of_chunk(v[3])));
            kq[1] = key_max(key_max(key_of_chunk(v[4]), key_of_chunk(v[5])), key_max(key_of_chunk(v[6]), key_of_chunk(v[7])));
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            // lanes with the same (lane >> 3) & 1 share a column half
#pragma unroll
            for (int o = 1; o <= 16; o <<= 1) {
                if (o == 8) continue;
                kq[r] = key_max(kq[r], __shfl_xor_sync(0xFFFFFFFFu, kq[r], o));
                nq[r] |= __shfl_xor_sync(0xFFFFFFFFu, nq[r], o);
            }
            if ((lane & 7) == 0 && lane < 16) { S.qkey[warp][2 * r + (lane >> 3)] = kq[r]; S.qnf[warp][2 * r + (lane >> 3)] = nq[r]; }
        }
    }
    if (col_piece) {
        // One key per column of the tile.  This thread holds 8 rows of 8 columns: per column the maximum and the
        // wrapped minimum over its rows, packed two columns to a word; lanes l and l ^ 16 hold the same columns of
        // other rows; the warps' results meet in the scratch and the tail warp finishes four columns per lane.
        uint32_t cf = 0u;
        if (!warp_nf && have_cols) {
            // (done above)
        } else if (!warp_nf) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t a[4] = {v[j].x & 0x7FFF7FFFu, v[j].y & 0x7FFF7FFFu, v[j].z & 0x7FFF7FFFu, v[j].w & 0x7FFF7FFFu};
#pragma unroll
                for (int i = 0; i < 4; ++i) { cm[i] = __vimax3_u16x2(cm[i], a[i], a[i]); cn[i] = __viaddmin_u16x2(a[i], 0xFFFFFFFFu, cn[i]); }
            }
        } else {
            // NaN or inf somewhere in the warp's data: element by element, finite ones only (rare path)
#pragma unroll
            for (int i = 0; i < 4; ++i) { cm[i] = 0u; cn[i] = 0xFFFFFFFFu; }
            for (int j = 0; j < 8; ++j) {
                const uint32_t w4[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
                for (int i = 0; i < 4; ++i)
                    for (int hf = 0; hf < 2; ++hf) {
                        const uint32_t x = (w4[i] >> (16 * hf)) & 0x7FFFu;
                        if (x >= kBf16Inf) { cf |= 1u << (2 * i + hf); continue; }
                        const uint32_t m = (cm[i] >> (16 * hf)) & 0xFFFFu, n = (cn[i] >> (16 * hf)) & 0xFFFFu;
                        const uint32_t m2 = max(m, x), n2 = min(n, (x - 1u) & 0xFFFFu);
                        cm[i] = (cm[i] & ~(0xFFFFu << (16 * hf))) | (m2 << (16 * hf));
                        cn[i] = (cn[i] & ~(0xFFFFu << (16 * hf))) | (n2 << (16 * hf));
                    }
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t om = __shfl_xor_sync(0xFFFFFFFFu, cm[i], 16), on = __shfl_xor_sync(0xFFFFFFFFu, cn[i], 16);
            cm[i] = __vimax3_u16x2(cm[i], om, om);
            cn[i] = __vimin3_u16x2(cn[i], on, on);
        }
        cf |= __shfl_xor_sync(0xFFFFFFFFu, cf, 16);
        if (lane < 16) {
#pragma unroll
            for (int i = 0; i < 4; ++i) { S.cm[warp][4 * lane + i] = cm[i]; S.cn[warp][4 * lane + i] = cn[i]; }
            S.cf[warp][lane] = cf;
        }
    }
    const uint32_t hi = __reduce_max_sync(0xFFFFFFFFu, all >> 16), lo = __reduce_max_sync(0xFFFFFFFFu, all & 0xFFFFu);
    nf = __reduce_add_sync(0xFFFFFFFFu, nf);
    nz = __reduce_add_sync(0xFFFFFFFFu, nz);
    if (lane == 0) { S.wkey[warp] = (hi << 16) | lo; S.wnf[warp] = nf; S.wnz[warp] = nz; }
    if (t == 0) S.meta = M;
}

// The tail warp's work on one tile, from the scratch the compute warps left: keys of the columns (four per lane),
// and by lane 0 the tile's key or quadrant keys, its count of finite non-zeros and the tensor amax.  `seen_ti`,
// `seen_amax`: lane 0 remembers the largest amax it has sent for the tensor it is on, so that the atomic goes out
// only when a tile raises it.
__device__ __forceinline__ void amax_tail(const BatchParams& bp, const AmaxShared& S, int lane, int& seen_ti, uint32_t& seen_amax)
{
    const AmaxMeta M = S.meta;
    const uint32_t local = M.local;
    const bool has_keys = (M.mode & kModeKeys) != 0u;
    const bool col_piece = (M.mode & kModeColPiece) != 0u;
    const bool per_piece = (M.mode & kModePerPiece) != 0u;
    if (col_piece) {
        // columns 4 lane .. 4 lane + 3: two words of two columns each per warp, flags in byte lane >> 1
        uint32_t m0 = 0u, m1 = 0u, n0 = 0xFFFFFFFFu, n1 = 0xFFFFFFFFu, f = 0u;
#pragma unroll
        for (int wp = 0; wp < kThreads / 32; ++wp) {
            m0 = __vimax3_u16x2(m0, S.cm[wp][2 * lane], S.cm[wp][2 * lane]);
            m1 = __vimax3_u16x2(m1, S.cm[wp][2 * lane + 1], S.cm[wp][2 * lane + 1]);
            n0 = __vimin3_u16x2(n0, S.cn[wp][2 * lane], S.cn[wp][2 * lane]);
            n1 = __vimin3_u16x2(n1, S.cn[wp][2 * lane + 1], S.cn[wp][2 * lane + 1]);
            f |= S.cf[wp][lane >> 1];
        }
        f >>= 4 * (lane & 1);
        uint4 kk;
        kk.x = ((m0 & 0xFFFFu) << 16) | (0xFFFFu - (n0 & 0xFFFFu)) | ((f & 1u) << 31);
        kk.y = ((m0 >> 16) << 16) | (0xFFFFu - (n0 >> 16)) | (((f >> 1) & 1u) << 31);
        kk.z = ((m1 & 0xFFFFu) << 16) | (0xFFFFu - (n1 & 0xFFFFu)) | (((f >> 2) & 1u) << 31);
        kk.w = ((m1 >> 16) << 16) | (0xFFFFu - (n1 >> 16)) | (((f >> 3) & 1u) << 31);
        *reinterpret_cast<uint4*>(M.col_keys + (size_t)local * kRowKeyStride + 4 * lane) = kk;
    }
    if (lane == 0) {
        uint32_t kk = S.wkey[0], nf = S.wnf[0], nz = S.wnz[0];
#pragma unroll
        for (int i = 1; i < kThreads / 32; ++i) { kk = key_max(kk, S.wkey[i]); nf += S.wnf[i]; nz += S.wnz[i]; }
        // finite non-zero elements of the tile (NaN and inf are non-zero patterns: taken off)
        if (has_keys) M.keys[(size_t)local * M.key_stride + (M.key_stride == (uint32_t)kRowKeyStride ? (uint32_t)kTileRows : 4u)] = nz - nf;
        if ((M.mode & kModeColsApart) != 0u) M.col_keys[(size_t)local * kRowKeyStride + kTileRows] = nz - nf;
        if ((M.mode & kModeBlk64) != 0u) {
            for (int q = 0; q < 4; ++q) {
                uint32_t kq = S.qkey[0][q], nq = S.qnf[0][q];
                for (int i = 1; i < kThreads / 32; ++i) { kq = key_max(kq, S.qkey[i][q]); nq |= S.qnf[i][q]; }
                M.keys[(size_t)local * kTileKeyStride + q] = kq | (nq ? 0x80000000u : 0u);
            }
        } else if (has_keys && !per_piece && !col_piece) {
            M.keys[(size_t)local * M.key_stride] = kk | (nf ? 0x80000000u : 0u);
        }
        // non-negative binary32 patterns order like the values
        const uint32_t amax_bits = (kk >> 16) << 16;
        if (M.ti != seen_ti) { seen_ti = M.ti; seen_amax = 0u; }
        if (amax_bits > seen_amax) {
            seen_amax = amax_bits;
            atomicMax(reinterpret_cast<unsigned int*>(bp.t[M.ti].amax_slot), amax_bits);
        }
    }
}

// The pre-pass kernel: persistent CTAs (two per SM) of 8 compute warps, a load warp and a tail warp.  One thread of
// the load warp streams the CTA's tiles (tile numbers blockIdx.x, + gridDim.x, ...) through a ring of three 32 KiB
// stages with TMA tile loads (zero fill past the tensor's edge), so that up to six tiles per SM are in flight
// whatever the compute warps are doing; a compute thread copies its eight 16-byte chunks of a landed tile to
// registers, the warp hands the stage back, reduces from the registers and leaves its results in one of two
// scratch areas; the tail warp combines the eight warps' results, writes the keys that span warps and raises the
// tensor amax, off the compute warps' path.  Every mbarrier wait is bounded; a wait that runs out sets the status
// word that the finalise kernel reports, and from then on the tail warp writes nothing.
constexpr int kAmaxStages = 3;
constexpr int kAmaxThreads = kThreads + 64;            // 8 compute warps, the load warp, the tail warp
constexpr int kAmaxStageBytes = kTileRows * kTileCols * 2;

struct AmaxControl {
    unsigned long long full[kAmaxStages];                // the tile has landed
    unsigned long long empty[kAmaxStages];               // the compute warps have their copies (one arrival per warp)
    AmaxMeta meta[kAmaxStages];                          // by the load warp, before the stage's copy is started
    volatile uint32_t abort;
    uint32_t issued;
    AmaxShared S[2];
};
constexpr int kAmaxSmemBytes = 1024 + kAmaxStages * kAmaxStageBytes + (int)sizeof(AmaxControl);
static_assert(2 * (kAmaxSmemBytes + 1024) <= 228 * 1024, "two CTAs per SM must fit in shared memory");

template <bool ROWS_ONLY>
__global__ void __launch_bounds__(kAmaxThreads, 2)
mor_amax_kernel(const __grid_constant__ MainParams p)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char* in = smem_raw + ((1024u - (smem_addr(smem_raw) & 1023u)) & 1023u);
    AmaxControl& C = *reinterpret_cast<AmaxControl*>(in + kAmaxStages * kAmaxStageBytes);
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    if (t == 0) {
        for (int s = 0; s < kAmaxStages; ++s) { mbar_init(&C.full[s], 1); mbar_init(&C.empty[s], kThreads / 32); }
        C.abort = 0u;
        C.issued = 0u;
        fence_mbar_init();
    }
    __syncthreads();
    pdl_trigger();                                       // the main kernel may move in as this kernel's CTAs leave
    const uint32_t n_it = (p.total_tiles - blockIdx.x + gridDim.x - 1u) / gridDim.x;

    if (warp == kThreads / 32) {
        // ---- load warp: one thread issues, the others leave ----
        if (lane != 0) return;
        // what changes only with the tensor is kept in registers: the CTA's tile numbers only grow, so the search for
        // a tile's tensor goes forward from the last one (reads of the records in the parameter space are slow)
        int ti = -1;
        uint32_t begin = 0u, end = 0u, nbc = 1u;
        AmaxMeta m;
        m.ti = 0; m.local = 0u; m.mode = 0u; m.key_stride = 0u; m.keys = nullptr; m.col_keys = nullptr;
#pragma unroll 1
        for (uint32_t it = 0; it < n_it; ++it) {
            const uint32_t s = it % kAmaxStages, tile = blockIdx.x + it * gridDim.x;
            if (ti < 0 || (tile >= end && ti < p.b.n - 1)) {
                if (ti < 0) { ti = 0; end = p.b.tile_end[0]; }
                while (tile >= end && ti < p.b.n - 1) { begin = end; ++ti; end = p.b.tile_end[ti]; }
                const TensorRec& R = p.b.t[ti];
                nbc = R.nbc;
                m.ti = ti; m.key_stride = R.key_stride; m.keys = R.keys; m.col_keys = R.col_keys;
                const bool cols = m.col_keys != nullptr;
                m.mode = (m.keys != nullptr ? kModeKeys : 0u) |
                         (m.keys != nullptr && m.key_stride == (uint32_t)kRowKeyStride && m.col_keys != m.keys ? kModePerPiece : 0u) |
                         (cols ? kModeColPiece : 0u) | (m.keys != nullptr && R.kind == KIND_BLK64 ? kModeBlk64 : 0u) |
                         (cols && m.col_keys != m.keys ? kModeColsApart : 0u);
            }
            if (it >= (uint32_t)kAmaxStages &&
                !mbar_wait(&C.empty[s], (it / kAmaxStages - 1u) & 1u, &C.abort, p.wait_cycles)) {
                C.abort = 1u;
                atomicOr(p.device_status, 1u);
                break;
            }
            m.local = tile - begin;
            const uint32_t bi = m.local / nbc, bj = m.local - bi * nbc;
            C.meta[s] = m;                               // (made visible by the arrival below)
            // (test hook: the load of one chosen tile is left out, so that the waits for it run out)
            if (tile != p.test_skip_tile) {
                mbar_arrive_expect_tx(&C.full[s], (uint32_t)kAmaxStageBytes);
                tma_load_tile(in + s * kAmaxStageBytes, &p.in_map[ti], (int)(bj * kTileCols), (int)(bi * kTileRows), &C.full[s]);
            }
            C.issued = it + 1u;
        }
        if (C.abort) {
            // copies that may still be in flight must land (or be given up on) before the CTA goes
            const uint32_t issued = C.issued;
            for (uint32_t k = 0; k < (uint32_t)kAmaxStages && k < issued; ++k) {
                const uint32_t it = issued - 1u - k;
                mbar_wait(&C.full[it % kAmaxStages], (it / kAmaxStages) & 1u, nullptr, p.wait_cycles);
            }
        }
        return;
    }

    if (warp == kThreads / 32 + 1) {
        // ---- tail warp ----
        int seen_ti = -1;
        uint32_t seen_amax = 0u;
#pragma unroll 1
        for (uint32_t it = 0; it < n_it; ++it) {
            const uint32_t b = it & 1u;
            scratch_full_sync(b);
            if (!C.abort) amax_tail(p.b, C.S[b], lane, seen_ti, seen_amax);
            __syncwarp();
            if (it + 2u < n_it) scratch_free_arrive(b);      // (the last two have no taker)
        }
        return;
    }

    // ---- compute warps ----
    bool dead = false;
    const uint32_t off = (uint32_t)((t >> 4) * 256 + (t & 15) * 16);
    const uint32_t off_row = (uint32_t)((t >> 1) * 256 + (t & 1) * 128 + ((((t >> 1) & 7) ^ ((t & 1) << 2)) << 4));
    const uint32_t in_base = smem_addr(in);
#pragma unroll 1
    for (uint32_t it = 0; it < n_it; ++it) {
        const uint32_t s = it % kAmaxStages, b = it & 1u;
        if (!dead) {
            bool ok = mbar_wait(&C.full[s], (it / kAmaxStages) & 1u, &C.abort, p.wait_cycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) {
                dead = true;
                if (lane == 0) { C.abort = 1u; atomicOr(p.device_status, 1u); }
            }
        }
        uint4 v[8], m0, m1;
        if (!dead) {
            m0 = lds128(smem_addr(&C.meta[s]));
            m1 = lds128(smem_addr(&C.meta[s]) + 16u);
            const uint32_t a = in_base + s * (uint32_t)kAmaxStageBytes;
            if (ROWS_ONLY) {
                // row keys alone: thread (row t >> 1, half t & 1) takes the eight chunks of its 128 bytes, in an order
                // that keeps the lanes of a load phase on distinct banks
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = lds128((a + off_row) ^ (uint32_t)(j << 4));
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = lds128(a + off + (uint32_t)(j * 16 * 256));
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&C.empty[s]);         // this warp's copies are in registers
        if (it >= 2u) scratch_free_sync(b);              // the tail warp has read what tile it - 2 left in this scratch
        if (!dead) {
            AmaxMeta M;
            M.ti = (int32_t)m0.x; M.local = m0.y; M.mode = m0.z; M.key_stride = m0.w;
            M.keys = reinterpret_cast<uint32_t*>(((unsigned long long)m1.y << 32) | m1.x);
            M.col_keys = reinterpret_cast<uint32_t*>(((unsigned long long)m1.w << 32) | m1.z);
            amax_thread_part<ROWS_ONLY>(M, v, C.S[b]);
        }
        scratch_full_arrive(b);
    }
}

// Per-channel partition: a block is a whole row (a whole column), so its key is the combination of the keys of the
// row's 128-element pieces over all tiles of the tile row (of the column's pieces over all tiles of the tile column).
// One CTA of 128 threads per (tile row or tile column, tensor).
__global__ void __launch_bounds__(kTileRows)
mor_row_keys_kernel(const __grid_constant__ BatchParams p)
{
    pdl_trigger();
    const TensorRec& R = p.t[blockIdx.y];
    const bool cols = R.kind == KIND_COLCH;
    if ((R.kind != KIND_CHANNEL && !cols) || R.row_keys == nullptr || blockIdx.x >= (cols ? R.nbc : R.nbr)) return;
    const uint32_t n = cols ? R.nbr : R.nbc;
    const size_t first = cols ? (size_t)blockIdx.x : (size_t)blockIdx.x * R.nbc, stride = cols ? (size_t)R.nbc : 1u;
    const uint32_t* src = R.keys + first * kRowKeyStride + threadIdx.x;
    uint32_t k = 0u, flag = 0u;
    for (uint32_t j = 0; j < n; ++j, src += stride * kRowKeyStride) {
        const uint32_t v = *src;
        flag |= v & 0x80000000u;
        k = key_max(k, v & 0x7FFFFFFFu);
    }
    R.row_keys[(size_t)blockIdx.x * kTileRows + threadIdx.x] = k | flag;
}

// Per-channel partition with a per-row decision (Algorithm 2 with one block per row) or per-row statistics: the
// row's sums are the sums of its tiles' parts, added in tile order in double (likewise for whole columns).  One CTA
// of 128 threads per (tile row or tile column, tensor); writes sel, block statistics and, into the partial of the
// line of tiles' first tile, the counts of rows (columns) per format, which the finalise kernel adds up.
__global__ void __launch_bounds__(kTileRows)
mor_row_decide_kernel(const __grid_constant__ BatchParams p, Partial* __restrict__ partials)
{
    __shared__ uint32_t s_n4[kTileRows / 32], s_nb[kTileRows / 32];
    pdl_wait();                                          // the main kernel's row parts are complete
    const TensorRec& R = p.t[blockIdx.y];
    const bool cols = R.kind == KIND_COLCH;              // blocks are whole columns: `row` below is a column
    if ((R.kind != KIND_CHANNEL && !cols) || R.row_part == nullptr || blockIdx.x >= (cols ? R.nbc : R.nbr)) return;
    const long long row = (long long)blockIdx.x * kTileRows + threadIdx.x;
    const bool valid = row < (cols ? R.cols : R.rows);
    const uint32_t n = cols ? R.nbr : R.nbc;
    const size_t first = cols ? (size_t)blockIdx.x : (size_t)blockIdx.x * R.nbc, stride = cols ? (size_t)R.nbc : 1u;
    double s43 = 0.0, s52 = 0.0;
    uint32_t nnz = 0u, nonf = 0u;
    if (valid) {
        const float4* src = R.row_part + first * kTileRows + threadIdx.x;
        for (uint32_t j = 0; j < n; ++j, src += stride * kTileRows) {
            const float4 v = *src;
            const uint32_t nz = __float_as_uint(v.z);
            s43 += (double)v.x; s52 += (double)v.y; nnz += nz & 0xFFFFu; nonf += nz >> 16;
        }
    }
    uint32_t sel = MOR_FMT_E4M3;
    if (valid) {
        if (nonf) sel = MOR_FMT_BF16;
        else if (R.criterion == MOR_CRIT_BLOCK_VS_E5M2) {
            const bool ok = (R.flags & MOR_FLAG_STRICT_TIES) ? (s43 < s52) : (s43 <= s52);
            sel = ok ? MOR_FMT_E4M3 : MOR_FMT_BF16;
        } else if (R.criterion == MOR_CRIT_BLOCK_MEAN_REL) {
            const double err = nnz ? s43 / (double)nnz : 0.0;
            sel = err < (double)R.threshold ? MOR_FMT_E4M3 : MOR_FMT_BF16;
        }
        if (R.criterion != MOR_CRIT_TENSOR_MEAN_REL && R.sel) R.sel[row] = (uint8_t)sel;   // (tensor-level: filled by the finalise kernel)
        if (R.block_stats) {
            const uint32_t key = R.row_keys[row] & 0x7FFFFFFFu;
            mor_block_stats_t bs;
            bs.amax = __uint_as_float((key >> 16) << 16);
            bs.min_abs_nz = __uint_as_float(0x7F800000u);           // kept for three formats only, which this partition does not take
            bs.nnz = nnz; bs.n_nonfinite = nonf;
            bs.sum_rel_e4m3 = (float)s43; bs.sum_rel_e5m2 = (float)s52;
            R.block_stats[row] = bs;
        }
    }
    if (R.criterion != MOR_CRIT_TENSOR_MEAN_REL) {
        const uint32_t b4 = __ballot_sync(0xFFFFFFFFu, valid && sel == MOR_FMT_E4M3), bb = __ballot_sync(0xFFFFFFFFu, valid && sel == MOR_FMT_BF16);
        if ((threadIdx.x & 31) == 0) { s_n4[threadIdx.x >> 5] = __popc(b4); s_nb[threadIdx.x >> 5] = __popc(bb); }
        __syncthreads();
        if (threadIdx.x == 0) {
            Partial& P = partials[R.tile_begin + first];
            P.n_e4m3 = s_n4[0] + s_n4[1] + s_n4[2] + s_n4[3];
            P.n_e5m2 = 0u;
            P.n_bf16 = s_nb[0] + s_nb[1] + s_nb[2] + s_nb[3];
        }
    }
}

// ----------------------------------------------------------------------- finalise ----

// One CTA per (tensor, slice).  Every slice repeats the reduction over the tensor's tile
// partials in the same order, so all slices agree; slice 0 writes the summary.  With the
// tensor-level criterion the slices share the work of filling the per-block selection.
template <int KIND>
__global__ void __launch_bounds__(kThreads)
mor_finalise_kernel(const __grid_constant__ BatchParams p, const Partial* __restrict__ partials)
{
    __shared__ WarpPart s_wp[kThreads / 32];
    pdl_wait();                                          // the main kernel's partials and outputs are complete
    const TensorRec& R = p.t[blockIdx.x];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;

    WarpPart a;
    a.s43 = a.s52 = 0.0; a.nnz = a.nonfinite = a.n4 = a.n5 = a.nb = 0u; a.mn = 0xFFFFu;
    unsigned long long nnz64 = 0, nonf64 = 0, n4 = 0, n5 = 0, nb = 0;
    for (uint32_t i = t; i < R.n_tiles; i += kThreads) {
        const Partial P = partials[R.tile_begin + i];
        a.s43 += P.sum43; a.s52 += P.sum52;
        nnz64 += P.nnz; nonf64 += P.nonfinite; n4 += P.n_e4m3; n5 += P.n_e5m2; nb += P.n_bf16;
        a.mn = min(a.mn, P.min_nz_bits);
    }
    a.s43 = warp_sum(a.s43);
    a.s52 = warp_sum(a.s52);
    a.mn = __reduce_min_sync(0xFFFFFFFFu, a.mn);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        nnz64 += __shfl_xor_sync(0xFFFFFFFFu, nnz64, o);
        nonf64 += __shfl_xor_sync(0xFFFFFFFFu, nonf64, o);
        n4 += __shfl_xor_sync(0xFFFFFFFFu, n4, o);
        n5 += __shfl_xor_sync(0xFFFFFFFFu, n5, o);
        nb += __shfl_xor_sync(0xFFFFFFFFu, nb, o);
    }
    __shared__ unsigned long long s_cnt[kThreads / 32][5];
    if (lane == 0) {
        s_wp[warp] = a;
        s_cnt[warp][0] = nnz64; s_cnt[warp][1] = nonf64; s_cnt[warp][2] = n4; s_cnt[warp][3] = n5; s_cnt[warp][4] = nb;
    }
    __syncthreads();
    __shared__ uint32_t s_fmt;
    if (t == 0) {
        WarpPart tot = s_wp[0];
        unsigned long long c[5] = {s_cnt[0][0], s_cnt[0][1], s_cnt[0][2], s_cnt[0][3], s_cnt[0][4]};
        for (int i = 1; i < kThreads / 32; ++i) {
            tot.s43 += s_wp[i].s43; tot.s52 += s_wp[i].s52; tot.mn = min(tot.mn, s_wp[i].mn);
            for (int j = 0; j < 5; ++j) c[j] += s_cnt[i][j];
        }
        const float g_amax = *R.amax;
        const uint32_t m_g = group_mantissa(g_amax, R.scale_mode);
        // Eq. 2: mean over the non-zeros of the tensor, strict '<'
        const double mean = c[0] ? tot.s43 / (double)c[0] : 0.0;
        const uint32_t fmt = (c[1] == 0 && mean < (double)R.threshold) ? MOR_FMT_E4M3 : MOR_FMT_BF16;
        unsigned long long n_blocks = (KIND == KIND_TENSOR) ? (R.n_tiles ? 1ull : 0ull) : R.n_units;
        uint32_t bsel = fmt;
        if (KIND == KIND_TENSOR) {
            if (R.criterion == MOR_CRIT_BLOCK_VS_E5M2) {
                const bool ok = (R.flags & MOR_FLAG_STRICT_TIES) ? (tot.s43 < tot.s52) : (tot.s43 <= tot.s52);
                bsel = (c[1] == 0 && ok) ? MOR_FMT_E4M3 : MOR_FMT_BF16;
            }
            c[2] = (n_blocks && bsel == MOR_FMT_E4M3); c[3] = 0; c[4] = (n_blocks && bsel == MOR_FMT_BF16);
            if (n_blocks && blockIdx.y == 0) {
                uint32_t s4b, s5b;
                const float b_amax = *R.amax_slot;
                block_scale(b_amax, m_g, R.scale_mode, s4b, s5b);
                if (R.sel) R.sel[0] = (uint8_t)bsel;
                if (R.scale_e8m0) R.scale_e8m0[0] = (uint8_t)(s4b >> 23);
                if (R.scale_f32) R.scale_f32[0] = __uint_as_float(s4b);
                if (R.block_stats) {
                    mor_block_stats_t bs;
                    bs.amax = b_amax;
                    bs.min_abs_nz = minnz_value(tot.mn);
                    bs.nnz = (uint32_t)(c[0] > 0xFFFFFFFFull ? 0xFFFFFFFFull : c[0]);
                    bs.n_nonfinite = (uint32_t)(c[1] > 0xFFFFFFFFull ? 0xFFFFFFFFull : c[1]);
                    bs.sum_rel_e4m3 = (float)tot.s43; bs.sum_rel_e5m2 = (float)tot.s52;
                    R.block_stats[0] = bs;
                }
            }
        } else if (R.criterion == MOR_CRIT_TENSOR_MEAN_REL) {
            c[2] = fmt == MOR_FMT_E4M3 ? n_blocks : 0; c[3] = 0; c[4] = fmt == MOR_FMT_BF16 ? n_blocks : 0;
        }
        if (blockIdx.y == 0) {
            mor_tensor_stats_t ts;
            ts.sum_rel_e4m3 = tot.s43; ts.nnz = c[0]; ts.mean_rel_e4m3 = mean;
            ts.group_amax = g_amax; ts.group_mantissa = m_g; ts.tensor_format = fmt;
            ts.status = *R.device_status ? MOR_ERR_TIMEOUT : MOR_OK;
            ts.n_blocks = n_blocks; ts.n_e4m3 = c[2]; ts.n_e5m2 = c[3]; ts.n_bf16 = c[4]; ts.n_nonfinite = c[1];
            *R.tensor_stats = ts;
            if (R.hist) {
                // Section 4.1.3: bins of 0.5 % of relative error, the last one open-ended
                uint32_t bin = 0;
                while (bin < MOR_ERROR_BINS - 1 && mean >= 0.005 * (double)(bin + 1)) ++bin;
                atomicAdd(&R.hist[bin], 1u);
            }
        }
        s_fmt = fmt;
    }
    __syncthreads();
    if (KIND != KIND_TENSOR && R.criterion == MOR_CRIT_TENSOR_MEAN_REL && R.sel) {
        const uint8_t f = (uint8_t)s_fmt;
        const unsigned long long n = R.n_units;
        for (unsigned long long i = (unsigned long long)blockIdx.y * kThreads + t; i < n;
             i += (unsigned long long)gridDim.y * kThreads)
            R.sel[i] = f;
    }
}

}  // namespace

template <bool ROWS_ONLY>
cudaError_t launch_amax_t(const MainParams& p, cudaStream_t s)
{
    auto kfn = mor_amax_kernel<ROWS_ONLY>;
    static std::atomic<int> sm_count[64];   // per instantiation and device; 0 = not set up yet
    static std::mutex setup;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int sms = sm_count[dev].load(std::memory_order_acquire);
    if (sms == 0) {
        std::lock_guard<std::mutex> lock(setup);         // host threads may make their first call together
        e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, kAmaxSmemBytes);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (sms <= 0) return cudaErrorInvalidDevice;
        sm_count[dev].store(sms, std::memory_order_release);
    }
    const uint32_t resident = 2u * (uint32_t)sms;
    const uint32_t grid = p.total_tiles < resident ? p.total_tiles : resident;
    kfn<<<grid, kAmaxThreads, kAmaxSmemBytes, s>>>(p);
    return cudaGetLastError();
}

// rows_only: every tensor of the launch wants one key per row piece and nothing else (1x128 blocks or per-channel
// rows, not paired with column blocks); the general instantiation serves every mix.
cudaError_t launch_amax(const MainParams& p, bool rows_only, cudaStream_t s)
{
    if (p.total_tiles == 0) return cudaSuccess;
    return rows_only ? launch_amax_t<true>(p, s) : launch_amax_t<false>(p, s);
}

cudaError_t launch_row_keys(const BatchParams& p, cudaStream_t s)
{
    uint32_t nbr = 0;
    for (int i = 0; i < p.n; ++i) {
        if (p.t[i].kind == KIND_CHANNEL && p.t[i].nbr > nbr) nbr = p.t[i].nbr;
        if (p.t[i].kind == KIND_COLCH && p.t[i].nbc > nbr) nbr = p.t[i].nbc;
    }
    if (nbr == 0) return cudaSuccess;
    mor_row_keys_kernel<<<dim3(nbr, (unsigned)p.n), kTileRows, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_row_decide(const BatchParams& p, Partial* partials, int kind, cudaStream_t s)
{
    uint32_t nbr = 0;
    for (int i = 0; i < p.n; ++i) {
        if (p.t[i].kind != kind || p.t[i].row_part == nullptr) continue;
        const uint32_t lines = kind == KIND_COLCH ? p.t[i].nbc : p.t[i].nbr;
        if (lines > nbr) nbr = lines;
    }
    if (nbr == 0) return cudaSuccess;
    return launch_dependent(mor_row_decide_kernel, dim3(nbr, (unsigned)p.n), dim3(kTileRows), 0, s, p, partials);
}

cudaError_t launch_finalise(const BatchParams& p, const Partial* partials, int kind, cudaStream_t s)
{
    if (p.n == 0) return cudaSuccess;
    // slices only help when the selection array has to be filled for a tensor-level decision
    unsigned slices = 1;
    for (int i = 0; i < p.n; ++i)
        if (kind != KIND_TENSOR && p.t[i].criterion == MOR_CRIT_TENSOR_MEAN_REL && p.t[i].sel && p.t[i].n_units > 65536u) slices = 16;
    dim3 grid((unsigned)p.n, slices);
    cudaError_t e = cudaSuccess;
    switch (kind) {
        case KIND_TENSOR: e = launch_dependent(mor_finalise_kernel<KIND_TENSOR>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_ROW128: e = launch_dependent(mor_finalise_kernel<KIND_ROW128>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_BLK128: e = launch_dependent(mor_finalise_kernel<KIND_BLK128>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_BLK64: e = launch_dependent(mor_finalise_kernel<KIND_BLK64>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_CHANNEL: e = launch_dependent(mor_finalise_kernel<KIND_CHANNEL>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_COL128: e = launch_dependent(mor_finalise_kernel<KIND_COL128>, grid, dim3(kThreads), 0, s, p, partials); break;
        case KIND_COLCH: e = launch_dependent(mor_finalise_kernel<KIND_COLCH>, grid, dim3(kThreads), 0, s, p, partials); break;
        default: return cudaErrorInvalidValue;
    }
    return e;
}

}  // namespace mor
