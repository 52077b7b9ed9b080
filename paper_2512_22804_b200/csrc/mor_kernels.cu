// Hand-written sm_100a kernels of the MoR analyse-and-quantise pass.
//
//   mor_amax_kernel      Algorithm 1, "g_amax <- max(abs(g))" with the tensor as one group
//   mor_main_kernel      per tile: block amax and GAM scale (Algorithm 1), cast to E4M3 and
//                        E5M2, relative-error sums (Eq. 1-3), range statistics (Eq. 4),
//                        per-block decision (Algorithm 2), packed stores
//   mor_finalise_kernel  tensor-wide aggregate and Eq. 2 decision
//
// Data movement per tile (128 segments x 128 BF16 = 32 KiB): 16-byte cp.async copies with
// zero fill for the ragged edge bring the tile into shared memory once; two threads own
// each segment and read it back conflict-free (the chunk order is rotated by the thread
// index); codes are staged in shared memory and leave as 16-byte coalesced stores.
//
// Arithmetic that must be exact: amax (integer compare of BF16 bit patterns), the scale
// (one IEEE binary32 division), the scaled value (one IEEE binary32 multiply) and the
// FP8 codes (cvt.rn.satfinite).  The error ratio uses an approximate reciprocal; it only
// feeds sums that are compared with a tolerance.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <float.h>

#include "mor_internal.h"

namespace mor {
namespace {

constexpr int kInBytes = kSegsPerTile * kSegElems * 2;   // 32768
constexpr int kOutBytes = kSegsPerTile * kSegElems;      // 16384
constexpr uint32_t kBf16Inf = 0x7F80u;

struct WarpPart {
    double s43, s52;
    uint32_t nnz, nonfinite, n4, n5, nb, mn;
};

struct TileShared {
    long long seg_off[kSegsPerTile];    // element offset of the segment's first element in x
    long long seg_coff[kSegsPerTile];   // byte offset of its first code
    int seg_n[kSegsPerTile];            // valid elements of the segment (0..128)
    WarpPart wp[kThreads / 32];
    uint32_t wmax[kThreads / 32];
    uint32_t bcast[4];
    uint8_t blk_sel[kSegsPerTile];
};

constexpr int kSmemBytes = kInBytes + kOutBytes + (int)sizeof(TileShared);

// ------------------------------------------------------------------ small helpers ----

__device__ __forceinline__ uint32_t smem_addr(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte asynchronous copy global -> shared; bytes past `src_bytes` are written as zero.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait_all()
{
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ uint4 lds128(const unsigned char* p) { return *reinterpret_cast<const uint4*>(p); }

// {hi, lo} -> two E4M3 codes, `lo` in the low byte (round to nearest even, saturate to 448).
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
// two E4M3 codes -> f16x2 (exact: every E4M3 value is a binary16 number)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t c)
{
    uint32_t r;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(static_cast<uint16_t>(c)));
    return r;
}
// an E5M2 code is the upper byte of the binary16 with the same value
__device__ __forceinline__ uint32_t e5m2x2_to_f16x2(uint32_t c) { return __byte_perm(c, 0u, 0x1404); }

// q (binary16) - y (binary32) in one binary32 operation; exact here because q is the FP8
// neighbour of y
__device__ __forceinline__ float diff_f16_f32(uint16_t q, float y)
{
    float d;
    asm("sub.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(q), "f"(y));
    return d;
}

__device__ __forceinline__ float rcp_approx(float a)
{
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// "ideal FP32 scaling factor" 448 / amax: one IEEE division; a quotient above the largest
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

__device__ __forceinline__ int find_tensor(const BatchParams& p, uint32_t tile, uint32_t& local)
{
    int ti = 0;
    uint32_t begin = 0;
#pragma unroll 1
    while (ti < p.n - 1 && tile >= p.tile_end[ti]) { begin = p.tile_end[ti]; ++ti; }
    local = tile - begin;
    return ti;
}

// Where segment `s` of tile `local` lives.  BLK128: row s of block `local`.  Otherwise the
// segments are the 128-element pieces of the rows in row-major order.
template <int KIND>
__device__ __forceinline__ void seg_geometry(const TensorRec& R, uint32_t local, int s,
                                             long long& off, long long& coff, int& n)
{
    long long row, cb;
    bool valid;
    if (KIND == KIND_BLK128) {
        const uint32_t bi = local / R.nbc, bj = local - bi * R.nbc;
        row = (long long)bi * 128 + s;
        cb = bj;
        valid = row < R.rows;
    } else {
        const uint32_t u = local * (uint32_t)kSegsPerTile + (uint32_t)s;
        const uint32_t r = u / R.nbc;
        row = r;
        cb = u - r * R.nbc;
        valid = u < R.n_units;
    }
    const long long c0 = cb * kSegElems;
    const long long left = R.cols - c0;
    n = valid ? (int)(left < kSegElems ? left : kSegElems) : 0;
    off = valid ? row * R.ld + c0 : 0;
    coff = valid ? row * R.codes_ld + c0 : 0;
}

__device__ __forceinline__ void load_tile_async(const TensorRec& R, const TileShared& sh, unsigned char* s_in, int t)
{
    const uint32_t base = smem_addr(s_in);
    const int k = t & 15;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int seg = (t >> 4) + 16 * j;
        int bytes = (sh.seg_n[seg] - 8 * k) * 2;
        bytes = bytes < 0 ? 0 : (bytes > 16 ? 16 : bytes);
        const uint16_t* src = R.x + (bytes > 0 ? sh.seg_off[seg] + 8 * k : 0);
        cp_async16(base + seg * 256 + k * 16, src, bytes);
    }
}

// max over |x| of a thread's 64 elements as BF16 bits; NaN and inf win (they compare above
// every finite pattern), which is how a non-finite input is noticed
__device__ __forceinline__ uint32_t raw_amax_half_segment(const unsigned char* half, int t)
{
    __nv_bfloat162 m = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 v = lds128(half + (((j + t) & 7) << 4));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&w[i]);
            m = __hmax2_nan(m, __habs2(a));
        }
    }
    const uint32_t mb = *reinterpret_cast<const uint32_t*>(&m);
    return max(mb & 0xFFFFu, mb >> 16);
}

// the same over finite elements only (used once a non-finite element has been seen)
__device__ __forceinline__ uint32_t finite_amax_half_segment(const unsigned char* half, int t)
{
    uint32_t m = 0;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        const uint4 v = lds128(half + (((j + t) & 7) << 4));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
            if (lo < kBf16Inf) m = max(m, lo);
            if (hi < kBf16Inf) m = max(m, hi);
        }
    }
    return m;
}

struct Acc {
    float a43[4], a52[4];
    uint32_t nnz, nbig, nonfinite, mn;   // mn: min over non-zeros of (|x| bits << 16) - 1
};

// One BF16 pair -> two E4M3 codes (and two E5M2 codes), with its terms of Eq. 1-3.
//   y = fl32(x * scale); c = RNE-saturating cast; q = value of c; term = |y - q| / |y|.
// Terms are accumulated only where |y| is a normal binary32; the few non-zero elements
// below that (they are flushed by both formats, term = 1) are added from the counts
// nnz - nbig by the caller.
template <bool YARD, bool THREE, bool SLOW>
__device__ __forceinline__ void convert_pair(uint32_t w, float s4, float s5, int lane, Acc& A,
                                             uint32_t& c4, uint32_t& c5)
{
    const uint32_t blo = w << 16, bhi = w & 0xFFFF0000u;
    const uint32_t alo = blo & 0x7FFFFFFFu, ahi = bhi & 0x7FFFFFFFu;
    const float xlo = __uint_as_float(blo), xhi = __uint_as_float(bhi);
    bool uselo = true, usehi = true;
    if (SLOW) {
        uselo = alo < 0x7F800000u;
        usehi = ahi < 0x7F800000u;
        A.nonfinite += (uselo ? 0u : 1u) + (usehi ? 0u : 1u);
    }
    A.nnz += ((alo != 0u && uselo) ? 1u : 0u) + ((ahi != 0u && usehi) ? 1u : 0u);
    if (THREE) {
        if (uselo) A.mn = min(A.mn, alo - 1u);
        if (usehi) A.mn = min(A.mn, ahi - 1u);
    }

    const float ylo = __fmul_rn(xlo, s4), yhi = __fmul_rn(xhi, s4);
    c4 = cvt_e4m3x2(yhi, ylo);
    const uint32_t q4 = e4m3x2_to_f16x2(c4);
    const float dlo = diff_f16_f32(static_cast<uint16_t>(q4 & 0xFFFFu), ylo);
    const float dhi = diff_f16_f32(static_cast<uint16_t>(q4 >> 16), yhi);
    const float aylo = fabsf(ylo), ayhi = fabsf(yhi);
    const bool biglo = (aylo >= FLT_MIN) && uselo, bighi = (ayhi >= FLT_MIN) && usehi;
    const float rlo = rcp_approx(aylo), rhi = rcp_approx(ayhi);
    if (biglo) { A.a43[lane] = fmaf(fabsf(dlo), rlo, A.a43[lane]); A.nbig++; }
    if (bighi) { A.a43[lane] = fmaf(fabsf(dhi), rhi, A.a43[lane]); A.nbig++; }

    if (YARD) {
        const float zlo = __fmul_rn(xlo, s5), zhi = __fmul_rn(xhi, s5);
        c5 = cvt_e5m2x2(zhi, zlo);
        const uint32_t q5 = e5m2x2_to_f16x2(c5);
        const float elo = diff_f16_f32(static_cast<uint16_t>(q5 & 0xFFFFu), zlo);
        const float ehi = diff_f16_f32(static_cast<uint16_t>(q5 >> 16), zhi);
        // |z - q'| / |z| = |z - q'| * (1/|y|) * (scale4/scale5); the power-of-two ratio is
        // applied once per block
        if (biglo) A.a52[lane] = fmaf(fabsf(elo), rlo, A.a52[lane]);
        if (bighi) A.a52[lane] = fmaf(fabsf(ehi), rhi, A.a52[lane]);
    } else {
        c5 = 0;
    }

    if (SLOW) {
        // stated reading for non-finite inputs: NaN -> 0x7F, +-inf -> +-largest finite
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
}

// A thread's 64 elements.  E4M3 codes go to shared memory at once unless the recipe is
// three-way, where both code sets wait in registers for the block's decision.
template <bool YARD, bool THREE, bool SLOW, bool STORE>
__device__ __forceinline__ void convert_half_segment(const unsigned char* half_in, unsigned char* half_out, int t,
                                                     float s4, float s5, Acc& A, uint2 (&k4)[8], uint2 (&k5)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int kk = (j + t) & 7;
        const uint4 v = lds128(half_in + (kk << 4));
        uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
        convert_pair<YARD, THREE, SLOW>(v.x, s4, s5, 0, A, a0, b0);
        convert_pair<YARD, THREE, SLOW>(v.y, s4, s5, 1, A, a1, b1);
        convert_pair<YARD, THREE, SLOW>(v.z, s4, s5, 2, A, a2, b2);
        convert_pair<YARD, THREE, SLOW>(v.w, s4, s5, 3, A, a3, b3);
        const uint2 c4 = make_uint2(a0 | (a1 << 16), a2 | (a3 << 16));
        if (THREE) {
            k4[j] = c4;
            k5[j] = make_uint2(b0 | (b1 << 16), b2 | (b3 << 16));
        } else if (STORE) {
            *reinterpret_cast<uint2*>(half_out + (kk << 3)) = c4;
        }
    }
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Algorithm 2 for one block with the per-block metrics (M_1 = Eq. 3, M_2 = Eq. 4, or
// Eq. 1-2 on the block alone).
__device__ __forceinline__ uint32_t decide_block(const TensorRec& R, double e43, double e52, uint32_t nnz,
                                                 uint32_t nonfinite, uint32_t amax_bits, uint32_t mn,
                                                 uint32_t n_elems)
{
    if (nonfinite) return MOR_FMT_BF16;
    if (R.criterion == MOR_CRIT_BLOCK_VS_E5M2) {
        const bool ok = (R.flags & MOR_FLAG_STRICT_TIES) ? (e43 < e52) : (e43 <= e52);
        if (ok) return MOR_FMT_E4M3;
        if (R.n_formats == 3) {
            // max|b| < (57344 * 2^14) * min|b|, exact in binary32 (11 significant bits)
            float mnv = (mn == 0xFFFFFFFFu) ? __uint_as_float(0x7F800000u) : __uint_as_float(mn + 1u);
            if ((R.flags & MOR_FLAG_RANGE_MIN_INCLUDES_ZERO) && nnz < n_elems) mnv = 0.0f;
            const float amax = __uint_as_float(amax_bits << 16);
            if (amax < 939524096.0f * mnv) return MOR_FMT_E5M2;
        }
        return MOR_FMT_BF16;
    }
    if (R.criterion == MOR_CRIT_BLOCK_MEAN_REL) {
        const double err = nnz ? e43 / (double)nnz : 0.0;
        return err < (double)R.threshold ? MOR_FMT_E4M3 : MOR_FMT_BF16;
    }
    return MOR_FMT_E4M3;   // tensor-level criterion: decided by the finalise kernel
}

// ---------------------------------------------------------------------- main kernel ----

template <int KIND, bool YARD, bool THREE, bool STORE>
__global__ void __launch_bounds__(kThreads, 3)
mor_main_kernel(const __grid_constant__ BatchParams p, Partial* __restrict__ partials)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* s_in = smem;
    unsigned char* s_out = smem + kInBytes;
    TileShared& sh = *reinterpret_cast<TileShared*>(smem + kInBytes + kOutBytes);

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    uint32_t local;
    const TensorRec& R = p.t[find_tensor(p, blockIdx.x, local)];

    if (t < kSegsPerTile) seg_geometry<KIND>(R, local, t, sh.seg_off[t], sh.seg_coff[t], sh.seg_n[t]);
    __syncthreads();
    load_tile_async(R, sh, s_in, t);

    // Algorithm 1, group part (every thread: one division, overlapped with the copy)
    const float g_amax = *R.amax;
    const uint32_t m_g = group_mantissa(g_amax, R.scale_mode);

    cp_async_commit_wait_all();
    __syncthreads();

    const int seg = t >> 1;
    const unsigned char* half_in = s_in + seg * 256 + (t & 1) * 128;
    unsigned char* half_out = s_out + seg * 128 + (t & 1) * 64;

    // ---- block amax (Algorithm 1) ----
    uint32_t amax_bits = raw_amax_half_segment(half_in, t);
    bool slow;
    if (KIND == KIND_ROW128) {
        amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, 1));
        slow = __any_sync(0xFFFFFFFFu, amax_bits >= kBf16Inf);
        if (slow) {
            amax_bits = finite_amax_half_segment(half_in, t);
            amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, 1));
        }
    } else {
        amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
        if (lane == 0) sh.wmax[warp] = amax_bits;
        __syncthreads();
        amax_bits = sh.wmax[0];
#pragma unroll
        for (int i = 1; i < kThreads / 32; ++i) amax_bits = max(amax_bits, sh.wmax[i]);
        slow = amax_bits >= kBf16Inf;
        if (slow) {                                         // CTA-uniform
            __syncthreads();
            amax_bits = __reduce_max_sync(0xFFFFFFFFu, finite_amax_half_segment(half_in, t));
            if (lane == 0) sh.wmax[warp] = amax_bits;
            __syncthreads();
            amax_bits = sh.wmax[0];
            for (int i = 1; i < kThreads / 32; ++i) amax_bits = max(amax_bits, sh.wmax[i]);
        }
    }
    // per-tensor partition: the block is the tensor, its amax is the group amax
    const float b_amax = (KIND == KIND_TENSOR) ? g_amax : __uint_as_float(amax_bits << 16);
    if (KIND == KIND_TENSOR) amax_bits = __float_as_uint(g_amax) >> 16;

    uint32_t s4b, s5b;
    block_scale(b_amax, m_g, R.scale_mode, s4b, s5b);
    const float s4 = __uint_as_float(s4b), s5 = __uint_as_float(s5b);

    // ---- cast and error terms ----
    Acc A;
#pragma unroll
    for (int i = 0; i < 4; ++i) { A.a43[i] = 0.0f; A.a52[i] = 0.0f; }
    A.nnz = A.nbig = A.nonfinite = 0u;
    A.mn = 0xFFFFFFFFu;
    uint2 k4[8], k5[8];
    if (slow) convert_half_segment<YARD, THREE, true, STORE>(half_in, half_out, t, s4, s5, A, k4, k5);
    else      convert_half_segment<YARD, THREE, false, STORE>(half_in, half_out, t, s4, s5, A, k4, k5);

    const float tiny = (float)(A.nnz - A.nbig);             // non-zeros below binary32's normal range: term 1
    float e43 = ((A.a43[0] + A.a43[1]) + (A.a43[2] + A.a43[3])) + tiny;
    // scale4 / scale5 = 2^(e4 - e5)
    const float ratio = __uint_as_float((127u - ((s5b >> 23) - (s4b >> 23))) << 23);
    float e52 = YARD ? ((A.a52[0] + A.a52[1]) + (A.a52[2] + A.a52[3])) * ratio + tiny : 0.0f;

    // ---- block sums, decision, per-tile partial ----
    WarpPart wp;
    uint32_t sel = MOR_FMT_E4M3;
    if (KIND == KIND_ROW128) {
        e43 += __shfl_xor_sync(0xFFFFFFFFu, e43, 1);
        e52 += __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
        const uint32_t nnz = A.nnz + __shfl_xor_sync(0xFFFFFFFFu, A.nnz, 1);
        const uint32_t nonf = A.nonfinite + __shfl_xor_sync(0xFFFFFFFFu, A.nonfinite, 1);
        const uint32_t mn = min(A.mn, __shfl_xor_sync(0xFFFFFFFFu, A.mn, 1));
        const int n_el = sh.seg_n[seg];
        sel = decide_block(R, (double)e43, (double)e52, nnz, nonf, amax_bits, mn, (uint32_t)n_el);
        const bool lead = (t & 1) == 0 && n_el > 0;
        if (lead) {
            const uint32_t b = local * (uint32_t)kSegsPerTile + (uint32_t)seg;
            const uint32_t sb = (sel == MOR_FMT_E5M2) ? s5b : s4b;
            if (R.sel) R.sel[b] = (uint8_t)sel;
            if (R.scale_e8m0) R.scale_e8m0[b] = (uint8_t)(sb >> 23);
            if (R.scale_f32) R.scale_f32[b] = __uint_as_float(sb);
            if (R.block_stats) {
                mor_block_stats_t bs;
                bs.amax = b_amax;
                bs.min_abs_nz = (mn == 0xFFFFFFFFu) ? __uint_as_float(0x7F800000u) : __uint_as_float(mn + 1u);
                bs.nnz = nnz; bs.n_nonfinite = nonf; bs.sum_rel_e4m3 = e43; bs.sum_rel_e5m2 = e52;
                R.block_stats[b] = bs;
            }
            sh.blk_sel[seg] = (uint8_t)sel;
        }
        wp.s43 = lead ? (double)e43 : 0.0;
        wp.s52 = lead ? (double)e52 : 0.0;
        wp.nnz = lead ? nnz : 0u;
        wp.nonfinite = lead ? nonf : 0u;
        wp.n4 = (lead && sel == MOR_FMT_E4M3) ? 1u : 0u;
        wp.n5 = (lead && sel == MOR_FMT_E5M2) ? 1u : 0u;
        wp.nb = (lead && sel == MOR_FMT_BF16) ? 1u : 0u;
        wp.mn = mn;
    } else {
        wp.s43 = (double)e43; wp.s52 = (double)e52;
        wp.nnz = A.nnz; wp.nonfinite = A.nonfinite;
        wp.n4 = wp.n5 = wp.nb = 0u;
        wp.mn = A.mn;
    }
    wp.s43 = warp_sum(wp.s43);
    wp.s52 = warp_sum(wp.s52);
    wp.nnz = __reduce_add_sync(0xFFFFFFFFu, wp.nnz);
    wp.nonfinite = __reduce_add_sync(0xFFFFFFFFu, wp.nonfinite);
    wp.n4 = __reduce_add_sync(0xFFFFFFFFu, wp.n4);
    wp.n5 = __reduce_add_sync(0xFFFFFFFFu, wp.n5);
    wp.nb = __reduce_add_sync(0xFFFFFFFFu, wp.nb);
    wp.mn = __reduce_min_sync(0xFFFFFFFFu, wp.mn);
    if (lane == 0) sh.wp[warp] = wp;
    __syncthreads();

    if (t == 0) {
        WarpPart tot = sh.wp[0];
        for (int i = 1; i < kThreads / 32; ++i) {
            const WarpPart& o = sh.wp[i];
            tot.s43 += o.s43; tot.s52 += o.s52; tot.nnz += o.nnz; tot.nonfinite += o.nonfinite;
            tot.n4 += o.n4; tot.n5 += o.n5; tot.nb += o.nb; tot.mn = min(tot.mn, o.mn);
        }
        if (KIND == KIND_BLK128) {
            const uint32_t bi = local / R.nbc, bj = local - bi * R.nbc;
            const long long rr = R.rows - (long long)bi * 128, cc = R.cols - (long long)bj * 128;
            const uint32_t n_el = (uint32_t)((rr < 128 ? rr : 128) * (cc < 128 ? cc : 128));
            const uint32_t bsel = decide_block(R, tot.s43, tot.s52, tot.nnz, tot.nonfinite, amax_bits, tot.mn, n_el);
            const uint32_t sb = (bsel == MOR_FMT_E5M2) ? s5b : s4b;
            if (R.sel) R.sel[local] = (uint8_t)bsel;
            if (R.scale_e8m0) R.scale_e8m0[local] = (uint8_t)(sb >> 23);
            if (R.scale_f32) R.scale_f32[local] = __uint_as_float(sb);
            if (R.block_stats) {
                mor_block_stats_t bs;
                bs.amax = b_amax;
                bs.min_abs_nz = (tot.mn == 0xFFFFFFFFu) ? __uint_as_float(0x7F800000u) : __uint_as_float(tot.mn + 1u);
                bs.nnz = tot.nnz; bs.n_nonfinite = tot.nonfinite;
                bs.sum_rel_e4m3 = (float)tot.s43; bs.sum_rel_e5m2 = (float)tot.s52;
                R.block_stats[local] = bs;
            }
            tot.n4 = bsel == MOR_FMT_E4M3; tot.n5 = bsel == MOR_FMT_E5M2; tot.nb = bsel == MOR_FMT_BF16;
            sh.bcast[0] = bsel;
        }
        Partial P;
        P.sum43 = tot.s43; P.sum52 = tot.s52; P.nnz = tot.nnz; P.nonfinite = tot.nonfinite;
        P.n_e4m3 = tot.n4; P.n_e5m2 = tot.n5; P.n_bf16 = tot.nb;
        P.min_nz_bits = tot.mn;
        partials[R.tile_begin + local] = P;
    }

    if (KIND == KIND_BLK128 && (THREE || R.fallback)) {
        __syncthreads();
        sel = sh.bcast[0];
    }
    if (THREE && STORE) {
        // the block's decision is known now: keep the code set of the chosen format
#pragma unroll
        for (int j = 0; j < 8; ++j)
            *reinterpret_cast<uint2*>(half_out + (((j + t) & 7) << 3)) = (sel == MOR_FMT_E5M2) ? k5[j] : k4[j];
    }
    if (STORE) {
        __syncthreads();
        // ---- coalesced code stores: 1024 chunks of 16 bytes, 4 per thread ----
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = t + kThreads * j, sg = c >> 3, k = c & 7;
            if (16 * k < sh.seg_n[sg])
                *reinterpret_cast<uint4*>(R.codes + sh.seg_coff[sg] + 16 * k) = lds128(s_out + sg * 128 + k * 16);
        }
        // ---- optional copy of the blocks that stay in BF16 ----
        if (R.fallback && KIND != KIND_TENSOR) {
            const int k = t & 15;
#pragma unroll 1
            for (int j = 0; j < 8; ++j) {
                const int sg = (t >> 4) + 16 * j;
                const uint32_t ssel = (KIND == KIND_BLK128) ? sel : sh.blk_sel[sg];
                const int left = sh.seg_n[sg] - 8 * k;
                if (left <= 0 || ssel != MOR_FMT_BF16) continue;
                uint16_t* dst = R.fallback + sh.seg_off[sg] + 8 * k;
                const unsigned char* src = s_in + sg * 256 + k * 16;
                if (left >= 8) *reinterpret_cast<uint4*>(dst) = lds128(src);
                else for (int i = 0; i < left; ++i) dst[i] = reinterpret_cast<const uint16_t*>(src)[i];
            }
        }
    }
}

// ------------------------------------------------------------------ amax pre-pass ----

// One tile of 128 row pieces per CTA; 16-byte loads straight to registers.  The packed BF16
// maximum lets NaN and inf through; a thread that meets one rescans its registers with a
// filter and counts them.
__global__ void __launch_bounds__(kThreads)
mor_amax_kernel(const __grid_constant__ BatchParams p, float* __restrict__ amax_slots_unused)
{
    (void)amax_slots_unused;
    __shared__ long long s_off[kSegsPerTile];
    __shared__ int s_n[kSegsPerTile];
    __shared__ uint32_t s_wmax[kThreads / 32], s_wnf[kThreads / 32];

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    uint32_t local;
    const TensorRec& R = p.t[find_tensor(p, blockIdx.x, local)];
    if (t < kSegsPerTile) {
        long long coff;
        seg_geometry<KIND_TENSOR>(R, local, t, s_off[t], coff, s_n[t]);
    }
    __syncthreads();

    uint4 v[8];
    const int k = t & 15;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int seg = (t >> 4) + 16 * j;
        const int left = s_n[seg] - 8 * k;
        v[j] = make_uint4(0u, 0u, 0u, 0u);
        if (left >= 8) {
            v[j] = *reinterpret_cast<const uint4*>(R.x + s_off[seg] + 8 * k);
        } else if (left > 0) {
            const uint16_t* src = R.x + s_off[seg] + 8 * k;
            uint16_t e[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int i = 0; i < left; ++i) e[i] = src[i];
            v[j] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
        }
    }
    __nv_bfloat162 m = __float2bfloat162_rn(0.0f);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) m = __hmax2_nan(m, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
    }
    const uint32_t mb = *reinterpret_cast<const uint32_t*>(&m);
    uint32_t amax = max(mb & 0xFFFFu, mb >> 16), nf = 0;
    if (amax >= kBf16Inf) {
        amax = 0;
        for (int j = 0; j < 8; ++j) {
            const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
            for (int i = 0; i < 4; ++i) {
                const uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
                if (lo < kBf16Inf) amax = max(amax, lo); else nf++;
                if (hi < kBf16Inf) amax = max(amax, hi); else nf++;
            }
        }
    }
    amax = __reduce_max_sync(0xFFFFFFFFu, amax);
    nf = __reduce_add_sync(0xFFFFFFFFu, nf);
    if (lane == 0) { s_wmax[warp] = amax; s_wnf[warp] = nf; }
    __syncthreads();
    if (t == 0) {
        for (int i = 1; i < kThreads / 32; ++i) { amax = max(amax, s_wmax[i]); nf += s_wnf[i]; }
        // non-negative binary32 patterns order like the values
        atomicMax(reinterpret_cast<unsigned int*>(const_cast<float*>(R.amax)), amax << 16);
        if (nf) atomicAdd(R.nonfinite_slot, nf);
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
    __shared__ WarpPart s_tot;
    const TensorRec& R = p.t[blockIdx.x];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;

    WarpPart a;
    a.s43 = a.s52 = 0.0; a.nnz = a.nonfinite = a.n4 = a.n5 = a.nb = 0u; a.mn = 0xFFFFFFFFu;
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
                block_scale(g_amax, m_g, R.scale_mode, s4b, s5b);
                if (R.sel) R.sel[0] = (uint8_t)bsel;
                if (R.scale_e8m0) R.scale_e8m0[0] = (uint8_t)(s4b >> 23);
                if (R.scale_f32) R.scale_f32[0] = __uint_as_float(s4b);
                if (R.block_stats) {
                    mor_block_stats_t bs;
                    bs.amax = g_amax;
                    bs.min_abs_nz = (tot.mn == 0xFFFFFFFFu) ? __uint_as_float(0x7F800000u) : __uint_as_float(tot.mn + 1u);
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
            ts.group_amax = g_amax; ts.group_mantissa = m_g; ts.tensor_format = fmt; ts.status = MOR_OK;
            ts.n_blocks = n_blocks; ts.n_e4m3 = c[2]; ts.n_e5m2 = c[3]; ts.n_bf16 = c[4]; ts.n_nonfinite = c[1];
            *R.tensor_stats = ts;
        }
        s_fmt = fmt;
        (void)s_tot;
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

template <int KIND, bool YARD, bool THREE, bool STORE>
cudaError_t launch_main_t(const BatchParams& p, Partial* partials, uint32_t tiles, cudaStream_t s)
{
    auto kfn = mor_main_kernel<KIND, YARD, THREE, STORE>;
    static bool configured = false;   // per instantiation; the attribute is per function, setting it twice is harmless
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kfn<<<tiles, kThreads, kSmemBytes, s>>>(p, partials);
    return cudaGetLastError();
}

template <int KIND>
cudaError_t launch_main_k(const MainVariant& v, const BatchParams& p, Partial* partials, uint32_t tiles, cudaStream_t s)
{
    if (v.three) {
        return v.store ? launch_main_t<KIND, true, true, true>(p, partials, tiles, s)
                       : launch_main_t<KIND, true, true, false>(p, partials, tiles, s);
    }
    if (v.yard) {
        return v.store ? launch_main_t<KIND, true, false, true>(p, partials, tiles, s)
                       : launch_main_t<KIND, true, false, false>(p, partials, tiles, s);
    }
    return v.store ? launch_main_t<KIND, false, false, true>(p, partials, tiles, s)
                   : launch_main_t<KIND, false, false, false>(p, partials, tiles, s);
}

}  // namespace

cudaError_t launch_amax(const BatchParams& p, uint32_t total_tiles, cudaStream_t s)
{
    if (total_tiles == 0) return cudaSuccess;
    mor_amax_kernel<<<total_tiles, kThreads, 0, s>>>(p, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_main(const MainVariant& v, const BatchParams& p, Partial* partials, uint32_t total_tiles, cudaStream_t s)
{
    if (total_tiles == 0) return cudaSuccess;
    switch (v.kind) {
        case KIND_TENSOR: return launch_main_k<KIND_TENSOR>(v, p, partials, total_tiles, s);
        case KIND_ROW128: return launch_main_k<KIND_ROW128>(v, p, partials, total_tiles, s);
        case KIND_BLK128: return launch_main_k<KIND_BLK128>(v, p, partials, total_tiles, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_finalise(const BatchParams& p, const Partial* partials, int kind, cudaStream_t s)
{
    if (p.n == 0) return cudaSuccess;
    // slices only help when the selection array has to be filled for a tensor-level decision
    unsigned slices = 1;
    for (int i = 0; i < p.n; ++i)
        if (kind != KIND_TENSOR && p.t[i].criterion == MOR_CRIT_TENSOR_MEAN_REL && p.t[i].sel && p.t[i].n_units > 65536u) slices = 16;
    dim3 grid((unsigned)p.n, slices);
    switch (kind) {
        case KIND_TENSOR: mor_finalise_kernel<KIND_TENSOR><<<grid, kThreads, 0, s>>>(p, partials); break;
        case KIND_ROW128: mor_finalise_kernel<KIND_ROW128><<<grid, kThreads, 0, s>>>(p, partials); break;
        case KIND_BLK128: mor_finalise_kernel<KIND_BLK128><<<grid, kThreads, 0, s>>>(p, partials); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace mor
