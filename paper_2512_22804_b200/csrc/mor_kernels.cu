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

// Block statistics of a thread's 64 elements in one pass over packed BF16 pairs:
//   mx  per-halfword max of the |x| bit patterns.  NaN and inf compare above every finite
//       pattern, which is how a non-finite input is noticed.
//   mn  per-halfword min of (|x| bits - 1) mod 2^16: zeros wrap to 0xFFFF and drop out, so
//       mn + 1 is the smallest non-zero |x| (Eq. 4, and the check for values that leave
//       binary32's normal range after scaling).
__device__ __forceinline__ void scan_half_segment(const unsigned char* half, int t, uint32_t& amax_bits, uint32_t& minm1_bits)
{
    uint32_t mx = 0u, mn = 0xFFFFFFFFu;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint4 v = lds128(half + (((j + t) & 7) << 4));
        const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu, a2 = v.z & 0x7FFF7FFFu, a3 = v.w & 0x7FFF7FFFu;
        mx = __vimax3_u16x2(mx, a0, a1);
        mx = __vimax3_u16x2(mx, a2, a3);
        mn = __viaddmin_u16x2(a0, 0xFFFFFFFFu, mn);
        mn = __viaddmin_u16x2(a1, 0xFFFFFFFFu, mn);
        mn = __viaddmin_u16x2(a2, 0xFFFFFFFFu, mn);
        mn = __viaddmin_u16x2(a3, 0xFFFFFFFFu, mn);
    }
    amax_bits = max(mx & 0xFFFFu, mx >> 16);
    minm1_bits = min(mn & 0xFFFFu, mn >> 16);
}

// the same over finite elements only (used once a non-finite element has been seen)
__device__ __forceinline__ void scan_half_segment_finite(const unsigned char* half, int t, uint32_t& amax_bits, uint32_t& minm1_bits)
{
    uint32_t m = 0u, n = 0xFFFFu;
#pragma unroll 1
    for (int j = 0; j < 8; ++j) {
        const uint4 v = lds128(half + (((j + t) & 7) << 4));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
            if (lo < kBf16Inf) { m = max(m, lo); n = min(n, (lo - 1u) & 0xFFFFu); }
            if (hi < kBf16Inf) { m = max(m, hi); n = min(n, (hi - 1u) & 0xFFFFu); }
        }
    }
    amax_bits = m;
    minm1_bits = n;
}

struct Acc {
    float a43[4], a52[4];
    uint32_t nnz, nbig, nonfinite;
};

__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
// two IEEE binary32 multiplies in one instruction (each lane rounds to nearest even)
__device__ __forceinline__ void mul_f32x2(unsigned long long a, unsigned long long b, float& lo, float& hi)
{
    unsigned long long r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ float rcp_ftz(float a)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}

// Fast path for one BF16 pair: two E4M3 codes (and two E5M2 codes) with their terms of
// Eq. 1-3.   y = fl32(x * scale); c = RNE-saturating cast; q = value of c;
// term = |y - q| / |y|, formed as |y - q| * rcp(|y| + 2^-126).  The caller guarantees that
// the block holds no NaN/inf and that every non-zero |y| is at least 2^-100, so the added
// constant changes a term by less than 2^-26 relative, and a zero element gives 0 * finite.
template <bool YARD>
__device__ __forceinline__ void convert_pair_fast(uint32_t w, unsigned long long s4x2, unsigned long long s5x2, int lane,
                                                  float (&a43)[4], float (&a52)[4], __nv_bfloat162& cnt,
                                                  uint32_t& c4, uint32_t& c5)
{
    const __nv_bfloat162 xb = *reinterpret_cast<const __nv_bfloat162*>(&w);
    cnt = __hadd2(cnt, __hneu2(xb, __float2bfloat162_rn(0.0f)));          // non-zero count, exact up to 256 per half
    const unsigned long long x2 = pack_f32x2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    float ylo, yhi;
    mul_f32x2(x2, s4x2, ylo, yhi);
    c4 = cvt_e4m3x2(yhi, ylo);
    const uint32_t q4 = e4m3x2_to_f16x2(c4);
    const float dlo = diff_f16_f32(static_cast<uint16_t>(q4 & 0xFFFFu), ylo);
    const float dhi = diff_f16_f32(static_cast<uint16_t>(q4 >> 16), yhi);
    const float rlo = rcp_ftz(fabsf(ylo) + FLT_MIN), rhi = rcp_ftz(fabsf(yhi) + FLT_MIN);
    a43[lane] = fmaf(fabsf(dlo), rlo, a43[lane]);
    a43[lane] = fmaf(fabsf(dhi), rhi, a43[lane]);
    if (YARD) {
        float zlo, zhi;
        mul_f32x2(x2, s5x2, zlo, zhi);
        c5 = cvt_e5m2x2(zhi, zlo);
        const uint32_t q5 = e5m2x2_to_f16x2(c5);
        const float elo = diff_f16_f32(static_cast<uint16_t>(q5 & 0xFFFFu), zlo);
        const float ehi = diff_f16_f32(static_cast<uint16_t>(q5 >> 16), zhi);
        // |z - q'| / |z| = |z - q'| * (1/|y|) * (scale4/scale5); the power-of-two ratio is applied once per block
        a52[lane] = fmaf(fabsf(elo), rlo, a52[lane]);
        a52[lane] = fmaf(fabsf(ehi), rhi, a52[lane]);
    } else {
        c5 = 0;
    }
}

// Careful path for one BF16 pair: handles NaN/inf elements (stated reading: ignored by
// every count and sum, NaN -> 0x7F, +-inf -> +-largest finite) and non-zero elements whose
// scaled value leaves binary32's normal range (flushed by both formats: term 1, added by
// the caller from the counts nnz - nbig).
template <bool YARD>
__device__ __forceinline__ void convert_pair_careful(uint32_t w, float s4, float s5, int lane, Acc& A,
                                                     uint32_t& c4, uint32_t& c5)
{
    const uint32_t blo = w << 16, bhi = w & 0xFFFF0000u;
    const uint32_t alo = blo & 0x7FFFFFFFu, ahi = bhi & 0x7FFFFFFFu;
    const float xlo = __uint_as_float(blo), xhi = __uint_as_float(bhi);
    const bool uselo = alo < 0x7F800000u, usehi = ahi < 0x7F800000u;
    A.nonfinite += (uselo ? 0u : 1u) + (usehi ? 0u : 1u);
    A.nnz += ((alo != 0u && uselo) ? 1u : 0u) + ((ahi != 0u && usehi) ? 1u : 0u);

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
        if (biglo) A.a52[lane] = fmaf(fabsf(elo), rlo, A.a52[lane]);
        if (bighi) A.a52[lane] = fmaf(fabsf(ehi), rhi, A.a52[lane]);
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

// A thread's 64 elements.  E4M3 codes go to shared memory at once unless the recipe is
// three-way, where both code sets wait in registers for the block's decision.
// Results: e43 = the thread's sum of E4M3 terms, complete; e52 = its sum of E5M2 terms still
// to be multiplied by scale4/scale5 and then increased by `tiny` (the count of non-zeros
// flushed below binary32's normal range, already inside e43); nnz; nonfinite.
template <bool YARD, bool THREE, bool CAREFUL, bool STORE>
__device__ __forceinline__ void convert_half_segment(const unsigned char* half_in, unsigned char* half_out, int t,
                                                     float s4, float s5, float& e43, float& e52, float& tiny,
                                                     uint32_t& nnz, uint32_t& nonfinite, uint2 (&k4)[8], uint2 (&k5)[8])
{
    Acc A;
#pragma unroll
    for (int i = 0; i < 4; ++i) { A.a43[i] = 0.0f; A.a52[i] = 0.0f; }
    A.nnz = A.nbig = A.nonfinite = 0u;
    __nv_bfloat162 cnt = __float2bfloat162_rn(0.0f);
    const unsigned long long s4x2 = pack_f32x2(s4, s4), s5x2 = pack_f32x2(s5, s5);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int kk = (j + t) & 7;
        const uint4 v = lds128(half_in + (kk << 4));
        uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
        if (CAREFUL) {
            convert_pair_careful<YARD>(v.x, s4, s5, 0, A, a0, b0);
            convert_pair_careful<YARD>(v.y, s4, s5, 1, A, a1, b1);
            convert_pair_careful<YARD>(v.z, s4, s5, 2, A, a2, b2);
            convert_pair_careful<YARD>(v.w, s4, s5, 3, A, a3, b3);
        } else {
            convert_pair_fast<YARD>(v.x, s4x2, s5x2, 0, A.a43, A.a52, cnt, a0, b0);
            convert_pair_fast<YARD>(v.y, s4x2, s5x2, 1, A.a43, A.a52, cnt, a1, b1);
            convert_pair_fast<YARD>(v.z, s4x2, s5x2, 2, A.a43, A.a52, cnt, a2, b2);
            convert_pair_fast<YARD>(v.w, s4x2, s5x2, 3, A.a43, A.a52, cnt, a3, b3);
        }
        const uint2 c4 = make_uint2(__byte_perm(a0, a1, 0x5410), __byte_perm(a2, a3, 0x5410));
        if (THREE) {
            k4[j] = c4;
            k5[j] = make_uint2(__byte_perm(b0, b1, 0x5410), __byte_perm(b2, b3, 0x5410));
        } else if (STORE) {
            *reinterpret_cast<uint2*>(half_out + (kk << 3)) = c4;
        }
    }
    tiny = 0.0f;
    if (CAREFUL) {
        nnz = A.nnz;
        nonfinite = A.nonfinite;
        tiny = (float)(A.nnz - A.nbig);
    } else {
        nnz = (uint32_t)(__low2float(cnt) + __high2float(cnt));
        nonfinite = 0u;
    }
    e43 = ((A.a43[0] + A.a43[1]) + (A.a43[2] + A.a43[3])) + tiny;
    e52 = (A.a52[0] + A.a52[1]) + (A.a52[2] + A.a52[3]);
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float minnz_value(uint32_t minm1_bits)
{
    return minm1_bits == 0xFFFFu ? __uint_as_float(0x7F800000u) : __uint_as_float((minm1_bits + 1u) << 16);
}

// Algorithm 2 for one block with the per-block metrics (M_1 = Eq. 3, M_2 = Eq. 4, or
// Eq. 1-2 on the block alone).
__device__ __forceinline__ uint32_t decide_block(const TensorRec& R, double e43, double e52, uint32_t nnz,
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

    // ---- block amax and smallest non-zero (Algorithm 1; Eq. 4) ----
    uint32_t amax_bits, minm1;
    scan_half_segment(half_in, t, amax_bits, minm1);
    bool nonfin;
    if (KIND == KIND_ROW128) {
        amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, 1));
        minm1 = min(minm1, __shfl_xor_sync(0xFFFFFFFFu, minm1, 1));
        nonfin = __any_sync(0xFFFFFFFFu, amax_bits >= kBf16Inf);          // warp-uniform
        if (nonfin) {
            scan_half_segment_finite(half_in, t, amax_bits, minm1);
            amax_bits = max(amax_bits, __shfl_xor_sync(0xFFFFFFFFu, amax_bits, 1));
            minm1 = min(minm1, __shfl_xor_sync(0xFFFFFFFFu, minm1, 1));
        }
    } else {
        amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
        minm1 = __reduce_min_sync(0xFFFFFFFFu, minm1);
        if (lane == 0) sh.wmax[warp] = (amax_bits << 16) | (0xFFFFu - minm1);   // both halves reduce with max
        __syncthreads();
        uint32_t hi = 0u, lo = 0u;
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) { hi = max(hi, sh.wmax[i] >> 16); lo = max(lo, sh.wmax[i] & 0xFFFFu); }
        amax_bits = hi; minm1 = 0xFFFFu - lo;
        nonfin = amax_bits >= kBf16Inf;                                   // CTA-uniform
        if (nonfin) {
            __syncthreads();
            scan_half_segment_finite(half_in, t, amax_bits, minm1);
            amax_bits = __reduce_max_sync(0xFFFFFFFFu, amax_bits);
            minm1 = __reduce_min_sync(0xFFFFFFFFu, minm1);
            if (lane == 0) sh.wmax[warp] = (amax_bits << 16) | (0xFFFFu - minm1);
            __syncthreads();
            hi = 0u; lo = 0u;
            for (int i = 0; i < kThreads / 32; ++i) { hi = max(hi, sh.wmax[i] >> 16); lo = max(lo, sh.wmax[i] & 0xFFFFu); }
            amax_bits = hi; minm1 = 0xFFFFu - lo;
        }
    }
    // per-tensor partition: the block is the tensor, its amax was reduced by the pre-pass
    const float b_amax = (KIND == KIND_TENSOR) ? *R.amax_slot : __uint_as_float(amax_bits << 16);
    if (KIND == KIND_TENSOR) amax_bits = __float_as_uint(b_amax) >> 16;

    uint32_t s4b, s5b;
    block_scale(b_amax, m_g, R.scale_mode, s4b, s5b);
    const float s4 = __uint_as_float(s4b), s5 = __uint_as_float(s5b);

    // The fast path needs every non-zero |x * scale| to be at least 2^-100 (see convert_pair_fast).
    // minm1 covers this thread's block (ROW128), this tile (BLK128, TENSOR).
    bool careful = nonfin;
    if (minm1 != 0xFFFFu) careful = careful || !(__fmul_rn(minnz_value(minm1), s4) >= 7.888609052210118e-31f);
    if (KIND == KIND_ROW128) careful = __any_sync(0xFFFFFFFFu, careful);

    // ---- cast and error terms ----
    float e43, e52, tiny;
    uint32_t nnz, nonf;
    uint2 k4[8], k5[8];
    if (careful) convert_half_segment<YARD, THREE, true, STORE>(half_in, half_out, t, s4, s5, e43, e52, tiny, nnz, nonf, k4, k5);
    else         convert_half_segment<YARD, THREE, false, STORE>(half_in, half_out, t, s4, s5, e43, e52, tiny, nnz, nonf, k4, k5);
    // scale4 / scale5 = 2^(e4 - e5)
    const float ratio = __uint_as_float((127u - ((s5b >> 23) - (s4b >> 23))) << 23);
    e52 = YARD ? e52 * ratio + tiny : 0.0f;

    // ---- block sums, decision, per-tile partial ----
    uint32_t sel = MOR_FMT_E4M3;
    float w43, w52;                 // what this thread adds to the tile's sums
    uint32_t wcnt = 0u;             // n_e4m3 | n_e5m2 << 8 | n_bf16 << 16 (at most 128 blocks per tile)
    uint32_t wnz = nnz | (nonf << 16);   // at most 64 per thread, 16384 per tile
    if (KIND == KIND_ROW128) {
        e43 += __shfl_xor_sync(0xFFFFFFFFu, e43, 1);
        e52 += __shfl_xor_sync(0xFFFFFFFFu, e52, 1);
        const uint32_t pz = wnz + __shfl_xor_sync(0xFFFFFFFFu, wnz, 1);
        const uint32_t bnnz = pz & 0xFFFFu, bnonf = pz >> 16;
        const int n_el = sh.seg_n[seg];
        sel = decide_block(R, (double)e43, (double)e52, bnnz, bnonf, amax_bits, minm1, (uint32_t)n_el);
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
                bs.min_abs_nz = THREE ? minnz_value(minm1) : __uint_as_float(0x7F800000u);
                bs.nnz = bnnz; bs.n_nonfinite = bnonf; bs.sum_rel_e4m3 = e43; bs.sum_rel_e5m2 = e52;
                R.block_stats[b] = bs;
            }
            sh.blk_sel[seg] = (uint8_t)sel;
            wcnt = 1u << (8 * sel);
        }
        w43 = lead ? e43 : 0.0f;
        w52 = lead ? e52 : 0.0f;
    } else {
        w43 = e43; w52 = e52;
    }
    WarpPart wp;
    if (KIND == KIND_ROW128) {
        // block sums are binary32 already; add them up in binary32 inside the warp
        wp.s43 = (double)warp_sum(w43);
        wp.s52 = (double)warp_sum(w52);
    } else {
        wp.s43 = warp_sum((double)w43);
        wp.s52 = warp_sum((double)w52);
    }
    wnz = __reduce_add_sync(0xFFFFFFFFu, wnz);
    wcnt = __reduce_add_sync(0xFFFFFFFFu, wcnt);
    wp.nnz = wnz & 0xFFFFu; wp.nonfinite = wnz >> 16;
    wp.n4 = wcnt & 0xFFu; wp.n5 = (wcnt >> 8) & 0xFFu; wp.nb = wcnt >> 16;
    wp.mn = (KIND == KIND_ROW128) ? __reduce_min_sync(0xFFFFFFFFu, minm1) : minm1;
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
            const uint32_t bsel = decide_block(R, tot.s43, tot.s52, tot.nnz, tot.nonfinite, amax_bits, minm1, n_el);
            const uint32_t sb = (bsel == MOR_FMT_E5M2) ? s5b : s4b;
            if (R.sel) R.sel[local] = (uint8_t)bsel;
            if (R.scale_e8m0) R.scale_e8m0[local] = (uint8_t)(sb >> 23);
            if (R.scale_f32) R.scale_f32[local] = __uint_as_float(sb);
            if (R.block_stats) {
                mor_block_stats_t bs;
                bs.amax = b_amax;
                bs.min_abs_nz = THREE ? minnz_value(minm1) : __uint_as_float(0x7F800000u);
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
            v[j] = make_uint4(e[0] | ((uint32_t)e[1] << 16), e[2] | ((uint32_t)e[3] << 16),
                              e[4] | ((uint32_t)e[5] << 16), e[6] | ((uint32_t)e[7] << 16));
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
        atomicMax(reinterpret_cast<unsigned int*>(R.amax_slot), amax << 16);
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
