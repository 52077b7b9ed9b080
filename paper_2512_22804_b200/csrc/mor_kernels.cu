// The two small kernels around the fused main kernel (mor_main.cu).
//
//   mor_amax_kernel      Algorithm 1, "g_amax <- max(abs(g))" with the tensor as one group
//   mor_finalise_kernel  tensor-wide aggregate of the per-tile partials and the Eq. 2 decision
#include <cuda_bf16.h>
#include <float.h>

#include "mor_internal.h"

namespace mor {
namespace {

constexpr uint32_t kBf16Inf = 0x7F80u;

struct WarpPart {
    double s43, s52;
    uint32_t nnz, nonfinite, n4, n5, nb, mn;
};

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

// Where row piece `s` of pre-pass tile `local` lives: the pieces are the 128-element pieces of
// the rows in row-major order.
__device__ __forceinline__ void piece_geometry(const TensorRec& R, uint32_t local, int s, long long& off, int& n)
{
    const uint32_t u = local * (uint32_t)kSegsPerTile + (uint32_t)s;
    const uint32_t r = u / R.nbc;
    const long long c0 = (long long)(u - r * R.nbc) * kSegElems;
    const bool valid = u < R.n_units;
    const long long left = R.cols - c0;
    n = valid ? (int)(left < kSegElems ? left : kSegElems) : 0;
    off = valid ? (long long)r * R.ld + c0 : 0;
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
    if (t < kSegsPerTile) piece_geometry(R, local, t, s_off[t], s_n[t]);
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
            ts.group_amax = g_amax; ts.group_mantissa = m_g; ts.tensor_format = fmt;
            ts.status = *R.device_status ? MOR_ERR_TIMEOUT : MOR_OK;
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

}  // namespace

cudaError_t launch_amax(const BatchParams& p, uint32_t total_tiles, cudaStream_t s)
{
    if (total_tiles == 0) return cudaSuccess;
    mor_amax_kernel<<<total_tiles, kThreads, 0, s>>>(p, nullptr);
    return cudaGetLastError();
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
