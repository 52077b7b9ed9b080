/*
 * mor.h -- C boundary of the B200 (sm_100a) MoR analyse-and-quantise library.
 *
 * MoR (Mixture of Representations) partitions a BF16 tensor into blocks, walks an ordered
 * list of formats from most to least aggressive for every block and keeps the first one
 * whose acceptance metric holds (Section 3, Algorithm 2 of the paper).  Scales follow the
 * Group Amax Mantissa scheme: one 23-bit mantissa per tensor plus one 8-bit exponent per
 * block (Section 2, Algorithm 1).
 *
 * Conventions for every entry point
 *   - Pointers inside descriptors are DEVICE pointers.  The descriptors themselves, and
 *     every argument named host_*, live in HOST memory and are read before the call returns.
 *   - The caller owns all buffers and the stream.  The library allocates nothing, keeps no
 *     state between calls and never synchronises: work is enqueued on `cuda_stream`
 *     (a cudaStream_t passed as void*, NULL = the default stream) and the call returns.
 *   - Argument problems are reported synchronously and nothing is launched.  Conditions
 *     found on the device (non-finite inputs) are reported in mor_tensor_stats_t.
 *   - Inputs are row-major BF16 with the last dimension contiguous.
 */
#ifndef MOR_H_
#define MOR_H_

#include <stddef.h>
#include <stdint.h>

/* The library is built with hidden symbol visibility; only the entry points below are exported. */
#if defined(__GNUC__)
#define MOR_API __attribute__((visibility("default")))
#else
#define MOR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOR_OK = 0,
    MOR_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, negative size, bad enum   */
    MOR_ERR_UNSUPPORTED = 2,   /* a recipe the paper defines no metric for, or a block shape
                                  this build has no kernel for                                */
    MOR_ERR_ALIGNMENT = 3,     /* base pointer or leading dimension not aligned as stated     */
    MOR_ERR_WORKSPACE = 4,     /* workspace NULL or smaller than mor_workspace_bytes()        */
    MOR_ERR_CUDA = 5,          /* a CUDA runtime call failed (launch, copy)                   */
    MOR_ERR_TIMEOUT = 6,       /* a bounded device-side wait expired (reported in
                                  mor_tensor_stats_t.status; the outputs are then incomplete)  */
    MOR_ERR_STATIC_SCRATCH = 7 /* mor_analyze_quantize_static: the tensor needs more scratch than
                                  the built-in array holds                                    */
} mor_status_t;

/* Representation types.  Section 3 orders the candidates by how much precision they give up,
 * E4M3 first and BF16 last.  E4M3: 4 exponent / 3 mantissa bits, finite range 2^-9..448.
 * E5M2: 5 / 2 bits, 2^-16..57344 (Sections 1-2).  Casts round to nearest even and
 * saturate to the largest finite value. */
typedef enum { MOR_FMT_E4M3 = 0, MOR_FMT_E5M2 = 1, MOR_FMT_BF16 = 2 } mor_format_t;

/* How a block's scale is formed.
 *   GAM        Algorithm 1: mantissa of 448/tensor_amax shared by all blocks, per-block
 *              exponent of 448/block_amax lowered by one when the shared mantissa is the
 *              larger, so that no block saturates.
 *   E8M0       power-of-two scale per block (the ablation of Section 4.1.2): Algorithm 1
 *              with a zero mantissa.
 *   FP32_AMAX  fl32(448/block_amax) per block (same ablation); the full scale is returned
 *              in mor_outputs_t.scale_f32. */
typedef enum { MOR_SCALE_GAM = 0, MOR_SCALE_E8M0 = 1, MOR_SCALE_FP32_AMAX = 2 } mor_scale_mode_t;

/* Acceptance metric for E4M3.
 *   TENSOR_MEAN_REL  Section 3.1, Eq. 1-2: one decision for the whole tensor; mean over its
 *                    non-zero elements of |x - Q(x)| / |x| must be < threshold.  The scales
 *                    may still be per block: the block sums are added up into the tensor's error.
 *   BLOCK_VS_E5M2    Section 3.2, Eq. 3: per block, E4M3 is kept when its summed relative
 *                    error does not exceed that of E5M2.  With three formats a rejected
 *                    block takes E5M2 when Eq. 4 holds (max|b|/min|b| < 57344/2^-14).
 *   BLOCK_MEAN_REL   Eq. 1-2 applied to each block alone (an instance of Algorithm 2 the
 *                    paper does not evaluate). */
typedef enum {
    MOR_CRIT_TENSOR_MEAN_REL = 0,
    MOR_CRIT_BLOCK_VS_E5M2 = 1,
    MOR_CRIT_BLOCK_MEAN_REL = 2
} mor_criterion_t;

enum {
    MOR_FLAG_STRICT_TIES = 1u,             /* Eq. 3 with its literal '<': a block that is
                                              equally good in both formats is rejected.
                                              Default: a tie keeps E4M3.                    */
    MOR_FLAG_RANGE_MIN_INCLUDES_ZERO = 2u  /* Eq. 4 with the literal min|b|: a block that
                                              holds a zero never takes E5M2.  Default: the
                                              minimum runs over non-zero elements.          */
};

/* One tensor and the recipe to analyse it with (inputs of Algorithm 2: tensor, partition,
 * ordered type list, metric; input of Algorithm 1: q_amax is 448, and 57344 for E5M2). */
typedef struct mor_tensor_desc {
    const void* x;          /* DEVICE.  BF16 [rows, ld], 16-byte aligned                     */
    int64_t rows, cols;     /* >= 0; an empty tensor is valid                                */
    int64_t ld;             /* elements between row starts; >= cols; multiple of 8           */
    int32_t block_rows;     /* partition: (0,0) whole tensor, (1,128) sub-channel rows,      */
    int32_t block_cols;     /*            (128,128) or (64,64) 2-D blocks (Section 4.1.2 runs
                                           the smaller size as an ablation); per channel (Section 3;
                                           the paper's most FP8-efficient partition): (1,0) one
                                           block per row, (0,1) one block per column, whichever is
                                           the operand's dot-product dimension, two formats only,
                                           decided for the tensor (Eq. 2) or per channel (Eq. 3, or
                                           Eq. 1-2 on the channel); (128,1) sub-column blocks.  The
                                           column partitions (128,1) and (0,1) serve the operand whose
                                           dot-product dimension runs down the rows: their codes come
                                           out transposed, see codes.  Edge blocks may overhang:
                                           missing elements take part in nothing                  */
    int32_t n_formats;      /* 2 or 3                                                        */
    int32_t formats[3];     /* {E4M3,BF16} or {E4M3,E5M2,BF16}, in this order                */
    int32_t criterion;      /* mor_criterion_t; three formats need BLOCK_VS_E5M2             */
    float   threshold;      /* th of Eq. 2 as a fraction (0.045 = the paper's 4.5 %)         */
    int32_t scale_mode;     /* mor_scale_mode_t                                              */
    uint32_t flags;         /* MOR_FLAG_*                                                    */
    const float* group_amax;/* DEVICE, optional.  g_amax of Algorithm 1 if the caller has it
                               already: it fixes the shared mantissa; block amaxes are still
                               taken from the data, so a stale value cannot cause saturation.
                               NULL = the library computes it with one extra read of the
                               tensor (always done for the (0,0) and (1,0) partitions, whose
                               block amax spans tiles; never needed for the E8M0 and FP32-amax
                               scale modes of the other partitions, which have no shared
                               mantissa: those read the tensor once)                         */
} mor_tensor_desc_t;

#define MOR_ERROR_BINS 12

/* Per-block quantities behind the decisions (Eq. 3 sums, Eq. 4 range). */
typedef struct mor_block_stats {
    float    amax;          /* max|x| over the block's finite elements                       */
    float    min_abs_nz;    /* min|x| over finite non-zero elements, +inf if none; filled
                               only for three-format recipes                                 */
    uint32_t nnz;           /* finite non-zero elements (n of Eq. 1 restricted to the block) */
    uint32_t n_nonfinite;   /* NaN or +-inf elements                                         */
    float    sum_rel_e4m3;  /* sum over non-zeros of |x - Q_E4M3(x)| / |x|                   */
    float    sum_rel_e5m2;  /* same for E5M2; filled when the criterion is BLOCK_VS_E5M2     */
} mor_block_stats_t;

/* Per-tensor summary; always written. */
typedef struct mor_tensor_stats {
    double   sum_rel_e4m3;  /* numerator of Eq. 2                                            */
    uint64_t nnz;           /* n of Eq. 1                                                    */
    double   mean_rel_e4m3; /* error of Eq. 2; 0 when n = 0                                  */
    float    group_amax;    /* g_amax of Algorithm 1 (finite elements only)                  */
    uint32_t group_mantissa;/* m_g of Algorithm 1: low 23 bits                               */
    uint32_t tensor_format; /* Eq. 2 decision with `threshold`: MOR_FMT_E4M3 or MOR_FMT_BF16;
                               filled whatever the criterion                                 */
    uint32_t status;        /* mor_status_t of device-side conditions, MOR_OK normally       */
    uint64_t n_blocks, n_e4m3, n_e5m2, n_bf16;   /* blocks by selected format                */
    uint64_t n_nonfinite;   /* NaN / inf elements: ignored by every amax, count and sum;
                               they force their block, and tensor_format, to BF16            */
} mor_tensor_stats_t;

/* Outputs of Algorithm 2 (X_Q and the block metadata D) and of Algorithm 1 (S; M is in
 * mor_tensor_stats_t.group_mantissa).  All DEVICE pointers.  Block arrays are row-major
 * over the block grid [ceil(rows/block_rows), ceil(cols/block_cols)]. */
typedef struct mor_outputs {
    uint8_t* codes;         /* [rows, codes_ld] FP8 codes, 16-byte aligned ((128,1) and (0,1) blocks:
                               transposed, [cols, codes_ld] with codes_ld >= roundup(rows,16),
                               so that every block is contiguous).  E4M3 codes
                               everywhere except in blocks that selected E5M2; blocks that
                               selected BF16 still hold their E4M3 codes.  The tile store works
                               on 16-byte pieces of a row: the bytes of a row from column cols
                               up to the next multiple of 16 are overwritten (with the code of
                               zero); bytes from there to codes_ld-1 are left untouched       */
    int64_t  codes_ld;      /* bytes between row starts; >= roundup(cols,16); multiple of 16 */
    uint8_t* scale_e8m0;    /* [n_blocks] biased binary32 exponent of the selected format's
                               scale.  The scale is bits((e << 23) | group_mantissa); the
                               consumer de-scales by dividing by it                          */
    uint8_t* sel;           /* [n_blocks] mor_format_t chosen for the block                  */
    float*   scale_f32;     /* [n_blocks] optional (required for MOR_SCALE_FP32_AMAX): the
                               selected format's scale as a binary32                         */
    void*    bf16_fallback; /* optional, BF16 [rows, ld] like x: receives a copy of every
                               block that selected BF16 (other blocks are left untouched).
                               NULL = the fallback is the input itself.  Per-block criteria
                               only                                                          */
    mor_block_stats_t*  block_stats;  /* [n_blocks] optional                                 */
    mor_tensor_stats_t* tensor_stats; /* required                                            */
    void*    fake_quant;    /* optional, BF16 [rows, ld] like x: the tensor after "quantise,
                               dequantise, de-scale" (Section 4, the form the paper trains with).
                               Per element: the FP8 value of the block's selected format divided
                               by the block's scale (one binary32 division), rounded to BF16;
                               blocks that stay in BF16 and NaN/inf elements are copied.  Where the
                               decision is taken for the whole tensor (tensor-level criterion,
                               (0,0) partition) the E4M3 values are written: keep the input
                               instead when tensor_format says BF16.  Per-channel partitions take
                               this output and bf16_fallback with the tensor-level criterion only
                               (a per-channel decision is known after the codes are written)      */
    uint32_t* error_histogram; /* optional, DEVICE, [MOR_ERROR_BINS] counters of the relative-error
                               histogram of Section 4.1.3: the call adds one to the bin that holds the
                               tensor's error of Eq. 1 (tensor_stats.mean_rel_e4m3).  Bin k covers
                               [0.5 k %, 0.5 (k+1) %), the last bin everything from 5.5 % up.  The
                               caller zeroes the counters when a period starts and may hand the same
                               array to many calls (one row of the paper's heat map per tensor)      */
} mor_outputs_t;

/* Bytes of DEVICE scratch the calls below need for these `n` descriptors (one partial result per
 * 128 x 128 tile, block keys handed from the amax pre-pass to the main kernel, one amax slot per
 * tensor, one status word).  Only shapes and block shapes are read.  Returns 0 on
 * a NULL or negative argument.  The scratch needs no initialisation and 256-byte alignment. */
MOR_API size_t mor_workspace_bytes(const mor_tensor_desc_t* host_descs, int n);

/* Section 3, Algorithm 2 on one tensor: block amax, GAM scale, cast to E4M3 (and E5M2),
 * relative-error sums, per-block or per-tensor decision; writes codes, scales, selection,
 * optional BF16 copies and statistics.  Launches: tensor amax (unless supplied), the fused
 * main kernel, a small finalise kernel. */
MOR_API mor_status_t mor_analyze_quantize(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same analysis for `n` tensors with one set of launches per block shape.
 * Section 3 applies the method to a tensor and to its transpose (the operand layouts of the forward
 * and the backward GEMM).  Two neighbouring entries that name the same tensor (same x, shape, ld,
 * recipe, group_amax) with block shape (1,128) first and (128,1) second, codes wanted, no BF16 copy or
 * fake-quantised output on the first, are served by one main kernel that reads every tile of the tensor
 * once and converts it along the rows and along the columns; every output equals that of two separate
 * calls. */
MOR_API mor_status_t mor_analyze_quantize_batched(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs,
                                          int n, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Optional CUDA events (cudaEvent_t passed as void*, created and owned by the caller, NULL to
 * skip) recorded on `cuda_stream` around the three stages, so that a caller can time each
 * stage of a call separately.  Order on the stream: amax_begin, [tensor-amax kernels],
 * main_begin, [all main kernels], main_end, [all finalise kernels], finalise_end. */
typedef struct mor_stage_events {
    void* amax_begin;
    void* main_begin;
    void* main_end;
    void* finalise_end;
} mor_stage_events_t;

/* mor_analyze_quantize_batched plus stage events (host_events may be NULL). */
MOR_API mor_status_t mor_analyze_quantize_batched_ex(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs,
                                             int n, void* workspace, size_t workspace_bytes, void* cuda_stream,
                                             const mor_stage_events_t* host_events);

/* Decisions and statistics only (Eq. 1-4 evaluated, nothing quantised out): reads the
 * tensor, writes `tensor_stats` and, when non-NULL, `block_stats`, `sel`, `scale_e8m0`.
 * Serves threshold calibration and the per-tensor error statistics of Section 4.1.3. */
MOR_API mor_status_t mor_select_stats(const mor_tensor_desc_t* host_desc, mor_block_stats_t* block_stats,
                              mor_tensor_stats_t* tensor_stats, uint8_t* sel, uint8_t* scale_e8m0,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* mor_select_stats for `n` tensors in one call (tensors sharing a partition and recipe share kernel launches,
 * 16 per launch).  host_outs[i].codes, .codes_ld, .bf16_fallback and .fake_quant are ignored; tensor_stats is
 * required, block_stats / sel / scale_e8m0 / scale_f32 / error_histogram are optional as in mor_analyze_quantize.
 * Same workspace as mor_analyze_quantize_batched for the same descriptors. */
MOR_API mor_status_t mor_select_stats_batched(const mor_tensor_desc_t* host_descs, const mor_outputs_t* host_outs, int n,
                                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The first step of Algorithm 1 alone (the group's largest magnitude), with the whole tensor as the group:
 * writes max|x| over finite elements of tensor i to amax_out[i] (DEVICE, n floats), so
 * that later calls can pass it as group_amax. */
MOR_API mor_status_t mor_group_amax(const mor_tensor_desc_t* host_descs, int n, float* amax_out,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* End-to-end variant for data that lives in HOST memory: copies the tensor to the device,
 * runs mor_analyze_quantize and copies codes, scales, selection and statistics back, all
 * on `cuda_stream`; returns after enqueueing (synchronise the stream before reading).
 * In `host_desc` and `host_out` every data pointer is a HOST pointer here (pinned memory
 * makes the copies asynchronous); host_desc->group_amax must be NULL.  `device_staging`
 * is DEVICE scratch of at least mor_host_staging_bytes() bytes. */
MOR_API size_t mor_host_staging_bytes(const mor_tensor_desc_t* host_desc);
MOR_API mor_status_t mor_analyze_quantize_host(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                       void* device_staging, size_t staging_bytes, void* cuda_stream);

/* No counterpart in the paper: a packaging variant of mor_analyze_quantize for callers that cannot
 * allocate device memory where they run (a plug-in inside a runtime that owns all device memory, a
 * latency-critical loop that must avoid the synchronisation an allocation implies, a process with a
 * memory budget fixed at start-up).  Inputs and outputs are the caller's as before; the scratch
 * comes from an array of MOR_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU
 * that loads the library holds that much memory until the process exits.  The call makes no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Limit: mor_workspace_bytes(host_desc, 1) must not exceed MOR_STATIC_SCRATCH_BYTES (2 MiB).
 *     The scratch holds 56 bytes per 128 x 128 tile, and 552 with the (1,128) partition (one key
 *     per block), so the limit is roughly 600 M elements, or 62 M elements for (1,128); larger
 *     tensors are refused with MOR_ERR_STATIC_SCRATCH and nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and keeps it for the life of the process; make that first call outside any stream
 *     capture.  The address belongs to the device that is current at the call, which must be the
 *     device of `cuda_stream`.  After a cudaDeviceReset() the remembered address is stale: a process
 *     that resets a device must not use this entry point on it afterwards.
 *   - All calls share the one array, and it keeps what the previous call left in it; the call
 *     clears the part that has to start at zero.  Two calls whose kernels overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them.  */
#define MOR_STATIC_SCRATCH_BYTES (2 * 1024 * 1024)
MOR_API mor_status_t mor_analyze_quantize_static(const mor_tensor_desc_t* host_desc, const mor_outputs_t* host_out,
                                         void* cuda_stream);

MOR_API const char* mor_status_string(mor_status_t status);
MOR_API int mor_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MOR_H_ */
