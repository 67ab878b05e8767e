/*
 * soar.h - C ABI of the SOAR NVFP4 weight quantizer for NVIDIA B200 (sm_100a).
 *
 * The library turns a bf16 weight matrix into the NVFP4 triple of the SOAR paper
 * (Sec. 3.1): 4-bit E2M1 codes, one FP8 E4M3 scale per 16 consecutive elements of
 * a row, one FP32 scale per tensor; the scales and codes are chosen by Closed-form
 * Joint Scale Optimization (Sec. 3.2, Eq. 4-6) and Decoupled Scale Search
 * (Sec. 3.3, Eq. 7-8) run as the loop of Algorithm 1.
 *
 * Conventions that hold for every call
 *   - "device" pointers are CUDA global memory owned by the caller; "host" pointers
 *     are ordinary memory.  The library never allocates or frees device memory and
 *     never synchronizes: work is enqueued on `stream` in order, so results are
 *     readable once the caller has synchronized that stream.
 *   - The int return value is a host-side status (SOAR_OK or a negative SOAR_ERR_*)
 *     for argument and launch errors; nothing is enqueued when it is an argument error.
 *     Conditions that depend on the data (non-finite input, all-zero tensor, magnitude
 *     outside the supported range) are reported in soar_result.status on the device.
 *   - Calls that share a workspace or output buffers must be ordered on one stream.
 */
#ifndef SOAR_H_
#define SOAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SOAR_OK 0
#define SOAR_ERR_INVALID_ARG (-1)      /* null pointer, bad struct size, bad count          */
#define SOAR_ERR_UNSUPPORTED (-2)      /* cols % 16, ld < cols, alignment, block != 16, ... */
#define SOAR_ERR_WORKSPACE (-3)        /* workspace missing or too small                    */
#define SOAR_ERR_CUDA (-4)             /* a CUDA runtime call or kernel launch failed       */
#define SOAR_ERR_TOO_LARGE (-5)        /* matrix exceeds the built-in scratch of soar_quantize_static,
                                          or the capacity of a pipeline slot                */

/* soar_result.status bits (device side, data dependent) */
#define SOAR_STATUS_ZERO_TENSOR 1      /* every element is zero: alpha = 1, scales = 0      */
#define SOAR_STATUS_NONFINITE 2        /* NaN or Inf in the input: outputs unspecified      */
#define SOAR_STATUS_RANGE 4            /* max |W| outside [2^-100, 2^100]: outputs unspecified */
#define SOAR_STATUS_INTERNAL 8         /* a bounded wait inside a kernel gave up: outputs unspecified */
#define SOAR_STATUS_BAD_WEIGHT 16      /* a column weight negative, not finite, or non-zero outside
                                          [2^-20, 2^20] (soar_quantize_weighted): outputs unspecified */

/* scale_layout bits */
#define SOAR_SCALES_LINEAR 1           /* row-major [rows][cols/16] bytes                   */
#define SOAR_SCALES_SWIZZLED 2         /* 128x4 tiles as Blackwell block-scaled MMA reads   */

/* presets for soar_default_cfg */
#define SOAR_PRESET_PAPER 0            /* T=15, stop 1e-3, 2 E4M3 neighbours, 101 beta (Sec. 4.1, App. B.3) */
#define SOAR_PRESET_SINGLE_PASS 1      /* T=1, no early stop, 2 neighbours, beta = {1}       */
#define SOAR_PRESET_RTN 2              /* T=0: the max-based rule of Eq. 1-3 only            */
#define SOAR_PRESET_CJSO_ONLY 3        /* Sec. 3.2 alone: T=15, stop 1e-3, nearest E4M3 code, coupled scale */
#define SOAR_PRESET_DSS_ONLY 4         /* Sec. 3.3 alone: one search (2 x 101) around the max-based start   */
#define SOAR_PRESET_COUPLED_PAIR 5     /* closed-form updates with both E4M3 codes bracketing the Eq. 6 solution,
                                          each tried with itself as the quantization scale (2 candidates per
                                          block instead of 202): T=15, stop 1e-3, coupled scale.  Not an arm of
                                          the paper; on synthetic weights it ends at the full search's error  */

/* soar_cfg.flags bits: the stand-alone arms of the paper's ablation (Table 4) */
#define SOAR_FLAG_COUPLED_SCALE 1      /* Sec. 3.2 "Refinement Scheme": one block scale quantizes and
                                          dequantizes; a candidate's quantization scale is its own E4M3
                                          value times beta, not the unrounded Eq. 6 solution times beta */
#define SOAR_FLAG_KEEP_ALPHA 2         /* skip Eq. 5: alpha stays the max-based value of Eq. 1 */
#define SOAR_FLAG_KEEP_BLOCK_SCALE 4   /* skip Eq. 6: candidate sets are centred on the stored scale
                                          (with KEEP_ALPHA: Sec. 3.3 (i),(ii) alone) */

#define SOAR_FLAG_DETERMINISTIC 8       /* bit-identical results from run to run.  By default the tensor-wide
                                          sums of Eq. 5 and of the error are binary64 additions in the order
                                          the thread blocks finish, so their last bits, and through alpha in
                                          rare cases a code, can differ between runs.  With this flag every
                                          thread block stores its sums in a slot of its own and the next kernel
                                          adds the slots in a fixed order.  Needs 56 KB more workspace per
                                          matrix (soar_workspace_bytes accounts for it).  soar_quantize,
                                          soar_quantize_batch, soar_quantize_host and the pipeline only:
                                          soar_quantize_stage and soar_quantize_weighted return
                                          SOAR_ERR_UNSUPPORTED */

#define SOAR_MAX_ITERS 64
#define SOAR_MAX_BETA 512
#define SOAR_MAX_DQ 16

/* Search settings (host memory).  Names follow Algorithm 1 and App. B.3. */
typedef struct soar_cfg {
  uint32_t struct_size;   /* sizeof(soar_cfg), checked                                      */
  int32_t block;          /* elements per E4M3 scale; 16 only (Sec. 3.1)                    */
  int32_t max_iters;      /* T of Algorithm 1, 0..SOAR_MAX_ITERS; 0 = Eq. 1-3 only           */
  float early_stop_rel;   /* stop after an iteration whose relative error gain is below this
                             (Sec. 4.1: 1e-3); <= 0 disables                                */
  int32_t n_dq;           /* E4M3 dequantization-scale candidates per block, 1..SOAR_MAX_DQ
                             (App. B.3: 2, the codes bracketing the Eq. 6 solution; 1 = the
                             nearest code; n >= 2: n/2 codes at or below, n/2 above)        */
  int32_t n_beta;         /* multipliers of the quantization scale, 1..SOAR_MAX_BETA
                             (App. B.3: 101, i.e. 0.50 .. 1.50); centred on 1.00            */
  int32_t beta_step_pct;  /* multiplier step in hundredths (App. B.3: 1)                     */
  int32_t scale_layout;   /* SOAR_SCALES_* bits: which scale outputs to write               */
  int32_t flags;          /* SOAR_FLAG_* bits; 0 = Algorithm 1                              */
} soar_cfg;

/* Per-call report (device memory, written by the last kernel of soar_quantize). */
typedef struct soar_result {
  int32_t status;                           /* SOAR_STATUS_* bits                            */
  int32_t iters_run;                        /* iterations of Algorithm 1 executed            */
  float alpha;                              /* the FP32 global scale (same as *out_global)   */
  float amax;                               /* max |W|                                       */
  double sse;                               /* sum (W - What)^2 of the returned state (Eq. 4) */
  double sse_init;                          /* same for the max-based start (Eq. 1-3)        */
  double sumsq;                             /* sum W^2                                       */
  int64_t zero_blocks;                      /* blocks whose 16 elements are all zero         */
  int64_t wide_candidates;                  /* candidate evaluations that took the binary64
                                               accumulation path (scale far below block max);
                                               soar_quantize_weighted: blocks (summed over the
                                               iterations) that visited every multiplier: the
                                               coupled arm and blocks with a zero column weight */
  double trace_alpha[SOAR_MAX_ITERS + 1];   /* alpha^(0), then alpha of each executed iteration */
  double trace_sse[SOAR_MAX_ITERS + 1];     /* error of the start, then after each iteration */
} soar_result;

/* Fill *cfg (host) with a preset.  Returns SOAR_ERR_INVALID_ARG for a null pointer or
 * unknown preset. */
int soar_default_cfg(soar_cfg* cfg, int preset);

/* Bytes of device scratch soar_quantize needs for this shape and cfg (0 on bad arguments).
 * It is a small fixed part for the tensor-wide sums of Eq. 5; 8 bytes per block of state
 * carried between iterations when cfg->max_iters > 0; and, when cfg->scale_layout lacks
 * SOAR_SCALES_LINEAR, rows*cols/16 bytes for the row-major scales the loop works on. */
size_t soar_workspace_bytes(int64_t rows, int64_t cols, const soar_cfg* cfg);

/* Bytes of the swizzled scale buffer: scales padded to multiples of 128 rows and 4 columns. */
size_t soar_swizzled_scale_bytes(int64_t rows, int64_t cols);

/*
 * Quantize one matrix with Algorithm 1 (max-based start of Eq. 1; per iteration the
 * global scale of Eq. 5, the block scales of Eq. 6 and the search of Eq. 8 over
 * cfg->n_beta x cfg->n_dq candidate pairs; early stop per Sec. 4.1).
 *
 *   W_bf16             device, read only: rows x cols bf16, row r at W + r*ld elements;
 *                      blocks are 16 consecutive columns.  Base 16-byte aligned, ld % 8 == 0,
 *                      ld >= cols, cols % 16 == 0, rows*cols/16 < 2^31.
 *   cfg                host.
 *   out_fp4_packed     device, rows*cols/2 bytes, 16-byte aligned.  Byte k of row r holds
 *                      columns 2k (low nibble) and 2k+1 (high nibble); a nibble is
 *                      sign<<3 | E2M1 magnitude code (0,.5,1,1.5,2,3,4,6 -> 0..7); the sign
 *                      bit is the input's sign bit, also on zeros.
 *   out_e4m3_scales    device, rows*cols/16 bytes row-major, or NULL when cfg->scale_layout
 *                      lacks SOAR_SCALES_LINEAR.  An all-zero block gets scale byte 0x00.
 *   out_e4m3_scales_sw device, soar_swizzled_scale_bytes() bytes, or NULL when
 *                      cfg->scale_layout lacks SOAR_SCALES_SWIZZLED.  Padding bytes are zero.
 *   out_global_fp32    device, one float: alpha, so that What = code value * alpha * scale (Eq. 3).
 *   workspace          device scratch of at least soar_workspace_bytes(), 256-byte aligned;
 *                      contents before the call are ignored, after it unspecified.
 *   out_result         device, one soar_result, or NULL.
 *   stream             a cudaStream_t passed as void* (NULL = the default stream).
 */
int soar_quantize(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                  const soar_cfg* cfg, void* out_fp4_packed, void* out_e4m3_scales,
                  void* out_e4m3_scales_sw, float* out_global_fp32, void* workspace,
                  size_t workspace_bytes, soar_result* out_result, void* stream);

/* One matrix of a batch: the arguments of soar_quantize that differ per matrix. */
typedef struct soar_tensor_desc {
  const void* W_bf16;        /* device, rows x cols bf16, row stride ld                       */
  int64_t rows, cols, ld;
  void* out_fp4_packed;      /* device, rows*cols/2 bytes                                     */
  void* out_e4m3_scales;     /* device, rows*cols/16 bytes, or NULL (see soar_quantize)       */
  void* out_e4m3_scales_sw;  /* device, soar_swizzled_scale_bytes(), or NULL                  */
  float* out_global_fp32;    /* device, one float                                             */
  soar_result* out_result;   /* device, or NULL                                               */
} soar_tensor_desc;

/* Bytes of device scratch soar_quantize_batch needs: the sum of soar_workspace_bytes over the
 * matrices (0 on bad arguments). */
size_t soar_batch_workspace_bytes(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg);

/*
 * Algorithm 1 on n independent matrices with shared settings; every matrix gets exactly the
 * outputs soar_quantize would give it.  The matrices' tiles are walked as one sequence by the
 * same kernels (up to 16 matrices per launch), so a model's many small matrices cost a few
 * launches per group instead of a few per matrix; matrices that stop early (Sec. 4.1) drop
 * out of later iterations on their own.  `tensors` is host memory (n descriptors, read before
 * the call returns); `workspace` is device scratch of soar_batch_workspace_bytes(), 256-byte
 * aligned.  Argument errors of any matrix are returned before anything is enqueued.
 */
int soar_quantize_batch(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * The accumulators at the head of a workspace.  Matrix i of a batch owns the
 * SOAR_WORKSPACE_HEADER_BYTES bytes at byte i * SOAR_WORKSPACE_HEADER_BYTES of `workspace`
 * (soar_quantize: i = 0), laid out as below.  They are all that couples the blocks of a tensor
 * (Algorithm 1: the maximum of Eq. 1, the two sums of Eq. 5, the error of Sec. 4.1's stop), and
 * they are public for one purpose: a caller that splits a tensor's rows over several GPUs runs
 * soar_quantize_stage on each part and, between stages, combines these fields over the parts.
 */
#define SOAR_WORKSPACE_HEADER_BYTES 2048
typedef struct soar_workspace_header {
  uint32_t amax_bits;               /* bf16 bit pattern of max |W|: combine with max           */
  uint32_t error;                   /* non-zero stops the remaining stages: combine with OR/max */
  uint64_t zero_blocks;             /* counters for the report: sum                            */
  uint64_t wide;
  double sumsq;                     /* sum W^2: sum                                            */
  double num[SOAR_MAX_ITERS + 1];   /* stage s: sum A_b * scale_b      (numerator of Eq. 5): sum   */
  double den[SOAR_MAX_ITERS + 1];   /* stage s: sum B_b * scale_b^2    (denominator of Eq. 5): sum */
  double gsum[SOAR_MAX_ITERS + 1];  /* stage s: error minus sum W^2    (Eq. 4): sum            */
} soar_workspace_header;

/*
 * soar_quantize_batch one stage at a time, for tensors whose rows are split over several
 * GPUs (or several calls).  The stages, in order: SOAR_STAGE_AMAX (clears the headers; writes
 * amax_bits, sumsq), SOAR_STAGE_INIT (stage-0 entries of num, den, gsum; zero_blocks),
 * iteration t = 0 .. max_iters-1 passed as `stage` = t (entries t+1 of num, den, gsum; wide),
 * SOAR_STAGE_FINALIZE (alpha, report, swizzled scales).  Each stage reads the header entries the
 * earlier stages wrote, so a caller that has split a tensor combines, after every stage, the
 * fields that stage wrote over all parts (sum or max as marked above, e.g. with an all-reduce
 * on the same stream) and every part then continues with the whole tensor's values: alpha, the
 * early stop and the report come out as for the unsplit tensor, up to the order of the
 * binary64 additions.  Run over one part with nothing combined, the stages in order are
 * exactly soar_quantize_batch.  Arguments, checks and error codes as soar_quantize_batch; an
 * unknown stage returns SOAR_ERR_INVALID_ARG.  The swizzled scale layout is tiled by 128 rows,
 * so a part's rows must be a multiple of 128 for its swizzled output to be a slice of the
 * whole tensor's.
 */
#define SOAR_STAGE_AMAX (-3)
#define SOAR_STAGE_INIT (-2)
#define SOAR_STAGE_FINALIZE (-1)
int soar_quantize_stage(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg, void* workspace,
                        size_t workspace_bytes, int stage, void* stream);

/* Device staging buffers for soar_quantize_host (all device memory, caller-owned, same sizes
 * and alignment as the matching soar_quantize arguments; W holds rows*ld bf16 elements). */
typedef struct soar_staging {
  void* W;
  void* packed;
  void* scales;        /* NULL when cfg lacks SOAR_SCALES_LINEAR   */
  void* scales_sw;     /* NULL when cfg lacks SOAR_SCALES_SWIZZLED */
  float* alpha;
  soar_result* result; /* NULL when no report is wanted            */
  void* workspace;
  size_t workspace_bytes;
} soar_staging;

/*
 * soar_quantize for a matrix that lives in host memory (Algorithm 1, same outputs): copies
 * W host->device into dev->W, runs soar_quantize on the staging buffers, and copies the
 * codes, scales, alpha and report back to the host pointers, all enqueued in order on
 * `stream`.  Host buffers should be page-locked for the copies to be asynchronous; they are
 * valid after the caller synchronizes the stream.  out_*_host pointers follow the rules of
 * the matching soar_quantize outputs (NULL where the layout is not requested).
 */
int soar_quantize_host(const void* W_host, int64_t rows, int64_t cols, int64_t ld,
                       const soar_cfg* cfg, void* out_fp4_packed_host, void* out_e4m3_scales_host,
                       void* out_e4m3_scales_sw_host, float* out_global_host,
                       soar_result* out_result_host, const soar_staging* dev, void* stream);

/*
 * Overlapped form of soar_quantize_host for a list of matrices in host memory (Algorithm 1 on each;
 * same outputs).  A pipeline owns three caller-supplied streams and a ring of caller-supplied device
 * staging slots: the copy of matrix i+1 into its slot (first stream) runs while matrix i is
 * quantized (second stream) and the results of matrix i-1 are copied back (third stream), chained
 * by the pipeline's own events, so that on a machine whose host link is slower than the quantizer
 * the list costs about as much as its copies.  Slots are taken in turn and the turn carries over
 * from one soar_pipeline_run to the next, so a new list starts on the slot that has been free the
 * longest and its copies overlap the previous list's work.
 *
 *   soar_pipeline_create   slots: n_slots >= 1 descriptors (host memory, copied): device buffers as in
 *                          soar_staging plus their capacities in bytes; a matrix fits a slot when its
 *                          rows*ld*2 input bytes, its outputs and its workspace need fit.  The three streams
 *                          (cudaStream_t as void*) must differ from each other and belong to the
 *                          current device.  Allocates no device memory (host bookkeeping and CUDA
 *                          events only).  *out receives the handle.
 *   soar_pipeline_run      enqueues the n matrices `mats` (host memory, read before the call returns).
 *                          Host buffers should be page-locked; they are valid once
 *                          soar_pipeline_synchronize (or a synchronize of the third stream) returns.
 *                          col_weights: NULL, or n device pointers (`cols` floats each, as in
 *                          soar_quantize_weighted; a NULL entry means unweighted); slots used with
 *                          weights need a workspace of soar_weighted_workspace_bytes().  Every
 *                          matrix is checked against every rule of soar_quantize and against the
 *                          slot capacities before anything is enqueued.
 *   soar_pipeline_synchronize  blocks the calling host thread until everything enqueued so far has
 *                          landed in the host buffers.
 *   soar_pipeline_destroy  waits for the pipeline's work, then releases its events.
 * Not thread-safe: one host thread drives a pipeline at a time.
 */
typedef struct soar_slot {
  soar_staging dev;          /* device buffers of the slot (see soar_staging)                         */
  size_t W_bytes;            /* capacity of dev.W                                                      */
  size_t packed_bytes;       /* capacity of dev.packed                                                 */
  size_t scales_bytes;       /* capacity of dev.scales (0 when NULL)                                   */
  size_t scales_sw_bytes;    /* capacity of dev.scales_sw (0 when NULL)                                */
} soar_slot;

typedef struct soar_host_matrix {
  const void* W_host;              /* rows x cols bf16, row stride ld elements                         */
  int64_t rows, cols, ld;
  void* out_fp4_packed_host;       /* rows*cols/2 bytes                                                */
  void* out_e4m3_scales_host;      /* rows*cols/16 bytes, or NULL when the layout is not requested     */
  void* out_e4m3_scales_sw_host;   /* soar_swizzled_scale_bytes(), or NULL                             */
  float* out_global_host;          /* one float                                                        */
  soar_result* out_result_host;    /* or NULL                                                          */
} soar_host_matrix;

typedef struct soar_pipeline soar_pipeline;
int soar_pipeline_create(soar_pipeline** out, const soar_slot* slots, int n_slots, void* stream_h2d,
                         void* stream_compute, void* stream_d2h);
int soar_pipeline_run(soar_pipeline* pipe, const soar_host_matrix* mats, int n, const soar_cfg* cfg,
                      const float* const* col_weights);
int soar_pipeline_synchronize(soar_pipeline* pipe);
void soar_pipeline_destroy(soar_pipeline* pipe);

/*
 * Reconstruction error of a stored NVFP4 triple against W (Eq. 3 and Eq. 4):
 * *out_sse = sum (W - code value * alpha * scale)^2 and *out_sumsq = sum W^2, both
 * accumulated in binary64.  All pointers device; scale_layout is exactly one SOAR_SCALES_*
 * bit and names the layout of e4m3_scales.  W, rows, cols, ld as in soar_quantize.
 */
int soar_dequant_error(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                       const void* fp4_packed, const void* e4m3_scales, int scale_layout,
                       const float* global_fp32, double* out_sse, double* out_sumsq,
                       void* stream);

/*
 * SOAR with a column-weighted objective: sum_ij h_j (W_ij - What_ij)^2, h = col_weight.
 * This is the diagonal form of the output-distortion objective ||(W - What) X||^2 that the
 * paper's Sec. 5 ("Discussions and Future Works") proposes for CJSO and DSS: h_j stands for the
 * second moment of input channel j over calibration data.  Algorithm 1 runs unchanged except
 * that every per-element term carries its column's weight: the block sums of Eq. 5 and Eq. 6
 * become A = sum h_j W_j Q_j and B = sum h_j Q_j^2, the error of Eq. 8 and of the early stop
 * (Sec. 4.1) is the weighted one, and the report's sse, sse_init and sumsq are weighted.  The
 * initialization (Eq. 1) does not depend on h; with every h_j = 1 the outputs are those of
 * soar_quantize.
 *
 *   col_weight  device, `cols` floats, 16-byte aligned, read-only.  Each must be zero or lie in
 *               [2^-20, 2^20]; anything else (negative, NaN, Inf, out of range) is reported as
 *               SOAR_STATUS_BAD_WEIGHT in out_result->status and the outputs are unspecified.
 *               Only ratios between weights matter to the minimiser.
 *   workspace   device, 256-byte aligned, >= soar_weighted_workspace_bytes(rows, cols, cfg):
 *               2 KB of accumulators plus, when max_iters > 0, 17 bytes per block (A and B in
 *               binary64 and the stored scale code), plus rows*cols/16 bytes when the row-major
 *               scale layout is not requested.
 * Every other argument, the stream semantics, ownership and the error codes are those of
 * soar_quantize.  The block sums are accumulated in binary64 in element order, so the pass is
 * bound by arithmetic, not by HBM, even with one candidate.
 *
 * soar_quantize_weighted_batch is the same on n independent matrices with shared settings, walked
 * by the same kernels (up to 16 matrices per launch) like soar_quantize_batch: `tensors` and
 * `col_weights` are host arrays of n entries (col_weights[i]: the device vector of matrix i's
 * `cols` weights), `workspace` is device scratch of soar_weighted_batch_workspace_bytes() (the sum
 * of soar_weighted_workspace_bytes over the matrices), 256-byte aligned.  Every matrix gets exactly
 * what soar_quantize_weighted gives it.
 */
size_t soar_weighted_workspace_bytes(int64_t rows, int64_t cols, const soar_cfg* cfg);
int soar_quantize_weighted(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                           const float* col_weight, const soar_cfg* cfg, void* out_fp4_packed,
                           void* out_e4m3_scales, void* out_e4m3_scales_sw, float* out_global_fp32,
                           void* workspace, size_t workspace_bytes, soar_result* out_result,
                           void* stream);
size_t soar_weighted_batch_workspace_bytes(const soar_tensor_desc* tensors, int n, const soar_cfg* cfg);
int soar_quantize_weighted_batch(const soar_tensor_desc* tensors, const float* const* col_weights, int n,
                                 const soar_cfg* cfg, void* workspace, size_t workspace_bytes,
                                 void* stream);

/*
 * soar_dequant_error under the same column weights: *out_sse = sum h_j (W - code value *
 * alpha * scale)^2 and *out_sumsq = sum h_j W^2 (binary64).  col_weight as above (not
 * validated here: a NaN weight gives NaN sums); the other arguments as soar_dequant_error.
 */
int soar_dequant_error_weighted(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                                const float* col_weight, const void* fp4_packed,
                                const void* e4m3_scales, int scale_layout, const float* global_fp32,
                                double* out_sse, double* out_sumsq, void* stream);

/*
 * MXFP4 with the decoupled scale search (Sec. 4.3, "DSS on MXFP4"): E2M1 codes in blocks of 32
 * consecutive elements of a row, one E8M0 scale byte per block (value 2^(byte - 127)), no tensor
 * scale.  The paper reports results for this combination and gives no procedure; the library
 * follows this reading of Sec. 3.3 with alpha = 1:
 *   n_beta == 0  the format's plain rule: shared exponent floor(log2 bmax) - 2, elements rounded to
 *                nearest (ties to even) and saturated at 6;
 *   n_beta >= 1  the search: the high-precision scale is Eq. 1's max-based one, D* = bmax / 6; the
 *                dequantization candidates are the n_dq E8M0 values around D* (n_dq = 1: the nearer
 *                one; n_dq >= 2: n_dq/2 at or below, n_dq/2 above; with two candidates the plain
 *                rule's exponent is always one of them), the quantization candidates D* times
 *                App. B.3's multipliers (n_beta of them, step beta_step_pct / 100, centred on 1.00);
 *                every pair is scored by Eq. 8 and the first minimum in (multiplier, code) order is kept.
 * A block whose largest magnitude is below 2^-120 is stored as a zero block (scale byte 0).
 *
 *   W_bf16            device, as soar_quantize, and cols % 32 == 0
 *   out_fp4_packed    device, rows*cols/2 bytes, 16-byte aligned, nibble layout as soar_quantize
 *   out_e8m0_scales   device, rows*cols/32 bytes, row-major
 *   out_result        device, one soar_mx_result, 8-byte aligned (required: it also carries the
 *                     call's running sums); status holds SOAR_STATUS_NONFINITE / _ZERO_TENSOR / _INTERNAL
 * One pass over W, no workspace, nothing allocated, enqueued on `stream`.
 */
typedef struct soar_mx_result {
  int32_t status;            /* SOAR_STATUS_* bits                                              */
  uint32_t amax_bits;        /* bf16 bit pattern of max |W|                                     */
  float amax;                /* max |W|                                                         */
  int32_t pad_;
  double sse;                /* sum (W - What)^2                                                */
  double sumsq;              /* sum W^2                                                         */
  double reserved;           /* internal: sse - sumsq before clamping                           */
  int64_t zero_blocks;       /* blocks stored as zero blocks                                    */
  int64_t wide_candidates;   /* candidate evaluations on the binary64 accumulation path         */
} soar_mx_result;
int soar_mx_quantize(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld, int n_dq, int n_beta,
                     int beta_step_pct, void* out_fp4_packed, void* out_e8m0_scales,
                     soar_mx_result* out_result, void* stream);

/*
 * soar_quantize without a workspace argument, for callers that must not allocate device
 * memory and have none to spare: code running inside another framework's memory pool, a
 * plugin or callback that is handed only its input and output buffers, a process whose
 * device memory is fully pre-assigned.  (The paper has no counterpart; this is a convenience
 * of the library.)  The scratch soar_quantize would take from `workspace` lives in a fixed
 * array inside the library image instead, so every GPU that loads the library holds
 * SOAR_STATIC_SCRATCH_BYTES of device memory until the process exits.  The call itself
 * makes no cudaMalloc/cudaFree and calls no allocating routine.
 *
 *   - Limit: rows*cols <= SOAR_STATIC_MAX_ELEMENTS, else SOAR_ERR_TOO_LARGE is returned and
 *     nothing is enqueued.  All other arguments, outputs and return codes are those of
 *     soar_quantize.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) before it enqueues anything; make that first call outside any stream capture.
 *   - There is one array per device, shared by every call and every stream.  The call
 *     clears the part that must start at zero, so leftovers of earlier calls do no harm,
 *     but two calls that overlap on the GPU (different streams, no ordering) race on it
 *     and give unspecified results: order them, or use soar_quantize with separate
 *     workspaces.
 */
#define SOAR_STATIC_MAX_ELEMENTS (1ll << 24)                 /* e.g. one 4096 x 4096 matrix */
#define SOAR_STATIC_SCRATCH_BYTES (2048 + 9 * (1 << 20))    /* 8 B of state + 1 scale byte per block */
int soar_quantize_static(const void* W_bf16, int64_t rows, int64_t cols, int64_t ld,
                         const soar_cfg* cfg, void* out_fp4_packed, void* out_e4m3_scales,
                         void* out_e4m3_scales_sw, float* out_global_fp32,
                         soar_result* out_result, void* stream);

/* Number of kernels soar_quantize enqueues for this cfg (host-side bookkeeping for callers
 * that count launches); 0 on bad arguments. */
int soar_quantize_launches(const soar_cfg* cfg);

/* Launch tracing for benchmarks (no counterpart in the paper).  Between soar_trace_begin()
 * and soar_trace_end(), every kernel the library launches is bracketed by two CUDA events on
 * its stream.  soar_trace_end() waits for those events and writes, per kernel name, the
 * number of launches and the summed device time in milliseconds into out[0..capacity)
 * (host); *count receives the number of distinct kernels seen.  Process-wide, not re-entrant. */
typedef struct soar_trace_entry {
  char kernel[32];
  int64_t launches;
  double total_ms;
} soar_trace_entry;
int soar_trace_begin(void);
int soar_trace_end(soar_trace_entry* out, int capacity, int* count);

/*
 * Self-test of an arithmetic shortcut (no counterpart in the paper).  The candidate loop of
 * soar_quantize needs 1/(alpha * dq) rounded to nearest (the reciprocal of Eq. 2's divisor) for
 * every candidate; it computes it as the hardware's approximate reciprocal plus one Newton
 * step, which on sm_100a equals the correctly rounded reciprocal for every input of the range
 * it is used on.  This call counts, on the device, the binary32 inputs with biased exponent
 * lo_exp..hi_exp (2 <= lo_exp <= hi_exp <= 252; all 2^23 significands each) on which the two
 * differ, into *out_mismatches (device, 8 bytes).  The full range takes about two seconds.
 */
int soar_selftest_reciprocal(int lo_exp, int hi_exp, unsigned long long* out_mismatches, void* stream);

/*
 * Test hook for the kernels' bounded waits (no counterpart in the paper).  Every wait inside a
 * kernel (a consumer warp waiting for the tile its producer fetches) counts its polls and gives
 * up at a limit; the call then reports SOAR_STATUS_INTERNAL instead of hanging.  While the hook
 * is on, kernels launched afterwards fetch no tiles at all, so their consumers' waits run to
 * the limit (a quarter of a million polls, about a second per kernel) with no copy in flight:
 * the pass kernels then return, the remaining kernels of the call return at once,
 * soar_result.status carries SOAR_STATUS_INTERNAL and the outputs are unspecified.  on = 0
 * restores normal operation.  Process-wide; not for production use.
 */
int soar_debug_fail_waits(int on);

/* Text for a host-side return value. */
const char* soar_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SOAR_H_ */
