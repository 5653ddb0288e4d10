/*
 * bof4.h -- C ABI of the B200 (sm_100a) library for block-wise 4-bit optimal-float
 * quantisation: BOF4 (absolute block maximum), BOF4-S (signed block maximum), the data-driven
 * EM/Lloyd codebook fit, and outlier-preserving quantisation (OPQ).
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 *  - Pointers named d_* are DEVICE pointers (memory of the current CUDA device); pointers
 *    named h_* and plain value arguments live on the HOST.  The library never takes ownership:
 *    the caller allocates and frees every buffer, including the workspace.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All work is
 *    enqueued on that stream and the call returns without synchronising; outputs are valid once
 *    the stream has reached the end of the enqueued work.
 *  - Weights are a flattened tensor of n elements cut into B = n / block_size contiguous blocks
 *    (Sec. 2.1).  block_size is a power of two from 32 to 4096.  opq_split_static and the gemv
 *    need n (cols) to be a multiple of it.  Every other entry point, the codebook fit
 *    included, also takes a ragged tensor: its last block is simply shorter (its own
 *    maximum; its own mean and deviation over its own length, the two tree sums padded with
 *    zeros to the next power of two; a one-weight block has no outliers), there are
 *    ceil(n / block_size) block constants and (n + 1) / 2 code bytes, and a code byte that holds a
 *    single weight has a zero low nibble.  The paper only uses whole blocks.
 *  - Weight tensors, code arrays and dequantised outputs are accessed with 32-byte vector
 *    instructions: their device pointers must be 32-byte aligned (BOF4_ERR_INVALID_ARG if not).
 *  - A codebook is 16 fp32 reconstruction levels in ASCENDING order, device resident.  Code c
 *    (0..15) is the 0-based rank of the level; decision thresholds are the fp32 midpoints
 *    (xhat[j] + xhat[j+1]) * 0.5f and a value equal to a threshold belongs to the upper level
 *    (Sec. 3.2: regions [xi(l-1), xi(l)), nearest-neighbour rule).
 *  - Every function returns a status (BOF4_OK = 0, negative = error).  On error nothing has
 *    been enqueued.  bof4_last_error() gives a message for the calling thread's last error.
 *  - All fp32 arithmetic that decides a stored value (block constant, normalisation, threshold
 *    comparison, dequantisation product, OPQ block statistics) is IEEE-754 round-to-nearest-even
 *    without flush-to-zero and without fused contraction.  Inputs must be finite.
 */
#ifndef BOF4_H
#define BOF4_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Exported from the shared library (the rest of it is built with hidden visibility). */
#if defined(__GNUC__)
#define BOF4_API __attribute__((visibility("default")))
#else
#define BOF4_API
#endif

/* ---- status codes ---- */
#define BOF4_OK 0
#define BOF4_ERR_INVALID_ARG (-1) /* NULL pointer, negative size, bad enum value            */
#define BOF4_ERR_SHAPE (-2)       /* block size unsupported, n not a multiple where it must be, n too large */
#define BOF4_ERR_DTYPE (-3)       /* dtype code unknown or combination not supported        */
#define BOF4_ERR_WORKSPACE (-4)   /* workspace NULL, misaligned or smaller than required    */
#define BOF4_ERR_CAPACITY (-5)    /* outlier list capacity negative / too large, or (bof4_outlier_count) exceeded */
#define BOF4_ERR_CUDA (-6)        /* a CUDA runtime call failed (message has the reason)    */

/* ---- enums (plain ints in the signatures) ---- */
#define BOF4_F32 0  /* IEEE binary32 */
#define BOF4_BF16 1 /* bfloat16      */

#define BOF4_NORM_ABS 0    /* block constant = max_i |w_i|                    (Eq. 1) */
#define BOF4_NORM_SIGNED 1 /* block constant = the element of largest |w_i|   (Eq. 4) */

#define BOF4_METRIC_MSE 0 /* weighted-mean centroid   (Eq. 6) */
#define BOF4_METRIC_MAE 1 /* weighted-median centroid (Eq. 8) */
/* The same two criteria on the NORMALISED weights (App. D): every sample has weight 1, i.e. the
 * plain mean / plain median of textbook Lloyd, and the error is measured on x, not on w. */
#define BOF4_METRIC_MSE_NORMALIZED 2
#define BOF4_METRIC_MAE_NORMALIZED 3

#define BOF4_OP_EM 0  /* bof4_em_step / bof4_fit_codebook workspace */
#define BOF4_OP_OPQ 1 /* opq_split / bof4_quantize_opq workspace    */

#define BOF4_LEVELS 16

/*
 * Result of one expectation + accumulation pass (device resident, written by bof4_em_step).
 * Index l is the 0-based level.  MSE (Eq. 6, App. B.3):
 *     s1[l] = sum over members of m^2 * x,   s0[l] = sum over members of m^2,
 *     err_sum = sum over all weights of (w - m * xhat[code])^2.
 * MAE (Eq. 8, App. B.3):
 *     s0[l] = sum over members of |m| (total weight of the weighted median), s1[l] = 0,
 *     median[l] = weighted median of the members (the first sample, in ascending order, whose
 *     cumulative weight reaches half of s0[l]); the input level where s0[l] == 0,
 *     err_sum = sum over all weights of |w - m * xhat[code]|.
 *     The weights |m| enter the selection as 31-bit fixed-point integers relative to the largest
 *     |w| of the data (all sums are integer sums, hence independent of their order): exact for
 *     |m| down to 2^-7 (fp32 weights) or 2^-23 (bf16 weights) of that magnitude, truncated below
 *     and zero beyond 2^-31 of it.  The median is the exact weighted median unless the truncated
 *     parts add up to more than the margin by which the cumulative weight passes half of s0[l]
 *     at the selected sample; s0[l] is the sum of the fixed-point weights, rescaled.
 * For the normalised-domain metrics m^2 and |m| are replaced by 1 and w by x in these sums.
 * count[l] is the number of members of region l, n_total the number of weights seen.
 * For MSE median[l] is the centroid s1[l]/s0[l] rounded to fp32 (input level where s0[l] == 0).
 */
typedef struct bof4_em_stats {
    double s1[BOF4_LEVELS];
    double s0[BOF4_LEVELS];
    uint64_t count[BOF4_LEVELS];
    double err_sum;
    int64_t n_total;
    float median[BOF4_LEVELS];
} bof4_em_stats;

/*
 * Bytes of device workspace an operation needs for tensors of at most n_max elements.  Host
 * function, no CUDA call.  The workspace must be 256-byte aligned.  Returns 0 for invalid arguments.
 *   op = BOF4_OP_EM : partial records of the deterministic two-stage reduction and, for
 *                     metric = MAE, the per-level selection histograms and candidate lists.
 *                     n_max = the TOTAL number of weights of the tensor list.  The candidate lists
 *                     grow with it (n_max / 8 bytes, between 8 MiB and 1 GiB); any workspace of at
 *                     least bof4_workspace_bytes(BOF4_OP_EM, 0, ...) is accepted, a smaller one
 *                     than asked for here only costs the MAE fit one more pass over the data per
 *                     iteration.  Results do not depend on the workspace size.
 *   op = BOF4_OP_OPQ: per-tile outlier staging and tile offsets of the ordered compaction.
 */
BOF4_API size_t bof4_workspace_bytes(int op, int64_t n_max, int block_size, int metric);

/*
 * One E+M accumulation pass with the codebook held fixed (Sec. 3.2; Eq. 6 or Eq. 8 with the
 * error of App. B.3 in the un-normalised weight domain) over the union of n_tensors tensors.
 *   h_w       host array of n_tensors DEVICE pointers to the tensors (dtype w_dtype each)
 *   h_n       host array of n_tensors element counts (any length; every tensor is cut into blocks
 *             from its own start, and a length that is not a multiple of block_size ends in a
 *             shorter block with its own constant: blocks never run across two tensors)
 *   d_codebook  [16] fp32 levels, read only
 *   d_stats   out: one bof4_em_stats record
 *   d_ws      workspace of at least bof4_workspace_bytes(BOF4_OP_EM, max_t h_n[t], ...)
 * The sums are accumulated in a fixed order that depends only on the shapes, so two calls on
 * the same inputs give bit-identical statistics.
 */
BOF4_API int bof4_em_step(const void* const* h_w, const int64_t* h_n, int n_tensors, int w_dtype,
                 int block_size, int norm, int metric, const float* d_codebook,
                 bof4_em_stats* d_stats, void* d_ws, size_t ws_bytes, void* stream);

/*
 * `iters` Lloyd iterations in place on d_codebook (Sec. 3.2): thresholds from the current
 * levels, assignment, then every level whose bit is NOT set in fixed_mask and whose region has
 * positive total weight is replaced by its centroid (weighted mean, Eq. 6, or weighted median,
 * Eq. 8); levels with their bit set keep their value ("initialise and skip recomputation").
 *   d_codebook  in: initial levels (ascending), out: fitted levels
 *   d_err_log   [iters] fp64 or NULL: entry t = mean error (MSE or MAE over all weights,
 *               un-normalised domain) of the levels that ENTER iteration t
 * No host synchronisation happens inside; the whole loop is enqueued on `stream`.
 */
BOF4_API int bof4_fit_codebook(const void* const* h_w, const int64_t* h_n, int n_tensors, int w_dtype,
                      int block_size, int norm, int metric, float* d_codebook,
                      uint32_t fixed_mask, int iters, double* d_err_log, void* d_ws,
                      size_t ws_bytes, void* stream);

/*
 * M step of a fit whose E-step statistics come from several bof4_em_step calls - the joint fit
 * over the shards of several GPUs: every GPU runs bof4_em_step on its shard, the records are
 * gathered in rank order (432 bytes per GPU and iteration, the only exchange the path needs), and
 * every GPU calls this with the same records, so that all hold the same levels (Sec. 3.2, Eq. 6:
 * the centroid is a ratio of sums, and sums over shards add).  The records are summed in index
 * order in fp64.  MSE metrics only: a weighted median of a union (Eq. 8) cannot be merged from
 * per-shard medians (BOF4_ERR_INVALID_ARG).
 *   d_stats     device, n_records records as written by bof4_em_step with the levels in d_codebook
 *   d_codebook  in: the levels the records were computed with; out: free levels updated
 *   d_err_slot  out or NULL: mean error of the incoming levels over all records' weights
 *   d_total     out or NULL: the summed record
 */
BOF4_API int bof4_m_step(const bof4_em_stats* d_stats, int n_records, int metric, float* d_codebook,
                uint32_t fixed_mask, double* d_err_slot, bof4_em_stats* d_total, void* stream);

/*
 * Block-wise quantisation (Sec. 2.1 Eq. 1-3, Sec. 3.1 Eq. 4): per block the constant m,
 * x = w / m (x = 0 for an all-zero block), code = region of x.
 *   d_codes   out [(n+1)/2] bytes; byte k = (code[2k] << 4) | code[2k+1]
 *   d_scales  out [ceil(n/block_size)] block constants, dtype scale_dtype.  The constant is stored
 *             exactly: scale_dtype must equal w_dtype, or be BOF4_F32 for bf16 weights.
 */
BOF4_API int bof4_quantize(const void* d_w, int w_dtype, int64_t n, int block_size, int norm,
                  const float* d_codebook, uint8_t* d_codes, void* d_scales, int scale_dtype,
                  void* stream);

/*
 * Outlier split of OPQ alone (Sec. 3.3 Eq. 9, App. E): per block the corrected sample standard
 * deviation sigma_b (two-pass formula in fp32, balanced binary summation tree over the block);
 * w is an outlier iff |w| > sigma_b * tau with tau = F_M^{-1}(q) (see bof4_opq_threshold).
 *   d_w_clean  out [n] copy of w with outliers replaced by +0 (same dtype), or NULL
 *   d_out_idx  out [capacity] int32 flattened indices of the outliers, ASCENDING
 *   d_out_val  out [capacity] bf16 outlier values (round-to-nearest-even from fp32 weights)
 *   d_n_out    out: the true number of outliers, also when it exceeds `capacity` (then only
 *              the first `capacity` entries are written)
 * n must be below 2^31.  Check the count with bof4_outlier_count before relying on the list.
 */
BOF4_API int opq_split(const void* d_w, int w_dtype, int64_t n, int block_size, float tau,
              void* d_w_clean, int32_t* d_out_idx, void* d_out_val, int64_t capacity,
              int64_t* d_n_out, void* d_ws, size_t ws_bytes, void* stream);

/*
 * Second half of the two-call pattern of the outlier lists (Sec. 3.3: outliers are PRESERVED, so
 * a list that did not fit must not pass unnoticed).  opq_split, opq_split_static and
 * bof4_quantize_opq are asynchronous and can only leave the true count in *d_n_out; this call
 * waits for `stream`, copies the count to the host and compares it with the capacity that was
 * passed to the producing call.
 *   d_n_out   device: the count written by the producing call on the same stream
 *   h_n_out   host, out (may be NULL): the true number of outliers
 * Returns BOF4_OK when count <= capacity, BOF4_ERR_CAPACITY when outliers were dropped (the
 * message names the capacity that would have sufficed; codes, scales and the stored part of the
 * list are valid, so only the producing call has to be repeated with larger arrays).
 * This is the one entry point that synchronises (the stream it is given, nothing else).
 */
BOF4_API int bof4_outlier_count(const int64_t* d_n_out, int64_t capacity, int64_t* h_n_out, void* stream);

/*
 * opq_split without a workspace argument and without any allocation.  (The paper has no
 * counterpart; this is a convenience of the library.)
 *
 * Meant for callers that are not in a position to obtain device memory: code that runs while
 * another component owns the whole device-memory pool, a plug-in whose host framework forbids
 * cudaMalloc / cudaFree on its streams because those calls synchronise the device, or a
 * start-up path that runs before the application's allocator exists.  The scratch that
 * opq_split takes from d_ws (tile counts, chunk offsets, staging slots) lives instead in a
 * 4 MiB array inside the library image; every GPU that loads the library holds that array
 * until the process exits.
 *
 *   - Same arguments, outputs and bit-exact results as opq_split, minus d_ws / ws_bytes, for
 *     tensors of whole blocks: n must be a multiple of block_size (BOF4_ERR_SHAPE otherwise; the
 *     ragged last block of opq_split is not offered here).
 *   - n is limited to 2^24 weights per call (BOF4_ERR_SHAPE beyond; split larger tensors at
 *     multiples of block_size and add the chunk's first index to its outlier indices, or use
 *     opq_split).
 *   - The first call on each device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.  The address
 *     is remembered per device ordinal for the life of the process: after a cudaDeviceReset of
 *     that device the remembered address is stale and this entry point must not be used again.
 *   - All calls on one device share the one array.  Every call rewrites each cell before it
 *     reads it, so nothing has to be cleared between calls, but two calls whose kernels
 *     overlap on the GPU (different streams, no ordering between them) race on it: order them.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine.
 */
BOF4_API int opq_split_static(const void* d_w, int w_dtype, int64_t n, int block_size, float tau,
                     void* d_w_clean, int32_t* d_out_idx, void* d_out_val, int64_t capacity,
                     int64_t* d_n_out, void* stream);

/*
 * OPQ fused with quantisation in one read of the weights (Sec. 3.3): outliers are listed as in
 * opq_split and replaced by zero BEFORE the block-constant search; the cleaned block is then
 * quantised as in bof4_quantize.
 */
BOF4_API int bof4_quantize_opq(const void* d_w, int w_dtype, int64_t n, int block_size, int norm,
                      const float* d_codebook, float tau, uint8_t* d_codes, void* d_scales,
                      int scale_dtype, int32_t* d_out_idx, void* d_out_val, int64_t capacity,
                      int64_t* d_n_out, void* d_ws, size_t ws_bytes, void* stream);

/*
 * Dequantisation (Eq. 3): out[i] = round_to_out_dtype( fp32(scale[b]) * xhat[code[i]] ), one
 * fp32 multiplication.  With OPQ (d_out_idx != NULL) the first min(*d_n_out, capacity)
 * outliers are then written back at their indices (Sec. 3.3, decoding side).
 *   d_out_idx / d_out_val / d_n_out  outlier list as produced by bof4_quantize_opq, or all NULL
 *   capacity   number of entries the outlier arrays can hold (ignored without OPQ)
 */
BOF4_API int bof4_dequantize(const uint8_t* d_codes, const void* d_scales, int scale_dtype, int64_t n,
                    int block_size, const float* d_codebook, const int32_t* d_out_idx,
                    const void* d_out_val, const int64_t* d_n_out, int64_t capacity,
                    void* d_out, int out_dtype, void* stream);

/*
 * bof4_quantize and bof4_dequantize (without an outlier list) over a list of tensors that share
 * block size, normalisation, codebook and dtypes: the model-wide case, where a launch and a table
 * set-up per matrix would cost as much as the matrix itself.  The rows of all tensors are dealt
 * over one grid (64 tensors per launch); results are those of n_tensors single calls, bit for bit.
 *   h_w / h_codes / h_scales / h_out   host arrays of n_tensors DEVICE pointers, one per tensor,
 *                                      each with the size, alignment and meaning of the single call
 *   h_n                                host array of n_tensors element counts (ragged lengths allowed)
 * The host arrays are read before the call returns.
 */
BOF4_API int bof4_quantize_batch(const void* const* h_w, const int64_t* h_n, int n_tensors, int w_dtype,
                        int block_size, int norm, const float* d_codebook, uint8_t* const* h_codes,
                        void* const* h_scales, int scale_dtype, void* stream);
BOF4_API int bof4_dequantize_batch(const uint8_t* const* h_codes, const void* const* h_scales, int scale_dtype,
                          const int64_t* h_n, int n_tensors, int block_size, const float* d_codebook,
                          void* const* h_out, int out_dtype, void* stream);

/*
 * Double quantisation of the block constants (Limitations; App. F).  The paper names the technique
 * and the extra sign bit per block that signed normalisation needs; it fixes no format.  Here, in
 * fp32: the constants of 256 consecutive blocks (fewer in the last group) share the group constant
 * g = max |m|; with t = g / 255, block b keeps q_b = min(255, round-half-even(|m_b| / t)) (0 when
 * t = 0) and, for norm = BOF4_NORM_SIGNED, its sign in bit (b mod 8) of byte (b div 8) of d_sign.
 * The decoder's constant is m^_b = +-(t * q_b); |m^ - m| <= g / 510 up to fp32 rounding.  The 4-bit
 * codes stay those formed with the exact constants, so the element of largest magnitude of a block
 * is no longer reconstructed exactly.  Storage: 8 (+1) bits per block and 32 bits per group.
 *   d_scales   device, n_blocks constants of scale_dtype, as written by the quantising calls
 *   d_q        out, device, n_blocks bytes
 *   d_group    out, device, ceil(n_blocks / 256) fp32
 *   d_sign     out, device, ceil(n_blocks / 8) bytes; ignored (may be NULL) for BOF4_NORM_ABS
 * One launch on `stream`, no workspace.  BOF4_ERR_INVALID_ARG / BOF4_ERR_DTYPE on bad arguments.
 */
BOF4_API int bof4_scales_compress(const void* d_scales, int scale_dtype, int64_t n_blocks, int norm,
                         uint8_t* d_q, float* d_group, uint8_t* d_sign, void* stream);

/*
 * The decoding side of the double quantisation: d_scales_out[b] = m^_b (fp32, n_blocks values),
 * to be passed to bof4_dequantize or bof4_gemv with scale_dtype = BOF4_F32.  d_sign = NULL:
 * all constants positive (absolute normalisation).  One launch on `stream`.
 */
BOF4_API int bof4_scales_expand(const uint8_t* d_q, const float* d_group, const uint8_t* d_sign,
                       int64_t n_blocks, float* d_scales_out, void* stream);

/*
 * Matrix-vector product with the 4-bit matrix decoded on the fly: Eq. 3 fused into its consumer,
 * the operation behind the paper's token-generation timings (App. E.2), with the OPQ outliers
 * applied as a sparse correction (Sec. 3.3, decoding side).  W is rows x cols, row-major, quantised
 * as one flat tensor of rows * cols weights (so a block never straddles two rows: block_size
 * divides cols).  In fp32:
 *   y[r] = sum over the blocks b of row r of  scale[b] * sum_{i in b} xhat[code[i]] * x[col(i)]
 *          + sum over the outliers k of row r of  (val[k] - scale[b(k)] * xhat[code[idx[k]]]) * x[col(idx[k])]
 * i.e. the dequantised weight is not rounded to bf16 in between, and an outlier contributes its
 * stored value instead of its quantised one.  The summation order is fixed (no atomics), so y is
 * bit-reproducible; it differs from a sequential sum by fp32 rounding only.
 *   d_codes     device, rows * cols / 2 bytes, 32-byte aligned
 *   d_scales    device, rows * cols / block_size block constants of scale_dtype
 *   cols        multiple of block_size, at most 32768
 *   d_x         device, cols values of x_dtype (BOF4_BF16 or BOF4_F32), 16-byte aligned
 *   d_out_idx / d_out_val / d_n_out / capacity   outlier list as for bof4_dequantize, or all NULL;
 *               with a list, rows * cols must fit 32-bit indices
 *   d_y         device, rows fp32 values, written
 * One launch (two with an outlier list) on `stream`; no workspace, no host synchronisation.
 */
BOF4_API int bof4_gemv(const uint8_t* d_codes, const void* d_scales, int scale_dtype, int64_t rows,
              int64_t cols, int block_size, const float* d_codebook, const void* d_x, int x_dtype,
              const int32_t* d_out_idx, const void* d_out_val, const int64_t* d_n_out,
              int64_t capacity, float* d_y, void* stream);

/*
 * The same product for a batch of right-hand sides on the tensor cores (App. E.2: the decode-side
 * consumer with several tokens in flight): Y = W_q X^T with W rows x cols as for bof4_gemv and
 * n_rhs = 16, 32, 48 or 64 right-hand sides.  Reading: the A operand is the dequantised weight
 * rounded to bf16 - bit for bit the output of bof4_dequantize (Eq. 3, round to nearest even) - X is
 * bf16, products are exact, sums are accumulated in fp32 by the tensor cores (tcgen05.mma into
 * tensor memory), whose summation order and intermediate rounding are the hardware's: the result
 * agrees with the fp64 sum of the same products within 2^-14 * sum |w x| (cols / 16 accumulation
 * steps of at most 2^-23 each for cols <= 8192 * 16).  With an outlier list (Sec. 3.3, decoding
 * side) the stored bf16 value replaces the decoded weight: a second launch adds
 * (val - decoded) * X[b][col] for every outlier, row by row in list order (fp32).
 *   rows       multiple of 128;  cols multiple of 64 and of block_size
 *   d_codes    device, rows * cols / 2 bytes, 16-byte aligned;  d_scales as for bof4_gemv
 *   d_x        device, bf16 [n_rhs][cols] (each right-hand side contiguous), 16-byte aligned
 *   d_out_idx / d_out_val / d_n_out / capacity   outlier list as for bof4_dequantize (ascending
 *              indices), or all NULL; with a list, rows * cols must fit 32-bit indices
 *   d_y        device, fp32 [rows][n_rhs], written
 *   d_status   device int, written: 0, or 1 when a bounded wait inside the kernel ran out (the result
 *              is then undefined; the kernel has still released its tensor memory and returned)
 *   d_ws       optional device workspace (16-byte aligned) of up to 8 * rows * n_rhs * 4 bytes, or NULL:
 *              with it the product is split along K into up to 8 partial products (enough CTAs to fill
 *              the GPU when rows / 128 is small) that a second launch sums in a fixed order
 * One to three launches on `stream` (preceded by a 4-byte clear of d_status); no synchronisation.
 */
BOF4_API int bof4_gemm_tc(const uint8_t* d_codes, const void* d_scales, int scale_dtype, int64_t rows,
                 int64_t cols, int block_size, const float* d_codebook, const void* d_x, int n_rhs,
                 const int32_t* d_out_idx, const void* d_out_val, const int64_t* d_n_out, int64_t capacity,
                 float* d_y, int* d_status, void* d_ws, size_t ws_bytes, void* stream);

/*
 * Data-free codebook for unit-variance Gaussian weights (Sec. 3.2 Eq. 5 / Eq. 7; App. B.2): `iters`
 * Lloyd iterations in which every free level becomes the theoretical centroid of its region,
 * a ratio (MSE) or root (MAE) of integrals over the absolute block maximum, evaluated by
 * Simpson quadrature in fp64 on the device.  Thresholds are midpoints of adjacent levels.
 *   block_size  any I >= 2 (the integrals only need I, not a power of two)
 *   metric      BOF4_METRIC_MSE or BOF4_METRIC_MAE
 *   d_codebook  in: starting levels (ascending), out: levels after `iters` iterations
 *   fixed_mask  must fix level 15 (= 1) and, for BOF4_NORM_ABS, level 0 (= -1): the outermost
 *               regions hold the point mass of the block maximum (App. B.2)
 *   d_ws        256 bytes of device workspace, 256-byte aligned (the fp64 state between iterations)
 * One small launch per iteration on `stream`; no host synchronisation.
 */
BOF4_API int bof4_theoretical_codebook(int block_size, int norm, int metric, float* d_codebook,
                              uint32_t fixed_mask, int iters, void* d_ws, size_t ws_bytes,
                              void* stream);

/*
 * The same for up to 128 problems at once (for instance every block size of a sweep under both
 * normalisations and metrics): problem p has block size h_block_size[p], normalisation
 * h_norm[p], metric h_metric[p], fixed levels h_fixed_mask[p] (host arrays, read before the call
 * returns) and its levels in d_codebooks[16 p .. 16 p + 15] (device, in/out).  All problems
 * advance together, one launch per iteration.  d_ws: 256 bytes per problem, 256-byte aligned.
 * Results equal those of n_problems single calls bit for bit.
 */
BOF4_API int bof4_theoretical_codebook_batch(int n_problems, const int* h_block_size, const int* h_norm,
                                    const int* h_metric, const uint32_t* h_fixed_mask,
                                    float* d_codebooks, int iters, void* d_ws, size_t ws_bytes,
                                    void* stream);

/*
 * Data-free codebook for ANY symmetric zero-mean weight density (Sec. 3.2 Eq. 5 / Eq. 7 before the
 * Gaussian simplification; App. B.1 for the cdf of the normalised weights given the block maximum
 * and the density of the maximum, App. B.2 for the centroid integrals).  p_W is passed as samples:
 *   d_pdf    device, n_grid fp64 values p_W(w_j) at w_j = j * w_max / (n_grid - 1), j = 0 .. n_grid-1
 *            (w >= 0 only; any positive scale: the samples are normalised to total mass 1 on
 *            [-w_max, w_max]); w_max must cover the range of the block maximum
 *   n_grid   3 ... 2^20
 * The integrals INT_0^w p_W and INT_0^w u p_W(u) du are cumulative trapezoid sums on the grid,
 * read between nodes by linear interpolation; the integrals over the block maximum are trapezoid
 * sums on the same grid, all in fp64.  Other arguments as for bof4_theoretical_codebook.
 *   d_ws     256 + 24 * n_grid bytes, 256-byte aligned
 * One set-up launch and one small launch per iteration on `stream`; no host synchronisation.
 */
BOF4_API int bof4_theoretical_codebook_general(int block_size, int norm, int metric, const double* d_pdf,
                                      int n_grid, double w_max, float* d_codebook, uint32_t fixed_mask,
                                      int iters, void* d_ws, size_t ws_bytes, void* stream);

/* ---- host helpers (no CUDA call) ---- */

/* tau = F_M^{-1}(q) for unit-variance Gaussian weights, F_M(m) = (2 G(m) - 1)^I the CDF of the
 * absolute block maximum (App. B.1): tau = G^{-1}((1 + q^(1/I)) / 2).  NaN for q outside (0,1)
 * or block_size < 1. */
BOF4_API double bof4_opq_threshold(double q, int block_size);

/* Starting codebook with the 7 negative / zero / 8 positive split of the printed codebooks
 * (Tab. 6): -1 + k/7 (k = 0..6), 0, k/8 (k = 1..8), and the fixed-level mask of the variant:
 * {-1, 0, 1} for BOF4_NORM_ABS, {0, 1} for BOF4_NORM_SIGNED (Sec. 3.1, Sec. 3.2). */
BOF4_API int bof4_default_init(int norm, float h_levels[BOF4_LEVELS], uint32_t* h_fixed_mask);

/* Message of the calling thread's most recent error ("" if none). */
BOF4_API const char* bof4_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BOF4_H */
