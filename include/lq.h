/*
 * lq.h -- C ABI of the B200 (sm_100a) LeanQuant per-linear-layer quantisation pass.
 *
 * The pass is Algorithm 1 of the paper ("LeanQuant for LLM quantization"), split
 * into its four stages.  Notation is the paper's: W is r x c (r output rows, c input
 * columns), X is c x n (n calibration tokens), H = 2 X X^T is c x c, b bits give
 * K = 2^b grid points, B is the block width of the column loop.
 *
 * Conventions for every call
 *   - Returns LQ_OK or an lq_status error code.  Argument errors are found on the host
 *     before anything is launched; nothing is enqueued when a call fails.
 *   - All pointers named "device" are device pointers owned by the caller; they must stay
 *     valid until the stream has executed the call.  The library allocates nothing per
 *     call: scratch memory is a caller-allocated workspace sized by the matching
 *     *_workspace query (256-byte aligned).
 *   - Work is enqueued on the given CUDA stream (a cudaStream_t passed as void*) and is
 *     asynchronous.  Failures found on the device (a non-positive pivot, a non-finite
 *     value, a wait that ran out) are recorded in the handle and read by lq_sync_status.
 *   - Matrices are row-major with a leading dimension in elements.
 *   - There is no CPU fallback: without a CUDA device every compute call fails.
 */
#ifndef LQ_H_
#define LQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LQ_OK = 0,
    LQ_ERR_INVALID_ARG = 1,
    LQ_ERR_UNSUPPORTED = 2,
    LQ_ERR_WORKSPACE_TOO_SMALL = 3,
    LQ_ERR_NOT_POSITIVE_DEFINITE = 4,  /* device: pivot <= 0 in the factorisation; info = column */
    LQ_ERR_NONFINITE = 5,              /* device: NaN/Inf met; info = index */
    LQ_ERR_CUDA = 6,                   /* a CUDA runtime / driver call failed */
    LQ_ERR_TIMEOUT = 7,                /* device: a bounded wait inside a kernel ran out */
    LQ_ERR_STATIC_SCRATCH_TOO_SMALL = 8 /* lq_fit_grid_noalloc: the problem needs more than the built-in scratch */
} lq_status;

typedef enum { LQ_F32 = 0, LQ_BF16 = 1 } lq_dtype;
typedef enum {
    LQ_FEATURE_MAJOR = 0,  /* X is c x n_chunk, tokens contiguous (what the contraction reads directly) */
    LQ_TOKEN_MAJOR = 1     /* X is n_chunk x c, features contiguous (activations as a model produces them);
                              transposed into the workspace first */
} lq_layout;
typedef enum { LQ_GRID_NONUNIFORM = 0, LQ_GRID_AFFINE = 1 } lq_grid_type;
typedef enum {
    LQ_INIT_UNIFORM = 0,           /* Eq. 6: evenly spaced between the row's minimum and maximum (the paper's choice) */
    LQ_INIT_WEIGHTED_QUANTILE = 1  /* the sorted weight at the first position whose cumulative sample weight
                                      reaches (k + 1/2) / K of the row's total; rows of at most 16384 weights */
} lq_init;

typedef struct lq_handle lq_handle;

/* Settings of stages 3 and 4 (inputs of Algorithm 1 plus the search parameters of Eq. 7). */
typedef struct {
    int32_t bits;        /* b: 2, 3 or 4                                                    */
    int32_t grid_type;   /* lq_grid_type                                                    */
    float   p;           /* outlier-preservation strength of Eq. 5 / Eq. 7 (paper: 4)       */
    int32_t n_iter;      /* Lloyd iterations, fixed count, no early stop                    */
    int32_t init;        /* lq_init                                                         */
    int32_t group_size;  /* affine: weights per (S, Z) group along a row; 0 = whole row     */
    int32_t T;           /* affine: partitions of the range R (paper: 2048)                 */
    int32_t t_count;     /* affine: t, t_min and t_max run over 0..t (Appendix B)           */
    int32_t block;       /* B: columns per block of the column loop; must be 128            */
    int32_t reserved;
} lq_config;

/* ---- handle ------------------------------------------------------------------------- */

/* Creates a handle bound to CUDA device `device` (allocates a few bytes of device memory
 * for the status word, three streams of different priority and a few events: lq_prepare_hinv forks
 * its sweep onto those streams and joins them back before it returns control of the caller's stream,
 * so to the caller everything still happens in stream order; one lq_prepare_hinv per handle at a time).  Fails with LQ_ERR_CUDA when no such
 * device exists. */
int lq_create(lq_handle** out, int device);
int lq_destroy(lq_handle* h);

/* Waits for `stream`, then returns the first device-detected failure recorded since the
 * last call (LQ_OK if none) in *status with its detail in *info, and clears it. */
int lq_sync_status(lq_handle* h, void* stream, int32_t* status, int64_t* info);

/* ---- stage 1: Algorithm 1 line 3 (H <- 2 X X^T), Section 2.2 ------------------------- */

/* H[0:c,0:c] += alpha * X X^T for one chunk of tokens; call once per chunk, H (device,
 * fp32, ldh >= c, ldh % 4 == 0, 16-byte aligned) is the in/out accumulator and must be
 * zeroed by the caller before the first chunk.  Only tiles touching the upper triangle are
 * updated: entries strictly below the diagonal are unspecified until lq_hessian_finalize.
 * X: device, 16-byte aligned, bf16 or fp32; feature-major c x n_chunk (ldx >= n_chunk elements,
 * ldx * sizeof(x) % 16 == 0) or token-major n_chunk x c (ldx >= c, ldx even for bf16).
 * bf16 products are exact in the fp32 accumulator; fp32 input is split into three bf16 terms
 * and keeps fp32-level accuracy.
 * workspace: lq_hessian_workspace bytes (0 for feature-major bf16 input; ws may then be NULL):
 * the staged copy of the chunk (transposed and / or split). */
int lq_hessian_workspace(int32_t x_dtype, int32_t layout, int64_t c, int64_t n_chunk, size_t* bytes);
int lq_hessian_accumulate(lq_handle* h, void* stream, const void* X, int32_t x_dtype,
                          int32_t layout, int64_t c, int64_t n_chunk, int64_t ldx,
                          float* H, int64_t ldh, float alpha, void* ws, size_t ws_bytes);
/* Copies the upper triangle of H onto the lower one. */
int lq_hessian_finalize(lq_handle* h, void* stream, float* H, int64_t c, int64_t ldh);

/* ---- stage 2: Algorithm 1 line 4, "Cholesky and Dampening" --------------------------- */

/* H_d = H + damp_frac * mean(diag H) * I;  U = upper Cholesky factor of H_d^-1
 * (H_d^-1 = U^T U, U_jj > 0; strictly lower part of U is written as 0);
 * dinv = diag(H_d^-1).  Only the upper triangle of H is read.  A zero diagonal entry of H
 * (an input channel that never fired) is replaced by 1 and, when W is given, that column of
 * W is zeroed in place (W: device r x c of w_dtype, may be NULL).
 * H: device fp32 c x c (not modified unless U aliases it, which is allowed).
 * U: device fp32 c x c, ldu >= c.  dinv: device fp32[c].
 * Internally factorises in fp64 (blocked, tensor-core FP64 MMA trailing updates).
 * A non-positive pivot records LQ_ERR_NOT_POSITIVE_DEFINITE (info = column). */
int lq_prepare_hinv_workspace(int64_t c, size_t* bytes);
int lq_prepare_hinv(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh,
                    float damp_frac, float* U, int64_t ldu, float* dinv,
                    void* W, int32_t w_dtype, int64_t r, int64_t ldw,
                    void* ws, size_t ws_bytes);

/* d[j] = U[j][j]: the diagonal of the factor written by lq_prepare_hinv.  Algorithm 1 keeps the
 * symbol H^-1 for the Cholesky factor after line 4, so its lines 6 and 8, read to the letter,
 * weight the grid objective by the diagonal of the factor, diag(U)^-p, instead of the diagonal of
 * the inverse that Eq. 5 / Eq. 7 name.  Passing d to lq_fit_grid in place of dinv gives that
 * variant (U_jj^2 is the inverse-Hessian diagonal of weight j at the moment the column loop
 * reaches it).  U: device fp32 c x c, ldu >= c; d: device fp32[c]. */
int lq_chol_diag(lq_handle* h, void* stream, const float* U, int64_t c, int64_t ldu, float* d);

/* ---- stage 3: loss-error-aware grid, Eq. 5 (non-uniform) / Eq. 7 (affine) ------------ */

/* Non-uniform: for every row k, K = 2^bits centroids by weighted 1-D k-means with sample
 * weights dinv^(-p) (normalised by their geometric mean), started from Eq. 6 and run for
 * exactly n_iter Lloyd iterations; grid (device fp32, r x K) gets the ascending centroids.
 * Affine: for every (row, group) the pair (S, Z) of Eq. 7 with least weighted squared
 * error over (t_min, t_max) in {0..t_count}^2, first minimum in t_min-major order;
 * scale (device fp32) and zero (device int32) are r x (c / group).
 * W: device r x c (bf16 or fp32).  dinv: device fp32[c] from stage 2. */
int lq_fit_grid_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes);
int lq_fit_grid(lq_handle* h, void* stream, const lq_config* cfg, const void* W,
                int32_t w_dtype, int64_t r, int64_t c, int64_t ldw, const float* dinv,
                float* grid, float* scale, int32_t* zero, void* ws, size_t ws_bytes);

/* The paper has no counterpart for this entry point; it exists for callers that must not
 * allocate device memory.  Examples: a process in which a framework's caching allocator or a
 * serving engine has already reserved all of HBM, so that cudaMalloc fails or fragments its
 * pool; a latency-critical section that cannot afford the device-wide synchronisation that
 * cudaMalloc / cudaFree imply; a plug-in or callback context whose host forbids allocation.
 * It computes exactly what lq_fit_grid computes (same kernels, same results) but takes no
 * workspace: the scratch (the per-column sample weights and two scalars) lives in an array
 * of 256 + 8 * LQ_FIT_GRID_NOALLOC_MAX_C bytes (128.25 KiB) that is part of the library image,
 * so every GPU on which the library's kernels are loaded holds it until the process exits.
 * The call itself calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - h may be NULL, so that not even lq_create (which allocates the 16-byte status word) is
 *     needed; device-detected failures (a non-finite or non-positive dinv entry) are then
 *     recorded in an internal word that no call reads.  With a handle they are reported by
 *     lq_sync_status as usual.  The handle's device must be the current device.
 *   - c > LQ_FIT_GRID_NOALLOC_MAX_C (or any future setting whose scratch need exceeds the
 *     array) fails with LQ_ERR_STATIC_SCRATCH_TOO_SMALL before anything is launched.
 *   - The first call on each device looks up the array's device address (one-time set-up,
 *     guarded by a mutex) with that device current, and the first call of each configuration
 *     (bit width, weight type, grid type and search path) on a device opts its kernel in to the
 *     shared memory it needs; make the first call of each configuration you use before any
 *     stream capture begins.  Later calls only launch kernels.
 *   - All calls on one device share the one array.  It keeps whatever the previous call left
 *     there; nothing has to be cleared because every word a call reads it has written first.
 *     Two calls whose kernels may overlap on the GPU (different streams, no ordering between
 *     them) race on it: order them on one stream or with events.
 * All other arguments, layouts and results are those of lq_fit_grid. */
#define LQ_FIT_GRID_NOALLOC_MAX_C 16384
int lq_fit_grid_noalloc(lq_handle* h, void* stream, const lq_config* cfg, const void* W,
                        int32_t w_dtype, int64_t r, int64_t c, int64_t ldw, const float* dinv,
                        float* grid, float* scale, int32_t* zero);

/* ---- stage 4: Algorithm 1 lines 10-21, the block-wise column loop -------------------- */

/* For each block of B = 128 columns: quantise column j of every row to its grid
 * (quant_nu: nearest centroid, a weight exactly on a midpoint takes the lower one;
 * quant_aff: clip(round(w/S) + Z, 0, K-1) with the group's (S, Z)),
 * E[:, j-i] = (W[:, j] - What[:, j]) / U[j, j], feed the error back inside the block, then
 * W[:, i+B:] -= E U[i:i+B, i+B:] on the tensor cores.  W is not modified (a fp32 working
 * copy lives in the workspace).
 * codes: device uint8 r x c (ld = c), one code per byte.  W_hat: device, what_dtype, r x c
 * with ldwh, or NULL.  loss_out: device double[1] = 1/2 * sum E^2 (Eq. 3), or NULL. */
int lq_quantize_layer_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes);
int lq_quantize_layer(lq_handle* h, void* stream, const lq_config* cfg, const void* W,
                      int32_t w_dtype, int64_t r, int64_t c, int64_t ldw,
                      const float* U, int64_t ldu,
                      const float* grid, const float* scale, const int32_t* zero,
                      uint8_t* codes, void* W_hat, int32_t what_dtype, int64_t ldwh,
                      double* loss_out, void* ws, size_t ws_bytes);

/* ---- storage format: the bit columns of the paper's result tables --------------------- */

/* Packs the codes of lq_quantize_layer (one per byte) into the b-bit form that the paper's bit
 * accounting assumes (b bits per weight plus a 2^b-entry table per row for non-uniform grids, or
 * (S, Z) per group for affine ones): row i of `packed` (device, ldp >= ceil(c * bits / 8) bytes per
 * row) is the little-endian bit stream of row i's codes, code j in bits [j * bits, (j + 1) * bits).
 * Unused high bits of a row's last byte are zero. */
int lq_pack_codes(lq_handle* h, void* stream, const uint8_t* codes, int64_t r, int64_t c,
                  int32_t bits, uint8_t* packed, int64_t ldp);

/* A whole quantised layer in the form the paper's bit accounting assumes (result tables, bit columns; Appendix A):
 *   non-uniform: b-bit codes plus a 2^b-entry fp16 table per output row      -> b + 16 * 2^b / c bits per weight
 *                (4.06 / 3.03 / 2.02 at c = 4096; 4.05 / 3.02 / 2.01 averaged over a Llama-3-8B-shaped block);
 *   affine:      b-bit codes plus an fp16 scale and an int16 zero point per group -> b + 32 / g bits per weight
 *                (4.25 with groups of 128, 4.00 row-wise at these widths).
 * record (device, 16-byte aligned, lq_pack_layer_bytes bytes): a 64-byte header {magic "LQP1", bits, grid type, group size,
 * r, c, byte offsets of the three sections, total bytes}, the packed codes (row i at codes_offset + i * ceil(c * bits / 8),
 * the bit stream of lq_pack_codes), then the tables (r x 2^b fp16) or the scales (r x c/g fp16) and zero points
 * (r x c/g int16); sections start on 16-byte boundaries.  grid / scale are rounded to fp16 (round to nearest even); a
 * zero point outside int16 records LQ_ERR_UNSUPPORTED (info = its index) and is stored saturated.
 * *bits_per_weight (may be NULL) is the figure above: header and alignment padding are not counted. */
int lq_pack_layer_bytes(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes, double* bits_per_weight);
int lq_pack_layer(lq_handle* h, void* stream, const lq_config* cfg, const uint8_t* codes, int64_t r, int64_t c,
                  const float* grid, const float* scale, const int32_t* zero, void* record, size_t record_bytes);
/* The weights a record stands for: W_hat[i][j] = table[i][code] or (code - Z) * S with the record's fp16 values
 * (device, what_dtype, r x c with ldwh).  A header that does not match (cfg, r, c) records LQ_ERR_INVALID_ARG. */
int lq_unpack_layer(lq_handle* h, void* stream, const lq_config* cfg, const void* record, size_t record_bytes,
                    int64_t r, int64_t c, void* W_hat, int32_t what_dtype, int64_t ldwh);

/* For layers that share a Hessian (the q / k / v projections of a block read the same activations): lq_prepare_hinv
 * zeroes the dead input channels' columns of the one W it is given; this does the same for another layer's W.
 * H: the accumulated Hessian as lq_prepare_hinv read it (so U must not have been written over it). */
int lq_zero_dead_columns(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, void* W, int32_t w_dtype,
                         int64_t r, int64_t ldw);

/* Variant of lq_quantize_layer for affine grids in which the (S, Z) of a group are not fitted beforehand on the
 * original weights (Algorithm 1 lines 5-9) but when the column loop reaches the group's first column, on that
 * group's columns as they stand then, i.e. with the errors of all earlier columns already fed back into them
 * (the usual practice of GPTQ implementations; the paper's pseudocode fits all grids first).  The search is that
 * of lq_fit_grid (Eq. 7 with cfg->T, cfg->t_count, cfg->p and the sample weights from dinv); scale / zero
 * (r x c / group_size) are outputs.  Supported group sizes: divisors of 128 that are multiples of 4 (refitted inside the
 * in-block kernel), multiples of 128 that divide 1024, multiples of 1024, and one group per row (which is the same as
 * fitting beforehand).  Other arguments as lq_quantize_layer;
 * workspace: lq_quantize_layer_lazy_workspace bytes. */
int lq_quantize_layer_lazy_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes);
int lq_quantize_layer_lazy(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                           int64_t r, int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* dinv,
                           float* scale, int32_t* zero, uint8_t* codes, void* W_hat, int32_t what_dtype,
                           int64_t ldwh, double* loss, void* ws, size_t ws_bytes);

/* ---- activation ordering (appendix "Experiment Details": the option the paper turns on for its GPTQ baseline) ------ */

/* The columns are quantised in the order of decreasing diag(H) (most active input channels first) instead of left to
 * right: the pass runs unchanged on the permuted layer and its outputs are put back.
 *   lq_act_order      perm[k] (device int32[c]) = the column taken k-th; equal diagonal entries: lower index first.  c <= 16384.
 *   lq_permute_hessian  Hp[a][b] = H[perm[a]][perm[b]] (Hp must not be H).
 *   lq_gather_columns   dst[i][k] = src[i][perm[k]]   (W into the order of the pass);
 *   lq_scatter_columns  dst[i][perm[k]] = src[i][k]   (codes and W_hat back into the layer's own order);
 *                       elements of elem_bytes = 1, 2 or 4 bytes, leading dimensions in elements, dst must not be src.
 * With a group-wise affine grid the groups are runs of group_size columns of the permuted order, so scale / zero stay
 * in that order and a consumer needs perm beside them. */
int lq_act_order(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, int32_t* perm);
int lq_permute_hessian(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, const int32_t* perm,
                       float* Hp, int64_t ldhp);
int lq_gather_columns(lq_handle* h, void* stream, const void* src, int32_t elem_bytes, int64_t r, int64_t c, int64_t lds,
                      const int32_t* perm, void* dst, int64_t ldd);
int lq_scatter_columns(lq_handle* h, void* stream, const void* src, int32_t elem_bytes, int64_t r, int64_t c, int64_t lds,
                       const int32_t* perm, void* dst, int64_t ldd);

/* ---- Algorithm 2 (Appendix, "LeanQuant-Exact"): greedy order, full downdate per row ---- */

/* For every row, with the grid fitted beforehand by lq_fit_grid (lines 3-7 of Algorithm 2) and the row's own
 * copy of the inverse Hessian Hinv = U^T U: c times, among the weights not yet quantised take the one with
 * the least loss error (quant(w_i) - w_i)^2 / (2 Hinv_ii) (ties: lowest index), quantise it, spread its
 * error over the others by Eq. 3 and remove it from the inverse by Eq. 9.  O(c^3) operations per row: meant
 * for layers of up to a few thousand input features.  Arithmetic in fp64.
 * U is the factor written by lq_prepare_hinv (so the inverse is the damped one; damp_frac = 0 there gives
 * (2 X X^T)^-1 to the letter).  Arguments, layouts and outputs as for lq_quantize_layer, except that `loss`
 * is the sum over all weights of the loss error at the moment each was quantised (equal to
 * 1/2 sum_rows (w - w_hat) H_d (w - w_hat)^T), cfg->block is ignored and any group size dividing c is
 * accepted.  c <= 8192.  Workspace: lq_quantize_exact_workspace bytes, 256-byte aligned (the fp64 inverse
 * plus one copy of it per resident CTA, 16 GiB of copies at most).  A non-positive pivot records LQ_ERR_NOT_POSITIVE_DEFINITE
 * (info = row * c + index). */
int lq_quantize_exact_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes);
int lq_quantize_exact(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                      int64_t r, int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* grid,
                      const float* scale, const int32_t* zero, uint8_t* codes, void* W_hat,
                      int32_t what_dtype, int64_t ldwh, double* loss, void* ws, size_t ws_bytes);

/* ---- measurement aid (no counterpart in the paper) ------------------------------------- */

/* Launches one dependent-free arithmetic loop that fills the device (2048 threads per SM, eight
 * independent chains per thread, `iters` iterations) and returns in *ops (host) the number of operations
 * it executes: fp32 lane-operations (one FMA each) for LQ_PROBE_F32_FMA, flops for the two fp64 kinds.
 * A benchmark times the launch with events on `stream`; ops / time is the rate of that pipe on this
 * machine at its clocks, the denominator for the stages that are bound by it (grid fitting: fp32
 * lanes; dampen / invert / factor and Algorithm 2: fp64). */
typedef enum { LQ_PROBE_F32_FMA = 0, LQ_PROBE_F64_FMA = 1, LQ_PROBE_F64_MMA = 2 } lq_probe_kind;
int lq_peak_probe(lq_handle* h, void* stream, int32_t kind, int64_t iters, double* ops);

/* Number of CUDA kernels this library has launched in this process so far (an atomic host counter;
 * for benchmarks and tests that want to see that the kernels ran). */
uint64_t lq_launch_count(void);

/* Library version string (static storage). */
const char* lq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LQ_H_ */
