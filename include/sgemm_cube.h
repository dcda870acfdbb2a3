/*
 * sgemm_cube.h -- C ABI of the SGEMM-cube library for NVIDIA B200 (sm_100a).
 *
 * SGEMM-cube approximates an FP32 GEMM C = A * B (FP32 in, FP32 out) with FP16 tensor-core
 * products.  Every FP32 operand x is split into an FP16 high word and a scaled FP16 residual,
 *
 *      hi = fl16(x),     lo = fl16((x - hi) * 2^s)            (round-to-nearest-even)
 *
 * and C is rebuilt from three FP16 x FP16 -> FP32 products, dropping lo*lo:
 *
 *      C  ~=  hi_A hi_B  +  2^-s ( lo_A hi_B  +  hi_A lo_B )
 *
 * (paper: Sec. 3.3, the two-component representation, Eq. fp16_high_low; Sec. 4.2, residual
 *  scaling, Eq. sf_bounds; Sec. 4.3, Eq. recover_eqn; Sec. 4.5, the two accumulation orders,
 *  Eq. elementwise / Eq. termwise).
 *
 * Conventions shared by every entry point
 *   - All matrices are ROW-MAJOR with a leading dimension counted in elements.
 *   - Pointers named *_dev are DEVICE pointers on the handle's device; pointers named *_host are
 *     host pointers.  The caller owns every buffer it passes; the handle owns only its internal
 *     workspace.  No entry point takes ownership of or frees a caller's buffer.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Device entry
 *     points enqueue work on it and return without synchronising.
 *   - Every function returns a status code (0 = success) and never throws or exits.  Argument
 *     errors are detected before anything is enqueued.  A failure inside a kernel (a bounded
 *     wait that ran out) is recorded in a device error word and reported by sgemm_cube_check().
 *   - FP16 matrices are passed as uint16_t bit patterns (IEEE binary16).
 *   - There is no CPU fallback: on a device that is not sm_100 sgemm_cube_create fails.
 */
#ifndef SGEMM_CUBE_H_
#define SGEMM_CUBE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sgemm_cube_ctx* sgemm_cube_handle;

/* status codes */
enum {
  SGEMM_CUBE_OK = 0,
  SGEMM_CUBE_INVALID_ARG = 1,      /* null pointer, negative size, ld too small, bad enum        */
  SGEMM_CUBE_MISALIGNED = 2,       /* pointer / leading dimension violates an alignment rule    */
  SGEMM_CUBE_CUDA_ERROR = 3,       /* a CUDA runtime or driver call failed                      */
  SGEMM_CUBE_DEVICE_TIMEOUT = 4,   /* a kernel gave up on a bounded wait (see sgemm_cube_check) */
  SGEMM_CUBE_UNSUPPORTED_ARCH = 5, /* device is not compute capability 10.x                     */
  SGEMM_CUBE_ALLOC_FAILED = 6,     /* workspace allocation failed                               */
  SGEMM_CUBE_TOO_LARGE = 7         /* problem exceeds the fixed scratch of the _static variant  */
};

/* accumulation order (paper Sec. 4.5) */
enum {
  SGEMM_CUBE_TERMWISE = 0,   /* Eq. termwise: streams summed separately, combined once at the end */
  SGEMM_CUBE_ELEMENTWISE = 1, /* Eq. elementwise: per k-block, products folded into one accumulator */
  /* The reordered elementwise order that Sec. 4.5 (last paragraph) proposes and leaves unmeasured:
   * per k-block the corrections are summed first, scaled, added to the block's hi*hi product, and
   * the block enters the accumulator once: acc = acc + ((R_A B + A R_B) / s_f + A B).  Uses the
   * elementwise k-block option.  Accepted wherever an accumulation order is.  For scale_exp <= 15
   * the block's value is formed inside the tensor core's accumulator (the instruction that adds
   * the first hi*hi product scales the accumulated corrections by 2^-s), which makes this the
   * fastest of the per-block orders: 450 against 340 TFLOP/s for the plain elementwise order at
   * 8192^3 (termwise 470). */
  SGEMM_CUBE_ELEMENTWISE_REORDERED = 2
};

/* options for sgemm_cube_set_option */
enum {
  /* Length, in k, of a chain accumulated inside the tensor core before it is added, in FP32 with
   * round-to-nearest, to the running sum held in registers (termwise: the hi*hi stream; the
   * correction stream is carried whole).  Multiple of 64, default 128.  This is the k-block g
   * of Sec. 4.5 as realised on this hardware.  The tensor core truncates (rounds toward zero)
   * each time it adds a 16-deep group of products to its accumulator; on data of one sign that
   * bias adds up along a chain, about 0.5 ulp per 16 k (measured Frobenius error on U[0,1)
   * inputs: 1.9e-7 / 4.7e-7 / 1.1e-6 for k-blocks 64 / 128 / 256, FP32 GEMM 4.3e-7; on
   * symmetric data 1.5e-7 / 2.1e-7 / 3.5e-7).  Shorter blocks cost throughput: about 2 % from
   * 256 to 128 and a further 5 % to 64 at 8192^3. */
  SGEMM_CUBE_OPT_TERMWISE_K_BLOCK = 0,
  /* Same for the elementwise order: the k-block of Eq. elementwise.  Multiple of 64, default 64. */
  SGEMM_CUBE_OPT_ELEMENTWISE_K_BLOCK = 1,
  /* 1: run the tensor-core kernels as clusters of two CTAs that share one
   * tcgen05.mma.cta_group::2 (256 x 256 tile per pair, each CTA loading half of the B tile);
   * 0: one CTA per 128 x 256 tile; 2 (default): the library chooses: pairs for the kernels that
   * read FP16 words (two-phase sgemm_cube, sgemm_cube_presplit, sgemm_cube_hgemm, ...) whenever
   * M > 128 and split-K (below, single CTAs only) does not apply, and for the fused converter
   * kernel whenever M > 128.  Same arithmetic, bit-identical results either way as long as
   * split-K does not apply.  (Pairs pull two thirds of the bytes of single CTAs from L2 into the SMs, which is
   * what bounds this kernel: 458 against 439 TFLOP/s at 8192^3, 407 against 378 at 4096^3.) */
  SGEMM_CUBE_OPT_CTA_PAIR = 2,
  /* How sgemm_cube computes (same arithmetic; same bracketing and bit-identical results except
   * where split-K, which only the two-phase strategy uses, re-brackets the k-block sums):
   * SGEMM_CUBE_STRATEGY_FUSED     one kernel; TMA stages FP32 tiles in shared memory, converter
   *                               warps split them there in place, no FP16 copy of A or B exists
   *                               in device memory, no workspace;
   * SGEMM_CUBE_STRATEGY_TWO_PHASE the split kernel writes the FP16 words of A and B once into the
   *                               handle's workspace (4 bytes per element of A and B, grown with
   *                               cudaMalloc on first use), then one kernel forms all three
   *                               products and the reconstruction;
   * SGEMM_CUBE_STRATEGY_AUTO      (default) TWO_PHASE when M*N*K >= 2^27 and the workspace can be
   *                               had, FUSED otherwise (measured crossover: 512^3). */
  SGEMM_CUBE_OPT_STRATEGY = 3,
  /* 1: sgemm_cube records CUDA events around its tensor-core kernel, for
   * sgemm_cube_last_kernel_ms and sgemm_cube_mean_kernel_ms.  Default 0. */
  SGEMM_CUBE_OPT_TIME_KERNEL = 4,
  /* 1 (default): when a problem has so few 128 x 256 tiles that more than half of the SMs would
   * idle and k is long enough, the three-product kernel (two-phase sgemm_cube,
   * sgemm_cube_presplit) cuts the k range into up to 16 slices of whole k-blocks, one work unit per
   * (tile, slice); the slices' sums go to a workspace (grown with cudaMalloc on first use) and a
   * reduction kernel adds them in slice order (termwise: hi*hi sums and correction sums
   * separately, combined once).  This is one more level of the blocked summation of Sec. 4.5 and
   * is deterministic.  0: never split. */
  SGEMM_CUBE_OPT_SPLIT_K = 5
};

enum {
  SGEMM_CUBE_STRATEGY_AUTO = 0,
  SGEMM_CUBE_STRATEGY_FUSED = 1,
  SGEMM_CUBE_STRATEGY_TWO_PHASE = 2
};

/* Create a handle bound to CUDA device `device`.  Allocates a small device error word; the
 * workspace of the unfused path and of the host-buffer path grows on demand.
 * Errors: INVALID_ARG (out == NULL), CUDA_ERROR, UNSUPPORTED_ARCH, ALLOC_FAILED. */
int sgemm_cube_create(sgemm_cube_handle* out, int device);

/* Synchronise the device, free the handle's workspace and the handle.  Returns DEVICE_TIMEOUT
 * if a kernel recorded a failure that was never collected by sgemm_cube_check. */
int sgemm_cube_destroy(sgemm_cube_handle h);

/* Set an option (see SGEMM_CUBE_OPT_*).  Errors: INVALID_ARG. */
int sgemm_cube_set_option(sgemm_cube_handle h, int option, int64_t value);

/* Operand split (paper Eq. recover_eqn, first two lines; Sec. 3.3; Sec. 4.2).
 *   hi[i,j] = fl16(X[i,j]);  lo[i,j] = fl16((X[i,j] - hi[i,j]) * 2^scale_exp)
 * RN-even conversions; the subtraction and the scaling are exact FP32 operations; FP16
 * subnormals are produced (gradual underflow is kept, nothing is flushed or clamped);
 * out-of-range inputs follow IEEE (|x| >= 65520 -> hi = inf, lo = NaN or inf).
 *   X_dev      rows x cols FP32, row-major, leading dimension ldx >= cols          (device, read)
 *   hi_dev/lo_dev  rows x cols FP16 bit patterns, leading dimension ldh >= cols    (device, written)
 *   scale_exp  s in [0, 24];  rows, cols >= 0 (nothing is done, and the pointers are not looked
 *   at, when either is 0)
 * Any alignment is accepted; 16-byte aligned pointers with ldx % 4 == 0 and ldh % 8 == 0 take
 * the vectorised path.  Errors: INVALID_ARG, CUDA_ERROR. */
int sgemm_cube_split(sgemm_cube_handle h, int rows, int cols,
                     const float* X_dev, int64_t ldx,
                     uint16_t* hi_dev, uint16_t* lo_dev, int64_t ldh,
                     int scale_exp, void* stream);

/* SGEMM-cube (paper Eq. recover_eqn with Eq. termwise or Eq. elementwise):
 *   C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B),
 * hi = fl16(x), lo = fl16((x - hi) 2^s) as in sgemm_cube_split, FP16 x FP16 products on the tensor
 * cores with FP32 accumulation, the reconstruction in FP32; C overwritten (no alpha/beta).
 * The operand split runs either inside the product kernel (converter warps, no FP16 copy of A or
 * B in device memory) or once up front into the handle's workspace: see SGEMM_CUBE_OPT_STRATEGY.
 * Both give bit-identical C unless split-K applies (SGEMM_CUBE_OPT_SPLIT_K).
 *   A_dev  M x K FP32, lda >= K     (device, read)
 *   B_dev  K x N FP32, ldb >= N     (device, read)
 *   C_dev  M x N FP32, ldc >= N     (device, written)
 *   scale_exp s in [0, 24]; accumulation_order SGEMM_CUBE_TERMWISE, SGEMM_CUBE_ELEMENTWISE or
 *   SGEMM_CUBE_ELEMENTWISE_REORDERED
 * Alignment: A_dev, B_dev 16-byte aligned and lda % 4 == 0, ldb % 4 == 0 (else MISALIGNED).
 * C_dev may have any alignment.  M, N, K >= 0, any values (ragged edges are handled).  Empty
 * problems are valid in every GEMM entry point of this header: M == 0 or N == 0 does nothing,
 * K == 0 stores C = 0 (the empty sum; left alone by sgemm_cube_hgemm with accumulate != 0); an
 * operand without elements may be a null pointer.
 * Once the workspace for a problem size exists (after the first call at that size or a larger
 * one) the call only enqueues work on `stream`: it can be captured into a CUDA graph and replayed.
 * A handle's workspace is shared by its calls, so calls that may overlap on the GPU need one
 * handle per stream.
 * Errors: INVALID_ARG, MISALIGNED, CUDA_ERROR (ALLOC_FAILED only with the TWO_PHASE strategy
 * forced; AUTO falls back to the fused kernel when the workspace cannot be had). */
int sgemm_cube(sgemm_cube_handle h, int M, int N, int K,
               const float* A_dev, int64_t lda,
               const float* B_dev, int64_t ldb,
               float* C_dev, int64_t ldc,
               int scale_exp, int accumulation_order, void* stream);

/* Unfused ablation of the same computation (paper Sec. 5.4: one GEMM pipeline per term):
 * split A and B into FP16 words in the handle's workspace, run three FP16 GEMM passes
 * (hi_A hi_B -> D_hh; lo_A hi_B -> D_x; hi_A lo_B added to D_x), then C = D_hh + 2^-s D_x.
 * Termwise only (accumulation_order must be SGEMM_CUBE_TERMWISE).  Same arguments and
 * alignment-free inputs (the workspace copies are padded).  The workspace
 * (4 bytes x (M K + K N) + 8 bytes x M N, rounded up) is grown with cudaMalloc on first use;
 * Errors: INVALID_ARG, ALLOC_FAILED, CUDA_ERROR. */
int sgemm_cube_unfused(sgemm_cube_handle h, int M, int N, int K,
                       const float* A_dev, int64_t lda,
                       const float* B_dev, int64_t ldb,
                       float* C_dev, int64_t ldc,
                       int scale_exp, int accumulation_order, void* stream);

/* SGEMM-cube on operands that were split beforehand with sgemm_cube_split (all three products
 * and the reconstruction in one kernel; useful when an operand is reused across calls).
 *   Ahi_dev/Alo_dev  M x K FP16 bit patterns, leading dimension lda16 >= K   (device, read)
 *   Bhi_dev/Blo_dev  K x N FP16 bit patterns, leading dimension ldb16 >= N   (device, read)
 * Alignment: the four FP16 pointers 16-byte aligned, lda16 % 8 == 0, ldb16 % 8 == 0.
 * scale_exp must be the value used for the split.  Errors as sgemm_cube. */
int sgemm_cube_presplit(sgemm_cube_handle h, int M, int N, int K,
                        const uint16_t* Ahi_dev, const uint16_t* Alo_dev, int64_t lda16,
                        const uint16_t* Bhi_dev, const uint16_t* Blo_dev, int64_t ldb16,
                        float* C_dev, int64_t ldc,
                        int scale_exp, int accumulation_order, void* stream);

/* Plain FP16 x FP16 -> FP32 GEMM on the tensor cores, D = A16 B16 (or D += A16 B16 when
 * accumulate != 0): one pass of the unfused path, and the plain FP16 GEMM the paper
 * contrasts with (Sec. 6.2).
 *   A16_dev M x K FP16 (lda16 >= K), B16_dev K x N FP16 (ldb16 >= N), D_dev M x N FP32 (ldd >= N).
 * Alignment as sgemm_cube_presplit.  Errors as sgemm_cube. */
int sgemm_cube_hgemm(sgemm_cube_handle h, int M, int N, int K,
                     const uint16_t* A16_dev, int64_t lda16,
                     const uint16_t* B16_dev, int64_t ldb16,
                     float* D_dev, int64_t ldd, int accumulate, void* stream);

/* Host-buffer convenience around sgemm_cube: copies A and B from HOST memory to the handle's
 * device workspace, runs the computation of sgemm_cube there (same strategy choice, see
 * SGEMM_CUBE_OPT_STRATEGY), copies C back to HOST memory and synchronises the stream before
 * returning.  Pinned host memory makes the copies asynchronous to the host but the
 * call still returns only when C_host is complete.  For M >= 1024 and M*N*K >= 2^30 (and a
 * strategy other than FUSED) the call is pipelined: B is copied and split once, A and C move in
 * about eight row panels on two internal copy streams so that the upload of one panel, the
 * products of the previous one and the download of the one before overlap.  The result is
 * bit-identical to sgemm_cube on device copies of the same operands when split-K applies to
 * neither (a panel of a tall problem may have few enough tiles to be split where the whole problem
 * is not; both results pass the same error gates).
 *   A_host M x K (lda >= K), B_host K x N (ldb >= N), C_host M x N (ldc >= N), all FP32 HOST.
 * Errors: INVALID_ARG, ALLOC_FAILED, CUDA_ERROR, DEVICE_TIMEOUT. */
int sgemm_cube_host(sgemm_cube_handle h, int M, int N, int K,
                    const float* A_host, int64_t lda,
                    const float* B_host, int64_t ldb,
                    float* C_host, int64_t ldc,
                    int scale_exp, int accumulation_order, void* stream);

/* Four-term variant: the low-low product that SGEMM-cube drops (paper Sec. 4.3, bounded by
 * Eq. ll_bound) is kept, i.e. the full expansion of (hi_A + lo_A 2^-s)(hi_B + lo_B 2^-s):
 *   C = hi_A hi_B + 2^-s (lo_A hi_B + hi_A lo_B) + 2^-2s lo_A lo_B.
 * It exists to measure what dropping that term costs; it is not part of the paper's method.
 * Termwise only: each stream is summed in k-blocks (SGEMM_CUBE_OPT_TERMWISE_K_BLOCK) and
 *   C = S_hh + (2^-s S_x + 2^-2s S_ll),
 * the small terms combined first.  Runs as: the split of both operands, one FP16 GEMM pass lo_A lo_B into
 * the handle's workspace, the three-product kernel writing its raw sums, one reduction kernel.
 * Arguments, layouts and alignment-free inputs as sgemm_cube_unfused.  Workspace:
 * 4 bytes x (M K + K N) + 12 bytes x M N, rounded up, grown with cudaMalloc on first use.
 * Errors: INVALID_ARG, ALLOC_FAILED, CUDA_ERROR. */
int sgemm_cube_four_term(sgemm_cube_handle h, int M, int N, int K,
                         const float* A_dev, int64_t lda,
                         const float* B_dev, int64_t ldb,
                         float* C_dev, int64_t ldc,
                         int scale_exp, void* stream);

/* Exponent window of a matrix's FP16 high words (paper Sec. 4.2: e_min and e_max of
 * Eq. sf_bounds are the smallest and largest unbiased exponents E' - 15 of the finite high
 * components).  One pass over X on the device; the call synchronises `stream` and writes to HOST
 * memory:
 *   window_out[0] = e_min, window_out[1] = e_max over the NORMAL high words (127 / -127 if none),
 *   window_out[2] = number of entries whose high word is subnormal (|x| < 2^-14: the 22-bit
 *                   guarantee cannot be kept by scaling the residual alone, Sec. 4.2),
 *   window_out[3] = number of entries whose high word is inf or NaN (|x| >= 65520),
 *   window_out[4] = number of entries whose high word is zero.
 *   X_dev rows x cols FP32, ldx >= cols (device, read); window_out 5 x int64 (host, written).
 * Errors: INVALID_ARG, CUDA_ERROR. */
int sgemm_cube_exponent_window(sgemm_cube_handle h, int rows, int cols,
                               const float* X_dev, int64_t ldx,
                               int64_t* window_out, void* stream);

/* Residual-overflow detection (paper Sec. 4.2, Rule 2, which allows a larger scale only if
 * overflowing residuals are caught): the number of entries of a split operand whose high word is finite
 * while its scaled residual word is inf or NaN, i.e. for which (x - hi) 2^s left the FP16 range
 * (the paper's example: x = 32784 at s_b = 12).  A non-zero count means the chosen scale exponent
 * is too large for this operand; sgemm_cube_choose_scale_exp gives one that cannot overflow.
 * One pass over the two word matrices; the call synchronises `stream`.
 *   hi_dev, lo_dev  rows x cols FP16 bit patterns as written by sgemm_cube_split, ldh >= cols
 *   count_out       1 x int64 (host, written)
 * Errors: INVALID_ARG, CUDA_ERROR. */
int sgemm_cube_residual_overflow_count(sgemm_cube_handle h, int rows, int cols,
                                       const uint16_t* hi_dev, const uint16_t* lo_dev, int64_t ldh,
                                       int64_t* count_out, void* stream);

/* Scale exponent for a pair of operands from their exponent windows (host arithmetic only).
 * Eq. sf_bounds:  -3 - e_min <= s_b <= 26 - e_max  over both operands; Sec. 4.2 advises moving
 * the residuals as far above the underflow threshold as the largest entry allows, so the upper end
 * is taken, capped at 15:  *scale_exp_out = min(26 - e_max, 15).  Full normal FP16 range
 * (e_max = 15) gives 11, e_max <= 14 gives at least 12.
 * *protected_out (optional) = 1 if that value also satisfies the lower end and no high word is
 * subnormal, inf or NaN, i.e. if Eq. split_error holds for every entry; else 0.
 * Errors: INVALID_ARG. */
int sgemm_cube_choose_scale_exp(const int64_t* window_a, const int64_t* window_b,
                                int* scale_exp_out, int* protected_out);

/* ---- Whole-input scaling (explicit exponent management).
 * The paper notes (Sec. 4.2, after Rule 1) that once a high word is subnormal, |x| < 2^-14,
 * scaling the residual alone cannot keep 22 bits and that the whole input must be scaled, and
 * leaves that outside its scope (Sec. 7 lists it as future work).  These entry points are that
 * extension: operands are multiplied by powers of two before the split (exact) and the product
 * is multiplied by the inverse power afterwards (exact unless the FP32 result leaves the normal
 * range, then rounded once). */

/* Range of the exponents the FP16 high words of X would have if FP16 had unbounded exponent
 * range: the unbiased exponent of |x| rounded (RN-even) to an 11-bit significand, over the
 * non-zero finite entries.  One pass over X; the call synchronises `stream` and writes HOST memory:
 *   range_out[0] = e_min, range_out[1] = e_max (127 / -127 if no entry qualifies),
 *   range_out[2] = number of inf / NaN entries.
 *   X_dev rows x cols FP32, ldx >= cols (device, read); range_out 3 x int64 (host, written).
 * Errors: INVALID_ARG, CUDA_ERROR. */
int sgemm_cube_hi_exponent_range(sgemm_cube_handle h, int rows, int cols,
                                 const float* X_dev, int64_t ldx,
                                 int64_t* range_out, void* stream);

/* Scaling exponents for a pair of operands from their ranges (host arithmetic only):
 * p = 15 - e_max per operand (its largest high word lands in the top normal FP16 binade, nothing
 * overflows), clamped to [-126, 126]; an operand without non-zero finite entries gets p = 0.  The
 * scaled windows may then span the whole normal range, for which Eq. sf_bounds leaves
 * *scale_exp_out = 11.  *protected_out (optional) = 1 if every non-zero entry of both scaled
 * operands has a normal high word (e_min + p >= -14), i.e. each operand spans at most 30 binades,
 * and there is no inf / NaN; else 0 (the smallest entries then keep fewer than 22 bits).
 * Errors: INVALID_ARG. */
int sgemm_cube_choose_input_scaling(const int64_t* range_a, const int64_t* range_b,
                                    int* p_a_out, int* p_b_out, int* scale_exp_out,
                                    int* protected_out);

/* C = 2^-(p_a + p_b) * sgemm_cube(2^p_a A, 2^p_b B): the split kernels scale while they read, one
 * three-product kernel, one pass over C for the way back (skipped when p_a + p_b == 0).  Always
 * the two-phase route (FP16 words in the handle's workspace), so inputs need no alignment.
 * p_a, p_b in [-126, 126]; the other arguments and layouts as sgemm_cube.
 * Errors: INVALID_ARG, ALLOC_FAILED, CUDA_ERROR. */
int sgemm_cube_scaled(sgemm_cube_handle h, int M, int N, int K,
                      const float* A_dev, int64_t lda,
                      const float* B_dev, int64_t ldb,
                      float* C_dev, int64_t ldc,
                      int p_a, int p_b, int scale_exp, int accumulation_order, void* stream);

/* sgemm_cube_hi_exponent_range on A and B, sgemm_cube_choose_input_scaling, sgemm_cube_scaled in
 * one call.  Synchronises `stream` twice (the ranges are read on the host) before it enqueues the
 * product.  chosen_out (optional, host, 4 x int): p_a, p_b, scale exponent, protected flag.
 * Errors: as the three calls. */
int sgemm_cube_auto_scaled(sgemm_cube_handle h, int M, int N, int K,
                           const float* A_dev, int64_t lda,
                           const float* B_dev, int64_t ldb,
                           float* C_dev, int64_t ldc,
                           int accumulation_order, void* stream, int* chosen_out);

/* Size in bytes of the fixed device scratch area used by sgemm_cube_unfused_static. */
#define SGEMM_CUBE_STATIC_SCRATCH_BYTES (32u << 20)

/* The unfused computation (same arithmetic, same kernels and same result as sgemm_cube_unfused,
 * termwise order) for callers that are not allowed to allocate device memory: code running inside
 * another framework's memory pool with a hard cap, real-time or safety-certified loops where
 * cudaMalloc/cudaFree (which may synchronise the whole device or fail late) are forbidden after
 * start-up, or a process whose remaining device memory is already committed.  The paper has no
 * counterpart of this entry point; it exists for such integrations only.
 *
 * It needs no handle and calls no cudaMalloc, cudaFree or other allocating routine.  Its scratch
 * (the FP16 words of A and B and two FP32 M x N partial results) lives in a fixed array of
 * SGEMM_CUBE_STATIC_SCRATCH_BYTES (32 MiB) that is part of the library's device image: every GPU
 * on which the library is loaded holds those 32 MiB until the process exits.
 *   Limit: 4*(M*K8 + K*N8) + 8*M*N4 bytes (K8, N8 = K, N rounded up to 8; N4 = N rounded up to 4;
 *   each of the six pieces rounded up to 256 bytes) must not exceed the array, e.g. up to
 *   1024 x 1024 x 1024 or 2048 x 512 x 1024.  Larger problems return SGEMM_CUBE_TOO_LARGE and
 *   enqueue nothing.
 *   Arguments, layouts and alignment as sgemm_cube_unfused, on the CURRENT device
 *   (A_dev, B_dev, C_dev must be on it).
 *   The first call on a device looks up the array's device address and configures the kernels;
 *   make that first call outside any stream capture, and at start-up: the 32 MiB are committed
 *   when the CUDA runtime loads the library's device code on that GPU, which with lazy module
 *   loading can be as late as this first call, so a process whose device memory is already
 *   exhausted gets CUDA_ERROR from it.  Later calls only launch and leave the amount of free
 *   device memory unchanged.
 *   All calls share the one array, which keeps whatever the last call left in it.  Every region a
 *   call reads is first overwritten by that call, so results never depend on earlier calls; but
 *   two calls that may overlap on the GPU (different streams without an ordering between them,
 *   whether from one host thread or several) race on the scratch and give undefined results.
 *   Host threads may call concurrently as far as the host side goes (enqueueing is serialised
 *   internally).
 *   A kernel-side bounded-wait failure (never expected) cannot be reported by this entry point;
 *   C is then unspecified.
 * Errors: INVALID_ARG, TOO_LARGE, UNSUPPORTED_ARCH, CUDA_ERROR. */
int sgemm_cube_unfused_static(int M, int N, int K,
                              const float* A_dev, int64_t lda,
                              const float* B_dev, int64_t ldb,
                              float* C_dev, int64_t ldc,
                              int scale_exp, void* stream);

/* Synchronise `stream` and report (then clear) the device error word.
 * Returns OK, DEVICE_TIMEOUT (detail in *detail_out if non-NULL: a code naming the wait that
 * gave up) or CUDA_ERROR. */
int sgemm_cube_check(sgemm_cube_handle h, void* stream, uint32_t* detail_out);

/* Number of kernels this handle has launched since creation (for launch accounting). */
int64_t sgemm_cube_launch_count(sgemm_cube_handle h);

/* Device time, in milliseconds, of the tensor-core kernel of the most recent sgemm_cube call
 * (requires SGEMM_CUBE_OPT_TIME_KERNEL = 1 before that call; waits for the kernel to finish).
 * Errors: INVALID_ARG (timing off, or no call yet), CUDA_ERROR. */
int sgemm_cube_last_kernel_ms(sgemm_cube_handle h, float* ms_out);

/* Mean device time, in milliseconds, of the tensor-core kernel over the sgemm_cube calls made
 * since SGEMM_CUBE_OPT_TIME_KERNEL was set to 1 or since the previous call of this function (at
 * most the 128 most recent ones: one CUDA event pair is kept per call); *calls_out (optional) =
 * how many calls were averaged.  Waits for those kernels to finish, then starts a new average.
 * Errors: INVALID_ARG (timing off, or no call since), CUDA_ERROR. */
int sgemm_cube_mean_kernel_ms(sgemm_cube_handle h, float* mean_ms_out, int* calls_out);

/* SM clock cycles and nanoseconds (device global timer) that the tensor-core kernel of the most
 * recent sgemm_cube call ran for, taken inside the kernel by its first CTA (requires
 * SGEMM_CUBE_OPT_TIME_KERNEL = 1 before that call; waits for the device to finish).  Their
 * quotient is the SM clock the kernel actually ran at, which under a power cap is well below the
 * clock that nvidia-smi shows between kernels; the three-GEMM roofline at that clock is
 * SMs x 8192 FP16 flop/clk x (cycles / ns) / 3.
 * Errors: INVALID_ARG (timing off), CUDA_ERROR. */
int sgemm_cube_last_kernel_clock(sgemm_cube_handle h, uint64_t* sm_cycles_out, uint64_t* ns_out);

/* ---- Diagnostics for the failure-reporting path (tests; nothing on the GEMM path calls them).
 * Every wait inside the kernels is bounded; a wait that runs out writes a code into the handle's
 * device error word, the CTA drains and exits, and sgemm_cube_check / sgemm_cube_destroy report
 * SGEMM_CUBE_DEVICE_TIMEOUT.  Neither function below makes a GEMM kernel fail.
 *
 * sgemm_cube_debug_inject_error: host-made failure.  Waits for the device, then copies `code`
 * into the error word, as if a kernel had recorded it.
 * sgemm_cube_debug_wait_timeout: enqueues a one-CTA kernel in which one thread runs the kernels'
 * bounded wait, with a limit of `limit_clocks` SM clocks (1 .. 10^8), on a barrier that nothing
 * signals; the wait gives up after the limit and records code 0x1F0.  The kernel then ends
 * normally and the context stays usable.
 * Errors: INVALID_ARG, CUDA_ERROR. */
int sgemm_cube_debug_inject_error(sgemm_cube_handle h, uint32_t code);
int sgemm_cube_debug_wait_timeout(sgemm_cube_handle h, int64_t limit_clocks, void* stream);

/* Text for a status code (static storage; never NULL). */
const char* sgemm_cube_status_string(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int sgemm_cube_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SGEMM_CUBE_H_ */
