/*
 * libsquat -- the KV-cache write path of SQuat (arXiv 2503.24358) on one NVIDIA B200 (sm_100a).
 *
 * Plain C ABI.  No exceptions, no C++ or framework types cross it.  Unless a parameter says
 * "host", every tensor pointer is a DEVICE pointer owned by the caller, 16-byte aligned, valid
 * until the stream work enqueued by the call has finished.  Calls enqueue kernels on the given
 * CUDA stream (a cudaStream_t passed as void*, NULL = default stream) and return without
 * synchronising, except where stated.  Arguments are validated on the host before anything
 * is launched; a rejected call launches nothing.  Kernels never trap or assert: numerical
 * trouble (non-finite input, a group whose values are all equal) sets bits in a device status
 * word, see squat_get_device_status.  There is no CPU fallback.
 *
 * Notation (the paper's): d = head dimension, r = subspace rank, lambda = regulariser of
 * Eq. (2), g = elements quantized per iteration (Appendix A "Block-Wise Quantization"),
 * G = quantization group size, b = bits, L = 2^b - 1.
 *
 * Cache layout written by the quantizers (the paper prescribes none):
 *   codes  token-major; token i of (batch, head) owns d*b/8 consecutive bytes; channel j's code
 *          sits at bit (j*b) mod 8 of byte floor(j*b/8), low bits first.
 *   keys   scale, zero: float32 [batch, head, token/G, d]   (one grid per channel per G tokens)
 *   values scale, zero: float32 [batch, head, token, d/G]   (one grid per G channels per token)
 *   deq(c) = zero + scale * c      (Section 2, "Quantization").
 */
#ifndef SQUAT_H
#define SQUAT_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SQUAT_OK = 0,
    SQUAT_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, negative size, bad enum            */
    SQUAT_ERR_SHAPE = 2,         /* sizes that do not divide as the method requires               */
    SQUAT_ERR_UNSUPPORTED = 3,   /* valid in the paper, not built here (e.g. head_dim != 128)     */
    SQUAT_ERR_ALLOC = 4,         /* device allocation failed                                      */
    SQUAT_ERR_CUDA = 5,          /* a CUDA runtime call failed; see squat_last_cuda_error         */
    SQUAT_ERR_NUMERIC = 6        /* the eigensolver did not converge                              */
} squat_status;

typedef enum { SQUAT_F32 = 0, SQUAT_BF16 = 1 } squat_dtype;
typedef enum { SQUAT_KEYS = 0, SQUAT_VALUES = 1 } squat_kind;

/* bits of the device status word */
#define SQUAT_FLAG_NONFINITE   1u   /* a NaN or infinity among the keys / values (its group's scale came out NaN/Inf) */
#define SQUAT_FLAG_ZERO_RANGE  2u   /* some group had max == min (scale 0, all codes 0)            */
#define SQUAT_FLAG_NO_CONVERGE 4u   /* eigensolver hit its sweep limit for some head               */
#define SQUAT_FLAG_BOUNDS 16u        /* only in the bounds-checked build of the library (-DSQUAT_CHECKED): a kernel computed an
                                       * address outside the buffer or on-chip region it belongs to; the access was skipped      */
#define SQUAT_FLAG_DEVICE_TIMEOUT 8u /* a bounded wait on the tensor core inside squat_quantize_keys ran
                                       * out: that call's outputs are invalid (the kernel still ends)  */

/* Opaque per-layer state: the update matrices of every KV head (shared by all samples of a
 * batch, Appendix C) plus the scratch the subspace build needs.  Owns device memory. */
typedef struct squat_subspace squat_subspace;

/* Allocates the state for n_kv_heads heads of dimension head_dim (only 128 is built) on the
 * current device.  Synchronous (cudaMalloc).  *out receives the handle; free it with
 * squat_subspace_destroy.  The update matrices start as zero (= plain round-to-nearest). */
int squat_subspace_create(int n_kv_heads, int head_dim, squat_subspace **out);
int squat_subspace_destroy(squat_subspace *s);

/*
 * Step 1 -- query subspace and update matrices  (Section 3.2; Algorithm 1 lines 5-9;
 * Prop. 1, Prop. 2, Lemma 3, Lemma 4; GQA and batch rules of Appendix C).
 *
 * q         prompt queries of ONE sample (the first of the batch), [n_q_heads, n_tokens, d],
 *           d contiguous, element strides stride_h (between query heads) and stride_t (between
 *           tokens).  Query heads h*(n_q/n_kv) .. (h+1)*(n_q/n_kv)-1 feed KV head h.
 * rank_r    top singular directions kept, 0 <= r <= d (r = 0 gives plain round-to-nearest).
 * lambda    >= 0, finite.          block_g   g, divides d; 1 = element by element (Prop. 1).
 *
 * Per KV head: Gram matrix of the stacked queries in fp64, its eigen-decomposition in fp64
 * (sigma_i^2 and v_i of the SVD of Alg. 1 line 5), P = I + lambda Qhat^T Qhat with
 * Qhat = diag(sigma[:r]) V[:r], and the update matrices B_t H_t of Lemma 3 for t = 1..d/g-1,
 * assembled as one block-strictly-lower-triangular W (float32):  quantizing channel j with
 * error e moves every later channel j' by e * W[j'][j].
 * Enqueues on `stream`; the handle may be used by later calls on the same stream at once.
 */
int squat_build_subspace(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                         long long stride_h, long long stride_t, int rank_r, double lambda,
                         int block_g, void *stream);

/*
 * The same build from Gram matrices the caller already has (Section 3.2: the subspace depends on the prompt's
 * queries only through M_h = Qc^T Qc, a sum over tokens).  This is the entry for a prompt whose tokens are spread
 * over several GPUs: every rank forms the Gram matrices of its own tokens (squat_gram_static), the ranks add them
 * up (one all-reduce of n_kv_heads * d * d float64), and every rank calls this with the sum.
 *   gram   [n_kv_heads, d, d] float64, device, 16-byte aligned, symmetric; copied into the handle.
 * rank_r, lambda, block_g and the result as for squat_build_subspace (rank_r is not checked against a token
 * count here: the caller knows how many rows went into the sum).
 */
int squat_build_subspace_from_gram(squat_subspace *s, const double *gram, int rank_r, double lambda, int block_g,
                                   void *stream);

/*
 * Step 1 with the block power method in place of the SVD (the accelerator the paper's comment on Algorithm 1 line 5
 * names; it gives no steps, these are the textbook ones).  Per KV head, with M the Gram matrix of the stacked queries:
 *     X <- orth(M X), `iters` times, from the start block X0;  B = X^T M X;  P = I + lambda X B X^T,
 * i.e. the compression of M to the iterated r-dimensional subspace stands where squat_build_subspace has the rank-r
 * truncation of M (the two agree once span(X) is the dominant eigenspace; P depends on span(X) only, so the Ritz
 * pairs of B are never formed).  W follows from P exactly as in squat_build_subspace; all of it in fp64.
 *   q .. block_g       as for squat_build_subspace, except rank_r <= 64 (SQUAT_ERR_UNSUPPORTED above).
 *   start_block        device, float64, 8-byte aligned: X0 as [d, rank_r] row-major (the random numbers the method
 *                      draws are the caller's); head h reads start_block + h * start_stride_h (elements; 0 = the
 *                      same block for every head, else >= d * rank_r).  Read only; may be NULL when rank_r = 0.
 *   iters              0 <= iters <= 64 multiplications by M (0: X = orth(X0)).
 * Orthonormalisation is Cholesky QR (twice for the last basis).  A direction whose pivot falls below 1e-13 of its
 * diagonal entry (start block or Gram matrix of rank < rank_r within the block, or cond(M) on the block beyond
 * ~1e6) is dropped and contributes nothing; squat_subspace_eig_sweeps then reports, per head, the number of basis
 * columns kept (= rank_r when nothing was dropped) instead of a sweep count.  The eigenvalue / eigenvector arrays
 * of squat_subspace_export are scratch after this call.  Enqueues on `stream`.
 */
int squat_build_subspace_power(squat_subspace *s, const void *q, int dtype, int n_q_heads, int n_tokens,
                               long long stride_h, long long stride_t, int rank_r, double lambda, int block_g,
                               const double *start_block, long long start_stride_h, int iters, void *stream);

/*
 * squat_build_subspace_power from Gram matrices the caller already has -- the block power method for a prompt whose
 * tokens are spread over several GPUs: Gram matrices of the local tokens (squat_gram_static), one all-reduce, then
 * this call on every rank with the same start block.  gram as for squat_build_subspace_from_gram, the other
 * arguments as for squat_build_subspace_power.
 */
int squat_build_subspace_power_from_gram(squat_subspace *s, const double *gram, int rank_r, double lambda, int block_g,
                                         const double *start_block, long long start_stride_h, int iters, void *stream);

/* Test / checkpoint hooks.  Both synchronise `stream`.  Host pointers; any may be NULL.
 *   W_host      [n_kv_heads, d, d] float32, row j' column j, block strictly lower triangular.
 *   gram_host   [n_kv_heads, d, d] float64 Gram matrices of the last build.
 *   eigval_host [n_kv_heads, d]    float64 eigenvalues, descending (sigma_i^2).
 *   eigvec_host [n_kv_heads, d, d] float64, row i = unit eigenvector of eigval i. */
int squat_subspace_export(const squat_subspace *s, void *stream, float *W_host, double *gram_host,
                          double *eigval_host, double *eigvec_host);
int squat_subspace_import(squat_subspace *s, const float *W_host, void *stream);
/* Diagnostics of the last build: Jacobi sweeps the eigensolver ran for each head.  Synchronises
 * `stream`.  sweeps_host is a host array of n_kv_heads ints. */
int squat_subspace_eig_sweeps(const squat_subspace *s, void *stream, int *sweeps_host);

/*
 * Step 2 -- key quantization with error feedback  (Algorithm 1, function Quant; Eq. (3) and
 * Eq. (update_block); quantizer of Section 2).
 *
 * k         [batch, n_kv_heads, n_tokens, d], d contiguous, element strides given.
 * n_tokens  multiple of group_size (the tail stays in the caller's residual buffer,
 *           Alg. 1 lines 10-11); groups are G consecutive tokens from the first one passed.
 * codes     [batch, n_kv_heads, *, d*bits/8] bytes; scales, zeros [batch, n_kv_heads, *, d].
 *           out_stride_b / out_stride_h are in TOKENS (a batch/head step moves the code pointer
 *           by stride*d*bits/8 bytes and the scale/zero pointers by (stride/G)*d floats), so a
 *           decode window can be written into a larger cache.  Must be multiples of G.
 * For every group and channel j in order: grid from min/max over the G tokens of the current
 * (corrected) values, round half to even, push each token's error on its later channels
 * through W.  Splitting n_tokens at multiples of G over several calls gives identical bytes.
 * bits in {2, 4}; group_size in {32, 64, 128}; d = 128; n_kv_heads must match the handle.
 * The updates that cross 32-channel blocks are computed on the tensor cores as three tf32
 * products per multiply-add (operands split hi + lo), accumulated in fp32; the result agrees
 * with fp32 arithmetic to a few 1e-7 of sum |e W|.  Every wait on the tensor core is bounded; if
 * one runs out the kernel still ends, SQUAT_FLAG_DEVICE_TIMEOUT is set in the device status word
 * and the outputs of that call are invalid.
 */
int squat_quantize_keys(const squat_subspace *s, const void *k, int dtype, int batch, int n_kv_heads,
                        int n_tokens, int head_dim, long long stride_b, long long stride_h,
                        long long stride_t, int bits, int group_size, unsigned char *codes,
                        float *scales, float *zeros, long long out_stride_b, long long out_stride_h,
                        void *stream);

/*
 * Which kernel squat_quantize_keys runs.  For element-wise updates (block_g = 1) the update matrix of Prop. 1 is
 * semiseparable, W[j'][j] = v_j' . c_j (the Woodbury identity the footnote to Prop. 4 points to, applied to the
 * trailing blocks of P): a token then carries a state of r numbers and the update costs 2 r d multiply-adds per key
 * vector instead of d (d - 1) / 2.  squat_build_subspace and squat_build_subspace_from_gram prepare that form when
 * block_g = 1, lambda > 0 and 1 <= rank_r <= 8, and squat_quantize_keys / _m16 then use it (FP32 pipes only, no
 * tensor-core hand-over); every other build, and an imported W, runs the dense kernel.  Both compute the same
 * function Quant; results agree up to rounding ties.
 *   prefer_dense   1: always run the dense kernel;  0: the default choice above.
 *   lowrank_rank   host, may be NULL: receives the rank the rank-r form is prepared for (0: not prepared).
 * Host-side state of the handle: like every call that takes the handle, issue it from one thread at a time, in the
 * order the work is to execute.
 */
int squat_subspace_select_key_kernel(squat_subspace *s, int prefer_dense, int *lowrank_rank);

/*
 * Step 3 -- per-token value quantization  (Section 2 "Quantization"; Appendix C: each token's d
 * channels in d/G groups of G).  Every operation is IEEE binary32 in the order
 *   Delta = (M - m) / L;  t = (x - m) / Delta;  c = clamp(rint(t), 0, L).
 * v [batch, n_kv_heads, n_tokens, d]; codes as for keys; scales, zeros
 * [batch, n_kv_heads, *, d/G] with out strides in tokens.  d % G == 0, d*bits % 64 == 0.
 * batch and n_kv_heads are grid dimensions: more than 65535 of either returns SQUAT_ERR_UNSUPPORTED.
 */
int squat_quantize_values(const void *v, int dtype, int batch, int n_kv_heads, int n_tokens,
                          int head_dim, long long stride_b, long long stride_h, long long stride_t,
                          int bits, int group_size, unsigned char *codes, float *scales, float *zeros,
                          long long out_stride_b, long long out_stride_h, void *stream);

/*
 * Step 4 -- dequantize  (Section 2: deq(c) = c * Delta + m), for either layout kind.
 * in strides in tokens as above; out is contiguous [batch, n_kv_heads, n_tokens, d] of out_dtype
 * (float32: fma(c, scale, zero) rounded once; bf16: that value rounded to nearest even).
 * d / 8 and the group size are powers of two and batch, n_kv_heads <= 65535, else SQUAT_ERR_UNSUPPORTED.
 */
int squat_dequantize(int kind, const unsigned char *codes, const float *scales, const float *zeros,
                     int batch, int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                     long long in_stride_b, long long in_stride_h, void *out, int out_dtype,
                     void *stream);

/*
 * The same steps with scale and zero-point stored in 16 bits (IEEE binary16).  The "KV size" columns of Tables 1-2
 * (19.1-21.4 % of the FP16 cache, residual tokens included) imply this storage: 2-bit codes plus two 16-bit numbers
 * per 32 elements are 18.75 %; with float32 metadata the cache is 25 %.  The paper says nothing more, so, as a reading:
 * the stored values are the float32 scale and zero-point rounded once more to the nearest binary16 (ties to even),
 * and every decision is taken against the STORED values -- t = (x - z16) / Delta16, c = clamp(rint(t), 0, L), and (for
 * keys) the error fed back is c * Delta16 + z16 - x -- so that a reader of the cache sees exactly what the writer
 * corrected for.  Codes are clamped because a rounded zero-point can lie above the group's minimum.  A scale that
 * rounds to 0 (or a range of 0) gives codes 0; one beyond the binary16 range gives codes 0 and SQUAT_FLAG_NONFINITE.
 * scales / zeros: the same shapes and strides as the float32 variants, element type binary16 (2 bytes), 16-byte
 * aligned.  Everything else (arguments, errors) as for the functions without the suffix.
 */
int squat_quantize_keys_m16(const squat_subspace *s, const void *k, int dtype, int batch, int n_kv_heads,
                            int n_tokens, int head_dim, long long stride_b, long long stride_h,
                            long long stride_t, int bits, int group_size, unsigned char *codes,
                            void *scales, void *zeros, long long out_stride_b, long long out_stride_h,
                            void *stream);
int squat_quantize_values_m16(const void *v, int dtype, int batch, int n_kv_heads, int n_tokens,
                              int head_dim, long long stride_b, long long stride_h, long long stride_t,
                              int bits, int group_size, unsigned char *codes, void *scales, void *zeros,
                              long long out_stride_b, long long out_stride_h, void *stream);
int squat_dequantize_m16(int kind, const unsigned char *codes, const void *scales, const void *zeros,
                         int batch, int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                         long long in_stride_b, long long in_stride_h, void *out, int out_dtype, void *stream);

/*
 * The whole write path from HOST buffers (prefill of one layer): copies q (sample 0,
 * [n_q_heads, n_tokens, d]), k and v ([batch, n_kv_heads, n_tokens, d]), all contiguous, to the
 * device workspace, runs steps 1-3, copies codes / scales / zeros back and synchronises the
 * stream.  Host buffers should be pinned for full copy speed.  `workspace` is caller-owned device
 * memory of at least squat_write_path_workspace_bytes(...) bytes, 256-byte aligned.
 */
size_t squat_write_path_workspace_bytes(int dtype, int batch, int n_q_heads, int n_kv_heads,
                                        int n_tokens, int head_dim, int bits, int group_size);
int squat_write_path_host(squat_subspace *s, const void *q_host, const void *k_host, const void *v_host,
                          int dtype, int batch, int n_q_heads, int n_kv_heads, int n_tokens,
                          int head_dim, int rank_r, double lambda, int block_g, int bits, int group_size,
                          unsigned char *k_codes_host, float *k_scales_host, float *k_zeros_host,
                          unsigned char *v_codes_host, float *v_scales_host, float *v_zeros_host,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same with the two variants of the write path selectable:
 *   meta16             1: scales and zero-points are stored and copied back as IEEE binary16 (the host metadata
 *                      buffers then hold 2-byte elements; semantics of the _m16 quantizers), 0: float32.
 *   start_block_host   NULL: step 1 by the SVD (squat_build_subspace).  Otherwise host float64 [d, rank_r]
 *                      row-major, one block for all heads: step 1 by the block power method
 *                      (squat_build_subspace_power, rank_r <= 64) with power_iters multiplications.
 * Everything else as squat_write_path_host; the workspace size is the same function's.
 */
int squat_write_path_host_ex(squat_subspace *s, const void *q_host, const void *k_host, const void *v_host,
                             int dtype, int batch, int n_q_heads, int n_kv_heads, int n_tokens,
                             int head_dim, int rank_r, double lambda, int block_g, int bits, int group_size,
                             unsigned char *k_codes_host, void *k_scales_host, void *k_zeros_host,
                             unsigned char *v_codes_host, void *v_scales_host, void *v_zeros_host,
                             int meta16, const double *start_block_host, int power_iters,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * One decode window from HOST buffers (Algorithm 1, decode branch: when the residual buffer holds R keys, Quant runs
 * on its R/G groups with the per-head matrices that were computed at prefill; values likewise, Appendix C).  Copies
 * k and v ([batch, n_kv_heads, n_tokens, d], contiguous, n_tokens a multiple of group_size) to the device workspace,
 * quantizes them with the update matrices the handle holds (nothing is built), copies codes / scales / zeros back to
 * the host buffers (contiguous, the shapes squat_quantize_keys / _values write) and synchronises the stream.
 * meta16 = 1: scales and zero-points are binary16 (2-byte elements).  Workspace: at least
 * squat_write_path_workspace_bytes(dtype, batch, n_kv_heads, n_kv_heads, n_tokens, d, bits, group_size) bytes of
 * caller-owned device memory, 256-byte aligned.  The copies run on two side streams of the handle and overlap the
 * kernels; calls on one handle must not overlap each other.
 */
int squat_append_window_host(squat_subspace *s, const void *k_host, const void *v_host, int dtype, int batch,
                             int n_kv_heads, int n_tokens, int head_dim, int bits, int group_size,
                             unsigned char *k_codes_host, void *k_scales_host, void *k_zeros_host,
                             unsigned char *v_codes_host, void *v_scales_host, void *v_zeros_host, int meta16,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * Reader of the cache -- one decode step of attention over the packed cache (Section 2, "(Masked) Attention
 * mechanism": softmax(q K^T / sqrt(d)) V for the newest token; the score vector w^deq of the proof of
 * Theorem 1; the most recent tokens come from the full-precision residual buffer of Algorithm 1).  This is
 * the step that follows the write path; the cache is read in its packed form, never dequantized to memory.
 *
 *   out[b][hq] = sum_i p_i v_i,   p = softmax_i( softmax_scale * <q[b][hq], k_i> ),
 *   i over the n_tokens dequantized rows of KV head hq / (n_q_heads / n_kv_heads) (GQA rule of Appendix C),
 *   then the n_res rows of the residual buffer.
 *
 * q            [batch, n_q_heads, d] device, dense, dtype q_dtype.
 * k_codes .. v_zeros   the cache as squat_quantize_keys / squat_quantize_values wrote it (device); token 0
 *              of (b, h) sits at token index b * cache_stride_b + h * cache_stride_h, strides in tokens and
 *              multiples of group_size, so a cache longer than n_tokens can be read.  n_tokens is the number
 *              of quantized tokens per (b, h): a multiple of group_size, may be 0.
 * k_res, v_res [batch, n_kv_heads, n_res, d] device, dense, dtype res_dtype: the residual buffer;
 *              n_res <= SQUAT_ATTN_MAX_RESIDUAL, may be 0 (then both may be NULL).  n_tokens + n_res >= 1.
 * softmax_scale  multiplies the scores; 0 selects the paper's 1 / sqrt(d).
 * out          [batch, n_q_heads, d] float32 device.
 * workspace    device, caller-owned, 256-byte aligned, at least squat_decode_attention_workspace_bytes(...);
 *              holds the per-chunk partial results, no state is kept between calls.
 * All arithmetic is float32.  Returns a status code; nothing is launched on an argument error.
 */
#define SQUAT_ATTN_MAX_RESIDUAL 128
size_t squat_decode_attention_workspace_bytes(int batch, int n_q_heads, int n_tokens);
int squat_decode_attention(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                           const unsigned char *k_codes, const float *k_scales, const float *k_zeros,
                           const unsigned char *v_codes, const float *v_scales, const float *v_zeros,
                           int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                           int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                           float softmax_scale, float *out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same decode step over a cache whose keys were quantized BEFORE the rotary position embedding (Section 4:
 * the variant of the method that "quantizes and stores the KV cache before applying RoPE" and applies the
 * embedding on the fly after dequantization).  The write path is the one above, fed with un-rotated keys and a
 * subspace built from un-rotated queries; the cost of the embedding moves to this reader.
 *
 *   k_i  =  rope( deq(cached row i),  first_pos + i ),   then the residual rows at the positions that follow;
 *   rope(x, P): every channel pair (c, c + d/2), c < d/2, turns by the angle P * base^(-2c/d)
 *               (x_c, x_{c+d/2}) <- (x_c cos - x_{c+d/2} sin, x_c sin + x_{c+d/2} cos)
 *   -- the pairing and angles of the Llama family the paper evaluates; the paper itself only names the embedding.
 *   q comes already rotated at its own position; values are not rotated.
 *
 * rope_table   device, 16-byte aligned, squat_rope_table_floats(table_positions) floats as filled (on the host, in
 *              float64, then rounded) by squat_rope_table_fill(base, d, table_positions, .) and copied by the
 *              caller: (cos, sin) of 32 a theta_c for a < ceil(table_positions / 32), then of l theta_c for l < 32.
 *              Must cover every position used: first_pos + n_tokens + n_res <= table_positions.
 * first_pos    position of cached token 0 of every (b, h); >= 0 and a multiple of 32.
 * Everything else as for squat_decode_attention.  Errors: the same, plus SQUAT_ERR_SHAPE for a first_pos that is
 * not a multiple of 32 or a table that is too short.
 */
/* The general form of the two readers: meta16 = 1 reads a cache whose scales and zero-points are binary16 (written
 * by the _m16 functions; the four metadata pointers then point to 2-byte elements); rope_table = NULL reads keys
 * stored after the rotary embedding (table_positions and first_pos are then ignored).  Everything else as above. */
int squat_decode_attention_ex(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                              const unsigned char *k_codes, const void *k_scales, const void *k_zeros,
                              const unsigned char *v_codes, const void *v_scales, const void *v_zeros, int meta16,
                              int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                              int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                              float softmax_scale, const float *rope_table, int table_positions, long long first_pos,
                              float *out, void *workspace, size_t workspace_bytes, void *stream);
size_t squat_rope_table_floats(int n_positions);
int squat_rope_table_fill(double base, int head_dim, int n_positions, float *table_host);
int squat_decode_attention_pre_rope(const void *q, int q_dtype, int batch, int n_q_heads, int n_kv_heads, int head_dim,
                                    const unsigned char *k_codes, const float *k_scales, const float *k_zeros,
                                    const unsigned char *v_codes, const float *v_scales, const float *v_zeros,
                                    int n_tokens, long long cache_stride_b, long long cache_stride_h, int bits,
                                    int group_size, const void *k_res, const void *v_res, int res_dtype, int n_res,
                                    float softmax_scale, const float *rope_table, int table_positions,
                                    long long first_pos, float *out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Gram matrices of the stacked prompt queries without any allocation.  (The paper has no counterpart:
 * this entry exists for callers that must not allocate.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they need the Gram step: code that
 * runs inside a memory-pool or allocator callback, inside a region where the framework has frozen its
 * allocator (for instance while it records work for later replay), or in a process whose device memory
 * has been handed out completely to a serving engine.  squat_subspace_create allocates its scratch; this
 * entry does not.  It computes, for every KV head h, M_h = Qc^T Qc in fp64 (the first stage of
 * squat_build_subspace, same kernels, same layout of q) into the caller's gram_out
 * [n_kv_heads, d, d] (device, float64), keeping its intermediate per-chunk partial sums in a fixed
 * 8 MiB array that is part of the library image on every GPU that loads it.
 *
 * Limits and rules:
 *   - n_kv_heads <= 64 (one 128 KiB partial per head and row chunk, 64 in all); more heads are rejected
 *     with SQUAT_ERR_UNSUPPORTED and nothing is launched.  head_dim must be 128.
 *   - no cudaMalloc, cudaFree or other allocating call is made, on any call.
 *   - the first call on each device looks up the array's device address (with that device current) and
 *     keeps it; make that first call outside any stream capture.
 *   - all calls share the one array.  It keeps whatever the previous call left; every element a call reads
 *     it has written first, so results never depend on earlier calls -- but two calls whose kernels overlap
 *     on the GPU (different streams, or different threads) race on it.  Serialise them.
 */
int squat_gram_static(const void *q, int dtype, int n_q_heads, int n_kv_heads, int n_tokens, int head_dim,
                      long long stride_h, long long stride_t, double *gram_out, void *stream);

/*
 * Measurement aid (the paper has no counterpart): launches one kernel of register-resident single-precision
 * multiply-add chains that keeps every FP32 lane of the GPU busy -- scalar fma.rn.f32 (packed = 0) or two-wide
 * fma.rn.f32x2 (packed = 1) -- so that a benchmark can time it (CUDA events around the call) and quote kernels
 * against the FP32 throughput this GPU actually reaches.  iters in [1, 2^20] sets the length (64 multiply-adds per
 * thread and iteration, twice that when packed); *flops_host (host, may be NULL) receives the floating-point
 * operations the launch performs; sink is a device float the kernel never really writes (it keeps the chains from
 * being optimised away).  Enqueues on `stream`.
 */
int squat_fp32_peak_probe(int packed, int iters, float *sink, long long *flops_host, void *stream);

/*
 * Self-test of the bounds-checked build (the paper has no counterpart).  In libsquat_checked.so (built with
 * -DSQUAT_CHECKED) a kernel forms one address on the last word of a small buffer and one a byte past it, touching
 * neither: *detected (host) is 1 iff the first passed the check and the second raised SQUAT_FLAG_BOUNDS.  The device
 * status word is left as it was.  Synchronises `stream`.  In the normal build: SQUAT_ERR_UNSUPPORTED, *detected = 0.
 */
int squat_checked_selftest(void *stream, int *detected);

/* Reads (and clears when `clear` != 0) the device status word of the current device.
 * Synchronises `stream`.  flags is a host pointer. */
int squat_get_device_status(void *stream, unsigned *flags, int clear);

/* Number of kernels this library has launched in this process (all devices). */
unsigned long long squat_kernel_launch_count(void);

const char *squat_status_string(int status);
/* Text of the last CUDA runtime error seen by the calling thread inside this library. */
const char *squat_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SQUAT_H */
