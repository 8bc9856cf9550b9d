/*
 * loqt.h - C ABI of the B200 (sm_100a) LoQT quantized low-rank linear layer.
 *
 * The layer (LoQT, arXiv 2405.16528, Section 2 and Algorithm 1) is
 *
 *     W_eff = deq(W_q) + s * deq(P_q) * B            (out x in)
 *
 * with W_q (out x in) and P_q (out x r) frozen and stored in NF4 (Section 5.1:
 * 64-weight blocks, each with one fp32 scale M = max|w| per block, 16 levels), B
 * (r x in) the only trained matrix, kept in bf16, and s the adapter scale of
 * Algorithm 1's merge line.
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library
 *     allocates no device memory and keeps no reference after the call's
 *     kernels have run.  `stream` is a cudaStream_t passed as void* (NULL =
 *     default stream).  Work is enqueued asynchronously on that stream.
 *   - Matrices are row-major with an explicit leading dimension in ELEMENTS.
 *     bf16 matrices: base 16-byte aligned, leading dimension a multiple of 8.
 *   - Return value: LOQT_OK or an error code; argument checking is synchronous
 *     and happens before anything is enqueued.  The library never aborts and
 *     never falls back to the CPU; on a device that is not sm_100 every compute
 *     entry point returns LOQT_ERR_ARCH.
 *   - Workspaces are caller-allocated, 256-byte aligned scratch.  Their first
 *     256 bytes hold a sticky device status word: zero it once after
 *     allocation.  Device-side waits are bounded; if one expires the kernel
 *     sets that word and returns.  Read it with loqt_device_status().
 */
#ifndef LOQT_H_
#define LOQT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LOQT_OK = 0,
  LOQT_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, ld too small      */
  LOQT_ERR_ALIGNMENT = 2,   /* pointer or leading dimension violates alignment    */
  LOQT_ERR_UNSUPPORTED = 3, /* block size other than 64, or a size beyond the stated limit */
  LOQT_ERR_WORKSPACE = 4,   /* workspace missing or smaller than required          */
  LOQT_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed                 */
  LOQT_ERR_TIMEOUT = 6,     /* a bounded device-side wait expired                  */
  LOQT_ERR_ARCH = 7,        /* current device is not compute capability 10.x       */
  LOQT_ERR_NUMERIC = 8      /* loqt_projection: an iterate was rank deficient to working precision */
} loqt_status;

/*
 * View of an NF4 matrix (Section 5.1).  DEVICE pointers, caller-owned.
 *   codes  : [rows][ld/2] bytes.  Element k of a row lives in byte k/2: low
 *            nibble when k is even, high nibble when k is odd.  Code c stands
 *            for the c-th NF4 level in ascending order (0 -> -1, 7 -> 0, 15 -> +1).
 *   absmax : [rows][ld/64] fp32, the scale M of each block.
 *   rows, cols : logical shape.   ld : padded row length, ld >= cols,
 *            ld % 64 == 0.  Blocks are 64 consecutive elements of one row; a
 *            row whose length is not a multiple of 64 ends in a short block
 *            whose scale covers its real elements only, and the padding
 *            elements hold code 7 (the exact zero level).
 *   block  : must be 64.
 * codes must be 16-byte aligned, absmax 4-byte aligned.
 */
typedef struct {
  uint8_t *codes;
  float *absmax;
  int32_t rows, cols, ld;
  int32_t block;
} loqt_nf4_mat;

/* Operation selector for loqt_workspace_bytes(). */
enum { LOQT_OP_FWD = 0, LOQT_OP_BWD = 1, LOQT_OP_MERGE = 2, LOQT_OP_MERGE_SPLIT = 3, LOQT_OP_COMPENSATE = 4, LOQT_OP_FULL_GRADIENT = 5,
       LOQT_OP_FWD_RIGHT = 6, LOQT_OP_BWD_RIGHT = 7, LOQT_OP_MERGE_RIGHT = 8, LOQT_OP_PROJECTION = 9,
       LOQT_OP_COMPENSATE_RIGHT = 10 };

/*
 * q_NF4 (Section 5.1, first two displayed equations): per block M = max|w|,
 * per element code = argmin_i |w / M - q_i| (fp32 division, lower index on a
 * tie; an all-zero block gets M = 0 and code 7).
 *   src : fp32 [dst.rows][ld_src] on the device, ld_src >= dst.cols.
 *   dst : receives codes and absmax, padding included.
 * rows * (ld / 64) must stay below 2^30 (LOQT_ERR_UNSUPPORTED otherwise).
 */
loqt_status loqt_nf4_quantize(const float *src, int64_t ld_src, loqt_nf4_mat dst, void *stream);

/*
 * q_NF4^{-1} (Section 5.1, last two displayed equations): w = M * q[code],
 * one fp32 multiply.  Writes src.rows x src.cols elements to `dst` (row-major,
 * ld_dst elements per row), as fp32 when dst_is_bf16 == 0, else rounded once
 * to bf16 (nearest even).  rows * (ld / 8) must stay below 2^31
 * (LOQT_ERR_UNSUPPORTED otherwise).
 */
loqt_status loqt_nf4_dequantize(loqt_nf4_mat src, void *dst, int64_t ld_dst, int dst_is_bf16,
                                void *stream);

/*
 * Forward (Section 2 "Equivalence of Gradient Updates"; Section 2.4 weight-only
 * quantisation; Algorithm 1 merge line for the scale):
 *     y = x deq(W_q)^T + s (x B^T) deq(P_q)^T
 *   Wq : out x in,  Pq : out x r,  B : bf16 [r][ldb] (r x in)
 *   x  : bf16 [T][ldx] (T x in)    y : bf16 [T][ldy] (T x out), overwritten
 * Dequantised operands are bf16 (one rounding of M*q); products accumulate in
 * fp32; the intermediate s*(x B^T) is rounded to bf16.  ws: workspace of at
 * least loqt_workspace_bytes(LOQT_OP_FWD, ...) bytes.
 */
loqt_status loqt_linear_fwd(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                            const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy, void *ws,
                            size_t ws_bytes, void *stream);

/*
 * Backward (same section: G^B = P^T G^W, evaluated factored):
 *     v  = dy deq(P_q)                 (T x r, scratch, kept as bf16 s*v)
 *     dx = dy deq(W_q) + s v B         (bf16 [T][lddx])
 *     dB = s v^T x                     (fp32 [r][lddb])
 * W_q and P_q are frozen: no other gradient is produced.  dB is overwritten,
 * or added to when accumulate_dB != 0 (gradient accumulation).  The split-K
 * reduction of dB is done in a fixed order, so results are reproducible.
 * dx may be NULL to skip the input gradient.  ws: workspace of at least
 * loqt_workspace_bytes(LOQT_OP_BWD, ...) bytes; besides s*v and the split-K
 * partial sums it holds deq(P_q) as bf16 (out x roundup(r, 64)), written once
 * per call so that the product for v need not dequantise P_q again for every
 * 256 token rows.
 */
loqt_status loqt_linear_bwd(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb, float s,
                            const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T,
                            void *dx, int64_t lddx, float *dB, int64_t lddb, int accumulate_dB,
                            void *ws, size_t ws_bytes, void *stream);

/*
 * Periodic merge + requantise (Section 2.4; Algorithm 1 merge line; Section 2.5):
 *     W_q <- q_NF4( deq(W_q) + s deq(P_q) B )        in place
 * deq(W_q) enters as the unrounded fp32 product M*q, deq(P_q) as the bf16
 * operand of the tensor-core product, the sum is formed in fp32.  Each block of
 * W_q depends only on its own previous contents, so the update is in place.
 * Two launches: deq(P_q) is written once, as bf16, into the workspace
 * (loqt_workspace_bytes(LOQT_OP_MERGE, ...) bytes), then the merge kernel forms
 * the product and requantises W_q in its epilogue.
 */
loqt_status loqt_merge_requant(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb,
                               float s, void *ws, size_t ws_bytes, void *stream);

/*
 * The requantising half of the merge on its own (Section 2.4; Algorithm 1 merge
 * line; quantiser of Section 5.1):
 *     W_q <- q_NF4( deq(W_q) + s * delta )            in place
 *   delta : fp32 [Wq.rows][ld_delta] on the device, ld_delta >= Wq.cols.
 * deq(W_q) is the unrounded fp32 product M*q; the sum is one fused multiply-add.
 * Padding elements of a short last block keep code 7.  rows * (ld / 64) must
 * stay below 2^30 (LOQT_ERR_UNSUPPORTED otherwise).
 */
loqt_status loqt_nf4_requantize(const float *delta, int64_t ld_delta, float s, loqt_nf4_mat Wq,
                                void *stream);

/*
 * The merge of loqt_merge_requant in two passes, with the same result bit for
 * bit: deq(P_q) B is written to the workspace as fp32 (out x roundup(in, 64)),
 * then loqt_nf4_requantize streams over it.  Workspace:
 * loqt_workspace_bytes(LOQT_OP_MERGE_SPLIT, ...).  The fused form is the faster
 * one at large shapes; this one exposes the streaming stage for measurement
 * and serves callers that already hold the product.
 */
loqt_status loqt_merge_requant_split(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb,
                                     float s, void *ws, size_t ws_bytes, void *stream);

/*
 * Right-side variant of the layer, for matrices with more rows than columns
 * (Section 2.1, the one-sided projection equation and the paragraph after it:
 * the gradient is projected from the right, G Q, when the matrix is taller than
 * wide, and the adapter derivation carries over with Q^T).  The frozen projection
 * sits on the input side and the trainable factor is tall:
 *     W = deq(W_q) + s B deq(Q_q)      Wq : out x in,  Qq : r x in (NF4, blocks along in),
 *                                     B  : bf16 [out][ldb] (out x r)
 *   forward   y  = x deq(W_q)^T + s (x deq(Q_q)^T) B^T
 *   backward  dx = dy deq(W_q) + s (dy B) deq(Q_q);   dB = s dy^T (x deq(Q_q)^T)   (fp32 [out][lddb])
 *   merge     W_q <- q_NF4( deq(W_q) + s B deq(Q_q) )   in place
 * Arguments, precisions and error behaviour as for loqt_linear_fwd / _bwd /
 * loqt_merge_requant; workspaces from loqt_workspace_bytes(LOQT_OP_FWD_RIGHT /
 * LOQT_OP_BWD_RIGHT / LOQT_OP_MERGE_RIGHT, out, in, r, T).  Forward and backward
 * each keep, in their workspace, a bf16 copy of deq(Q_q) that they write once per
 * call for the product x deq(Q_q)^T (the operand is the same rounding of the same
 * values as the in-product dequantisation gives).
 */
loqt_status loqt_linear_fwd_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb, float s,
                                  const void *x, int64_t ldx, int32_t T, void *y, int64_t ldy,
                                  void *ws, size_t ws_bytes, void *stream);
loqt_status loqt_linear_bwd_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb, float s,
                                  const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T,
                                  void *dx, int64_t lddx, float *dB, int64_t lddb, int accumulate_dB,
                                  void *ws, size_t ws_bytes, void *stream);
loqt_status loqt_merge_requant_right(loqt_nf4_mat Wq, loqt_nf4_mat Qq, const void *B, int64_t ldb,
                                     float s, void *ws, size_t ws_bytes, void *stream);

/*
 * Full-rank gradient of the layer's weight, formed only at merge steps to find
 * the next projection (Algorithm 1: G^W is computed before Initialize; Algorithm
 * 2 takes its leading singular vectors):
 *     G = dy^T x        (fp32 [out][ldg]; overwritten, or added to when accumulate != 0)
 *   x : bf16 [T][ldx],  dy : bf16 [T][lddy].  bf16 products, fp32 accumulation,
 * split over T with a fixed-order reduction when the tiles alone would not fill
 * the GPU.  Workspace: loqt_workspace_bytes(LOQT_OP_FULL_GRADIENT, out, in, 0, T).
 */
loqt_status loqt_full_gradient(const void *x, int64_t ldx, const void *dy, int64_t lddy, int32_t T,
                               int32_t out, int32_t in, float *G, int64_t ldg, int accumulate,
                               void *ws, size_t ws_bytes, void *stream);

/*
 * The projection from the full-rank gradient (Section 2.1, the rank-r factorisation
 * of the gradient; Algorithm 2, the SVD lines: P = the r leading left singular
 * vectors of G^W).  Only the subspace those vectors span enters the method
 * (P P^T G), and the library approximates it by randomised subspace iteration
 * (Halko, Martinsson and Tropp, "Finding structure with randomness", Algorithm 4.4):
 *     Q = orth(G Omega);   repeat iters times:   Z = orth(G^T Q);   Q = orth(G Z);   P = Q
 * The span of P tends to the leading subspace at the rate
 * (sigma_(r+1) / sigma_r)^(2 iters + 1).
 *   G     : fp32 [out][ldg] on the device (from loqt_full_gradient); 16-byte
 *           aligned.  It enters the products rounded once to bf16 (the paper
 *           trains in BF16, so its gradients carry no more).
 *   Omega : bf16 [in][ldo], the in x r test matrix (independent standard normal
 *           entries drawn by the caller; the random numbers are an input).
 *   P     : fp32 [out][ldp], receives out x r with orthonormal columns.
 *   1 <= r <= min(out, in), r <= 4096;  0 <= iters <= 16.
 * Products: tcgen05, bf16 operands with fp32 accumulation; an orthonormalised
 * iterate enters the next product as the sum of two bf16 matrices (value and
 * rounding remainder), so it carries 16 significant bits.  orth() is Cholesky QR
 * in double precision (Gram matrix, blocked Cholesky factorisation, triangular
 * solve).  If an iterate is rank deficient to working precision (G of rank below
 * r, or cond(G Omega) beyond about 1e7) the factorisation meets a non-positive
 * pivot: the kernels then finish with that pivot replaced by one, set the
 * status word, and loqt_device_status() returns LOQT_ERR_NUMERIC; P is then
 * not a valid basis.  Workspace: loqt_workspace_bytes(LOQT_OP_PROJECTION, out, in, r, 0).
 */
loqt_status loqt_projection(const float *G, int64_t ldg, int32_t out, int32_t in, int32_t r,
                            const void *Omega, int64_t ldo, int32_t iters, float *P, int64_t ldp,
                            void *ws, size_t ws_bytes, void *stream);

/*
 * The same for the right-side variant (Section 2.1, the one-sided projection of a
 * matrix with more rows than columns: G Q with Q spanning the leading right
 * singular vectors).  The iteration above runs on G^T:
 *     Q = orth(G^T Omega);   repeat iters times:   Z = orth(G Q);   Q = orth(G^T Z)
 *   Omega : bf16 [out][ldo], the out x r test matrix.
 *   Q     : fp32 [r][ldq], receives the basis transposed, r x in with orthonormal
 *           rows: the layout of the factor Q_q of loqt_linear_fwd_right.
 * Everything else (G, limits, precisions, LOQT_ERR_NUMERIC, workspace) as for
 * loqt_projection.
 */
loqt_status loqt_projection_right(const float *G, int64_t ldg, int32_t out, int32_t in, int32_t r,
                                  const void *Omega, int64_t ldo, int32_t iters, float *Q,
                                  int64_t ldq, void *ws, size_t ws_bytes, void *stream);

/*
 * Error-compensated initialisation of a layer for a new projection P
 * (Section 2.5 "Compensating for Quantization Errors"; Algorithm 2, the loop over
 * compensation steps; appendix: B = P^+ (W - Q)).  Alternating minimisation of
 * || Q + P B - W || with P fixed:
 *     B_0 = 0;   for c = 1..steps:   Q_c = q_NF4( W - P B_{c-1} ),   B_c = P^T ( W - deq(Q_c) )
 *   W  : fp32 [out][ldw] on the device (the full-precision weights to approximate),
 *        16-byte aligned, ldw % 4 == 0.
 *   P  : fp32 [out][ldp], orthonormal columns (so that P^+ = P^T).
 *   Wq : receives Q_steps;  Pq : receives q_NF4(P);  B : receives B_steps as bf16 [r][ldb].
 * W and W - P B are 32-bit; P, the residual W - deq(Q_c) and B enter the
 * tensor-core products as bf16, sums in fp32.  1 <= steps <= 16 (the paper uses
 * at most five).  Workspace: loqt_workspace_bytes(LOQT_OP_COMPENSATE, out, in, r, 0).
 */
loqt_status loqt_compensated_init(const float *W, int64_t ldw, const float *P, int64_t ldp,
                                  int32_t steps, loqt_nf4_mat Wq, loqt_nf4_mat Pq, void *B,
                                  int64_t ldb, void *ws, size_t ws_bytes, void *stream);

/*
 * The same initialisation for the right-side variant W = deq(W_q) + s B deq(Q_q)
 * (Section 2.5 carried over to the right-side factorisation of Section 2.1):
 *     B_0 = 0;   for c = 1..steps:   Q_c = q_NF4( W - B_{c-1} Q ),   B_c = ( W - deq(Q_c) ) Q^T
 *   W  : fp32 [out][ldw], 16-byte aligned, ldw % 4 == 0.
 *   Q  : fp32 [r][ldq], orthonormal rows (from loqt_projection_right).
 *   Wq : receives Q_steps;  Qq : receives q_NF4(Q) (r x in);  B : receives B_steps as bf16 [out][ldb].
 * Precisions and limits as for loqt_compensated_init.  Workspace:
 * loqt_workspace_bytes(LOQT_OP_COMPENSATE_RIGHT, out, in, r, 0).
 */
loqt_status loqt_compensated_init_right(const float *W, int64_t ldw, const float *Q, int64_t ldq,
                                        int32_t steps, loqt_nf4_mat Wq, loqt_nf4_mat Qq, void *B,
                                        int64_t ldb, void *ws, size_t ws_bytes, void *stream);

/*
 * One optimiser step on the trainable factor (Algorithm 1, update line
 * B <- B - rho(G^B); rho = Adam, Section 2.1; optimiser states in BF16 per the
 * hyper-parameter appendix).  Adam as published by Kingma & Ba, with decoupled
 * weight decay:
 *     m <- beta1 m + (1 - beta1) g;   v <- beta2 v + (1 - beta2) g^2
 *     B <- B - lr ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay B )
 *   B  : bf16 [r][ldb], updated in place;  dB : fp32 [r][lddb], the gradient from loqt_linear_bwd;
 *   m, v : bf16 [r][ld_state], updated in place (zero before the first step).
 * fp32 arithmetic, one rounding of B, m, v to bf16.  step counts from 1.  The
 * hyper-parameters are carried as fp32: beta = 0.999 means the fp32 number nearest
 * to it, also inside 1 - beta.
 */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t step;
} loqt_adam_params;

loqt_status loqt_adam_step(void *B, int64_t ldb, const float *dB, int64_t lddb, void *m, void *v,
                           int64_t ld_state, int32_t r, int32_t in, loqt_adam_params hp, void *stream);

/*
 * The same step with the two moments held in 8 bits (the paper trains B with
 * "8-bit Adam": memory comparison of Section 3.2, the 13B run, the continued
 * pretraining appendix; it cites Dettmers et al., "8-bit Optimizers via Block-wise
 * Quantization", whose scheme is taken).  The row-major flattened r x in moments
 * are cut into blocks of 2048 elements; each block has one fp32 scale (its largest
 * magnitude) and one code per element in the dynamic tree data type: bit 7 sign,
 * then a run of E zero bits (a base-10 exponent), an indicator bit and f fraction
 * bits j: magnitude = 10^-E (0.1 + 0.9 (j + 1) / 2^f) times the block scale; code 0
 * is zero.  The non-negative second moment uses bit 7 as a further fraction bit.
 *   st.m8, st.v8 : uint8 [r * in] codes;  st.m_absmax, st.v_absmax : fp32 [ceil(r * in / 2048)]
 *   (all zero before the first step).  B, dB, hp as for loqt_adam_step.
 * Per block: dequantise, Adam update in fp32 (as loqt_adam_step), new block
 * scales, nearest-magnitude quantisation of the new moments.
 */
typedef struct {
  uint8_t *m8;
  float *m_absmax;
  uint8_t *v8;
  float *v_absmax;
} loqt_adam8_state;

loqt_status loqt_adam8_step(void *B, int64_t ldb, const float *dB, int64_t lddb, loqt_adam8_state st,
                            int32_t r, int32_t in, loqt_adam_params hp, void *stream);

/*
 * The same merge for n independent matrices in one call (a whole model at a
 * merge step).  Wq, Pq, B, ldb are HOST arrays of length n; the workspace is
 * shared and must satisfy the largest matrix.  A workspace of 256 + k times the
 * largest matrix's scratch (k up to 8) lets the call stage k matrices ahead,
 * which keeps the GPU from draining between products.
 */
loqt_status loqt_merge_requant_many(int32_t n, const loqt_nf4_mat *Wq, const loqt_nf4_mat *Pq,
                                    const void *const *B, const int64_t *ldb, float s, void *ws,
                                    size_t ws_bytes, void *stream);

/*
 * Double quantisation of the block scales (Section 2.4, last paragraph: the
 * quantiser's own state is quantised a second time, as in QLoRA; the paper gives
 * no parameters, the scheme taken is QLoRA's: the fp32 scales of a matrix, in row-major order
 * [rows][ld/64], are centred by their mean and stored as 8-bit floats - OCP FP8
 * E4M3 - in blocks of 256 with one fp32 second-level scale per block).
 *   codes8 : [n] bytes, n = rows * ld / 64     c1 : [ceil(n / 256)] fp32
 *   offset : one fp32 (device memory)          all DEVICE pointers, caller-owned
 *   encode: offset = mean(c2); per block d = c2 - offset, m = max|d|,
 *           code = E4M3((d / m) * 448) (nearest, ties to even), c1 = m / 448
 *   decode: c2' = E4M3(code) * c1 + offset      (each operation rounded to fp32)
 * Storage per weight: 4 + 8/64 + 32/(64*256) = 4.127 bits instead of 4.5.
 *
 * loqt_scales_double_quantize / _dequantize convert between the fp32 scales of
 * a loqt_nf4_mat and this form (ws: loqt_scales_workspace_bytes() bytes; the
 * mean is summed in double precision in a fixed order, so results are
 * reproducible).  loqt_nf4_dequantize_dq, loqt_linear_fwd_dq and
 * loqt_linear_bwd_dq are loqt_nf4_dequantize, loqt_linear_fwd and
 * loqt_linear_bwd reading the scales of W_q and P_q from this form inside the
 * kernels (the absmax pointers of the loqt_nf4_mat arguments are not read and
 * may be NULL); same arguments, workspaces and error behaviour otherwise.  The
 * merge works on fp32 scales: expand them, merge, and encode the new ones.
 */
typedef struct {
  uint8_t *codes8;
  float *c1;
  float *offset;
  int64_t n;
} loqt_dq_scales;

size_t loqt_scales_workspace_bytes(void);
loqt_status loqt_scales_double_quantize(const float *absmax, loqt_dq_scales dst, void *ws, size_t ws_bytes,
                                        void *stream);
loqt_status loqt_scales_double_dequantize(loqt_dq_scales src, float *absmax, void *stream);
loqt_status loqt_nf4_dequantize_dq(loqt_nf4_mat src, loqt_dq_scales dq, void *dst, int64_t ld_dst,
                                   int dst_is_bf16, void *stream);
loqt_status loqt_linear_fwd_dq(loqt_nf4_mat Wq, loqt_dq_scales Wdq, loqt_nf4_mat Pq, loqt_dq_scales Pdq,
                               const void *B, int64_t ldb, float s, const void *x, int64_t ldx, int32_t T,
                               void *y, int64_t ldy, void *ws, size_t ws_bytes, void *stream);
loqt_status loqt_linear_bwd_dq(loqt_nf4_mat Wq, loqt_dq_scales Wdq, loqt_nf4_mat Pq, loqt_dq_scales Pdq,
                               const void *B, int64_t ldb, float s, const void *x, int64_t ldx,
                               const void *dy, int64_t lddy, int32_t T, void *dx, int64_t lddx, float *dB,
                               int64_t lddb, int accumulate_dB, void *ws, size_t ws_bytes, void *stream);

/*
 * Forward for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a convenience of this library, not part of the method.)
 *
 * Some code that wants to run a LoQT layer has no way to obtain a workspace:
 * a plug-in that is handed tensors by a host framework whose allocator it must
 * not call, code running where cudaMalloc is forbidden because it would
 * synchronise the device (inside a latency-critical serving loop, between the
 * nodes of a pre-planned memory budget), or a small C program that simply owns
 * no allocator.  For them this entry point computes exactly what
 * loqt_linear_fwd computes - same arguments for W_q, P_q, B, s, x, y - but the
 * intermediate s*(x B^T) and the status word live in a fixed array compiled
 * into the library instead of a caller workspace.
 *
 *   - Limit: T * roundup(r, 64) * 2 bytes must not exceed
 *     LOQT_STATIC_FWD_MAX_SCRATCH (8 MiB: e.g. T = 4096 tokens at r = 1024, or
 *     16384 tokens at r = 256).  Larger problems return LOQT_ERR_WORKSPACE and
 *     enqueue nothing; split the tokens or use loqt_linear_fwd.
 *   - Cost: every GPU on which the library is loaded holds the 8 MiB + 256 B
 *     array until the process exits, whether or not this function is called.
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address
 *     (once per device, with that device current).  Make that first call
 *     outside any stream capture.
 *   - All calls on a device share the one array.  Two calls whose kernels can
 *     overlap on the GPU (different streams without an ordering between them)
 *     race on it and produce garbage; calls on one stream are safe.  The array
 *     keeps the previous call's contents; the status word is cleared at the
 *     start of every call, nothing else needs clearing.
 *   - check_device_status != 0: after enqueuing, wait for `stream` and return
 *     LOQT_ERR_TIMEOUT if a bounded device-side wait expired; 0: return as
 *     soon as the work is enqueued (a device-side timeout then goes unreported).
 */
#define LOQT_STATIC_FWD_MAX_SCRATCH (8u * 1024u * 1024u)
loqt_status loqt_linear_fwd_static(loqt_nf4_mat Wq, loqt_nf4_mat Pq, const void *B, int64_t ldb,
                                   float s, const void *x, int64_t ldx, int32_t T, void *y,
                                   int64_t ldy, int check_device_status, void *stream);

/* Bytes of workspace `op` needs for the given shape (never less than 256: the
 * first 256 bytes always hold the device status word). */
size_t loqt_workspace_bytes(int op, int32_t out, int32_t in, int32_t r, int32_t T);

/* Copies the status word at the start of a workspace back to the host
 * (synchronises `stream`) and maps it to LOQT_OK, LOQT_ERR_TIMEOUT (a bounded wait
 * expired) or LOQT_ERR_NUMERIC (loqt_projection met a rank-deficient iterate). */
loqt_status loqt_device_status(const void *ws, void *stream);

/* Number of kernels this library has launched in this process (all entry
 * points, all streams); monotone, for instrumentation. */
uint64_t loqt_launch_count(void);

/*
 * Testing and tuning hooks of the product engine.  (No counterpart in the
 * paper: every product of Section 2 and the merge of Section 2.4 run through one
 * GEMM kernel that exists in several tile shapes, picked per product by a cost
 * model.)
 *
 * loqt_set_tile_override forces a tile shape for every later product of this
 * process that supports it: bn = 128 or 256 output columns per tile, rows = 128
 * or 256 token rows per CTA, pair = 1 to run two CTAs as one tcgen05 pair
 * (needs bn = 256, else LOQT_ERR_UNSUPPORTED).  Products that cannot run the
 * forced shape keep the automatic choice: split-K products never pair, and the
 * merge runs single 128-row tiles only.  bn = 0 restores the automatic choice.
 * The override is process-global and not synchronised with concurrent calls.
 *
 * loqt_variant_launches returns how often the kernel instantiation
 * (bn, rows, pair, nf4) has been launched so far; nf4 = 1 counts the variant
 * that dequantises NF4 operands in its main loop, 0 the one fed by TMA alone.
 */
loqt_status loqt_set_tile_override(int32_t bn, int32_t rows, int32_t pair);
uint64_t loqt_variant_launches(int32_t bn, int32_t rows, int32_t pair, int32_t nf4);

/*
 * Self-test of the bounded device-side wait (no counterpart in the paper).
 * Every wait inside the kernels gives up after a time limit, sets the status
 * word of the workspace and lets the kernel drain and return.  This call
 * launches a one-warp kernel that runs the same wait routine on a barrier
 * nothing ever arrives on, with a limit of limit_us microseconds (1..100000),
 * so that afterwards loqt_device_status(ws) reports LOQT_ERR_TIMEOUT and the
 * context stays usable.  ws: at least 256 bytes, 256-byte aligned; word 0 is
 * the status word, word 2 receives the number of lanes whose wait completed
 * (must be 0), word 3 the CTA's abort flag (must be 1).
 */
loqt_status loqt_selftest_wait_timeout(void *ws, size_t ws_bytes, uint32_t limit_us, void *stream);

const char *loqt_status_string(loqt_status st);

#ifdef __cplusplus
}
#endif
#endif /* LOQT_H_ */
