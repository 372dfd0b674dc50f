/*
 * fp4q -- transposition-invariant 2D-block FP4 quantization and the block-scaled
 * GEMMs it feeds, for NVIDIA B200 (sm_100a).  C ABI of libfp4q.so.
 *
 * Method: "Stable FP4 Training via Transposition-Invariant Block Quantization".
 *   Section 3      2D square blocks (32x32) share one scale; S(B_ij) = S(B_ij^T).
 *   Section 3.1    truncation-free scale S = 2^ceil(log2(2M/(Qp-Qn))); stochastic rounding
 *                  with E[roundS(x)] = x for the backward pass.
 *   Section 3.2    MXFP8 for the query and key projections.
 *   Section 3, "Application to linear layers":  Y = X W^T,  dX = dY W,  dW = dY^T X.
 *
 * Conventions common to every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller; the descriptor structs
 *     themselves (fp4q_tensor, fp4q_groups) are read on the HOST during the call.
 *   - The library allocates no device memory and the compute entry points (quantizers, GEMMs)
 *     never synchronise: they only enqueue work on `stream` (a cudaStream_t passed as void*;
 *     NULL = default stream).  The three small workspace calls (fp4q_workspace_status,
 *     fp4q_workspace_set_wait_limit, fp4q_debug_withhold_load) copy a few bytes and DO
 *     synchronise `stream`.  The first call on a device creates per-device state (module load,
 *     driver entry point lookup, kernel attributes) and should be made outside stream capture.
 *   - Every function returns an fp4q_status; nothing throws, traps or aborts.  Argument
 *     errors are reported before any work is enqueued.  Device-side anomalies (a bounded
 *     wait that ran out) are recorded in the workspace status word and read back with
 *     fp4q_workspace_status(); the kernel then skips its remaining work and exits normally.
 *   - Matrices are row-major with an explicit leading dimension.
 */
#ifndef FP4Q_H
#define FP4Q_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FP4Q_OK = 0,
    FP4Q_ERR_NULL = 1,        /* a required pointer is NULL                                   */
    FP4Q_ERR_SHAPE = 2,       /* negative size, mismatched operand shapes, leading dim too small */
    FP4Q_ERR_ALIGN = 3,       /* pointer or leading dimension violates an alignment rule      */
    FP4Q_ERR_UNSUPPORTED = 4, /* valid request this build does not implement                  */
    FP4Q_ERR_WORKSPACE = 5,   /* workspace missing or smaller than fp4q_workspace_bytes()     */
    FP4Q_ERR_CUDA = 6,        /* a CUDA runtime/driver call failed (launch, tensor map)       */
    FP4Q_ERR_TIMEOUT = 7      /* device status word: a bounded wait expired inside a kernel   */
} fp4q_status;

typedef enum {
    FP4Q_ROUND_NEAREST = 0,    /* round to nearest, ties to even code (forward pass)           */
    FP4Q_ROUND_STOCHASTIC = 1  /* stochastic rounding (gradient tensors in the backward pass) */
} fp4q_round;

typedef enum { FP4Q_OUT_BF16 = 0, FP4Q_OUT_F32 = 1 } fp4q_out;

/* fp4q_quantize2d flag: key the stochastic-rounding stream on the element's index in the
 * TRANSPOSED tensor (j*rows + i instead of i*cols + j), so that quantize(A^T) with this flag
 * reproduces quantize(A) transposed bit for bit. */
#define FP4Q_INDEX_TRANSPOSED 1u
/* Block-size study (Table 4 of the paper): quantize with 16 x 16 or 64 x 64 blocks instead of 32 x 32.
 * FP4Q_BLOCK_64: the scale matrix keeps its 32-granular shape, each block's scale written to its four entries, so the
 *   tensor is a valid operand of every GEMM entry point (the hardware's scale vectors are 32 wide).
 * FP4Q_BLOCK_16: scale is [ceil(rows/16), ld_s >= ceil(cols/16)]; such a tensor is an operand of the three
 *   fp4q_gemm_*_b16 products only (16-element scale vectors are a different mode of the tensor cores). */
#define FP4Q_BLOCK_16 2u
#define FP4Q_BLOCK_64 4u

/*
 * A 2D-block-quantized tensor with logical source shape [rows, cols] (Section 3; appendix
 * "2D Block Scaling and Transposition Consistency").  One UE8M0 scale byte (code = e + 127,
 * S = 2^e) per 32x32 block serves both payload layouts:
 *   q_rm  [rows, ld_rm] bytes: element (i,j) is nibble (j&1) of q_rm[i*ld_rm + j/2]
 *   q_t   [cols, ld_t ] bytes: element (i,j) is nibble (i&1) of q_t [j*ld_t  + i/2]   (may be NULL)
 *   scale [ceil(rows/32), ld_s] bytes: block (I,J) at scale[I*ld_s + J]
 * The low nibble holds the even index.  Element codes are E2M1: bit 3 sign, bits 2..0
 * magnitude code for {0, 0.5, 1, 1.5, 2, 3, 4, 6}.
 * Alignment: q_rm and q_t 16-byte aligned; ld_rm and ld_t multiples of 16 bytes with
 * ld_rm >= ceil32(cols)/2 and ld_t >= ceil32(rows)/2 (ceil32 = round up to 32);
 * ld_s >= ceil(cols/32).  The quantizer writes every payload byte of every block it
 * touches (codes beyond the logical extent are 0); bytes beyond ceil32(.)/2 are left alone.
 */
typedef struct {
    int64_t rows, cols;
    uint8_t *q_rm;
    int64_t ld_rm;
    uint8_t *q_t;
    int64_t ld_t;
    uint8_t *scale;
    int64_t ld_s;
} fp4q_tensor;

/*
 * Token groups of a grouped (mixture-of-experts) product: group g owns rows
 * row_offsets[g] .. row_offsets[g+1]-1 of the token matrices.  row_offsets is a DEVICE array
 * of n_groups+1 non-decreasing int64 values, each a multiple of 128, with row_offsets[0] = 0
 * and row_offsets[n_groups] = the token matrices' row count; padding rows inside a group must
 * hold zeros (the boundary-block rule of the appendix then makes them inert).  Groups may be
 * empty.  row_alignment is the caller's statement about the offsets: 0 or 128 = multiples of 128 (the general
 * case); 256 = every offset is a multiple of 256, which lets the grouped forward and input-gradient products
 * run on the 256-row CTA-pair tiles of the dense products (a wrong statement gives wrong results for the rows
 * of a tile that straddles two groups, nothing worse).  Other values: FP4Q_ERR_UNSUPPORTED.
 */
typedef struct {
    int32_t n_groups;
    int32_t row_alignment;
    const int64_t *row_offsets;
} fp4q_groups;

/*
 * fp4q_quantize2d -- Sections 3 and 3.1; appendix "2D Block Scaling ..." and "Rounding ...".
 * Cuts x (BF16, [rows, cols], leading dimension ld_x in ELEMENTS, any 2-byte-aligned pointer;
 * fastest when 16-byte aligned with ld_x a multiple of 8) into 32x32 blocks; per block takes the
 * maximum magnitude M over the valid entries, the truncation-free scale S = 2^e with e the
 * smallest integer such that 6*2^e >= M (clamped to [-127, 127]; M = 0 gives e = -127), and
 * rounds every x/S to E2M1: to nearest (ties to even) or stochastically.  In stochastic mode
 * an element between neighbours lo <= v < hi goes up iff floor(256*(v-lo)/(hi-lo)) + r8 >= 256
 * where r8 is byte (idx & 15) of Philox4x32-10(counter = (idx>>4 low, idx>>4 high, tensor_id, 0),
 * key = (seed low, seed high)) and idx = i*cols + j.  The same code is written to out->q_rm and
 * (unless NULL) out->q_t, and the scale byte to out->scale.  Inputs are expected finite; for
 * completeness M ignores non-finite entries, +-Inf becomes +-6 and NaN becomes +0.
 * out->rows/cols must equal rows/cols.  rows == 0 or cols == 0 is a no-op.
 */
fp4q_status fp4q_quantize2d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                            const fp4q_tensor *out, fp4q_round mode, uint64_t seed,
                            uint32_t tensor_id, uint32_t flags, void *stream);

/*
 * fp4q_quantize2d_multi -- fp4q_quantize2d applied to several independent tensors by one call (same arithmetic, same
 * bytes as one call per tensor; the rounding stream of tensor j is keyed on jobs[j].tensor_id).  The operands of a
 * layer do not depend on one another and many of them are small (a 4096 x 4096 weight is a few waves of CTAs), so the
 * call enqueues one kernel per tensor on `stream` with each kernel after the first configured as the programmatic
 * dependent of its predecessor: it starts beside the predecessor's last wave instead of after it and completes after
 * it, and whatever is enqueued after the call sees all tensors.  `jobs` is a HOST array of n_jobs descriptors, read
 * during the call; the pointers inside are device pointers as for fp4q_quantize2d.  32 x 32 blocks only (flags: 0 or
 * FP4Q_INDEX_TRANSPOSED).  The tensors must not overlap one another's outputs.  Every job is validated before anything
 * is enqueued; empty tensors are skipped.
 */
typedef struct {
    const void *x_bf16;
    int64_t rows, cols, ld_x;
    const fp4q_tensor *out;
    uint32_t tensor_id;
    uint32_t flags;
} fp4q_quantize_job;

fp4q_status fp4q_quantize2d_multi(const fp4q_quantize_job *jobs, int32_t n_jobs, fp4q_round mode, uint64_t seed,
                                  void *stream);

/* GEMM workspace: fp4q_workspace_bytes() bytes of device memory, 256-byte aligned, zeroed once by
 * the caller before first use (the kernels restore what they use).  Holds the device status word.
 * Calls that share a workspace must not overlap on the GPU. */
size_t fp4q_workspace_bytes(void);

/* Reads the status word of a workspace (synchronous 4-byte device-to-host copy on `stream`
 * followed by a stream synchronise) and clears it.  FP4Q_OK, FP4Q_ERR_TIMEOUT or FP4Q_ERR_CUDA.
 * After FP4Q_ERR_TIMEOUT the outputs of the calls that used the workspace since the last read
 * are unspecified; the context stays usable and later calls are unaffected. */
fp4q_status fp4q_workspace_status(void *ws, void *stream);

/* Every wait inside the GEMM kernels is bounded by a number of polls (default 2^22, far beyond
 * anything a healthy run needs; the one wait that spans a whole tile scales it with the tile's
 * contraction length).  This call stores another limit in the workspace (0 restores the default);
 * it applies to every later call that uses the workspace.  Synchronises `stream`. */
fp4q_status fp4q_workspace_set_wait_limit(void *ws, uint32_t polls, void *stream);

/* Development aid for exercising the timeout path without faulting or hanging anything: with
 * nth_load = n > 0 stored in the workspace, the first CTA of every later GEMM call that uses the
 * workspace leaves out its n-th operand load, so the wait for it runs out, the kernel records
 * FP4Q_ERR_TIMEOUT and leaves through its normal exit.  0 switches the hook off (the state of a
 * zeroed workspace).  Combine with a small wait limit.  Synchronises `stream`. */
fp4q_status fp4q_debug_withhold_load(void *ws, uint32_t nth_load, void *stream);

/*
 * fp4q_gemm_fwd -- Y[T,N] = X^[T,K] W^[N,K]^T  (Section 3, first product), FP32 accumulation.
 * Reads X.q_rm and W.q_rm (both contraction-contiguous) with scales X.scale[t/32, k/32] and
 * W.scale[n/32, k/32].  Y is BF16 or FP32 (dt), leading dimension ldy in elements; Y must be
 * 16-byte aligned and ldy*sizeof(element) a multiple of 16.  T, N arbitrary; K = X.cols = W.cols.
 * Grouped form (g != NULL): X is the permuted token matrix, W the expert stack [n_groups*N, K];
 * row t of group g is multiplied by rows g*N .. g*N+N-1 of the stack.
 */
fp4q_status fp4q_gemm_fwd(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy,
                          fp4q_out dt, const fp4q_groups *g, void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_dgrad -- dX[T,K] = dY^[T,N] W^[N,K]  (Section 3, second product).
 * Reads dY.q_rm and W.q_t; the scale of W for output column k and contraction block nb is
 * W.scale[nb, k/32] -- the same bytes the forward product used, read transposed.
 * Grouped form: W is the stack [n_groups*N, K]; rows of group g contract over stack rows g*N...
 */
fp4q_status fp4q_gemm_dgrad(const fp4q_tensor *dY, const fp4q_tensor *W, void *dX, int64_t ldx,
                            fp4q_out dt, const fp4q_groups *g, void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_wgrad -- dW[N,K] = dY^[T,N]^T X^[T,K]  (Section 3, third product).
 * Reads dY.q_t and X.q_t (both token-contiguous) with scales dY.scale[t/32, n/32] and
 * X.scale[t/32, k/32].  accumulate != 0 adds to the existing dW (FP32 output only).
 * Grouped form: dW is the stack [n_groups*N, K]; block g contracts over the rows of group g
 * only; an empty group yields zeros (or leaves dW unchanged when accumulating).
 */
fp4q_status fp4q_gemm_wgrad(const fp4q_tensor *dY, const fp4q_tensor *X, void *dW, int64_t ldw,
                            fp4q_out dt, int accumulate, const fp4q_groups *g, void *ws,
                            size_t ws_bytes, void *stream);

/*
 * fp4q_mxfp8_quantize1d -- Section 3.2 operand format: x (BF16 [rows, cols], ld_x elements) to
 * E4M3 payload q[rows, ld_q] (bytes; ld_q multiple of 16, q 16-byte aligned) with one UE8M0 scale
 * per 32 consecutive elements of a row, scale[rows, ld_s], ld_s >= ceil(cols/32).  The block scale
 * is the smallest power of two with 448*S >= M (clamped as above); rounding to nearest even;
 * +-Inf -> +-448, NaN -> 0.  Payload bytes from cols to ceil32(cols) are written as 0.
 */
fp4q_status fp4q_mxfp8_quantize1d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                                  uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s,
                                  void *stream);

/*
 * fp4q_mxfp8_qk -- the query and key projections in MXFP8 (Section 3.2):
 *   Q[T,N] = X^ Wq^^T,  K[T,N] = X^ Wk^^T,  FP32 accumulation,
 * on operands produced by fp4q_mxfp8_quantize1d: xq [T, ld_xq] / xs [T, ld_xs];
 * wq_q, wk_q [N, ld_wq] / wq_s, wk_s [N, ld_ws]; contraction length Kdim.
 * Q_out and K_out are BF16 or FP32 with leading dimension ldo (elements).  Either weight may be
 * NULL to skip that projection.
 */
fp4q_status fp4q_mxfp8_qk(const uint8_t *xq, int64_t ld_xq, const uint8_t *xs, int64_t ld_xs,
                          int64_t T, int64_t Kdim,
                          const uint8_t *wq_q, const uint8_t *wq_s,
                          const uint8_t *wk_q, const uint8_t *wk_s, int64_t ld_wq, int64_t ld_ws,
                          int64_t N, void *Q_out, void *K_out, int64_t ldo, fp4q_out dt,
                          void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_quantize1d -- 1D-block FP4 quantization, the layout the paper keeps for activations (Section 3,
 * "Application to linear layers"; appendix "Quantization Placement"): one UE8M0 scale per 32 consecutive elements of a
 * row of x[rows, cols], otherwise the arithmetic of fp4q_quantize2d (truncation-free scale with bound 6, E2M1 codes,
 * nearest-even or stochastic rounding with the random byte of element index i*cols + j, non-finite inputs as there).
 * q [rows, ld_q] packed two codes per byte (low nibble = even column; ld_q >= ceil32(cols)/2, multiple of 16, q
 * 16-byte aligned; bytes up to ceil32(cols)/2 are written, padding codes are 0), scale [rows, ld_s],
 * ld_s >= ceil(cols/32).  Stochastic rounding needs cols % 16 == 0 (FP4Q_ERR_UNSUPPORTED otherwise).
 */
fp4q_status fp4q_quantize1d(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                            uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s,
                            fp4q_round mode, uint64_t seed, uint32_t tensor_id, void *stream);

/*
 * fp4q_quantize1d_t -- the same encoding of the TRANSPOSE: q [cols, ld_q] (q[j, i/2] nibble i&1 encodes x[i, j];
 * ld_q >= ceil32(rows)/2), scale [cols, ld_s] with one scale per column j and 32 consecutive rows i,
 * ld_s >= ceil(rows/32).  Nearest-even rounding (activations are quantized in the forward pass).  This is the operand
 * of the weight-gradient product, which contracts over the rows of x; with 1D blocks it is a second quantization of x
 * whose scales differ from those of fp4q_quantize1d - the inconsistency Figure 1 of the paper illustrates.
 */
fp4q_status fp4q_quantize1d_t(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                              uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s, void *stream);

/*
 * fp4q_gemm_fwd_act1d -- the forward product with the paper's mixed layout (Section 3.1: 2D blocks for weights, 1D
 * blocks for activations): Y[T, N] = X^ W^T, X given by its 1D-block encoding along the contraction axis as written
 * by fp4q_quantize1d (xq [T, ld_xq] packed payload, xs [T, ld_xs] per-row scales; K = W->cols), W a 2D-block tensor
 * (row-major payload used).  Dense only.  Output, workspace, alignment and error behaviour as fp4q_gemm_fwd.
 */
fp4q_status fp4q_gemm_fwd_act1d(const uint8_t *xq, int64_t ld_xq, const uint8_t *xs, int64_t ld_xs, int64_t T,
                                const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt,
                                void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_wgrad_act1d -- the weight-gradient product with a 1D-block activation: dW[N, K] (+)= dY^^T X^_t, dY a
 * 2D-block tensor (transposed payload used; T = dY->rows, N = dY->cols), X given by the 1D-block encoding of its
 * transpose as written by fp4q_quantize1d_t (xtq [K, ld_xtq], xts [K, ld_xts], blocks along the token axis).  This is
 * the product in which 1D blocks force the activation to be quantized a second time with different scales
 * (Figure 1 of the paper).  Dense only.  Output, accumulate, workspace and errors as fp4q_gemm_wgrad.
 */
fp4q_status fp4q_gemm_wgrad_act1d(const fp4q_tensor *dY, const uint8_t *xtq, int64_t ld_xtq, const uint8_t *xts,
                                  int64_t ld_xts, int64_t K, void *dW, int64_t ldw, fp4q_out dt, int accumulate,
                                  void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_mxfp8_quantize1d_t -- the same MXFP8 encoding of the TRANSPOSE of x[rows, cols]: payload q[cols, ld_q]
 * (q[j, i] encodes x[i, j]; ld_q >= ceil32(rows), multiple of 16; q 16-byte aligned) with one UE8M0 scale per
 * column j and 32 consecutive rows i, scale[cols, ld_s], ld_s >= ceil(rows/32).  The paper applies MXFP8 to the
 * query/key projections (Section 3.2) and does not describe their backward pass; the reading taken here is that the
 * backward products re-quantize their operands along the new contraction axis with the same rule, which is what
 * this call produces without a separate transposition.  Payload bytes from rows to ceil32(rows) are written as 0.
 */
fp4q_status fp4q_mxfp8_quantize1d_t(const void *x_bf16, int64_t rows, int64_t cols, int64_t ld_x,
                                    uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s,
                                    void *stream);

/*
 * fp4q_mxfp8_gemm -- C[M,N] = A^ B^^T, FP32 accumulation, on two MXFP8 operands whose rows run along the
 * contraction axis: aq [M, ld_aq] / as [M, ld_as], bq [N, ld_bq] / bs [N, ld_bs], contraction length Kdim
 * (payload pitch >= ceil32(Kdim), scale pitch >= ceil(Kdim/32)).  C is BF16 or FP32 with leading dimension ldc.
 * With the two quantizers above it gives the backward products of an MXFP8 projection Y = X W^T:
 *   dX[T,K] = dY W      : A = quantize1d(dY)   [T, N],  B = quantize1d_t(W)  [K, N],  Kdim = N
 *   dW[N,K] = dY^T X    : A = quantize1d_t(dY) [N, T],  B = quantize1d_t(X)  [K, T],  Kdim = T
 * fp4q_mxfp8_qk is this call applied to the two forward projections.  ws/ws_bytes/stream as for fp4q_gemm_fwd.
 */
fp4q_status fp4q_mxfp8_gemm(const uint8_t *aq, int64_t ld_aq, const uint8_t *as, int64_t ld_as, int64_t M,
                            const uint8_t *bq, int64_t ld_bq, const uint8_t *bs, int64_t ld_bs, int64_t N,
                            int64_t Kdim, void *C, int64_t ldc, fp4q_out dt,
                            void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_fwd_quantized -- the dense forward product with the output quantization fused into the GEMM's epilogue
 * (Section 3.1 feeds each layer's BF16 output to the next layer's quantizer; here the tile is quantized while it is
 * still in registers):
 *   Y = X^ W^^T with FP32 accumulation, rounded to BF16, then Yq = 2D-block FP4 of Y exactly as fp4q_quantize2d
 *   computes it from that BF16 matrix with the same mode, seed and tensor_id (element index i*N + j): same block
 *   maxima, scales, codes, both payload layouts; Y itself is never written.
 * X [T,K], W [N,K] as for fp4q_gemm_fwd (dense form).  Yq: rows = T, cols = N, layouts and alignment as for
 * fp4q_quantize2d (q_t may be NULL).  N must be a multiple of 16 (FP4Q_ERR_UNSUPPORTED otherwise); T is free.
 * Grouped form (g != NULL; NULL = dense): as fp4q_gemm_fwd, with g->row_alignment = 256 required (the epilogue lives
 * in the CTA-pair kernel, whose tiles span 256 rows; FP4Q_ERR_UNSUPPORTED otherwise).
 * ws/ws_bytes/stream and the asynchronous FP4Q_ERR_TIMEOUT report are those of fp4q_gemm_fwd.
 */
fp4q_status fp4q_gemm_fwd_quantized(const fp4q_tensor *X, const fp4q_tensor *W, const fp4q_tensor *Yq,
                                    fp4q_round mode, uint64_t seed, uint32_t tensor_id, const fp4q_groups *g,
                                    void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_dgrad_quantized -- the dense input-gradient product with the same fused epilogue: dX = dY^ W^ with FP32
 * accumulation, rounded to BF16, then dXq = 2D-block FP4 of dX exactly as fp4q_quantize2d computes it (element index
 * i*K + j): the layer's dX is the previous layer's dY, which the backward pass quantizes with stochastic rounding
 * (Section 3.1), so that quantization can happen here and dX never reaches memory in BF16.
 * dY [T,N] (row-major payload used), W [N,K] (transposed payload used) as for fp4q_gemm_dgrad (dense form).
 * dXq: rows = T, cols = K (multiple of 16), otherwise as Yq of fp4q_gemm_fwd_quantized; errors and grouped form as
 * there (W then is the stack [n_groups*N, K], N a multiple of 64).
 */
fp4q_status fp4q_gemm_dgrad_quantized(const fp4q_tensor *dY, const fp4q_tensor *W, const fp4q_tensor *dXq,
                                      fp4q_round mode, uint64_t seed, uint32_t tensor_id, const fp4q_groups *g,
                                      void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_fwd_b16 / fp4q_gemm_dgrad_b16 / fp4q_gemm_wgrad_b16 -- the three products of Section 3 on tensors
 * quantized in 16 x 16 blocks (the block-size study of Table 4 and the appendix "Block size"): operands are
 * fp4q_tensor descriptors written by fp4q_quantize2d with FP4Q_BLOCK_16, i.e. the usual two payloads and a scale
 * matrix [ceil(rows/16), ld_s >= ceil(cols/16)]; the scale of element (i, j) is scale[i/16, j/16], read transposed for
 * the transposed payload exactly as in the 32 x 32 case.  Same outputs, accumulation, alignment rules, workspace and
 * error behaviour as fp4q_gemm_fwd / _dgrad / _wgrad; dense form only.  Mixing block sizes in one product is not
 * supported (both operands must be 16-block tensors; the library cannot tell, the scale matrix's shape is the caller's
 * statement).
 */
fp4q_status fp4q_gemm_fwd_b16(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy, fp4q_out dt,
                              void *ws, size_t ws_bytes, void *stream);
fp4q_status fp4q_gemm_dgrad_b16(const fp4q_tensor *dY, const fp4q_tensor *W, void *dX, int64_t ldx, fp4q_out dt,
                                void *ws, size_t ws_bytes, void *stream);
fp4q_status fp4q_gemm_wgrad_b16(const fp4q_tensor *dY, const fp4q_tensor *X, void *dW, int64_t ldw, fp4q_out dt,
                                int accumulate, void *ws, size_t ws_bytes, void *stream);

/*
 * fp4q_gemm_fwd_static_workspace -- no counterpart in the paper: the dense forward product of
 * fp4q_gemm_fwd for callers that cannot allocate device memory (code living inside an application that
 * owns the device heap, a loop that must stay out of the allocator, a sandbox restricted to buffers it was
 * handed).  It calls no cudaMalloc, cudaFree or allocating library routine: the kernel's workspace is a
 * fixed 1024-byte array inside the library's device image (held by every GPU that loads the library
 * until the process exits).  A request is refused with FP4Q_ERR_WORKSPACE if the workspace the kernels
 * need (fp4q_workspace_bytes()) exceeds those 1024 bytes; the workspace does not grow with T, N or K, so
 * no problem size is refused on its account.  X, W, Y, ldy and dt mean what they mean for fp4q_gemm_fwd
 * (dense form only).  status_out, if not NULL, is a DEVICE pointer to 4 bytes that receives the kernel's
 * status word (0, or FP4Q_ERR_TIMEOUT) in stream order after the product.
 * The first call on a device looks up the array's device address (and, like fp4q_gemm_fwd, sets the
 * kernel's shared-memory attribute): make that first call before any stream capture.
 * Every call shares the one array and clears it first: two calls that overlap on the GPU (different
 * streams, or different host threads) race on it, so keep calls to this entry point in one stream order.
 */
fp4q_status fp4q_gemm_fwd_static_workspace(const fp4q_tensor *X, const fp4q_tensor *W, void *Y, int64_t ldy,
                                           fp4q_out dt, uint32_t *status_out, void *stream);

const char *fp4q_status_string(fp4q_status s);

/* Library version: major*10000 + minor*100 + patch. */
int fp4q_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FP4Q_H */
