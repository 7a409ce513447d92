/*
 * quest.h -- C ABI of the B200 (sm_100a) QuEST quantized-linear library.
 *
 * The library implements the forward pass of one QuEST linear layer (Algorithm 1 of
 * "QuEST: Stable Training of LLMs with 1-Bit Weights and Activations", arXiv 2502.05003):
 *
 *     x_h = HT(x);  xq_h = proj_{alpha*}(x_h);  w_h = HT(w);  wq_h = proj_{alpha*}(w_h);
 *     y   = xq_h wq_h^T;   return y, xq_h, wq_h, M(x_h; xq_h), M(w_h; wq_h)
 *
 * and, further down, its backward pass (Algorithm 2), the FP4 grid of Section 4.4 and the
 * weight-only variant of Section 4.5.
 *
 * General rules for every entry point
 *   - Pointers named in "device" are CUDA device pointers owned by the caller; the library
 *     allocates no device memory.  Inputs are never written; inputs and outputs must not alias.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and the call returns without synchronising; outputs are valid once the stream reaches
 *     that point.
 *   - The return value is a quest_status; 0 is success.  All argument checks run on the host
 *     before anything is launched: on an argument error nothing is enqueued.  The library
 *     never throws, aborts or traps.
 *   - Tensors are row-major.  `dtype`: QUEST_F32 (binary32) or QUEST_BF16 (bfloat16).
 *
 * Packed formats (shared by every entry point)
 *   - Level index k in [0, 2^b - 1]; the grid value is c = 2k - (2^b - 1), an odd integer, and
 *     the dequantised element is scale[row] * c (Eq. 1's zero-free uniform grid).
 *   - Codes: container(b) = 1, 2, 4, 4, 8, 8, 8, 8 bits for b = 1..8; a row of `cols` codes
 *     occupies cols*container/8 bytes, rows are dense; element e of a row sits in byte
 *     e / (8/container) at bit offset (e mod (8/container)) * container (element 0 lowest).
 *   - Trust mask: one bit per element, row of cols/8 bytes, element e at bit (e mod 8) of
 *     byte e/8; 1 = trusted (gradient passes), 0 = masked.
 *   - Scales: one binary32 per row, the half step of the row's grid in the orthonormal
 *     Hadamard domain: alpha*(b) * RMS(x_h) / (2^b - 1).
 */
#ifndef QUEST_H_
#define QUEST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum quest_status {
    QUEST_OK = 0,
    QUEST_ERR_NULL = 1,           /* a required pointer is NULL */
    QUEST_ERR_SHAPE = 2,          /* rows/cols/M/N/K/ld out of range or not a supported multiple */
    QUEST_ERR_BITS = 3,           /* bits outside 1..8 */
    QUEST_ERR_HAD_BLOCK = 4,      /* had_block not a power of two, does not divide cols, or > 16384 */
    QUEST_ERR_DTYPE = 5,          /* unknown dtype code */
    QUEST_ERR_ALIGN = 6,          /* a pointer or leading dimension is not aligned as required */
    QUEST_ERR_TRUST = 7,          /* trust_factor negative, infinite or NaN */
    QUEST_ERR_WORKSPACE = 8,      /* workspace NULL or smaller than quest_workspace_bytes() */
    QUEST_ERR_OVERFLOW = 9,       /* K*(2^bx-1)*(2^bw-1) does not fit in int32 */
    QUEST_ERR_DEVICE = 10,        /* current device is not compute capability 10.x */
    QUEST_ERR_CUDA = 11,          /* a CUDA runtime/driver call failed; see quest_last_cuda_error() */
    QUEST_ERR_DEVICE_TIMEOUT = 12,/* a bounded wait inside a kernel expired (see quest_device_status) */
    QUEST_ERR_STATIC_LIMIT = 13   /* quest_lowbit_gemm_static: problem needs more than QUEST_STATIC_SCRATCH_BYTES */
} quest_status;

enum { QUEST_F32 = 0, QUEST_BF16 = 1 };

/*
 * quest_quantize -- the rotation and projection steps of Algorithm 1 for every row of x: the Hadamard
 * rotation of Eq. 2, the RMS normalisation and alpha*(b) clipping of Section 3.1 ("Gaussian
 * Fitting"), rounding onto Eq. 1's b-bit grid, and the trust mask of Section 3.2.
 *
 *   x            device, [rows x cols], row stride ld_elems elements, dtype as given; 16-byte
 *                aligned, ld_elems*sizeof(elem) a multiple of 16
 *   rows, cols   rows >= 0 (0 is a no-op); 8 <= cols <= 16384, cols % 8 == 0
 *   bits         b in 1..8
 *   had_block    g: the rotation is block-diagonal with the Sylvester-Hadamard matrix H_g on
 *                contiguous blocks of g elements; a power of two dividing cols (1 = no rotation)
 *   trust_factor s >= 0: M = [|x_h - xq_h| <= s * alpha* RMS/(2^b-1)] ("The 1-bit Case": s = 1.3
 *                at b = 1; 1.0 otherwise)
 *   codes        device out, rows*cols*container/8 bytes, 16-byte aligned; may be NULL
 *   scales       device out, rows binary32; may be NULL
 *   mask         device out, rows*cols/8 bytes, 4-byte aligned; may be NULL
 * Rounding decisions are taken in binary32 in a fixed operation order (descending-stride
 * butterflies, pairwise sum of squares, one fused multiply-add onto the level axis, ties to
 * even), so codes and masks are reproducible bit for bit.  A row of zeros gets scale 0, the
 * middle level and an all-ones mask (for s >= 1).
 */
int quest_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                   int bits, int had_block, float trust_factor,
                   uint8_t *codes, float *scales, uint8_t *mask, void *stream);

/*
 * quest_trust_mask -- the trust mask M_{alpha*}(x_h; xq_h) of Section 3.2 alone (what Algorithm 1
 * returns for the backward pass), recomputed from x.  Same arguments and rules as
 * quest_quantize; `mask` is required.
 */
int quest_trust_mask(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                     int bits, int had_block, float trust_factor, uint8_t *mask, void *stream);

/*
 * quest_lowbit_gemm -- the product step of Algorithm 1 on packed codes: acc[i][j] = sum_k cx[i][k]*cw[j][k]
 * exactly, reported as int32 (tensor cores: int8 operands, or E2M1 operands on the FP4 path when both
 * widths are at most 2, whose grid values +-1 and +-3 are E2M1 numbers), then
 * y[i][j] = sx[i]*sw[j]*acc[i][j] (Section 5: integer matmul with the dequantisation fused into the
 * epilogue).
 *
 *   xq, sx, bits_x   device: codes [M x K] and scales [M] of the activations
 *   wq, sw, bits_w   device: codes [N x K] and scales [N] of the weights (both operands K-major)
 *   M, N, K          M, N >= 0; 32 <= K <= 65504, K % 32 == 0; K*(2^bx-1)*(2^bw-1) < 2^31
 *   y, y_dtype, ldy  device out [M x N], row stride ldy elements, QUEST_F32 or QUEST_BF16;
 *                    may be NULL if only acc is wanted
 *   acc              device out, dense [M x N] int32 raw accumulators; may be NULL
 *   workspace        device scratch of at least quest_workspace_bytes(M, N, K, bits_x, bits_w)
 *                    bytes, 256-byte aligned; holds the operands the tensor cores read.
 *                    Its contents are undefined afterwards; two calls that overlap on the GPU
 *                    must not share it.
 */
int quest_lowbit_gemm(const uint8_t *xq, const float *sx, int bits_x,
                      const uint8_t *wq, const float *sw, int bits_w,
                      int64_t M, int64_t N, int64_t K,
                      void *y, int y_dtype, int64_t ldy_elems, int32_t *acc,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * quest_lowbit_gemm_static -- quest_lowbit_gemm without a workspace argument.  The paper has no
 * counterpart: this exists for callers that cannot allocate device memory, such as a plug-in that
 * only receives input and output pointers from its host application, a server that handed all of
 * device memory to its own pools at start-up (a later cudaMalloc would fail), or a loop that cannot
 * afford the device-wide synchronisation an allocation implies.  The int8 operands go to a fixed
 * array of QUEST_STATIC_SCRATCH_BYTES inside the library image; each GPU that loads the library holds
 * that much memory until the process exits.
 *
 *   Arguments, results and error codes are those of quest_lowbit_gemm (caller still passes codes,
 *   scales and outputs).  In addition QUEST_ERR_STATIC_LIMIT is returned, before anything is
 *   launched, when quest_workspace_bytes(M, N, K, bits_x, bits_w) exceeds
 *   QUEST_STATIC_SCRATCH_BYTES, i.e. roughly when (M + N) * K > 4 Mi elements.
 *   The call itself allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine.
 *   The first call on each device looks up the array's device address (one cudaGetSymbolAddress,
 *   with that device current); make that first call outside any stream capture.
 *   All calls in the process share the one array per device and it keeps whatever the last call
 *   left there.  Nothing in it has to start at zero (every byte the kernels read is rewritten by the
 *   same call first), but two calls whose kernels overlap on the GPU (different streams, or
 *   different host threads) race on it and produce garbage: serialise them on one stream.
 */
#define QUEST_STATIC_SCRATCH_BYTES (4u << 20)
int quest_lowbit_gemm_static(const uint8_t *xq, const float *sx, int bits_x,
                             const uint8_t *wq, const float *sw, int bits_w,
                             int64_t M, int64_t N, int64_t K,
                             void *y, int y_dtype, int64_t ldy_elems, int32_t *acc,
                             void *stream);

/*
 * quest_linear_fwd -- Algorithm 1 end to end: quantize x rows, quantize w rows (unless cached),
 * contract, scale.  No inverse transform is applied to y: the same rotation on both operands
 * cancels in the product ("Implementation" paragraph of Section 3.3).
 *
 *   x [M x K], w [N x K]   device, dense row-major, `dtype`
 *   y [M x N]              device out, dense, `y_dtype`
 *   xq, sx, mx             device out: codes, scales, trust mask of x (the values Algorithm 1 returns);
 *                          xq and sx are required, mx may be NULL
 *   wq, sw, mw             the same for w.  If w_is_cached != 0, w may be NULL and wq/sw are
 *                          INPUTS produced by an earlier call with the same bits and had_block
 *                          (the inference pipeline of Section 5); mw is then untouched
 *   w_is_cached            0: quantize w.  1: take wq/sw and unpack wq into the workspace.
 *                          2: as 1, and the workspace already holds the tensor-core operand of this
 *                          w: it was filled by an earlier call (w_is_cached 0 or 1) with the same
 *                          workspace pointer, w, N, K and bits, and nothing else wrote the workspace
 *                          since.  M may differ between those calls (w's operand sits at the start of
 *                          the workspace); the workspace must be large enough for this call's M.
 *                          Other values: QUEST_ERR_SHAPE.
 *   workspace              as for quest_lowbit_gemm with bits_x = bits_w = bits
 */
int quest_linear_fwd(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                     int bits, int had_block, float trust_factor,
                     void *y, int y_dtype,
                     uint8_t *xq, float *sx, uint8_t *mx,
                     uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                     void *workspace, size_t workspace_bytes, void *stream);

/*
 * quest_linear_fwd in two calls, for callers that schedule the two halves of Algorithm 1 themselves (weights
 * quantized once and contracted with several batches of activations; a half run on another stream; a half timed
 * alone).  quest_linear_fwd_quantize is the rotation and projection steps: it writes the codes, scales and masks
 * exactly as quest_linear_fwd does (same arguments, without y) and leaves the tensor-core operands of x and w in
 * `workspace`.  quest_linear_fwd_contract is the product step: it contracts the operands that the first call left
 * in the same `workspace` (same M, N, K, bits; nothing else may have written the workspace in between) and applies
 * the scales.  The pair, in this order on one stream, is quest_linear_fwd.
 */
int quest_linear_fwd_quantize(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                              int bits, int had_block, float trust_factor,
                              uint8_t *xq, float *sx, uint8_t *mx,
                              uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                              void *workspace, size_t workspace_bytes, void *stream);
int quest_linear_fwd_contract(const float *sx, const float *sw, int64_t M, int64_t N, int64_t K, int bits,
                              void *y, int y_dtype, void *workspace, size_t workspace_bytes, void *stream);

/*
 * quest_mlp_fwd -- forward pass of a Llama-style MLP block (the model family of the paper's experiments;
 * hyper-parameter table: MLP width 8/3 of the hidden size) in which each of the three linear layers is
 * Algorithm 1:
 *
 *     gate = QuEST_linear(x, w_gate);  up = QuEST_linear(x, w_up);     x is rotated and quantized once
 *     h    = bf16( silu(gate) * up ),  silu(z) = z / (1 + exp(-z))     gate, up and the product in binary32
 *     y    = QuEST_linear(h, w_down)
 *
 * Four launches on `stream`: quantizer (x, w_gate, w_up), contraction of x_q with both weight matrices with
 * the SwiGLU in its epilogue (gate and up never reach memory; Section 5 fuses the dequantisation into the
 * matmul epilogue for the same reason), quantizer (h, w_down), contraction with the dequantising epilogue.
 * No allocation and no synchronisation, so the call can be captured into a CUDA graph.
 *
 *   x [T x H], w_gate [I x H], w_up [I x H], w_down [H x I]   device, dense row-major, `dtype`
 *   T, H, I          tokens, hidden size, MLP width; H and I multiples of 32 (and of had_block), <= 16384
 *   h [T x I]        device out, bfloat16, dense, 16-byte aligned: the hidden activations the down projection
 *                    quantizes (a backward pass needs them as well)
 *   y [T x H]        device out, dense, y_dtype
 *   saved            device out: codes, per-row scales and trust masks of all five quantized tensors (what
 *                    Algorithm 1 returns for each layer); codes and scales are required, masks may be NULL
 *   workspace        device scratch of at least quest_mlp_workspace_bytes(T, H, I) bytes, 256-byte aligned
 * Errors as for quest_linear_fwd.
 */
typedef struct quest_mlp_saved {
    uint8_t *xq;  float *sx;  uint8_t *mx;      /* x       [T x H] */
    uint8_t *wgq; float *swg; uint8_t *mwg;     /* w_gate  [I x H] */
    uint8_t *wuq; float *swu; uint8_t *mwu;     /* w_up    [I x H] */
    uint8_t *hq;  float *sh;  uint8_t *mh;      /* h       [T x I] */
    uint8_t *wdq; float *swd; uint8_t *mwd;     /* w_down  [H x I] */
} quest_mlp_saved;
int quest_mlp_fwd(const void *x, const void *w_gate, const void *w_up, const void *w_down, int dtype,
                  int64_t T, int64_t H, int64_t I, int bits, int had_block, float trust_factor,
                  void *h, void *y, int y_dtype, const quest_mlp_saved *saved,
                  void *workspace, size_t workspace_bytes, void *stream);
size_t quest_mlp_workspace_bytes(int64_t T, int64_t H, int64_t I);

/*
 * quest_linear_bwd -- Algorithm 2 (QuEST training backward) for one linear layer, from what
 * quest_linear_fwd saved:
 *
 *     dL/dxq_h = dL/dy wq_h;   dL/dx = IHT(M(x_h; xq_h) * dL/dxq_h)
 *     dL/dwq_h = dL/dy^T xq_h; dL/dw = IHT(M(w_h; wq_h) * dL/dwq_h)
 *
 * with the trust estimator of Section 3.2 applied in the Hadamard domain and IHT the inverse of
 * the orthonormal block Hadamard transform.  The two products run on the tensor cores with
 * bfloat16 operands and binary32 accumulation (Section 3.3 keeps the backward products in 16 bits): dL/dy as
 * given, the quantized operand dequantised to bfloat16 (scale * grid value, one rounding per element).
 *
 *   dy                 device, [M x N] bfloat16, dense, 16-byte aligned
 *   M, N, K            M, N > 0 and multiples of 8; 32 <= K <= 16384, K % 32 == 0
 *   bits, had_block    as in the forward call that produced the codes
 *   xq, sx, mx         device: codes [M x K], scales [M], trust mask [M x K/8] of x (forward outputs);
 *                      masks 16-byte aligned, codes 4-byte aligned
 *   wq, sw, mw         the same for w ([N x K])
 *   dx, dw             device out: [M x K] and [N x K], dense, out_dtype (QUEST_F32 or QUEST_BF16),
 *                      16-byte aligned; either may be NULL to skip that gradient
 *   workspace          device scratch of at least quest_bwd_workspace_bytes(M, N, K) bytes, 256-byte
 *                      aligned (dequantised bfloat16 operands and the masked binary32 products)
 */
int quest_linear_bwd(const void *dy, int64_t M, int64_t N, int64_t K, int bits, int had_block,
                     const uint8_t *xq, const float *sx, const uint8_t *mx,
                     const uint8_t *wq, const float *sw, const uint8_t *mw,
                     void *dx, void *dw, int out_dtype,
                     void *workspace, size_t workspace_bytes, void *stream);
size_t quest_bwd_workspace_bytes(int64_t M, int64_t N, int64_t K);

/*
 * FP4 variant -- Section 4.4, "The FP4 Format": the rounding of Eq. 1 is replaced by rounding to the
 * FP4 (E2M1) grid +-{0, .5, 1, 1.5, 2, 3, 4, 6} scaled to [-1, 1], with alpha*_FP4 the minimiser of the
 * same Gaussian MSE on that grid and the trust bound T its largest half-interval (times
 * trust_factor).  Formats: codes are E2M1 nibbles (sign << 3 | magnitude index, two per byte,
 * element 0 in the low nibble, rounded to nearest even and saturated by the hardware conversion);
 * scale[row] = alpha*_FP4 RMS(x_h) / 6, so the dequantised element is scale * E2M1 value; masks as for
 * the uniform grid.  The contraction runs on the FP4 tensor-core path (tcgen05 kind::mxf4 with every
 * block scale 2^0) directly on the packed codes; its binary32 accumulators hold sum_k v_x v_w exactly
 * (multiples of 1/4 below 2^22 for every supported K), reported as acc4[i][j] = 4 sum_k v_x v_w in int32,
 * and y = sx[i] sw[j] acc4 / 4.
 * Arguments and rules are those of quest_quantize / quest_lowbit_gemm / quest_linear_fwd with
 * bits = 4; cols (K) must be a multiple of 32 and xq, wq 16-byte aligned.  Nothing is unpacked, so
 * the workspace arguments of the two GEMM-bearing calls are unused and may be NULL / 0.
 */
float quest_alpha_star_fp4(void);
int quest_quantize_fp4(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld_elems,
                       int had_block, float trust_factor,
                       uint8_t *codes, float *scales, uint8_t *mask, void *stream);
int quest_lowbit_gemm_fp4(const uint8_t *xq, const float *sx, const uint8_t *wq, const float *sw,
                          int64_t M, int64_t N, int64_t K,
                          void *y, int y_dtype, int64_t ldy_elems, int32_t *acc4,
                          void *workspace, size_t workspace_bytes, void *stream);
int quest_linear_fwd_fp4(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                         int had_block, float trust_factor,
                         void *y, int y_dtype,
                         uint8_t *xq, float *sx, uint8_t *mx,
                         uint8_t *wq, float *sw, uint8_t *mw, int w_is_cached,
                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * Weight-only variant -- Section 4.5, "Weight-only quantization": the weights are quantized to bits_w
 * bits as in Algorithm 1 (its two weight steps), the activations keep 16 bits.  The paper gives no algorithm of
 * its own for this case; here it is Algorithm 1 with the rounding of the activations left out:
 *   x_h = bf16(HT(x))         every butterfly and the factor 1/sqrt(had_block) in binary32, in the
 *                             quantizer's order, one rounding to bfloat16 (nearest even) at the end
 *   w_q, sw, mw               exactly the outputs of quest_quantize(w, bits_w, had_block, trust_factor)
 *   y[m][n] = sw[n] * sum_k x_h[m][k] c_w[n][k],   c_w = 2 k_w - (2^bits_w - 1)
 * The sum runs on the tensor cores over bfloat16 operands (both exact) with binary32 accumulation in an
 * order the hardware chooses, so y agrees with the exact sum to a few units of K * 2^-24 * sw[n] *
 * sum_k |x_h c_w|, plus the rounding of y_dtype; x_h, w_q, sw and mw are reproducible bit for bit.
 *
 *   x [M x K], w [N x K]   device, QUEST_F32 or QUEST_BF16 each, row strides ldx / ldw elements,
 *                          16-byte aligned rows; K a multiple of 32, 32 <= K <= 16384
 *   y [M x N]              device, y_dtype, row stride ldy elements
 *   xh                     optional device output [M x K] bfloat16, dense, 16-byte aligned
 *   wq, sw, mw             optional device outputs as in quest_quantize
 *   workspace              device scratch of at least quest_weight_only_workspace_bytes(M, N, K)
 *                          bytes, 256-byte aligned; nothing is allocated by the call
 * Errors as for quest_linear_fwd; M = 0 or N = 0 is QUEST_OK and launches nothing.
 */
int quest_linear_fwd_weight_only(const void *x, int x_dtype, int64_t ldx, const void *w, int w_dtype, int64_t ldw,
                                 int64_t M, int64_t N, int64_t K, int bits_w, int had_block, float trust_factor,
                                 void *y, int y_dtype, int64_t ldy, void *xh, uint8_t *wq, float *sw, uint8_t *mw,
                                 void *workspace, size_t workspace_bytes, void *stream);
size_t quest_weight_only_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Bytes of scratch quest_lowbit_gemm / quest_linear_fwd need (0 on invalid arguments). */
size_t quest_workspace_bytes(int64_t M, int64_t N, int64_t K, int bits_x, int bits_w);

/* rows*cols*container(bits)/8, the size of a packed code tensor (0 on invalid arguments). */
size_t quest_codes_bytes(int64_t rows, int64_t cols, int bits);

/* The binary32 table entry alpha*(b) of Section 3.1 (0 outside 1..8). */
float quest_alpha_star(int bits);

/*
 * Kernels never spin without bound: a wait that expires records a non-zero word on the device
 * and the kernel returns.  quest_device_status synchronises `stream`, reads that word, clears
 * it, and returns QUEST_OK or QUEST_ERR_DEVICE_TIMEOUT (QUEST_ERR_CUDA if the read fails).
 */
int quest_device_status(void *stream);
/* The same call under a second name ("status of the last kernels on this stream"); kept so that code
 * written against either spelling links. */
int quest_last_device_status(void *stream);

/*
 * quest_selftest_bounded_wait -- diagnostic (no counterpart in the paper): runs the time-out path of the
 * kernels' bounded waits on purpose and harmlessly.  A one-warp kernel waits on a barrier that nothing will
 * complete, with a limit of `limit_cycles` SM clock cycles (1e3 .. 4e9; 2e6 is about a millisecond); the wait
 * gives up, records the time-out in the device status word and returns; a second wait in the same CTA is
 * then refused at once.  No fault, no trap, the context stays usable.  After the stream has run it,
 * quest_device_status returns QUEST_ERR_DEVICE_TIMEOUT once and QUEST_OK from then on.
 *   report   optional device array of 4 ints: [0] first wait satisfied (expect 0), [1] second wait satisfied
 *            (expect 0), [2] abort flag of the CTA (expect 1), [3] second wait shorter than the first (expect 1)
 */
int quest_selftest_bounded_wait(int64_t limit_cycles, int *report, void *stream);

/*
 * Measurement aid (no counterpart in the paper): per-stage device times.  While enabled, every
 * entry point brackets each of its stages with a pair of CUDA events on the caller's stream.
 * quest_stage_times waits for the events of the most recent call, adds their elapsed times to
 * running totals, copies totals (milliseconds) and counts into the caller's HOST arrays of
 * QUEST_NUM_STAGES entries (either may be NULL), and zeroes the totals if reset != 0.  Call it
 * after every timed call: events are reused from call to call.  A call made while its stream is
 * being captured records its events as graph nodes instead: every replay of the graph re-times
 * the stages, and quest_stage_times, called after a replay, collects the stages of the LAST call
 * in the graph (until reset == 2 forgets the captured stages).  Not thread-safe; leave it disabled
 * (the default) in production.
 */
enum {
    QUEST_STAGE_QUANT_X = 0,   /* quantizer launch on x (or the only launch of quest_quantize) */
    QUEST_STAGE_QUANT_W = 1,   /* quantizer launch on w inside quest_linear_fwd */
    QUEST_STAGE_UNPACK = 2,    /* packed codes -> int8 operands (and row sums) */
    QUEST_STAGE_GEMM = 3,      /* the tensor-core contraction with its epilogue */
    QUEST_NUM_STAGES = 4
};
int quest_stage_timing(int enable);
int quest_stage_times(double *total_ms, long long *counts, int reset);

/* Text for a status code; for QUEST_ERR_CUDA, quest_last_cuda_error() has the CUDA message of
 * the most recent failure on the calling thread. */
const char *quest_status_string(int status);
const char *quest_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* QUEST_H_ */
