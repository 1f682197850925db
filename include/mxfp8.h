/*
 * mxfp8.h -- C ABI of the B200 (sm_100a) MXFP8 conversion + block-scaled GEMM library.
 *
 * The operations are those of "Recipes for Pre-training LLMs with MXFP8" (arXiv 2506.08027):
 * conversion of FP32/BF16 tensors to MXFP8 (Sec. 2, Sec. 3.3, Algorithm 1, App. A.1, A.2),
 * along rows and/or columns (Sec. 3.2), decoding (Sec. 2), and the block-scaled matrix
 * product that consumes the result (Sec. 2, App. A.3), optionally re-quantizing its FP32
 * output to MXFP8 (Sec. 2).
 *
 * Conventions shared by every call
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns
 *     every buffer; the library never allocates, frees or keeps a pointer after returning.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream).  Nothing synchronises except mxfp8_device_status() and the *_host calls.
 *     Calls may be made from several host threads and on several streams at once.  The
 *     conversion kernels keep a few words of device state per stream (the first 64 streams
 *     of a device that convert large tensors; later ones, the per-thread default stream and
 *     launches inside a stream capture work without it, a little slower on tensors of
 *     hundreds of megabytes); nothing a caller has to manage.
 *   - Return value: MXFP8_OK or a negative mxfp8_status.  Nothing is printed, nothing aborts.
 *   - Tensors are row-major.  A block is K = 32 consecutive elements (Sec. 2) along a row
 *     (MXFP8_ROW) or down a column (MXFP8_COL).  Quantized data keeps the shape and the
 *     row-major order of the source in both orientations: one byte per element.
 *   - A scale is one UE8M0 byte b meaning X = 2^(b-127); b = 0xFF means NaN (Sec. 2).
 *     mxfp8_quantize never produces 0xFF.
 *
 * Scale layouts (the paper leaves the memory layout of the scales open)
 *   The scales of a tensor form a logical matrix S[mn, kb]: for MXFP8_ROW blocks mn = source
 *   row and kb = column / 32; for MXFP8_COL blocks mn = source column and kb = row / 32.
 *   MXFP8_SF_LINEAR   : ROW -> [rows, cols/32] row-major;  COL -> [rows/32, cols] row-major.
 *   MXFP8_SF_SWIZZLED : what the tensor cores read.  S is cut into atoms of 128 mn x 4 kb
 *                       (512 bytes); atoms are ordered mn-outer, kb-inner; inside an atom the
 *                       byte of (mn, kb) is at (mn%32)*16 + ((mn%128)/32)*4 + kb%4.  mn is
 *                       padded to a multiple of 128 and kb to a multiple of 4; pad bytes are 0.
 *                       See mxfp8_sf_offset().
 */
#ifndef MXFP8_H_
#define MXFP8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MXFP8_OK = 0,
    MXFP8_ERR_NULL = -1,           /* a required pointer is NULL                         */
    MXFP8_ERR_ENUM = -2,           /* an enum argument is out of range                   */
    MXFP8_ERR_SHAPE = -3,          /* non-positive size, or blocked dimension % 32 != 0   */
    MXFP8_ERR_ALIGN = -4,          /* a pointer or a row pitch misses its alignment       */
    MXFP8_ERR_UNSUPPORTED = -5,    /* valid request this build does not implement         */
    MXFP8_ERR_CUDA = -6,           /* a CUDA runtime/driver call or a launch failed       */
    MXFP8_ERR_DEVICE_TIMEOUT = -7, /* a bounded wait inside a kernel ran out              */
    MXFP8_ERR_WORKSPACE = -8,      /* workspace missing or too small                      */
    MXFP8_ERR_DEVICE_ARGS = -9     /* a kernel found invalid values in a device-side argument array */
} mxfp8_status;

enum { MXFP8_FP32 = 0, MXFP8_BF16 = 1 };                 /* source / destination dtype   */
enum { MXFP8_ROW = 1, MXFP8_COL = 2, MXFP8_BOTH = 3 };   /* block orientation (bit mask) */
enum { MXFP8_RULE_PAPER = 0, MXFP8_RULE_OCP = 1 };       /* scale rounding rule          */
/* Element encodings (Table 1).  E4M3 / E5M2 are the MXFP8 elements, one code per byte.  E2M3 / E3M2
 * (MXFP6) and E2M1 (MXFP4) share the block size, the scale type and both scale rules; they have no Inf
 * and no NaN (a NaN input becomes +max, +-Inf becomes +-max).  Their codes are stored the way the tensor
 * cores read them: every 16 consecutive codes of a row share one 16-byte slot, code i in bits
 * [w*i, w*i + w) of the slot taken as a little-endian integer (w = 6 or 4), the other bytes zero.  A
 * [rows, cols] code tensor therefore still has `cols` bytes per row and needs cols % 16 == 0
 * (MXFP8_ERR_UNSUPPORTED otherwise).  Every entry point takes all five, except the fused GEMM output
 * (8-bit elements only).  The values are the tensor cores' own format codes. */
enum { MXFP8_E4M3 = 0, MXFP8_E5M2 = 1, MXFP8_E2M3 = 3, MXFP8_E3M2 = 4, MXFP8_E2M1 = 5 };
enum { MXFP8_SF_LINEAR = 0, MXFP8_SF_SWIZZLED = 1 };     /* scale layout                 */
enum { MXFP8_K_MAJOR = 0, MXFP8_MN_MAJOR = 1 };          /* GEMM operand storage         */

/*
 * mxfp8_quantize -- FP32/BF16 -> MXFP8 (Sec. 3.3, Algorithm 1, App. A.1, A.2; two
 * orientations per Sec. 3.2).
 *
 * Per block of 32: amax = max |V_i| over the finite elements (0 if none); scale byte b by
 *   MXFP8_RULE_PAPER: X = amax/destmax rounded UP to a power of two, at least 2^-127
 *                     (Algorithm 1, App. A.1);  b = log2(X) + 127;
 *   MXFP8_RULE_OCP  : exponent floor(log2 amax) - emax(elem), clamped to [-127, 127]
 *                     (the OCP v1.0 suggestion Sec. 3.3 compares against);
 * then Q_i = V_i / X rounded to nearest-even on the element grid and saturated to +-destmax
 * (448 for E4M3, 57344 for E5M2).  NaN elements stay NaN, +-Inf become +-destmax, and neither
 * enters amax.  FP32 subnormal inputs are honoured (no flush to zero).
 *
 *   src          [rows, cols] row-major, dtype MXFP8_FP32 or MXFP8_BF16, 16-byte aligned.
 *   orientation  MXFP8_ROW (needs cols % 32 == 0), MXFP8_COL (needs rows % 32 == 0) or
 *                MXFP8_BOTH (needs both); BOTH reads src once.
 *   q_row, s_row outputs of the ROW orientation (ignored unless orientation & MXFP8_ROW):
 *                q_row [rows, cols] bytes; s_row mxfp8_scale_bytes(rows, cols, ROW, layout).
 *   q_col, s_col the same for the COL orientation.
 *   q_* must be 16-byte aligned, s_* 16-byte aligned; outputs must not overlap src.
 *   Errors: ERR_NULL, ERR_ENUM, ERR_SHAPE, ERR_ALIGN, ERR_CUDA (launch failure).
 */
int mxfp8_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                   int orientation, int scale_rule, int elem,
                   void* q_row, void* s_row, void* q_col, void* s_col,
                   int sf_layout, void* stream);

/*
 * mxfp8_dequantize -- decoded value Q_i * X (Sec. 2), written as FP32 or BF16 (one RNE
 * rounding of the exact product; overflow gives +-Inf, scale byte 0xFF gives NaN).
 *   q [rows, cols] bytes; s in `sf_layout` for `orientation` (MXFP8_ROW or MXFP8_COL only);
 *   dst [rows, cols] of dst_dtype.  Same alignment rules and errors as mxfp8_quantize.
 */
int mxfp8_dequantize(const void* q, const void* s, int64_t rows, int64_t cols,
                     int orientation, int elem, int sf_layout,
                     void* dst, int dst_dtype, void* stream);

/*
 * mxfp8_quantize_multi -- mxfp8_quantize of up to MXFP8_QUANTIZE_MULTI_MAX tensors in ONE launch.
 * A training step casts several tensors at the same point (Sec. 3.2: activations, weights and
 * gradients each need their MXFP8 copies before the GEMMs that read them); small tensors do not fill
 * the machine alone, and one launch shares the ramp-up and the tail between them.  The results are
 * those of separate mxfp8_quantize calls, bit for bit.  (The batching itself has no counterpart in
 * the paper.)
 *   items   HOST array of `count` entries: source, shape and the outputs the orientation needs
 *           (same meaning, layout and alignment as in mxfp8_quantize; device pointers).
 *   All tensors share src_dtype, orientation, scale_rule, elem and sf_layout.
 *   Every tensor needs cols % 16 == 0 (ERR_UNSUPPORTED otherwise).
 */
#define MXFP8_QUANTIZE_MULTI_MAX 8
typedef struct mxfp8_quantize_item {
    const void* src;
    int64_t rows, cols;
    void* q_row;
    void* s_row;
    void* q_col;
    void* s_col;
} mxfp8_quantize_item;
int mxfp8_quantize_multi(const mxfp8_quantize_item* items, int count, int src_dtype,
                         int orientation, int scale_rule, int elem, int sf_layout, void* stream);

/*
 * mxfp8_act_quantize -- an elementwise activation fused ahead of the conversion.  Sec. 3.2 keeps the
 * activation function in high precision and converts its result for the next GEMM; this call reads
 * the pre-activation once and writes only the MXFP8 copies: y = act(x) evaluated in FP32 and rounded
 * once to the source dtype (BF16 round-to-nearest-even; unchanged for FP32), then exactly
 * mxfp8_quantize(y).  The paper names no particular function; provided are
 *   MXFP8_ACT_RELU       x > 0 ? x : 0            (NaN -> 0)
 *   MXFP8_ACT_RELU2      x > 0 ? x * x : 0
 *   MXFP8_ACT_SILU       x / (1 + exp(-x))
 *   MXFP8_ACT_GELU_TANH  0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
 * The first two are exact FP32 arithmetic (bit-reproducible); the last two use the device's fast FP32
 * exponential and division (relative error of a few 2^-22 before the rounding to the source dtype).
 * Arguments as mxfp8_quantize; needs cols % 16 == 0 (ERR_UNSUPPORTED otherwise).
 */
enum { MXFP8_ACT_NONE = 0, MXFP8_ACT_RELU = 1, MXFP8_ACT_RELU2 = 2, MXFP8_ACT_SILU = 3, MXFP8_ACT_GELU_TANH = 4 };
int mxfp8_act_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int act,
                       int orientation, int scale_rule, int elem,
                       void* q_row, void* s_row, void* q_col, void* s_col,
                       int sf_layout, void* stream);

/*
 * mxfp8_glu_quantize -- a gated activation fused ahead of the conversion: the source is [rows, 2 * cols]
 * with the gate in columns 0 .. cols-1 and the up projection in columns cols .. 2*cols-1 (one tensor,
 * as a fused gate/up GEMM writes it), and
 *     y[r, c] = act(gate[r, c]) * up[r, c]
 * is evaluated in FP32 (act as in mxfp8_act_quantize, then one FP32 product), rounded once to the source
 * dtype, and converted exactly as mxfp8_quantize(y) of the [rows, cols] result (MXFP8_ACT_SILU: SwiGLU,
 * MXFP8_ACT_GELU_TANH: GeGLU, MXFP8_ACT_RELU: ReGLU, MXFP8_ACT_NONE: the bilinear form).  Same place in
 * the recipe as mxfp8_act_quantize (Sec. 3.2).  cols must be a multiple of 128 (BF16 source) or 64 (FP32
 * source) -- MXFP8_ERR_UNSUPPORTED otherwise; other arguments as mxfp8_quantize.
 */
int mxfp8_glu_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols, int act,
                       int orientation, int scale_rule, int elem,
                       void* q_row, void* s_row, void* q_col, void* s_col,
                       int sf_layout, void* stream);

/*
 * mxfp8_act_grad_quantize -- the backward of such an activation ahead of the conversion: dz = act'(z) * dh, the
 * gradient with respect to the activation's input, is an activation gradient and gets converted (Sec. 3.2).
 * `z` (the activation's input saved by the forward pass) and `dh` (the incoming gradient) are device tensors
 * [rows, cols] of `src_dtype`; act is MXFP8_ACT_RELU .. MXFP8_ACT_GELU_TANH.  act'(z) is evaluated in FP32 (relu: 0 or
 * 1; squared relu: 2z or 0; silu and tanh-gelu with the fast FP32 exponential and division), multiplied by dh (one
 * FP32 product), rounded once to the source dtype, then converted exactly like mxfp8_quantize of a tensor holding
 * that value.  One launch; nothing is written besides the MXFP8 outputs; cols a multiple of 16; other arguments,
 * layouts and errors as mxfp8_quantize.
 */
int mxfp8_act_grad_quantize(const void* dh, const void* z, int src_dtype, int64_t rows, int64_t cols, int act,
                            int orientation, int scale_rule, int elem,
                            void* q_row, void* s_row, void* q_col, void* s_col,
                            int sf_layout, void* stream);

/*
 * mxfp8_rmsnorm_quantize -- RMS normalisation fused ahead of the conversion (Sec. 3.2 keeps the
 * normalisation layers in high precision and converts their output for the next GEMM).  Two launches:
 *   rstd[r] = 1 / sqrt(mean_c(x[r, c]^2) + eps)     FP32 accumulation over the row, written to `rstd`
 *                                                    (device, `rows` floats; the backward pass wants it)
 *   y[r, c] = (x[r, c] * rstd[r]) * gamma[c]        two FP32 products in this order, rounded once to the
 *                                                    source dtype, then exactly mxfp8_quantize(y)
 * gamma: device, `cols` values of the source dtype, 16-byte aligned.  eps >= 0.  The sum of squares is
 * accumulated in FP32 in a fixed order (reproducible run to run), so rstd agrees with an FP64 evaluation
 * to FP32 rounding, not bit for bit.  Other arguments as mxfp8_quantize; needs cols % 16 == 0.
 * The source is read twice (statistics, then conversion) and no normalised tensor is written.
 */
int mxfp8_rmsnorm_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                           const void* gamma, float eps, float* rstd,
                           int orientation, int scale_rule, int elem,
                           void* q_row, void* s_row, void* q_col, void* s_col,
                           int sf_layout, void* stream);

/*
 * mxfp8_layernorm_quantize -- the same with a layer normalisation: y = ((x - mean[row]) * rstd[row]) * gamma[col] + beta[col],
 * four FP32 operations in that order (no fused multiply-add), rounded once to the source dtype, then converted.
 * mean[row] and rstd[row] = 1 / sqrt(mean_c (x - mean)^2 + eps) are computed by a statistics launch (FP32 sums in a
 * fixed order of x - pivot and its square, pivot = the row's first element, in one pass over the row; a row whose
 * pivot turns out to lie more than about four standard deviations from the mean is summed a second time around
 * that mean, so an outlier in the first column costs time, not digits) and written to `mean` and `rstd` (device,
 * FP32 [rows]) for the backward pass.  `gamma`, `beta`: device, source dtype, [cols], 16-byte aligned.  Everything else as mxfp8_rmsnorm_quantize.
 * (Sec. 3.2 keeps normalisation in high precision and converts its output; the paper names no particular one.)
 */
int mxfp8_layernorm_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                             const void* gamma, const void* beta, float eps, float* mean, float* rstd,
                             int orientation, int scale_rule, int elem,
                             void* q_row, void* s_row, void* q_col, void* s_col,
                             int sf_layout, void* stream);

/*
 * mxfp8_rmsnorm_quantize_static -- mxfp8_rmsnorm_quantize for callers that do not want the row
 * statistics and have no buffer to lend: the statistics go to a fixed array inside the library
 * (file-scope device memory, 65536 rows x 4 bytes = 256 KB, part of the module image), so the call
 * takes no scratch from the caller and allocates nothing, on the host or on the device.  It is meant
 * for callers that cannot call cudaMalloc where they stand: code inside a stream capture, a real-time
 * loop that must not take the allocator's lock, a plugin that was handed its buffers and nothing else.
 * The array used is the one of the device that is current on the calling thread (every device that
 * loads the library holds its own copy until the process ends); its address is looked up on the first
 * call on that device, so make that first call before any stream capture begins.
 * Errors: those of mxfp8_rmsnorm_quantize, checked in the same order, and after them
 * MXFP8_ERR_UNSUPPORTED for more than mxfp8_rmsnorm_quantize_static_max_rows() rows (nothing is launched).
 * The array is shared by all calls on a device and keeps the last call's statistics: every call
 * overwrites the rows it uses before it reads them, and calls that overlap on the GPU (two streams,
 * two threads) race on it -- order them on one stream.
 * Results are those of mxfp8_rmsnorm_quantize.  (A packaging for convenience: the paper has no
 * counterpart.)
 */
int64_t mxfp8_rmsnorm_quantize_static_max_rows(void);
int mxfp8_rmsnorm_quantize_static(const void* src, int src_dtype, int64_t rows, int64_t cols,
                                  const void* gamma, float eps,
                                  int orientation, int scale_rule, int elem,
                                  void* q_row, void* s_row, void* q_col, void* s_col,
                                  int sf_layout, void* stream);

/*
 * mxfp8_fake_quantize -- the MXFP8 round trip in one pass: dst = decode(quantize(src)) in the source's
 * own dtype (BF16 -> MXFP8 -> BF16 is how the paper's accuracy runs emulated MX arithmetic ahead of
 * BF16 GEMMs, Sec. 3.1).  Same block / scale / cast rules and the same special-value handling as
 * mxfp8_quantize; the result equals mxfp8_dequantize(mxfp8_quantize(src)) bit for bit.
 *   dst_row / dst_col  [rows, cols] of src_dtype, one per requested orientation, 16-byte aligned.
 *   Needs cols % 16 == 0 (ERR_UNSUPPORTED otherwise) besides the rules of mxfp8_quantize.
 */
int mxfp8_fake_quantize(const void* src, int src_dtype, int64_t rows, int64_t cols,
                        int orientation, int scale_rule, int elem,
                        void* dst_row, void* dst_col, void* stream);

/*
 * Optional fused epilogue of mxfp8_gemm: the FP32 accumulator tile is converted to MXFP8
 * exactly as mxfp8_quantize would convert the FP32 output D[M, N] (Sec. 2: the FP32 output is
 * quantized to MX format when its consumer needs it).  ROW blocks run along N, COL blocks
 * along M.  Scales are written in MXFP8_SF_SWIZZLED layout.
 */
typedef struct {
    int orientation;   /* MXFP8_ROW, MXFP8_COL or MXFP8_BOTH */
    int scale_rule;
    int elem;
    void* q_row;       /* [M, N] bytes */
    void* s_row;       /* mxfp8_scale_bytes(M, N, MXFP8_ROW, MXFP8_SF_SWIZZLED) */
    void* q_col;
    void* s_col;       /* mxfp8_scale_bytes(M, N, MXFP8_COL, MXFP8_SF_SWIZZLED) */
} mxfp8_epilogue;

/*
 * mxfp8_gemm -- block-scaled product on the tensor cores (Sec. 2, App. A.3):
 *     D[m, n] = sum over K-blocks kb of  2^(sa[m,kb]-127) * 2^(sb[n,kb]-127)
 *                                        * sum_{k in kb} Aq[m,k] * Bq[n,k],
 * accumulated in FP32.  A is logically [M, K], B logically [N, K].
 *   a_major / b_major  MXFP8_K_MAJOR : stored [MN, K] row-major, quantized with ROW blocks;
 *                      MXFP8_MN_MAJOR: stored [K, MN] row-major, quantized with COL blocks
 *                      (blocks run down K).  fprop = (K,K), dgrad = (K,MN), wgrad = (MN,MN).
 *   As, Bs             scales in MXFP8_SF_SWIZZLED layout, logically [MN, K/32] in both cases
 *                      -- exactly what mxfp8_quantize writes for the matching orientation.
 *   D                  [M, N] row-major, out_dtype MXFP8_FP32 or MXFP8_BF16 (RNE); may be NULL
 *                      when `epi` is given and only the quantized output is wanted.
 *   epi                NULL, or the fused MXFP8 output described above.
 *   workspace          device scratch of at least mxfp8_gemm_workspace_bytes(); may be NULL
 *                      when that is 0.  Contents are undefined afterwards.
 * Requirements: K % 32 == 0 (else ERR_SHAPE).  Ragged M, N and K (not multiples of the tile) are
 * handled by the hardware's out-of-bounds fill and clipping; what remains are the 16-byte row
 * pitches TMA needs: M % 16 == 0 for an MN-major A, N % 16 == 0 for an MN-major B, N % 8 == 0 for
 * BF16 output, N % 4 == 0 for FP32 output; with `epi`, M % 128 == 0 and N % 128 == 0
 * (ERR_UNSUPPORTED otherwise).  All pointers 16-byte aligned.
 * A bounded wait that expires inside the kernel sets the device status word; read it with
 * mxfp8_device_status().  The result is deterministic (same inputs, same bytes).
 */
int mxfp8_gemm(const void* Aq, const void* As, const void* Bq, const void* Bs,
               int64_t M, int64_t N, int64_t K,
               int a_major, int b_major, int a_elem, int b_elem,
               void* D, int out_dtype, const mxfp8_epilogue* epi,
               void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of the scale buffer of a [rows, cols] tensor for one orientation (ROW or COL). */
size_t mxfp8_scale_bytes(int64_t rows, int64_t cols, int orientation, int sf_layout);

/* Byte offset of scale (mn, kblock) in a scale buffer with n_kblocks K-blocks per mn and
 * (for LINEAR/COL only) mn_count columns.  LINEAR: ROW uses mn*n_kblocks + kblock; a COL
 * buffer is addressed by the caller as kblock*mn_count + mn and is not handled here.
 * SWIZZLED: the 128x4 atom formula in the header comment.  Host helper, no device work. */
int64_t mxfp8_sf_offset(int64_t mn, int64_t kblock, int64_t n_kblocks, int sf_layout);

/*
 * mxfp8_gemm_multi -- up to 3 independent block-scaled products in ONE launch.  FPROP, DGRAD and WGRAD of
 * a layer (Sec. 3.2) are independent once the MXFP8 copies exist; dealt out as one pool of tiles they fill
 * the machine evenly where each alone would end on a partly idle wave.  Every product follows
 * mxfp8_gemm's definition, argument rules and tolerance (no fused MXFP8 output here); the outputs share
 * `out_dtype`.  `problems`: HOST array of `count` entries with device pointers; outputs must not
 * overlap each other or any operand.  (The batching itself has no counterpart in the paper.)
 */
typedef struct mxfp8_gemm_problem {
    const void* Aq;
    const void* As;
    const void* Bq;
    const void* Bs;
    int64_t M, N, K;
    int a_major, b_major, a_elem, b_elem;
    void* D;
} mxfp8_gemm_problem;
int mxfp8_gemm_multi(const mxfp8_gemm_problem* problems, int count, int out_dtype, void* stream);

/*
 * mxfp8_grouped_gemm -- the per-expert products of a mixture-of-experts layer in one launch (App. A.4
 * trains a mixture-of-experts model with the same recipe; each expert's FPROP / DGRAD / WGRAD is the
 * block-scaled product of Sec. 2 restricted to the tokens routed to that expert).
 *
 * Tokens are sorted by expert; group_offsets (DEVICE pointer, num_groups + 1 int32 values, 4-byte
 * aligned) gives the first token of every expert and the end of the last: non-negative,
 * non-decreasing, multiples of 128, at most the token count.  The kernel reads and checks them
 * on the device (no host synchronisation); a violation makes the launch store nothing and leaves
 * MXFP8_ERR_DEVICE_ARGS in the device status word.  Rows before group_offsets[0] and from
 * group_offsets[num_groups] on belong to no expert and are left untouched (GROUP_M) / unused (GROUP_K).
 *
 * mode MXFP8_GROUP_M (FPROP, DGRAD): M = tokens.
 *     Aq [M, K] K-major with ROW blocks, As its swizzled scales (logical [M, K/32]).
 *     B = the experts' matrices stacked, quantized as ONE tensor by mxfp8_quantize:
 *         b_major K:  Bq [G*N, K], ROW blocks, scales logical [G*N, K/32]   (expert g = rows g*N ..)
 *         b_major MN: Bq [G*K, N], COL blocks, scales logical [N, G*K/32]   (expert g = rows g*K ..)
 *     D [M, N]: row t = A[t, :] . B_g^T for the expert g that owns token t.
 * mode MXFP8_GROUP_K (WGRAD): K = tokens; b_major must be MN.
 *     Aq [K, M] and Bq [K, N], both with COL blocks (blocks run down the token axis), scales
 *     logical [M, K/32] and [N, K/32].
 *     D [G*M, N]: rows g*M .. = A_g^T . B_g summed over expert g's tokens; zeros for an expert
 *     without tokens.
 * M, N, K multiples of 128; num_groups <= 256; element formats and output dtype as mxfp8_gemm;
 * FP32 accumulation; all pointers device, 16-byte aligned; nothing is allocated.
 */
enum { MXFP8_GROUP_M = 1, MXFP8_GROUP_K = 2 };
int mxfp8_grouped_gemm(const void* Aq, const void* As, const void* Bq, const void* Bs,
                       const int32_t* group_offsets, int num_groups, int mode,
                       int64_t M, int64_t N, int64_t K, int b_major, int a_elem, int b_elem,
                       void* D, int out_dtype, void* stream);

/*
 * Data-parallel exchange.  The recipe casts weights, activations and output gradients (Sec. 3.2); when
 * the tokens of a step are split over GPUs and every GPU owns a row range of each weight, two exchanges
 * follow from that arithmetic: the MXFP8 copies of the weight shards are gathered (1 + 1/32 bytes per
 * element and orientation instead of 2 for BF16), and the WGRAD partial results, one per GPU over its
 * own tokens, are summed and scattered to the owners of the rows.  (The paper states no multi-GPU
 * algorithm; these two calls are what its per-tensor arithmetic needs when the tensors are sharded.)
 *
 * mxfp8_sf_concat_k -- joins swizzled scale arrays along the block axis.  `parts` holds `num_parts`
 * swizzled arrays one after another, each for logical [mn, k_part/32] scales (k_part a multiple of 128,
 * so every part is whole 512-byte atoms); `dst` receives the swizzled array for logical
 * [mn, num_parts * k_part/32], part r supplying blocks r*k_part/32 .. .  This is what the column-blocked
 * scales of row-sharded weights need after an all-gather (blocks run down the sharded axis); the element
 * bytes of both orientations and the row-blocked scales of row shards are already in place when
 * each shard is written at its row offset.  Device pointers, 16-byte aligned; one launch; a pure permutation of bytes.
 *
 * mxfp8_gemm_reduce_scatter -- D_owner[r][m - r*M/num_owners, n] += sum_k A[m,k] * B[n,k] for every m:
 * the block-scaled product of mxfp8_gemm (operands as there) whose FP32 result is ADDED, tile by tile
 * while the product runs, into one FP32 buffer [M/num_owners, N] per owner of a row range.  `D_owner`
 * is a HOST array of `num_owners` (1..8) device pointers; a pointer may be another GPU's memory mapped
 * into this process (peer access or an IPC mapping): the additions then cross NVLink as they are produced.
 * `first_owner` (0 .. num_owners-1) is the owner whose tiles this launch produces first; giving each
 * rank its own index spreads the traffic over the owners.  The caller zeroes the buffers, makes sure every rank has done so before any
 * rank launches, and waits for all ranks' launches before reading its own buffer; the order in
 * which different launches' contributions are added is not fixed (two contributions: exact and order-free;
 * more: equal up to FP32 rounding order).  M a multiple of 128 * num_owners, N of 4 (16 with an MN-major B), K of 32.
 * Nothing is allocated; never waits on another GPU inside the kernel.  With num_owners = 1 and a local buffer the
 * call is a product that accumulates into an FP32 output (D += A * B^T): WGRAD summed over micro-batches.
 */
/* Lets kernels launched on the current device read and write memory of `peer_device` (needed once per pair of
 * devices before a pointer into the peer's memory is given to mxfp8_gemm_reduce_scatter).  MXFP8_OK when access
 * is, or already was, enabled or the peer is the current device; MXFP8_ERR_SHAPE for a device that does not
 * exist; MXFP8_ERR_UNSUPPORTED when the two devices have no peer path.  Changes this process's context only. */
int mxfp8_enable_peer_access(int peer_device);
int mxfp8_sf_concat_k(const void* parts, int num_parts, int64_t mn, int64_t k_part, void* dst, void* stream);
#define MXFP8_REDUCE_SCATTER_MAX_OWNERS 8
int mxfp8_gemm_reduce_scatter(const void* Aq, const void* As, const void* Bq, const void* Bs,
                              int64_t M, int64_t N, int64_t K,
                              int a_major, int b_major, int a_elem, int b_elem,
                              void* const* D_owner, int num_owners, int first_owner, void* stream);

/* Scratch bytes mxfp8_gemm needs for this problem (0 when none). */
size_t mxfp8_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int out_dtype, int has_epilogue);

/* Waits for `stream`, then returns and clears the device status word of the current device:
 * MXFP8_OK, MXFP8_ERR_DEVICE_TIMEOUT, MXFP8_ERR_DEVICE_ARGS, or MXFP8_ERR_CUDA if the wait itself failed.
 * This is the only device-pointer call that synchronises. */
int mxfp8_device_status(void* stream);

/* Measurement aid (no counterpart in the paper): waits for `stream`, then reports the SM clock that the most recent
 * GEMM launch of this library on the current device really ran at -- SM cycles divided by wall nanoseconds, both read
 * by the kernel's first CTA at its start and end -- and that CTA's lifetime in microseconds.  A sampled
 * driver clock cannot resolve a kernel of a few hundred microseconds; this can, and shows a power-capped run. */
int mxfp8_gemm_last_clock(void* stream, double* sm_mhz, double* kernel_us);

/* Human-readable name of a status code (static string). */
const char* mxfp8_status_string(int status);

/* Number of kernels this library has launched in this process (for launch accounting). */
int64_t mxfp8_launch_count(void);

/*
 * Host-buffer variants: the same operations with HOST pointers for inputs and outputs.  The
 * caller provides a device staging buffer `dev_ws` of at least the returned *_host_ws_bytes;
 * the call copies inputs host->device, runs the device path, copies results device->host,
 * all on `stream`, and waits for the stream before returning.  Host buffers should be pinned
 * for full PCIe bandwidth.  (No counterpart in the paper; provided for end-to-end use.)
 */
size_t mxfp8_quantize_host_ws_bytes(int src_dtype, int64_t rows, int64_t cols, int orientation);
int mxfp8_quantize_host(const void* src_host, int src_dtype, int64_t rows, int64_t cols,
                        int orientation, int scale_rule, int elem,
                        void* q_row_host, void* s_row_host, void* q_col_host, void* s_col_host,
                        int sf_layout, void* dev_ws, size_t dev_ws_bytes, void* stream);


/*
 * mxfp8_linear -- one training step of a linear layer Y = X * W^T through the MXFP8 path on
 * DEVICE buffers (Sec. 3.2, the FPROP / DGRAD / WGRAD workflow): X [T, H], W [F, H], dY [T, F]
 * in BF16 are each converted once to MXFP8-E4M3 in BOTH orientations under `scale_rule`, then
 *     FPROP  Y  [T, F] = X  * W^T   (row-blocked X,  row-blocked W)
 *     DGRAD  dX [T, H] = dY * W     (row-blocked dY, column-blocked W)
 *     WGRAD  dW [F, H] = dY^T * X   (column-blocked dY, column-blocked X)
 * run as block-scaled GEMMs with BF16 output (the call only enqueues work: it can be captured in a CUDA
 * graph and replayed): two kernel launches on `stream` (the three casts
 * share one, the three GEMMs share one), no wait.  Y, dX, dW must not overlap.
 * T, H, F must be multiples of 128 (ERR_UNSUPPORTED).  ws: device scratch for the quantized
 * copies, mxfp8_linear_ws_bytes() bytes, 256-byte aligned, owned by the caller.  All tensors
 * 16-byte aligned, row-major, dense.
 */
size_t mxfp8_linear_ws_bytes(int64_t T, int64_t H, int64_t F);
int mxfp8_linear(const void* x, const void* w, const void* dy,
                 int64_t T, int64_t H, int64_t F, int scale_rule,
                 void* y, void* dx, void* dw, void* ws, size_t ws_bytes, void* stream);

/*
 * mxfp8_linear_host -- one training step of a linear layer Y = X * W^T through the MXFP8 path
 * (Sec. 3.2, the FPROP / DGRAD / WGRAD workflow), with HOST inputs and outputs:
 *   X [T, H], W [F, H], dY [T, F] in BF16 (host) are copied to the device, each is converted
 *   once to MXFP8-E4M3 in BOTH orientations under `scale_rule`, then
 *     FPROP  Y  [T, F] = X  * W^T   (row-blocked X,  row-blocked W)
 *     DGRAD  dX [T, H] = dY * W     (row-blocked dY, column-blocked W)
 *     WGRAD  dW [F, H] = dY^T * X   (column-blocked dY, column-blocked X)
 *   run as block-scaled GEMMs with BF16 output, and Y, dX, dW are copied back to the host.
 * T, H, F must be multiples of 128.  dev_ws: device scratch of mxfp8_linear_host_ws_bytes(),
 * 256-byte aligned.  Waits for `stream` before returning.  The token axis goes through in four row
 * chunks when T is a multiple of 512, so that uploads, products and downloads overlap (two helper
 * streams per device, created on first use, ordered after the work already in `stream`): FPROP and
 * DGRAD run per chunk, the column-blocked copies and WGRAD once everything is there; same results as
 * mxfp8_linear, bit for bit.  (The composition is the paper's
 * workflow; the host-buffer packaging has no counterpart in the paper.)
 */
size_t mxfp8_linear_host_ws_bytes(int64_t T, int64_t H, int64_t F);
int mxfp8_linear_host(const void* x_host, const void* w_host, const void* dy_host,
                      int64_t T, int64_t H, int64_t F, int scale_rule,
                      void* y_host, void* dx_host, void* dw_host,
                      void* dev_ws, size_t dev_ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MXFP8_H_ */
