/*
 * nq.h -- C boundary of the B200 (sm_100a) NestQuant hot path.
 *
 * NestQuant ("Post-Training Integer-Nesting Quantization for On-Device DNN") stores an INTn
 * quantised weight as two integers, w_int = w_high * 2^l + w_low with n = h + l (Eq. 5), so that a
 * model can run "part-bit" on w_high alone (scale inflated to s * 2^l, Eq. 9) and be upgraded to
 * the "full-bit" INTn model by paging w_low back in and recomposing.  This library is the
 * data-parallel part of that: decomposition, recomposition, dropping the low part, and the integer
 * GEMM / convolution on the nested weights in both modes.
 *
 * General rules for every entry point
 *   - Pointers marked (device) are device memory of the current CUDA device, owned by the caller and
 *     alive until the work queued on `stream` has finished.  Pointers marked (host) are read before
 *     the call returns.  The library allocates no device memory.
 *   - `stream` is a cudaStream_t passed as void* (0 = the default stream).  Calls only enqueue work
 *     and return; they never synchronise, except nq_device_status.
 *   - Return value: NQ_OK or an nq_status error.  Argument errors are found before anything is
 *     launched.  Nothing aborts, traps or throws.
 *   - Weight matrices are [rows, cols] = [output channels, K] with K contiguous.
 *   - Nesting parameters: n_bits in [2, 8]; h_bits in [1, n_bits - 1]; l = n_bits - h_bits;
 *     compensate != 0 keeps w_low in l + 1 bits ("Full-Bit Model: Performance Compensation"),
 *     compensate == 0 clips it to l bits (Eq. 10).  Unpacked weights are int8 holding INTn values;
 *     for n_bits < 8 values outside [-2^(n-1), 2^(n-1) - 1] give unspecified results.
 *
 * Packed ("sliced") layout of a [rows, cols] tensor of k-bit two's-complement fields
 *   The tensor is padded with zero fields to multiples of 128 rows and 128 columns and cut into blocks of
 *   128 rows x 128 columns.  A block is 2048*k contiguous bytes; block (rb, g) -- row block rb, column group g
 *   of G = ceil(cols / 128) -- is block number rb*G + g.  The whole tensor takes nq_packed_bytes(rows, cols, k)
 *   = (rows padded to 128) * nq_packed_row_bytes(cols, k) bytes.
 *   k is split into powers of two (8, 4, 2, 1), widest first; the slice of width s holds s bits of every field
 *   (the widest slice the most significant bits) and takes 2048*s bytes of the block: the block's 128 rows one
 *   after the other, 16*s bytes each.  In a row's 16*s bytes, element e (= column % 128) lives in byte
 *   ((e/32)*s + ((e%32)/4) / (8/s)) * 4 + e%4, at bits [8 - s*(sub+1), 8 - s*sub) with sub = ((e%32)/4) % (8/s).
 *   (The paper only fixes the field width and its two's-complement content.  This placement lets four fields be
 *   extracted with one mask per 32-bit word, and makes the 128 rows x 128 columns that one thread block of the
 *   GEMM consumes per step one contiguous run of memory.)  The base address of a packed tensor must be 16-byte
 *   aligned.  Kernels that write a packed tensor write its padding as zero fields; kernels that read one never
 *   depend on the padding's content.
 */
#ifndef NQ_H_
#define NQ_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define NQ_API __attribute__((visibility("default")))
#else
#define NQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NQ_OK = 0,
    NQ_ERR_INVALID_ARG = 1, /* null pointer, negative size, inconsistent shapes                 */
    NQ_ERR_UNSUPPORTED = 2, /* nesting (n, h) or shape outside what the kernels implement        */
    NQ_ERR_ALIGNMENT = 3,   /* a pointer or pitch breaks the stated alignment rule               */
    NQ_ERR_WORKSPACE = 4,   /* workspace missing or too small                                    */
    NQ_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed (launch, descriptor encoding) */
    NQ_ERR_TIMEOUT = 6      /* a bounded on-device wait expired (reported by nq_device_status)   */
} nq_status;

typedef enum { NQ_F32 = 0, NQ_BF16 = 1 } nq_dtype;

/* Text for a status code (host, static storage). */
NQ_API const char *nq_status_str(int status);

/* Bits of the stored low field: l + 1 with compensation, l without.  Returns -1 for a bad (n, h). */
NQ_API int nq_low_bits(int n_bits, int h_bits, int compensate);

/* Bytes per row of the padded tensor (a size unit: 16 * bits per 128 columns; a row's bytes are not contiguous) and
 * size of a whole packed tensor in bytes, rows padded to a multiple of 128 (host, pure).  -1 on bad arguments. */
NQ_API int64_t nq_packed_row_bytes(int64_t cols, int bits);
NQ_API int64_t nq_packed_bytes(int64_t rows, int64_t cols, int bits);

/*
 * Decomposition -- Eq. 5, Eq. 6, Algorithm 1 step 2, Eq. 10 and the compensation subsection.
 * Per element: w_high = clip(round(w_int / 2^l)) to INTh, where the rounding is DOWN (the
 * RightShift of Eq. 6) where mask == 0 and UP where mask != 0 (an exact multiple of 2^l is left
 * alone); w_low = w_int - w_high * 2^l, clipped to l bits when compensate == 0.
 *   w_int (device)  int8 [rows, cols], row pitch ld_w elements (>= cols)
 *   mask  (device)  uint8 [rows, cols], same pitch: the given adaptive-rounding decision
 *   packed_high, packed_low (device, out)  sliced tensors of h_bits and nq_low_bits() bits
 * Fast path when w_int, mask are 16-byte aligned and ld_w is a multiple of 16; otherwise a slower
 * byte-wise path is taken (same results).
 */
NQ_API int nq_decompose(const int8_t *w_int, const uint8_t *mask, int64_t rows, int64_t cols, int64_t ld_w,
                 int n_bits, int h_bits, int compensate,
                 void *packed_high, void *packed_low, void *stream);

/*
 * Rounding masks of the baselines NestQuant is compared with ("Higher-Bit Weights: Integer Data Optimization" and
 * its ablation; the rows of the "Nesting Numerical Errors" table): for nq_decompose's `mask` argument when no
 * adaptive-rounding optimiser supplies one.
 *   NQ_ROUND_DOWN     BitShift: always the floor (mask 0 everywhere)
 *   NQ_ROUND_UP       always the ceiling (mask 1 everywhere; nq_decompose leaves exact multiples of 2^l alone)
 *   NQ_ROUND_NEAREST  RTN: the nearer neighbour of w_int / 2^l, a tie going to the even one
 *   w_int (device) int8 [rows, cols] pitch ld_w;  mask_out (device, out) uint8 0 / 1, [rows, cols] pitch ld_mask
 */
enum { NQ_ROUND_DOWN = 0, NQ_ROUND_UP = 1, NQ_ROUND_NEAREST = 2 };
NQ_API int nq_rounding_mask(const int8_t *w_int, int64_t ld_w, int64_t rows, int64_t cols, int n_bits, int h_bits,
                     int mode, uint8_t *mask_out, int64_t ld_mask, void *stream);

/*
 * Recomposition / page-in -- Eq. 5 read as the upgrade of "Nesting Mechanism of Decomposed
 * Weights": w_int = clip_INTn(w_high * 2^l + w_low), a shift and an ADD of the sign-extended low
 * field.  Output int8 [rows, cols] with row pitch ld_out elements (device, out).
 */
NQ_API int nq_recompose(const void *packed_high, const void *packed_low, int64_t rows, int64_t cols,
                 int n_bits, int h_bits, int compensate,
                 int8_t *w_int_out, int64_t ld_out, void *stream);

/*
 * Drop-low / page-out -- the downgrade of the same subsection.  The full-bit resident state is
 * {w_int, packed_low}; this derives packed_high = (w_int - w_low) / 2^l from it (no mask needed),
 * after which the caller may free w_int and packed_low.
 */
NQ_API int nq_drop_low(const int8_t *w_int, int64_t ld_w, const void *packed_low, int64_t rows, int64_t cols,
                int n_bits, int h_bits, int compensate,
                void *packed_high_out, void *stream);

/* Test aids: a sliced tensor of `bits`-bit fields <-> sign-extended int8 values. */
NQ_API int nq_unpack(const void *packed, int bits, int64_t rows, int64_t cols,
              int8_t *out, int64_t ld_out, void *stream);
NQ_API int nq_pack(const int8_t *values, int64_t ld, int bits, int64_t rows, int64_t cols,
            void *packed_out, void *stream);

/*
 * The paper's packed-bit tensor ("Deployment": nested weights are stored as packed-bit tensors in unsigned
 * INT64 words, e.g. twenty-one 3-bit or twelve 5-bit weights per word) and conversion to and from the sliced
 * layout, on the device.  A [rows, cols] tensor of k-bit fields takes nq_word64_row_words(cols, k) words per
 * row, rows dense; word w of a row holds the fields of elements w * (64 / k) ... in order, field j at bits
 * [j * k, j * k + k), two's complement, unused top bits and fields past `cols` zero.  (The paper fixes the count
 * per word; the order of the fields inside a word is this library's reading.)
 *   words (device)  uint64, 8-byte aligned;  packed (device)  sliced tensor, 16-byte aligned
 * nq_word64_row_words returns -1 on bad arguments.
 */
NQ_API int64_t nq_word64_row_words(int64_t cols, int bits);
NQ_API int nq_word64_to_sliced(const uint64_t *words, int bits, int64_t rows, int64_t cols, void *packed_out, void *stream);
NQ_API int nq_sliced_to_word64(const void *packed, int bits, int64_t rows, int64_t cols, uint64_t *words_out, void *stream);

/*
 * Whole-model page-in / page-out in ONE launch.  A model is a list of tensors; the caller builds
 * the list once with nq_batch_plan and then switches the model with a single call.
 *   descs (host)   count entries
 *   table (device) at least nq_batch_table_bytes(descs, count) bytes, 16-byte aligned; filled by
 *                  nq_batch_plan with a copy queued on `stream`.  It lists the tensors and cuts the model
 *                  into work items (one thread block each) that never straddle two tensors.
 *   work_items     the number of work items nq_batch_plan reports; pass it back to the batched calls
 * Every tensor of a batch shares (n_bits, h_bits, compensate).  w_int must be 16-byte aligned with
 * ld a multiple of 16 for every tensor of a batch (NQ_ERR_ALIGNMENT otherwise).
 */
typedef struct {
    int64_t rows, cols, ld;   /* ld: row pitch of w_int in elements */
    void *packed_high;        /* (device) */
    void *packed_low;         /* (device) */
    int8_t *w_int;            /* (device) */
} nq_tensor_desc;

NQ_API int64_t nq_batch_table_bytes(const nq_tensor_desc *descs, int count);
NQ_API int nq_batch_plan(const nq_tensor_desc *descs, int count, void *table, int64_t table_bytes,
                  int64_t *work_items_out, void *stream);
NQ_API int nq_recompose_batched(const void *table, int count, int64_t work_items,
                         int n_bits, int h_bits, int compensate, void *stream);
NQ_API int nq_drop_low_batched(const void *table, int count, int64_t work_items,
                        int n_bits, int h_bits, int compensate, void *stream);

/*
 * Full-bit GEMM -- the integer layer on the recomposed weights with the dequantisation of Eq. 2:
 *   acc[m, j] = sum_k X[m, k] * W[j, k]                       (int32, exact)
 *   Y[m, j]   = fl(float(acc[m, j]) * fl(act_scale * w_scale[j]))  (+ bias[j], one more rounding)
 *   X (device) int8 [M, K] pitch ldx;  W (device) int8 [N, K] pitch ldw;  both 16-byte aligned with
 *   pitches that are multiples of 16.  w_scale (device) fp32 [N]; bias (device) fp32 [N] or NULL.
 *   acc_out (device, out) int32 [M, N] pitch ld_acc, or NULL.  Y (device, out) [M, N] pitch ldy of
 *   y_dtype, or NULL.  At least one of acc_out, Y must be given.  Outputs whose base address and row pitch
 *   (in bytes) are multiples of 16 are written with TMA tile stores; any other element-aligned output takes a
 *   slower path with ordinary stores (same results).  K < 2^17 so that the int32 accumulator cannot overflow.
 */
NQ_API int nq_gemm_full(const int8_t *X, int64_t ldx, const int8_t *W, int64_t ldw,
                 const float *w_scale, float act_scale, const float *bias,
                 int64_t M, int64_t N, int64_t K,
                 int32_t *acc_out, int64_t ld_acc, void *Y, int64_t ldy, int y_dtype, void *stream);

/*
 * Part-bit GEMM -- the same layer on w_high alone, unpacked from the sliced tensor inside the
 * kernel, with the inflated scale of Eq. 9:
 *   acc[m, j] = sum_k X[m, k] * w_high[j, k];   Y = fl(float(acc) * fl(fl(act_scale*w_scale[j]) * 2^l))
 *   packed_high (device) sliced [N, K] tensor of h_bits fields, h_bits in [2, 7] here.
 */
NQ_API int nq_gemm_part(const int8_t *X, int64_t ldx, const void *packed_high, int n_bits, int h_bits,
                 const float *w_scale, float act_scale, const float *bias,
                 int64_t M, int64_t N, int64_t K,
                 int32_t *acc_out, int64_t ld_acc, void *Y, int64_t ldy, int y_dtype, void *stream);

/*
 * Nested full-bit GEMM -- the full-bit layer computed straight from the two stored parts, with no INT8 copy of
 * the weights in memory: the kernel rebuilds w_int = w_high * 2^l + w_low (Eq. 5) in shared memory while it
 * unpacks.  A model then occupies (n + 1) / 8 bytes per weight in full-bit mode and h / 8 in part-bit mode, and
 * the upgrade is the arrival of w_low alone, the byte model of the paper's switching-overhead analysis.
 *   acc, Y      exactly those of nq_gemm_full on the tensor nq_recompose would write
 *   packed_high (device) sliced [N, K] tensor of h_bits fields
 *   packed_low  (device) sliced [N, K] tensor of (n_bits - h_bits + 1)-bit fields: the COMPENSATED lower-bit
 *               weights, as nq_decompose writes them with compensate != 0.  For such a pair Eq. 5 is exact and
 *               stays inside INTn; for other field values the sum wraps modulo 2^n instead of being clipped.
 *   n_bits 8 with h_bits in [2, 7], or n_bits 6 with h_bits in [2, 5]; anything else NQ_ERR_UNSUPPORTED.
 *   The other arguments are those of nq_gemm_full.
 */
NQ_API int nq_gemm_nested(const int8_t *X, int64_t ldx, const void *packed_high, const void *packed_low,
                   int n_bits, int h_bits, const float *w_scale, float act_scale, const float *bias,
                   int64_t M, int64_t N, int64_t K,
                   int32_t *acc_out, int64_t ld_acc, void *Y, int64_t ldy, int y_dtype, void *stream);

/*
 * Implicit-GEMM convolution on the nested weights, zero padding (the zero-point is 0):
 *   acc[b, p, q, co] = sum_{r, s, ci} x[b, p*stride - pad + r, q*stride - pad + s, ci] * w[co, r, s, ci]
 *   Y = dequantisation as in nq_gemm_full (part_bit == 0) or nq_gemm_part (part_bit != 0).
 *   X (device) int8, NHWC [B, H, W, Cin] when x_nchw == 0, NCHW [B, Cin, H, W] when x_nchw != 0 (then
 *     a transposing pre-pass writes an NHWC copy into the workspace).
 *   Wt (device) weights as a [Cout, K] matrix with K = R*S*Cin in (r, s, ci) order (OHWI):
 *     int8 with row pitch ldw (a multiple of 16, >= K) when part_bit == 0, the sliced h_bits tensor
 *     of that matrix when part_bit != 0 (ldw ignored).
 *   acc_out / Y: NHWC, i.e. the [M = B*Ho*Wo, N = Cout] matrix, dense.
 *   workspace (device): nq_conv_workspace_bytes(desc) bytes, 1024-byte aligned.
 */
typedef struct {
    int32_t B, Cin, H, W, Cout, R, S, stride, pad;
    int32_t x_nchw;
} nq_conv_desc;

NQ_API int64_t nq_conv_workspace_bytes(const nq_conv_desc *desc);
NQ_API int nq_conv_implicit_gemm(const int8_t *X, const void *Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                          const nq_conv_desc *desc, const float *w_scale, float act_scale,
                          const float *bias, int32_t *acc_out, void *Y, int y_dtype,
                          void *workspace, int64_t workspace_bytes, void *stream);

/*
 * The convolution in nested full-bit mode: nq_conv_implicit_gemm's result for part_bit == 0 on the tensor
 * nq_recompose would write, computed from the two packed parts as in nq_gemm_nested (same operands, same limits
 * on n_bits / h_bits; both are sliced tensors of the [Cout, K] weight matrix in (r, s, ci) order).
 */
NQ_API int nq_conv_implicit_gemm_nested(const int8_t *X, const void *packed_high, const void *packed_low,
                                 int n_bits, int h_bits, const nq_conv_desc *desc, const float *w_scale,
                                 float act_scale, const float *bias, int32_t *acc_out, void *Y, int y_dtype,
                                 void *workspace, int64_t workspace_bytes, void *stream);

/*
 * The same three layers with a requantising epilogue: the output is the next layer's INT8 activations, so layers
 * can be chained on the device and the output traffic is a quarter of fp32.  The paper quantises activations to
 * 8 bits with the uniform quantiser of Eq. 1 (zero-point 0) but does not say how one layer's output becomes the
 * next layer's input; this is the library's own definition (fp32, one rounding per operation):
 *   v = the dequantised value of nq_gemm_full / nq_gemm_part (+ bias[j])
 *   v = max(v, 0)                                   when relu != 0
 *   q = clip(round_half_even(fl(v * fl(1 / out_scale))), -128, 127)
 *   Yq (device, out) int8 [M, N] pitch ldyq (convolution: NHWC, dense).  out_scale > 0 is the activation scale of
 *   the next layer (its act_scale).  The other arguments are those of the fp32 / bf16 entry points.
 */
NQ_API int nq_gemm_full_q8(const int8_t *X, int64_t ldx, const int8_t *W, int64_t ldw, const float *w_scale,
                    float act_scale, const float *bias, float out_scale, int relu,
                    int64_t M, int64_t N, int64_t K, int8_t *Yq, int64_t ldyq, void *stream);
NQ_API int nq_gemm_part_q8(const int8_t *X, int64_t ldx, const void *packed_high, int n_bits, int h_bits,
                    const float *w_scale, float act_scale, const float *bias, float out_scale, int relu,
                    int64_t M, int64_t N, int64_t K, int8_t *Yq, int64_t ldyq, void *stream);
NQ_API int nq_conv_implicit_gemm_q8(const int8_t *X, const void *Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                             const nq_conv_desc *desc, const float *w_scale, float act_scale, const float *bias,
                             float out_scale, int relu, int8_t *Yq,
                             void *workspace, int64_t workspace_bytes, void *stream);

/* The nested full-bit layers (nq_gemm_nested, nq_conv_implicit_gemm_nested) with the same requantising epilogue. */
NQ_API int nq_gemm_nested_q8(const int8_t *X, int64_t ldx, const void *packed_high, const void *packed_low,
                      int n_bits, int h_bits, const float *w_scale, float act_scale, const float *bias,
                      float out_scale, int relu, int64_t M, int64_t N, int64_t K,
                      int8_t *Yq, int64_t ldyq, void *stream);
NQ_API int nq_conv_implicit_gemm_nested_q8(const int8_t *X, const void *packed_high, const void *packed_low,
                                    int n_bits, int h_bits, const nq_conv_desc *desc, const float *w_scale,
                                    float act_scale, const float *bias, float out_scale, int relu, int8_t *Yq,
                                    void *workspace, int64_t workspace_bytes, void *stream);


/*
 * Pieces a chained model needs between its layers.  The paper runs its models with 8-bit activations but defines
 * none of this arithmetic (how a block's skip path, or a pooling layer, treats the INT8 tensors), so these are the
 * library's own definitions, all in fp32 with one rounding per operation:
 *
 * Residual blocks -- the requantising convolution (nq_conv_implicit_gemm_q8, and its nested full-bit form) with a
 * skip tensor added before the activation:
 *   v = dequantised convolution output (+ bias[j]);   v = fl(v + fl(float(residual[m, j]) * residual_scale))
 *   v = max(v, 0) when relu != 0;   q = clip(round_half_even(fl(v * fl(1 / out_scale))), -128, 127)
 *   residual (device) int8, the output's shape [B, Ho, Wo, Cout], dense NHWC: the block's input (identity skip) or
 *   the requantised output of its 1 x 1 down-sampling convolution; residual_scale is that tensor's activation scale.
 *   A 16-byte aligned residual with Cout a multiple of 16 takes the fast path; anything else is read byte-wise.
 *   Every other argument is that of nq_conv_implicit_gemm_q8 / nq_conv_implicit_gemm_nested_q8.
 */
NQ_API int nq_conv_implicit_gemm_q8_res(const int8_t *X, const void *Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                                 const nq_conv_desc *desc, const float *w_scale, float act_scale, const float *bias,
                                 const int8_t *residual, float residual_scale, float out_scale, int relu, int8_t *Yq,
                                 void *workspace, int64_t workspace_bytes, void *stream);
NQ_API int nq_conv_implicit_gemm_nested_q8_res(const int8_t *X, const void *packed_high, const void *packed_low,
                                        int n_bits, int h_bits, const nq_conv_desc *desc, const float *w_scale,
                                        float act_scale, const float *bias, const int8_t *residual,
                                        float residual_scale, float out_scale, int relu, int8_t *Yq,
                                        void *workspace, int64_t workspace_bytes, void *stream);

/*
 * Max pooling of INT8 NHWC activations [B, H, W, C] -> [B, Ho, Wo, C], Ho = (H + 2*pad - ksize) / stride + 1:
 * the integer maximum over the window's taps that lie inside the image (padding never wins); the activation scale
 * is unchanged.  pad < ksize.  C a multiple of 16 with 16-byte aligned tensors takes 16-byte accesses.
 */
NQ_API int nq_maxpool_nhwc_i8(const int8_t *X, int B, int H, int W, int C, int ksize, int stride, int pad, int8_t *Y,
                       void *stream);

/*
 * Global average pooling with requantisation, INT8 NHWC [B, H, W, C] -> INT8 [B, C]:
 *   sum = integer sum over the H*W pixels;  a = fl(in_scale / float(H*W));
 *   q = clip(round_half_even(fl(fl(float(sum) * a) * fl(1 / out_scale))), -128, 127)
 */
NQ_API int nq_avgpool_requant_nhwc_i8(const int8_t *X, int B, int H, int W, int C, float in_scale, float out_scale,
                               int8_t *Y, void *stream);

/*
 * The convolution again, for callers that must not allocate.  (The paper has no counterpart; this is a
 * convenience of the library.)  nq_conv_implicit_gemm needs a workspace whenever it re-lays the input
 * (NCHW activations, or a channel count it cannot gather in place), and somebody has to allocate that.
 * Code that runs where cudaMalloc is off the table -- a plug-in handed a fixed set of buffers by its host
 * application, a real-time loop that may not touch the allocator, a process whose memory budget was
 * pinned at start-up -- can call this variant instead: it takes the same inputs and outputs and no
 * workspace, and stages through an array that is part of the library image itself.
 *   - The array is NQ_CONV_STATIC_SCRATCH_BYTES (16 MiB) of device memory.  Every GPU on which the library
 *     is loaded carries it from load to process exit, used or not.
 *   - A layer whose nq_conv_workspace_bytes() exceeds that size is refused with NQ_ERR_WORKSPACE and
 *     nothing is launched; use nq_conv_implicit_gemm with your own buffer for those.
 *   - The first call on each device looks the array's device address up (one runtime query, with that
 *     device current).  Make that first call before you start capturing a stream.
 *   - All calls share the one array and it keeps whatever the previous call left there.  The kernels
 *     overwrite every byte they later read, so nothing has to be cleared between calls; but two calls
 *     whose work overlaps on the GPU (different streams, or different host threads) would scribble over
 *     each other's staging data.  Keep calls on one stream, or order them yourself.
 *   - Host side: the looked-up address is cached per device (devices 0..63) in the library; host threads may
 *     make their calls in any order, the first one included.  A cached address does not survive
 *     cudaDeviceReset: a process that resets a device must not call this function on it afterwards.
 *   - No cudaMalloc, cudaFree or allocating library routine is called.
 * Arguments, layouts, results and error codes are otherwise those of nq_conv_implicit_gemm.
 */
#define NQ_CONV_STATIC_SCRATCH_BYTES (16 * 1024 * 1024)
NQ_API int nq_conv_implicit_gemm_static(const int8_t *X, const void *Wt, int64_t ldw, int part_bit, int n_bits,
                                        int h_bits, const nq_conv_desc *desc, const float *w_scale, float act_scale,
                                        const float *bias, int32_t *acc_out, void *Y, int y_dtype, void *stream);

/*
 * Test aid (the paper has no counterpart).  The GEMM / convolution kernels have two pairs of equivalent code paths:
 * outputs written by TMA tile stores or by ordinary stores, and part-bit fields of 1, 2 and 4 bits read straight
 * from the packed matrix or through the shared-memory ring of packed tiles.  The library picks by alignment and
 * field width; this switch forces the second of each pair so that a test can compare the two bit for bit.
 * Process-wide and not synchronised: set it only while no call of another thread is in flight.
 */
enum { NQ_DEBUG_PLAIN_STORES = 0, NQ_DEBUG_PACKED_RING = 1 };
NQ_API int nq_debug_set(int which, int enabled);

/*
 * Measurement aid (the paper has no counterpart: it times no integer kernel).  Enqueues ONE launch of a kernel
 * that only issues the tensor instruction of the GEMM / convolution kernels -- tcgen05.mma kind::i8 on CTA pairs,
 * 256 x 256 x 32 per instruction -- on operands that already sit in shared memory (small signed pseudo-random
 * bytes), accumulating in tensor memory: no global loads, no epilogue.  Every CTA pair (one per two SMs) runs
 * stage_iters stages of four instructions.  Timed with CUDA events by the caller, ops / time is the ceiling of
 * the INT8 tensor path on this GPU under its power limit, the denominator of the GEMM roofline.
 *   stage_iters  in [1, 2^21] (a launch of 3700 stages lasts about a millisecond)
 *   ops_out (host, out, may be NULL)  integer operations of the launch: pairs * stage_iters * 4 * 2*256*256*32
 * Allocates nothing; the wait at its end is bounded like every other (nq_device_status).
 */
NQ_API int nq_i8_mma_ceiling(int64_t stage_iters, double *ops_out, void *stream);

/*
 * Every on-device wait in the GEMM / convolution kernels is bounded.  If one expires the kernel
 * records it and returns instead of hanging.  This call synchronises `stream`, reads and clears
 * the record of the current device: returns NQ_OK, NQ_ERR_TIMEOUT (with *where_out = an internal
 * code of the wait that gave up) or NQ_ERR_CUDA.
 */
NQ_API int nq_device_status(void *stream, int *where_out);

#ifdef __cplusplus
}
#endif
#endif /* NQ_H_ */
