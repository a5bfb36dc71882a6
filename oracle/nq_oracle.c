/*
 * nq_oracle.c -- plain CPU restatement of NestQuant's nested-integer arithmetic.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is checked
 * against; it is never part of the product path.  It shares no code, header, table
 * or helper with the CUDA sources and is written for the eye, not for speed: one
 * loop nest per definition, 32-bit integer intermediates, no blocking, no
 * intrinsics.  The only concession to wall-clock is an OpenMP "parallel for" over
 * the outermost independent index.
 *
 * What follows the paper, and where:
 *   decompose   Eq. 5 (w_int = w_high * 2^l + w_low, n = h + l), Eq. 6 (w_high is
 *               the clipped rounding of w_int / 2^l), Algorithm 1 step 2 (the
 *               rounding direction of every element is decided by the adaptive
 *               rounding, here an input mask), Eq. 10 (clipped w_low) and the
 *               "Full-Bit Model: Performance Compensation" subsection (w_low kept in
 *               l+1 bits, unclipped).
 *   recompose   Eq. 5 read right to left: shift w_high left by l and ADD w_low.
 *   drop_low    the downgrade of "Nesting Mechanism of Decomposed Weights":
 *               w_high = (w_int - w_low) / 2^l.
 *   word64      "Deployment" paragraph: 64 // k fields per unsigned 64-bit word.
 *   gemm/conv   the integer layer the nested weights feed (x_hat = s * x_int in the
 *               Background, Eq. 2, Eq. 9): int8 x int8 -> int32, then one fp32
 *               scale per output channel, times 2^l in part-bit mode.
 *
 * Parity pins (tests/test_oracle_*.py): the worked example of the compensation
 * figure, all 40 entries of the numerical-error table, exhaustive exact
 * recomposition, range invariants, brute force and library cross-checks for the
 * contraction.  The bit positions of the "sliced" packed layout are this
 * library's own choice (the paper fixes only the field width and two's complement
 * content): that layout is parity unpinned by the paper and pinned only by
 * round-trip, by its size function and by a hand-written example.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>

/* ------------------------------------------------------------------------- */
/* helpers                                                                   */
/* ------------------------------------------------------------------------- */

static int32_t clip_i32(int32_t v, int32_t lo, int32_t hi)
{
    if (v < lo) return lo;
    if (v > hi) return hi;
    return v;
}

/* floor(w / 2^l) for any sign of w, written without relying on >> of negatives */
static int32_t floor_div_pow2(int32_t w, int l)
{
    int32_t d = (int32_t)1 << l;
    int32_t q = w / d;              /* C division truncates toward zero */
    if ((w % d) != 0 && w < 0) q -= 1;
    return q;
}

static int valid_bits(int n_bits, int h_bits)
{
    return n_bits >= 2 && n_bits <= 8 && h_bits >= 1 && h_bits < n_bits;
}

/* ------------------------------------------------------------------------- */
/* O1  decomposition (Eq. 5, Eq. 6, Eq. 10, Algorithm 1 step 2, compensation) */
/* ------------------------------------------------------------------------- */

/*
 * mask[i] == 0 : round w_int / 2^l down (floor; this is the RightShift of Eq. 6)
 * mask[i] != 0 : round it up (ceil; an exact multiple of 2^l stays where it is)
 * then clip to the signed h-bit range.  w_low is what is left; with compensate
 * it is stored as is (it fits l+1 signed bits), without it is clipped to l bits
 * as Eq. 10 prints.
 * Returns 0, or -1 for an unsupported (n, h).
 */
int nqo_decompose(const int8_t *w_int, const uint8_t *mask, int64_t count,
                  int n_bits, int h_bits, int compensate,
                  int8_t *w_high, int8_t *w_low)
{
    if (!valid_bits(n_bits, h_bits)) return -1;
    const int l = n_bits - h_bits;
    const int32_t two_l = (int32_t)1 << l;
    const int32_t min_high = -((int32_t)1 << (h_bits - 1));
    const int32_t max_high = ((int32_t)1 << (h_bits - 1)) - 1;
    const int32_t min_low = -((int32_t)1 << (l - 1));
    const int32_t max_low = ((int32_t)1 << (l - 1)) - 1;
    for (int64_t i = 0; i < count; ++i) {
        int32_t w = w_int[i];
        int32_t down = floor_div_pow2(w, l);
        int32_t exact = (down * two_l == w);
        int32_t rounded = (mask[i] != 0 && !exact) ? down + 1 : down;
        int32_t wh = clip_i32(rounded, min_high, max_high);
        int32_t wl = w - wh * two_l;
        if (!compensate) wl = clip_i32(wl, min_low, max_low);
        w_high[i] = (int8_t)wh;
        w_low[i] = (int8_t)wl;
    }
    return 0;
}

/* Round-to-nearest mask for the RTN row of the numerical-error table: the mask
 * that makes the rounding of w / 2^l land on the nearest integer, ties to even. */
int nqo_mask_rtn(const int8_t *w_int, int64_t count, int n_bits, int h_bits, uint8_t *mask)
{
    if (!valid_bits(n_bits, h_bits)) return -1;
    const int l = n_bits - h_bits;
    const int32_t two_l = (int32_t)1 << l;
    for (int64_t i = 0; i < count; ++i) {
        int32_t w = w_int[i];
        int32_t down = floor_div_pow2(w, l);
        int32_t rem = w - down * two_l;           /* 0 .. 2^l - 1 */
        int up;
        if (2 * rem > two_l) up = 1;
        else if (2 * rem < two_l) up = 0;
        else up = (down & 1) != 0;                /* tie: go to the even neighbour */
        mask[i] = (uint8_t)up;
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O2  recomposition / page-in (Eq. 5): shift and ADD, then the INTn clip     */
/* ------------------------------------------------------------------------- */
int nqo_recompose(const int8_t *w_high, const int8_t *w_low, int64_t count,
                  int n_bits, int h_bits, int8_t *w_int)
{
    if (!valid_bits(n_bits, h_bits)) return -1;
    const int l = n_bits - h_bits;
    const int32_t lo = -((int32_t)1 << (n_bits - 1));
    const int32_t hi = ((int32_t)1 << (n_bits - 1)) - 1;
    for (int64_t i = 0; i < count; ++i) {
        int32_t v = (int32_t)w_high[i] * ((int32_t)1 << l) + (int32_t)w_low[i];
        w_int[i] = (int8_t)clip_i32(v, lo, hi);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O3  drop-low / page-out: w_high = (w_int - w_low) / 2^l                    */
/* ------------------------------------------------------------------------- */
int nqo_drop_low(const int8_t *w_int, const int8_t *w_low, int64_t count,
                 int n_bits, int h_bits, int8_t *w_high)
{
    if (!valid_bits(n_bits, h_bits)) return -1;
    const int l = n_bits - h_bits;
    for (int64_t i = 0; i < count; ++i) {
        int32_t d = (int32_t)w_int[i] - (int32_t)w_low[i];
        w_high[i] = (int8_t)floor_div_pow2(d, l);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O4a  the paper's packed-bit tensor: 64 // k fields per unsigned 64-bit word */
/* ------------------------------------------------------------------------- */
int64_t nqo_word64_fields_per_word(int bits) { return 64 / bits; }

int64_t nqo_word64_row_words(int64_t cols, int bits)
{
    int64_t per = 64 / bits;
    return (cols + per - 1) / per;
}

/* field j of a word sits at bits [j*k, j*k + k); unused top bits are zero */
void nqo_pack_word64(const int8_t *v, int64_t rows, int64_t cols, int bits, uint64_t *out)
{
    const int64_t per = 64 / bits;
    const int64_t words = nqo_word64_row_words(cols, bits);
    const uint64_t field_mask = (bits == 64) ? ~0ull : (((uint64_t)1 << bits) - 1);
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t wd = 0; wd < words; ++wd) out[r * words + wd] = 0;
        for (int64_t c = 0; c < cols; ++c) {
            uint64_t field = ((uint64_t)(int64_t)v[r * cols + c]) & field_mask;
            out[r * words + c / per] |= field << ((c % per) * bits);
        }
    }
}

void nqo_unpack_word64(const uint64_t *in, int64_t rows, int64_t cols, int bits, int8_t *v)
{
    const int64_t per = 64 / bits;
    const int64_t words = nqo_word64_row_words(cols, bits);
    const uint64_t field_mask = ((uint64_t)1 << bits) - 1;
    const int64_t sign = (int64_t)1 << (bits - 1);
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            int64_t u = (int64_t)((in[r * words + c / per] >> ((c % per) * bits)) & field_mask);
            if (u >= sign) u -= (int64_t)1 << bits;       /* two's complement field */
            v[r * cols + c] = (int8_t)u;
        }
}

/* ------------------------------------------------------------------------- */
/* O4b  the "sliced" layout (this library's storage format, not the paper's)  */
/* ------------------------------------------------------------------------- */
/*
 * A [rows, cols] tensor of k-bit two's-complement fields is padded with zero fields to
 * multiples of 128 in both directions and cut into blocks of 128 rows x 128 columns.
 * A block takes 2048*k bytes; blocks follow one another row-block by row-block
 * (block (rb, g) of a tensor with G = ceil(cols/128) column groups is block number
 * rb*G + g).  k is written as a sum of distinct powers of two (8, 4, 2, 1), widest
 * first; each power s is a "slice" that holds s bits of every field, the widest slice
 * holding the most significant bits.  Inside a block the slices follow one another,
 * the slice of width s occupying 2048*s bytes: the 128 rows of the block one after the
 * other, 16*s bytes each.  Inside a row's 16*s bytes, element e of the row's 128
 * (e = column % 128) is placed as
 *      unit = e / 32        a unit is 32 elements = s little-endian 32-bit words
 *      q    = (e % 32) / 4  which of the unit's eight 4-element quads
 *      lane = e % 4         byte lane inside the word
 *      word = q / (8 / s)   8/s slices share one byte
 *      sub  = q % (8 / s)   sub 0 sits in the TOP bits of the byte
 * i.e. byte (unit*s + word)*4 + lane, bits [8 - s*sub - s, 8 - s*sub).
 * With s = 8 this is the plain byte order of the block's rows.
 */
static int slice_widths(int bits, int widths[4])
{
    int n = 0;
    for (int s = 8; s >= 1; s >>= 1)
        if (bits & s) widths[n++] = s;
    return n;
}

/* bytes per row of the padded tensor (a size unit only: a row's bytes are not contiguous) */
int64_t nqo_sliced_row_bytes(int64_t cols, int bits)
{
    int64_t groups = (cols + 127) / 128;
    return groups * 16 * bits;
}

int64_t nqo_sliced_padded_rows(int64_t rows) { return (rows + 127) / 128 * 128; }

/* where slice `s` keeps the bits of element e of a row: byte offset inside the row's 16*s bytes, shift inside the byte */
static void slice_place(int s, int e, int64_t *byte_off, int *shift)
{
    int unit = e / 32, q = (e % 32) / 4, lane = e % 4;
    int per_byte = 8 / s;
    int word = q / per_byte, sub = q % per_byte;
    *byte_off = (int64_t)(unit * s + word) * 4 + lane;
    *shift = 8 - s * sub - s;
}

/* start of the 16*s bytes that slice number k (preceded by `bits_before` bits of wider slices) keeps for row r, column c */
static int64_t slice_row_start(int64_t r, int64_t c, int64_t groups, int bits, int bits_before, int s)
{
    int64_t block = (r / 128) * groups + c / 128;
    return block * 2048 * bits + (int64_t)2048 * bits_before + (r % 128) * 16 * s;
}

int nqo_pack_sliced(const int8_t *v, int64_t rows, int64_t cols, int bits, uint8_t *out)
{
    if (bits < 1 || bits > 8) return -1;
    int widths[4];
    const int nslices = slice_widths(bits, widths);
    const int64_t groups = (cols + 127) / 128;
    memset(out, 0, (size_t)(nqo_sliced_padded_rows(rows) * groups * 16 * bits));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            uint32_t field = ((uint32_t)(int32_t)v[r * cols + c]) & ((1u << bits) - 1u);
            int e = (int)(c % 128);
            int consumed = 0;                     /* field bits already placed, from the top */
            for (int k = 0; k < nslices; ++k) {
                int s = widths[k];
                uint32_t part = (field >> (bits - consumed - s)) & ((1u << s) - 1u);
                int64_t off; int sh;
                slice_place(s, e, &off, &sh);
                out[slice_row_start(r, c, groups, bits, consumed, s) + off] |= (uint8_t)(part << sh);
                consumed += s;
            }
        }
    return 0;
}

int nqo_unpack_sliced(const uint8_t *in, int64_t rows, int64_t cols, int bits, int8_t *v)
{
    if (bits < 1 || bits > 8) return -1;
    int widths[4];
    const int nslices = slice_widths(bits, widths);
    const int64_t groups = (cols + 127) / 128;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            int e = (int)(c % 128);
            uint32_t field = 0;
            int consumed = 0;
            for (int k = 0; k < nslices; ++k) {
                int s = widths[k];
                int64_t off; int sh;
                slice_place(s, e, &off, &sh);
                uint32_t part = ((uint32_t)in[slice_row_start(r, c, groups, bits, consumed, s) + off] >> sh) & ((1u << s) - 1u);
                field = (field << s) | part;
                consumed += s;
            }
            int32_t val = (int32_t)field;
            if (val >= (1 << (bits - 1))) val -= (1 << bits);   /* two's complement field */
            v[r * cols + c] = (int8_t)val;
        }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* O5  integer contraction: acc[m, j] = sum_k x[m, k] * w[j, k]               */
/* ------------------------------------------------------------------------- */
void nqo_gemm_acc(const int8_t *x, int64_t ldx, const int8_t *w, int64_t ldw,
                  int64_t M, int64_t N, int64_t K, int32_t *acc, int64_t ldacc)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t j = 0; j < N; ++j) {
            int32_t s = 0;
            for (int64_t k = 0; k < K; ++k)
                s += (int32_t)x[m * ldx + k] * (int32_t)w[j * ldw + k];
            acc[m * ldacc + j] = s;
        }
}

/* ------------------------------------------------------------------------- */
/* O6  dequantisation (Eq. 2 full-bit, Eq. 9 part-bit): one fp32 rounding per  */
/*     operation, in this order:                                              */
/*        scale_j = fl(fl(act_scale * w_scale[j]) * 2^l)   (l = 0 in full-bit) */
/*        y       = fl(float(acc) * scale_j)  [+ bias_j, one more rounding]    */
/*     y_ref is the same quantity carried in double with no fp32 rounding.    */
/* ------------------------------------------------------------------------- */
void nqo_dequant(const int32_t *acc, int64_t ldacc, int64_t M, int64_t N,
                 const float *w_scale, float act_scale, int l_shift, const float *bias,
                 float *y, int64_t ldy, double *y_ref)
{
    const float pow2 = (float)(1 << l_shift);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t j = 0; j < N; ++j) {
            volatile float sj = act_scale * w_scale[j];
            volatile float scale = sj * pow2;
            volatile float prod = (float)acc[m * ldacc + j] * scale;
            float out = prod;
            if (bias) { volatile float t = prod + bias[j]; out = t; }
            y[m * ldy + j] = out;
            if (y_ref) {
                double d = (double)acc[m * ldacc + j] * (double)act_scale * (double)w_scale[j]
                         * (double)(1 << l_shift);
                if (bias) d += (double)bias[j];
                y_ref[m * N + j] = d;
            }
        }
}

/* ------------------------------------------------------------------------- */
/* O6b  requantisation of a layer's output to INT8 for the next layer.  The    */
/*      paper quantises activations to 8 bits ("8-bit activations") with the   */
/*      uniform quantiser of Eq. 1 and zero-point 0, but does not say how a    */
/*      layer's output becomes the next layer's input: PARITY UNPINNED by the  */
/*      paper; this is the library's own definition, in fp32, one rounding per */
/*      operation, in this order:                                              */
/*        v = dequantised output as in O6 (+ bias)                             */
/*        v = max(v, 0)                       when relu                        */
/*        t = fl(v * fl(1 / out_scale))                                        */
/*        q = clip(round-half-even(t), -128, 127)          (Eq. 1 with Z = 0)  */
/* ------------------------------------------------------------------------- */
void nqo_requant(const int32_t *acc, int64_t ldacc, int64_t M, int64_t N,
                 const float *w_scale, float act_scale, int l_shift, const float *bias,
                 int relu, float out_scale, int8_t *q, int64_t ldq)
{
    const float pow2 = (float)(1 << l_shift);
    volatile float inv = 1.0f / out_scale;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t j = 0; j < N; ++j) {
            volatile float sj = act_scale * w_scale[j];
            volatile float scale = sj * pow2;
            volatile float v = (float)acc[m * ldacc + j] * scale;
            if (bias) { volatile float t = v + bias[j]; v = t; }
            if (relu && v < 0.0f) v = 0.0f;
            volatile float t = v * inv;
            float r = nearbyintf(t);              /* default rounding mode: to nearest, ties to even */
            if (r < -128.0f) r = -128.0f;
            if (r > 127.0f) r = 127.0f;
            q[m * ldq + j] = (int8_t)r;
        }
}

/* ------------------------------------------------------------------------- */
/* O6c  the same hand-over with a residual connection (the skip path of a      */
/*      ResNet block): the skip tensor r is INT8 with its own scale and is     */
/*      added, dequantised, before the activation.  PARITY UNPINNED by the     */
/*      paper (it says "8-bit activations" and nothing about the blocks'       */
/*      arithmetic); the library's own definition, fp32, one rounding each:    */
/*        v = dequantised output as in O6 (+ bias)                             */
/*        v = fl(v + fl(float(r) * res_scale))                                 */
/*        v = max(v, 0) when relu;  t = fl(v * fl(1 / out_scale))              */
/*        q = clip(round-half-even(t), -128, 127)                              */
/* ------------------------------------------------------------------------- */
void nqo_requant_res(const int32_t *acc, int64_t ldacc, int64_t M, int64_t N,
                     const float *w_scale, float act_scale, int l_shift, const float *bias,
                     const int8_t *res, int64_t ldres, float res_scale,
                     int relu, float out_scale, int8_t *q, int64_t ldq)
{
    const float pow2 = (float)(1 << l_shift);
    volatile float inv = 1.0f / out_scale;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t j = 0; j < N; ++j) {
            volatile float sj = act_scale * w_scale[j];
            volatile float scale = sj * pow2;
            volatile float v = (float)acc[m * ldacc + j] * scale;
            if (bias) { volatile float t = v + bias[j]; v = t; }
            volatile float skip = (float)res[m * ldres + j] * res_scale;
            volatile float sum = v + skip;
            v = sum;
            if (relu && v < 0.0f) v = 0.0f;
            volatile float t = v * inv;
            float r = nearbyintf(t);
            if (r < -128.0f) r = -128.0f;
            if (r > 127.0f) r = 127.0f;
            q[m * ldq + j] = (int8_t)r;
        }
}

/* ------------------------------------------------------------------------- */
/* O8   pooling between the layers of a chained model (library's own           */
/*      definitions, PARITY UNPINNED by the paper).  Activations are INT8,     */
/*      NHWC [B, H, W, C].                                                     */
/*      max pooling: the integer maximum over the window's taps that lie       */
/*      inside the image (padding never wins); the scale is unchanged.         */
/*      global average pooling with requantisation:                            */
/*        sum = integer sum over the H * W pixels of a channel                 */
/*        a   = fl(in_scale / float(H * W))                                    */
/*        t   = fl(fl(float(sum) * a) * fl(1 / out_scale))                     */
/*        q   = clip(round-half-even(t), -128, 127)                            */
/* ------------------------------------------------------------------------- */
void nqo_maxpool_nhwc(const int8_t *x, int64_t B, int64_t H, int64_t W, int64_t C,
                      int64_t ksize, int64_t stride, int64_t pad, int8_t *y)
{
    const int64_t Ho = (H + 2 * pad - ksize) / stride + 1, Wo = (W + 2 * pad - ksize) / stride + 1;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t p = 0; p < Ho; ++p)
            for (int64_t q = 0; q < Wo; ++q)
                for (int64_t c = 0; c < C; ++c) {
                    int best = -128;
                    for (int64_t r = 0; r < ksize; ++r)
                        for (int64_t s = 0; s < ksize; ++s) {
                            int64_t ih = p * stride - pad + r, iw = q * stride - pad + s;
                            if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                            int v = x[((b * H + ih) * W + iw) * C + c];
                            if (v > best) best = v;
                        }
                    y[((b * Ho + p) * Wo + q) * C + c] = (int8_t)best;
                }
}

void nqo_avgpool_requant_nhwc(const int8_t *x, int64_t B, int64_t H, int64_t W, int64_t C,
                              float in_scale, float out_scale, int8_t *y)
{
    volatile float a = in_scale / (float)(H * W);
    volatile float inv = 1.0f / out_scale;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t c = 0; c < C; ++c) {
            int32_t sum = 0;
            for (int64_t i = 0; i < H * W; ++i) sum += x[(b * H * W + i) * C + c];
            volatile float v = (float)sum * a;
            volatile float t = v * inv;
            float r = nearbyintf(t);
            if (r < -128.0f) r = -128.0f;
            if (r > 127.0f) r = 127.0f;
            y[b * C + c] = (int8_t)r;
        }
}

/* fp32 -> bf16, round to nearest, ties to even (finite inputs) */
void nqo_f32_to_bf16(const float *x, int64_t count, uint16_t *out)
{
    for (int64_t i = 0; i < count; ++i) {
        uint32_t u;
        memcpy(&u, &x[i], 4);
        uint32_t keep = u >> 16, drop = u & 0xFFFFu;
        if (drop > 0x8000u || (drop == 0x8000u && (keep & 1u))) keep += 1;
        out[i] = (uint16_t)keep;
    }
}

/* ------------------------------------------------------------------------- */
/* O7  direct convolution, zero padding (the zero-point is 0):                */
/*   acc[b, co, p, q] = sum_{ci, r, s} x[b, ci, p*st - pad + r, q*st - pad + s] */
/*                                     * w[co, ci, r, s]                      */
/*   x is NCHW, w is OIHW, acc is N(Cout)HoWo -- the framework layout the      */
/*   paper's models use.                                                      */
/* ------------------------------------------------------------------------- */
int64_t nqo_conv_out_dim(int64_t in, int64_t ksize, int64_t stride, int64_t pad)
{
    return (in + 2 * pad - ksize) / stride + 1;
}

void nqo_conv_acc(const int8_t *x, int64_t B, int64_t C, int64_t H, int64_t W,
                  const int8_t *w, int64_t Cout, int64_t R, int64_t S,
                  int64_t stride, int64_t pad, int32_t *acc)
{
    const int64_t Ho = nqo_conv_out_dim(H, R, stride, pad);
    const int64_t Wo = nqo_conv_out_dim(W, S, stride, pad);
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t co = 0; co < Cout; ++co)
            for (int64_t p = 0; p < Ho; ++p)
                for (int64_t q = 0; q < Wo; ++q) {
                    int32_t s = 0;
                    for (int64_t ci = 0; ci < C; ++ci)
                        for (int64_t r = 0; r < R; ++r)
                            for (int64_t t = 0; t < S; ++t) {
                                int64_t ih = p * stride - pad + r;
                                int64_t iw = q * stride - pad + t;
                                if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                                s += (int32_t)x[((b * C + ci) * H + ih) * W + iw]
                                   * (int32_t)w[((co * C + ci) * R + r) * S + t];
                            }
                    acc[((b * Cout + co) * Ho + p) * Wo + q] = s;
                }
}

/* the same definition evaluated at listed output pixels only (all Cout channels):
 * pix[3*i + 0..2] = (b, p, q); acc_out[i*Cout + co] */
void nqo_conv_acc_pixels(const int8_t *x, int64_t B, int64_t C, int64_t H, int64_t W,
                         const int8_t *w, int64_t Cout, int64_t R, int64_t S,
                         int64_t stride, int64_t pad,
                         const int64_t *pix, int64_t npix, int32_t *acc_out)
{
    (void)B;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < npix; ++i) {
        int64_t b = pix[3 * i], p = pix[3 * i + 1], q = pix[3 * i + 2];
        for (int64_t co = 0; co < Cout; ++co) {
            int32_t s = 0;
            for (int64_t ci = 0; ci < C; ++ci)
                for (int64_t r = 0; r < R; ++r)
                    for (int64_t t = 0; t < S; ++t) {
                        int64_t ih = p * stride - pad + r;
                        int64_t iw = q * stride - pad + t;
                        if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                        s += (int32_t)x[((b * C + ci) * H + ih) * W + iw]
                           * (int32_t)w[((co * C + ci) * R + r) * S + t];
                    }
            acc_out[i * Cout + co] = s;
        }
    }
}

int nqo_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
