// Implicit-GEMM convolution on the nested weights: layout pre-passes, tile geometry, launch.
//
// The contraction itself is the kernel of nq_contraction.cuh.  Here the activations are brought to the
// form its TMA producer reads:
//   - Cin = 64 or a multiple of 128 (every ResNet layer but the stem): NHWC activations are read in place,
//     one rectangle of output pixels and one filter tap at a time, by 4-D tile loads whose out-of-image
//     coordinates return zeros (the zero padding).  NCHW input is first transposed into the workspace.
//   - any other Cin (the 3-channel stem): the [M, K] patch matrix is written out explicitly into the
//     workspace and the plain GEMM path runs on it.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <stdint.h>

#include "../../include/nq.h"
#include "nq_contraction.cuh"
#include "nq_internal.cuh"

// Staging memory of nq_conv_implicit_gemm_static: lives in the library image, one copy per GPU that loads it.
// In host code this name is only a handle for cudaGetSymbolAddress -- it is not a device address.  The extra
// 1 KiB lets the host round the address up to the 1 KiB alignment nq_conv_implicit_gemm asks of a workspace.
static __device__ __align__(256) unsigned char g_conv_static_scratch[NQ_CONV_STATIC_SCRATCH_BYTES + 1024];

namespace nq {
namespace {

// [B, C, HW] int8 -> [B, HW, C]; a block moves 64 channels x 128 pixels.  A thread loads one word (four pixels)
// of each of eight channels -- a warp's load is 128 contiguous bytes of one channel -- turns them into the eight
// channel bytes of each of its four pixels with byte permutes in registers (two 4 x 4 byte transposes), and
// parks those in shared memory, from where whole 16-byte pieces of pixel rows go out.  (Scattering single bytes
// into shared memory, as a first version did, ran at under a third of the memory bandwidth.)
__global__ void __launch_bounds__(256) nchw_to_nhwc_kernel(const int8_t* __restrict__ in, int8_t* __restrict__ out,
                                                           int C, int HW) {
    __shared__ __align__(16) uint8_t tile[128][80];           // [pixel slot][channel]; pixel p sits in slot (p % 4) * 32 + p / 4
    const int b = blockIdx.z, c0 = blockIdx.y * 64, p0 = blockIdx.x * 128;
    const int8_t* src = in + ((size_t)b * C + c0) * HW;
    int8_t* dst = out + (size_t)b * HW * C;
    const int t = threadIdx.x;
    const int pq = t & 31, cg = t >> 5;                       // pixel quad of the block, group of eight channels
    const bool words = ((HW & 3) == 0) && ((reinterpret_cast<uintptr_t>(in) & 3) == 0);
    const int px = p0 + 4 * pq;
    uint32_t w[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int c = cg * 8 + k;
        uint32_t v = 0;
        if (c0 + c < C && px < HW) {
            if (words) {                                       // HW is a multiple of 4, so the whole quad is inside
                v = __ldg(reinterpret_cast<const uint32_t*>(src + (size_t)c * HW + px));
            } else {
                for (int j = 0; j < 4; ++j)
                    if (px + j < HW) v |= (uint32_t)(uint8_t)src[(size_t)c * HW + px + j] << (8 * j);
            }
        }
        w[k] = v;
    }
    uint32_t o[4][2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t t0 = __byte_perm(w[4 * h], w[4 * h + 1], 0x5140), t1 = __byte_perm(w[4 * h + 2], w[4 * h + 3], 0x5140);
        const uint32_t t2 = __byte_perm(w[4 * h], w[4 * h + 1], 0x7362), t3 = __byte_perm(w[4 * h + 2], w[4 * h + 3], 0x7362);
        o[0][h] = __byte_perm(t0, t1, 0x5410); o[1][h] = __byte_perm(t0, t1, 0x7632);
        o[2][h] = __byte_perm(t2, t3, 0x5410); o[3][h] = __byte_perm(t2, t3, 0x7632);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint2*>(&tile[i * 32 + pq][cg * 8]) = make_uint2(o[i][0], o[i][1]);
    __syncthreads();
    const bool pieces = ((C & 15) == 0) && ((reinterpret_cast<uintptr_t>(out) & 15) == 0);
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int idx = t + 256 * r;
        const int pix = idx >> 2, cq = (idx & 3) * 16;
        const int slot = (pix & 3) * 32 + (pix >> 2);
        if (p0 + pix >= HW) continue;
        if (pieces && c0 + cq + 16 <= C) {
            *reinterpret_cast<uint4*>(dst + (size_t)(p0 + pix) * C + c0 + cq) = *reinterpret_cast<const uint4*>(&tile[slot][cq]);
        } else {
            for (int j = 0; j < 16; ++j)
                if (c0 + cq + j < C) dst[(size_t)(p0 + pix) * C + c0 + cq + j] = (int8_t)tile[slot][cq + j];
        }
    }
}

// explicit patch matrix A[m, k], k = (r*S + s)*Cin + ci, row pitch ld (a multiple of 16), zero beyond K
__global__ void __launch_bounds__(256) im2col_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a, nq_conv_desc d,
                                                     int Ho, int Wo, int K, int ld, long long chunks_total) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= chunks_total) return;
    const int chunks_per_row = ld / 16;
    const long long m = idx / chunks_per_row;
    const int k0 = (int)(idx - m * chunks_per_row) * 16;
    const int q = (int)(m % Wo);
    const long long t = m / Wo;
    const int p = (int)(t % Ho), b = (int)(t / Ho);
    uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int k = k0 + j;
        uint32_t v = 0;
        if (k < K) {
            const int tap = k / d.Cin, ci = k - tap * d.Cin;
            const int r = tap / d.S, s = tap - r * d.S;
            const int ih = p * d.stride - d.pad + r, iw = q * d.stride - d.pad + s;
            if (ih >= 0 && ih < d.H && iw >= 0 && iw < d.W) {
                const size_t off = d.x_nchw ? (((size_t)b * d.Cin + ci) * d.H + ih) * d.W + iw
                                            : (((size_t)b * d.H + ih) * d.W + iw) * d.Cin + ci;
                v = (uint8_t)x[off];
            }
        }
        w[j >> 2] |= v << (8 * (j & 3));
    }
    *reinterpret_cast<uint4*>(a + m * ld + k0) = make_uint4(w[0], w[1], w[2], w[3]);
}

// The same patch matrix for layers with few input channels (the stem): one block per output row (b, p).  The
// R input rows it needs are staged in shared memory PIXEL-INTERLEAVED ([r][padded pixel][ci], padding already zero),
// so that the bytes of a patch row that belong to one filter row -- k = (r * S + s) * Cin + ci for all s, ci -- are
// one contiguous run of S * Cin bytes starting at (q * stride) * Cin in staged row r.  A thread owns one 16-byte
// chunk column of the output (k0 fixed) and walks the output pixels: each of its four words is two aligned
// shared-memory reads and a funnel shift (the start offsets, loop-invariant, sit in registers); only a word that
// straddles two filter rows or the end of K is put together byte by byte.  (The first version staged the rows channel
// by channel and read every output byte on its own, two shared-memory reads each: 206 us of the 346 us stem layer
// at batch 128.)  blockDim.x = (ld / 16) * pixels-per-pass.
__global__ void __launch_bounds__(512) im2col_rows_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a,
                                                          nq_conv_desc d, int Ho, int Wo, int K, int ld, int rowbytes) {
    extern __shared__ uint8_t sm[];
    uint8_t* patch = sm;                                   // [R][rowbytes] (+ 8 bytes of slack, zero)
    const int p = blockIdx.x, b = blockIdx.y;
    const int cpr = ld / 16;
    const int run = d.S * d.Cin;                           // bytes of one filter row in a patch row
    for (int i = threadIdx.x; i < (d.R * rowbytes + 8) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(patch)[i] = 0u;
    __syncthreads();
    if (d.x_nchw) {
        // one input word = four pixels of one channel -> four byte stores, Cin apart
        const bool words = ((d.W & 3) == 0) && ((reinterpret_cast<uintptr_t>(x) & 3) == 0);
        const int wpr = words ? d.W >> 2 : d.W;
        for (int i = threadIdx.x; i < d.R * d.Cin * wpr; i += blockDim.x) {
            const int rc = i / wpr, wc = i - rc * wpr;
            const int r = rc / d.Cin, ci = rc - r * d.Cin;
            const int ih = p * d.stride - d.pad + r;
            if (ih < 0 || ih >= d.H) continue;
            const int8_t* src = x + (((size_t)b * d.Cin + ci) * d.H + ih) * d.W;
            uint8_t* dst = patch + r * rowbytes + d.pad * d.Cin + ci;
            if (words) {
                const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(src) + wc);
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[(4 * wc + j) * d.Cin] = (uint8_t)(v >> (8 * j));
            } else {
                dst[wc * d.Cin] = (uint8_t)src[wc];
            }
        }
    } else {
        // NHWC rows are interleaved already: W * Cin contiguous bytes
        const int nb = d.W * d.Cin;
        for (int r = 0; r < d.R; ++r) {
            const int ih = p * d.stride - d.pad + r;
            if (ih < 0 || ih >= d.H) continue;
            const int8_t* src = x + ((size_t)b * d.H + ih) * nb;
            uint8_t* dst = patch + r * rowbytes + d.pad * d.Cin;
            if (((nb & 3) == 0) && ((reinterpret_cast<uintptr_t>(src) & 3) == 0) && (((d.pad * d.Cin) & 3) == 0)) {
                for (int i = threadIdx.x; i < nb / 4; i += blockDim.x)
                    reinterpret_cast<uint32_t*>(dst)[i] = __ldg(reinterpret_cast<const uint32_t*>(src) + i);
            } else {
                for (int i = threadIdx.x; i < nb; i += blockDim.x) dst[i] = (uint8_t)src[i];
            }
        }
    }
    __syncthreads();
    // this thread's chunk column: where each of its 16 bytes starts in the staged rows (relative to q * stride * Cin)
    const int c = threadIdx.x % cpr, q0 = threadIdx.x / cpr, qstep = blockDim.x / cpr;
    const int k0 = c * 16;
    // word j = bytes k .. k + 3: those of filter row r come from offset off_a (mask_a says which), the rest -- a word
    // may straddle two filter rows -- from filter row r + 1 at off_b (mask_b; bytes at or beyond K stay zero)
    int off_a[4], off_b[4];
    uint32_t mask_a[4], mask_b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int k = k0 + 4 * j;
        const int r = k / run;
        const int n_a = min(4, (r + 1) * run - k);         // bytes of this word inside filter row r
        off_a[j] = r * rowbytes + (k - r * run);
        off_b[j] = (r + 1) * rowbytes + (k - (r + 1) * run);      // byte i of a read there is element k + i of row r + 1
        uint32_t ma = 0, mb = 0;
        for (int i = 0; i < 4; ++i) {
            if (k + i >= K) continue;
            if (i < n_a) ma |= 0xffu << (8 * i); else mb |= 0xffu << (8 * i);
        }
        mask_a[j] = ma; mask_b[j] = mb;
        if (ma == 0) off_a[j] = 0;                         // nothing to read: keep the address inside the staged rows
        if (mb == 0) off_b[j] = -1;
    }
    int8_t* out = a + ((size_t)b * Ho + p) * Wo * ld;
    for (int q = q0; q < Wo; q += qstep) {
        const int base = q * d.stride * d.Cin;
        uint32_t w[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = off_a[j] + base;
            const uint32_t* wp = reinterpret_cast<const uint32_t*>(patch + (o & ~3));
            w[j] = __funnelshift_r(wp[0], wp[1], 8 * (o & 3)) & mask_a[j];
            if (off_b[j] >= 0) {
                const int o2 = off_b[j] + base;
                const uint32_t* wq = reinterpret_cast<const uint32_t*>(patch + (o2 & ~3));
                w[j] |= __funnelshift_r(wq[0], wq[1], 8 * (o2 & 3)) & mask_b[j];
            }
        }
        *reinterpret_cast<uint4*>(out + (size_t)q * ld + k0) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

bool implicit_ok(const nq_conv_desc& d) { return d.Cin == 64 || (d.Cin > 0 && d.Cin % 128 == 0); }

bool desc_ok(const nq_conv_desc* d) {
    return d && d->B > 0 && d->Cin > 0 && d->H > 0 && d->W > 0 && d->Cout > 0 && d->R > 0 && d->S > 0 && d->stride > 0 &&
           d->pad >= 0 && d->H + 2 * d->pad >= d->R && d->W + 2 * d->pad >= d->S;
}

int out_dim(int in, int k, int stride, int pad) { return (in + 2 * pad - k) / stride + 1; }

// rectangle of 2^tw x 2^th output pixels of 128 / 2^(tw+th) images that wastes the fewest tile rows
void choose_tile(int B, int Ho, int Wo, int& tw_log2, int& th_log2) {
    double best = 1e300;
    tw_log2 = 3; th_log2 = 3;
    for (int a = 7; a >= 0; --a)
        for (int b = 7 - a; b >= 0; --b) {
            const long long tw = 1 << a, th = 1 << b, tb = 128 >> (a + b);
            const double cover = (double)((Wo + tw - 1) / tw * tw) * ((Ho + th - 1) / th * th) * ((B + tb - 1) / tb * tb);
            if (cover < best) { best = cover; tw_log2 = a; th_log2 = b; }
        }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace nq

extern "C" {

int64_t nq_conv_workspace_bytes(const nq_conv_desc* d) {
    if (!nq::desc_ok(d)) return -1;
    if (nq::implicit_ok(*d)) return d->x_nchw ? (int64_t)d->B * d->H * d->W * d->Cin : 0;
    const int64_t Ho = nq::out_dim(d->H, d->R, d->stride, d->pad), Wo = nq::out_dim(d->W, d->S, d->stride, d->pad);
    const int64_t K = (int64_t)d->R * d->S * d->Cin;
    return (int64_t)d->B * Ho * Wo * ((K + 15) / 16 * 16);
}

static int conv_common(const int8_t* X, const void* Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                       const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                       int32_t* acc_out, void* Y, int y_dtype, void* workspace, int64_t workspace_bytes, void* stream_,
                       const nq::OutQuant* oq, const void* Wlow = nullptr) {
    using namespace nq;
    // Wlow given: nested full-bit mode -- Wt is the packed higher-bit tensor, Wlow the packed compensated lower-bit one
    if (Wlow && ((n_bits != 8 && n_bits != 6) || h_bits < 2 || h_bits >= n_bits)) return NQ_ERR_UNSUPPORTED;
    if (Wlow && !aligned16(Wlow)) return NQ_ERR_ALIGNMENT;
    if (!desc_ok(d)) return NQ_ERR_INVALID_ARG;
    if (y_dtype != NQ_F32 && y_dtype != NQ_BF16 && !(y_dtype == kOutI8 && oq)) return NQ_ERR_INVALID_ARG;
    if (oq && !(oq->out_scale > 0.0f)) return NQ_ERR_INVALID_ARG;
    if (part_bit && (n_bits < 2 || n_bits > 8 || h_bits < 1 || h_bits >= n_bits)) return NQ_ERR_UNSUPPORTED;
    if (!X || !Wt || (!acc_out && !Y) || (Y && !w_scale)) return NQ_ERR_INVALID_ARG;
    const int Ho = out_dim(d->H, d->R, d->stride, d->pad), Wo = out_dim(d->W, d->S, d->stride, d->pad);
    const int64_t M = (int64_t)d->B * Ho * Wo, N = d->Cout, K = (int64_t)d->R * d->S * d->Cin;
    if (K >= (1 << 17) || M > (1ll << 30)) return NQ_ERR_UNSUPPORTED;
    if (!part_bit && (ldw < K || (ldw & 15))) return ldw < K ? NQ_ERR_INVALID_ARG : NQ_ERR_ALIGNMENT;
    if (!aligned16(Wt) || !aligned16(X)) return NQ_ERR_ALIGNMENT;
    const int64_t need = nq_conv_workspace_bytes(d);
    if (need > 0 && (!workspace || workspace_bytes < need)) return NQ_ERR_WORKSPACE;
    if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 1023)) return NQ_ERR_ALIGNMENT;
    cudaStream_t stream = (cudaStream_t)stream_;
    CUtensorMap tmA;

    if (!implicit_ok(*d)) {
        // explicit patch matrix, then the plain GEMM path
        const int ld = (int)((K + 15) / 16 * 16);
        const long long chunks = M * (ld / 16);
        const int cpr = ld / 16;
        const size_t rowbytes = (((size_t)d->W + 2 * d->pad) * d->Cin + 3) & ~size_t(3);
        const size_t rows_smem = (size_t)d->R * rowbytes + 8;
        if (rows_smem <= 48 * 1024 && cpr <= 64 && Ho <= 65535 * 32 && d->B <= 65535) {
            const int per_pass = 256 / cpr > 0 ? 256 / cpr : 1;           // output pixels a block handles at a time
            im2col_rows_kernel<<<dim3(Ho, d->B), cpr * per_pass, rows_smem, stream>>>(X, (int8_t*)workspace, *d, Ho, Wo, (int)K,
                                                                                     ld, (int)rowbytes);
        } else {
            im2col_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, stream>>>(X, (int8_t*)workspace, *d, Ho, Wo, (int)K, ld, chunks);
        }
        if (cudaGetLastError() != cudaSuccess) return NQ_ERR_CUDA;
        int st = encode_tensor_map_2d(&tmA, workspace, (uint64_t)K, (uint64_t)M, (uint64_t)ld, kBK, kBM, 128);
        if (st != NQ_OK) return st;
        return run_contraction(tmA, kModeGemm, nullptr, (int)((M + kBM - 1) / kBM), (int)((K + kBK - 1) / kBK), Wt, ldw,
                               part_bit != 0, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, acc_out, N, Y, N, y_dtype,
                               stream, oq, Wlow);
    }

    const int8_t* x_nhwc = X;
    if (d->x_nchw) {
        const int HW = d->H * d->W;
        dim3 grid((HW + 127) / 128, (d->Cin + 63) / 64, d->B);
        nchw_to_nhwc_kernel<<<grid, 256, 0, stream>>>(X, (int8_t*)workspace, d->Cin, HW);
        if (cudaGetLastError() != cudaSuccess) return NQ_ERR_CUDA;
        x_nhwc = (const int8_t*)workspace;
    }
    if (d->R == 1 && d->S == 1 && d->stride == 1 && d->pad == 0 && d->Cin % 128 == 0) {
        // A pointwise convolution of NHWC activations IS the GEMM [B*H*W, Cin] x [Cout, Cin]^T: plain 2-D tile loads of
        // 128 contiguous rows instead of the 4-D gather, and every tile policy of the GEMM path (pairs, wide tiles).
        // (Measured on the ResNet-101-shaped stack: 3-10 % per such layer; 64-channel inputs are faster on their own mode.)
        int st = encode_tensor_map_2d(&tmA, x_nhwc, (uint64_t)K, (uint64_t)M, (uint64_t)K, kBK, kBM, 128);
        if (st != NQ_OK) return st;
        return run_contraction(tmA, kModeGemm, nullptr, (int)((M + kBM - 1) / kBM), (int)((K + kBK - 1) / kBK), Wt, ldw,
                               part_bit != 0, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, acc_out, N, Y, N, y_dtype,
                               stream, oq, Wlow);
    }
    ConvGeom g{};
    g.B = d->B; g.Ho = Ho; g.Wo = Wo; g.S = d->S; g.taps = d->R * d->S; g.stride = d->stride; g.pad = d->pad;
    choose_tile(d->B, Ho, Wo, g.tw_log2, g.th_log2);
    const int tw = 1 << g.tw_log2, th = 1 << g.th_log2, tb = 128 >> (g.tw_log2 + g.th_log2);
    g.tiles_w = (Wo + tw - 1) / tw;
    g.tiles_h = (Ho + th - 1) / th;
    const int tiles_b = (d->B + tb - 1) / tb;
    const int m_tiles = g.tiles_w * g.tiles_h * tiles_b;
    int mode, k_blocks, st;
    if (d->Cin == 64) {
        mode = kModeConv64;
        g.cblocks = 1;
        k_blocks = (g.taps + 1) / 2;
        st = encode_tensor_map_nhwc(&tmA, x_nhwc, d->Cin, d->W, d->H, d->B, 64, tw, th, tb, d->stride, 64);
    } else {
        mode = kModeConv128;
        g.cblocks = d->Cin / 128;
        k_blocks = g.taps * g.cblocks;
        st = encode_tensor_map_nhwc(&tmA, x_nhwc, d->Cin, d->W, d->H, d->B, 128, tw, th, tb, d->stride, 128);
    }
    if (st != NQ_OK) return st;
    return run_contraction(tmA, mode, &g, m_tiles, k_blocks, Wt, ldw, part_bit != 0, n_bits, h_bits, w_scale, act_scale,
                           bias, M, N, K, acc_out, N, Y, N, y_dtype, stream, oq, Wlow);
}

int nq_conv_implicit_gemm(const int8_t* X, const void* Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                          const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                          int32_t* acc_out, void* Y, int y_dtype, void* workspace, int64_t workspace_bytes, void* stream) {
    if (y_dtype != NQ_F32 && y_dtype != NQ_BF16) return NQ_ERR_INVALID_ARG;
    return conv_common(X, Wt, ldw, part_bit, n_bits, h_bits, d, w_scale, act_scale, bias, acc_out, Y, y_dtype, workspace,
                       workspace_bytes, stream, nullptr);
}

int nq_conv_implicit_gemm_nested(const int8_t* X, const void* packed_high, const void* packed_low, int n_bits, int h_bits,
                                 const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                                 int32_t* acc_out, void* Y, int y_dtype, void* workspace, int64_t workspace_bytes,
                                 void* stream) {
    if (y_dtype != NQ_F32 && y_dtype != NQ_BF16) return NQ_ERR_INVALID_ARG;
    if (!packed_low) return NQ_ERR_INVALID_ARG;
    return conv_common(X, packed_high, 0, 1, n_bits, h_bits, d, w_scale, act_scale, bias, acc_out, Y, y_dtype, workspace,
                       workspace_bytes, stream, nullptr, packed_low);
}

int nq_conv_implicit_gemm_nested_q8(const int8_t* X, const void* packed_high, const void* packed_low, int n_bits,
                                    int h_bits, const nq_conv_desc* d, const float* w_scale, float act_scale,
                                    const float* bias, float out_scale, int relu, int8_t* Yq, void* workspace,
                                    int64_t workspace_bytes, void* stream) {
    const nq::OutQuant oq{out_scale, relu};
    if (!Yq || !packed_low) return NQ_ERR_INVALID_ARG;
    return conv_common(X, packed_high, 0, 1, n_bits, h_bits, d, w_scale, act_scale, bias, nullptr, Yq, nq::kOutI8, workspace,
                       workspace_bytes, stream, &oq, packed_low);
}

int nq_conv_implicit_gemm_q8(const int8_t* X, const void* Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                             const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                             float out_scale, int relu, int8_t* Yq, void* workspace, int64_t workspace_bytes, void* stream) {
    const nq::OutQuant oq{out_scale, relu};
    if (!Yq) return NQ_ERR_INVALID_ARG;
    return conv_common(X, Wt, ldw, part_bit, n_bits, h_bits, d, w_scale, act_scale, bias, nullptr, Yq, nq::kOutI8, workspace,
                       workspace_bytes, stream, &oq);
}

int nq_conv_implicit_gemm_q8_res(const int8_t* X, const void* Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                                 const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                                 const int8_t* residual, float residual_scale, float out_scale, int relu, int8_t* Yq,
                                 void* workspace, int64_t workspace_bytes, void* stream) {
    const nq::OutQuant oq{out_scale, relu, residual, residual_scale};
    if (!Yq || !residual) return NQ_ERR_INVALID_ARG;
    return conv_common(X, Wt, ldw, part_bit, n_bits, h_bits, d, w_scale, act_scale, bias, nullptr, Yq, nq::kOutI8, workspace,
                       workspace_bytes, stream, &oq);
}

int nq_conv_implicit_gemm_nested_q8_res(const int8_t* X, const void* packed_high, const void* packed_low, int n_bits,
                                        int h_bits, const nq_conv_desc* d, const float* w_scale, float act_scale,
                                        const float* bias, const int8_t* residual, float residual_scale, float out_scale,
                                        int relu, int8_t* Yq, void* workspace, int64_t workspace_bytes, void* stream) {
    const nq::OutQuant oq{out_scale, relu, residual, residual_scale};
    if (!Yq || !packed_low || !residual) return NQ_ERR_INVALID_ARG;
    return conv_common(X, packed_high, 0, 1, n_bits, h_bits, d, w_scale, act_scale, bias, nullptr, Yq, nq::kOutI8, workspace,
                       workspace_bytes, stream, &oq, packed_low);
}

int nq_conv_implicit_gemm_static(const int8_t* X, const void* Wt, int64_t ldw, int part_bit, int n_bits, int h_bits,
                                 const nq_conv_desc* d, const float* w_scale, float act_scale, const float* bias,
                                 int32_t* acc_out, void* Y, int y_dtype, void* stream) {
    const int64_t need = nq_conv_workspace_bytes(d);
    if (need < 0) return NQ_ERR_INVALID_ARG;
    if (need > (int64_t)NQ_CONV_STATIC_SCRATCH_BYTES) return NQ_ERR_WORKSPACE;   // does not fit the built-in staging array
    // device address of the array, looked up once per device with that device current
    // (atomic slots: two host threads that both make a device's first call store the same address)
    static std::atomic<unsigned char*> base[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NQ_ERR_CUDA;
    unsigned char* ptr = base[dev].load(std::memory_order_relaxed);
    if (!ptr) {
        if (cudaGetSymbolAddress((void**)&ptr, g_conv_static_scratch) != cudaSuccess || !ptr) return NQ_ERR_CUDA;
        base[dev].store(ptr, std::memory_order_relaxed);
    }
    unsigned char* ws = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(ptr) + 1023) & ~uintptr_t(1023));
    return nq_conv_implicit_gemm(X, Wt, ldw, part_bit, n_bits, h_bits, d, w_scale, act_scale, bias, acc_out, Y, y_dtype,
                                 ws, NQ_CONV_STATIC_SCRATCH_BYTES, stream);
}

}  // extern "C"
