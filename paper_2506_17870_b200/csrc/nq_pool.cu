// Pooling between the layers of a chained model: INT8 NHWC activations in, INT8 out.  Both kernels are plain
// bandwidth-bound passes (the stem's max pooling reads 4 x what it writes; the global average reads a 7 x 7 map).
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"

namespace {

// One thread per output pixel and group of 16 channels: 16-byte loads of every tap inside the image, per-byte
// signed maximum.  Taps outside the image are skipped (padding never wins).
__global__ void __launch_bounds__(256) maxpool_nhwc_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int B, int H, int W,
                                                           int C, int ksize, int stride, int pad, int Ho, int Wo, long long total) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int groups = (C + 15) / 16;
    const int g = (int)(idx % groups);
    long long t = idx / groups;
    const int q = (int)(t % Wo);
    t /= Wo;
    const int p = (int)(t % Ho), b = (int)(t / Ho);
    const int c0 = g * 16;
    const bool vec = ((C & 15) == 0) && ((reinterpret_cast<uintptr_t>(x) & 15) == 0) && ((reinterpret_cast<uintptr_t>(y) & 15) == 0);
    int8_t* dst = y + (((long long)b * Ho + p) * Wo + q) * C + c0;
    if (vec) {
        uint32_t m[4] = {0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u};      // -128 in every byte
        for (int r = 0; r < ksize; ++r) {
            const int ih = p * stride - pad + r;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < ksize; ++s) {
                const int iw = q * stride - pad + s;
                if (iw < 0 || iw >= W) continue;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + (((long long)b * H + ih) * W + iw) * C + c0));
                m[0] = __vmaxs4(m[0], v.x); m[1] = __vmaxs4(m[1], v.y); m[2] = __vmaxs4(m[2], v.z); m[3] = __vmaxs4(m[3], v.w);
            }
        }
        *reinterpret_cast<uint4*>(dst) = make_uint4(m[0], m[1], m[2], m[3]);
    } else {
        for (int j = 0; j < 16 && c0 + j < C; ++j) {
            int best = -128;
            for (int r = 0; r < ksize; ++r) {
                const int ih = p * stride - pad + r;
                if (ih < 0 || ih >= H) continue;
                for (int s = 0; s < ksize; ++s) {
                    const int iw = q * stride - pad + s;
                    if (iw < 0 || iw >= W) continue;
                    const int v = x[(((long long)b * H + ih) * W + iw) * C + c0 + j];
                    best = v > best ? v : best;
                }
            }
            dst[j] = (int8_t)best;
        }
    }
}

// One thread per (image, channel): integer sum over the map (adjacent threads read adjacent channels), then
// a = fl(in_scale / (H * W)), t = fl(fl(float(sum) * a) * inv_out), round half to even, clip.
__global__ void __launch_bounds__(256) avgpool_requant_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ y, int B, int HW,
                                                              int C, float a, float inv_out) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * C) return;
    const int b = idx / C, c = idx - b * C;
    const int8_t* src = x + (long long)b * HW * C + c;
    int sum = 0;
    for (int i = 0; i < HW; ++i) sum += src[(long long)i * C];
    const float t = __fmul_rn(__fmul_rn(__int2float_rn(sum), a), inv_out);
    int qv = __float2int_rn(t);
    qv = qv < -128 ? -128 : (qv > 127 ? 127 : qv);
    y[idx] = (int8_t)qv;
}

}  // namespace

extern "C" {

int nq_maxpool_nhwc_i8(const int8_t* X, int B, int H, int W, int C, int ksize, int stride, int pad, int8_t* Y, void* stream) {
    if (B < 0 || H <= 0 || W <= 0 || C <= 0 || ksize <= 0 || stride <= 0 || pad < 0 || pad >= ksize ||
        H + 2 * pad < ksize || W + 2 * pad < ksize)
        return NQ_ERR_INVALID_ARG;
    if (B == 0) return NQ_OK;
    if (!X || !Y) return NQ_ERR_INVALID_ARG;
    const int Ho = (H + 2 * pad - ksize) / stride + 1, Wo = (W + 2 * pad - ksize) / stride + 1;
    const long long total = (long long)B * Ho * Wo * ((C + 15) / 16);
    if (total > (1ll << 40)) return NQ_ERR_UNSUPPORTED;
    maxpool_nhwc_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(X, Y, B, H, W, C, ksize, stride, pad,
                                                                                           Ho, Wo, total);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

int nq_avgpool_requant_nhwc_i8(const int8_t* X, int B, int H, int W, int C, float in_scale, float out_scale, int8_t* Y,
                               void* stream) {
    if (B < 0 || H <= 0 || W <= 0 || C <= 0 || !(out_scale > 0.0f) || (long long)H * W > (1 << 23)) return NQ_ERR_INVALID_ARG;
    if (B == 0) return NQ_OK;
    if (!X || !Y || (long long)B * C > 0x7fffffffLL) return NQ_ERR_INVALID_ARG;
    const float a = in_scale / (float)(H * W);          // one IEEE division each, as the definition says
    const float inv_out = 1.0f / out_scale;
    avgpool_requant_kernel<<<(B * C + 255) / 256, 256, 0, (cudaStream_t)stream>>>(X, Y, B, H * W, C, a, inv_out);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

}  // extern "C"
