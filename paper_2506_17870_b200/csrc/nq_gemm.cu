// Host side of the nested GEMM entry points: argument checks, TMA descriptors, launch.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/nq.h"

#include "nq_contraction_pair.cuh"
#include "nq_internal.cuh"

namespace nq {

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn encode_fn() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess || !sym ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeFn>(sym);
    }
    return fn;
}
CUtensorMapSwizzle swizzle_of(int bytes) {
    return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE;
}
}  // namespace

int encode_tensor_map_2d(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_bytes,
                         uint32_t box_inner, uint32_t box_outer, int swizzle_bytes) {
    EncodeFn fn = encode_fn();
    if (!fn) return NQ_ERR_CUDA;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NQ_OK : NQ_ERR_CUDA;
}

int encode_tensor_map_nhwc(CUtensorMap* map, const void* base, uint64_t C, uint64_t W, uint64_t H, uint64_t B,
                           uint32_t box_c, uint32_t tw, uint32_t th, uint32_t tb, uint32_t stride, int swizzle_bytes) {
    EncodeFn fn = encode_fn();
    if (!fn) return NQ_ERR_CUDA;
    cuuint64_t dims[4] = {C, W, H, B};
    cuuint64_t strides[3] = {C, C * W, C * W * H};
    // the box spans (t - 1) * stride + 1 input positions, of which every stride-th is taken: t elements
    cuuint32_t box[4] = {box_c, (tw - 1) * stride + 1, (th - 1) * stride + 1, tb};
    cuuint32_t estr[4] = {1, stride, stride, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NQ_OK : NQ_ERR_CUDA;
}

int encode_tensor_map_out(CUtensorMap* map, const void* base, uint64_t row_bytes, uint64_t pitch_bytes, uint64_t d1,
                          uint64_t d2, uint64_t d3, uint32_t b1, uint32_t b2, uint32_t b3, uint32_t box_bytes) {
    EncodeFn fn = encode_fn();
    if (!fn) return NQ_ERR_CUDA;
    cuuint64_t dims[4] = {row_bytes, d1, d2, d3};
    cuuint64_t strides[3] = {pitch_bytes, pitch_bytes * d1, pitch_bytes * d1 * d2};
    cuuint32_t box[4] = {box_bytes, b1, b2, b3};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, box_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NQ_OK : NQ_ERR_CUDA;
}

namespace {

// The two output maps of a launch (Y and the int32 accumulators); a map that is not used is a copy of tmA, so
// that the kernel parameter is always a valid descriptor.
struct OutMaps {
    CUtensorMap y, acc;
};

template <int BN, bool PART, int MODE>
int launch(const CUtensorMap& tmA, const CUtensorMap& tmB, const OutMaps& om, const ContractionArgs& a, cudaStream_t stream) {
    const int smem = contraction_smem_bytes(BN, PART, a.h_bits, a.packed_stages);
    static int configured[64] = {0};       // largest opt-in done so far, per device, for this instantiation
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NQ_ERR_CUDA;
    if (smem > configured[dev]) {
        if (cudaFuncSetAttribute(contraction_kernel<BN, PART, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 smem) != cudaSuccess)
            return NQ_ERR_CUDA;
        configured[dev] = smem;
    }
    const int tiles = a.m_tiles * a.n_tiles;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    contraction_kernel<BN, PART, MODE><<<grid, contraction_threads(PART), smem, stream>>>(tmA, tmB, om.y, om.acc, a);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

template <int BN, bool PART>
int launch_mode(int mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const OutMaps& om, const ContractionArgs& a,
                cudaStream_t s) {
    if (mode == kModeConv128) return launch<BN, PART, kModeConv128>(tmA, tmB, om, a, s);
    if (mode == kModeConv64) return launch<BN, PART, kModeConv64>(tmA, tmB, om, a, s);
    return launch<BN, PART, kModeGemm>(tmA, tmB, om, a, s);
}

// CTA-pair kernel: a cluster of two CTAs per 256 x 256 tile
template <bool PART, int MODE, bool DIRECT = false, int NEST = 0>
int launch_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const OutMaps& om, const ContractionArgs& a,
                cudaStream_t stream) {
    const int smem = pair_smem_bytes(PART, a.ring_bits, a.packed_stages);
    static int configured[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return NQ_ERR_CUDA;
    if (smem > configured[dev]) {
        if (cudaFuncSetAttribute(contraction_pair_kernel<PART, MODE, DIRECT, NEST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 smem) != cudaSuccess)
            return NQ_ERR_CUDA;
        configured[dev] = smem;
    }
    const int tiles = a.m_tiles * a.n_tiles;
    const int max_pairs = sm_count() / 2;
    const int pairs = tiles < max_pairs ? tiles : max_pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(pair_threads(PART, DIRECT), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, contraction_pair_kernel<PART, MODE, DIRECT, NEST>, tmA, tmB, om.y, om.acc, a) != cudaSuccess) {
        (void)cudaGetLastError();
        return NQ_ERR_CUDA;
    }
    return NQ_OK;
}

template <bool PART, bool DIRECT = false>
int launch_pair_mode(int mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const OutMaps& om, const ContractionArgs& a,
                     cudaStream_t s) {
    if (mode == kModeConv128) return launch_pair<PART, kModeConv128, DIRECT>(tmA, tmB, om, a, s);
    if (mode == kModeConv64) return launch_pair<PART, kModeConv64, DIRECT>(tmA, tmB, om, a, s);
    return launch_pair<PART, kModeGemm, DIRECT>(tmA, tmB, om, a, s);
}

// Test switches (nq_debug_set): keep the epilogue on ordinary global stores / keep every part-bit pair launch on the
// TMA-fed ring of packed tiles, so that tests can compare those paths with the default ones bit for bit.
int g_debug[2] = {0, 0};
bool tile_stores_enabled() { return g_debug[NQ_DEBUG_PLAIN_STORES] == 0; }
bool direct_fetch_enabled() { return g_debug[NQ_DEBUG_PACKED_RING] == 0; }

// Tile-store map of one output ([M, N] of esize-byte elements, pitch ld): possible when base and pitch are
// 16-byte aligned.  Convolution outputs are NHWC, addressed by (pixel column, pixel row, image) in boxes that
// match the 32 consecutive tile rows of an epilogue warp.
bool make_out_map(CUtensorMap* map, const void* base, int esize, int64_t M, int64_t N, int64_t ld, const ConvGeom* g) {
    if (!base || !tile_stores_enabled()) return false;
    const uint64_t pitch = (uint64_t)ld * esize, row_bytes = (uint64_t)N * esize;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || (pitch & 15) || pitch >= (1ull << 40)) return false;
    const uint32_t box_bytes = esize == 1 ? 32 : 64;      // 32 columns of the output
    if (!g) return encode_tensor_map_out(map, base, row_bytes, pitch, (uint64_t)M, 1, 1, 32, 1, 1, box_bytes) == NQ_OK;
    const uint32_t tw = 1u << g->tw_log2, th = 1u << g->th_log2;
    const uint32_t bw = tw < 32 ? tw : 32;
    const uint32_t bh = (32 / bw) < th ? (32 / bw) : th;
    const uint32_t bb = 32 / (bw * bh);
    return encode_tensor_map_out(map, base, row_bytes, pitch, (uint64_t)g->Wo, (uint64_t)g->Ho, (uint64_t)g->B, bw, bh, bb,
                                 box_bytes) == NQ_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

// The A operand is reached through tmA, built by the caller: a plain 2-D map of an [M, K] matrix
// (kModeGemm, geom == nullptr) or a 4-D map of NHWC activations (convolution modes, geom given; then M
// tiles are geom's pixel rectangles and k_blocks follows the filter taps).
int run_contraction(const CUtensorMap& tmA, int mode, const ConvGeom* geom, int m_tiles, int k_blocks,
                    const void* Bmat, int64_t ldb, bool part, int n_bits, int h_bits,
                    const float* w_scale, float act_scale, const float* bias, int64_t M, int64_t N, int64_t K,
                    int32_t* acc_out, int64_t ld_acc, void* Y, int64_t ldy, int y_dtype, cudaStream_t stream,
                    const OutQuant* oq, const void* Blow) {
    // Blow given: nested full-bit mode -- Bmat is the packed higher-bit matrix, Blow the packed (l + 1)-bit
    // lower-bit matrix, and the unpack warps of the pair kernel rebuild w_int from both: the
    // wider field through the ring of packed tiles, the narrower one by direct reads.
    const bool nest = Blow != nullptr;
    // Tile shape: the widest tile reuses operands best, but a small problem must first of all fill the
    // machine.  Estimate, for each candidate, (waves of tiles over the SMs) x (stages per tile) x (cycles per
    // stage, measured orders of magnitude: narrow tiles are load-bound, the wide single-CTA tile is
    // shared-memory-bound) and take the cheapest.
    const int sms = sm_count();
    int bn = 64;
    bool pair = false;
    {
        double best = 1e300;
        const int cand_bn[4] = {64, 128, 256, 256};
        const bool cand_pair[4] = {false, false, false, true};
        const double stage_cycles[4] = {260.0, 330.0, 800.0, 560.0};
        for (int c = 0; c < 4; ++c) {
            if (nest && !cand_pair[c]) continue;
            if (cand_pair[c] && !nest && m_tiles < 2) continue;
            if (c > 0 && N <= cand_bn[c - 1] && !(c == 3)) continue;          // no wider than the output needs
            if (c == 3 && N <= 128 && !nest) continue;
            const long long nt = (N + cand_bn[c] - 1) / cand_bn[c];
            const long long tiles = (cand_pair[c] ? (m_tiles + 1) / 2 : m_tiles) * nt;
            const long long slots = cand_pair[c] ? sms / 2 : sms;
            const double waves = (double)((tiles + slots - 1) / slots);
            const double cost = waves * (k_blocks * stage_cycles[c] + 2500.0);   // + per-tile epilogue / fill
            if (cost < best) { best = cost; bn = cand_bn[c]; pair = cand_pair[c]; }
        }
    }
    // Full-bit with short K: a CTA's epilogue warps need a time that does not depend on K for their 128 x 256
    // outputs (about 6500 cycles; 7800 when the accumulator hand-back crosses a CTA pair), so once the MMAs of a tile
    // take less than that the tile is epilogue-bound and single CTAs are faster (measured at M = 50432, K = 768:
    // N = 2304 122 -> 102 us, N = 3072 150 -> 135 us; K = 3072 stays on pairs, 90 against 126 us).
    if (pair && !part && N > 128 && k_blocks * 560.0 < 7800.0) {
        const long long nt = (N + 255) / 256;
        const double waves_pair = (double)((((m_tiles + 1) / 2) * nt + sms / 2 - 1) / (sms / 2));
        const double waves_single = (double)(((long long)m_tiles * nt + sms - 1) / sms);
        const double mma_single = k_blocks * 800.0;
        if (waves_single * (mma_single > 6500.0 ? mma_single : 6500.0) < waves_pair * 7800.0) { pair = false; bn = 256; }
    }
    const int b_box_rows = pair ? kPairBN / 2 : bn;
    ContractionArgs a{};
    if (geom) a.g = *geom;
    a.M = (int)M; a.N = (int)N; a.K = (int)K;
    a.m_tiles = pair ? (m_tiles + 1) / 2 : m_tiles;
    a.n_tiles = (int)((N + bn - 1) / bn);
    a.k_blocks = k_blocks;
    // Rasterisation: a group of M-tiles shares a band of N-tiles, so that the group's rows of A stay in L2 while the
    // N-tiles go by.  The band must fit beside the stream of B and the output: about 32 MB of A rows per group
    // (16 M-tiles up to K = 8192 on pairs; 8 at K = 16384, where 16 made every wave re-read its 67 MB band: measured
    // 5.2-7.0 GB of DRAM traffic per 16384^3 launch against 1.07 GB algorithmic).
    {
        const double band_rows = (pair ? 256.0 : 128.0) * kGroupM;
        int gl = 4;
        while (gl > 2 && band_rows / kGroupM * (1 << gl) * (double)K > 34.0e6) --gl;
        a.group_log2 = gl;
    }
    a.div_group = make_fastdiv((uint32_t)((1 << a.group_log2) * a.n_tiles));
    a.div_last = make_fastdiv((uint32_t)((a.m_tiles % (1 << a.group_log2)) ? (a.m_tiles % (1 << a.group_log2)) : 1));
    a.w_scale = w_scale; a.bias = bias; a.act_scale = act_scale;
    a.acc_out = acc_out; a.ld_acc = ld_acc; a.y = Y; a.ldy = ldy; a.y_is_bf16 = (y_dtype == NQ_BF16);
    a.y_is_i8 = (y_dtype == kOutI8 && oq) ? 1 : 0;
    a.relu = oq ? oq->relu : 0;
    a.inv_out_scale = oq ? 1.0f / oq->out_scale : 1.0f;
    a.residual = (oq && a.y_is_i8) ? oq->residual : nullptr;      // dense, like the output
    a.ld_res = N;
    a.res_scale = oq ? oq->res_scale : 0.0f;
    a.status = status_word();
    if (!a.status) return NQ_ERR_CUDA;
    OutMaps om;
    om.y = tmA; om.acc = tmA;
    a.y_tma = make_out_map(&om.y, Y, a.y_is_i8 ? 1 : (y_dtype == NQ_BF16 ? 2 : 4), M, N, ldy, geom) ? 1 : 0;
    a.acc_tma = make_out_map(&om.acc, acc_out, 4, M, N, ld_acc, geom) ? 1 : 0;
    CUtensorMap tmB;
    bool direct = false;
    if (part) {
        const int l = n_bits - h_bits;
        a.pow2_l = nest ? 1.0f : (float)(1 << l);
        a.acc_shift = nest ? 8 - n_bits : 8 - h_bits;        // nested: w_int sits in the top n bits of the byte
        a.unshift = 1.0f / (float)(1 << a.acc_shift);
        a.h_bits = h_bits;
        // as deep a ring of packed tiles as shared memory allows: it is what hides the load latency of B
        // (pair kernel: a multiple of its unpack group count, see nq_contraction_pair.cuh)
        a.packed_stages = 0;
        // pair kernel, part-bit: fields of 1, 2 and 4 bits are read straight from the packed tensor's blocks (one
        // coalesced load per 32 fields); wider fields come through the ring, whose slots are filled by one bulk copy
        // per block (measured, 16384^3: direct reads of h = 5 / 6 / 7 need two or three loads per unit in flight for
        // four stages and fall to 2.3 / 2.3 / 1.75 POP/s against 2.97 / 2.64 / 2.35 through the ring)
        direct = !nest && pair && (h_bits == 1 || h_bits == 2 || h_bits == 4) && direct_fetch_enabled();
        const bool high_in_ring = !nest || h_bits > l + 1;
        const int ring_bits = high_in_ring ? h_bits : l + 1;
        const int direct_bits = nest ? (high_in_ring ? l + 1 : h_bits) : h_bits;
        const void* ring_mat = high_in_ring ? Bmat : Blow;
        const void* direct_mat = nest ? (high_in_ring ? Blow : Bmat) : Bmat;
        const bool ring2 = nest && direct_bits == 3;
        a.ring2 = ring2 ? 1 : 0;
        a.ring_field_bits = ring_bits;
        a.ring_bits = ring_bits + (ring2 ? 1 : 0);
        const int step = pair ? kUnpackGroups : 1;
        for (int d = direct ? 0 : kMaxPackedStages; d >= step; d -= step)
            if ((pair ? pair_smem_bytes(true, a.ring_bits, d) : contraction_smem_bytes(bn, true, h_bits, d)) <= kSmemLimit) {
                a.packed_stages = d;
                break;
            }
        if (a.packed_stages == 0 && !direct) return NQ_ERR_UNSUPPORTED;
        a.packed_b = static_cast<const uint8_t*>(direct_mat);     // read directly by the unpack warps (DIRECT, nested)
        a.ring_b = static_cast<const uint8_t*>(ring_mat);         // copied block by block into the ring of packed tiles
        a.packed_groups = (int)((K + 127) / 128);
        a.packed_blocks = (int)((N + 127) / 128);
        tmB = tmA;                                                // packed operands need no tensor map: blocks are contiguous
    } else {
        a.pow2_l = 1.0f; a.unshift = 1.0f; a.acc_shift = 0; a.h_bits = 0;
        int st = (mode == kModeConv64)
                     ? encode_tensor_map_2d(&tmB, Bmat, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, 64, b_box_rows, 64)
                     : encode_tensor_map_2d(&tmB, Bmat, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, kBK, b_box_rows, 128);
        if (st != NQ_OK) return st;
    }
    if (nest) {
        if (!pair) return NQ_ERR_UNSUPPORTED;
        if (mode == kModeConv128)
            return n_bits == 8 ? launch_pair<true, kModeConv128, false, 8>(tmA, tmB, om, a, stream)
                               : launch_pair<true, kModeConv128, false, 6>(tmA, tmB, om, a, stream);
        if (mode == kModeConv64)
            return n_bits == 8 ? launch_pair<true, kModeConv64, false, 8>(tmA, tmB, om, a, stream)
                               : launch_pair<true, kModeConv64, false, 6>(tmA, tmB, om, a, stream);
        return n_bits == 8 ? launch_pair<true, kModeGemm, false, 8>(tmA, tmB, om, a, stream)
                           : launch_pair<true, kModeGemm, false, 6>(tmA, tmB, om, a, stream);
    }
    if (pair && direct) return launch_pair_mode<true, true>(mode, tmA, tmB, om, a, stream);
    if (pair) return part ? launch_pair_mode<true>(mode, tmA, tmB, om, a, stream) : launch_pair_mode<false>(mode, tmA, tmB, om, a, stream);
    if (part) {
        if (bn == 256) return launch_mode<256, true>(mode, tmA, tmB, om, a, stream);
        if (bn == 128) return launch_mode<128, true>(mode, tmA, tmB, om, a, stream);
        return launch_mode<64, true>(mode, tmA, tmB, om, a, stream);
    }
    if (bn == 256) return launch_mode<256, false>(mode, tmA, tmB, om, a, stream);
    if (bn == 128) return launch_mode<128, false>(mode, tmA, tmB, om, a, stream);
    return launch_mode<64, false>(mode, tmA, tmB, om, a, stream);
}

namespace {

int gemm_common(const int8_t* X, int64_t ldx, const void* Bmat, int64_t ldb, bool part, int n_bits, int h_bits,
                const float* w_scale, float act_scale, const float* bias, int64_t M, int64_t N, int64_t K,
                int32_t* acc_out, int64_t ld_acc, void* Y, int64_t ldy, int y_dtype, void* stream,
                const OutQuant* oq = nullptr, const void* Blow = nullptr) {
    if (M < 0 || N < 0 || K < 0) return NQ_ERR_INVALID_ARG;
    if (y_dtype != NQ_F32 && y_dtype != NQ_BF16 && !(y_dtype == kOutI8 && oq)) return NQ_ERR_INVALID_ARG;
    if (oq && !(oq->out_scale > 0.0f)) return NQ_ERR_INVALID_ARG;
    if (part && (n_bits < 2 || n_bits > 8 || h_bits < 1 || h_bits >= n_bits)) return NQ_ERR_UNSUPPORTED;
    if (Blow && ((n_bits != 8 && n_bits != 6) || h_bits < 2)) return NQ_ERR_UNSUPPORTED;
    if (Blow && !aligned16(Blow)) return NQ_ERR_ALIGNMENT;
    if (K >= (1 << 17) || M > (1ll << 30) || N > (1ll << 30)) return NQ_ERR_UNSUPPORTED;
    if (M == 0 || N == 0) return NQ_OK;
    if (!acc_out && !Y) return NQ_ERR_INVALID_ARG;
    if (!w_scale && Y) return NQ_ERR_INVALID_ARG;
    if ((acc_out && ld_acc < N) || (Y && ldy < N)) return NQ_ERR_INVALID_ARG;
    if (K == 0) return NQ_ERR_UNSUPPORTED;
    if (!X || !Bmat || ldx < K || (!part && ldb < K)) return NQ_ERR_INVALID_ARG;
    if (!aligned16(X) || (ldx & 15) || !aligned16(Bmat) || (!part && (ldb & 15))) return NQ_ERR_ALIGNMENT;
    if ((acc_out && (reinterpret_cast<uintptr_t>(acc_out) & 3)) || (Y && y_dtype != kOutI8 && (reinterpret_cast<uintptr_t>(Y) & 1)))
        return NQ_ERR_ALIGNMENT;
    CUtensorMap tmA;
    int st = encode_tensor_map_2d(&tmA, X, (uint64_t)K, (uint64_t)M, (uint64_t)ldx, kBK, kBM, 128);
    if (st != NQ_OK) return st;
    return run_contraction(tmA, kModeGemm, nullptr, (int)((M + kBM - 1) / kBM), (int)((K + kBK - 1) / kBK), Bmat, ldb,
                           part, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, acc_out, ld_acc, Y, ldy, y_dtype,
                           (cudaStream_t)stream, oq, Blow);
}

}  // namespace
}  // namespace nq

extern "C" {

int nq_debug_set(int which, int enabled) {
    if (which != NQ_DEBUG_PLAIN_STORES && which != NQ_DEBUG_PACKED_RING) return NQ_ERR_INVALID_ARG;
    nq::g_debug[which] = enabled ? 1 : 0;
    return NQ_OK;
}

int nq_gemm_full(const int8_t* X, int64_t ldx, const int8_t* W, int64_t ldw, const float* w_scale, float act_scale,
                 const float* bias, int64_t M, int64_t N, int64_t K, int32_t* acc_out, int64_t ld_acc, void* Y,
                 int64_t ldy, int y_dtype, void* stream) {
    return nq::gemm_common(X, ldx, W, ldw, false, 8, 0, w_scale, act_scale, bias, M, N, K, acc_out, ld_acc, Y, ldy,
                           y_dtype, stream);
}

int nq_gemm_full_q8(const int8_t* X, int64_t ldx, const int8_t* W, int64_t ldw, const float* w_scale, float act_scale,
                    const float* bias, float out_scale, int relu, int64_t M, int64_t N, int64_t K, int8_t* Yq,
                    int64_t ldyq, void* stream) {
    const nq::OutQuant oq{out_scale, relu};
    if (!Yq) return NQ_ERR_INVALID_ARG;
    return nq::gemm_common(X, ldx, W, ldw, false, 8, 0, w_scale, act_scale, bias, M, N, K, nullptr, 0, Yq, ldyq, nq::kOutI8,
                           stream, &oq);
}

int nq_gemm_part_q8(const int8_t* X, int64_t ldx, const void* packed_high, int n_bits, int h_bits, const float* w_scale,
                    float act_scale, const float* bias, float out_scale, int relu, int64_t M, int64_t N, int64_t K,
                    int8_t* Yq, int64_t ldyq, void* stream) {
    const nq::OutQuant oq{out_scale, relu};
    if (!Yq) return NQ_ERR_INVALID_ARG;
    return nq::gemm_common(X, ldx, packed_high, 0, true, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, nullptr, 0, Yq,
                           ldyq, nq::kOutI8, stream, &oq);
}

int nq_gemm_nested(const int8_t* X, int64_t ldx, const void* packed_high, const void* packed_low, int n_bits, int h_bits,
                   const float* w_scale, float act_scale, const float* bias, int64_t M, int64_t N, int64_t K,
                   int32_t* acc_out, int64_t ld_acc, void* Y, int64_t ldy, int y_dtype, void* stream) {
    if (!packed_low) return (M == 0 || N == 0) && M >= 0 && N >= 0 && K >= 0 ? NQ_OK : NQ_ERR_INVALID_ARG;
    return nq::gemm_common(X, ldx, packed_high, 0, true, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, acc_out,
                           ld_acc, Y, ldy, y_dtype, stream, nullptr, packed_low);
}

int nq_gemm_nested_q8(const int8_t* X, int64_t ldx, const void* packed_high, const void* packed_low, int n_bits, int h_bits,
                      const float* w_scale, float act_scale, const float* bias, float out_scale, int relu, int64_t M,
                      int64_t N, int64_t K, int8_t* Yq, int64_t ldyq, void* stream) {
    const nq::OutQuant oq{out_scale, relu};
    if (!Yq || !packed_low) return NQ_ERR_INVALID_ARG;
    return nq::gemm_common(X, ldx, packed_high, 0, true, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, nullptr, 0, Yq,
                           ldyq, nq::kOutI8, stream, &oq, packed_low);
}

int nq_gemm_part(const int8_t* X, int64_t ldx, const void* packed_high, int n_bits, int h_bits, const float* w_scale,
                 float act_scale, const float* bias, int64_t M, int64_t N, int64_t K, int32_t* acc_out, int64_t ld_acc,
                 void* Y, int64_t ldy, int y_dtype, void* stream) {
    return nq::gemm_common(X, ldx, packed_high, 0, true, n_bits, h_bits, w_scale, act_scale, bias, M, N, K, acc_out,
                           ld_acc, Y, ldy, y_dtype, stream);
}

}  // extern "C"
