// The INT8 contraction kernel shared by the GEMM and the implicit-GEMM convolution.
//
//   acc[m, j] = sum_k A[m, k] * B[j, k]   (int8 x int8 -> int32 on the tcgen05 tensor cores)
//   Y[m, j]   = float(acc) * scale[j] (+ bias[j])       fused epilogue, fp32 or bf16
//
// One persistent CTA per SM walks a list of 128 x BN output tiles.  Roles (warp-specialised):
//   warp 0      TMA producer: A tile (128 rows x 128 B) and B tile (BN rows x 128 B, or the packed
//               INTh tile in part-bit mode) into a ring of shared-memory stages
//   warp 1      MMA issuer: one thread issues four tcgen05.mma kind::i8 (K = 32 each) per stage into
//               a TMEM accumulator; owns the TMEM allocation
//   warps 2-9   epilogue: tcgen05.ld the accumulator (each warp a 32-lane quarter and half of the columns), scale, store.
//               Two accumulators alternate so the epilogue of tile i overlaps the MMAs of tile i+1
//   warps 10-17 (part-bit only) unpackers: expand packed INTh fields into the swizzled int8 B tile.
//               The field goes to the TOP h bits of the byte, i.e. the byte is w_high * 2^(8-h); the
//               accumulator is then 2^(8-h) times too large, exactly, and the epilogue takes it out
//               (arithmetic shift for the int32 output, an exact power-of-two factor in the scale).
// Every mbarrier wait is bounded (see mbar_wait); when one gives up every role leaves its loop,
// the block joins, frees its TMEM and returns, and the host can read the record.  Every TMA load
// has a single destination CTA.
#pragma once
#include <cuda_bf16.h>

#include "nq_sm100.cuh"

namespace nq {

constexpr int kBM = 128;           // tile rows (M) = TMEM lanes
constexpr int kBK = 128;           // K bytes per stage = one 128-byte swizzle row
// Ring depth by tile width: narrow tiles have small stages and little work per stage, so they need more of
// them in flight to cover the load latency (full-bit 8 / 6 / 4 stages of 24 / 32 / 48 KB; part-bit leaves
// room for the packed ring).
__host__ __device__ constexpr int stages_for(int bn, bool part) {
    return part ? (bn == 64 ? 6 : bn == 128 ? 4 : 3) : (bn == 64 ? 8 : bn == 128 ? 6 : 4);
}
constexpr int kMaxPackedStages = 8;     // ring of packed (still INTh) B tiles; the depth in use is chosen by the host
constexpr int kGroupM = 16;        // tile rasterisation: at most 16 M-tiles share a band of N-tiles (the host picks 4, 8 or 16)

// How the A operand is gathered.
//   kModeGemm    A is a plain [M, K] matrix: one 2-D tile per stage.
//   kModeConv128 implicit GEMM, Cin a multiple of 128: a stage is 128 channels of ONE filter tap for a
//                tw x th x tb rectangle of output pixels, fetched by one 4-D tile load from the NHWC tensor.
//   kModeConv64  implicit GEMM, Cin = 64: a stage is TWO taps x 64 channels, held as two sub-tiles of
//                64-byte rows (64-byte swizzle) for A and for B alike.
constexpr int kModeGemm = 0, kModeConv128 = 1, kModeConv64 = 2;

struct ConvGeom {
    int B, Ho, Wo, S, taps, stride, pad;
    int cblocks;                     // kModeConv128: Cin / 128
    int tw_log2, th_log2;            // tile = 2^tw x 2^th output pixels of 128 / (2^tw * 2^th) images
    int tiles_w, tiles_h;
};

// Division by a number fixed at launch: q = (umulhi(n, magic) + n) >> shift, exact for n < 2^31 (magic = 0 for a
// power of two).  The tile walk of every role divides twice per tile; the hardware's integer division cost the
// epilogue warps about as much as one of their four output chunks.
struct FastDiv {
    uint32_t magic, shift;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f{0u, 0u};
    while ((1u << f.shift) < d) ++f.shift;
    if ((1u << f.shift) != d) f.magic = (uint32_t)(((1ull << 32) * ((1ull << f.shift) - d)) / d + 1);
    return f;
}
__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f) { return (__umulhi(n, f.magic) + n) >> f.shift; }

struct ContractionArgs {
    ConvGeom g;
    int M, N, K;
    int m_tiles, n_tiles, k_blocks;
    int group_log2;                // M-tiles per rasterisation group = 2^group_log2
    FastDiv div_group, div_last;   // by (group size) * n_tiles, and by the row count of the last (short) group of M-tiles
    const float* w_scale;
    const float* bias;
    float act_scale;
    float pow2_l;        // 2^l in part-bit mode, 1 otherwise
    float unshift;       // 2^-(8-h) in part-bit mode, 1 otherwise (exact)
    int acc_shift;       // 8-h in part-bit mode, 0 otherwise
    int h_bits;          // part-bit: width of the packed field
    int packed_stages;   // part-bit: depth of the packed-tile ring (1..kMaxPackedStages)
    // Packed operands (part-bit, nested): tensors in the sliced layout, blocks of 128 rows x 128 fields, 2048 * bits
    // contiguous bytes each, block (rb, g) at ((rb * packed_groups + g) * 2048 * bits).
    const uint8_t* packed_b;   // the tensor the unpack warps read straight from global memory (part-bit: packed_high; nested:
                               // the narrower of the two fields)
    const uint8_t* ring_b;     // the tensor that comes through the shared-memory ring (part-bit: packed_high; nested: the wider field)
    int packed_groups;         // column groups G = ceil(K / 128) of both
    int packed_blocks;         // row blocks ceil(N / 128) that exist; a tile may reach one block further, which is not read
    int ring_bits;       // bits per field of a ring slot (h_bits in part-bit mode; in nested full-bit mode the wider of the two
                         // fields, plus one when ring2 is set)
    int ring_field_bits; // ... of the tensor behind ring_b
    int ring2;           // nested mode, 3-bit narrow field: its 1-bit slice is copied into the ring slot as well
    int32_t* acc_out;
    long long ld_acc;
    void* y;
    long long ldy;
    int y_is_bf16;
    int y_tma, acc_tma;  // the output is written with tile stores through tmY / tmAcc (aligned base and pitch)
    int y_is_i8;         // requantised INT8 output: q = clip(rint(fl(relu(v) * inv_out_scale)))
    int relu;
    float inv_out_scale;
    const int8_t* residual;   // requantised output only: INT8 skip tensor [M, N], row pitch ld_res, added dequantised
    long long ld_res;         //   (fl(float(r) * res_scale)) before the activation; nullptr = none
    float res_scale;
    unsigned int* status;
};

// Thread layout of a block: warp 0 producer, warp 1 MMA issuer, then the epilogue warps, then (part-bit) the
// unpack warps.  Eight epilogue warps: two per TMEM lane quarter, each taking half of the tile's columns -- a
// single warp per scheduler cannot hide the latency of its own convert-and-store chain (measured: the
// epilogue, not the stores, capped output-bound problems at 1.3 TB/s with four warps).
constexpr int kEpiWarps = 8;
constexpr int kFirstUnpackWarp = 2 + kEpiWarps;
constexpr int kBaseThreads = (2 + kEpiWarps) * 32;
// Output staging of one epilogue warp: 32 rows x 64 bytes, rows 80 bytes apart (an odd multiple of 16 keeps
// the row-wise writes free of bank conflicts).
constexpr int kEpiRowPitch = 80;
constexpr int kEpiStageBytes = 32 * kEpiRowPitch;

__host__ __device__ constexpr int a_stage_bytes() { return kBM * kBK; }
__host__ __device__ constexpr int b_stage_bytes(int bn) { return bn * kBK; }

// dynamic shared memory: [A stages][B stages][packed stages][scale + bias per epilogue warp][barriers]
constexpr int kSmemLimit = 227 * 1024;   // dynamic shared memory a block may opt in to

__host__ __device__ inline int contraction_smem_bytes(int bn, bool part, int h_bits, int packed_stages) {
    int stages = stages_for(bn, part);
    int bytes = stages * (a_stage_bytes() + b_stage_bytes(bn));
    if (part) bytes += packed_stages * bn * 16 * h_bits;
    bytes += 4 * 2 * bn * (int)sizeof(float);   // scale and bias: each epilogue warp keeps those of its half of the columns
    bytes += kEpiWarps * kEpiStageBytes;        // output staging, one per epilogue warp
    bytes += 512;                       // barriers, TMEM base, abort flag
    return bytes + 1024;                // slack to align the base to 1024 B
}

__device__ __forceinline__ void tile_coords(int tile, const ContractionArgs& p, int& mt, int& nt) {
    const int gm = 1 << p.group_log2;
    const int per_group = gm * p.n_tiles;
    const int g = (int)fast_div((uint32_t)tile, p.div_group);
    const int first = g * gm;
    const int local = tile - g * per_group;
    if (p.m_tiles - first >= gm) {                       // a full group: its size is a power of two
        mt = first + (local & (gm - 1));
        nt = local >> p.group_log2;
    } else {
        const int gsz = p.m_tiles - first;
        nt = (int)fast_div((uint32_t)local, p.div_last);
        mt = first + local - nt * gsz;
    }
}

// One 32-element unit of packed H-bit fields as it sits in the shared-memory tile ...
struct PackedUnit {
    uint4 a;       // 4-bit slice
    uint2 c;       // 2-bit slice
    uint32_t d;    // 1-bit slice
};
// Out of a ring slot holding ROWS rows of a block slice by slice ([ROWS][64 B] of the 4-bit slice, [ROWS][32 B] of the
// 2-bit slice, [ROWS][16 B] of the 1-bit slice): unit ru = row * 4 + unit.  Consecutive lanes read consecutive pieces.
template <int H, int ROWS>
__device__ __forceinline__ void load_packed_unit(const uint8_t* slot, int ru, PackedUnit& r) {
    int off = 0;
    if (H & 4) { r.a = *reinterpret_cast<const uint4*>(slot + ru * 16); off = ROWS * 64; }
    if (H & 2) { r.c = *reinterpret_cast<const uint2*>(slot + off + ru * 8); off += ROWS * 32; }
    if (H & 1) { r.d = *reinterpret_cast<const uint32_t*>(slot + off + ru * 4); }
}
// ... and its expansion to 32 bytes with the field in the TOP H bits of each byte.  All shifts and masks are
// immediates: the 4-bit slice costs one AND (or shift + AND) per word, every narrower slice one shift and one
// masked OR per word.
template <int H>
__device__ __forceinline__ void expand_packed_unit(const PackedUnit& r, uint32_t (&T)[8]) {
#pragma unroll
    for (int q = 0; q < 8; ++q) T[q] = 0;
    int used = 0;
    if (H & 4) {
        T[0] = r.a.x & 0xf0f0f0f0u; T[1] = (r.a.x << 4) & 0xf0f0f0f0u;
        T[2] = r.a.y & 0xf0f0f0f0u; T[3] = (r.a.y << 4) & 0xf0f0f0f0u;
        T[4] = r.a.z & 0xf0f0f0f0u; T[5] = (r.a.z << 4) & 0xf0f0f0f0u;
        T[6] = r.a.w & 0xf0f0f0f0u; T[7] = (r.a.w << 4) & 0xf0f0f0f0u;
        used = 4;
    }
    if (H & 2) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t word = (q < 4) ? r.c.x : r.c.y;
            const int net = 2 * (q & 3) - used;
            const uint32_t moved = net >= 0 ? (word << net) : (word >> (-net));
            T[q] |= moved & (0xc0c0c0c0u >> used);
        }
        used += 2;
    }
    if (H & 1) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int net = q - used;
            const uint32_t moved = net >= 0 ? (r.d << net) : (r.d >> (-net));
            T[q] |= moved & (0x80808080u >> used);
        }
    }
}

// The same expansion with the field placed SKIP bits below the top of each byte (SKIP + H <= 8).
template <int H, int SKIP>
__device__ __forceinline__ void expand_packed_unit_at(const PackedUnit& r, uint32_t (&T)[8]) {
    static_assert(SKIP >= 0 && SKIP + H <= 8, "field does not fit in a byte");
#pragma unroll
    for (int q = 0; q < 8; ++q) T[q] = 0;
    int used = SKIP;
    if (H & 4) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t word = (q < 2) ? r.a.x : (q < 4) ? r.a.y : (q < 6) ? r.a.z : r.a.w;
            const int net = 4 * (q & 1) - used;
            const uint32_t moved = net >= 0 ? (word << net) : (word >> (-net));
            T[q] = moved & (0xf0f0f0f0u >> used);
        }
        used += 4;
    }
    if (H & 2) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t word = (q < 4) ? r.c.x : r.c.y;
            const int net = 2 * (q & 3) - used;
            const uint32_t moved = net >= 0 ? (word << net) : (word >> (-net));
            T[q] |= moved & (0xc0c0c0c0u >> used);
        }
        used += 2;
    }
    if (H & 1) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int net = q - used;
            const uint32_t moved = net >= 0 ? (r.d << net) : (r.d >> (-net));
            T[q] |= moved & (0x80808080u >> used);
        }
    }
}

// Eq. 5 on 32 fields at once, for INTn weights kept in the top n bits of a byte: T holds w_high * 2^l (the
// higher-bit field at the top of the byte), L the (l+1)-bit compensated lower-bit field ending at bit 8 - n.
// The two overlap in one bit, the lower field's sign: w_int = (hi | lo without its sign bit) - sign bit, a
// per-byte subtraction done on the whole word (bit 7 of every byte is set first so that no borrow crosses a
// byte, and put right afterwards).  The sum is taken modulo 256: for a compensated decomposition Eq. 5 is exact
// and stays inside INTn, so the clip of the definition never acts.
template <int NB, int L1>
__device__ __forceinline__ void recompose_unit(uint32_t (&T)[8], const uint32_t (&L)[8]) {
    static_assert(NB - L1 >= 1 && NB - L1 <= 6, "the sign of the lower field must lie below bit 7");
    constexpr uint32_t SIGN = 0x80808080u >> (NB - L1);
    constexpr uint32_t TOP = 0x80808080u;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const uint32_t v = T[q] | (L[q] & ~SIGN);
        const uint32_t m = L[q] & SIGN;
        T[q] = ((v | TOP) - m) ^ (~v & TOP);
    }
}

// Write the 32 expanded bytes of one unit where the MMA expects them in the swizzled int8 tile of ROWS rows.
template <int ROWS, int MODE>
__device__ __forceinline__ void store_expanded_unit(uint8_t* __restrict__ dst, int row, int unit, const uint32_t (&T)[8]) {
    if (MODE == kModeConv64) {
        // two sub-tiles of 64-byte rows: units 0,1 feed the first, 2,3 the second; 64-byte swizzle
        uint8_t* drow = dst + (unit >> 1) * (ROWS * 64) + row * 64;
        const int sw = (row >> 1) & 3, c = (unit & 1) * 2;
        *reinterpret_cast<uint4*>(drow + ((c ^ sw) << 4)) = make_uint4(T[0], T[1], T[2], T[3]);
        *reinterpret_cast<uint4*>(drow + (((c + 1) ^ sw) << 4)) = make_uint4(T[4], T[5], T[6], T[7]);
    } else {
        uint8_t* drow = dst + row * 128;
        const int sw = row & 7;
        *reinterpret_cast<uint4*>(drow + (((2 * unit) ^ sw) << 4)) = make_uint4(T[0], T[1], T[2], T[3]);
        *reinterpret_cast<uint4*>(drow + (((2 * unit + 1) ^ sw) << 4)) = make_uint4(T[4], T[5], T[6], T[7]);
    }
}

// The same unit fetched straight from a block of the packed tensor in global memory (ru = row-in-block * 4 + unit):
// the 32 lanes of a warp read 512 / 256 / 128 contiguous bytes.  A row past the end of the matrix reads as zeros.
template <int H>
__device__ __forceinline__ void fetch_packed_unit(const uint8_t* block, int ru, bool in_range, PackedUnit& r) {
    r.a = make_uint4(0u, 0u, 0u, 0u); r.c = make_uint2(0u, 0u); r.d = 0u;
    if (!in_range) return;
    int off = 0;
    if (H & 4) { r.a = sm100::ldg_stream_v4(block + ru * 16); off = 8192; }
    if (H & 2) { r.c = sm100::ldg_stream_v2(block + off + ru * 8); off += 4096; }
    if (H & 1) { r.d = sm100::ldg_stream_u32(block + off + ru * 4); }
}

constexpr int kUnpackWarps = 8;
constexpr int kUnpackThreads = kUnpackWarps * 32;

// Expand one packed B tile (ROWS rows x 128 fields, in a ring slot) into the swizzled int8 tile the MMA reads, with
// THREADS threads (tid = 0 .. THREADS-1); four consecutive threads share a row.  A slot holds SLOT_ROWS rows slice by
// slice; tiles of 256 rows are two such runs (two blocks of the packed tensor), one after the other.
template <int ROWS, int MODE, int H, int THREADS>
__device__ __forceinline__ void unpack_tile(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int tid) {
    constexpr int TASKS = ROWS * 4 / THREADS;              // units per thread
    constexpr int CHUNK = TASKS < 4 ? TASKS : 4;           // units whose loads are issued together
    constexpr int SLOT_ROWS = ROWS < 128 ? ROWS : 128;
    static_assert(TASKS >= 1 && TASKS % CHUNK == 0, "tile does not divide over the threads");
#pragma unroll
    for (int base = 0; base < TASKS; base += CHUNK) {
        PackedUnit raw[CHUNK];
#pragma unroll
        for (int i = 0; i < CHUNK; ++i) {
            const int task = (base + i) * THREADS + tid;
            load_packed_unit<H, SLOT_ROWS>(src + (task >> 9) * (2048 * H), task & 511, raw[i]);
        }
#pragma unroll
        for (int i = 0; i < CHUNK; ++i) {
            const int task = (base + i) * THREADS + tid;
            const int row = task >> 2, unit = task & 3;
            uint32_t T[8];
            expand_packed_unit<H>(raw[i], T);
            store_expanded_unit<ROWS, MODE>(dst, row, unit, T);
        }
    }
}

// The packed-tile producer's copies of one ring slot of a ROWS-row tile whose first row is row0 (a multiple of ROWS):
// whole blocks for tiles of 128 and 256 rows, the tile's 64 rows of every slice for tiles of 64 rows.  A block beyond
// the tensor's last is not copied (its rows are beyond N: their products are never stored).  Announces the bytes first.
template <int ROWS>
__device__ __forceinline__ void load_ring_slot(const ContractionArgs& p, uint32_t slot, int row0, int group, uint32_t bar) {
    const int fb = p.ring_field_bits;
    if (ROWS >= 128) {
        const int rb0 = row0 >> 7;
        int n = 0;
        for (int j = 0; j < ROWS / 128; ++j) n += (rb0 + j < p.packed_blocks) ? 1 : 0;
        sm100::mbar_arrive_expect_tx(bar, (uint32_t)(n * 2048 * fb));
        for (int j = 0; j < ROWS / 128; ++j)
            if (rb0 + j < p.packed_blocks)
                sm100::bulk_load(slot + j * 2048 * fb, p.ring_b + ((long long)(rb0 + j) * p.packed_groups + group) * (2048 * fb),
                                 2048 * fb, bar);
    } else {
        const uint8_t* block = p.ring_b + ((long long)(row0 >> 7) * p.packed_groups + group) * (2048 * fb);
        const int r0 = row0 & 127;
        sm100::mbar_arrive_expect_tx(bar, (uint32_t)(ROWS * 16 * fb));
        int done = 0;                                   // bits of the wider slices already placed
        for (int w = 4; w >= 1; w >>= 1) {
            if (!(fb & w)) continue;
            sm100::bulk_load(slot + ROWS * 16 * done, block + 2048 * done + r0 * 16 * w, ROWS * 16 * w, bar);
            done += w;
        }
    }
}

struct TileOrigin {      // where an M-tile starts, in output-pixel coordinates (convolution modes)
    int b0, p0, q0;
};
__device__ __forceinline__ TileOrigin conv_tile_origin(const ConvGeom& g, int mt) {
    TileOrigin o;
    const int qt = mt % g.tiles_w;
    const int rest = mt / g.tiles_w;
    o.q0 = qt << g.tw_log2;
    o.p0 = (rest % g.tiles_h) << g.th_log2;
    o.b0 = (rest / g.tiles_h) << (7 - g.tw_log2 - g.th_log2);
    return o;
}

// Four dequantised values -> four INT8 activations in one word (byte i = value i): one multiply by fl(1 / out_scale),
// round half to even, clip.  The conversion saturates to int32, the packing instruction to INT8; with ReLU the
// packing saturates to [0, 255] instead and a per-byte minimum brings that to [0, 127] (a negative value rounds to
// a non-positive integer, so clipping at zero after the rounding equals ReLU before it).
__device__ __forceinline__ uint32_t requant4(float v0, float v1, float v2, float v3, float inv, int relu) {
    const int q0 = __float2int_rn(__fmul_rn(v0, inv)), q1 = __float2int_rn(__fmul_rn(v1, inv));
    const int q2 = __float2int_rn(__fmul_rn(v2, inv)), q3 = __float2int_rn(__fmul_rn(v3, inv));
    uint32_t hi, out;
    if (relu) {
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0u));
        asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(q1), "r"(q0), "r"(hi));
        return __vminu4(out, 0x7f7f7f7fu);
    }
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(q3), "r"(q2), "r"(0u));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(q1), "r"(q0), "r"(hi));
    return out;
}

// 32 accumulator values of one output row -> dequantised fp32 in the stated rounding order:
// v = fl(float(acc) * scale_j), then + bias_j with one more rounding.  The 32 factors are the same for every lane:
// they are read four at a time (a scalar read per column costs a shared-memory wavefront each, and the load/store
// data path is the busiest unit of this epilogue).
__device__ __forceinline__ void dequant_chunk(const ContractionArgs& p, const uint32_t (&r)[32], const float* sc,
                                              const float* bs, float (&v)[32]) {
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
        const float4 s4 = *reinterpret_cast<const float4*>(sc + j);
        v[j] = __fmul_rn(__int2float_rn((int)r[j]), s4.x);
        v[j + 1] = __fmul_rn(__int2float_rn((int)r[j + 1]), s4.y);
        v[j + 2] = __fmul_rn(__int2float_rn((int)r[j + 2]), s4.z);
        v[j + 3] = __fmul_rn(__int2float_rn((int)r[j + 3]), s4.w);
    }
    if (p.bias) {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            const float4 b4 = *reinterpret_cast<const float4*>(bs + j);
            v[j] = __fadd_rn(v[j], b4.x);
            v[j + 1] = __fadd_rn(v[j + 1], b4.y);
            v[j + 2] = __fadd_rn(v[j + 2], b4.z);
            v[j + 3] = __fadd_rn(v[j + 3], b4.w);
        }
    }
}

// The skip path of a residual block: v += fl(float(r) * res_scale), r the INT8 skip values of the same 32 columns
// (eight words, byte i of word q = column 4q + i).
__device__ __forceinline__ void add_residual(float (&v)[32], const uint32_t (&w)[8], float res_scale) {
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int r = (int)(int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xffu);
        v[j] = __fadd_rn(v[j], __fmul_rn(__int2float_rn(r), res_scale));
    }
}

// Epilogue of one thread for 32 consecutive columns of its output row: optional int32 copy (with the
// part-bit shift), dequantisation in the stated rounding order, fp32 or bf16 store; vector stores when
// the chunk is whole and the pointers and pitches allow.
__device__ __forceinline__ void store_chunk(const ContractionArgs& p, long long row, int col0, const uint32_t (&r)[32],
                                            const float* sc, const float* bs, bool vec_acc, bool vec_f32, bool vec_bf16) {
    const bool full_chunk = col0 + 32 <= p.N;
    if (p.acc_out) {
        int32_t* dst = p.acc_out + row * p.ld_acc + col0;
        if (full_chunk && vec_acc) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<int4*>(dst + j) =
                    make_int4((int)r[j] >> p.acc_shift, (int)r[j + 1] >> p.acc_shift,
                              (int)r[j + 2] >> p.acc_shift, (int)r[j + 3] >> p.acc_shift);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) dst[j] = (int)r[j] >> p.acc_shift;
        }
    }
    if (p.y) {
        float v[32];
        dequant_chunk(p, r, sc, bs, v);
        if (p.residual) {
            const int8_t* rp = p.residual + row * p.ld_res + col0;
            uint32_t w[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                uint32_t x = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (col0 + 4 * q + i < p.N) x |= (uint32_t)(uint8_t)rp[4 * q + i] << (8 * i);
                w[q] = x;
            }
            add_residual(v, w, p.res_scale);
        }
        if (p.y_is_i8) {
            // the next layer's INT8 activations: ReLU, one multiply by fl(1 / out_scale), round half to even, clip
            int8_t* dst = reinterpret_cast<int8_t*>(p.y) + row * p.ldy + col0;
            uint32_t w[8];
#pragma unroll
            for (int j = 0; j < 32; j += 4) w[j >> 2] = requant4(v[j], v[j + 1], v[j + 2], v[j + 3], p.inv_out_scale, p.relu);
            const bool vec_i8 = ((p.ldy & 15) == 0) && ((reinterpret_cast<uintptr_t>(p.y) & 15) == 0);
            if (full_chunk && vec_i8) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4*>(dst + 16) = make_uint4(w[4], w[5], w[6], w[7]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < p.N) dst[j] = (int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xffu);
            }
        } else if (!p.y_is_bf16) {
            float* dst = reinterpret_cast<float*>(p.y) + row * p.ldy + col0;
            if (full_chunk && vec_f32) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < p.N) dst[j] = v[j];
            }
        } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.y) + row * p.ldy + col0;
            if (full_chunk && vec_bf16) {
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    __nv_bfloat162 a = __floats2bfloat162_rn(v[j], v[j + 1]);
                    __nv_bfloat162 b = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
                    __nv_bfloat162 c2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]);
                    __nv_bfloat162 d = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
                    uint4 o;
                    o.x = *reinterpret_cast<uint32_t*>(&a);
                    o.y = *reinterpret_cast<uint32_t*>(&b);
                    o.z = *reinterpret_cast<uint32_t*>(&c2);
                    o.w = *reinterpret_cast<uint32_t*>(&d);
                    *reinterpret_cast<uint4*>(dst + j) = o;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < p.N) dst[j] = __float2bfloat16_rn(v[j]);
            }
        }
    }
}

// 64 bytes of each of the warp's 32 rows, written with coalesced stores.  In the accumulator a lane owns one ROW,
// so storing from registers makes every store instruction touch 32 different cache lines with 16 bytes each,
// and the load/store unit spends a cycle per line: on output-bound problems that, not HBM, set the pace.  Here
// the warp lays the 32 x 64-byte block out in shared memory and reads it back with four consecutive lanes on
// one row: every instruction then touches 8 lines with 64 contiguous bytes each.  `q` is the lane's own row,
// `row` / `row_ok` its row index and validity; all 32 lanes must call.
__device__ __forceinline__ void store_rows64(uint8_t* stage, int lane, const uint4 (&q)[4], int row, bool row_ok,
                                             uint8_t* base, long long pitch_bytes, long long col_byte) {
    // a tile store of the other output may still be reading this block (accumulators by ordinary stores next to a
    // Y written by tile stores, or the reverse): wait for it before overwriting what it reads
    if (lane == 0) sm100::bulk_wait_read_all();
    __syncwarp();
    uint4* mine = reinterpret_cast<uint4*>(stage + lane * kEpiRowPitch);
    mine[0] = q[0]; mine[1] = q[1]; mine[2] = q[2]; mine[3] = q[3];
    __syncwarp();
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int rr = pass * 8 + (lane >> 2), cg = lane & 3;
        const int grow = __shfl_sync(0xffffffffu, row, rr);
        const bool ok = __shfl_sync(0xffffffffu, (int)row_ok, rr) != 0;
        const uint4 v = *reinterpret_cast<const uint4*>(stage + rr * kEpiRowPitch + cg * 16);
        if (ok) *reinterpret_cast<uint4*>(base + grow * pitch_bytes + col_byte + cg * 16) = v;
    }
    __syncwarp();
}

// Where the 32 rows of an epilogue warp sit in the output, as tile-store coordinates (dimensions 1..3 of the
// output map; dimension 0 is the byte offset of the columns).
struct OutCoords {
    int c1, c2, c3;
};
// The same 32 x 64-byte block handed to the TMA unit instead: the lanes lay their rows down in the 64-byte
// swizzle (no bank conflicts), one lane issues a tile store, and nobody reads the block back or issues a global
// store -- the load/store unit was the busiest unit of output-bound problems, and most of its shared-memory
// traffic was that read-back.  Rows and columns outside the output are clipped by the store.
// The buffer is reused once the previous store from it has finished reading.
__device__ __forceinline__ void store_rows64_tma(uint8_t* stage, int lane, const uint4 (&q)[4], const CUtensorMap* map,
                                                 int x_byte, const OutCoords& oc) {
    using namespace sm100;
    if (lane == 0) bulk_wait_read_all();
    __syncwarp();
    uint8_t* mine = stage + lane * 64;
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(mine + ((j ^ sw) << 4)) = q[j];
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        tma_store_4d(map, smem_u32(stage), x_byte, oc.c1, oc.c2, oc.c3);
        bulk_commit_group();
    }
}

// The same for 32-byte rows (INT8 output): a 32 x 32-byte block in the 32-byte swizzle.
__device__ __forceinline__ void store_rows32_tma(uint8_t* stage, int lane, const uint4 (&q)[2], const CUtensorMap* map,
                                                 int x_byte, const OutCoords& oc) {
    using namespace sm100;
    if (lane == 0) bulk_wait_read_all();
    __syncwarp();
    uint8_t* mine = stage + lane * 32;
    const int sw = (lane >> 2) & 1;
    *reinterpret_cast<uint4*>(mine + ((0 ^ sw) << 4)) = q[0];
    *reinterpret_cast<uint4*>(mine + ((1 ^ sw) << 4)) = q[1];
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        tma_store_4d(map, smem_u32(stage), x_byte, oc.c1, oc.c2, oc.c3);
        bulk_commit_group();
    }
}

// The epilogue of one warp for 32 consecutive columns: same arithmetic as store_chunk, coalesced stores.
__device__ __forceinline__ void store_chunk_warp(const ContractionArgs& p, int row, bool row_ok, int col0,
                                                 const uint32_t (&r)[32], const float* sc, const float* bs,
                                                 bool vec_acc, bool vec_f32, bool vec_bf16, uint8_t* stage, int lane,
                                                 const CUtensorMap* tmY, const CUtensorMap* tmAcc, const OutCoords& oc) {
    const bool full_chunk = col0 + 32 <= p.N;
    const bool acc_fast = p.acc_out == nullptr || p.acc_tma || (full_chunk && vec_acc);
    const bool res_fast = p.residual == nullptr ||
                          (full_chunk && ((p.ld_res & 15) == 0) && ((reinterpret_cast<uintptr_t>(p.residual) & 15) == 0));
    const bool y_fast = (p.y == nullptr || p.y_tma || (!p.y_is_i8 && full_chunk && (p.y_is_bf16 ? vec_bf16 : vec_f32))) && res_fast;
    if (!acc_fast || !y_fast) {                        // ragged or unaligned: the plain per-row path
        if (row_ok) store_chunk(p, row, col0, r, sc, bs, vec_acc, vec_f32, vec_bf16);
        return;
    }
    uint4 q[4];
    if (p.acc_out) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                q[j] = make_uint4((uint32_t)((int)r[half * 16 + 4 * j] >> p.acc_shift), (uint32_t)((int)r[half * 16 + 4 * j + 1] >> p.acc_shift),
                                  (uint32_t)((int)r[half * 16 + 4 * j + 2] >> p.acc_shift), (uint32_t)((int)r[half * 16 + 4 * j + 3] >> p.acc_shift));
            if (p.acc_tma) store_rows64_tma(stage, lane, q, tmAcc, (col0 + half * 16) * 4, oc);
            else store_rows64(stage, lane, q, row, row_ok, reinterpret_cast<uint8_t*>(p.acc_out), p.ld_acc * 4,
                              (long long)(col0 + half * 16) * 4);
        }
    }
    if (p.y) {
        float v[32];
        dequant_chunk(p, r, sc, bs, v);
        if (p.residual) {                              // a row outside the output adds zeros (its values are clipped by the store)
            uint4 ra = make_uint4(0u, 0u, 0u, 0u), rb = ra;
            if (row_ok) {
                const uint4* rp = reinterpret_cast<const uint4*>(p.residual + (long long)row * p.ld_res + col0);
                ra = __ldg(rp); rb = __ldg(rp + 1);
            }
            const uint32_t w[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
            add_residual(v, w, p.res_scale);
        }
        if (p.y_is_i8) {
            // the next layer's INT8 activations: ReLU, one multiply by fl(1 / out_scale), round half to even, clip
            uint32_t w8[8];
#pragma unroll
            for (int j = 0; j < 32; j += 4) w8[j >> 2] = requant4(v[j], v[j + 1], v[j + 2], v[j + 3], p.inv_out_scale, p.relu);
            const uint4 q2[2] = {make_uint4(w8[0], w8[1], w8[2], w8[3]), make_uint4(w8[4], w8[5], w8[6], w8[7])};
            store_rows32_tma(stage, lane, q2, tmY, col0, oc);
        } else if (!p.y_is_bf16) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    q[j] = make_uint4(__float_as_uint(v[half * 16 + 4 * j]), __float_as_uint(v[half * 16 + 4 * j + 1]),
                                      __float_as_uint(v[half * 16 + 4 * j + 2]), __float_as_uint(v[half * 16 + 4 * j + 3]));
                if (p.y_tma) store_rows64_tma(stage, lane, q, tmY, (col0 + half * 16) * 4, oc);
                else store_rows64(stage, lane, q, row, row_ok, reinterpret_cast<uint8_t*>(p.y), p.ldy * 4,
                                  (long long)(col0 + half * 16) * 4);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                __nv_bfloat162 a = __floats2bfloat162_rn(v[8 * j], v[8 * j + 1]);
                __nv_bfloat162 b = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
                __nv_bfloat162 c2 = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
                __nv_bfloat162 d = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
                q[j] = make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                                  *reinterpret_cast<uint32_t*>(&c2), *reinterpret_cast<uint32_t*>(&d));
            }
            if (p.y_tma) store_rows64_tma(stage, lane, q, tmY, col0 * 2, oc);
            else store_rows64(stage, lane, q, row, row_ok, reinterpret_cast<uint8_t*>(p.y), p.ldy * 2, (long long)col0 * 2);
        }
    }
}

// Tile-store coordinates of the 32 rows that start at tile row ml0 (a multiple of 32) of M-tile mt.
template <int MODE>
__device__ __forceinline__ OutCoords out_coords(const ContractionArgs& p, int mt, int ml0) {
    OutCoords oc;
    if (MODE == kModeGemm) {
        oc.c1 = mt * kBM + ml0; oc.c2 = 0; oc.c3 = 0;
    } else {
        const TileOrigin o = conv_tile_origin(p.g, mt);
        oc.c1 = o.q0 + (ml0 & ((1 << p.g.tw_log2) - 1));
        oc.c2 = o.p0 + ((ml0 >> p.g.tw_log2) & ((1 << p.g.th_log2) - 1));
        oc.c3 = o.b0 + (ml0 >> (p.g.tw_log2 + p.g.th_log2));
    }
    return oc;
}

// Per-channel output factors of 32 * PER_LANE consecutive columns starting at col_base, lane-strided:
// fl(fl(act * w_scale) * 2^l), then the exact 2^-(8-h) that undoes the top-aligned unpack; and the bias.
template <int PER_LANE>
__device__ __forceinline__ void fetch_scales(const ContractionArgs& p, int col_base, int lane, float (&sc)[PER_LANE],
                                             float (&bs)[PER_LANE]) {
#pragma unroll
    for (int i = 0; i < PER_LANE; ++i) {
        const int col = col_base + lane + 32 * i;
        sc[i] = 0.f;
        bs[i] = 0.f;
        if (col < p.N) {
            sc[i] = __fmul_rn(__fmul_rn(__fmul_rn(p.act_scale, __ldg(p.w_scale + col)), p.pow2_l), p.unshift);
            if (p.bias) bs[i] = __ldg(p.bias + col);
        }
    }
}

// What an epilogue warp needs from its kernel: where scales, staging blocks and accumulator barriers live, and
// which tiles the block walks.
struct EpilogueCtx {
    float* sScale;
    float* sBias;
    uint8_t* sStage;
    uint64_t* tfull;
    uint64_t* tempty;
    uint32_t* signal_sink;        // pair kernel: landing place of signal stores in the leader
    volatile int* abort_flag;
    uint32_t tmem_base;
    int first_tile, tile_step, num_tiles;
    uint32_t rank;                // pair kernel: this CTA's rank in the pair (0 = leader); 0 otherwise
};

// The epilogue role of both contraction kernels (warps 2 .. 2 + kEpiWarps - 1): for every tile of the block, wait
// for the accumulator, read this warp's lane quarter and half of the columns 32 columns at a time, hand the
// accumulator back after the last read, dequantise and store.  BN: tile columns.  PAIR: the block is one CTA of a
// pair -- it owns rows [128 * rank, 128 * rank + 128) of a 256-row tile, the accumulator barriers are signalled
// across the pair (tfull by the leader's commit in both CTAs; tempty lives in the leader, to which the partner's
// warps send 4 announced bytes each).
template <int BN, int MODE, bool PAIR>
__device__ __forceinline__ void epilogue_role(const ContractionArgs& p, const CUtensorMap* tmY, const CUtensorMap* tmAcc,
                                              const EpilogueCtx& ex, int warp, int lane) {
    using namespace sm100;
    const int quarter = warp & 3;                  // TMEM lanes this warp may read
    const int chalf = (warp - 2) >> 2;             // which half of the tile's columns it handles
    int staged_nt = -1;                            // column tile whose scales sit in shared memory
    constexpr int SCALES_PER_LANE = BN / 64;       // a warp stages BN / 2 scales
    uint32_t tl = 0;
    bool ok = true;
    const bool vec_f32 = (p.y != nullptr) && !p.y_is_bf16 && ((p.ldy & 3) == 0) &&
                         ((reinterpret_cast<uintptr_t>(p.y) & 15) == 0);
    const bool vec_bf16 = (p.y != nullptr) && p.y_is_bf16 && ((p.ldy & 7) == 0) &&
                          ((reinterpret_cast<uintptr_t>(p.y) & 15) == 0);
    const bool vec_acc = (p.acc_out != nullptr) && ((p.ld_acc & 3) == 0) &&
                         ((reinterpret_cast<uintptr_t>(p.acc_out) & 15) == 0);
    // per-channel factor: fl(fl(act * w_scale) * 2^l), then the exact 2^-(8-h) of the unpack.
    // Each warp keeps a private copy, so the epilogue warps never wait on one another.
    float* sc_w = ex.sScale + (warp - 2) * (BN / 2);      // scales of this warp's half of the columns
    float* bs_w = ex.sBias + (warp - 2) * (BN / 2);
    for (int tile = ex.first_tile; ok && tile < ex.num_tiles; tile += ex.tile_step, ++tl) {
        int mt, nt;
        tile_coords(tile, p, mt, nt);
        if (PAIR) mt = mt * 2 + (int)ex.rank;          // this CTA's 128-row tile of the pair's 256 rows
        const uint32_t buf = tl & 1, buse = tl >> 1;
        const int n0 = nt * BN;
        __syncwarp();
        if (nt != staged_nt) {                         // only the first tile: later ones are prefetched below
            float sc_r[SCALES_PER_LANE], bs_r[SCALES_PER_LANE];
            fetch_scales<SCALES_PER_LANE>(p, n0 + chalf * (BN / 2), lane, sc_r, bs_r);
#pragma unroll
            for (int i = 0; i < SCALES_PER_LANE; ++i) { sc_w[lane + 32 * i] = sc_r[i]; bs_w[lane + 32 * i] = bs_r[i]; }
            staged_nt = nt;
        }
        __syncwarp();
        // The next tile's scales are fetched now and land in registers while this tile is converted and
        // stored; they go to shared memory at the end of the iteration.  (Fetched at the top of the next
        // iteration instead, the global-memory round trip sat on every tile's critical path.)
        int next_nt = -1;
        float sc_n[SCALES_PER_LANE], bs_n[SCALES_PER_LANE];
        if (tile + ex.tile_step < ex.num_tiles) {
            int mt_n;
            tile_coords(tile + ex.tile_step, p, mt_n, next_nt);
            if (next_nt != nt) fetch_scales<SCALES_PER_LANE>(p, next_nt * BN + chalf * (BN / 2), lane, sc_n, bs_n);
        }
        ok = PAIR ? mbar_wait_cluster(smem_u32(&ex.tfull[buf]), buse & 1, ex.abort_flag, p.status, 0x130u)
                  : mbar_wait(smem_u32(&ex.tfull[buf]), buse & 1, ex.abort_flag, p.status, 0x30u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        long long row;
        bool row_ok;
        if (MODE == kModeGemm) {
            row = (long long)mt * kBM + quarter * 32 + lane;
            row_ok = row < p.M;
        } else {
            // tile row -> output pixel: the low bits walk the width, then the height, then the images
            const TileOrigin o = conv_tile_origin(p.g, mt);
            const int ml = quarter * 32 + lane;
            const int qq = o.q0 + (ml & ((1 << p.g.tw_log2) - 1));
            const int pp = o.p0 + ((ml >> p.g.tw_log2) & ((1 << p.g.th_log2) - 1));
            const int bb = o.b0 + (ml >> (p.g.tw_log2 + p.g.th_log2));
            row_ok = qq < p.g.Wo && pp < p.g.Ho && bb < p.g.B;
            row = ((long long)bb * p.g.Ho + pp) * p.g.Wo + qq;
        }
        const OutCoords oc = out_coords<MODE>(p, mt, quarter * 32);
        constexpr int CHUNKS = BN / 64;                // 32-column chunks per warp (half of the tile)
#pragma unroll 1
        for (int cc = 0; cc < CHUNKS; ++cc) {
            const int c = chalf * CHUNKS + cc;
            uint32_t r[32];
            tmem_ld_32x32(ex.tmem_base + buf * BN + c * 32 + ((uint32_t)(quarter * 32) << 16), r);
            tmem_ld_wait();
            if (cc == CHUNKS - 1) {                    // last read of the accumulator: hand it back before storing
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if (!PAIR || ex.rank == 0) mbar_arrive(smem_u32(&ex.tempty[buf]));
                    else signal_remote_tx4(map_to_cta(smem_u32(ex.signal_sink), 0), map_to_cta(smem_u32(&ex.tempty[buf]), 0));
                }
            }
            const int col0 = n0 + c * 32;
            if (col0 >= p.N) continue;
            store_chunk_warp(p, (int)row, row_ok, col0, r, sc_w + cc * 32, bs_w + cc * 32, vec_acc, vec_f32, vec_bf16,
                             ex.sStage + (warp - 2) * kEpiStageBytes, lane, tmY, tmAcc, oc);
        }
        if (next_nt >= 0 && next_nt != nt) {
            __syncwarp();
#pragma unroll
            for (int i = 0; i < SCALES_PER_LANE; ++i) { sc_w[lane + 32 * i] = sc_n[i]; bs_w[lane + 32 * i] = bs_n[i]; }
            staged_nt = next_nt;
        }
    }
    if (lane == 0) bulk_wait_all();                    // this lane's tile stores are done before the block leaves
}

// Part-bit blocks end with one more warp, the producer of the packed-tile ring: two producers that spin in one
// warp hold each other up for the length of a barrier probe.
constexpr int kPackedProducerWarp = kFirstUnpackWarp + kUnpackWarps;
__host__ __device__ constexpr int contraction_threads(bool part) {
    return part ? kBaseThreads + kUnpackThreads + 32 : kBaseThreads;
}

template <int BN, bool PART, int MODE>
__global__ void __launch_bounds__(contraction_threads(PART), 1)
contraction_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmAcc,
                   const ContractionArgs p) {
    using namespace sm100;
    constexpr int STAGES = stages_for(BN, PART);
    constexpr int A_BYTES = a_stage_bytes();
    constexpr int B_BYTES = b_stage_bytes(BN);
    constexpr uint32_t TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;       // power of two >= 32
    constexpr uint32_t IDESC = idesc_i8(kBM, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = sA + STAGES * A_BYTES;
    const int packed_bytes = PART ? BN * 16 * p.h_bits : 0;
    uint8_t* sP = sB + STAGES * B_BYTES;
    float* sScale = reinterpret_cast<float*>(sP + (PART ? p.packed_stages * packed_bytes : 0));   // [4 warps][BN]
    float* sBias = sScale + 4 * BN;                                                             // [4 warps][BN]
    uint8_t* sStage = reinterpret_cast<uint8_t*>(sBias + 4 * BN);                               // [kEpiWarps][kEpiStageBytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sStage + kEpiWarps * kEpiStageBytes);
    // barrier map: full[STAGES], empty[STAGES], pfull[2], pempty[2], tfull[2], tempty[2]
    uint64_t* full = bars;
    uint64_t* empty = full + STAGES;
    uint64_t* pfull = empty + STAGES;
    uint64_t* pempty = pfull + kMaxPackedStages;
    uint64_t* tfull = pempty + kMaxPackedStages;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&full[s]), PART ? 1 + kUnpackWarps : 1);   // producer (+ one arrival per unpack warp)
            mbar_init(smem_u32(&empty[s]), 1);                 // tcgen05.commit
        }
        for (int s = 0; s < kMaxPackedStages; ++s) {
            mbar_init(smem_u32(&pfull[s]), 1);
            mbar_init(smem_u32(&pempty[s]), kUnpackWarps);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tfull[b]), 1);
            mbar_init(smem_u32(&tempty[b]), kEpiWarps);        // one arrival per epilogue warp
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        if (p.y_tma) prefetch_tensormap(&tmY);
        if (p.acc_tma) prefetch_tensormap(&tmAcc);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                int mt, nt;
                tile_coords(tile, p, mt, nt);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, use = it / STAGES;
                    if (!(ok = mbar_wait(smem_u32(&empty[s]), (use & 1) ^ 1, abort_flag, p.status, 0x10u))) break;
                    const uint32_t fb = smem_u32(&full[s]);
                    // bytes this stage brings in: A always; B too in full-bit mode
                    int n_sub = 1;                                       // kModeConv64: taps present in this stage
                    if (MODE == kModeConv64) n_sub = min(2, p.g.taps - 2 * kb);
                    const uint32_t a_bytes = (MODE == kModeConv64) ? n_sub * (A_BYTES / 2) : A_BYTES;
                    const uint32_t b_bytes = PART ? 0u : ((MODE == kModeConv64) ? n_sub * (B_BYTES / 2) : B_BYTES);
                    mbar_arrive_expect_tx(fb, a_bytes + b_bytes);
                    if (MODE == kModeGemm) {
                        tma_load_2d(smem_u32(sA + s * A_BYTES), &tmA, kb * kBK, mt * kBM, fb);
                    } else {
                        const TileOrigin o = conv_tile_origin(p.g, mt);
                        for (int sub = 0; sub < n_sub; ++sub) {
                            const int tap = (MODE == kModeConv64) ? 2 * kb + sub : kb / p.g.cblocks;
                            const int c0 = (MODE == kModeConv64) ? 0 : (kb % p.g.cblocks) * 128;
                            const int r = tap / p.g.S, sx = tap - r * p.g.S;
                            tma_load_4d(smem_u32(sA + s * A_BYTES + sub * (A_BYTES / 2)), &tmA, c0,
                                        o.q0 * p.g.stride - p.g.pad + sx, o.p0 * p.g.stride - p.g.pad + r, o.b0, fb);
                        }
                    }
                    if (PART) {
                        // the packed tiles have a ring and a producer lane of their own (below)
                    } else if (MODE == kModeConv64) {
                        for (int sub = 0; sub < n_sub; ++sub)
                            tma_load_2d(smem_u32(sB + s * B_BYTES + sub * (B_BYTES / 2)), &tmB, kb * kBK + sub * 64, nt * BN, fb);
                    } else {
                        tma_load_2d(smem_u32(sB + s * B_BYTES), &tmB, kb * kBK, nt * BN, fb);
                    }
                }
            }
            if (!ok) {
                // gave up: let the copies already in flight land before the block releases its shared memory
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 22)) { }
            }
        }
    } else if (PART && warp == kPackedProducerWarp) {
        if (lane == 0) {
            // ---- packed-tile producer: runs ahead of the A loads by up to the depth of its own ring, which
            //      is what hides the latency of fetching the weights
            uint32_t pit = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                int mt, nt;
                tile_coords(tile, p, mt, nt);
                for (int kb = 0; kb < p.k_blocks; ++kb, ++pit) {
                    const uint32_t ps = pit % p.packed_stages, puse = pit / p.packed_stages;
                    if (!(ok = mbar_wait(smem_u32(&pempty[ps]), (puse & 1) ^ 1, abort_flag, p.status, 0x11u))) break;
                    load_ring_slot<BN>(p, smem_u32(sP + ps * packed_bytes), nt * BN, kb, smem_u32(&pfull[ps]));
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 22)) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++tl) {
                const uint32_t buf = tl & 1, buse = tl >> 1;
                if (!(ok = mbar_wait(smem_u32(&tempty[buf]), (buse & 1) ^ 1, abort_flag, p.status, 0x20u))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, use = it / STAGES;
                    if (!(ok = mbar_wait(smem_u32(&full[s]), use & 1, abort_flag, p.status, 0x21u))) break;
                    tc_fence_after_sync();
                    if (MODE == kModeConv64) {
                        const int n_sub = min(2, p.g.taps - 2 * kb);
                        for (int sub = 0; sub < n_sub; ++sub) {
                            const uint64_t da = smem_desc_sw64(smem_u32(sA + s * A_BYTES + sub * (A_BYTES / 2)));
                            const uint64_t db = smem_desc_sw64(smem_u32(sB + s * B_BYTES + sub * (B_BYTES / 2)));
#pragma unroll
                            for (int k = 0; k < 2; ++k)
                                mma_i8(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | sub | k) != 0);
                        }
                    } else {
                        const uint64_t da = smem_desc_sw128(smem_u32(sA + s * A_BYTES));
                        const uint64_t db = smem_desc_sw128(smem_u32(sB + s * B_BYTES));
#pragma unroll
                        for (int k = 0; k < kBK / 32; ++k)   // 32 bytes of K per instruction: +2 in the address field
                            mma_i8(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | k) != 0);
                    }
                    mma_commit(smem_u32(&empty[s]));       // stage reusable once these MMAs have read it
                }
                if (ok) mma_commit(smem_u32(&tfull[buf]));   // accumulator complete
            }
        }
    } else if (warp < kFirstUnpackWarp) {
        // ------------------------------------------------------------------ epilogue
        EpilogueCtx ex;
        ex.sScale = sScale; ex.sBias = sBias; ex.sStage = sStage; ex.tfull = tfull; ex.tempty = tempty;
        ex.signal_sink = nullptr; ex.abort_flag = abort_flag; ex.tmem_base = tmem_base;
        ex.first_tile = blockIdx.x; ex.tile_step = gridDim.x; ex.num_tiles = num_tiles; ex.rank = 0;
        epilogue_role<BN, MODE, false>(p, &tmY, &tmAcc, ex, warp, lane);
    } else if (PART && warp < kPackedProducerWarp) {
        // ------------------------------------------------------------------ unpackers
        const int utid = threadIdx.x - kBaseThreads;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                const uint32_t s = it % STAGES, use = it / STAGES;
                const uint32_t ps = it % p.packed_stages, puse = it / p.packed_stages;
                ok = mbar_wait(smem_u32(&pfull[ps]), puse & 1, abort_flag, p.status, 0x40u) &&
                     mbar_wait(smem_u32(&empty[s]), (use & 1) ^ 1, abort_flag, p.status, 0x41u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint8_t* src = sP + ps * packed_bytes;
                uint8_t* dst = sB + s * B_BYTES;
                switch (p.h_bits) {                    // one specialised expansion per field width
                    case 1: unpack_tile<BN, MODE, 1, kUnpackThreads>(src, dst, utid); break;
                    case 2: unpack_tile<BN, MODE, 2, kUnpackThreads>(src, dst, utid); break;
                    case 3: unpack_tile<BN, MODE, 3, kUnpackThreads>(src, dst, utid); break;
                    case 4: unpack_tile<BN, MODE, 4, kUnpackThreads>(src, dst, utid); break;
                    case 5: unpack_tile<BN, MODE, 5, kUnpackThreads>(src, dst, utid); break;
                    case 6: unpack_tile<BN, MODE, 6, kUnpackThreads>(src, dst, utid); break;
                    default: unpack_tile<BN, MODE, 7, kUnpackThreads>(src, dst, utid); break;
                }
                fence_proxy_async_smem();              // these writes feed tcgen05.mma (async proxy)
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&full[s]));
                    mbar_arrive(smem_u32(&pempty[ps]));
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// Output type used inside the library for the requantised INT8 result, and its parameters.
constexpr int kOutI8 = 2;
struct OutQuant {
    float out_scale;
    int relu;
    const int8_t* residual;   // INT8 skip tensor of the output's shape (dense), or nullptr
    float res_scale;
};

// Host launcher (defined with the GEMM entry points).  The A operand is reached through tmA: a plain 2-D map
// of an [M, K] matrix (kModeGemm, geom == nullptr) or a 4-D map of NHWC activations (convolution modes).
int run_contraction(const CUtensorMap& tmA, int mode, const ConvGeom* geom, int m_tiles, int k_blocks,
                    const void* Bmat, int64_t ldb, bool part, int n_bits, int h_bits,
                    const float* w_scale, float act_scale, const float* bias, int64_t M, int64_t N, int64_t K,
                    int32_t* acc_out, int64_t ld_acc, void* Y, int64_t ldy, int y_dtype, cudaStream_t stream,
                    const OutQuant* oq = nullptr, const void* Blow = nullptr);

}  // namespace nq
