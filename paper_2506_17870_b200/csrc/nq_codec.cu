// Bandwidth-bound codec kernels: decomposition, recomposition (page-in), drop-low (page-out) and
// the plain pack / unpack test aids, all on the sliced sub-byte layout described in nq.h.
//
// Work unit: 32 consecutive elements of one row = eight 32-bit words of int8 on the unpacked side
// and, per slice of width s, s words on the packed side.  Units are walked block by block (128 rows x 128
// columns, the packed layout's storage unit), rows fastest: the 32 lanes of a warp hold four units of each of
// eight consecutive rows, so every packed access of a warp is one contiguous run (512 / 256 / 128 bytes of the
// 4- / 2- / 1-bit slice) and every int8 access covers eight whole 128-byte lines.  One thread takes a PAIR of units
// per loop trip -- the same columns, 64 rows apart in the block, so one index decode serves both and the loads of
// both are in flight together -- and keeps each in registers as eight "top-aligned" words T[q]: byte lane i of T[q] holds the k-bit
// field of element 4q+i in its TOP k bits.  In that form every slice is a fixed bit range of every
// byte, so moving between T and the slices is a mask, a shift and an OR per word -- four elements
// per instruction -- and the nesting arithmetic (Eq. 5, 6, 10) is done on four bytes at a time.
//
// These kernels move 2-3 bytes per weight, so at HBM speed an SM has only a few integer
// instructions per weight to spend.  For INT8 nesting (n = 8) every (h, compensate) pair therefore
// gets its own instantiation with all shifts and masks as immediates; other n run a generic kernel
// that takes them from registers.
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/nq.h"
#include "nq_internal.cuh"

namespace {

constexpr uint32_t H4 = 0x80808080u;
constexpr uint32_t L7 = 0x7f7f7f7fu;

__host__ __device__ constexpr uint32_t rep8(uint32_t b) { return (b & 0xffu) * 0x01010101u; }

// per-byte wrapping subtract
__device__ __forceinline__ uint32_t sub4(uint32_t a, uint32_t b) {
    return ((a | H4) - (b & L7)) ^ ((a ^ ~b) & H4);
}
// per-byte unsigned saturating subtract for a subtrahend whose bytes are all below 0x80
__device__ __forceinline__ uint32_t subsat_small_u4(uint32_t a, uint32_t s) {
    uint32_t d = ((a | H4) - s) ^ (~a & H4);      // wrapping a - s
    uint32_t under = ~a & d & H4;                 // top bit went 0 -> 1: the byte wrapped below zero
    uint32_t kill = (under >> 7) * 0xffu;
    return d & ~kill;
}
// the same for any subtrahend
__device__ __forceinline__ uint32_t subsat_u4(uint32_t a, uint32_t b) {
    uint32_t d = sub4(a, b);
    uint32_t borrow = ((~a & b) | (~(a ^ b) & d)) & H4;   // borrow out of each byte
    uint32_t kill = (borrow >> 7) * 0xffu;
    return d & ~kill;
}
// 1 in every byte that is non-zero
__device__ __forceinline__ uint32_t nonzero4(uint32_t x) {
    return ((((x & L7) + L7) | x) & H4) >> 7;
}

// ---------------------------------------------------------------------------------------------
// nesting parameters: the same member names at run time (Nest) and at compile time (SNest)
// ---------------------------------------------------------------------------------------------
struct Nest {
    int n, h, l, lb, comp;
    uint32_t bias, mask_n, mask_h, mask_l, mask_lb, bit_l;
    __device__ Nest(int n_, int h_, int comp_) : n(n_), h(h_), l(n_ - h_), lb(n_ - h_ + (comp_ ? 1 : 0)), comp(comp_) {
        bias = rep8(1u << (n - 1));
        mask_n = rep8((1u << n) - 1u);
        mask_h = rep8((1u << h) - 1u);
        mask_l = rep8((1u << l) - 1u);
        mask_lb = rep8((1u << lb) - 1u);
        bit_l = rep8(1u << l);
    }
};

template <int N_, int H_, int COMP_>
struct SNest {
    static constexpr int n = N_, h = H_, l = N_ - H_, lb = N_ - H_ + (COMP_ ? 1 : 0), comp = COMP_;
    static constexpr uint32_t bias = rep8(1u << (N_ - 1));
    static constexpr uint32_t mask_n = rep8((1u << N_) - 1u);
    static constexpr uint32_t mask_h = rep8((1u << H_) - 1u);
    static constexpr uint32_t mask_l = rep8((1u << (N_ - H_)) - 1u);
    static constexpr uint32_t mask_lb = rep8((1u << (N_ - H_ + (COMP_ ? 1 : 0))) - 1u);
    static constexpr uint32_t bit_l = rep8(1u << (N_ - H_));
    __device__ SNest(int, int, int) {}
};

// ---------------------------------------------------------------------------------------------
// packed side: one unit <-> eight top-aligned words
// ---------------------------------------------------------------------------------------------
struct PackedRaw {
    uint4 a, b;      // 8-bit slice (two 16-byte halves) or, for narrower fields, a = the 4-bit slice
    uint2 c;         // 2-bit slice
    uint32_t d;      // 1-bit slice
};

// `block` is the start of a 128 x 128 block of `bits`-bit fields, `ru` = row-in-block * 4 + unit (0 .. 511): the
// slice of width s starts 2048 * (bits of the wider slices) bytes into the block and keeps 4 * s bytes per unit.
__device__ __forceinline__ void load_packed_raw(const uint8_t* __restrict__ block, int ru, int bits, PackedRaw& r) {
    if (bits == 8) {
        const uint4* p = reinterpret_cast<const uint4*>(block + ru * 32);
        r.a = __ldg(p); r.b = __ldg(p + 1);
        return;
    }
    int off = 0;
    if (bits & 4) { r.a = __ldg(reinterpret_cast<const uint4*>(block + ru * 16)); off = 8192; }
    if (bits & 2) { r.c = __ldg(reinterpret_cast<const uint2*>(block + off + ru * 8)); off += 4096; }
    if (bits & 1) { r.d = __ldg(reinterpret_cast<const uint32_t*>(block + off + ru * 4)); }
}

__device__ __forceinline__ void expand_packed_raw(const PackedRaw& r, int bits, uint32_t (&T)[8]) {
    if (bits == 8) {
        T[0] = r.a.x; T[1] = r.a.y; T[2] = r.a.z; T[3] = r.a.w; T[4] = r.b.x; T[5] = r.b.y; T[6] = r.b.z; T[7] = r.b.w;
        return;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) T[q] = 0;
    int used = 0;
    if (bits & 4) {
        T[0] = r.a.x & 0xf0f0f0f0u; T[1] = (r.a.x << 4) & 0xf0f0f0f0u;
        T[2] = r.a.y & 0xf0f0f0f0u; T[3] = (r.a.y << 4) & 0xf0f0f0f0u;
        T[4] = r.a.z & 0xf0f0f0f0u; T[5] = (r.a.z << 4) & 0xf0f0f0f0u;
        T[6] = r.a.w & 0xf0f0f0f0u; T[7] = (r.a.w << 4) & 0xf0f0f0f0u;
        used = 4;
    }
    // a narrower slice lands below the bits already placed: one net shift and one masked OR per word
    if (bits & 2) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const uint32_t word = (q < 4) ? r.c.x : r.c.y;
            const int net = 2 * (q & 3) - used;          // left shift if positive
            const uint32_t moved = net >= 0 ? (word << net) : (word >> (-net));
            T[q] |= moved & (0xc0c0c0c0u >> used);
        }
        used += 2;
    }
    if (bits & 1) {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int net = q - used;
            const uint32_t moved = net >= 0 ? (r.d << net) : (r.d >> (-net));
            T[q] |= moved & (H4 >> used);
        }
    }
}

__device__ __forceinline__ void store_unit_top(uint8_t* __restrict__ block, int ru, int bits,
                                               const uint32_t (&T)[8]) {
    if (bits == 8) {
        uint4* p = reinterpret_cast<uint4*>(block + ru * 32);
        p[0] = make_uint4(T[0], T[1], T[2], T[3]);
        p[1] = make_uint4(T[4], T[5], T[6], T[7]);
        return;
    }
    int off = 0, used = 0;
    if (bits & 4) {
        uint4 w;
        w.x = (T[0] & 0xf0f0f0f0u) | ((T[1] >> 4) & 0x0f0f0f0fu);
        w.y = (T[2] & 0xf0f0f0f0u) | ((T[3] >> 4) & 0x0f0f0f0fu);
        w.z = (T[4] & 0xf0f0f0f0u) | ((T[5] >> 4) & 0x0f0f0f0fu);
        w.w = (T[6] & 0xf0f0f0f0u) | ((T[7] >> 4) & 0x0f0f0f0fu);
        *reinterpret_cast<uint4*>(block + ru * 16) = w;
        off = 8192; used = 4;
    }
    if (bits & 2) {
        uint2 w = make_uint2(0u, 0u);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int net = used - 2 * (q & 3);          // left shift if positive
            const uint32_t moved = net >= 0 ? (T[q] << net) : (T[q] >> (-net));
            const uint32_t piece = moved & (0xc0c0c0c0u >> (2 * (q & 3)));
            if (q < 4) w.x |= piece; else w.y |= piece;
        }
        *reinterpret_cast<uint2*>(block + off + ru * 8) = w;
        off += 4096; used += 2;
    }
    if (bits & 1) {
        uint32_t w = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int net = used - q;
            const uint32_t moved = net >= 0 ? (T[q] << net) : (T[q] >> (-net));
            w |= moved & (H4 >> q);
        }
        *reinterpret_cast<uint32_t*>(block + off + ru * 4) = w;
    }
}

// ---------------------------------------------------------------------------------------------
// unpacked side: 32 int8 of one row <-> eight words, with a byte-wise path for ragged / unaligned rows
// ---------------------------------------------------------------------------------------------
struct I8Raw {
    uint4 a, b;
    bool vec;        // loaded with vector loads; otherwise the byte-wise path runs at use time
};

__device__ __forceinline__ void load_unit_i8_bytes(const int8_t* __restrict__ row, int64_t c0, int64_t cols, uint32_t (&V)[8]) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        uint32_t w = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t c = c0 + q * 4 + i;
            uint32_t b = (c < cols) ? (uint32_t)(uint8_t)row[c] : 0u;
            w |= b << (8 * i);
        }
        V[q] = w;
    }
}

__device__ __forceinline__ void load_i8_raw(const int8_t* __restrict__ row, int64_t c0, int64_t cols, bool vec_ok, I8Raw& r) {
    r.vec = vec_ok && c0 + 32 <= cols;
    if (r.vec) {
        const uint4* p = reinterpret_cast<const uint4*>(row + c0);
        r.a = __ldg(p); r.b = __ldg(p + 1);
    }
}
__device__ __forceinline__ void expand_i8_raw(const I8Raw& r, const int8_t* __restrict__ row, int64_t c0, int64_t cols,
                                              uint32_t (&V)[8]) {
    if (r.vec) {
        V[0] = r.a.x; V[1] = r.a.y; V[2] = r.a.z; V[3] = r.a.w; V[4] = r.b.x; V[5] = r.b.y; V[6] = r.b.z; V[7] = r.b.w;
    } else {
        load_unit_i8_bytes(row, c0, cols, V);
    }
}

__device__ __forceinline__ void store_unit_i8(int8_t* __restrict__ row, int64_t c0, int64_t cols,
                                              bool vec_ok, const uint32_t (&V)[8]) {
    if (vec_ok && c0 + 32 <= cols) {
        uint4* p = reinterpret_cast<uint4*>(row + c0);
        p[0] = make_uint4(V[0], V[1], V[2], V[3]);
        p[1] = make_uint4(V[4], V[5], V[6], V[7]);
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                int64_t c = c0 + q * 4 + i;
                if (c < cols) row[c] = (int8_t)((V[q] >> (8 * i)) & 0xffu);
            }
    }
}

// ---------------------------------------------------------------------------------------------
// the nesting arithmetic on four bytes at a time.  "Biased" means value + 2^(n-1), an unsigned
// n-bit number; in that domain w_high + 2^(h-1) is simply the top h bits.
// ---------------------------------------------------------------------------------------------

// Eq. 6 with the mask-given rounding, then Eq. 10 / compensation.  V, M: int8 weights and mask bytes.
template <class NestT>
__device__ __forceinline__ void decompose_word(const NestT& N, uint32_t V, uint32_t M, uint32_t& Thi, uint32_t& Tlo) {
    uint32_t wu = (V ^ N.bias) & N.mask_n;                 // w + 2^(n-1)
    uint32_t down = (wu >> N.l) & N.mask_h;                // floor(w / 2^l) + 2^(h-1)
    uint32_t rem_nz = ((wu & N.mask_l) + L7) & H4;         // remainder != 0 (it is below 0x80: the add stays in its byte)
    uint32_t up = (rem_nz >> 7) & nonzero4(M);             // round up only off a multiple of 2^l
    uint32_t whb = down + up;                              // <= 2^h per byte: no carry between bytes
    whb -= (whb >> N.h) & 0x01010101u;                     // clip to 2^h - 1 (max_high, biased)
    Thi = (whb << (8 - N.h)) ^ H4;                         // two's complement again, field in the top h bits
    // w_low = w - w_high * 2^l; modulo 2^(l+1) that is the low l bits of w plus one borrow bit
    uint32_t lo = (wu ^ (whb << N.l)) & rep8((2u << N.l) - 1u);
    if (!N.comp) {
        // clip to [-2^(l-1), 2^(l-1) - 1]: in the domain lo + 2^l that is [2^(l-1), 3*2^(l-1) - 1]
        uint32_t lob = lo ^ N.bit_l;
        uint32_t half = 1u << (N.l - 1);
        lob = __vminu4(__vmaxu4(lob, rep8(half)), rep8(3u * half - 1u));
        lo = lob & N.mask_l;
    }
    Tlo = lo << (8 - N.lb);
}

// Eq. 5: shift, add the signed low field, clip to INTn.  Returns int8 bytes.
template <class NestT>
__device__ __forceinline__ uint32_t recompose_word(const NestT& N, uint32_t Thi, uint32_t Tlo) {
    uint32_t x = ((Thi >> (8 - N.n)) & N.mask_n) ^ N.bias;     // (w_high + 2^(h-1)) << l
    const uint32_t lo = Tlo >> (8 - N.lb);                      // low-aligned field; stray neighbour bits are masked below
    uint32_t a, s;
    if (N.comp) {          // l+1-bit field: low l bits drop in, the sign bit subtracts 2^l
        a = x | (lo & N.mask_l);
        s = lo & N.bit_l;
    } else {               // l-bit field: lo + 2^(l-1) drops in, then 2^(l-1) comes off
        uint32_t half = rep8(1u << (N.l - 1));
        a = x | ((lo & N.mask_l) ^ half);
        s = half;
    }
    // the only clip that can bind is the lower one (result below -2^(n-1)): an unsigned saturating subtract
    uint32_t wu = (N.comp && N.l == 7) ? subsat_u4(a, s) : subsat_small_u4(a, s);
    return N.n == 8 ? (wu ^ H4) : sub4(wu, N.bias);             // back from the biased domain
}

// (w_int - w_low) / 2^l as an h-bit field
template <class NestT>
__device__ __forceinline__ uint32_t drop_low_word(const NestT& N, uint32_t V, uint32_t Tlo) {
    uint32_t lo = (Tlo >> (8 - N.lb)) & N.mask_lb;
    uint32_t m = rep8(1u << (N.lb - 1));
    uint32_t lo_signed = sub4(lo ^ m, m);
    uint32_t d = sub4(V, lo_signed);
    return ((d >> N.l) & N.mask_h) << (8 - N.h);
}

__device__ __forceinline__ uint32_t values_to_top(uint32_t V, int bits) {
    return (V << (8 - bits)) & rep8(0xffu << (8 - bits));
}
__device__ __forceinline__ uint32_t top_to_values(uint32_t T, int bits) {
    if (bits == 8) return T;
    uint32_t x = (T >> (8 - bits)) & rep8((1u << bits) - 1u);
    uint32_t m = rep8(1u << (bits - 1));
    return sub4(x ^ m, m);
}

// ---------------------------------------------------------------------------------------------
// kernels.  A tensor is rows * groups_per_row * 4 units; the grid strides over units.
// ---------------------------------------------------------------------------------------------
struct TensorView {
    int64_t rows, cols, ld;
    uint8_t* hi;
    uint8_t* lo;
    int8_t* w;
    const uint8_t* mask;
};

enum Op { OP_DECOMPOSE = 0, OP_RECOMPOSE = 1, OP_DROP_LOW = 2, OP_UNPACK = 3, OP_PACK = 4 };

// One unit: `hi` / `lo` point at the unit's block of the respective packed tensor, ru = row-in-block * 4 + unit,
// wrow at the int8 row, c0 is the unit's first column.  A row beyond the tensor (padding of the last row block) is
// written as zero fields by the kernels that produce packed tensors and skipped by the others.
template <int OP, class NestT>
__device__ __forceinline__ void unit_body(const TensorView& t, const NestT& N, int bits, uint8_t* hi, uint8_t* lo, int ru,
                                          int8_t* wrow, const int8_t* mrow, uint32_t c0, bool row_in, bool vec_ok) {
    const bool to_packed = OP == OP_DECOMPOSE || OP == OP_DROP_LOW || OP == OP_PACK;
    if (!row_in && !to_packed) return;
    const int64_t cols = row_in ? t.cols : 0;                 // a padding row reads nothing: all its fields are zero
    uint32_t A[8], Bv[8];
    PackedRaw p0, p1;
    I8Raw v0, v1;
    if (OP == OP_DECOMPOSE) {
        load_i8_raw(wrow, c0, cols, vec_ok, v0);
        load_i8_raw(mrow, c0, cols, vec_ok, v1);
        expand_i8_raw(v0, wrow, c0, cols, A);
        expand_i8_raw(v1, mrow, c0, cols, Bv);
#pragma unroll
        for (int q = 0; q < 8; ++q) decompose_word(N, A[q], Bv[q], A[q], Bv[q]);
        store_unit_top(hi, ru, N.h, A);
        store_unit_top(lo, ru, N.lb, Bv);
    } else if (OP == OP_RECOMPOSE) {
        load_packed_raw(hi, ru, N.h, p0);
        load_packed_raw(lo, ru, N.lb, p1);
        expand_packed_raw(p0, N.h, A);
        expand_packed_raw(p1, N.lb, Bv);
#pragma unroll
        for (int q = 0; q < 8; ++q) A[q] = recompose_word(N, A[q], Bv[q]);
        store_unit_i8(wrow, c0, t.cols, vec_ok, A);
    } else if (OP == OP_DROP_LOW) {
        load_i8_raw(wrow, c0, cols, vec_ok, v0);
        load_packed_raw(lo, ru, N.lb, p1);
        expand_i8_raw(v0, wrow, c0, cols, A);
        expand_packed_raw(p1, N.lb, Bv);
#pragma unroll
        for (int q = 0; q < 8; ++q) A[q] = row_in ? drop_low_word(N, A[q], Bv[q]) : 0u;
        store_unit_top(hi, ru, N.h, A);
    } else if (OP == OP_UNPACK) {
        load_packed_raw(hi, ru, bits, p0);
        expand_packed_raw(p0, bits, A);
#pragma unroll
        for (int q = 0; q < 8; ++q) A[q] = top_to_values(A[q], bits);
        store_unit_i8(wrow, c0, t.cols, vec_ok, A);
    } else {
        load_i8_raw(wrow, c0, cols, vec_ok, v0);
        expand_i8_raw(v0, wrow, c0, cols, A);
#pragma unroll
        for (int q = 0; q < 8; ++q) A[q] = values_to_top(A[q], bits);
        store_unit_top(hi, ru, bits, A);
    }
}

// A thread's share of the work is a PAIR of units 64 rows apart in the same 128 x 128 block, so that one index
// decode and one set of base pointers serves both (these kernels are bound by integer instructions, not by
// bandwidth).  pair_index walks the tensor in this order, fastest first: the 32 lanes of a warp (four units of each
// of eight consecutive rows of one block), the column groups, the eight 8-row bands of the block's upper half, the
// row blocks.  Consecutive warps read or write consecutive 128-byte lines of the same int8 rows; every packed access
// of a warp is one contiguous run of 512 / 256 / 128 bytes.  All index arithmetic is 32-bit (the entry points refuse
// tensors of 2^31 rows, columns or blocks); only the final byte offsets are widened.
template <int OP, class NestT>
__device__ __forceinline__ void do_pair(const TensorView& t, uint32_t pair_index, const NestT& N, int bits) {
    const uint32_t groups = (uint32_t)((t.cols + 127) >> 7);
    const uint32_t wi = pair_index >> 5, x = pair_index & 31u;
    const uint32_t band = wi / groups, g = wi - band * groups;
    const uint32_t rb = band >> 3, r8 = band & 7u;
    const uint32_t blk = rb * groups + g;
    const int ru = (int)(r8 * 32u + x);                       // row-in-block * 4 + unit of the first unit of the pair
    const uint32_t row = rb * 128u + (uint32_t)(ru >> 2);
    const uint32_t c0 = (g * 4u + (x & 3u)) * 32u;
    const int hbits = (OP == OP_UNPACK || OP == OP_PACK) ? bits : N.h;
    uint8_t* hi = t.hi + (uint64_t)blk * (uint32_t)(2048 * hbits);
    uint8_t* lo = (OP == OP_UNPACK || OP == OP_PACK) ? nullptr : t.lo + (uint64_t)blk * (uint32_t)(2048 * N.lb);
    const bool vec_ok = ((t.ld & 15) == 0) && ((reinterpret_cast<uintptr_t>(t.w) & 15) == 0) &&
                        (OP != OP_DECOMPOSE || (reinterpret_cast<uintptr_t>(t.mask) & 15) == 0);
    const uint32_t ld = (uint32_t)t.ld, rows = (uint32_t)t.rows;
    int8_t* wrow = t.w + (uint64_t)row * ld;
    const int8_t* mrow = OP == OP_DECOMPOSE ? reinterpret_cast<const int8_t*>(t.mask) + (uint64_t)row * ld : nullptr;
    if (OP == OP_RECOMPOSE || OP == OP_UNPACK) {
        // packed -> int8 moves few bytes per thread: both units' loads are issued before either is expanded
        const int fb = OP == OP_UNPACK ? bits : N.h;
        PackedRaw a0, a1, b0, b1;
        const bool in0 = row < rows, in1 = row + 64u < rows;
        if (in0) { load_packed_raw(hi, ru, fb, a0); if (OP == OP_RECOMPOSE) load_packed_raw(lo, ru, N.lb, a1); }
        if (in1) { load_packed_raw(hi, ru + 256, fb, b0); if (OP == OP_RECOMPOSE) load_packed_raw(lo, ru + 256, N.lb, b1); }
        uint32_t A[8], Bv[8];
        if (in0) {
            expand_packed_raw(a0, fb, A);
            if (OP == OP_RECOMPOSE) {
                expand_packed_raw(a1, N.lb, Bv);
#pragma unroll
                for (int q = 0; q < 8; ++q) A[q] = recompose_word(N, A[q], Bv[q]);
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) A[q] = top_to_values(A[q], bits);
            }
            store_unit_i8(wrow, c0, t.cols, vec_ok, A);
        }
        if (in1) {
            expand_packed_raw(b0, fb, A);
            if (OP == OP_RECOMPOSE) {
                expand_packed_raw(b1, N.lb, Bv);
#pragma unroll
                for (int q = 0; q < 8; ++q) A[q] = recompose_word(N, A[q], Bv[q]);
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) A[q] = top_to_values(A[q], bits);
            }
            store_unit_i8(wrow + (uint64_t)64 * ld, c0, t.cols, vec_ok, A);
        }
        return;
    }
    unit_body<OP>(t, N, bits, hi, lo, ru, wrow, mrow, c0, row < rows, vec_ok);
    unit_body<OP>(t, N, bits, hi, lo, ru + 256, wrow + (uint64_t)64 * ld, OP == OP_DECOMPOSE ? mrow + (uint64_t)64 * ld : nullptr, c0,
                  row + 64u < rows, vec_ok);
}

template <int OP, class NestT>
__global__ void __launch_bounds__(256, 4) codec_kernel(TensorView t, int64_t total_units, int n, int h, int comp, int bits) {
    const NestT N(n, h, comp);
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total_units; u += stride)
        do_pair<OP>(t, (uint32_t)u, N, bits);
}

// One launch over a whole model.  The model is cut into work items of 256 consecutive unit pairs -- one 128 x 128
// block of one tensor, one pair per thread of a block -- and every item carries all a block needs (base pointers,
// shape, pitch, first pair), so that a thread block reads ONE 48-byte descriptor per item, with no second look-up
// behind it.  Block b takes items b, b + grid, ...; the next item's descriptor is fetched before the current item
// is worked on.  (The first version read an item, then the tensor's table entry, then the data: three dependent
// trips to memory per item, a third of the time of a ResNet-101-sized switch.)
constexpr int kItemUnits = 256;      // unit pairs per work item
constexpr int kBatchBlocksPerSM = 4;
struct BatchItem {
    uint8_t* hi;
    uint8_t* lo;
    int8_t* w;
    int32_t rows, cols, ld;
    uint32_t first_pair;    // first pair of the item inside its tensor
    uint32_t pad_[2];
};
static_assert(sizeof(BatchItem) == 48, "work item is three 16-byte words");

__device__ __forceinline__ BatchItem load_item(const BatchItem* items, int b) {
    const uint4* p = reinterpret_cast<const uint4*>(items + b);
    const uint4 a = __ldg(p), c = __ldg(p + 1), d = __ldg(p + 2);
    BatchItem it;
    it.hi = reinterpret_cast<uint8_t*>(((uint64_t)a.y << 32) | a.x);
    it.lo = reinterpret_cast<uint8_t*>(((uint64_t)a.w << 32) | a.z);
    it.w = reinterpret_cast<int8_t*>(((uint64_t)c.y << 32) | c.x);
    it.rows = (int32_t)c.z; it.cols = (int32_t)c.w; it.ld = (int32_t)d.x; it.first_pair = d.y;
    return it;
}

template <int OP, class NestT>
__global__ void __launch_bounds__(256, 4) codec_batched_kernel(const BatchItem* __restrict__ items, int n_items,
                                                               int n, int h, int comp) {
    const NestT N(n, h, comp);
    int b = blockIdx.x;
    if (b >= n_items) return;
    BatchItem cur = load_item(items, b);
    while (true) {
        const int nb = b + (int)gridDim.x;
        BatchItem nxt = cur;
        if (nb < n_items) nxt = load_item(items, nb);          // in flight while this item is worked on
        TensorView t;
        t.rows = cur.rows; t.cols = cur.cols; t.ld = cur.ld;
        t.hi = cur.hi; t.lo = cur.lo; t.w = cur.w; t.mask = nullptr;
        do_pair<OP>(t, cur.first_pair + threadIdx.x, N, 0);
        if (nb >= n_items) break;
        cur = nxt;
        b = nb;
    }
}

// The paper's packed-bit words (64 // BITS fields per 64-bit word) -> sliced layout.  One thread per 32-element
// unit: it walks the words that hold its fields, drops each field into the top bits of its byte lane of the
// eight top-aligned words, and lets store_unit_top cut the slices -- the same last step as every codec kernel.
template <int BITS>
__global__ void __launch_bounds__(256) word64_to_sliced_kernel(const uint64_t* __restrict__ words, int64_t rows,
                                                               int64_t cols, uint8_t* __restrict__ packed) {
    constexpr int PER = 64 / BITS;
    constexpr uint32_t MASK = (1u << BITS) - 1u;
    const int64_t groups = (cols + 127) >> 7;
    const int64_t units_per_row = groups << 2;
    const int64_t row_words = (cols + PER - 1) / PER;
    const int64_t rows_pad = (rows + 127) / 128 * 128;          // the padding rows of the last block are written as zeros
    const int64_t total = rows_pad * units_per_row;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = u / units_per_row, ur = u - row * units_per_row;
        const int64_t c0 = ur * 32;
        const uint64_t* wrow = words + row * row_words;
        const int64_t cols_here = row < rows ? cols : 0;
        int64_t wi = c0 / PER;
        int fi = (int)(c0 - wi * PER);
        uint64_t w = (c0 < cols_here) ? __ldg(wrow + wi) >> (fi * BITS) : 0ull;
        uint32_t T[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t t = 0;
#pragma unroll
            for (int lane = 0; lane < 4; ++lane) {
                const int j = q * 4 + lane;
                const uint32_t f = (c0 + j < cols_here) ? ((uint32_t)w & MASK) : 0u;
                t |= f << (8 * lane + 8 - BITS);
                w >>= BITS;
                if (++fi == PER) {
                    fi = 0;
                    ++wi;
                    w = (c0 + j + 1 < cols_here) ? __ldg(wrow + wi) : 0ull;
                }
            }
            T[q] = t;
        }
        store_unit_top(packed + ((row >> 7) * groups + (ur >> 2)) * 2048 * BITS, (int)((row & 127) * 4 + (ur & 3)), BITS, T);
    }
}

// unit pairs (the work of one thread, see do_pair) of a [rows, cols] tensor: 256 per 128 x 128 block
inline int64_t walk_units(int64_t rows, int64_t cols) {
    return ((rows + 127) / 128) * ((cols + 127) / 128) * 256;
}
// the 32-bit index arithmetic of the kernels covers tensors below 2^31 rows, row pitch and pairs
inline bool walk_fits(int64_t rows, int64_t cols, int64_t ld) {
    return rows < (1ll << 31) - 128 && cols < (1ll << 31) - 128 && ld < (1ll << 31) && walk_units(rows, cols) < (1ll << 31);
}

inline int launch_blocks(int64_t total_units) {
    int64_t need = (total_units + 255) / 256;
    int64_t cap = (int64_t)nq::sm_count() * 8 * 4;
    return (int)(need < cap ? need : cap);
}

inline bool nest_ok(int n, int h) { return n >= 2 && n <= 8 && h >= 1 && h < n; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// launchers: INT8 nesting gets the compile-time instantiation of its (h, compensate)
template <int OP, class NestT>
void launch_one(const TensorView& t, int64_t total, int n, int h, int comp, int bits, cudaStream_t s) {
    codec_kernel<OP, NestT><<<launch_blocks(total), 256, 0, s>>>(t, total, n, h, comp, bits);
}
template <int OP, class NestT>
void launch_batch(const BatchItem* list, int64_t items, int n, int h, int comp, cudaStream_t s) {
    // as many blocks as are resident at once (four per SM); a block walks the items b, b + grid, ...: with small
    // items the last round is a small part of the whole
    const int64_t resident = (int64_t)nq::sm_count() * kBatchBlocksPerSM;
    const unsigned grid = (unsigned)(items < resident ? items : resident);
    codec_batched_kernel<OP, NestT><<<grid, 256, 0, s>>>(list, (int)items, n, h, comp);
}

template <int OP, int H>
void dispatch_comp(bool batched, const TensorView& t, const BatchItem* table, int count, int64_t total, int comp,
                   cudaStream_t s) {
    if (comp) {
        if (batched) launch_batch<OP, SNest<8, H, 1>>(table, total, 8, H, 1, s);
        else launch_one<OP, SNest<8, H, 1>>(t, total, 8, H, 1, 0, s);
    } else {
        if (batched) launch_batch<OP, SNest<8, H, 0>>(table, total, 8, H, 0, s);
        else launch_one<OP, SNest<8, H, 0>>(t, total, 8, H, 0, 0, s);
    }
}

template <int OP>
void dispatch_nest(bool batched, const TensorView& t, const BatchItem* table, int count, int64_t total, int n, int h,
                   int comp, cudaStream_t s) {
    if (n == 8) {
        switch (h) {
            case 1: return dispatch_comp<OP, 1>(batched, t, table, count, total, comp, s);
            case 2: return dispatch_comp<OP, 2>(batched, t, table, count, total, comp, s);
            case 3: return dispatch_comp<OP, 3>(batched, t, table, count, total, comp, s);
            case 4: return dispatch_comp<OP, 4>(batched, t, table, count, total, comp, s);
            case 5: return dispatch_comp<OP, 5>(batched, t, table, count, total, comp, s);
            case 6: return dispatch_comp<OP, 6>(batched, t, table, count, total, comp, s);
            default: return dispatch_comp<OP, 7>(batched, t, table, count, total, comp, s);
        }
    }
    if (batched) launch_batch<OP, Nest>(table, total, n, h, comp, s);
    else launch_one<OP, Nest>(t, total, n, h, comp, 0, s);
}

template <int OP>
int run_single(TensorView t, int n, int h, int comp, int bits, void* stream) {
    if (t.rows == 0 || t.cols == 0) return NQ_OK;
    if (!walk_fits(t.rows, t.cols, t.ld)) return NQ_ERR_UNSUPPORTED;
    int64_t total = walk_units(t.rows, t.cols);
    if (OP == OP_UNPACK || OP == OP_PACK) launch_one<OP, Nest>(t, total, n, h, comp, bits, (cudaStream_t)stream);
    else dispatch_nest<OP>(false, t, nullptr, 0, total, n, h, comp, (cudaStream_t)stream);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

}  // namespace

namespace nq {
int word64_to_sliced_launch(const uint64_t* words, int bits, int64_t rows, int64_t cols, uint8_t* packed, cudaStream_t s) {
    const int64_t units = ((rows + 127) / 128 * 128) * (((cols + 127) >> 7) << 2);
    const int blocks = launch_blocks(units);
    switch (bits) {
        case 1: word64_to_sliced_kernel<1><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 2: word64_to_sliced_kernel<2><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 3: word64_to_sliced_kernel<3><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 4: word64_to_sliced_kernel<4><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 5: word64_to_sliced_kernel<5><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 6: word64_to_sliced_kernel<6><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        case 7: word64_to_sliced_kernel<7><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
        default: word64_to_sliced_kernel<8><<<blocks, 256, 0, s>>>(words, rows, cols, packed); break;
    }
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}
}  // namespace nq

extern "C" {

int nq_low_bits(int n_bits, int h_bits, int compensate) {
    if (!nest_ok(n_bits, h_bits)) return -1;
    return n_bits - h_bits + (compensate ? 1 : 0);
}

int64_t nq_packed_row_bytes(int64_t cols, int bits) {
    if (cols < 0 || bits < 1 || bits > 8) return -1;
    return ((cols + 127) / 128) * 16 * bits;
}

int64_t nq_packed_bytes(int64_t rows, int64_t cols, int bits) {
    if (rows < 0) return -1;
    int64_t r = nq_packed_row_bytes(cols, bits);
    return r < 0 ? -1 : r * ((rows + 127) / 128 * 128);
}

int nq_decompose(const int8_t* w_int, const uint8_t* mask, int64_t rows, int64_t cols, int64_t ld_w,
                 int n_bits, int h_bits, int compensate, void* packed_high, void* packed_low, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (!nest_ok(n_bits, h_bits)) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!w_int || !mask || !packed_high || !packed_low || ld_w < cols) return NQ_ERR_INVALID_ARG;
    if (!aligned16(packed_high) || !aligned16(packed_low)) return NQ_ERR_ALIGNMENT;
    TensorView t{rows, cols, ld_w, (uint8_t*)packed_high, (uint8_t*)packed_low, (int8_t*)w_int, mask};
    return run_single<OP_DECOMPOSE>(t, n_bits, h_bits, compensate ? 1 : 0, 0, stream);
}

int nq_recompose(const void* packed_high, const void* packed_low, int64_t rows, int64_t cols,
                 int n_bits, int h_bits, int compensate, int8_t* w_int_out, int64_t ld_out, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (!nest_ok(n_bits, h_bits)) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!w_int_out || !packed_high || !packed_low || ld_out < cols) return NQ_ERR_INVALID_ARG;
    if (!aligned16(packed_high) || !aligned16(packed_low)) return NQ_ERR_ALIGNMENT;
    TensorView t{rows, cols, ld_out, (uint8_t*)packed_high, (uint8_t*)packed_low, w_int_out, nullptr};
    return run_single<OP_RECOMPOSE>(t, n_bits, h_bits, compensate ? 1 : 0, 0, stream);
}

int nq_drop_low(const int8_t* w_int, int64_t ld_w, const void* packed_low, int64_t rows, int64_t cols,
                int n_bits, int h_bits, int compensate, void* packed_high_out, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (!nest_ok(n_bits, h_bits)) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!w_int || !packed_high_out || !packed_low || ld_w < cols) return NQ_ERR_INVALID_ARG;
    if (!aligned16(packed_high_out) || !aligned16(packed_low)) return NQ_ERR_ALIGNMENT;
    TensorView t{rows, cols, ld_w, (uint8_t*)packed_high_out, (uint8_t*)packed_low, (int8_t*)w_int, nullptr};
    return run_single<OP_DROP_LOW>(t, n_bits, h_bits, compensate ? 1 : 0, 0, stream);
}

int nq_unpack(const void* packed, int bits, int64_t rows, int64_t cols, int8_t* out, int64_t ld_out, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (bits < 1 || bits > 8) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!packed || !out || ld_out < cols) return NQ_ERR_INVALID_ARG;
    if (!aligned16(packed)) return NQ_ERR_ALIGNMENT;
    TensorView t{rows, cols, ld_out, (uint8_t*)packed, nullptr, out, nullptr};
    return run_single<OP_UNPACK>(t, 8, 4, 1, bits, stream);
}

int nq_pack(const int8_t* values, int64_t ld, int bits, int64_t rows, int64_t cols, void* packed_out, void* stream) {
    if (rows < 0 || cols < 0) return NQ_ERR_INVALID_ARG;
    if (bits < 1 || bits > 8) return NQ_ERR_UNSUPPORTED;
    if (rows == 0 || cols == 0) return NQ_OK;
    if (!values || !packed_out || ld < cols) return NQ_ERR_INVALID_ARG;
    if (!aligned16(packed_out)) return NQ_ERR_ALIGNMENT;
    TensorView t{rows, cols, ld, (uint8_t*)packed_out, nullptr, (int8_t*)values, nullptr};
    return run_single<OP_PACK>(t, 8, 4, 1, bits, stream);
}

static int64_t items_of(const nq_tensor_desc& d) {
    return walk_units(d.rows, d.cols) / kItemUnits;
}

int64_t nq_batch_table_bytes(const nq_tensor_desc* descs, int count) {
    if (count < 0 || (count > 0 && !descs)) return -1;
    int64_t items = 0;
    for (int i = 0; i < count; ++i) {
        if (descs[i].rows < 0 || descs[i].cols < 0) return -1;
        items += items_of(descs[i]);
    }
    return (items > 0 ? items : 1) * (int64_t)sizeof(BatchItem);
}

int nq_batch_plan(const nq_tensor_desc* descs, int count, void* table, int64_t table_bytes,
                  int64_t* work_items_out, void* stream) {
    if (count < 0 || (count > 0 && !descs) || !table || !work_items_out) return NQ_ERR_INVALID_ARG;
    const int64_t need = nq_batch_table_bytes(descs, count);
    if (need < 0) return NQ_ERR_INVALID_ARG;
    if (table_bytes < need) return NQ_ERR_WORKSPACE;
    if (!aligned16(table)) return NQ_ERR_ALIGNMENT;
    std::vector<BatchItem> host((size_t)(need / (int64_t)sizeof(BatchItem)));
    int64_t n_items = 0;
    for (int i = 0; i < count; ++i) {
        const nq_tensor_desc& d = descs[i];
        if (d.ld < d.cols) return NQ_ERR_INVALID_ARG;
        if (!walk_fits(d.rows, d.cols, d.ld)) return NQ_ERR_UNSUPPORTED;
        if (d.rows > 0 && d.cols > 0) {
            if (!d.packed_high || !d.packed_low || !d.w_int) return NQ_ERR_INVALID_ARG;
            if (!aligned16(d.packed_high) || !aligned16(d.packed_low) || !aligned16(d.w_int) || (d.ld & 15))
                return NQ_ERR_ALIGNMENT;
        }
        const int64_t pairs = (d.rows > 0 && d.cols > 0) ? walk_units(d.rows, d.cols) : 0;
        for (int64_t u = 0; u < pairs; u += kItemUnits) {
            BatchItem& it = host[(size_t)n_items++];
            it.hi = (uint8_t*)d.packed_high; it.lo = (uint8_t*)d.packed_low; it.w = d.w_int;
            it.rows = (int32_t)d.rows; it.cols = (int32_t)d.cols; it.ld = (int32_t)d.ld;
            it.first_pair = (uint32_t)u; it.pad_[0] = it.pad_[1] = 0;
        }
    }
    *work_items_out = n_items;
    if (count == 0 || n_items == 0) return NQ_OK;
    // the source is pageable host memory: the runtime stages it before this call returns
    cudaError_t err = cudaMemcpyAsync(table, host.data(), (size_t)n_items * sizeof(BatchItem), cudaMemcpyHostToDevice,
                                      (cudaStream_t)stream);
    return err == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

static int run_batched(int op, const void* table, int count, int64_t units, int n, int h, int comp, void* stream) {
    if (count < 0 || units < 0 || units > 0x7fffffffLL || !table) return NQ_ERR_INVALID_ARG;
    if (!nest_ok(n, h)) return NQ_ERR_UNSUPPORTED;
    if (count == 0 || units == 0) return NQ_OK;
    const BatchItem* entries = reinterpret_cast<const BatchItem*>(table);
    TensorView none{};
    if (op == OP_RECOMPOSE) dispatch_nest<OP_RECOMPOSE>(true, none, entries, count, units, n, h, comp, (cudaStream_t)stream);
    else dispatch_nest<OP_DROP_LOW>(true, none, entries, count, units, n, h, comp, (cudaStream_t)stream);
    return cudaGetLastError() == cudaSuccess ? NQ_OK : NQ_ERR_CUDA;
}

int nq_recompose_batched(const void* table, int count, int64_t work_items, int n_bits, int h_bits, int compensate,
                         void* stream) {
    return run_batched(OP_RECOMPOSE, table, count, work_items, n_bits, h_bits, compensate ? 1 : 0, stream);
}

int nq_drop_low_batched(const void* table, int count, int64_t work_items, int n_bits, int h_bits, int compensate,
                        void* stream) {
    return run_batched(OP_DROP_LOW, table, count, work_items, n_bits, h_bits, compensate ? 1 : 0, stream);
}

}  // extern "C"
