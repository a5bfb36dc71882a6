// The INT8 contraction on CTA pairs (tcgen05 cta_group::2): 256 x 256 output tiles.
//
// Why pairs: with one CTA per 128 x 256 tile every K = 128 stage moves 48 KB into shared memory and the
// tensor core reads 48 KB back out in 512 cycles -- the shared-memory port, not the tensor core, sets the
// pace (measured: ~66 % tensor-pipe activity).  In a pair each CTA stages its own 128 rows of A and only
// HALF of the B tile (128 of 256 rows); the tensor cores of both SMs read the two halves of B from both
// shared memories.  Per SM that is 32 KB in and 32 KB out per stage, and in part-bit mode each SM unpacks
// half as many weights.
//
// Roles per CTA are those of the single-CTA kernel (nq_contraction.cuh): warp 0 TMA producer, warp 1 MMA
// issuer (only in the even, "leader" CTA; it also owns the TMEM allocation in both), warps 2-9 epilogue,
// warps 10-17 unpackers (part-bit), warp 18 producer of the packed-tile ring (part-bit, ring variant).  Barrier protocol, all barriers at the same offsets in both CTAs:
//   full[s]    lives in the leader: 1 arrival by the leader's producer, which announces the bytes of BOTH
//              CTAs' loads; the partner's loads complete on it through its cluster address.  In part-bit
//              mode the leader's unpack warps arrive on it, and each of the partner's unpack warps sends it
//              4 announced bytes with an asynchronous remote store (a cluster-scope release arrival costs
//              the issuing warp over a thousand cycles; measured)
//   empty[s]   one per CTA, arrived on in both CTAs at once by the leader's tcgen05.commit
//   tfull[b]   likewise (accumulator b complete)
//   tempty[b]  lives in the leader: its own epilogue warps arrive, the partner's send 4 announced bytes each
//   pfull / pempty  packed-tile ring, private to each CTA
// DIRECT (part-bit, h = 1, 2, 4): the packed fields never pass through shared memory; each unpack thread reads its
// fields straight from the packed matrix into registers, one turn ahead of their use.  Reason, measured: the
// shared-memory port carries per stage and SM 32 KB of operand reads, 16 KB of A, 16 KB of expanded B and the
// packed tile twice (in by TMA, out to the unpack warps), 64 + 4h KB against 64 KB in the stage's 512 tensor
// cycles, and the part-bit rate followed that sum (0.80 / 0.76 / 0.73 / 0.70 of the full-bit rate for h = 4 .. 7).
// Direct reads lifted h = 4 from 2.40 to 2.93 POP/s at 8192^3; for h >= 5 the narrow slices need two or three
// small loads per unit and the load/store unit becomes the limit instead (h = 7 fell to 1.7), so those keep the
// ring, and so does h = 3 (two loads: 2.71 against 3.14 POP/s).  Tried for h >= 5 and dropped: the 4-bit slice by
// direct reads and only the narrow slices through the ring (2.52 / 2.41 / 1.93 against 2.76 / 2.72 / 2.34, same
// box) -- a direct read exposes the latency of global memory to the unpack warps, the ring's TMA loads run ahead.
// NESTED (full-bit from the two stored parts, Eq. 5): the wider of the two fields (5 to 7 bits) comes through the
// ring of packed tiles, the narrower one (2 to 4 bits) by direct reads -- except the 1-bit slice of a 3-bit narrow
// field, which is loaded into the ring tile behind the wide field's rows, so that every unit needs one direct
// load -- and the unpack warps add them.  Both
// through direct reads ran at a third of the tensor rate: 16 small loads and 36 registers of fields in flight
// per thread spilled, and the reloads sat on the unpack warps' critical path (a block of 18 or 19 warps cannot
// have more than 96 registers per thread: five warps share each quarter of the register file).
// Every wait is bounded; every TMA load has a single destination CTA.
#pragma once
#include "nq_contraction.cuh"

namespace nq {

constexpr int kPairBN = 256;              // tile columns
constexpr int kPairStagesFull = 6;
constexpr int kPairStagesPart = 4;
// The unpack warps work in groups: group g expands the stages whose counter is g modulo the group count, so a
// group has that many stage times for one tile and the fixed per-stage costs (waits, proxy fence, the arrival
// on the leader's barrier across the cluster) of different stages overlap.  Ring depths are multiples of the
// group count, so that a ring slot is always served by the same group, in order: a parity wait is only valid
// for a waiter that is at most one phase behind.
constexpr int kUnpackGroups = 4;
constexpr int kUnpackGroupWarps = kUnpackWarps / kUnpackGroups;
constexpr int kUnpackGroupThreads = kUnpackGroupWarps * 32;
static_assert(kPairStagesPart % kUnpackGroups == 0, "a stage slot must belong to one unpack group");
constexpr int kPairUnitsPerThread = (kPairBN / 2) * 4 / kUnpackGroupThreads;   // 32-field units per stage and thread

__host__ __device__ inline int pair_smem_bytes(bool part, int h_bits, int packed_stages) {
    const int stages = part ? kPairStagesPart : kPairStagesFull;
    int bytes = stages * (a_stage_bytes() + b_stage_bytes(kPairBN / 2));
    if (part) bytes += packed_stages * (kPairBN / 2) * 16 * h_bits;
    bytes += 4 * 2 * kPairBN * (int)sizeof(float);
    bytes += kEpiWarps * kEpiStageBytes;
    bytes += 512;
    return bytes + 1024;
}

struct PairUnpackCtx {
    uint8_t* sB;
    uint64_t* full;
    uint64_t* empty;
    uint32_t* signal_sink;
    volatile int* abort_flag;
    uint32_t rank;
    int pair, num_pairs, num_tiles, group, utid, lane;
};

// A group's position in the pair's sequence of K stages: iteration counter, tile and K block.
struct StageCursor {
    uint32_t it;
    int tile, kb;
};
__device__ __forceinline__ void advance_cursor(StageCursor& c, int steps, int k_blocks, int num_pairs, int num_tiles) {
    c.it += steps;
    c.kb += steps;
    while (c.kb >= k_blocks && c.tile < num_tiles) { c.kb -= k_blocks; c.tile += num_pairs; }
}

// The packed fields of one stage (this CTA's 128 rows of B x one 128-field group: one block of the packed tensor,
// contiguous in memory) into registers.  GROUP_BITS > H: only the leading H bits' worth of slices of a tensor of
// GROUP_BITS-bit fields (they start the block).
template <int H, int GROUP_BITS = H>
__device__ __forceinline__ void fetch_stage(const ContractionArgs& p, const PairUnpackCtx& cx, const StageCursor& c,
                                            PackedUnit (&raw)[kPairUnitsPerThread]) {
    int mt2, nt;
    tile_coords(c.tile, p, mt2, nt);
    const int rb = nt * 2 + (int)cx.rank;                       // this CTA's row block of B
    const int brow = rb * (kPairBN / 2);
    const uint8_t* block = p.packed_b + ((long long)rb * p.packed_groups + c.kb) * (2048 * GROUP_BITS);
#pragma unroll
    for (int i = 0; i < kPairUnitsPerThread; ++i) {
        const int task = i * kUnpackGroupThreads + cx.utid;
        fetch_packed_unit<H>(block, task, brow + (task >> 2) < p.N, raw[i]);
    }
}

// One unpack group of the DIRECT variant: for each of its stages wait for the slot, expand the fields fetched a
// turn earlier into the int8 tile, tell the leader's MMA thread, and only then fetch the fields of its next
// stage -- they have until the group's next turn to arrive.  (Fetching before the proxy fence was slower.)
template <int MODE, int H>
__device__ __forceinline__ void pair_unpack_direct(const ContractionArgs& p, const PairUnpackCtx& cx) {
    using namespace sm100;
    constexpr int HALF = kPairBN / 2;
    constexpr int B_BYTES = b_stage_bytes(HALF);
    PackedUnit raw[kPairUnitsPerThread];
    StageCursor cur{0u, cx.pair, 0};
    advance_cursor(cur, cx.group, p.k_blocks, cx.num_pairs, cx.num_tiles);
    if (cur.tile < cx.num_tiles) fetch_stage<H>(p, cx, cur, raw);
    while (cur.tile < cx.num_tiles) {
        const uint32_t s = cur.it % kPairStagesPart, use = cur.it / kPairStagesPart;
        bool ok = mbar_wait_cluster(smem_u32(&cx.empty[s]), (use & 1) ^ 1, cx.abort_flag, p.status, 0x141u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint8_t* dst = cx.sB + s * B_BYTES;
#pragma unroll
        for (int i = 0; i < kPairUnitsPerThread; ++i) {
            const int task = i * kUnpackGroupThreads + cx.utid;
            uint32_t T[8];
            expand_packed_unit<H>(raw[i], T);
            store_expanded_unit<HALF, MODE>(dst, task >> 2, task & 3, T);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (cx.lane == 0) {
            if (cx.rank == 0) mbar_arrive(smem_u32(&cx.full[s]));
            else signal_remote_tx4(map_to_cta(smem_u32(cx.signal_sink), 0), map_to_cta(smem_u32(&cx.full[s]), 0));
        }
        advance_cursor(cur, kUnpackGroups, p.k_blocks, cx.num_pairs, cx.num_tiles);
        if (cur.tile < cx.num_tiles) fetch_stage<H>(p, cx, cur, raw);
    }
}

// One unpack group of the NESTED variant, INT(NB|H) with the compensated lower field of L1 = NB - H + 1 bits.  The
// wider field is read from the ring tile in shared memory, the narrower one was fetched from global memory a
// turn earlier (p.packed_b is that tensor); Eq. 5 joins them and the stage is handed over as in part-bit mode.
template <int MODE, int H, int NB>
__device__ __forceinline__ void pair_unpack_nested(const ContractionArgs& p, const PairUnpackCtx& cx, const uint8_t* sP,
                                                   int packed_bytes, uint64_t* pfull, uint64_t* pempty) {
    using namespace sm100;
    constexpr int HALF = kPairBN / 2;
    constexpr int B_BYTES = b_stage_bytes(HALF);
    constexpr int L1 = NB - H + 1;
    constexpr bool HIGH_IN_RING = H > L1;
    constexpr int RING_BITS = HIGH_IN_RING ? H : L1;
    constexpr int DIRECT_BITS = HIGH_IN_RING ? L1 : H;
    static_assert(DIRECT_BITS >= 1 && DIRECT_BITS <= 4 && RING_BITS <= 7, "field widths");
    // A 3-bit narrow field would take two small loads per unit (measured a third slower than one): its 1-bit slice
    // rides in the ring tile instead, behind the wide field's rows (a second tile load, 16 bytes a row), and only
    // its 2-bit slice is fetched directly.
    constexpr bool BIT_IN_RING = DIRECT_BITS == 3;
    constexpr int FETCH_BITS = BIT_IN_RING ? 2 : DIRECT_BITS;
    PackedUnit raw[kPairUnitsPerThread];
    StageCursor cur{0u, cx.pair, 0};
    advance_cursor(cur, cx.group, p.k_blocks, cx.num_pairs, cx.num_tiles);
    if (cur.tile < cx.num_tiles) fetch_stage<FETCH_BITS, DIRECT_BITS>(p, cx, cur, raw);
    while (cur.tile < cx.num_tiles) {
        const uint32_t s = cur.it % kPairStagesPart, use = cur.it / kPairStagesPart;
        const uint32_t ps = cur.it % p.packed_stages, puse = cur.it / p.packed_stages;
        bool ok = mbar_wait(smem_u32(&pfull[ps]), puse & 1, cx.abort_flag, p.status, 0x140u) &&
                  mbar_wait_cluster(smem_u32(&cx.empty[s]), (use & 1) ^ 1, cx.abort_flag, p.status, 0x141u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint8_t* src = sP + ps * packed_bytes;
        uint8_t* dst = cx.sB + s * B_BYTES;
#pragma unroll
        for (int i = 0; i < kPairUnitsPerThread; ++i) {
            const int task = i * kUnpackGroupThreads + cx.utid;
            PackedUnit ring;
            load_packed_unit<RING_BITS, HALF>(src, task, ring);
            PackedUnit narrow = raw[i];
            if (BIT_IN_RING)
                narrow.d = *reinterpret_cast<const uint32_t*>(src + HALF * 16 * RING_BITS + task * 4);
            uint32_t T[8], L[8];
            expand_packed_unit<H>(HIGH_IN_RING ? ring : narrow, T);
            expand_packed_unit_at<L1, NB - L1>(HIGH_IN_RING ? narrow : ring, L);
            recompose_unit<NB, L1>(T, L);
            store_expanded_unit<HALF, MODE>(dst, task >> 2, task & 3, T);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (cx.lane == 0) {
            if (cx.rank == 0) mbar_arrive(smem_u32(&cx.full[s]));
            else signal_remote_tx4(map_to_cta(smem_u32(cx.signal_sink), 0), map_to_cta(smem_u32(&cx.full[s]), 0));
            mbar_arrive(smem_u32(&pempty[ps]));
        }
        advance_cursor(cur, kUnpackGroups, p.k_blocks, cx.num_pairs, cx.num_tiles);
        if (cur.tile < cx.num_tiles) fetch_stage<FETCH_BITS, DIRECT_BITS>(p, cx, cur, raw);
    }
}

// The ring variant of part-bit gives the packed-tile producer a warp of its own (the last one): two producers
// that spin in one warp hold each other up for the length of a barrier probe.
__host__ __device__ constexpr int pair_threads(bool part, bool direct) {
    return part ? (direct ? kBaseThreads + kUnpackThreads : kBaseThreads + kUnpackThreads + 32) : kBaseThreads;
}

template <bool PART, int MODE, bool DIRECT = false, int NEST = 0>
__global__ void __launch_bounds__(pair_threads(PART, DIRECT), 1)
contraction_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmAcc,
                        const ContractionArgs p) {
    using namespace sm100;
    constexpr int BN = kPairBN;
    constexpr int HALF = BN / 2;                              // rows of B held by this CTA
    constexpr int STAGES = PART ? kPairStagesPart : kPairStagesFull;
    constexpr int A_BYTES = a_stage_bytes();
    constexpr int B_BYTES = b_stage_bytes(HALF);
    constexpr uint32_t TMEM_COLS = 2 * BN;
    constexpr uint32_t IDESC = idesc_i8(2 * kBM, BN);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = sA + STAGES * A_BYTES;
    const int packed_bytes = PART ? HALF * 16 * p.ring_bits : 0;
    uint8_t* sP = sB + STAGES * B_BYTES;
    float* sScale = reinterpret_cast<float*>(sP + (PART ? p.packed_stages * packed_bytes : 0));   // [4 warps][BN]
    float* sBias = sScale + 4 * BN;
    uint8_t* sStage = reinterpret_cast<uint8_t*>(sBias + 4 * BN);
    uint64_t* full = reinterpret_cast<uint64_t*>(sStage + kEpiWarps * kEpiStageBytes);
    uint64_t* empty = full + STAGES;
    uint64_t* pfull = empty + STAGES;
    uint64_t* pempty = pfull + kMaxPackedStages;
    uint64_t* tfull = pempty + kMaxPackedStages;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint32_t* signal_sink = tmem_slot + 2;                    // landing place of the partner's signal stores

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                  // 0 = leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.m_tiles * p.n_tiles;              // m_tiles counts 256-row tiles here

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&full[s]), PART ? 1 + kUnpackGroupWarps : 1);   // + the leader's unpack group
            mbar_init(smem_u32(&empty[s]), 1);
        }
        for (int s = 0; s < kMaxPackedStages; ++s) {
            mbar_init(smem_u32(&pfull[s]), 1);
            mbar_init(smem_u32(&pempty[s]), kUnpackGroupWarps);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&tfull[b]), 1);
            // the leader's epilogue warps arrive; the partner's send 4 bytes each, announced by the MMA thread
            mbar_init(smem_u32(&tempty[b]), kEpiWarps + 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        if (p.y_tma) prefetch_tensormap(&tmY);
        if (p.acc_tma) prefetch_tensormap(&tmAcc);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                        // both CTAs' barriers exist before anyone signals across
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                int mt2, nt;
                tile_coords(tile, p, mt2, nt);
                const int mt = mt2 * 2 + (int)rank;            // this CTA's 128-row tile
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, use = it / STAGES;
                    if (!(ok = mbar_wait_cluster(smem_u32(&empty[s]), (use & 1) ^ 1, abort_flag, p.status, 0x110u))) break;
                    const uint32_t fb = map_to_cta(smem_u32(&full[s]), 0);        // the leader's barrier
                    int n_sub = 1;
                    if (MODE == kModeConv64) n_sub = min(2, p.g.taps - 2 * kb);
                    const uint32_t a_bytes = (MODE == kModeConv64) ? n_sub * (A_BYTES / 2) : A_BYTES;
                    const uint32_t b_bytes = PART ? 0u : ((MODE == kModeConv64) ? n_sub * (B_BYTES / 2) : B_BYTES);
                    // (part-bit: + 4 bytes from each warp of the partner's unpack group)
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&full[s]), 2 * (a_bytes + b_bytes) + (PART ? 4 * kUnpackGroupWarps : 0));
                    if (MODE == kModeGemm) {
                        tma_load_2d_pair(smem_u32(sA + s * A_BYTES), &tmA, kb * kBK, mt * kBM, fb);
                    } else {
                        const TileOrigin o = conv_tile_origin(p.g, mt);
                        for (int sub = 0; sub < n_sub; ++sub) {
                            const int tap = (MODE == kModeConv64) ? 2 * kb + sub : kb / p.g.cblocks;
                            const int c0 = (MODE == kModeConv64) ? 0 : (kb % p.g.cblocks) * 128;
                            const int r = tap / p.g.S, sx = tap - r * p.g.S;
                            tma_load_4d_pair(smem_u32(sA + s * A_BYTES + sub * (A_BYTES / 2)), &tmA, c0,
                                             o.q0 * p.g.stride - p.g.pad + sx, o.p0 * p.g.stride - p.g.pad + r, o.b0, fb);
                        }
                    }
                    const int brow = nt * BN + (int)rank * HALF;                   // this CTA's half of the B tile
                    if (PART) {
                        // the packed tiles have a ring and a producer lane of their own (below)
                    } else if (MODE == kModeConv64) {
                        for (int sub = 0; sub < n_sub; ++sub)
                            tma_load_2d_pair(smem_u32(sB + s * B_BYTES + sub * (B_BYTES / 2)), &tmB, kb * kBK + sub * 64, brow, fb);
                    } else {
                        tma_load_2d_pair(smem_u32(sB + s * B_BYTES), &tmB, kb * kBK, brow, fb);
                    }
                }
            }
            if (!ok) {
                const long long t0 = clock64();                // let copies in flight land before shared memory is released
                while (clock64() - t0 < (1ll << 22)) { }
            }
        }
    } else if (PART && !DIRECT && warp == kPackedProducerWarp) {
        if (lane == 0) {
            // ---- packed-tile producer: runs ahead of the A loads by up to the depth of its own ring, which
            //      is what hides the latency of fetching the weights
            uint32_t pit = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                int mt2, nt;
                tile_coords(tile, p, mt2, nt);
                const int brow = nt * BN + (int)rank * HALF;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++pit) {
                    const uint32_t ps = pit % p.packed_stages, puse = pit / p.packed_stages;
                    if (!(ok = mbar_wait(smem_u32(&pempty[ps]), (puse & 1) ^ 1, abort_flag, p.status, 0x111u))) break;
                    const uint32_t pb = smem_u32(&pfull[ps]);
                    const int rb = brow >> 7;
                    const bool extra = NEST != 0 && p.ring2 && rb < p.packed_blocks;
                    // the 1-bit slice of a 3-bit narrow field rides behind the wide field's block: 128 rows x 16 bytes, the
                    // last 2048 bytes of the narrow tensor's block
                    if (extra) mbar_expect_tx(pb, 2048);
                    load_ring_slot<HALF>(p, smem_u32(sP + ps * packed_bytes), brow, kb, pb);
                    if (extra)
                        bulk_load(smem_u32(sP + ps * packed_bytes + 2048 * p.ring_field_bits),
                                  p.packed_b + ((long long)rb * p.packed_groups + kb) * (2048 * 3) + 4096, 2048, pb);
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 22)) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs, ++tl) {
                const uint32_t buf = tl & 1, buse = tl >> 1;
                if (!(ok = mbar_wait_cluster(smem_u32(&tempty[buf]), (buse & 1) ^ 1, abort_flag, p.status, 0x120u))) break;
                // this use's hand-back: the leader's warps arrive, the partner's warps each send 4 bytes
                mbar_arrive_expect_tx(smem_u32(&tempty[buf]), 4 * kEpiWarps);
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, use = it / STAGES;
                    if (!(ok = mbar_wait_cluster(smem_u32(&full[s]), use & 1, abort_flag, p.status, 0x121u))) break;
                    tc_fence_after_sync();
                    if (MODE == kModeConv64) {
                        const int n_sub = min(2, p.g.taps - 2 * kb);
                        for (int sub = 0; sub < n_sub; ++sub) {
                            const uint64_t da = smem_desc_sw64(smem_u32(sA + s * A_BYTES + sub * (A_BYTES / 2)));
                            const uint64_t db = smem_desc_sw64(smem_u32(sB + s * B_BYTES + sub * (B_BYTES / 2)));
#pragma unroll
                            for (int k = 0; k < 2; ++k)
                                mma_i8_pair(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | sub | k) != 0);
                        }
                    } else {
                        const uint64_t da = smem_desc_sw128(smem_u32(sA + s * A_BYTES));
                        const uint64_t db = smem_desc_sw128(smem_u32(sB + s * B_BYTES));
#pragma unroll
                        for (int k = 0; k < kBK / 32; ++k)
                            mma_i8_pair(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | k) != 0);
                    }
                    mma_commit_pair(smem_u32(&empty[s]));      // frees the stage in both CTAs
                }
                if (ok) mma_commit_pair(smem_u32(&tfull[buf]));
            }
        }
    } else if (warp < kFirstUnpackWarp) {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        EpilogueCtx ex;
        ex.sScale = sScale; ex.sBias = sBias; ex.sStage = sStage; ex.tfull = tfull; ex.tempty = tempty;
        ex.signal_sink = signal_sink; ex.abort_flag = abort_flag; ex.tmem_base = tmem_base;
        ex.first_tile = pair; ex.tile_step = num_pairs; ex.num_tiles = num_tiles; ex.rank = rank;
        epilogue_role<BN, MODE, true>(p, &tmY, &tmAcc, ex, warp, lane);
    } else if (PART && DIRECT) {
        // ------------------------------------------------------------------ unpackers reading global memory (h <= 4)
        PairUnpackCtx cx;
        cx.sB = sB; cx.full = full; cx.empty = empty; cx.signal_sink = signal_sink; cx.abort_flag = abort_flag;
        cx.rank = rank; cx.pair = pair; cx.num_pairs = num_pairs; cx.num_tiles = num_tiles;
        cx.group = (warp - kFirstUnpackWarp) / kUnpackGroupWarps;
        cx.utid = (threadIdx.x - kBaseThreads) % kUnpackGroupThreads;
        cx.lane = lane;
        switch (p.h_bits) {
            case 1: pair_unpack_direct<MODE, 1>(p, cx); break;
            case 2: pair_unpack_direct<MODE, 2>(p, cx); break;
            case 3: pair_unpack_direct<MODE, 3>(p, cx); break;
            case 4: pair_unpack_direct<MODE, 4>(p, cx); break;
            case 5: pair_unpack_direct<MODE, 5>(p, cx); break;
            case 6: pair_unpack_direct<MODE, 6>(p, cx); break;
            default: pair_unpack_direct<MODE, 7>(p, cx); break;
        }
    } else if (PART && NEST != 0 && warp < kPackedProducerWarp) {
        // ------------------------------------------------------------------ unpackers joining both parts (Eq. 5)
        PairUnpackCtx cx;
        cx.sB = sB; cx.full = full; cx.empty = empty; cx.signal_sink = signal_sink; cx.abort_flag = abort_flag;
        cx.rank = rank; cx.pair = pair; cx.num_pairs = num_pairs; cx.num_tiles = num_tiles;
        cx.group = (warp - kFirstUnpackWarp) / kUnpackGroupWarps;
        cx.utid = (threadIdx.x - kBaseThreads) % kUnpackGroupThreads;
        cx.lane = lane;
        if constexpr (NEST == 8) {
            switch (p.h_bits) {
                case 2: pair_unpack_nested<MODE, 2, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 3: pair_unpack_nested<MODE, 3, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 4: pair_unpack_nested<MODE, 4, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 5: pair_unpack_nested<MODE, 5, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 6: pair_unpack_nested<MODE, 6, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
                default: pair_unpack_nested<MODE, 7, 8>(p, cx, sP, packed_bytes, pfull, pempty); break;
            }
        } else if constexpr (NEST == 6) {
            switch (p.h_bits) {
                case 2: pair_unpack_nested<MODE, 2, 6>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 3: pair_unpack_nested<MODE, 3, 6>(p, cx, sP, packed_bytes, pfull, pempty); break;
                case 4: pair_unpack_nested<MODE, 4, 6>(p, cx, sP, packed_bytes, pfull, pempty); break;
                default: pair_unpack_nested<MODE, 5, 6>(p, cx, sP, packed_bytes, pfull, pempty); break;
            }
        }
    } else if (PART && warp < kPackedProducerWarp) {
        // ------------------------------------------------------------------ unpackers (both CTAs, own half of B)
        const int group = (warp - kFirstUnpackWarp) / kUnpackGroupWarps;
        const int utid = (threadIdx.x - kBaseThreads) % kUnpackGroupThreads;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
            for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                if ((int)(it % kUnpackGroups) != group) continue;
                const uint32_t s = it % STAGES, use = it / STAGES;
                const uint32_t ps = it % p.packed_stages, puse = it / p.packed_stages;
                ok = mbar_wait(smem_u32(&pfull[ps]), puse & 1, abort_flag, p.status, 0x140u) &&
                     mbar_wait_cluster(smem_u32(&empty[s]), (use & 1) ^ 1, abort_flag, p.status, 0x141u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint8_t* src = sP + ps * packed_bytes;
                uint8_t* dst = sB + s * B_BYTES;
                switch (p.h_bits) {
                    case 1: unpack_tile<HALF, MODE, 1, kUnpackGroupThreads>(src, dst, utid); break;
                    case 2: unpack_tile<HALF, MODE, 2, kUnpackGroupThreads>(src, dst, utid); break;
                    case 3: unpack_tile<HALF, MODE, 3, kUnpackGroupThreads>(src, dst, utid); break;
                    case 4: unpack_tile<HALF, MODE, 4, kUnpackGroupThreads>(src, dst, utid); break;
                    case 5: unpack_tile<HALF, MODE, 5, kUnpackGroupThreads>(src, dst, utid); break;
                    case 6: unpack_tile<HALF, MODE, 6, kUnpackGroupThreads>(src, dst, utid); break;
                    default: unpack_tile<HALF, MODE, 7, kUnpackGroupThreads>(src, dst, utid); break;
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&full[s]));
                    else signal_remote_tx4(map_to_cta(smem_u32(signal_sink), 0), map_to_cta(smem_u32(&full[s]), 0));
                    mbar_arrive(smem_u32(&pempty[ps]));
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();          // the partner's shared memory and TMEM stay alive until both CTAs are done
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace nq
