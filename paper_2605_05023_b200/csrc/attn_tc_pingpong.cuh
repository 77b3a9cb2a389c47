// bf16 attention forward on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
// A work item is two query tiles of 128 rows that share every K / V tile: 256 consecutive rows of one (batch,
// query head), or, with an even GQA group, the same 128 rows of two neighbouring heads of one KV group.  Its key
// loop walks the key tiles (128 keys) that any of its rows can see (the Appendix A.2 masks handled here leave
// every row one contiguous key interval; tiles outside it are never loaded: block-level skipping).  The grid has one CTA per work
// item, ordered heaviest first inside L2-sized groups of heads, but a CTA that finishes its item asks
// the hardware scheduler for the next unstarted CTA's index (cluster launch control) and runs that
// item too: one resident CTA per SM processes many items, and the next item's loads and first MMAs
// overlap the previous item's epilogue.
//
// Roles, linked by mbarriers:
//   scheduler warp  one thread fetches the next work item (clusterlaunchcontrol.try_cancel), one item ahead,
//                   decodes it (indices, mask intervals, tile bounds) and publishes it to the other roles;
//   producer warp   TMA loads Q, then K_j / V_j tiles into a ring of shared-memory slots (128-byte
//                   swizzle, the layout tcgen05.mma reads directly);
//   MMA warp        one thread issues S = Q K_j^T (operands in shared memory, fp32 accumulator in
//                   TMEM) and O += P V_j (P read from TMEM, V from shared memory as an MN-major
//                   operand); tcgen05.commit signals completion;
//   softmax groups  128 threads per S buffer, one thread per query row (tcgen05.ld 32x32b: thread i
//                   holds row i): score modifier (Appendix A.1), mask on partial tiles only (loop
//                   splitting, Sec. 3.4), online softmax with lazy rescaling of O, or the sigmoid / ReLU
//                   normaliser (Appendix A.3); P goes back to TMEM over the S columns in two halves so
//                   that P V can start on the first 64 keys.  The same threads run the epilogue.
// D <= 128: NQ = 2, the two query tiles ping-pong so that the softmax of one overlaps the MMAs of the
// other (TMEM: S0 S1 O0 O1).  D = 256 has no TMEM room for two accumulators and runs in attn_tc_pair.cu.
//
// Every mbarrier wait is bounded: after kWaitLimitNs the waiting role records ATTN_ERR_TIMEOUT in the
// caller's status word, raises a CTA-wide abort flag and all roles drain to the common exit, where
// TMEM is released.
#pragma once
#include <algorithm>
#include <cstdlib>
#include <type_traits>

#include <cuda.h>

#include "../../include/attn.h"
#include "attn_params.cuh"
#include "attn_score.cuh"
#include "sm100_ptx.cuh"
#include "attn_tc_common.cuh"

namespace b200attn {

namespace {

using namespace tc;

constexpr int kItemWords = 26;                   // {handed over} + the 25 words of a work item, as published in shared memory


template <int D, int NQ, bool TMA_OUT = false>
struct Cfg {
    static constexpr int kBoxBytes = 64 * 128 * 2;                      // one 64-column TMA box of 128 rows
    static constexpr int kSlotBytes = (D == 64) ? kBoxBytes : 2 * kBoxBytes;
    static constexpr int kSlotsPerTile = 1;                             // one ring slot per K or V tile (used by the producer and MMA roles)
    static constexpr int kStages = (D == 64) ? 8 : 4;
    static constexpr int kQBytes = kBM * D * 2;
    static constexpr int kDataBytes = NQ * kQBytes + kStages * kSlotBytes;
    static constexpr int kBarBytes = 1024;
    static constexpr int kMaxOrdered = TMA_OUT ? 256 : 1024;            // query blocks per head that the weight-ordered work list covers
    static constexpr int kOrderBytes = 2 * kMaxOrdered * 2;             // query-block order and weights (packed documents)
    static constexpr int kStageBytes = 32 * 32 * 2;                     // a 32-row x 32-column bf16 box of O
    static constexpr int kOutBytes = TMA_OUT ? NQ * 4 * 2 * kStageBytes : 0;   // two such boxes per softmax warp
    static constexpr int kSmemBytes = kDataBytes + kOutBytes + kBarBytes + kOrderBytes + 1024;    // + slack to align the base to 1024
    static_assert(kSmemBytes <= 232448, "shared memory budget");
    // Softmax warpgroups first, then one warpgroup holding the producer, MMA and scheduler warps.
    // With NQ = 2 setmaxnreg moves registers from that last warpgroup to the softmax groups.
    static constexpr int kThreads = NQ * 128 + 128;
    static constexpr int kProducerWarp = NQ * 4;
    static constexpr int kMmaWarp = NQ * 4 + 1;
    static constexpr int kSchedWarp = NQ * 4 + 2;
    static constexpr int kRegsSoftmax = 208;
    static constexpr int kRegsOther = 88;
    // setmaxnreg moves registers inside what the CTA was launched with (384 threads x 168 registers, the most that
    // __launch_bounds__(384, 1) allows): a larger sum would leave setmaxnreg.inc waiting for registers for ever.
    static_assert(NQ * 128 * kRegsSoftmax + 128 * kRegsOther <= (NQ * 128 + 128) * 168, "register budget");
    static constexpr int kItemConsumers = NQ * 4 + 2;                   // softmax warps, producer, MMA thread
    static constexpr int kTmemCols = 512;
    static constexpr int kTmemO = 256;                                  // first O column
    static_assert(D == 64 || D == 128, "head dimension");
    static_assert(NQ == 2, "two query tiles per work item");
};

struct Barriers {
    uint64_t q_full[2];      // Q tile landed (TMA)
    uint64_t q_empty[2];     // last QK^T of the item done: the Q tile may be overwritten
    uint64_t full[8];        // ring slot landed (TMA)
    uint64_t empty[8];       // ring slot consumed (tcgen05.commit)
    uint64_t s_full[2];      // S buffer written by QK^T
    uint64_t p_half[2];      // first 64 keys of P written
    uint64_t p_full[2];      // all of P written (and O rescaled if needed)
    uint64_t pv_done[2];     // P V of one key tile done
    uint64_t o_free[2];      // epilogue has read O: the next item may overwrite it
    uint64_t clc;            // response of the hardware scheduler landed (waited on by the scheduler thread only)
    uint64_t item_full;      // next work item published in item_value
    uint64_t item_empty;     // every role has read the published item
    alignas(16) uint64_t item_response[2];   // 16 bytes written by the hardware scheduler (16-byte aligned)
    int item_msg[kItemWords + 1];   // {a work item was handed over, the decoded Item}, written by the scheduler thread
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= 1024, "barrier block");

struct TileRange {
    int jlo, jhi;      // key tiles [jlo, jhi)
};

struct Item {
    int q0t[2], ht[2]; // per query tile: first query row, query head
    int b, g;          // batch, kv head
    // Key tiles per query tile, as positions in the item's key-tile list.  Without global tokens the list is the
    // plain sequence of key tiles (position = tile index).  With global tokens a row sees two pieces, the global
    // keys [0, global_len) and its own interval, so the item's list is {tiles [0, pend)} followed by {tiles
    // [pend + jshift, ...)}: position v stands for tile v when v < pend and for tile v + jshift otherwise, both
    // query tiles walk the whole list (tr[0] = tr[1]; a tile that one of them does not see is masked element-wise
    // there), and only the producer and the softmax groups, which need the real tile, ever translate.
    TileRange tr[2];
    int lo_max[2], hi_min[2];   // per query tile: keys in [lo_max, hi_min] are visible to every row of the tile
    int doc_first[2], doc_last[2];   // per query tile: documents of its first and last row (first > last: unknown)
    float slope[2];    // per query tile: linear-bias slope of its query head (0 without a slope table)
    // Key tiles are walked downwards, from the last one to the first, when rev_top >= 0: position v of the list then
    // stands for tile rev_top - v and tr[] holds positions.  The scheduler asks for it when the heads' position bias
    // has a negative slope (ALiBi): the bias, and with it the row maximum, then falls from tile to tile instead of
    // growing by slope * 128 per tile, which at the steeper slopes forced a rescaling of O at every key step.
    int rev_top;
};
// What the instances for masks with global tokens carry in addition.
struct ItemG : Item {
    int pend, jshift;
    int pre_min[2];    // per query tile: keys below pre_min are visible to every row of the tile
};
template <bool GLB> using ItemT = std::conditional_t<GLB, ItemG, Item>;
// Key tile at position pos of an item's key-tile list.  REV: instances whose scheduler may reverse the walk.
template <bool GLB, bool REV, typename I>
__device__ __forceinline__ int tile_of(const I& it, int pos) {
    if constexpr (GLB) return pos >= it.pend ? pos + it.jshift : pos;
    else if constexpr (REV) return it.rev_top >= 0 ? it.rev_top - pos : pos;
    else return pos;
}


// Key tiles that the rows [q0, q0 + 128) can see, and the keys all of them see.
__device__ __forceinline__ TileRange tile_range(const AttnParams& p, int q0, int& lo_max, int& hi_min, int& doc_first,
                                                int& doc_last) {
    const TileBounds t = tile_bounds(p, q0, kBM);
    lo_max = t.lo_max;
    hi_min = t.hi_min;
    doc_first = t.doc_first;
    doc_last = t.doc_last;
    if (!t.any) return TileRange{0, 0};
    return TileRange{t.lo_min / kBN, t.hi_max / kBN + 1};
}

// Work item of a linear index (work_order in attn_params.cuh: sections of heads whose K/V fit in L2, heaviest query
// block first, the lightest blocks of every head at the very end).  `order`, when not null, lists the query blocks of
// a head heaviest first (packed documents, see build_block_order); otherwise the blocks are taken from the last to
// the first (most keys under a causal mask).
template <int NQ, bool GLB>
__device__ __forceinline__ ItemG decode_item(const AttnParams& p, int lin, const uint16_t* order) {
    // The two query tiles of an item share every K / V tile.  With an even GQA group they are the same 128 rows
    // of two neighbouring query heads of one KV group (identical key ranges: no step in which only one of them
    // has work); otherwise they are 256 consecutive rows of one head (under a causal mask the second tile then
    // sees one key tile more than the first).
    const int pair = p.head_pair;                        // 1: two heads x 128 rows, 0: one head x 256 rows
    const int rows = pair ? kBM : NQ * kBM;
    const int nqb = (p.Sq + rows - 1) / rows;
    const int units = pair ? 2 : 1;                      // query heads per item
    const int bh_total = p.B * p.Hq / units;
    const int sec_units = p.sec_heads / units;
    int rank, bh;                                        // rank of the block among its head's blocks, heaviest first
    // (only masks with global tokens have leading blocks; the other instances keep the plain order's code)
    if constexpr (GLB) work_order_front(lin, bh_total, sec_units, nqb, p.defer_blocks, p.front_blocks, rank, bh, p.sec_merge_from);
    else work_order(lin, bh_total, sec_units, nqb, p.defer_blocks, rank, bh, p.sec_merge_from);
    const int qb = order ? (int)order[rank] : nqb - 1 - rank;
    const int hq_units = p.Hq / units;
    ItemG it;
    it.b = bh / hq_units;
    const int h0 = (bh - it.b * hq_units) * units;
    it.g = h0 / p.group;
    it.ht[0] = h0;
    it.ht[1] = h0 + (pair ? 1 : 0);
    it.q0t[0] = qb * rows;
    it.q0t[1] = qb * rows + (pair ? 0 : kBM);
    it.pend = 0; it.jshift = 0; it.pre_min[0] = it.pre_min[1] = 0;
    if (p.mask_flags & kMaskGlobal) {
        // Union of the two query tiles' key tiles: prefix tiles [0, pend) and window tiles [jlo, jhi).
        int pend = 0, jlo = 0x7fffffff, jhi = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const TileBounds tb = tile_bounds(p, it.q0t[t], kBM);
            it.lo_max[t] = tb.lo_max; it.hi_min[t] = tb.hi_min; it.doc_first[t] = tb.doc_first; it.doc_last[t] = tb.doc_last;
            it.pre_min[t] = tb.pre_min;
            if (!tb.any) continue;
            pend = max(pend, (tb.pre_max + kBN - 1) / kBN);
            if (!(tb.hi_max < 0 || tb.lo_min > tb.hi_max)) { jlo = min(jlo, tb.lo_min / kBN); jhi = max(jhi, tb.hi_max / kBN + 1); }
        }
        if (jlo >= jhi) { jlo = jhi = pend; }                           // only the global tokens are visible
        if (jlo <= pend) { jhi = max(jhi, pend); jlo = 0; pend = 0; }   // the two pieces touch: one sequence
        it.pend = pend;
        it.jshift = jlo - pend;
        it.tr[0] = it.tr[1] = TileRange{0, pend + (jhi - jlo)};
    } else {
        it.tr[0] = tile_range(p, it.q0t[0], it.lo_max[0], it.hi_min[0], it.doc_first[0], it.doc_last[0]);
        if (pair) {
            it.tr[1] = it.tr[0];
            it.lo_max[1] = it.lo_max[0]; it.hi_min[1] = it.hi_min[0];
            it.doc_first[1] = it.doc_first[0]; it.doc_last[1] = it.doc_last[0];
        } else {
            it.tr[1] = tile_range(p, it.q0t[1], it.lo_max[1], it.hi_min[1], it.doc_first[1], it.doc_last[1]);
        }
    }
    it.slope[0] = p.slopes ? __ldg(p.slopes + it.ht[0]) : 0.f;
    it.slope[1] = p.slopes ? __ldg(p.slopes + it.ht[1]) : 0.f;
    it.rev_top = -1;
    if (!GLB && !(p.mask_flags & kMaskGlobal) && (it.slope[0] < 0.f || it.slope[1] < 0.f)) {   // (the global-token instances walk by position only)
        // walk the key tiles downwards: tile j becomes position (top - j)
        int top = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) top = max(top, it.tr[t].jhi);
        if (top > 0) {
#pragma unroll
            for (int t = 0; t < 2; ++t)
                it.tr[t] = (it.tr[t].jlo < it.tr[t].jhi) ? TileRange{top - it.tr[t].jhi, top - it.tr[t].jlo} : TileRange{0, 0};
            it.rev_top = top - 1;
        }
    }
    return it;
}

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* status_word) {
    return bounded_wait_on<false>(bar, parity, &bars->abort_flag, status_word);
}

// Packed documents (Appendix A.2, causal blockwise mask): the number of key tiles of a query block follows its
// position inside its document, not its index, so "last block first" is no longer "heaviest first" and the grid
// would end with a few long items on a few SMs.  Every CTA builds the same heaviest-first order of the query
// blocks once, in shared memory, before its roles start: weight = key tiles of the block's work item; rank =
// blocks that are heavier, plus equally heavy blocks of lower index (a stable counting of all pairs, spread over
// the CTA's threads, with no atomics, so that all CTAs agree on the order).  The order is used when the mask has a
// document (or global-token) clause and the blocks fit the table.
template <int NQ>
__device__ __forceinline__ bool has_block_order(const AttnParams& p, int capacity) {
    const int rows = p.head_pair ? kBM : NQ * kBM;
    return (p.mask_flags & (kMaskDocument | kMaskGlobal)) && (p.Sq + rows - 1) / rows <= capacity;
}
template <int NQ>
__device__ __noinline__ void build_block_order(const AttnParams& p, uint16_t* order, uint16_t* weight, int capacity) {   // (its own registers)
    const int rows = p.head_pair ? kBM : NQ * kBM;
    const int nqb = (p.Sq + rows - 1) / rows;
    if (!has_block_order<NQ>(p, capacity)) return;
    for (int qb = threadIdx.x; qb < nqb; qb += blockDim.x) {
        // key tiles of the block's work item, as decode_item counts them: the window / document tiles [jlo, jhi) and,
        // in front of them, the tiles [0, pend) of the global tokens (the prompt of a Share Question mask is most of
        // an item's keys)
        int jlo = 0x7fffffff, jhi = 0, pend = 0;
        for (int t = 0; t < (p.head_pair ? 1 : NQ); ++t) {
            const TileBounds tb = tile_bounds(p, qb * rows + t * kBM, kBM);
            if (!tb.any) continue;
            pend = max(pend, (tb.pre_max + kBN - 1) / kBN);
            if (tb.hi_max >= 0 && tb.lo_min <= tb.hi_max) { jlo = min(jlo, tb.lo_min / kBN); jhi = max(jhi, tb.hi_max / kBN + 1); }
        }
        const int tiles = (jlo >= jhi) ? pend : (jlo <= pend ? max(jhi, pend) : pend + (jhi - jlo));
        weight[qb] = (uint16_t)min(tiles, 65535);
    }
    __syncthreads();
    for (int qb = threadIdx.x; qb < nqb; qb += blockDim.x) {
        const int w = weight[qb];
        int rank = 0;
        for (int o = 0; o < nqb; ++o) {
            const int wo = weight[o];
            rank += (wo > w || (wo == w && o < qb)) ? 1 : 0;
        }
        order[rank] = (uint16_t)qb;
    }
}

// Waits for the next work item published by the scheduler thread, copies it and (kRelease) releases it.  The
// softmax warps call it with every lane (all lanes need the item) and release once per warp afterwards.
// Returns false when the grid has no unstarted CTA left (or the wait was abandoned).
template <bool kRelease = true, bool GLB = false, bool REV = false>
__device__ __forceinline__ bool next_item(Barriers* bars, uint32_t& phase, int32_t* status_word, ItemT<GLB>& it) {
    if (!bounded_wait(ptx::smem_u32(&bars->item_full), phase, bars, status_word)) return false;
    phase ^= 1u;
    const volatile int* m = bars->item_msg;
    const int got = m[0];
    it.q0t[0] = m[1]; it.q0t[1] = m[2]; it.ht[0] = m[3]; it.ht[1] = m[4]; it.b = m[17]; it.g = m[18];
    it.tr[0].jlo = m[5]; it.tr[0].jhi = m[6]; it.tr[1].jlo = m[7]; it.tr[1].jhi = m[8];
    it.lo_max[0] = m[9]; it.hi_min[0] = m[10]; it.lo_max[1] = m[11]; it.hi_min[1] = m[12];
    it.doc_first[0] = m[13]; it.doc_last[0] = m[14]; it.doc_first[1] = m[15]; it.doc_last[1] = m[16];
    it.slope[0] = __int_as_float(m[19]); it.slope[1] = __int_as_float(m[20]);
    if constexpr (GLB) { it.pend = m[21]; it.jshift = m[22]; it.pre_min[0] = m[23]; it.pre_min[1] = m[24]; }
    if constexpr (REV) it.rev_top = m[25];
    if constexpr (kRelease) ptx::mbar_arrive(ptx::smem_u32(&bars->item_empty));
    return got != 0;
}

// ------------------------------------------------------------------------------------------------
// scheduler: one thread
// ------------------------------------------------------------------------------------------------
// Fetches work items one ahead and decodes them for everybody: the first item is this CTA's own index, the
// following ones are CTAs of the grid that have not started, taken over with cluster launch control (clc_fetch:
// only this thread touches the hardware scheduler's response).  It publishes {handed over, decoded item} with
// ordinary stores for the other roles, so that no role spends time on index arithmetic and mask intervals.
template <int NQ, bool GLB>
__device__ __forceinline__ void scheduler_role(const AttnParams& p, Barriers* bars, int order_capacity) {
    // the heaviest-first order of the query blocks sits right behind the barrier block (see build_block_order)
    const uint16_t* order = has_block_order<NQ>(p, order_capacity) ? reinterpret_cast<const uint16_t*>(reinterpret_cast<const uint8_t*>(bars) + 1024) : nullptr;
    int32_t* status_word = p.status_word;
    uint32_t clc_phase = 0, empty_phase = 0;
    auto publish = [&](bool got, int lin) {
        volatile int* m = bars->item_msg;
        m[0] = got ? 1 : 0;
        if (got) {
            const ItemG it = decode_item<NQ, GLB>(p, lin, order);
            m[1] = it.q0t[0]; m[2] = it.q0t[1]; m[3] = it.ht[0]; m[4] = it.ht[1]; m[17] = it.b; m[18] = it.g;
            m[5] = it.tr[0].jlo; m[6] = it.tr[0].jhi; m[7] = it.tr[1].jlo; m[8] = it.tr[1].jhi;
            m[9] = it.lo_max[0]; m[10] = it.hi_min[0]; m[11] = it.lo_max[1]; m[12] = it.hi_min[1];
            m[13] = it.doc_first[0]; m[14] = it.doc_last[0]; m[15] = it.doc_first[1]; m[16] = it.doc_last[1];
            m[19] = __float_as_int(it.slope[0]); m[20] = __float_as_int(it.slope[1]);
            m[21] = it.pend; m[22] = it.jshift; m[23] = it.pre_min[0]; m[24] = it.pre_min[1];
            m[25] = it.rev_top;
        }
        ptx::mbar_arrive(ptx::smem_u32(&bars->item_full));
    };
    publish(true, (int)blockIdx.x);
    while (true) {
        // every role has copied the published item: fetch the next one
        if (!bounded_wait(ptx::smem_u32(&bars->item_empty), empty_phase, bars, status_word)) return;
        empty_phase ^= 1u;
        bool got;
        uint32_t x;
        if (!clc_fetch(ptx::smem_u32(&bars->clc), bars->item_response, clc_phase, &bars->abort_flag, status_word, got, x)) return;
        publish(got, (int)x);
        if (!got) return;                           // no item left: stop asking
    }
}

// ------------------------------------------------------------------------------------------------
// producer: TMA
// ------------------------------------------------------------------------------------------------
template <int D, int NQ, bool GLB, bool REV>
__device__ __forceinline__ void producer_role(const CUtensorMap* tmap_q, const CUtensorMap* tmap_k,
                                              const CUtensorMap* tmap_v, const AttnParams& p, Barriers* bars,
                                              uint32_t q_smem, uint32_t ring_smem) {
    using C = Cfg<D, NQ>;
    ptx::prefetch_tensormap(tmap_q);
    ptx::prefetch_tensormap(tmap_k);
    ptx::prefetch_tensormap(tmap_v);
    int ps = 0;
    uint32_t pph = 0, item_phase = 0;
    int q_uses[2] = {0, 0};                         // items in which this Q buffer was loaded so far

    using ItemP = ItemT<GLB>;
    // One K tile: one slot holding D/64 boxes of [128 keys x 64 columns].
    auto produce_k = [&](const ItemP& it, int j) -> bool {
#pragma unroll
        for (int sl = 0; sl < C::kSlotsPerTile; ++sl) {
            if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return false;
            const uint32_t bar = ptx::smem_u32(&bars->full[ps]);
            const uint32_t dst = ring_smem + ps * C::kSlotBytes;
            ptx::mbar_arrive_expect_tx(bar, C::kSlotBytes);
#pragma unroll
            for (int bx = 0; bx < C::kSlotBytes / C::kBoxBytes; ++bx)
                ptx::tma_load_4d(dst + bx * C::kBoxBytes, tmap_k, bar, sl * 128 + bx * 64, tile_of<GLB, REV>(it, j) * kBN, it.g, it.b);
            if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        }
        return true;
    };
    // One V tile: one slot of D/64 boxes [128 keys x 64 columns].
    auto produce_v = [&](const ItemP& it, int j) -> bool {
#pragma unroll
        for (int sl = 0; sl < C::kSlotsPerTile; ++sl) {
            if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return false;
            const uint32_t bar = ptx::smem_u32(&bars->full[ps]);
            const uint32_t dst = ring_smem + ps * C::kSlotBytes;
            ptx::mbar_arrive_expect_tx(bar, C::kSlotBytes);
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx)
                ptx::tma_load_4d(dst + bx * C::kBoxBytes, tmap_v, bar, bx * 64, tile_of<GLB, REV>(it, j) * kBN, it.g, it.b);
            if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        }
        return true;
    };

    while (true) {
        ItemP it;
        if (!next_item<true, GLB, REV>(bars, item_phase, p.status_word, it)) return;
        int J0 = 0x7fffffff, J1 = 0;
#pragma unroll
        for (int t = 0; t < NQ; ++t) {
            if (it.tr[t].jlo < it.tr[t].jhi) {
                J0 = min(J0, it.tr[t].jlo);
                J1 = max(J1, it.tr[t].jhi);
                // The previous item's last QK^T must have finished reading this Q buffer.
                if (q_uses[t] > 0 &&
                    !bounded_wait(ptx::smem_u32(&bars->q_empty[t]), (uint32_t)((q_uses[t] - 1) & 1), bars, p.status_word))
                    return;
                ++q_uses[t];
                const uint32_t bar = ptx::smem_u32(&bars->q_full[t]);
                ptx::mbar_arrive_expect_tx(bar, C::kQBytes);
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx)
                    ptx::tma_load_4d(q_smem + t * C::kQBytes + bx * C::kBoxBytes, tmap_q, bar, bx * 64, it.q0t[t], it.ht[t], it.b);
            }
        }
        if (J0 < J1) {
            if (!produce_k(it, J0)) return;
            for (int j = J0; j < J1; ++j) {
                if (!produce_v(it, j)) return;
                if (j + 1 < J1 && !produce_k(it, j + 1)) return;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// MMA issuer (one thread)
// ------------------------------------------------------------------------------------------------
template <int D, int NQ, bool P_HI_LO>
__device__ __forceinline__ void mma_role(const AttnParams& p, Barriers* bars, uint32_t tmem, uint32_t q_smem,
                                         uint32_t ring_smem) {
    using C = Cfg<D, NQ>;
    constexpr int KS = C::kSlotsPerTile;
    constexpr uint32_t kIdescQK = instr_desc(kBM, kBN, false);
    constexpr uint32_t kIdescPV = instr_desc(kBM, D, true);
    // Descriptor halves (128-byte swizzle, SBO = 1024 B, sm_100 version bit): hi is constant per operand kind,
    // lo = (address >> 4) | (LBO >> 4) << 16 advances by compile-time constants inside a tile.
    constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kLoKMajor = 1u << 16;                                             // LBO unused for K-major
    constexpr uint32_t kLoV = (uint32_t)(C::kBoxBytes >> 4) << 16;   // LBO between 64-column blocks
    const uint32_t q_lo = (q_smem >> 4) | kLoKMajor;
    const uint32_t ring_lo = ring_smem >> 4;
    const uint32_t bar_s_full = ptx::smem_u32(&bars->s_full[0]);
    const uint32_t bar_pv_done = ptx::smem_u32(&bars->pv_done[0]);
    const uint32_t bar_p_half = ptx::smem_u32(&bars->p_half[0]);
    const uint32_t bar_p_full = ptx::smem_u32(&bars->p_full[0]);
    const uint32_t bar_full = ptx::smem_u32(&bars->full[0]);
    const uint32_t bar_empty = ptx::smem_u32(&bars->empty[0]);

    int cs = 0;
    uint32_t cph = 0, item_phase = 0;
    uint32_t pph[2] = {0u, 0u};                     // phases of p_half / p_full per S buffer
    int q_uses[2] = {0, 0};                         // items in which tile t was active so far

    auto next_slot = [&](int& slot) -> bool {
        if (!bounded_wait(bar_full + cs * 8, cph, bars, p.status_word)) return false;
        slot = cs;
        if (++cs == C::kStages) { cs = 0; cph ^= 1u; }
        return true;
    };
    // S[buf] = Q[qt] K^T over the whole head dimension; signals s_full[buf].
    auto issue_qk = [&](int qt, int buf, const int (&kslot)[KS]) {
        const uint32_t a_lo = q_lo + (uint32_t)(qt * C::kQBytes >> 4);
        uint32_t b_lo[KS];
#pragma unroll
        for (int sl = 0; sl < KS; ++sl) b_lo[sl] = (ring_lo + (uint32_t)kslot[sl] * (C::kSlotBytes >> 4)) | kLoKMajor;
        const uint32_t d = tmem + buf * kBN;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            constexpr int kPerSlot = D / 16;
            const uint32_t a_off = (uint32_t)(((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            const uint32_t b_off = (uint32_t)((((kk % kPerSlot) / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            ptx::mma_ss_lohi(d, a_lo + a_off, kDescHi, b_lo[kk / kPerSlot] + b_off, kDescHi, kIdescQK, kk > 0 ? 1u : 0u);
        }
        ptx::tc_commit(bar_s_full + buf * 8);
    };
    // O[ocol..] (+)= P[buf] V over keys [16 * kk0, 16 * kk1) of the tile; the second half signals pv_done[qt].
    auto issue_pv = [&](int qt, int buf, uint32_t ocol, const int (&vslot)[KS], bool accumulate, int kk0, int kk1) {
        uint32_t b_lo[KS];
#pragma unroll
        for (int sl = 0; sl < KS; ++sl) b_lo[sl] = (ring_lo + (uint32_t)vslot[sl] * (C::kSlotBytes >> 4)) | kLoV;
        const uint32_t d = tmem + ocol, a = tmem + buf * kBN;
#pragma unroll
        for (int kk = kk0; kk < kk1; ++kk) {
            constexpr int kPerSlot = 8;
            ptx::mma_ts_lohi(d, a + kk * 8, b_lo[kk / kPerSlot] + (uint32_t)(((kk % kPerSlot) * 2048) >> 4), kDescHi, kIdescPV,
                             (accumulate || kk > 0) ? 1u : 0u);
        }
        if (kk1 == kBN / 16) ptx::tc_commit(bar_pv_done + qt * 8);
    };
    // Both halves of P V for one key tile: the first 64 keys as soon as they are written.
    auto wait_p_and_issue_pv = [&](int qt, int buf, uint32_t ocol, const int (&vslot)[KS], bool accumulate) -> bool {
        if (!bounded_wait(bar_p_half + buf * 8, pph[buf], bars, p.status_word)) return false;
        ptx::tc_fence_after_sync();
        issue_pv(qt, buf, ocol, vslot, accumulate, 0, 4);
        if (!bounded_wait(bar_p_full + buf * 8, pph[buf], bars, p.status_word)) return false;
        pph[buf] ^= 1u;
        ptx::tc_fence_after_sync();
        if constexpr (P_HI_LO) {
            // P = P_hi + P_lo (two bf16 tiles, columns [0,64) and [64,128) of the S buffer): the residual tile
            // goes through the same V descriptors before the pass that signals pv_done.
            const uint32_t d = tmem + ocol, a = tmem + buf * kBN + 64;
            uint32_t b_lo[KS];
#pragma unroll
            for (int sl = 0; sl < KS; ++sl) b_lo[sl] = (ring_lo + (uint32_t)vslot[sl] * (C::kSlotBytes >> 4)) | kLoV;
#pragma unroll
            for (int kk = 0; kk < kBN / 16; ++kk) {
                constexpr int kPerSlot = 8;
                ptx::mma_ts_lohi(d, a + kk * 8, b_lo[kk / kPerSlot] + (uint32_t)(((kk % kPerSlot) * 2048) >> 4), kDescHi, kIdescPV, 1u);
            }
        }
        issue_pv(qt, buf, ocol, vslot, true, 4, 8);
        return true;
    };
    // First use of tile t in this item: its Q must have landed.
    auto wait_q = [&](int t) -> bool {
        const bool ok = bounded_wait(ptx::smem_u32(&bars->q_full[t]), (uint32_t)(q_uses[t] & 1), bars, p.status_word);
        ptx::tc_fence_after_sync();
        return ok;
    };
    // Before the first P V of an item overwrites O: the epilogue of the previous item that used this
    // accumulator must have read it.
    auto wait_o_free = [&](int t) -> bool {
        if (q_uses[t] == 0) return true;
        const bool ok = bounded_wait(ptx::smem_u32(&bars->o_free[t]), (uint32_t)((q_uses[t] - 1) & 1), bars, p.status_word);
        ptx::tc_fence_after_sync();
        return ok;
    };

    while (true) {
        Item it;
        if (!next_item(bars, item_phase, p.status_word, it)) return;
        int J0 = 0x7fffffff, J1 = 0;
#pragma unroll
        for (int t = 0; t < NQ; ++t)
            if (it.tr[t].jlo < it.tr[t].jhi) { J0 = min(J0, it.tr[t].jlo); J1 = max(J1, it.tr[t].jhi); }

        if (J0 < J1) {
            int kslot[KS], vslot[KS];
            {
                if (!next_slot(kslot[0])) return;
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (it.tr[t].jlo <= J0 && J0 < it.tr[t].jhi) {
                        if (!wait_q(t)) return;
                        issue_qk(t, t, kslot);
                        if (it.tr[t].jhi == J0 + 1) ptx::tc_commit(ptx::smem_u32(&bars->q_empty[t]));
                    }
                }
                ptx::tc_commit(bar_empty + kslot[0] * 8);
                for (int j = J0; j < J1; ++j) {
                    const bool has_next = (j + 1 < J1);
                    if (!next_slot(vslot[0])) return;
                    if (has_next && !next_slot(kslot[0])) return;
                    ptx::tc_fence_after_sync();
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        const bool act = (it.tr[t].jlo <= j && j < it.tr[t].jhi);
                        const bool act_next = has_next && (it.tr[t].jlo <= j + 1 && j + 1 < it.tr[t].jhi);
                        if (act) {
                            if (j == it.tr[t].jlo && !wait_o_free(t)) return;
                            if (!wait_p_and_issue_pv(t, t, C::kTmemO + t * D, vslot, j > it.tr[t].jlo)) return;
                        }
                        if (act_next) {
                            if (!act && !wait_q(t)) return;     // first key tile of this query tile
                            issue_qk(t, t, kslot);
                            if (it.tr[t].jhi == j + 2) ptx::tc_commit(ptx::smem_u32(&bars->q_empty[t]));
                        }
                    }
                    ptx::tc_commit(bar_empty + vslot[0] * 8);
                    if (has_next) ptx::tc_commit(bar_empty + kslot[0] * 8);
                }
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (it.tr[t].jlo < it.tr[t].jhi) ++q_uses[t];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// softmax / sigmoid groups and epilogue: one thread per query row
// ------------------------------------------------------------------------------------------------

template <int D, int NQ, int SCORE, int NORM, bool GLB, bool TMA_OUT>
__device__ __forceinline__ void softmax_role(const AttnParams& p, Barriers* bars, uint32_t tmem, int qt, const CUtensorMap* tmap_o,
                                             uint32_t stage_smem, uint8_t* stage_ptr) {
    using C = Cfg<D, NQ, TMA_OUT>;
    constexpr bool SIGMOID = (NORM == kNormSigmoid);   // out_scale * sigmoid(s + b), P as a bf16 hi + lo pair
    constexpr bool RELU = (NORM == kNormRelu);         // out_scale * max(s, 0), no exponential at all
    const int wg_thread = threadIdx.x & 127;                 // row within the tile
    const uint32_t lane_base = (uint32_t)((threadIdx.x >> 5) & 3) * 32u;   // TMEM lanes this warp may touch
    const uint32_t tm = tmem + (lane_base << 16);
    const uint32_t ocol = C::kTmemO + (NQ == 2 ? qt * D : 0);

    const float cs = p.scale * kLog2e;                       // raw score -> log2 units
    const float sig_bias2 = p.sigmoid_bias * kLog2e;

    uint32_t g = 0;                                          // key tiles of this query tile processed so far
    uint32_t item_phase = 0;

    while (true) {
        // Every lane copies the published item; the warp releases it once all of them have.
        ItemT<GLB> it;
        const bool got = next_item<false, GLB, SCORE != kScorePlain>(bars, item_phase, p.status_word, it);
        __syncwarp();
        if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->item_empty));
        if (!got) return;
        const int q0 = it.q0t[qt];
        const TileRange tr = it.tr[qt];
        const int row = q0 + wg_thread;
        const int row_c = min(row, p.Sq - 1);                // rows past Sq compute on a valid interval, never stored
        const RowInterval riv = row_interval(p, row_c, it.doc_first[qt], it.doc_last[qt]);
        const int lo_last = it.lo_max[qt], hi_first = it.hi_min[qt];   // keys in [lo_last, hi_first] are visible to every row
        const int ip = row_c + p.Sk - p.Sq;
        ScoreConsts sc = {};
        if constexpr (SCORE != kScorePlain) sc = make_score_consts(p.scale, p.softcap, it.slope[qt]);
        const int niter = tr.jhi - tr.jlo;
        const bool relu_raw = RELU && p.softcap == 0.f && it.slope[qt] == 0.f && p.scale > 0.f;
        const bool sig_raw = SIGMOID && p.softcap == 0.f && it.slope[qt] == 0.f;
        CapPoly poly = {};                                   // softcap: coefficients of a tile's second pass
        float m_used = -INFINITY, l = 0.f;
        // Bias-only score (Appendix A.1): s*scale + slope*(i' - j) in log2 units = s*cs + slope2*(rowoff_chunk - i).
        // The column part -slope2*i is the same for every chunk and key tile: it sits in registers for the whole
        // item and joins the scale multiplication as the addend of one FMA; the chunk part slope2*rowoff_chunk is one
        // scalar per chunk that is added to the chunk's maximum and folded into the exponent's offset.
        uint64_t bias_col[SCORE == kScoreBias ? 16 : 1];
        if constexpr (SCORE == kScoreBias) {
#pragma unroll
            for (int k2 = 0; k2 < 16; ++k2) bias_col[k2] = ptx::pack2(-sc.slope2 * (float)(2 * k2), -sc.slope2 * (float)(2 * k2 + 1));
        }

        for (int n = 0; n < niter; ++n, ++g) {
            const int pos = tr.jlo + n;                          // position in the item's key-tile list (see Item)
            const int kv0 = tile_of<GLB, SCORE != kScorePlain>(it, pos) * kBN;
            const int buf = (NQ == 2) ? qt : (int)(g & 1u);
            const uint32_t ph = (NQ == 2) ? (g & 1u) : ((g >> 1) & 1u);
            // Mask (Appendix A.2): element-wise tests only on tiles that straddle an interval edge.
            bool full_tile = (kv0 >= lo_last) && (kv0 + kBN - 1 <= hi_first);
            if constexpr (GLB) full_tile = full_tile || (kv0 + kBN - 1 < it.pre_min[qt]);
            const int mask_a = riv.lo - kv0, mask_e = riv.hi - kv0;
            const int mask_p = GLB ? riv.pre - kv0 : 0;          // global tokens: the columns below it are visible too
            const float rowoff = (float)(ip - kv0);
            if (!bounded_wait(ptx::smem_u32(&bars->s_full[buf]), ph, bars, p.status_word)) return;
            ptx::tc_fence_after_sync();

            // y: scores in log2 units (SCORE plain: raw, scaled inside the max / exp steps; bias-only: without the
            // chunk's share of the bias), masked to -inf.
            uint32_t y[kBN];
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            float bias_chunk[kBN / 32] = {};
            float mt_bias = -INFINITY;
            float zmax = 0.f;                                    // largest squared raw score of the row in this tile (softcap)
            if constexpr (SCORE == kScoreBias) {
#pragma unroll
                for (int c = 0; c < kBN / 32; ++c) bias_chunk[c] = sc.slope2 * (rowoff - (float)(c * 32));
            }
            // Loading, score modifier, mask and row maximum, compiled twice: the copy for full tiles is straight-line
            // code without the mask blocks (for the softcap instance, whose score code is long, there is one copy
            // with a run-time test instead).
            auto load_score_max = [&](auto masked_tag, bool masked_rt, auto redo_tag) {
                constexpr bool kTag = decltype(masked_tag)::value;
                constexpr bool kRedo = decltype(redo_tag)::value;     // softcap: second pass over a tile (see below)
                (void)kRedo;
                const bool kMasked = kTag || masked_rt;
                ptx::tmem_ld_32x32(tm + buf * kBN, *reinterpret_cast<uint32_t(*)[32]>(&y[0]));
                ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[0]));
    #pragma unroll
                for (int c = 0; c < kBN / 32; ++c) {
                    if (c + 1 < kBN / 32)     // next chunk's TMEM read overlaps this chunk's arithmetic
                        ptx::tmem_ld_32x32(tm + buf * kBN + (c + 1) * 32, *reinterpret_cast<uint32_t(*)[32]>(&y[(c + 1) * 32]));
                    // Score (Appendix A.1)
                    if constexpr (SCORE == kScoreBias) {
                        const uint64_t cs2b = ptx::pack2(sc.cs, sc.cs);
    #pragma unroll
                        for (int k2 = 0; k2 < 16; ++k2) {
                            const uint64_t s2 = ptx::pack2(__uint_as_float(y[c * 32 + 2 * k2]), __uint_as_float(y[c * 32 + 2 * k2 + 1]));
                            float s0, s1;
                            ptx::unpack2(ptx::fma2(s2, cs2b, bias_col[k2]), s0, s1);
                            y[c * 32 + 2 * k2] = __float_as_uint(s0);
                            y[c * 32 + 2 * k2 + 1] = __float_as_uint(s1);
                        }
                    } else if constexpr (SCORE != kScorePlain) {
                        if constexpr (SIGMOID || RELU) {
                            // (ReLU of a plainly scaled score: max(scale * s, 0) = scale * max(s, 0) for scale > 0, so
                            // the raw scores go on and the scale joins the epilogue's factor.)
                            // (Sigmoid of a plainly scaled score: the scale rides in the sigmoid's first FMA, below.)
                            if (!((RELU && relu_raw) || (SIGMOID && sig_raw))) score_chunk32<true>(&y[c * 32], sc, rowoff - (float)(c * 32));
                        }
                        else if constexpr (kRedo) score_chunk32_tile(&y[c * 32], sc, rowoff - (float)(c * 32), poly, zmax);
                        else score_chunk32_lin(&y[c * 32], sc, rowoff - (float)(c * 32), zmax);
                    }
                    if (kMasked) {
                        // One bit test per element (two compares per element made partial tiles cost half as much
                        // again as full ones); the sigmoid and ReLU instances are faster with the compare form.
                        if constexpr (GLB) {
                            if constexpr (SIGMOID || RELU) mask_chunk32_cmp(&y[c * 32], mask_a - c * 32, mask_e - c * 32, mask_p - c * 32);
                            else mask_chunk32_bits(&y[c * 32], mask_a - c * 32, mask_e - c * 32, mask_p - c * 32);
                        } else {
                            if constexpr (SIGMOID || RELU) mask_chunk32_cmp(&y[c * 32], mask_a - c * 32, mask_e - c * 32);
                            else mask_chunk32_bits(&y[c * 32], mask_a - c * 32, mask_e - c * 32);
                        }
                    }
                    if constexpr (!SIGMOID && !RELU) {
    #pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            mx[0] = ptx::max3(mx[0], __uint_as_float(y[c * 32 + i]), __uint_as_float(y[c * 32 + i + 1]));
                            mx[1] = ptx::max3(mx[1], __uint_as_float(y[c * 32 + i + 2]), __uint_as_float(y[c * 32 + i + 3]));
                            mx[2] = ptx::max3(mx[2], __uint_as_float(y[c * 32 + i + 4]), __uint_as_float(y[c * 32 + i + 5]));
                            mx[3] = ptx::max3(mx[3], __uint_as_float(y[c * 32 + i + 6]), __uint_as_float(y[c * 32 + i + 7]));
                        }
                        if constexpr (SCORE == kScoreBias) {     // the chunk's maximum gets the chunk's share of the bias
                            mt_bias = fmaxf(mt_bias, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) + bias_chunk[c]);
                            mx[0] = mx[1] = mx[2] = mx[3] = -INFINITY;
                        }
                    }
                    if (c + 1 < kBN / 32) ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[(c + 1) * 32]));
                }
            };
            if constexpr (SCORE == kScoreGeneric) {
                load_score_max(std::false_type{}, !full_tile, std::false_type{});
                if constexpr (!SIGMOID && !RELU) {
                    // Softcap: the first pass caps with a + b s^2 (scores up to 0.2 of the cap).  A score of this
                    // warp's rows beyond that (rare)?  Then the pass runs once more: with the cubic (up to half the
                    // cap), or, beyond that too, on the tile capped exactly in TMEM with the identity coefficients.
                    if (__any_sync(0xffffffffu, zmax > sc.zl_limit)) {
                        const bool exact = __any_sync(0xffffffffu, zmax > sc.z_limit);
                        if (exact) softcap_exact_in_tmem(tm + buf * kBN, kBN / 32, sc.cap_in, sc.cap_out);
                        poly = cap_poly(sc, exact);
                        mx[0] = mx[1] = mx[2] = mx[3] = -INFINITY;
                        load_score_max(std::false_type{}, !full_tile, std::true_type{});
                    }
                }
            } else {
                if (full_tile) load_score_max(std::false_type{}, false, std::false_type{});
                else load_score_max(std::true_type{}, false, std::false_type{});
            }
            if constexpr (SIGMOID) {
                // Appendix A.3: p = sigmoid(s + b); a masked score (-inf) gives exactly 0.  An unnormalised row can
                // be carried by a few large weights, so bf16 rounding of P (up to 2^-8 relative) would show in O: P is split into
                // P_hi = bf16(p) in columns [0,64) and the residual P_lo = bf16(p - P_hi) in columns [64,128) of the
                // S buffer; the MMA thread accumulates both.  out_scale is applied in the epilogue.
                const float neg_mul = sig_raw ? -sc.cs : -1.0f;     // raw scores in, or scores in log2 units
                const uint64_t nb2 = ptx::pack2(-sig_bias2, -sig_bias2), neg1 = ptx::pack2(neg_mul, neg_mul);
#pragma unroll
                for (int cc = 0; cc < kBN / 32; ++cc) {
                    uint32_t pk[16], pl[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint64_t yy = ptx::pack2(__uint_as_float(y[cc * 32 + 2 * i]), __uint_as_float(y[cc * 32 + 2 * i + 1]));
                        float z0, z1;
                        ptx::unpack2(ptx::fma2(yy, neg1, nb2), z0, z1);                  // -(s + b) in log2 units
                        const float p0 = ptx::rcp_approx(1.0f + ptx::ex2_approx(z0));
                        const float p1 = ptx::rcp_approx(1.0f + ptx::ex2_approx(z1));
                        const uint32_t hi = ptx::pack_bf16x2(p0, p1);
                        pk[i] = hi;
                        pl[i] = ptx::pack_bf16x2(p0 - __uint_as_float(hi << 16), p1 - __uint_as_float(hi & 0xffff0000u));
                    }
                    ptx::tmem_st_32x16(tm + buf * kBN + cc * 16, pk);
                    if (cc == 1) warp_arrive_after_tmem_st(ptx::smem_u32(&bars->p_half[buf]));   // keys 0..63 of P_hi in place
                    // (All 128 scores of the row are already in registers, so the S columns may be overwritten.)
                    ptx::tmem_st_32x16(tm + buf * kBN + 64 + cc * 16, pl);
                }
            } else if constexpr (RELU) {
                // Appendix A.3: p = max(s, 0) in log2 units (the epilogue multiplies by out_scale * ln 2); a masked
                // score (-inf) gives exactly 0.
#pragma unroll
                for (int cc = 0; cc < kBN / 32; ++cc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        pk[i] = ptx::pack_bf16x2(fmaxf(__uint_as_float(y[cc * 32 + 2 * i]), 0.f), fmaxf(__uint_as_float(y[cc * 32 + 2 * i + 1]), 0.f));
                    ptx::tmem_st_32x16(tm + buf * kBN + cc * 16, pk);
                    if (cc == 1) warp_arrive_after_tmem_st(ptx::smem_u32(&bars->p_half[buf]));
                }
            } else {
                float mt = (SCORE == kScoreBias) ? mt_bias : fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                if constexpr (SCORE == kScorePlain) mt *= cs;
                const float m_new = fmaxf(m_used, mt);
                if (n == 0) {
                    m_used = m_new;
                } else {
                    // Lazy rescaling: O and l keep a stale maximum until a row's maximum grows by more than
                    // 2^8; the decision is taken per warp because the TMEM accesses are warp collective.
                    const bool need = (m_new - m_used) > kRescaleThreshold;
                    if (__any_sync(0xffffffffu, need)) {
                        if (!bounded_wait(ptx::smem_u32(&bars->pv_done[qt]), (g - 1u) & 1u, bars, p.status_word)) return;
                        ptx::tc_fence_after_sync();
                        const float alpha = (m_new == -INFINITY) ? 1.0f : ptx::ex2_approx(m_used - m_new);
                        l *= alpha;
                        m_used = m_new;
#pragma unroll 1
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t orr[32];
                            ptx::tmem_ld_32x32(tm + ocol + c * 32, orr);
                            ptx::tmem_wait_ld_regs(orr);
#pragma unroll
                            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * alpha);
                            ptx::tmem_st_32x32(tm + ocol + c * 32, orr);
                        }
                    }
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int cc = 0; cc < kBN / 32; ++cc) {
                    uint32_t pk[16];
                    exp_chunk<SCORE>(&y[cc * 32], cs, (SCORE == kScoreBias) ? neg_m + bias_chunk[cc] : neg_m, sum2, pk);
                    ptx::tmem_st_32x16(tm + buf * kBN + cc * 16, pk);
                    if (cc == 1) warp_arrive_after_tmem_st(ptx::smem_u32(&bars->p_half[buf]));
                }
                float s0, s1, s2, s3;
                ptx::unpack2(ptx::add2(sum2[0], sum2[1]), s0, s1);
                ptx::unpack2(ptx::add2(sum2[2], sum2[3]), s2, s3);
                l += (s0 + s1) + (s2 + s3);
            }
            warp_arrive_after_tmem_st(ptx::smem_u32(&bars->p_full[buf]));
        }

        // Epilogue: O / l (softmax), O * out_scale (sigmoid) or O * out_scale * ln 2 (ReLU: P was kept in log2 units);
        // LSE = ln 2 * (m + log2 l).
        const bool store_row = row < p.Sq;
        if (niter > 0) {
            if (!bounded_wait(ptx::smem_u32(&bars->pv_done[qt]), (g - 1u) & 1u, bars, p.status_word)) return;
            ptx::tc_fence_after_sync();
        }
        const float inv = SIGMOID ? p.out_scale : (RELU ? (relu_raw ? p.out_scale * p.scale : p.out_scale * kLn2) : (l > 0.f ? 1.0f / l : 0.f));
        char* obase = reinterpret_cast<char*>(p.o) +
                      ((long long)it.b * p.os[0] + (long long)it.ht[qt] * p.os[1] + (long long)row * p.os[2]) * (p.o_fp32 ? 4 : 2);
        if constexpr (TMA_OUT) {
            // bf16 output, two heads x 128 rows per item (both tiles end together and their epilogues compete for
            // the load/store unit): the warp's 32 rows x 32 columns go through one of its own two 2 KB boxes
            // in shared memory (64-byte swizzle: the 16-byte piece k of row r sits at piece k ^ ((r >> 1) & 3),
            // conflict free) and leave as one TMA tile store, which also clips rows beyond Sq.  A thread-owns-a-row
            // store to global memory touches 32 lines per instruction; this way the stores cost the load/store
            // unit an eighth of that.  The whole accumulator row is read first: one wait covers all the loads, and
            // the next item's first P V may overwrite the accumulator that much earlier.
            uint32_t oall[D / 32][32];
            if (niter > 0) {
#pragma unroll
                for (int c = 0; c < D / 32; ++c) ptx::tmem_ld_32x32(tm + ocol + c * 32, oall[c]);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) ptx::tmem_wait_ld_regs(oall[c]);
                ptx::tc_fence_before_sync();
                __syncwarp();
                if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->o_free[qt]));
            } else {
#pragma unroll
                for (int c = 0; c < D / 32; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i) oall[c][i] = 0u;
            }
            const int r = threadIdx.x & 31;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                const uint32_t (&orr)[32] = oall[c];
                if (r == 0) ptx::bulk_wait_group_read1();        // the store before last has been read out of its box
                __syncwarp();
                uint4* dst = reinterpret_cast<uint4*>(stage_ptr + (c & 1) * C::kStageBytes + r * 64);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 w;
                    w.x = ptx::pack_bf16x2(__uint_as_float(orr[8 * i]) * inv, __uint_as_float(orr[8 * i + 1]) * inv);
                    w.y = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv);
                    w.z = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv);
                    w.w = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv);
                    dst[i ^ ((r >> 1) & 3)] = w;
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (r == 0) {
                    ptx::tma_store_4d(tmap_o, stage_smem + (c & 1) * C::kStageBytes, c * 32, q0 + (wg_thread & ~31), it.ht[qt], it.b);
                    ptx::bulk_commit_group();
                }
            }
        } else {
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
                uint32_t orr[32];
                if (niter > 0) {
                    ptx::tmem_ld_32x32(tm + ocol + c * 32, orr);
                    ptx::tmem_wait_ld_regs(orr);
                    if (c == D / 32 - 1) {
                        // All of O is in registers: the next item's first P V may overwrite the accumulator.
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(ptx::smem_u32(&bars->o_free[qt]));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) orr[i] = 0u;
                }
                if (p.o_fp32) {
                    if (store_row) {
                        float4* dst = reinterpret_cast<float4*>(obase + c * 128);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[i] = make_float4(__uint_as_float(orr[4 * i]) * inv, __uint_as_float(orr[4 * i + 1]) * inv,
                                                 __uint_as_float(orr[4 * i + 2]) * inv, __uint_as_float(orr[4 * i + 3]) * inv);
                    }
                } else {
                    // bf16 output, 256 consecutive rows per item: under a causal mask the first tile's epilogue runs under the
                    // second tile's last key step, and the threads go on at once, so plain stores by the row's owner are best:
                    // 32 bytes at a time (a whole sector per thread and instruction; with 16-byte stores the exposed epilogue
                    // of the second tile took 3.7 k cycles, nearly all of them in the load/store unit).
                    if (store_row) {
                        char* dst = obase + c * 64;
                        const bool aligned32 = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;     // (always, for dense rows)
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            uint32_t w[8];
#pragma unroll
                            for (int k2 = 0; k2 < 8; ++k2)
                                w[k2] = ptx::pack_bf16x2(__uint_as_float(orr[16 * i + 2 * k2]) * inv, __uint_as_float(orr[16 * i + 2 * k2 + 1]) * inv);
                            if (aligned32) {
                                ptx::st_global_v8(dst + i * 32, w);
                            } else {
                                reinterpret_cast<uint4*>(dst + i * 32)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                                reinterpret_cast<uint4*>(dst + i * 32)[1] = make_uint4(w[4], w[5], w[6], w[7]);
                            }
                        }
                    }
                }
            }
        }
        if (!SIGMOID && !RELU && p.lse && store_row)
            p.lse[((long long)it.b * p.Hq + it.ht[qt]) * p.Sq + row] = (l > 0.f) ? (m_used + ptx::lg2_approx(l)) * kLn2 : -INFINITY;
    }
}

// ------------------------------------------------------------------------------------------------
// kernel
// ------------------------------------------------------------------------------------------------
// GLB: masks with global tokens (two key pieces per row).  TMA_OUT: bf16 output through shared memory and TMA tile
// stores (work items of two heads x 128 rows).
template <int D, int NQ, int SCORE, int NORM, bool GLB, bool TMA_OUT>
__global__ void __launch_bounds__(Cfg<D, NQ>::kThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                   const __grid_constant__ AttnParams p) {
    using C = Cfg<D, NQ, TMA_OUT>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t q_smem = base;
    const uint32_t ring_smem = base + NQ * C::kQBytes;
    Barriers* bars = reinterpret_cast<Barriers*>(smem + C::kDataBytes + C::kOutBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(ptx::smem_u32(&bars->q_full[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->q_empty[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->s_full[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->p_half[t]), 4);
            ptx::mbar_init(ptx::smem_u32(&bars->p_full[t]), 4);
            ptx::mbar_init(ptx::smem_u32(&bars->pv_done[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->o_free[t]), 4);
        }
        for (int s = 0; s < 8; ++s) {
            ptx::mbar_init(ptx::smem_u32(&bars->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&bars->clc), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->item_full), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->item_empty), C::kItemConsumers);
        bars->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0) {
        ptx::tmem_alloc<C::kTmemCols>(ptx::smem_u32(&bars->tmem_base));
        ptx::tmem_relinquish();
    }
    static_assert(C::kBarBytes == 1024, "scheduler_role finds the block order 1024 bytes behind the barriers");
    {
        uint16_t* order = reinterpret_cast<uint16_t*>(smem + C::kDataBytes + C::kOutBytes + C::kBarBytes);
        build_block_order<NQ>(p, order, order + C::kMaxOrdered, C::kMaxOrdered);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

    // NQ = 2: 384 threads x 168 registers at launch; 2 x 128 x 208 + 128 x 88 fits the same budget.
    if (warp < NQ * 4) {
        if constexpr (NQ == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsSoftmax));
        softmax_role<D, NQ, SCORE, NORM, GLB, TMA_OUT>(p, bars, tmem, warp >> 2, &tmap_o, base + C::kDataBytes + warp * 2 * C::kStageBytes,
                                              smem + C::kDataBytes + warp * 2 * C::kStageBytes);
        if (TMA_OUT && lane == 0) ptx::bulk_wait_group0();          // this warp's output boxes have left shared memory
    } else {
        if constexpr (NQ == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
        if (warp == C::kProducerWarp) {
            if (lane == 0) producer_role<D, NQ, GLB, SCORE != kScorePlain>(&tmap_q, &tmap_k, &tmap_v, p, bars, q_smem, ring_smem);
        } else if (warp == C::kMmaWarp) {
            if (lane == 0) mma_role<D, NQ, NORM == kNormSigmoid>(p, bars, tmem, q_smem, ring_smem);
        } else if (warp == C::kSchedWarp) {
            if (lane == 0) scheduler_role<NQ, GLB>(p, bars, C::kMaxOrdered);
        } else if (blockIdx.x == 0 && (p.mask_flags & kMaskDocument)) {
            check_offsets_warp(p.cu, p.num_docs, p.Sq, p.status_word);     // the spare warp of the first CTA
        }
        __syncwarp();
    }

    // Common exit.  After an abort, give copies and MMAs still in flight time to land before
    // shared memory and TMEM are handed back.
    if (*reinterpret_cast<volatile int*>(&bars->abort_flag)) __nanosleep(1000000);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc<C::kTmemCols>(tmem);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// Heads per section of the work order: as many KV heads as keep the section's K and V within about 40 MB of L2, in
// equal sections, whole GQA groups.
inline long long section_heads(const AttnParams& p) {
    const long long kv_bytes = 2ll * p.Sk * p.D * 2;
    long long kv_heads = (40ll << 20) / kv_bytes;
    if (kv_heads < 1) kv_heads = 1;
    const long long bh = (long long)p.B * p.Hq;
    long long sec_max = kv_heads * p.group;
    if (sec_max > bh) sec_max = bh;
    const long long n_sec = (bh + sec_max - 1) / sec_max;
    long long sec = (bh + n_sec - 1) / n_sec;
    return (sec + p.group - 1) / p.group * p.group;
}
// Query blocks per head that open the work order (leading_blocks in attn_params.cuh) when the call runs on the
// global-token instances, the ones that decode such an order: work items of two heads x 128 rows with an even GQA
// group, else one head x 256 rows; the weight-ordered list must cover the blocks (those instances: 1024).
inline int planned_leading_blocks(const AttnParams& p) {
    const int units = (p.group % 2 == 0) ? 2 : 1;
    const long long rows = (units == 2) ? kBM : 2 * kBM;
    const long long nqb = (p.Sq + rows - 1) / rows;
    if (nqb > Cfg<128, 2, false>::kMaxOrdered) return 0;
    return leading_blocks(p, (int)rows, kBN, (int)nqb, section_heads(p) / units, (long long)p.B * p.Hq / units, device_sm_count());
}

template <int D, int NQ, int SCORE, int NORM, bool GLB, bool TMA_OUT>
int launch_instance(AttnParams p, cudaStream_t stream) {
    using C = Cfg<D, NQ, TMA_OUT>;
    auto kernel = attn_fwd_tc_kernel<D, NQ, SCORE, NORM, GLB, TMA_OUT>;
    // The opt-in shared-memory size is a per-device function attribute: set it once per device.
    static SmemAttrFlags attr_set;
    if (!set_smem_attr_once(attr_set, kernel, C::kSmemBytes)) return ATTN_ERR_CUDA;
    CUtensorMap mq, mk, mv, mo;
    if (!make_map(&mq, p.q, p.B, p.Hq, p.Sq, D, p.qs, 128) || !make_map(&mk, p.k, p.B, p.Hkv, p.Sk, D, p.ks, 128) ||
        !make_map(&mv, p.v, p.B, p.Hkv, p.Sk, D, p.vs, 128))
        return ATTN_ERR_CUDA;
    // TMA_OUT instances store bf16 output as tiles of 32 rows x 32 columns; the others get a placeholder map that
    // they never use.
    if (!TMA_OUT) mo = mq;
    else if (!make_map(&mo, p.o, p.B, p.Hq, p.Sq, D, p.os, 32, 32, 64)) return ATTN_ERR_CUDA;
    // Heads per section of the work order: as many KV heads as keep the section's K and V within
    // about 40 MB of L2, in equal sections, whole GQA groups.
    const long long bh = (long long)p.B * p.Hq;
    const long long sec = section_heads(p);
    p.sec_heads = (int)sec;
    // Work items: two heads x 128 rows with an even GQA group, else one head x 256 rows (see decode_item).
    p.head_pair = (p.group % 2 == 0) ? 1 : 0;
    const long long rows = p.head_pair ? kBM : NQ * kBM;
    const long long nqb = (p.Sq + rows - 1) / rows;
    const long long grid = nqb * (bh / (p.head_pair ? 2 : 1));
    if (grid > 0x7fffffffLL) return ATTN_ERR_SHAPE;
    p.defer_blocks = deferred_blocks(p, (int)rows, kBN, (int)nqb, bh / (p.head_pair ? 2 : 1), device_sm_count());
    // (the blocks of global tokens' rows are the first of the weight-ordered list, which needs its table)
    // Packed documents: a section is one or a few heads, and its longest items (a document's last blocks) can take
    // longer than an SM's share of the section, so the last two sections are handed out as one.
    {
        const long long sec_units = sec / (p.head_pair ? 2 : 1), units = bh / (p.head_pair ? 2 : 1);
        const long long sections = (units + sec_units - 1) / sec_units;
        p.sec_merge_from = ((p.mask_flags & kMaskDocument) && sections >= 2) ? (int)(sections - 2) : 0x7fffffff;
    }
    // (the leading blocks are the first of the weight-ordered list; only the global-token instances decode them)
    p.front_blocks = GLB ? planned_leading_blocks(p) : 0;
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(mq, mk, mv, mo, p);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

template <int D, int NQ, bool GLB, bool TMA_OUT>
int launch_for_mask(const AttnParams& p, cudaStream_t stream) {
    if (p.normalizer == kNormSigmoid) return launch_instance<D, NQ, kScoreGeneric, kNormSigmoid, GLB, TMA_OUT>(p, stream);
    if (p.normalizer == kNormRelu) return launch_instance<D, NQ, kScoreGeneric, kNormRelu, GLB, TMA_OUT>(p, stream);
    if (p.softcap > 0.f) return launch_instance<D, NQ, kScoreGeneric, kNormSoftmax, GLB, TMA_OUT>(p, stream);
    if (p.slopes) return launch_instance<D, NQ, kScoreBias, kNormSoftmax, GLB, TMA_OUT>(p, stream);
    return launch_instance<D, NQ, kScorePlain, kNormSoftmax, GLB, TMA_OUT>(p, stream);
}
}  // namespace

}  // namespace b200attn
