// bf16 attention forward on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
// A work item is one query tile of 128 rows of one (batch, query head); its key loop walks the key
// tiles (128 keys) that any of its rows can see (Appendix A.2 masks leave every row one contiguous key
// interval; tiles outside it are never loaded: block-level skipping).  The grid has one CTA per work
// item, ordered heaviest first inside L2-sized groups of heads, but a CTA that finishes its item asks
// the hardware scheduler for the next unstarted CTA's index (cluster launch control) and runs that
// item too: one resident CTA per SM processes many items, and the next item's loads and first MMAs
// overlap the previous item's epilogue.
//
// Roles, linked by mbarriers:
//   scheduler warp  fetches the next work item (clusterlaunchcontrol.try_cancel), one item ahead;
//   producer warp   TMA loads Q, then K_j / V_j tiles into a ring of shared-memory slots (128-byte
//                   swizzle, the layout tcgen05.mma reads directly);
//   MMA warp        one thread issues S = Q K_j^T (operands in shared memory, fp32 accumulator in
//                   TMEM) and O += P V_j (P read from TMEM, V from shared memory as an MN-major
//                   operand); tcgen05.commit signals completion.  S is double buffered: Q K_{j+1}^T
//                   runs while the softmax groups work on S_j;
//   softmax groups  two groups of 128 threads share every S tile: thread i of group w owns row i and
//                   the 64 key columns [64 w, 64 w + 64) (tcgen05.ld 32x32b).  Score modifier
//                   (Appendix A.1), mask on partial tiles only (loop splitting, Sec. 3.4), online
//                   softmax with lazy rescaling of O (row maxima are exchanged between the two
//                   groups through shared memory), or the sigmoid normaliser (Appendix A.3).  P goes
//                   back to TMEM as bf16 over the group's own S columns.  The same threads run the
//                   epilogue, each group on half of the O columns.
// TMEM columns: S0 [0,128), S1 [128,256), O [256, 256 + D).
//
// Every mbarrier wait is bounded: after kWaitLimitNs the waiting role records ATTN_ERR_TIMEOUT in the
// caller's status word, raises a CTA-wide abort flag and all roles drain to the common exit, where
// TMEM is released.  No role waits on anything but mbarriers and the final __syncthreads.
#include <cuda.h>

#include "../../include/attn.h"
#include "attn_params.cuh"
#include "attn_score.cuh"
#include "sm100_ptx.cuh"
#include "attn_tc_common.cuh"

namespace b200attn {

namespace {

using namespace tc;

constexpr int kWgCols = 64;                      // S columns per softmax group


template <int D>
struct Cfg {
    static constexpr int kBoxBytes = 64 * 128 * 2;                      // one 64-column TMA box of 128 rows
    static constexpr int kSlotBytes = (D == 64) ? kBoxBytes : 2 * kBoxBytes;
    static constexpr int kSlotsPerTile = (D == 256) ? 2 : 1;            // K split by d halves, V by key halves
    static constexpr int kStages = (D == 64) ? 8 : (D == 128 ? 6 : 5);
    static constexpr int kQBytes = kBM * D * 2;
    static constexpr int kDataBytes = kQBytes + kStages * kSlotBytes;
    static constexpr int kBarBytes = 1024;
    static constexpr int kXchgBytes = 2 * 2 * kBM * 4;                  // row maxima / sums: [parity][group][row]
    static constexpr int kSmemBytes = kDataBytes + kBarBytes + kXchgBytes;
    // Two softmax warpgroups, then one warpgroup holding the producer, MMA and scheduler warps.
    static constexpr int kThreads = 384;
    static constexpr int kSoftmaxWarps = 8;
    static constexpr int kProducerWarp = 8;
    static constexpr int kMmaWarp = 9;
    static constexpr int kSchedWarp = 10;
    static constexpr int kItemConsumers = kSoftmaxWarps + 2;            // softmax warps, producer, MMA thread
    static constexpr int kTmemCols = 512;
    static constexpr int kTmemO = 256;                                  // first O column
    static_assert(D == 64 || D == 128 || D == 256, "head dimension");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

struct Barriers {
    uint64_t q_full;         // Q tile landed (TMA)
    uint64_t q_empty;        // last QK^T of the item done: the Q tile may be overwritten
    uint64_t full[8];        // ring slot landed (TMA)
    uint64_t empty[8];       // ring slot consumed (tcgen05.commit)
    uint64_t s_full[2];      // S buffer written by QK^T
    uint64_t p_full[2];      // all of P written (and O rescaled if needed)
    uint64_t pv_done;        // P V of one key tile done
    uint64_t o_done;         // last P V of the item done: O is complete
    uint64_t o_free;         // epilogue has read O: the next item may overwrite it
    uint64_t xchg[2];        // both softmax groups have posted their row values
    uint64_t clc;            // response of the hardware scheduler landed (waited on by the scheduler thread only)
    uint64_t item_full;      // next work item published in item_value
    uint64_t item_empty;     // every role has read the published item
    alignas(16) uint64_t item_response[2];   // 16 bytes written by the hardware scheduler (16-byte aligned)
    uint32_t item_value[2];  // {a work item was handed over, its linear index}, written by the scheduler thread
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= 1024, "barrier block");

struct TileRange {
    int jlo, jhi;      // key tiles [jlo, jhi)
    int pend;          // before them the key tiles [0, pend) of the global tokens (pend <= jlo; 0 without them)
};
__device__ __forceinline__ int tile_count(const TileRange& r) { return r.pend + (r.jhi - r.jlo); }
__device__ __forceinline__ int tile_at(const TileRange& r, int n) { return n < r.pend ? n : r.jlo + (n - r.pend); }

struct Item {
    int q0, h, b, g;   // first query row, query head, batch, kv head
    TileRange tr;
};

// Key tiles that the rows [q0, q0 + 128) can see.
__device__ __forceinline__ TileRange tile_range(const AttnParams& p, int q0) {
    const TileBounds t = tile_bounds(p, q0, kBM);
    if (!t.any) return TileRange{0, 0, 0};
    int pend = (t.pre_max + kBN - 1) / kBN;
    if (t.hi_max < 0 || t.lo_min > t.hi_max) return TileRange{pend, pend, pend};     // only the global tokens are visible
    int jlo = t.lo_min / kBN, jhi = t.hi_max / kBN + 1;
    if (jlo <= pend) { jlo = 0; jhi = max(jhi, pend); pend = 0; }                      // the two pieces touch
    return TileRange{jlo, jhi, pend};
}

// Work item of a linear index (work_order in attn_params.cuh: sections of heads whose K/V fit in L2, last query tile
// first).
__device__ __forceinline__ Item decode_item(const AttnParams& p, int lin) {
    const int nqb = (p.Sq + kBM - 1) / kBM;
    const int bh_total = p.B * p.Hq;
    int rank, bh;
    work_order_front(lin, bh_total, p.sec_heads, nqb, 0, p.front_blocks, rank, bh);      // (this kernel defers no blocks)
    // the first blocks (rows of global tokens under a non-causal mask) open the order, the others run from the last down
    const int qb = rank < p.front_blocks ? rank : nqb - 1 - (rank - p.front_blocks);
    Item it;
    it.b = bh / p.Hq;
    it.h = bh - it.b * p.Hq;
    it.g = it.h / p.group;
    it.q0 = qb * kBM;
    it.tr = tile_range(p, it.q0);
    return it;
}

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* status_word) {
    return bounded_wait_on<false>(bar, parity, &bars->abort_flag, status_word);
}

// Waits for the next work item published by the scheduler thread and releases it.
// Returns false when the grid has no unstarted CTA left (or the wait was abandoned).
__device__ __forceinline__ bool next_item(Barriers* bars, uint32_t& phase, int32_t* status_word, int& lin) {
    if (!bounded_wait(ptx::smem_u32(&bars->item_full), phase, bars, status_word)) return false;
    phase ^= 1u;
    const uint32_t got = *reinterpret_cast<volatile uint32_t*>(&bars->item_value[0]);
    lin = (int)*reinterpret_cast<volatile uint32_t*>(&bars->item_value[1]);
    ptx::mbar_arrive(ptx::smem_u32(&bars->item_empty));
    return got != 0;
}

// ------------------------------------------------------------------------------------------------
// scheduler: one thread
// ------------------------------------------------------------------------------------------------
// Only this thread touches the hardware scheduler's response (clc_fetch); it publishes {handed over, index} with
// ordinary stores for the other roles.
__device__ __forceinline__ void scheduler_role(Barriers* bars, int32_t* status_word) {
    uint32_t clc_phase = 0, empty_phase = 1;        // the first wait on item_empty passes at once
    while (true) {
        if (!bounded_wait(ptx::smem_u32(&bars->item_empty), empty_phase, bars, status_word)) return;
        empty_phase ^= 1u;
        bool got;
        uint32_t x;
        if (!clc_fetch(ptx::smem_u32(&bars->clc), bars->item_response, clc_phase, &bars->abort_flag, status_word, got, x)) return;
        *reinterpret_cast<volatile uint32_t*>(&bars->item_value[0]) = got ? 1u : 0u;
        *reinterpret_cast<volatile uint32_t*>(&bars->item_value[1]) = x;
        ptx::mbar_arrive(ptx::smem_u32(&bars->item_full));
        if (!got) return;                           // no item left: stop asking
    }
}

// ------------------------------------------------------------------------------------------------
// producer: TMA
// ------------------------------------------------------------------------------------------------
template <int D>
__device__ __forceinline__ void producer_role(const CUtensorMap* tmap_q, const CUtensorMap* tmap_k,
                                              const CUtensorMap* tmap_v, const AttnParams& p, Barriers* bars,
                                              uint32_t q_smem, uint32_t ring_smem) {
    using C = Cfg<D>;
    ptx::prefetch_tensormap(tmap_q);
    ptx::prefetch_tensormap(tmap_k);
    ptx::prefetch_tensormap(tmap_v);
    int ps = 0;
    uint32_t pph = 0, item_phase = 0;
    int q_uses = 0;                                 // items whose Q was loaded so far
    int lin = blockIdx.x;

    // One K tile: D <= 128 one slot holding D/64 boxes; D = 256 two slots, one per 128-column half.
    auto produce_k = [&](const Item& it, int j) -> bool {
#pragma unroll
        for (int sl = 0; sl < C::kSlotsPerTile; ++sl) {
            if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return false;
            const uint32_t bar = ptx::smem_u32(&bars->full[ps]);
            const uint32_t dst = ring_smem + ps * C::kSlotBytes;
            ptx::mbar_arrive_expect_tx(bar, C::kSlotBytes);
#pragma unroll
            for (int bx = 0; bx < C::kSlotBytes / C::kBoxBytes; ++bx)
                ptx::tma_load_4d(dst + bx * C::kBoxBytes, tmap_k, bar, sl * 128 + bx * 64, j * kBN, it.g, it.b);
            if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        }
        return true;
    };
    // One V tile: D <= 128 one slot of D/64 boxes [128 keys x 64]; D = 256 two slots, one per 64-key half,
    // each holding four boxes [64 keys x 64].
    auto produce_v = [&](const Item& it, int j) -> bool {
#pragma unroll
        for (int sl = 0; sl < C::kSlotsPerTile; ++sl) {
            if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return false;
            const uint32_t bar = ptx::smem_u32(&bars->full[ps]);
            const uint32_t dst = ring_smem + ps * C::kSlotBytes;
            ptx::mbar_arrive_expect_tx(bar, C::kSlotBytes);
            if constexpr (D == 256) {
#pragma unroll
                for (int bx = 0; bx < 4; ++bx)
                    ptx::tma_load_4d(dst + bx * (C::kBoxBytes / 2), tmap_v, bar, bx * 64, j * kBN + sl * 64, it.g, it.b);
            } else {
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx)
                    ptx::tma_load_4d(dst + bx * C::kBoxBytes, tmap_v, bar, bx * 64, j * kBN, it.g, it.b);
            }
            if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        }
        return true;
    };

    while (true) {
        const Item it = decode_item(p, lin);
        const int nt = tile_count(it.tr);
        if (nt > 0) {
            // The previous item's last QK^T must have finished reading the Q buffer.
            if (q_uses > 0 && !bounded_wait(ptx::smem_u32(&bars->q_empty), (uint32_t)((q_uses - 1) & 1), bars, p.status_word))
                return;
            ++q_uses;
            const uint32_t bar = ptx::smem_u32(&bars->q_full);
            ptx::mbar_arrive_expect_tx(bar, C::kQBytes);
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx)
                ptx::tma_load_4d(q_smem + bx * C::kBoxBytes, tmap_q, bar, bx * 64, it.q0, it.h, it.b);
            if (!produce_k(it, tile_at(it.tr, 0))) return;
            for (int n = 0; n < nt; ++n) {
                if (!produce_v(it, tile_at(it.tr, n))) return;
                if (n + 1 < nt && !produce_k(it, tile_at(it.tr, n + 1))) return;
            }
        }
        if (!next_item(bars, item_phase, p.status_word, lin)) return;
    }
}

// ------------------------------------------------------------------------------------------------
// MMA issuer (one thread)
// ------------------------------------------------------------------------------------------------
template <int D, bool P_HI_LO>
__device__ __forceinline__ void mma_role(const AttnParams& p, Barriers* bars, uint32_t tmem, uint32_t q_smem,
                                         uint32_t ring_smem) {
    using C = Cfg<D>;
    constexpr int KS = C::kSlotsPerTile;
    constexpr uint32_t kIdescQK = instr_desc(kBM, kBN, false);
    constexpr uint32_t kIdescPV = instr_desc(kBM, D, true);
    // Descriptor halves (128-byte swizzle, SBO = 1024 B, sm_100 version bit): hi is constant per operand kind,
    // lo = (address >> 4) | (LBO >> 4) << 16 advances by compile-time constants inside a tile.
    constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kLoKMajor = 1u << 16;                                             // LBO unused for K-major
    constexpr uint32_t kLoV = (uint32_t)((D == 256 ? C::kBoxBytes / 2 : C::kBoxBytes) >> 4) << 16;   // LBO between 64-column blocks
    const uint32_t q_lo = (q_smem >> 4) | kLoKMajor;
    const uint32_t ring_lo = ring_smem >> 4;
    const uint32_t bar_s_full = ptx::smem_u32(&bars->s_full[0]);
    const uint32_t bar_pv_done = ptx::smem_u32(&bars->pv_done);
    const uint32_t bar_p_full = ptx::smem_u32(&bars->p_full[0]);
    const uint32_t bar_full = ptx::smem_u32(&bars->full[0]);
    const uint32_t bar_empty = ptx::smem_u32(&bars->empty[0]);
    const uint32_t bar_q_empty = ptx::smem_u32(&bars->q_empty);

    int cs = 0;
    uint32_t cph = 0, item_phase = 0;
    uint32_t pph[2] = {0u, 0u};                     // phase of p_full per S buffer
    int q_uses = 0;                                 // items with at least one key tile so far
    uint32_t g = 0;                                 // key tiles processed so far (selects the S buffer)
    int lin = blockIdx.x;

    auto next_slot = [&](int& slot) -> bool {
        if (!bounded_wait(bar_full + cs * 8, cph, bars, p.status_word)) return false;
        slot = cs;
        if (++cs == C::kStages) { cs = 0; cph ^= 1u; }
        return true;
    };
    // S[buf] = Q K^T over the whole head dimension; signals s_full[buf].
    auto issue_qk = [&](int buf, const int (&kslot)[KS]) {
        uint32_t b_lo[KS];
#pragma unroll
        for (int sl = 0; sl < KS; ++sl) b_lo[sl] = (ring_lo + (uint32_t)kslot[sl] * (C::kSlotBytes >> 4)) | kLoKMajor;
        const uint32_t d = tmem + buf * kBN;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            constexpr int kPerSlot = (D == 256) ? 8 : D / 16;
            const uint32_t a_off = (uint32_t)(((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            const uint32_t b_off = (uint32_t)((((kk % kPerSlot) / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            ptx::mma_ss_lohi(d, q_lo + a_off, kDescHi, b_lo[kk / kPerSlot] + b_off, kDescHi, kIdescQK, kk > 0 ? 1u : 0u);
        }
        ptx::tc_commit(bar_s_full + buf * 8);
    };
    // O (+)= P[buf] V over the 128 keys of the tile.  Softmax group w wrote the bf16 P of keys [64 w, 64 w + 64)
    // over its own S columns, starting at column 64 w (+ col_off for the residual tile of the sigmoid path).
    auto issue_pv = [&](int buf, const int (&vslot)[KS], bool accumulate, uint32_t col_off) {
        uint32_t b_lo[KS];
#pragma unroll
        for (int sl = 0; sl < KS; ++sl) b_lo[sl] = (ring_lo + (uint32_t)vslot[sl] * (C::kSlotBytes >> 4)) | kLoV;
        const uint32_t d = tmem + C::kTmemO, a = tmem + buf * kBN + col_off;
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk) {
            constexpr int kPerSlot = (D == 256) ? 4 : 8;
            ptx::mma_ts_lohi(d, a + (kk / 4) * kWgCols + (kk % 4) * 8,
                             b_lo[kk / kPerSlot] + (uint32_t)(((kk % kPerSlot) * 2048) >> 4), kDescHi, kIdescPV,
                             (accumulate || kk > 0) ? 1u : 0u);
        }
    };

    while (true) {
        const Item it = decode_item(p, lin);
        const int J0 = 0, J1 = tile_count(it.tr);     // positions in the item's key-tile list (the ring holds them in order)
        if (J0 < J1) {
            int kslot[KS], vslot[KS];
#pragma unroll
            for (int sl = 0; sl < KS; ++sl)
                if (!next_slot(kslot[sl])) return;
            if (!bounded_wait(ptx::smem_u32(&bars->q_full), (uint32_t)(q_uses & 1), bars, p.status_word)) return;
            ptx::tc_fence_after_sync();
            issue_qk((int)(g & 1u), kslot);
            if (J1 == J0 + 1) ptx::tc_commit(bar_q_empty);
#pragma unroll
            for (int sl = 0; sl < KS; ++sl) ptx::tc_commit(bar_empty + kslot[sl] * 8);
            for (int j = J0; j < J1; ++j, ++g) {
                const int buf = (int)(g & 1u);
                const bool has_next = (j + 1 < J1);
#pragma unroll
                for (int sl = 0; sl < KS; ++sl)
                    if (!next_slot(vslot[sl])) return;
                if (has_next) {
#pragma unroll
                    for (int sl = 0; sl < KS; ++sl)
                        if (!next_slot(kslot[sl])) return;
                    ptx::tc_fence_after_sync();
                    issue_qk(buf ^ 1, kslot);
                    if (J1 == j + 2) ptx::tc_commit(bar_q_empty);
#pragma unroll
                    for (int sl = 0; sl < KS; ++sl) ptx::tc_commit(bar_empty + kslot[sl] * 8);
                }
                // Before the first P V of an item overwrites O: the epilogue of the previous item must have read it.
                if (j == J0 && q_uses > 0) {
                    if (!bounded_wait(ptx::smem_u32(&bars->o_free), (uint32_t)((q_uses - 1) & 1), bars, p.status_word)) return;
                }
                if (!bounded_wait(bar_p_full + buf * 8, pph[buf], bars, p.status_word)) return;
                pph[buf] ^= 1u;
                ptx::tc_fence_after_sync();
                if constexpr (P_HI_LO) {
                    // P = P_hi + P_lo, two bf16 tiles 32 columns apart inside each group's S columns.
                    issue_pv(buf, vslot, j > J0, 32u);
                    issue_pv(buf, vslot, true, 0u);
                } else {
                    issue_pv(buf, vslot, j > J0, 0u);
                }
                ptx::tc_commit(bar_pv_done);
                if (!has_next) ptx::tc_commit(ptx::smem_u32(&bars->o_done));
#pragma unroll
                for (int sl = 0; sl < KS; ++sl) ptx::tc_commit(bar_empty + vslot[sl] * 8);
            }
            ++q_uses;
        }
        if (!next_item(bars, item_phase, p.status_word, lin)) return;
    }
}

// ------------------------------------------------------------------------------------------------
// softmax / sigmoid groups and epilogue: thread i of group w owns row i, key columns [64 w, 64 w + 64)
// ------------------------------------------------------------------------------------------------

template <int D, int SCORE, int NORM>
__device__ __forceinline__ void softmax_role(const AttnParams& p, Barriers* bars, float* xchg, uint32_t tmem, int wg) {
    using C = Cfg<D>;
    constexpr bool SIGMOID = (NORM == kNormSigmoid);   // out_scale * sigmoid(s + b), P as a bf16 hi + lo pair
    constexpr bool RELU = (NORM == kNormRelu);         // out_scale * max(s, 0), no exponential at all
    constexpr int kOC = D / 2;                                // O columns handled by each group
    const int wg_thread = threadIdx.x & 127;                 // row within the tile
    const uint32_t lane_base = (uint32_t)((threadIdx.x >> 5) & 3) * 32u;   // TMEM lanes this warp may touch
    const uint32_t tm = tmem + (lane_base << 16);
    const int col0 = wg * kWgCols;                            // first S column of this group
    const uint32_t ocol = C::kTmemO + wg * kOC;

    const float cs = p.scale * kLog2e;                       // raw score -> log2 units
    const float sig_bias2 = p.sigmoid_bias * kLog2e;

    uint32_t g = 0;                                          // key tiles processed so far
    uint32_t xg = 0;                                         // exchange steps so far
    uint32_t items_done = 0;                                 // items with at least one key tile finished so far

    uint32_t item_phase = 0;
    int lin = blockIdx.x;

    // Posts this thread's value for its row and returns the other group's value for the same row.
    auto exchange = [&](float mine, float& theirs) -> bool {
        const uint32_t par = xg & 1u, ph = (xg >> 1) & 1u;
        ++xg;
        xchg[(par * 2 + wg) * kBM + wg_thread] = mine;
        warp_arrive(ptx::smem_u32(&bars->xchg[par]));
        if (!bounded_wait(ptx::smem_u32(&bars->xchg[par]), ph, bars, p.status_word)) return false;
        theirs = xchg[(par * 2 + (wg ^ 1)) * kBM + wg_thread];
        return true;
    };

    while (true) {
        const Item it = decode_item(p, lin);
        const int q0 = it.q0;
        const TileRange tr = it.tr;
        const int row = q0 + wg_thread;
        const int row_c = min(row, p.Sq - 1);                // rows past Sq compute on a valid interval, never stored
        const RowInterval riv = row_interval(p, row_c);
        const TileBounds tb = tile_bounds(p, q0, kBM);
        const int lo_last = tb.lo_max, hi_first = tb.hi_min;   // keys in [lo_last, hi_first] are visible to every row
        const int ip = row_c + p.Sk - p.Sq;
        ScoreConsts sc = {};
        if constexpr (SCORE != kScorePlain) sc = make_score_consts(p.scale, p.softcap, p.slopes ? __ldg(p.slopes + it.h) : 0.f);
        const int niter = tile_count(tr);
        float m_used = -INFINITY, l = 0.f;                   // l: this group's share of the row sum
        // D = 256 (values of larger magnitude, 256 columns per row): the row sum that normalises O is taken over the
        // bf16-rounded weights that P V uses, so that O is an exactly normalised average of V rows (the rounding of a
        // dominant weight would otherwise show in O); the LSE uses a second, unrounded sum.
        constexpr bool kRoundedSum = (D == 256);
        float l_exact = 0.f;

        for (int n = 0; n < niter; ++n, ++g) {
            const int kv0 = tile_at(tr, n) * kBN;
            const int buf = (int)(g & 1u);
            const uint32_t ph = (g >> 1) & 1u;
            // Mask (Appendix A.2): element-wise tests only on tiles that straddle an interval edge.
            const bool full_tile = ((kv0 >= lo_last) && (kv0 + kBN - 1 <= hi_first)) || (kv0 + kBN - 1 < tb.pre_min);
            const int mask_a = riv.lo - kv0 - col0, mask_e = riv.hi - kv0 - col0;   // visible columns of this group
            const int mask_p = riv.pre - kv0 - col0;                                // and the columns below it (global tokens)
            const float rowoff = (float)(ip - kv0 - col0);
            const uint32_t ts = tm + buf * kBN + col0;        // this thread's lane, this group's S / P columns
            if (!bounded_wait(ptx::smem_u32(&bars->s_full[buf]), ph, bars, p.status_word)) return;
            ptx::tc_fence_after_sync();

            // y: scores in log2 units (SCORE plain: raw, scaled inside the max / exp steps), masked to -inf.
            uint32_t y[kWgCols];
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            ptx::tmem_ld_32x32(ts, *reinterpret_cast<uint32_t(*)[32]>(&y[0]));
            ptx::tmem_ld_32x32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&y[32]));
            ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[0]));
            ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[32]));
#pragma unroll
            for (int c = 0; c < kWgCols / 32; ++c) {
                // Score (Appendix A.1)
                if constexpr (SCORE != kScorePlain) score_chunk32<SCORE == kScoreGeneric>(&y[c * 32], sc, rowoff - (float)(c * 32));
                // the row's interval and, for global tokens, the columns below mask_p
                if (!full_tile) mask_chunk32_bits(&y[c * 32], mask_a - c * 32, mask_e - c * 32, mask_p - c * 32);
                if constexpr (!SIGMOID && !RELU) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        mx[0] = ptx::max3(mx[0], __uint_as_float(y[c * 32 + i]), __uint_as_float(y[c * 32 + i + 1]));
                        mx[1] = ptx::max3(mx[1], __uint_as_float(y[c * 32 + i + 2]), __uint_as_float(y[c * 32 + i + 3]));
                        mx[2] = ptx::max3(mx[2], __uint_as_float(y[c * 32 + i + 4]), __uint_as_float(y[c * 32 + i + 5]));
                        mx[3] = ptx::max3(mx[3], __uint_as_float(y[c * 32 + i + 6]), __uint_as_float(y[c * 32 + i + 7]));
                    }
                }
            }

            if constexpr (SIGMOID) {
                // Appendix A.3: p = sigmoid(s + b); a masked score (-inf) gives exactly 0.  An unnormalised row can
                // be carried by a few large weights, so bf16 rounding of P (up to 2^-8 relative) would show in O: P is split into
                // P_hi = bf16(p) in this group's columns [0,32) and the residual P_lo = bf16(p - P_hi) in its columns
                // [32,64); the MMA thread accumulates both.  out_scale is applied in the epilogue.
                const uint64_t nb2 = ptx::pack2(-sig_bias2, -sig_bias2), neg1 = ptx::pack2(-1.0f, -1.0f);
#pragma unroll
                for (int cc = 0; cc < kWgCols / 32; ++cc) {
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
                    ptx::tmem_st_32x16(ts + cc * 16, pk);
                    ptx::tmem_st_32x16(ts + 32 + cc * 16, pl);
                }
            } else if constexpr (RELU) {
                // Appendix A.3: p = max(s, 0) in log2 units (the epilogue multiplies by out_scale * ln 2); a masked
                // score (-inf) gives exactly 0.
#pragma unroll
                for (int cc = 0; cc < kWgCols / 32; ++cc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        pk[i] = ptx::pack_bf16x2(fmaxf(__uint_as_float(y[cc * 32 + 2 * i]), 0.f), fmaxf(__uint_as_float(y[cc * 32 + 2 * i + 1]), 0.f));
                    ptx::tmem_st_32x16(ts + cc * 16, pk);
                }
            } else {
                float mt = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                if constexpr (SCORE == kScorePlain) mt *= cs;
                float mt_other;
                if (!exchange(mt, mt_other)) return;
                const float m_new = fmaxf(m_used, fmaxf(mt, mt_other));   // identical in both groups
                if (n == 0) {
                    m_used = m_new;
                } else {
                    // Lazy rescaling: O and l keep a stale maximum until a row's maximum grows by more than
                    // 2^8; the decision is taken per warp because the TMEM accesses are warp collective (the
                    // two groups see the same values and decide alike; each rescales its half of the O columns).
                    const bool need = (m_new - m_used) > kRescaleThreshold;
                    if (__any_sync(0xffffffffu, need)) {
                        if (!bounded_wait(ptx::smem_u32(&bars->pv_done), (g - 1u) & 1u, bars, p.status_word)) return;
                        ptx::tc_fence_after_sync();
                        const float alpha = (m_new == -INFINITY) ? 1.0f : ptx::ex2_approx(m_used - m_new);
                        l *= alpha;
                        l_exact *= alpha;
                        m_used = m_new;
#pragma unroll
                        for (int c = 0; c < kOC / 32; ++c) {
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
                uint64_t sume[2] = {0ull, 0ull};
#pragma unroll
                for (int cc = 0; cc < kWgCols / 32; ++cc) {
                    uint32_t pk[16];
                    exp_chunk<SCORE, kRoundedSum>(&y[cc * 32], cs, neg_m, sum2, pk, sume);
                    ptx::tmem_st_32x16(ts + cc * 16, pk);
                }
                float s0, s1, s2, s3;
                ptx::unpack2(ptx::add2(sum2[0], sum2[1]), s0, s1);
                ptx::unpack2(ptx::add2(sum2[2], sum2[3]), s2, s3);
                l += (s0 + s1) + (s2 + s3);
                if constexpr (kRoundedSum) {
                    ptx::unpack2(ptx::add2(sume[0], sume[1]), s0, s1);
                    l_exact += s0 + s1;
                }
            }
            warp_arrive_after_tmem_st(ptx::smem_u32(&bars->p_full[buf]));
        }

        // Epilogue: O / l (softmax), O * out_scale (sigmoid) or O * out_scale * ln 2 (ReLU: P was kept in log2 units);
        // LSE = ln 2 * (m + log2 l).
        const bool store_row = row < p.Sq;
        float l_row = l;
        if constexpr (!SIGMOID && !RELU) {
            float l_other;
            if (!exchange(l, l_other)) return;
            l_row = l + l_other;
        }
        float l_lse = l_row;                                 // the LSE is the log of the sum of the unrounded weights
        if constexpr (!SIGMOID && !RELU && kRoundedSum) {
            float le_other;
            if (!exchange(l_exact, le_other)) return;
            l_lse = l_exact + le_other;
        }
        if (niter > 0) {
            // pv_done cannot serve here: the MMA thread may lag two key tiles behind, and a parity wait only
            // tells apart "one phase behind" from "caught up".  o_done completes once per item.
            if (!bounded_wait(ptx::smem_u32(&bars->o_done), items_done & 1u, bars, p.status_word)) return;
            ++items_done;
            ptx::tc_fence_after_sync();
        }
        const float inv = SIGMOID ? p.out_scale : (RELU ? p.out_scale * kLn2 : (l_row > 0.f ? 1.0f / l_row : 0.f));
        char* obase = reinterpret_cast<char*>(p.o) +
                      ((long long)it.b * p.os[0] + (long long)it.h * p.os[1] + (long long)row * p.os[2] + wg * kOC) * (p.o_fp32 ? 4 : 2);
#pragma unroll
        for (int c = 0; c < kOC / 32; ++c) {
            uint32_t orr[32];
            if (niter > 0) {
                ptx::tmem_ld_32x32(tm + ocol + c * 32, orr);
                ptx::tmem_wait_ld_regs(orr);
                if (c == kOC / 32 - 1) {
                    // This group's share of O is in registers: once both groups say so, the next item's first
                    // P V may overwrite the accumulator.
                    ptx::tc_fence_before_sync();
                    warp_arrive(ptx::smem_u32(&bars->o_free));
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) orr[i] = 0u;
            }
            if (store_row) {
                if (p.o_fp32) {
                    float4* dst = reinterpret_cast<float4*>(obase + c * 128);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[i] = make_float4(__uint_as_float(orr[4 * i]) * inv, __uint_as_float(orr[4 * i + 1]) * inv,
                                             __uint_as_float(orr[4 * i + 2]) * inv, __uint_as_float(orr[4 * i + 3]) * inv);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>(obase + c * 64);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 w;
                        w.x = ptx::pack_bf16x2(__uint_as_float(orr[8 * i]) * inv, __uint_as_float(orr[8 * i + 1]) * inv);
                        w.y = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 2]) * inv, __uint_as_float(orr[8 * i + 3]) * inv);
                        w.z = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 4]) * inv, __uint_as_float(orr[8 * i + 5]) * inv);
                        w.w = ptx::pack_bf16x2(__uint_as_float(orr[8 * i + 6]) * inv, __uint_as_float(orr[8 * i + 7]) * inv);
                        dst[i] = w;
                    }
                }
            }
        }
        if (!SIGMOID && !RELU && wg == 0 && p.lse && store_row)
            p.lse[((long long)it.b * p.Hq + it.h) * p.Sq + row] = (l_lse > 0.f) ? (m_used + ptx::lg2_approx(l_lse)) * kLn2 : -INFINITY;


        // Next work item: one lane reads the fetched index and shares it with the warp.
        int got = 0;
        if ((threadIdx.x & 31) == 0) got = next_item(bars, item_phase, p.status_word, lin) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        lin = __shfl_sync(0xffffffffu, lin, 0);
        if (!got) return;
    }
}

// ------------------------------------------------------------------------------------------------
// kernel
// ------------------------------------------------------------------------------------------------
template <int D, int SCORE, int NORM>
__global__ void __launch_bounds__(Cfg<D>::kThreads, 1)
attn_fwd_split_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                   const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnParams p) {
    using C = Cfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = ptx::smem_u32(smem);
    // The swizzled tiles need a 1024-byte aligned base (dynamic shared memory starts right after the 1 KB the
    // driver reserves).  If that ever failed to hold, report it instead of computing garbage.
    if ((base & 1023u) != 0u) {
        if (threadIdx.x == 0 && p.status_word) atomicExch(p.status_word, (int)ATTN_ERR_ALIGN);
        return;
    }
    const uint32_t q_smem = base;
    const uint32_t ring_smem = base + C::kQBytes;
    Barriers* bars = reinterpret_cast<Barriers*>(smem + C::kDataBytes);
    float* xchg = reinterpret_cast<float*>(smem + C::kDataBytes + C::kBarBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&bars->q_full), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->q_empty), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->pv_done), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->o_done), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->o_free), C::kSoftmaxWarps);
        for (int t = 0; t < 2; ++t) {
            ptx::mbar_init(ptx::smem_u32(&bars->s_full[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->p_full[t]), C::kSoftmaxWarps);
            ptx::mbar_init(ptx::smem_u32(&bars->xchg[t]), C::kSoftmaxWarps);
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
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

    if (warp < C::kSoftmaxWarps) {
        softmax_role<D, SCORE, NORM>(p, bars, xchg, tmem, warp >> 2);
    } else {
        if (warp == C::kProducerWarp) {
            if (lane == 0) producer_role<D>(&tmap_q, &tmap_k, &tmap_v, p, bars, q_smem, ring_smem);
        } else if (warp == C::kMmaWarp) {
            if (lane == 0) mma_role<D, NORM == kNormSigmoid>(p, bars, tmem, q_smem, ring_smem);
        } else if (warp == C::kSchedWarp) {
            if (lane == 0) scheduler_role(bars, p.status_word);
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
template <int D, int SCORE, int NORM>
int launch_instance(AttnParams p, cudaStream_t stream) {
    using C = Cfg<D>;
    auto kernel = attn_fwd_split_kernel<D, SCORE, NORM>;
    // The opt-in shared-memory size is a per-device function attribute: set it once per device.
    static SmemAttrFlags attr_set;
    if (!set_smem_attr_once(attr_set, kernel, C::kSmemBytes)) return ATTN_ERR_CUDA;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, p.q, p.B, p.Hq, p.Sq, D, p.qs, 128) || !make_map(&mk, p.k, p.B, p.Hkv, p.Sk, D, p.ks, 128) ||
        !make_map(&mv, p.v, p.B, p.Hkv, p.Sk, D, p.vs, D == 256 ? 64 : 128))
        return ATTN_ERR_CUDA;
    // Heads per section of the work order: as many KV heads as keep the section's K and V within
    // about 40 MB of L2, in equal sections, whole GQA groups.
    const long long kv_bytes = 2ll * p.Sk * D * 2;
    long long kv_heads = (40ll << 20) / kv_bytes;
    if (kv_heads < 1) kv_heads = 1;
    const long long bh = (long long)p.B * p.Hq;
    long long sec_max = kv_heads * p.group;
    if (sec_max > bh) sec_max = bh;
    const long long n_sec = (bh + sec_max - 1) / sec_max;
    long long sec = (bh + n_sec - 1) / n_sec;
    sec = (sec + p.group - 1) / p.group * p.group;
    p.sec_heads = (int)sec;
    const long long nqb = (p.Sq + kBM - 1) / kBM;
    const long long grid = nqb * bh;
    if (grid > 0x7fffffffLL) return ATTN_ERR_SHAPE;
    // (global tokens only: their rows are the first blocks; this kernel's order already starts a section with the last blocks)
    p.front_blocks = (p.mask_flags & kMaskGlobal) ? leading_blocks(p, kBM, kBN, (int)nqb, sec, bh, device_sm_count()) : 0;
    kernel<<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(mq, mk, mv, p);
    return cudaGetLastError() == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

template <int D>
int launch_for_d(const AttnParams& p, cudaStream_t stream) {
    if (p.normalizer == kNormSigmoid) return launch_instance<D, kScoreGeneric, kNormSigmoid>(p, stream);
    if (p.normalizer == kNormRelu) return launch_instance<D, kScoreGeneric, kNormRelu>(p, stream);
    if (p.softcap > 0.f) return launch_instance<D, kScoreGeneric, kNormSoftmax>(p, stream);
    if (p.slopes) return launch_instance<D, kScoreBias, kNormSoftmax>(p, stream);
    return launch_instance<D, kScorePlain, kNormSoftmax>(p, stream);
}

}  // namespace

// One query tile per work item, S double buffered, two column-split softmax groups: the kernel for D = 256
// (its accumulator leaves no TMEM room for a second query tile).  It is also correct for D = 64 and 128, where
// the two-tile kernel of attn_tc_pingpong.cuh is faster because it reads K and V from L2 half as often.
int launch_attn_fwd_bf16_split(const AttnParams& p, cudaStream_t stream) {
    switch (p.D) {
        case 64: return launch_for_d<64>(p, stream);
        case 128: return launch_for_d<128>(p, stream);
        case 256: return launch_for_d<256>(p, stream);
        default: return ATTN_ERR_UNSUPPORTED;
    }
}

}  // namespace b200attn
