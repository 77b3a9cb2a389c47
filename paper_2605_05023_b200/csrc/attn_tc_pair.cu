// bf16 attention forward on tcgen05 with CTA pairs (cta_group::2): two SMs share every K / V tile.
//
// A work item is two adjacent query tiles of 128 rows of one (batch, query head), one per CTA of a
// cluster of two.  Each CTA loads only half of every key tile (64 of the 128 keys of K, half of the
// head-dimension columns of V); the pair's leader CTA (rank 0) issues tcgen05.mma.cta_group::2
// instructions with M = 256 that read the A operand (Q from shared memory, P from TMEM) of both CTAs
// and the two halves of the B operand from both CTAs' shared memory, and leave each CTA's 128 rows of
// S and O in that CTA's own TMEM.  Against one tile per CTA this halves the K / V traffic from L2 to
// shared memory, which is what bounds the one-tile kernel (D = 256 above all).
//
// Per CTA the roles are those of the one-tile kernel (attn_tc_split.cu): a producer warp (TMA), two
// softmax groups that split the 128 key columns of every S tile, a scheduler warp (cluster launch
// control, leader only, which forwards each fetched item to its peer), and on the leader the MMA thread.
// S is double buffered at D = 256 and triple buffered at D = 128 (Q K^T runs that many key tiles ahead of the
// softmax groups).  TMEM columns per CTA: S buffers of 128 columns each, then O (D columns).
// The key loop of a pair covers the key tiles either of its two query tiles can see; a tile outside one
// CTA's own interval is masked element-wise there (its P is exactly zero).
//
// Cross-CTA signalling: TMA loads of both CTAs count their bytes on the leader's `full` / `q_full`
// barriers; tcgen05.commit arrives on the same barrier of both CTAs; the softmax warps of both CTAs
// arrive on the leader's `p_full` / `o_free` barriers through the shared::cluster window.
// Sigmoid normaliser (Appendix A.3): the weights are not normalised per row, so the 8 significant bits of a bf16
// P show in O; P is written as fp16 (11 bits, scaled by 2^10 away from fp16's subnormals) and, because
// tcgen05.mma wants A and B of one type, every V tile is converted from bf16 to fp16 in shared memory, in place,
// by a fourth warpgroup of each CTA once its TMA load has landed (exact for |v| < 65536; anything larger is
// reported as ATTN_ERR_UNSUPPORTED in the status word).  P V is then one pass over fp16 operands.
// Every mbarrier wait is bounded (see bounded_wait); the only unbounded waits are the cluster barriers at
// start and exit, which every thread of both CTAs reaches.
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
constexpr int kMaxStages = 12;


template <int D>
struct Cfg {
    static constexpr int kBoxBytes = 64 * 128 * 2;                      // TMA box of 128 rows x 64 columns
    static constexpr int kSlotBytes = kBM * D;                          // half a K tile = half a V tile, in bytes
    static constexpr int kStages = (D == 128) ? 12 : 5;
    static constexpr int kQBytes = kBM * D * 2;
    static constexpr int kDataBytes = kQBytes + kStages * kSlotBytes;
    static constexpr int kBarBytes = 1024;
    static constexpr int kXchgBytes = 2 * 2 * kBM * 4;                  // row maxima / sums: [parity][group][row]
    static constexpr int kSmemBytes = kDataBytes + kBarBytes + kXchgBytes;
    static constexpr int kThreads = 384;
    static constexpr int kSoftmaxWarps = 8;
    static constexpr int kProducerWarp = 8;
    static constexpr int kMmaWarp = 9;
    static constexpr int kSchedWarp = 10;
    static constexpr int kSpareWarp = 11;
    static constexpr int kConverterWarp = 12;                           // sigmoid instances: a fourth warpgroup turns V into fp16
    static constexpr int kThreadsSigmoid = 512;
    static constexpr int kRegsSoftmax = 168, kRegsOther = 80, kRegsConverter = 80;   // sigmoid instances (setmaxnreg)
    static_assert(2 * 128 * kRegsSoftmax + 128 * kRegsOther + 128 * kRegsConverter <= 512 * 128, "register budget");
    static constexpr int kItemConsumers = kSoftmaxWarps + 3;            // local warps that read each fetched item
    static constexpr int kTmemCols = 512;
    static constexpr int kSBufs = (D == 128) ? 3 : 2;                   // S buffers: as many as fit beside O in TMEM
    static constexpr int kTmemO = kSBufs * kBN;                         // first O column
    static_assert(kTmemO + D <= kTmemCols, "TMEM budget");
    static_assert(D == 128 || D == 256, "head dimension");
    static_assert(kStages <= kMaxStages, "barrier arrays");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

// Same layout in both CTAs.  L: only the leader's copy is waited on.  B: each CTA waits on its own copy.
struct Barriers {
    uint64_t q_full;             // L  both Q tiles landed (TMA of both CTAs)
    uint64_t q_empty;            // B  last QK^T of the item done: the Q tile may be overwritten
    uint64_t full[kMaxStages];   // L  both halves of a ring slot landed (V of a sigmoid instance: and converted)
    uint64_t empty[kMaxStages];  // B  ring slot consumed (tcgen05.commit to both CTAs)
    uint64_t s_full[3];          // B  S buffer written by QK^T
    uint64_t p_full[3];          // L  all of P written in both CTAs (16 warp arrivals)
    uint64_t pv_done[3];         // B  P V of the key tile held in that S buffer done
    uint64_t o_done;             // B  last P V of the item done: O is complete
    uint64_t o_free;             // L  both epilogues have read O (16 warp arrivals)
    uint64_t xchg[2];            // B  both softmax groups of this CTA have posted their row values
    uint64_t clc;                // L  response of the hardware scheduler landed
    uint64_t item_full;          // B  next work item published by the leader's scheduler thread
    uint64_t item_empty;         // B  every local role has read the published item
    uint64_t item_ready;         // L  both CTAs are ready for the next item (2 arrivals)
    alignas(16) uint64_t clc_response[2];    // L  16 bytes written by the hardware scheduler (16-byte aligned)
    uint32_t item_value[2];      // B  {got, linear CTA index of the pair's first CTA}
    uint32_t tmem_base;
    int abort_flag;
    uint64_t landed[kMaxStages]; // B  sigmoid instances: this CTA's half of a V tile landed (TMA), ready to be converted
    uint64_t converted;          // B  sigmoid instances: the four converter warps are done with a V slot (4 arrivals)
};
static_assert(sizeof(Barriers) <= 1024, "barrier block");

struct TileRange {
    int jlo, jhi;      // key tiles [jlo, jhi)
};

struct Item {
    int q0, h, b, g;   // first query row of the pair, query head, batch, kv head
    TileRange tr;      // key tiles that any row of the pair can see
};

// Key tiles that the rows [q0, q0 + 256) can see.
__device__ __forceinline__ TileRange pair_range(const AttnParams& p, int q0) {
    const TileBounds t = tile_bounds(p, q0, 2 * kBM);
    if (!t.any) return TileRange{0, 0};
    return TileRange{t.lo_min / kBN, t.hi_max / kBN + 1};
}

// Work item of a pair index (work_order in attn_params.cuh: sections of heads whose K/V fit in L2, last query block
// first, the first blocks of every head at the very end).
__device__ __forceinline__ Item decode_item(const AttnParams& p, int pair) {
    const int nqb = (p.Sq + 2 * kBM - 1) / (2 * kBM);
    const int bh_total = p.B * p.Hq;
    int rank, bh;
    work_order(pair, bh_total, p.sec_heads, nqb, p.defer_blocks, rank, bh);
    const int qb = nqb - 1 - rank;
    Item it;
    it.b = bh / p.Hq;
    it.h = bh - it.b * p.Hq;
    it.g = it.h / p.group;
    it.q0 = qb * 2 * kBM;
    it.tr = pair_range(p, it.q0);
    return it;
}

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* status_word) {
    return bounded_wait_on<false>(bar, parity, &bars->abort_flag, status_word);
}
// For barriers that the other CTA of the pair arrives on.
__device__ __forceinline__ bool bounded_wait_cluster(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* status_word) {
    return bounded_wait_on<true>(bar, parity, &bars->abort_flag, status_word);
}

// Waits for the next work item published by the leader's scheduler thread and releases the slot.
// Returns false when the grid has no unstarted cluster left (or the wait was abandoned).
__device__ __forceinline__ bool next_item(Barriers* bars, uint32_t& phase, int32_t* status_word, int& pair) {
    if (!bounded_wait_cluster(ptx::smem_u32(&bars->item_full), phase, bars, status_word)) return false;
    phase ^= 1u;
    const uint32_t got = *reinterpret_cast<volatile uint32_t*>(&bars->item_value[0]);
    const uint32_t lin = *reinterpret_cast<volatile uint32_t*>(&bars->item_value[1]);
    ptx::mbar_arrive(ptx::smem_u32(&bars->item_empty));
    pair = (int)(lin >> 1);
    return got != 0u;
}

// ------------------------------------------------------------------------------------------------
// scheduler: one thread per CTA; the leader's asks the hardware for the next cluster and publishes it
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void scheduler_role(Barriers* bars, int32_t* status_word, uint32_t rank) {
    uint32_t item_phase = 0, empty_phase = 1, ready_phase = 0, clc_phase = 0;   // first wait on item_empty passes at once
    const uint32_t ready_on_leader = ptx::mapa(ptx::smem_u32(&bars->item_ready), 0);
    while (true) {
        // Every local role has read the previous item: this CTA is ready for the next one.
        if (!bounded_wait(ptx::smem_u32(&bars->item_empty), empty_phase, bars, status_word)) return;
        empty_phase ^= 1u;
        ptx::mbar_arrive_cluster(ready_on_leader);
        if (rank == 0) {
            if (!bounded_wait_cluster(ptx::smem_u32(&bars->item_ready), ready_phase, bars, status_word)) return;
            ready_phase ^= 1u;
            bool handed;
            uint32_t x;
            if (!clc_fetch(ptx::smem_u32(&bars->clc), bars->clc_response, clc_phase, &bars->abort_flag, status_word, handed, x)) return;
            const uint32_t got = handed ? 1u : 0u;
            // Publish {got, index} in both CTAs, then signal each CTA's item_full.
#pragma unroll
            for (uint32_t r = 0; r < 2; ++r) {
                ptx::st_cluster_u32(ptx::mapa(ptx::smem_u32(&bars->item_value[0]), r), got);
                ptx::st_cluster_u32(ptx::mapa(ptx::smem_u32(&bars->item_value[1]), r), x);
                ptx::mbar_arrive_cluster(ptx::mapa(ptx::smem_u32(&bars->item_full), r));
            }
        }
        int pair;
        if (!next_item(bars, item_phase, status_word, pair)) return;   // no item left: stop
    }
}

// ------------------------------------------------------------------------------------------------
// producer: TMA (this CTA's Q tile, its 64 keys of every K tile, its half of the columns of every V tile)
// ------------------------------------------------------------------------------------------------
template <int D, bool V_F16>
__device__ __forceinline__ void producer_role(const CUtensorMap* tmap_q, const CUtensorMap* tmap_k,
                                              const CUtensorMap* tmap_v, const AttnParams& p, Barriers* bars,
                                              uint32_t q_smem, uint32_t ring_smem, uint32_t rank) {
    using C = Cfg<D>;
    ptx::prefetch_tensormap(tmap_q);
    ptx::prefetch_tensormap(tmap_k);
    ptx::prefetch_tensormap(tmap_v);
    int ps = 0;
    uint32_t pph = 0, item_phase = 0;
    int q_uses = 0;                                 // items whose Q was loaded so far
    int pair = (int)(blockIdx.x >> 1);

    // Waits for the slot to be free in this CTA; the leader arms its `full` barrier for the bytes of both CTAs.
    // V of a sigmoid instance (V_F16): the bytes are counted on this CTA's own `landed` barrier instead; the
    // converter warps of both CTAs complete the leader's `full` barrier (two arrivals, so a K slot adds one).
    auto open_slot = [&](uint32_t& dst, uint32_t& bar, bool is_v) -> bool {
        if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return false;
        dst = ring_smem + ps * C::kSlotBytes;
        if (V_F16 && is_v) {
            bar = ptx::smem_u32(&bars->landed[ps]);
            ptx::mbar_arrive_expect_tx(bar, C::kSlotBytes);
        } else {
            bar = ptx::smem_u32(&bars->full[ps]);
            if (rank == 0) {
                ptx::mbar_arrive_expect_tx(bar, 2 * C::kSlotBytes);
                if (V_F16) ptx::mbar_arrive(bar);
            }
        }
        if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        return true;
    };
    // Keys [128 j + 64 rank, + 64) of K, all D columns: D/64 boxes of [64 keys x 64 columns].
    auto produce_k = [&](const Item& it, int j) -> bool {
        uint32_t dst, bar;
        if (!open_slot(dst, bar, false)) return false;
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            ptx::tma_load_4d_pair(dst + bx * (C::kBoxBytes / 2), tmap_k, bar, bx * 64, j * kBN + (int)rank * 64, it.g, it.b);
        return true;
    };
    // All 128 keys of V, columns [rank D/2, + D/2): D/128 boxes of [128 keys x 64 columns].
    auto produce_v = [&](const Item& it, int j) -> bool {
        uint32_t dst, bar;
        if (!open_slot(dst, bar, true)) return false;
#pragma unroll
        for (int bx = 0; bx < D / 128; ++bx) {
            if constexpr (V_F16) ptx::tma_load_4d(dst + bx * C::kBoxBytes, tmap_v, bar, (int)rank * (D / 2) + bx * 64, j * kBN, it.g, it.b);
            else ptx::tma_load_4d_pair(dst + bx * C::kBoxBytes, tmap_v, bar, (int)rank * (D / 2) + bx * 64, j * kBN, it.g, it.b);
        }
        return true;
    };

    while (true) {
        const Item it = decode_item(p, pair);
        const int J0 = it.tr.jlo, J1 = it.tr.jhi;
        if (J0 < J1) {
            // The previous item's last QK^T must have finished reading the Q buffer.
            if (q_uses > 0 && !bounded_wait(ptx::smem_u32(&bars->q_empty), (uint32_t)((q_uses - 1) & 1), bars, p.status_word))
                return;
            ++q_uses;
            const uint32_t bar = ptx::smem_u32(&bars->q_full);
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar, 2 * C::kQBytes);
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx)
                ptx::tma_load_4d_pair(q_smem + bx * C::kBoxBytes, tmap_q, bar, bx * 64, it.q0 + (int)rank * kBM, it.h, it.b);
            // Slot order = the order in which the MMA thread consumes: Q K^T runs kSBufs - 1 key tiles ahead of P V.
#pragma unroll
            for (int t = 0; t < C::kSBufs - 1; ++t)
                if (J0 + t < J1 && !produce_k(it, J0 + t)) return;
            for (int j = J0; j < J1; ++j) {
                if (j + C::kSBufs - 1 < J1 && !produce_k(it, j + C::kSBufs - 1)) return;
                if (!produce_v(it, j)) return;
            }
        }
        if (!next_item(bars, item_phase, p.status_word, pair)) return;
    }
}

// ------------------------------------------------------------------------------------------------
// converter (sigmoid instances): a warpgroup per CTA turns each landed V tile from bf16 into fp16, in place
// ------------------------------------------------------------------------------------------------
// It walks the ring in the producer's order and acts on the V slots only.  bf16 -> fp16 is exact for normal
// values below 65536 in magnitude (8 significant bits fit in 11); smaller than 2^-14 they lose bits that no
// output can show (absolute error below 2^-25 per product).  A value of 65536 or more (or a non-finite one)
// cannot be represented: the group reports ATTN_ERR_UNSUPPORTED in the status word.
template <int D>
__device__ __forceinline__ void converter_role(const AttnParams& p, Barriers* bars, uint8_t* ring_ptr) {
    using C = Cfg<D>;
    const int lane = threadIdx.x & 31;
    const int cthread = threadIdx.x & 127;          // thread within the converter warpgroup
    int ps = 0;
    uint32_t landed_phase = 0;                      // bit s: parity of the next completion of landed[s]
    uint32_t item_phase = 0;
    int pair = (int)(blockIdx.x >> 1);
    uint32_t too_large = 0;
    uint32_t slots_done = 0;
    const uint32_t full_on_leader = ptx::mapa(ptx::smem_u32(&bars->full[0]), 0);

    auto skip_slot = [&]() { if (++ps == C::kStages) ps = 0; };
    // All 32 lanes of a warp take every decision together (the waits are made by lane 0 and shared), so that a run
    // that is being abandoned leaves the warp-collective operations below with all their lanes.
    auto warp_wait = [&](uint32_t bar, uint32_t parity) -> bool {
        int ok = 1;
        if (lane == 0) ok = bounded_wait(bar, parity, bars, p.status_word) ? 1 : 0;
        return __shfl_sync(0xffffffffu, ok, 0) != 0;
    };
    auto convert_slot = [&]() -> bool {
        if (!warp_wait(ptx::smem_u32(&bars->landed[ps]), (landed_phase >> ps) & 1u)) return false;
        landed_phase ^= 1u << ps;
        uint4* slot = reinterpret_cast<uint4*>(ring_ptr + ps * C::kSlotBytes);
#pragma unroll 4
        for (int i = cthread; i < C::kSlotBytes / 16; i += 128) {
            uint4 w = slot[i];
            uint32_t* x = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                too_large = __vmaxu2(too_large, x[e] & 0x7fff7fffu);       // largest |bf16| bit pattern seen
                x[e] = ptx::pack_f16x2(__uint_as_float(x[e] << 16), __uint_as_float(x[e] & 0xffff0000u));
            }
            slot[i] = w;
        }
        ptx::fence_proxy_async_smem();              // these generic writes come before the MMA's reads of the slot
        // The four warps meet on a (bounded) mbarrier: none goes on to the next slot, and the first one does not
        // tell the leader's MMA thread, before all four are done with this one.
        warp_arrive(ptx::smem_u32(&bars->converted));
        if (!warp_wait(ptx::smem_u32(&bars->converted), slots_done & 1u)) return false;
        if (cthread == 0) ptx::mbar_arrive_cluster(full_on_leader + ps * 8);
        ++slots_done;
        skip_slot();
        return true;
    };

    bool ok = true;
    while (ok) {
        const Item it = decode_item(p, pair);
        const int J0 = it.tr.jlo, J1 = it.tr.jhi;
        if (J0 < J1) {
#pragma unroll
            for (int t = 0; t < C::kSBufs - 1; ++t)
                if (J0 + t < J1) skip_slot();                                   // K
            for (int j = J0; j < J1 && ok; ++j) {
                if (j + C::kSBufs - 1 < J1) skip_slot();                        // K
                ok = convert_slot();                                            // V
            }
        }
        if (!ok) break;
        int got = 0;
        if (lane == 0) got = next_item(bars, item_phase, p.status_word, pair) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        pair = __shfl_sync(0xffffffffu, pair, 0);
        if (!got) break;
    }
    // 0x4780 is bf16 65536: that and everything above (infinities and NaNs included) has no fp16 counterpart
    const bool bad = ((too_large & 0xffffu) >= 0x4780u) || ((too_large >> 16) >= 0x4780u);
    if (__any_sync(0xffffffffu, bad) && lane == 0 && p.status_word) atomicCAS(p.status_word, 0, (int)ATTN_ERR_UNSUPPORTED);
}

// ------------------------------------------------------------------------------------------------
// MMA issuer (one thread of the leader CTA)
// ------------------------------------------------------------------------------------------------
template <int D, bool V_F16>
__device__ __forceinline__ void mma_role(const AttnParams& p, Barriers* bars, uint32_t tmem, uint32_t q_smem,
                                         uint32_t ring_smem) {
    using C = Cfg<D>;
    constexpr uint32_t kIdescQK = instr_desc(2 * kBM, kBN, false);
    constexpr uint32_t kIdescPV = instr_desc(2 * kBM, D, true, V_F16);    // sigmoid instances: P and V are fp16
    // Descriptor halves (128-byte swizzle, SBO = 1024 B, sm_100 version bit): hi is constant per operand kind,
    // lo = (address >> 4) | (LBO >> 4) << 16 advances by compile-time constants inside a tile.
    constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kLoKMajor = 1u << 16;                                     // LBO unused for K-major
    constexpr uint32_t kLoV = (uint32_t)(C::kBoxBytes >> 4) << 16;               // LBO between 64-column blocks of V
    const uint32_t q_lo = ((q_smem & 0x3FFFFu) >> 4) | kLoKMajor;
    const uint32_t ring_lo = (ring_smem & 0x3FFFFu) >> 4;
    const uint32_t bar_s_full = ptx::smem_u32(&bars->s_full[0]);
    const uint32_t bar_pv_done = ptx::smem_u32(&bars->pv_done[0]);
    const uint32_t bar_p_full = ptx::smem_u32(&bars->p_full[0]);
    const uint32_t bar_full = ptx::smem_u32(&bars->full[0]);
    const uint32_t bar_empty = ptx::smem_u32(&bars->empty[0]);
    const uint32_t bar_q_empty = ptx::smem_u32(&bars->q_empty);

    constexpr int NS = C::kSBufs;
    int cs = 0;
    uint32_t cph = 0, item_phase = 0;
    int q_uses = 0;                                 // items with at least one key tile so far
    uint32_t g = 0;                                 // key tiles whose P V was issued so far
    int pair = (int)(blockIdx.x >> 1);

    auto next_slot = [&](int& slot) -> bool {
        // (V_F16: the peer's converter warp arrives on this barrier after writing its shared memory)
        if (!(V_F16 ? bounded_wait_cluster(bar_full + cs * 8, cph, bars, p.status_word)
                    : bounded_wait(bar_full + cs * 8, cph, bars, p.status_word)))
            return false;
        slot = cs;
        if (++cs == C::kStages) { cs = 0; cph ^= 1u; }
        return true;
    };
    // S[buf] (both CTAs) = Q K^T over the whole head dimension; signals s_full[buf] in both CTAs.
    // B operand: this CTA's 64 keys, D/64 boxes of [64 keys x 128 B]; the peer's half sits at the same offsets.
    auto issue_qk = [&](int buf, int kslot) {
        const uint32_t b_lo = (ring_lo + (uint32_t)kslot * (C::kSlotBytes >> 4)) | kLoKMajor;
        const uint32_t d = tmem + buf * kBN;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t a_off = (uint32_t)(((kk / 4) * C::kBoxBytes + (kk % 4) * 32) >> 4);
            const uint32_t b_off = (uint32_t)(((kk / 4) * (C::kBoxBytes / 2) + (kk % 4) * 32) >> 4);
            ptx::mma_ss_pair(d, q_lo + a_off, kDescHi, b_lo + b_off, kDescHi, kIdescQK, kk > 0 ? 1u : 0u);
        }
        ptx::tc_commit_pair(bar_s_full + buf * 8);
    };
    // O (+)= P[buf] V over the 128 keys of the tile.  Softmax group w wrote the 16-bit P of keys [64 w, 64 w + 64)
    // over its own S columns, starting at column 64 w.
    // B operand: this CTA's D/2 columns of V for all 128 keys, D/128 boxes of [128 keys x 128 B].
    auto issue_pv = [&](int buf, int vslot, bool accumulate, uint32_t col_off) {
        const uint32_t b_lo = (ring_lo + (uint32_t)vslot * (C::kSlotBytes >> 4)) | kLoV;
        const uint32_t d = tmem + C::kTmemO, a = tmem + buf * kBN + col_off;
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk)
            ptx::mma_ts_pair(d, a + (kk / 4) * kWgCols + (kk % 4) * 8, b_lo + (uint32_t)((kk * 2048) >> 4), kDescHi, kIdescPV,
                             (accumulate || kk > 0) ? 1u : 0u);
    };
    // Q K^T of key tile j into the S buffer of global tile index gt; releases the K slot (and Q after the last one).
    auto qk_step = [&](int j, uint32_t gt, int J1) -> bool {
        int kslot;
        if (!next_slot(kslot)) return false;
        ptx::tc_fence_after_sync();
        issue_qk((int)(gt % NS), kslot);
        if (j == J1 - 1) ptx::tc_commit_pair(bar_q_empty);
        ptx::tc_commit_pair(bar_empty + kslot * 8);
        return true;
    };

    while (true) {
        const Item it = decode_item(p, pair);
        const int J0 = it.tr.jlo, J1 = it.tr.jhi;
        if (J0 < J1) {
            if (!bounded_wait(ptx::smem_u32(&bars->q_full), (uint32_t)(q_uses & 1), bars, p.status_word)) return;
            // Q K^T runs NS - 1 key tiles ahead of P V: tile j + NS - 1 lands in the buffer that tile j - 1 has left.
#pragma unroll
            for (int t = 0; t < NS - 1; ++t)
                if (J0 + t < J1 && !qk_step(J0 + t, g + t, J1)) return;
            for (int j = J0; j < J1; ++j, ++g) {
                const int buf = (int)(g % NS);
                const uint32_t ph = (g / NS) & 1u;
                if (j + NS - 1 < J1 && !qk_step(j + NS - 1, g + NS - 1, J1)) return;
                int vslot;
                if (!next_slot(vslot)) return;
                // Before the first P V of an item overwrites O: both epilogues of the previous item must have read it.
                if (j == J0 && q_uses > 0) {
                    if (!bounded_wait(ptx::smem_u32(&bars->o_free), (uint32_t)((q_uses - 1) & 1), bars, p.status_word)) return;
                }
                if (!bounded_wait(bar_p_full + buf * 8, ph, bars, p.status_word)) return;
                ptx::tc_fence_after_sync();
                issue_pv(buf, vslot, j > J0, 0u);
                ptx::tc_commit_pair(bar_pv_done + buf * 8);
                if (j == J1 - 1) ptx::tc_commit_pair(ptx::smem_u32(&bars->o_done));
                ptx::tc_commit_pair(bar_empty + vslot * 8);
            }
            ++q_uses;
        }
        if (!next_item(bars, item_phase, p.status_word, pair)) return;
    }
}

// ------------------------------------------------------------------------------------------------
// softmax / sigmoid groups and epilogue: thread i of group w owns row i, key columns [64 w, 64 w + 64)
// ------------------------------------------------------------------------------------------------

// The same on a barrier of the pair's leader CTA (address in the shared::cluster window).  What the arrival
// publishes lives in TMEM and is ordered by the tcgen05 fences around it.
__device__ __forceinline__ void warp_arrive_on_leader(uint32_t cluster_addr) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) ptx::mbar_arrive_cluster_relaxed(cluster_addr);
}

template <int D, int SCORE, int NORM>
__device__ __forceinline__ void softmax_role(const AttnParams& p, Barriers* bars, float* xchg, uint32_t tmem, int wg,
                                             uint32_t rank) {
    using C = Cfg<D>;
    constexpr bool SIGMOID = (NORM == kNormSigmoid);   // out_scale * sigmoid(s + b), P and V as fp16
    constexpr bool RELU = (NORM == kNormRelu);         // out_scale * max(s, 0), no exponential at all
    constexpr int kOC = D / 2;                                // O columns handled by each group
    const int wg_thread = threadIdx.x & 127;                 // row within the tile
    const uint32_t lane_base = (uint32_t)((threadIdx.x >> 5) & 3) * 32u;   // TMEM lanes this warp may touch
    const uint32_t tm = tmem + (lane_base << 16);
    const int col0 = wg * kWgCols;                            // first S column of this group
    const uint32_t ocol = C::kTmemO + wg * kOC;
    const uint32_t p_full_on_leader = ptx::mapa(ptx::smem_u32(&bars->p_full[0]), 0);
    const uint32_t o_free_on_leader = ptx::mapa(ptx::smem_u32(&bars->o_free), 0);

    const float cs = p.scale * kLog2e;                       // raw score -> log2 units
    const float sig_bias2 = p.sigmoid_bias * kLog2e;

    uint32_t g = 0;                                          // key tiles processed so far
    uint32_t xg = 0;                                         // exchange steps so far
    uint32_t items_done = 0;                                 // items with at least one key tile finished so far
    uint32_t item_phase = 0;
    int pair = (int)(blockIdx.x >> 1);

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
        const Item it = decode_item(p, pair);
        const int q0 = it.q0 + (int)rank * kBM;              // this CTA's tile
        const TileRange tr = it.tr;
        const int row = q0 + wg_thread;
        const int row_c = min(row, p.Sq - 1);                // rows past Sq compute on a valid interval, never stored
        const RowInterval riv = row_interval(p, row_c);
        const TileBounds tb = tile_bounds(p, min(q0, p.Sq - 1), kBM);
        const int lo_last = tb.lo_max, hi_first = tb.hi_min;   // keys in [lo_last, hi_first] are visible to every row
        const int ip = row_c + p.Sk - p.Sq;
        ScoreConsts sc = {};
        if constexpr (SCORE != kScorePlain) sc = make_score_consts(p.scale, p.softcap, p.slopes ? __ldg(p.slopes + it.h) : 0.f);
        const int niter = tr.jhi - tr.jlo;
        float m_used = -INFINITY, l = 0.f;                   // l: this group's share of the row sum
        // A softcap without a position bias bounds every score by C: a fixed reference 32 octaves below that bound
        // keeps every exponential inside [2^-104, 2^40] whatever the row holds, so the running maximum, its exchange
        // between the two groups and the rescaling of O are not needed at all.
        const bool fixed_max = (SCORE == kScoreGeneric) && p.softcap > 0.f && p.slopes == nullptr && p.softcap * kLog2e < 72.5f;
        if (fixed_max) m_used = p.softcap * kLog2e - 32.0f;
        // D = 256, and always with the fixed reference: the row sum that normalises O is taken over the bf16-rounded
        // weights that P V uses, so that O is an exactly normalised average of V rows (the rounding of a dominant
        // weight would otherwise show in O); the LSE uses a second sum over the unrounded weights.
        const bool rounded_sum = fixed_max || D == 256;
        float l_exact = 0.f;                                 // rounded_sum only: sum of the unrounded weights

        for (int n = 0; n < niter; ++n, ++g) {
            const int kv0 = (tr.jlo + n) * kBN;
            const int buf = (int)(g % C::kSBufs);
            const uint32_t ph = (g / C::kSBufs) & 1u;
            // Mask (Appendix A.2): element-wise tests only on tiles that straddle an interval edge of this CTA's
            // rows (or lie outside their intervals: the pair's key loop covers both tiles).
            const bool full_tile = (kv0 >= lo_last) && (kv0 + kBN - 1 <= hi_first);
            const int mask_a = riv.lo - kv0 - col0, mask_e = riv.hi - kv0 - col0;   // visible columns of this group
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
            // Score (Appendix A.1).  Softcap in the softmax instances: the polynomial tanh on all columns and one range
            // check per tile; if a score of this warp's columns lies beyond the polynomial's range (rare), the raw
            // scores are read again and capped through the exponential form.
            // (These instances are launched with a softcap only.)
            constexpr bool kTileCap = (SCORE == kScoreGeneric) && !SIGMOID && !RELU;
            if constexpr (kTileCap) {
                float zmax = 0.f;
#pragma unroll
                for (int c = 0; c < kWgCols / 32; ++c) softcap_lin_chunk32(&y[c * 32], sc, zmax);
                if (__any_sync(0xffffffffu, zmax > sc.zl_limit)) {
                    // beyond the first polynomial's range: the cubic (up to half the cap) or the exponential form, on the raw scores
                    const bool exact = __any_sync(0xffffffffu, zmax > sc.z_limit);
                    ptx::tmem_ld_32x32(ts, *reinterpret_cast<uint32_t(*)[32]>(&y[0]));
                    ptx::tmem_ld_32x32(ts + 32, *reinterpret_cast<uint32_t(*)[32]>(&y[32]));
                    ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[0]));
                    ptx::tmem_wait_ld_regs(*reinterpret_cast<uint32_t(*)[32]>(&y[32]));
                    if (exact) {
#pragma unroll
                        for (int c = 0; c < kWgCols / 32; ++c) softcap_exact_chunk32(&y[c * 32], sc);
                    } else {
                        float zdummy = 0.f;
#pragma unroll
                        for (int c = 0; c < kWgCols / 32; ++c) softcap_poly_chunk32(&y[c * 32], sc, zdummy);
                    }
                }
                if (sc.has_bias) {
#pragma unroll
                    for (int c = 0; c < kWgCols / 32; ++c) bias_add_chunk32(&y[c * 32], sc, rowoff - (float)(c * 32));
                }
            }
#pragma unroll
            for (int c = 0; c < kWgCols / 32; ++c) {
                if constexpr (SCORE != kScorePlain && !kTileCap) {
                    // (Sigmoid without softcap or bias: the scale rides in the sigmoid's own first FMA, below.  ReLU of a
                    // plainly scaled score: max(scale * s, 0) = scale * max(s, 0) for scale > 0, so the raw scores go
                    // on and the scale joins the epilogue's factor.)
                    if (!((SIGMOID || (RELU && p.scale > 0.f)) && !sc.softcap && !sc.has_bias))
                        score_chunk32<SCORE == kScoreGeneric>(&y[c * 32], sc, rowoff - (float)(c * 32));
                }
                if (!full_tile) mask_chunk32_cmp(&y[c * 32], mask_a - c * 32, mask_e - c * 32);   // (the bit-test form cost this kernel 2 %)
                if (!SIGMOID && !RELU && !fixed_max) {
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
                // be carried by a few large weights, so the 8 significant bits of a bf16 P would show in O: P is
                // written as fp16, scaled by 2^10 (2^10 * sigmoid(x) = 1 / (2^-10 + 2^(-x log2 e - 10)): the scale
                // rides in the constants; the epilogue takes it out again together with out_scale).
                const float neg_mul = (!sc.softcap && !sc.has_bias) ? -sc.cs : -1.0f;      // raw scores in, or scores in log2 units
                const uint64_t nb2 = ptx::pack2(-sig_bias2 - 10.0f, -sig_bias2 - 10.0f), neg1 = ptx::pack2(neg_mul, neg_mul);
                constexpr float kTwoToMinus10 = 0.0009765625f;
                // Two special-function operations per score (ex2, rcp) make that unit the busiest at D = 128, where a key
                // step has half the tensor work of D = 256: there every other pair of scores takes its reciprocal on
                // the FMA pipe instead (sweep sigmoid rows +7 to 11 % at S <= 4k; at D = 256 the same costs c4b 2 %).
                constexpr int kNewtonEvery = (D == 128) ? 2 : 0;
#pragma unroll
                for (int cc = 0; cc < kWgCols / 32; ++cc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint64_t yy = ptx::pack2(__uint_as_float(y[cc * 32 + 2 * i]), __uint_as_float(y[cc * 32 + 2 * i + 1]));
                        float z0, z1;
                        ptx::unpack2(ptx::fma2(yy, neg1, nb2), z0, z1);                  // -(s + b) in log2 units, - 10
                        const float t0 = kTwoToMinus10 + ptx::ex2_approx(z0), t1 = kTwoToMinus10 + ptx::ex2_approx(z1);
                        float p0, p1;
                        if (kNewtonEvery > 0 && (i % kNewtonEvery) == 0) {
                            // Reciprocal on the FMA pipe: bit-trick seed (12 % off at worst) and two Newton steps,
                            // relative error 2.4e-4, half of what the fp16 rounding of P adds.
                            // (A masked score arrives here as t = +inf: bounded, so that the steps stay finite; the
                            // result, below 1e-30, still rounds to an fp16 zero.)
                            const float u0 = fminf(t0, 1e30f), u1 = fminf(t1, 1e30f);
                            const uint64_t nt2 = ptx::pack2(-u0, -u1), two2 = ptx::pack2(2.0f, 2.0f);
                            uint64_t r = ptx::pack2(__int_as_float(0x7EF311C7 - __float_as_int(u0)),
                                                    __int_as_float(0x7EF311C7 - __float_as_int(u1)));
                            r = ptx::mul2(r, ptx::fma2(nt2, r, two2));
                            r = ptx::mul2(r, ptx::fma2(nt2, r, two2));
                            ptx::unpack2(r, p0, p1);
                        } else {
                            p0 = ptx::rcp_approx(t0);
                            p1 = ptx::rcp_approx(t1);
                        }
                        pk[i] = ptx::pack_f16x2(p0, p1);
                    }
                    ptx::tmem_st_32x16(ts + cc * 16, pk);
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
                if (!fixed_max) {
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
                        // P V of the previous key tile (buffer (g-1) % kSBufs) must be done.  That barrier's earlier
                        // completion is known (S of this tile exists), so the parity wait cannot be mistaken.
                        if (!bounded_wait(ptx::smem_u32(&bars->pv_done[(g - 1u) % C::kSBufs]), ((g - 1u) / C::kSBufs) & 1u, bars, p.status_word)) return;
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
                }
                const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
                uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
                uint64_t sume[2] = {0ull, 0ull};
#pragma unroll
                for (int cc = 0; cc < kWgCols / 32; ++cc) {
                    uint32_t pk[16];
                    if (rounded_sum) exp_chunk<SCORE, true>(&y[cc * 32], cs, neg_m, sum2, pk, sume);
                    else exp_chunk<SCORE, false>(&y[cc * 32], cs, neg_m, sum2, pk);
                    ptx::tmem_st_32x16(ts + cc * 16, pk);
                }
                float s0, s1, s2, s3;
                ptx::unpack2(ptx::add2(sum2[0], sum2[1]), s0, s1);
                ptx::unpack2(ptx::add2(sum2[2], sum2[3]), s2, s3);
                l += (s0 + s1) + (s2 + s3);
                if (rounded_sum) {
                    ptx::unpack2(ptx::add2(sume[0], sume[1]), s0, s1);
                    l_exact += s0 + s1;
                }
            }
            // Publish this warp's P (and any rescaled O) to the MMA thread of the leader CTA.
            ptx::tmem_wait_st();
            ptx::tc_fence_before_sync();
            warp_arrive_on_leader(p_full_on_leader + buf * 8);
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
        if (!SIGMOID && !RELU && rounded_sum) {
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
        const bool relu_raw = RELU && p.scale > 0.f && !sc.softcap && !sc.has_bias;       // P holds max(s, 0) of the raw scores
        const float inv = SIGMOID ? p.out_scale * 0.0009765625f
                                  : (RELU ? (relu_raw ? p.out_scale * p.scale : p.out_scale * kLn2) : (l_row > 0.f ? 1.0f / l_row : 0.f));
        char* obase = reinterpret_cast<char*>(p.o) +
                      ((long long)it.b * p.os[0] + (long long)it.h * p.os[1] + (long long)row * p.os[2] + wg * kOC) * (p.o_fp32 ? 4 : 2);
#pragma unroll
        for (int c = 0; c < kOC / 32; ++c) {
            uint32_t orr[32];
            if (niter > 0) {
                ptx::tmem_ld_32x32(tm + ocol + c * 32, orr);
                ptx::tmem_wait_ld_regs(orr);
                if (c == kOC / 32 - 1) {
                    // This group's share of O is in registers: once all four groups of the pair say so, the next
                    // item's first P V may overwrite the accumulators.
                    ptx::tc_fence_before_sync();
                    warp_arrive_on_leader(o_free_on_leader);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) orr[i] = 0u;
            }
            if (store_row) {
                // 32-byte stores where the row piece is 32-byte aligned (always, for dense rows): a whole sector per
                // thread and instruction, half as many trips through the load/store unit as with 16-byte stores.
                if (p.o_fp32) {
                    char* dst = obase + c * 128;
                    const bool aligned32 = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w[8];
#pragma unroll
                        for (int k2 = 0; k2 < 8; ++k2) w[k2] = __float_as_uint(__uint_as_float(orr[8 * i + k2]) * inv);
                        if (aligned32) {
                            ptx::st_global_v8(dst + i * 32, w);
                        } else {
                            reinterpret_cast<uint4*>(dst + i * 32)[0] = make_uint4(w[0], w[1], w[2], w[3]);
                            reinterpret_cast<uint4*>(dst + i * 32)[1] = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                    }
                } else {
                    char* dst = obase + c * 64;
                    const bool aligned32 = (reinterpret_cast<uintptr_t>(dst) & 31u) == 0;
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
        if (!SIGMOID && !RELU && wg == 0 && p.lse && store_row)
            p.lse[((long long)it.b * p.Hq + it.h) * p.Sq + row] = (l_lse > 0.f) ? (m_used + ptx::lg2_approx(l_lse)) * kLn2 : -INFINITY;

        // Next work item: one lane reads the published index and shares it with the warp.
        int got = 0;
        if ((threadIdx.x & 31) == 0) got = next_item(bars, item_phase, p.status_word, pair) ? 1 : 0;
        got = __shfl_sync(0xffffffffu, got, 0);
        pair = __shfl_sync(0xffffffffu, pair, 0);
        if (!got) return;
    }
}

// ------------------------------------------------------------------------------------------------
// kernel (cluster of two CTAs)
// ------------------------------------------------------------------------------------------------
template <int D, int SCORE, int NORM>
__global__ void __launch_bounds__(NORM == kNormSigmoid ? Cfg<D>::kThreadsSigmoid : Cfg<D>::kThreads, 1)
attn_fwd_pair_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                     const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ AttnParams p) {
    using C = Cfg<D>;
    constexpr bool kVF16 = (NORM == kNormSigmoid);     // P and V as fp16 (see the top of this file)
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = ptx::smem_u32(smem);
    const uint32_t rank = ptx::cluster_ctarank();
    // The swizzled tiles need a 1024-byte aligned base (dynamic shared memory starts right after the 1 KB the
    // driver reserves).  Both CTAs see the same offset, so both leave together if that ever failed to hold.
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
        ptx::mbar_init(ptx::smem_u32(&bars->o_done), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->o_free), 2 * C::kSoftmaxWarps);
        for (int t = 0; t < 3; ++t) {
            ptx::mbar_init(ptx::smem_u32(&bars->s_full[t]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->p_full[t]), 2 * C::kSoftmaxWarps);
            ptx::mbar_init(ptx::smem_u32(&bars->pv_done[t]), 1);
        }
        for (int t = 0; t < 2; ++t) ptx::mbar_init(ptx::smem_u32(&bars->xchg[t]), C::kSoftmaxWarps);
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&bars->landed[s]), 1);
            if (s == 0) ptx::mbar_init(ptx::smem_u32(&bars->converted), 4);
            ptx::mbar_init(ptx::smem_u32(&bars->full[s]), kVF16 ? 2 : 1);   // sigmoid: two arrivals per use (see open_slot)
            ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_u32(&bars->clc), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->item_full), 1);
        ptx::mbar_init(ptx::smem_u32(&bars->item_empty), (rank == 0 ? C::kItemConsumers : C::kItemConsumers - 1) + (kVF16 ? 4 : 0));   // no MMA thread on the peer; sigmoid: four converter warps
        ptx::mbar_init(ptx::smem_u32(&bars->item_ready), 2);
        bars->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0) {
        ptx::tmem_alloc_pair<C::kTmemCols>(ptx::smem_u32(&bars->tmem_base));
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    ptx::cluster_sync_all();          // barriers of both CTAs are initialised before anyone signals across
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

    if (warp < C::kSoftmaxWarps) {
        if constexpr (kVF16) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsSoftmax));
        softmax_role<D, SCORE, NORM>(p, bars, xchg, tmem, warp >> 2, rank);
    } else if (kVF16 && warp >= C::kConverterWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsConverter));
        converter_role<D>(p, bars, smem + C::kQBytes);
    } else {
        if constexpr (kVF16) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
        if (warp == C::kProducerWarp) {
            if (lane == 0) producer_role<D, kVF16>(&tmap_q, &tmap_k, &tmap_v, p, bars, q_smem, ring_smem, rank);
        } else if (warp == C::kMmaWarp) {
            if (lane == 0 && rank == 0) mma_role<D, kVF16>(p, bars, tmem, q_smem, ring_smem);
        } else if (warp == C::kSchedWarp) {
            if (lane == 0) scheduler_role(bars, p.status_word, rank);
        } else if (warp == C::kSpareWarp && blockIdx.x == 0 && (p.mask_flags & kMaskDocument)) {
            check_offsets_warp(p.cu, p.num_docs, p.Sq, p.status_word);     // the spare warp of the first CTA
        }
        __syncwarp();
    }

    // Common exit: both CTAs meet before either gives back shared memory or TMEM that the other may still
    // signal into.  After an abort, give copies and MMAs still in flight time to land first.
    if (*reinterpret_cast<volatile int*>(&bars->abort_flag)) __nanosleep(1000000);
    ptx::tc_fence_before_sync();
    ptx::cluster_sync_all();
    if (warp == 0) ptx::tmem_dealloc_pair<C::kTmemCols>(tmem);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <int D, int SCORE, int NORM>
int launch_instance(AttnParams p, cudaStream_t stream) {
    using C = Cfg<D>;
    auto kernel = attn_fwd_pair_kernel<D, SCORE, NORM>;
    // The opt-in shared-memory size is a per-device function attribute: set it once per device.
    static SmemAttrFlags attr_set;
    if (!set_smem_attr_once(attr_set, kernel, C::kSmemBytes)) return ATTN_ERR_CUDA;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, p.q, p.B, p.Hq, p.Sq, D, p.qs, 128) || !make_map(&mk, p.k, p.B, p.Hkv, p.Sk, D, p.ks, 64) ||
        !make_map(&mv, p.v, p.B, p.Hkv, p.Sk, D, p.vs, 128))
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
    const long long nqb = (p.Sq + 2 * kBM - 1) / (2 * kBM);
    const long long grid = 2 * nqb * bh;
    if (grid > 0x7fffffffLL) return ATTN_ERR_SHAPE;
    p.defer_blocks = deferred_blocks(p, 2 * kBM, kBN, (int)nqb, bh, device_sm_count() / 2);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NORM == kNormSigmoid ? C::kThreadsSigmoid : C::kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, p) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
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

// CTA-pair kernel: D = 128 and D = 256.
int launch_attn_fwd_bf16_pair(const AttnParams& p, cudaStream_t stream) {
    switch (p.D) {
        case 128: return launch_for_d<128>(p, stream);
        case 256: return launch_for_d<256>(p, stream);
        default: return ATTN_ERR_UNSUPPORTED;
    }
}

}  // namespace b200attn
