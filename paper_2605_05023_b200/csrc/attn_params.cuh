// Kernel-side parameter block and the per-row visibility interval shared by the
// attention-forward kernels.  Every mask of Appendix A.2 that this library builds
// (causal, two-sided window, same-document, PrefixLM, the test-query clause of the
// causal blockwise mask) leaves each query row one contiguous interval of visible keys
// [lo, hi].  hi is non-decreasing in the row index; lo is non-decreasing too, except
// that it falls back to the window / sequence start at row test_query_start.
#pragma once
#include <algorithm>
#include <cstdint>
#include <cuda_runtime.h>

namespace b200attn {

enum : uint32_t { kMaskCausal = 1u, kMaskWindow = 2u, kMaskDocument = 4u, kMaskPrefix = 8u, kMaskTestQuery = 16u,
                  kMaskGlobal = 32u };
enum : int { kNormSoftmax = 0, kNormSigmoid = 1, kNormRelu = 2 };

struct AttnParams {
    const void* q;
    const void* k;
    const void* v;
    void* o;
    float* lse;                 // may be null
    int B, Hq, Hkv, Sq, Sk, D;
    int group;                  // Hq / Hkv
    long long qs[3], ks[3], vs[3], os[3];   // element strides: batch, head, row
    float scale;                // multiplies q.k
    float softcap;              // 0 = off
    const float* slopes;        // [Hq] or null
    float sigmoid_bias;
    float out_scale;
    uint32_t mask_flags;
    int window_left, window_right;   // < 0 = unbounded; host clamps large values
    const int32_t* cu;          // [num_docs + 1] or null
    int num_docs;
    int normalizer;
    int o_fp32;                 // output element type is fp32
    int32_t* status_word;       // may be null
    int sec_heads;              // tensor-core kernel: (batch, head) pairs per L2-sized section of the work order
    int prefix_len;             // PrefixLM: keys j < prefix_len are visible to every row (0 = none)
    int test_query_start;       // rows i >= this ignore the document clause (Sq = none)
    int global_len;             // global tokens: positions < global_len pass the window / document clauses (0 = none)
    int head_pair;              // ping-pong kernel: a work item is two heads x 128 rows (1) or one head x 256 rows (0)
    int defer_blocks;           // tensor-core kernels: query blocks per head whose work items end the work order (see work_order)
    int front_blocks;           // ... and whose work items open it (see leading_blocks)
    int sec_merge_from;         // ping-pong kernel: the sections from this one on are handed out as one (see work_order)
};

struct RowInterval {
    int lo, hi;                 // inclusive; lo > hi means no visible key
    int pre;                    // with global tokens: keys j < pre are visible too (0 otherwise; then pre <= lo - 1)
    int doc;                    // document of the row when the document clause was evaluated, else 0
};

// Index d of the document that holds token t: cu[d] <= t < cu[d+1].  Empty documents
// (cu[d] == cu[d+1]) are stepped over.  The result is clamped to [0, num_docs - 1].
// A caller that knows the answer lies in [first, last] passes that range (a query tile's threads get the
// documents of the tile's first and last row from the work item).
__device__ __forceinline__ int find_document(const int32_t* __restrict__ cu, int num_docs, int t, int first = 0, int last = -1) {
    int a = first, b = (last < 0) ? num_docs : last + 1;   // invariant: cu[a] <= t (cu[0] = 0), answer in [a, b)
    while (b - a > 1) {
        const int mid = (a + b) >> 1;
        if (__ldg(cu + mid) <= t) a = mid; else b = mid;
    }
    return a;
}

// Visible key interval of query row i (Appendix A.2 clauses combined by AND).
__device__ __forceinline__ RowInterval row_interval(const AttnParams& p, int i, int doc_first = 0, int doc_last = -1) {
    const int ip = i + p.Sk - p.Sq;
    int lo = 0, hi = p.Sk - 1, doc = 0;
    if (p.mask_flags & kMaskCausal) hi = min(hi, max(ip, p.prefix_len - 1));
    // A global token's row keeps only the causal clause.  (Tested on the flag: with Sq > Sk a row has i' < 0, which
    // is below global_len = 0 of a call without global tokens.)
    if ((p.mask_flags & kMaskGlobal) && ip < p.global_len) return RowInterval{0, hi, 0, 0};
    if (p.mask_flags & kMaskWindow) {
        if (p.window_left >= 0) lo = max(lo, ip - p.window_left);
        if (p.window_right >= 0) hi = min(hi, ip + p.window_right);
    }
    if ((p.mask_flags & kMaskDocument) && i < p.test_query_start) {
        doc = find_document(p.cu, p.num_docs, i, doc_first, doc_last);
        lo = max(lo, __ldg(p.cu + doc));
        hi = min(hi, __ldg(p.cu + doc + 1) - 1);
    }
    // Global tokens as keys: [0, global_len) joins the interval when they touch, else it is a second piece.
    int pre = 0;
    if (p.mask_flags & kMaskGlobal) {
        if (lo > hi) { lo = 0; hi = p.global_len - 1; }          // (the causal clause holds: global_len <= i')
        else if (lo <= p.global_len) { lo = 0; hi = max(hi, p.global_len - 1); }
        else pre = p.global_len;
    }
    return RowInterval{lo, hi, pre, doc};
}

// Bounds over the query rows [q0, q0 + rows) (clipped to Sq) of a tile: the keys that any row sees are inside
// [lo_min, hi_max]; the keys that every row sees are [lo_max, hi_min].  hi is monotone; lo is monotone on each
// side of test_query_start, so the extremes are at the tile's ends and at the row before test_query_start.
struct TileBounds {
    int lo_min, lo_max, hi_min, hi_max;
    int pre_min, pre_max;       // global-token prefix: every row sees keys < pre_min, some row sees keys < pre_max
    int doc_first, doc_last;    // documents of the first and last row (document clause; rows from the test query on: 0)
    bool any;                   // some row of the tile sees some key
};
__device__ __forceinline__ TileBounds tile_bounds(const AttnParams& p, int q0, int rows) {
    TileBounds t;
    t.doc_first = 0; t.doc_last = -1;
    if (q0 >= p.Sq) { t.lo_min = t.lo_max = 0; t.hi_min = t.hi_max = -1; t.pre_min = t.pre_max = 0; t.any = false; return t; }
    const int q1 = min(q0 + rows - 1, p.Sq - 1);
    const RowInterval a = row_interval(p, q0);
    const RowInterval b = row_interval(p, q1);
    // Rows between two rows of the document clause lie in documents between theirs; a tile that reaches the test
    // query (whose rows skip the clause) gives no such range.
    if ((p.mask_flags & kMaskDocument) && q1 < p.test_query_start) { t.doc_first = a.doc; t.doc_last = b.doc; }
    t.lo_min = min(a.lo, b.lo);
    t.lo_max = max(a.lo, b.lo);
    t.hi_min = a.hi;
    t.hi_max = b.hi;
    if ((p.mask_flags & kMaskDocument) && q0 < p.test_query_start && p.test_query_start <= q1)
        t.lo_max = max(t.lo_max, row_interval(p, p.test_query_start - 1).lo);
    t.pre_min = min(a.pre, b.pre);
    t.pre_max = max(a.pre, b.pre);
    if (p.mask_flags & kMaskGlobal) {
        // Rows of global tokens see up to the causal bound, the others up to their window: hi is not monotone
        // across position global_len, and with a test query the prefix piece is not either.  A tile that holds
        // such a break takes the union of its ends and classifies no key tile as fully visible.
        const int off = p.Sk - p.Sq;
        const bool breaks = (q0 + off < p.global_len && p.global_len <= q1 + off) ||
                            (q0 < p.test_query_start && p.test_query_start <= q1);
        t.hi_max = max(a.hi, b.hi);
        t.hi_min = min(a.hi, b.hi);
        if (breaks) {
            t.lo_min = 0;
            t.lo_max = 0x3fffffff;
            t.pre_min = 0;
            t.pre_max = p.global_len;
        }
    }
    t.any = !(t.hi_max < 0 || t.lo_min > t.hi_max) || t.pre_max > 0;
    return t;
}

// Work order of the tensor-core kernels: the (batch, head) unit and the query block of linear work index `lin`.
// Units are taken in sections of `sec_units` whose K/V fit in L2; inside a section the query block is the slow
// coordinate and runs from the heaviest block of a unit (rank 0) to the lightest, so the hardware hands out the
// heaviest items first.  The `defer` lightest blocks of every unit come after all sections, again heaviest first
// (see deferred_blocks).  rank: position of the block among its unit's `nqb` blocks, heaviest first.
// The sections from `merge_from` on form one section: a last section that holds less work per SM than its longest
// item takes ends the grid with idle SMs; as part of a longer section its long items start earlier and its light
// ones fill the end.
__device__ __forceinline__ void work_order(int lin, int units_total, int sec_units, int nqb, int defer, int& rank, int& unit,
                                           int merge_from = 0x7fffffff) {
    const int nh = nqb - defer;                          // blocks per unit that are taken section by section
    if (lin < units_total * nh) {
        const int per_sec = sec_units * nh;
        const int sec = min(lin / per_sec, merge_from);
        const int r = lin - sec * per_sec;
        const int sec_start = sec * sec_units;
        const int sh = min(sec >= merge_from ? units_total : sec_units, units_total - sec_start);
        rank = r / sh;
        unit = sec_start + r % sh;
    } else {                                             // the deferred blocks: one last section of all units
        const int r = lin - units_total * nh;
        rank = nh + r / units_total;
        unit = r % units_total;
    }
}

// The same with `front` blocks per unit that open the work order, before all sections, block by block over all units
// (rank < front): the blocks that hold the rows of global tokens under a non-causal mask, whose items walk every
// key tile while the others walk a window (see leading_blocks).  Every (rank, unit) pair still has exactly one index.
__device__ __forceinline__ void work_order_front(int lin, int units_total, int sec_units, int nqb, int defer, int front,
                                                 int& rank, int& unit, int merge_from = 0x7fffffff) {
    const int front_items = units_total * front;
    if (lin < front_items) {
        rank = lin / units_total;
        unit = lin - rank * units_total;
    } else {
        work_order(lin - front_items, units_total, sec_units, nqb - front, defer, rank, unit, merge_from);
        rank += front;
    }
}

// ------------------------------------------------------------------------------------------------ host side
// How many query blocks of every head open the work order, ahead of the sections: blocks whose work items are the
// longest of their head by far, which, handed out section by section, can end the grid on a few SMs when the last
// section starts late.  Two cases.  (a) Global Sliding Window (Appendix A.2), non-causal two-sided window: the blocks
// that hold a global token's row (such a row sees every key, the others a window).  (b) The causal blockwise mask with
// its test-query clause: the blocks of the test query's rows (they see every key up to their own position, the
// others their own document).  0 when there is little to gain: the long items have fewer than four times the key tiles
// of the others (for documents, estimated from the mean document length), a section lasts longer than a long item
// anyway (then the long items of the last section are hidden in it, and section order keeps its K and V in L2), or
// more than a quarter of the blocks would qualify.  `sec_units`: work-order units ((batch, head) or head pairs) per
// section, `units_total`: all of them; `workers`: CTAs that run at once.
inline int leading_blocks(const AttnParams& p, int rows, int key_tile, int nqb, long long sec_units, long long units_total, int workers) {
    if (nqb < 4) return 0;
    long long light_tiles, long_rows;
    if ((p.mask_flags & kMaskGlobal) && !(p.mask_flags & kMaskCausal)) {
        if (!(p.mask_flags & kMaskWindow) || p.window_left < 0 || p.window_right < 0) return 0;
        light_tiles = ((long long)p.window_left + p.window_right + rows) / key_tile + 2;
        long_rows = std::min<long long>(std::max<long long>((long long)p.global_len - (p.Sk - p.Sq), 0), p.Sq);
    } else if ((p.mask_flags & kMaskTestQuery) && (p.mask_flags & kMaskCausal) && !(p.mask_flags & kMaskGlobal)) {
        if (units_total <= 2 * sec_units) return 0;      // one section after the merge of the last two: the long blocks lead it anyway
        light_tiles = ((long long)p.Sk / std::max(p.num_docs, 1) + rows) / key_tile / 2 + 2;
        long_rows = std::max<long long>((long long)p.Sq - p.test_query_start, 0);
    } else {
        return 0;
    }
    const long long long_tiles = (long long)p.Sk / key_tile;
    if (long_tiles < 4 * light_tiles) return 0;
    const int blocks = (int)((long_rows + rows - 1) / rows);
    if (blocks == 0 || blocks * 4 > nqb) return 0;
    const long long section_steps = sec_units * (blocks * long_tiles + (nqb - blocks) * light_tiles) / std::max(workers, 1);
    return (section_steps >= long_tiles) ? 0 : blocks;
}

// How many of the first (lightest) query blocks of every head go to the end of the work order (decode_item of the
// ping-pong and of the CTA-pair kernel).  Causal masks without documents or global tokens only: there a block's key
// tiles grow with its index, and the count follows from the row intervals.  `rows`: query rows of a work item;
// `key_tile`: keys per key tile; `workers`: CTAs (or CTA pairs) that run at once.  As many blocks as hold about
// 0.6 x workers x (heaviest item) key tiles of work, at most half of the blocks; none when that is more than a quarter
// of all work (a small grid) or when the items do not differ by a factor of two (equal items need no filler).
inline int deferred_blocks(const AttnParams& p, int rows, int key_tile, int nqb, long long items_per_block, int workers) {
    if (!(p.mask_flags & kMaskCausal) || (p.mask_flags & (kMaskDocument | kMaskGlobal)) || nqb < 4) return 0;
    auto tiles = [&](int qb) -> long long {           // key tiles of the block's item (union over its rows)
        const long long first = (long long)qb * rows + p.Sk - p.Sq;
        const long long last = std::min<long long>((long long)(qb + 1) * rows, p.Sq) - 1 + p.Sk - p.Sq;
        long long hi = std::max<long long>(last, (long long)p.prefix_len - 1);
        hi = std::min<long long>(hi, p.Sk - 1);
        long long lo = 0;
        if ((p.mask_flags & kMaskWindow) && p.window_left >= 0) lo = std::max<long long>(0, first - p.window_left);
        if (p.prefix_len > 0 && first < p.prefix_len) lo = 0;
        if (hi < 0 || lo > hi) return 0;
        return hi / key_tile - lo / key_tile + 1;
    };
    long long total = 0, w_max = 0, w_min = 1ll << 40;
    for (int qb = 0; qb < nqb; ++qb) { const long long w = tiles(qb); total += w; w_max = std::max(w_max, w); w_min = std::min(w_min, w); }
    if (w_max < 2 * std::max<long long>(w_min, 1)) return 0;
    const long long target = (long long)workers * w_max * 6 / 10;
    if (target > total * items_per_block / 4) return 0;      // a small grid: the "filler" would be most of the work
    long long cum = 0;
    int d = 0;
    while (d < nqb / 2 && cum < target) { cum += tiles(d) * items_per_block; ++d; }
    return d;
}

}  // namespace b200attn
