// Kernel-side parameter block and the per-row visibility interval shared by the
// attention-forward kernels.  Every mask of Appendix A.2 that this library builds
// (causal, two-sided window, same-document, PrefixLM, the test-query clause of the
// causal blockwise mask) leaves each query row one contiguous interval of visible keys
// [lo, hi].  hi is non-decreasing in the row index; lo is non-decreasing too, except
// that it falls back to the window / sequence start at row test_query_start.
#pragma once
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

}  // namespace b200attn
