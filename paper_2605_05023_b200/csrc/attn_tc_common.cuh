// Pieces shared by the three tensor-core attention kernels (attn_tc_pingpong.cuh, attn_tc_pair.cu,
// attn_tc_split.cu): tile sizes and constants, the tcgen05 instruction descriptor, the element-wise mask of a
// partial tile, the exponential step of the online softmax, and the host-side TMA tensor maps.  (Bounded waits,
// the work-item fetch and the warp-level arrivals are in sm100_sync.cuh.)
#pragma once
#include <algorithm>
#include <atomic>

#include <cuda.h>
#include <cuda_runtime.h>

#include "sm100_ptx.cuh"
#include "sm100_sync.cuh"

namespace b200attn {
namespace tc {

constexpr int kBM = 128;                         // query rows per tile
constexpr int kBN = 128;                         // keys per tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;        // log2 units: P stays below 2^8

// Score instances compiled per kernel: no modifier, linear bias only, anything (softcap and / or bias).
enum : int { kScorePlain = 0, kScoreBias = 1, kScoreGeneric = 2 };

// Instruction descriptor of tcgen05.mma kind::f16: bf16 x bf16 -> fp32 (or, with f16_operands, f16 x f16 -> fp32),
// A K-major.  (A and B must have the same element type: an f16 A operand with a bf16 B operand is rejected by
// the hardware.)
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major, bool f16_operands = false) {
    return (1u << 4) | (f16_operands ? 0u : ((1u << 7) | (1u << 10))) | (b_mn_major ? (1u << 16) : 0u) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Mask of a partial tile (Appendix A.2; loop splitting, Sec. 3.4: only tiles that straddle an edge of a row's
// interval come here).  y holds 32 score columns of one row; columns outside [a, e] (chunk-relative, inclusive)
// become -inf.  Two forms with the same result: one bit test per element against a visibility word built with
// two shifts, or two compares per element (a few kernel instances are faster with the latter).
// `pre` adds a second visible piece: the columns below it (global tokens; 0 = none).
__device__ __forceinline__ void mask_chunk32_bits(uint32_t* y, int a, int e, int pre = 0) {
    const int lo = max(a, 0), hi = min(e, 31);
    uint32_t vis = (lo <= hi) ? ((0xffffffffu << lo) & (0xffffffffu >> (31 - hi))) : 0u;
    if (pre > 0) vis |= (pre >= 32) ? 0xffffffffu : ((1u << pre) - 1u);
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (!(vis & (1u << i))) y[i] = __float_as_uint(-INFINITY);
}
__device__ __forceinline__ void mask_chunk32_cmp(uint32_t* y, int a, int e, int pre = 0) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if ((i < a || i > e) && i >= pre) y[i] = __float_as_uint(-INFINITY);
}

// exp2 of 32 shifted scores -> 16 packed bf16 pairs; accumulates the fp32 row sum in four packed lanes.
// kSumRounded: the row sum is taken over the bf16-rounded weights that P V will use, so that the output is an
// exactly normalised average of V rows even when no weight is exactly 1 (fixed reference instead of the row
// maximum); the unrounded sum, which the LSE wants, goes to sum_exact.
template <int SCORE, bool kSumRounded = false>
__device__ __forceinline__ void exp_chunk(const uint32_t* y, float cs, float neg_m, uint64_t (&sum2)[4], uint32_t (&pk)[16],
                                          uint64_t* sum_exact = nullptr) {
    const uint64_t cs2 = ptx::pack2(cs, cs), nm2 = ptx::pack2(neg_m, neg_m), one2 = ptx::pack2(1.0f, 1.0f);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint64_t yy = ptx::pack2(__uint_as_float(y[2 * i]), __uint_as_float(y[2 * i + 1]));
        const uint64_t e = (SCORE == kScorePlain) ? ptx::fma2(yy, cs2, nm2) : ptx::fma2(yy, one2, nm2);
        float e0, e1;
        ptx::unpack2(e, e0, e1);
        const float p0 = ptx::ex2_approx(e0), p1 = ptx::ex2_approx(e1);
        pk[i] = ptx::pack_bf16x2(p0, p1);
        if constexpr (kSumRounded) {
            sum2[i & 3] = ptx::add2(sum2[i & 3], ptx::pack2(__uint_as_float(pk[i] << 16), __uint_as_float(pk[i] & 0xffff0000u)));
            sum_exact[i & 1] = ptx::add2(sum_exact[i & 1], ptx::pack2(p0, p1));
        } else {
            sum2[i & 3] = ptx::add2(sum2[i & 3], ptx::pack2(p0, p1));
        }
    }
}

// ------------------------------------------------------------------------------------------------ host side
// The opt-in shared-memory size is a per-device attribute of each kernel: set by the first call on a device.
// `done` is the calling launcher's own flag array (one per kernel instance).  Host threads may race on the first
// call: the flags are atomic and setting the attribute twice is harmless.
using SmemAttrFlags = std::atomic<bool>[64];
template <typename Kernel>
inline bool set_smem_attr_once(SmemAttrFlags& done, Kernel kernel, int bytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const bool tracked = dev >= 0 && dev < 64;
    if (tracked && done[dev].load(std::memory_order_acquire)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (tracked) done[dev].store(true, std::memory_order_release);
    return true;
}

// SMs of the current device (cached per device; 148 on a B200), for the kernels' work-order heuristics.
inline int device_sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    const bool tracked = dev >= 0 && dev < 64;
    if (tracked) { const int c = cached[dev].load(std::memory_order_acquire); if (c > 0) return c; }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    if (tracked) cached[dev].store(n, std::memory_order_release);
    return n;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// bf16 tensor [B, H, S, D] with element strides st (batch, head, row): box = box_cols columns x box_rows rows,
// 128-byte swizzle (the layout tcgen05.mma reads directly).
struct MapKey {
    const void* ptr;
    int B, H, S, D;
    long long st[3];
    int box_rows, box_cols;
    int swizzle_bytes;      // 128 (operand tiles) or 64 (32-column output boxes)
};
inline bool encode_map(CUtensorMap* map, const MapKey& k) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)k.D, (cuuint64_t)k.S, (cuuint64_t)k.H, (cuuint64_t)k.B};
    const cuuint64_t strides[3] = {(cuuint64_t)k.st[2] * 2, (cuuint64_t)k.st[1] * 2, (cuuint64_t)k.st[0] * 2};
    const cuuint32_t box[4] = {(cuuint32_t)k.box_cols, (cuuint32_t)k.box_rows, 1u, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(k.ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, k.swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Encoded maps are cached by key (attn_api.cu; emptied by attn_clear_cache()).
bool cached_map(CUtensorMap* out, const MapKey& key);
void clear_map_cache();
long long map_cache_hits();

inline bool make_map(CUtensorMap* map, const void* ptr, int B, int H, int S, int D, const long long st[3], int box_rows,
                     int box_cols = 64, int swizzle_bytes = 128) {
    const MapKey key = {ptr, B, H, S, D, {st[0], st[1], st[2]}, box_rows, box_cols, swizzle_bytes};
    return cached_map(map, key);
}

}  // namespace tc
}  // namespace b200attn
