// bf16 GEMM with a fused row-sum epilogue on tcgen05 with CTA pairs (cta_group::2).
//
// C = A B and rowsum[m] = sum_n C[m, n] in one kernel (the operator of the paper's GEMM case study, Table
// "GEMM+ReduceSum").  A is [M, K] row-major (the K-major A operand), B is [K, N] row-major (an N-major B
// operand: the same shared-memory form as V in the attention kernels), accumulation in fp32 in TMEM.
//
// A cluster of two CTAs owns a 256 x 256 tile of C: each CTA loads its own 128 rows of A and its own 128
// columns of B per 64-wide K step (32 KB instead of the 48 KB a lone CTA needs for 128 x 256: the pair halves
// the B traffic from L2 per FLOP), and the leader CTA issues tcgen05.mma.cta_group::2 with M = 256, N = 256
// that leaves each CTA's 128 rows of the accumulator in that CTA's own TMEM.  The accumulator is double
// buffered (2 x 256 of the 512 TMEM columns), so the epilogue of one tile runs under the main loop of the next.
// Pairs are persistent and take tiles round-robin.  When the 256 x 256 tiles do not fill the last round (or there
// are fewer of them than pairs), the launcher splits the tiles of that round into 256 x 128 halves so that more
// pairs share it: a narrow tile loads one box of B per CTA and runs the MMA with N = 128.
//
// Roles per CTA: warp 0 = TMA producer (one thread), warp 1 = MMA issuer (one thread, leader only), warps 2-5 =
// epilogue, thread = row: tcgen05.ld 32 columns at a time, add them to the thread's fp32 row sum (taken from the
// unrounded accumulators; no cross-thread step is needed because a thread holds a whole row of the tile),
// round to bf16 and store C, then one atomic add per row and tile into rowsum.
// Edges: TMA zero-fills rows >= M, columns >= N and the K tail, so they add nothing; stores are guarded.
//
// Cross-CTA signalling as in the CTA-pair attention kernel: TMA loads of both CTAs count on the leader's
// `full` barrier; tcgen05.commit arrives on the same barrier in both CTAs; the epilogue warps of both CTAs
// arrive on the leader's `acc_empty`.  Every mbarrier wait is bounded: after kWaitLimitNs the waiting role
// records ATTN_ERR_TIMEOUT in the caller's status word, raises a CTA-wide abort flag and all roles drain to
// the common exit (cluster barrier, which every thread of both CTAs reaches; TMEM released after it).
#include <cstdlib>

#include <cuda.h>

#include "../../include/attn.h"
#include "gemm_rowsum_params.cuh"
#include "sm100_ptx.cuh"
#include "attn_tc_common.cuh"

namespace b200attn {

namespace {

using namespace tc;

constexpr int kTileM = 128;                      // rows of C per CTA (256 per pair)
constexpr int kTileN = 256;                      // columns of C per pair
constexpr int kHalfN = kTileN / 2;               // columns of B that each CTA loads
constexpr int kTileK = 64;                       // K step: one 128-byte swizzle row of bf16
constexpr int kMaxStages = 6;
constexpr int kABytes = kTileM * kTileK * 2;     // [128 rows x 64 k] = 16 KB
constexpr int kBBoxBytes = kTileK * 64 * 2;      // [64 k x 64 columns] = 8 KB
constexpr int kBarBytes = 1024;
constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
constexpr int kFirstEpiWarp = 2;
constexpr int kTmemCols = 512;                   // two accumulators of kTileN columns

// kAccs = 1: tiles of 256 x 256, the two TMEM accumulators alternate between consecutive tiles (the epilogue of one
// tile runs under the main loop of the next).  kAccs = 2: tiles of 256 x 512, both accumulators belong to one tile:
// per K step each CTA loads 48 KB for twice the work (a third less traffic from L2 per FLOP, which is what bounds
// the 256 x 256 form when every SM is busy), and only the second accumulator's epilogue overlaps the next tile.
template <int kAccs>
struct Cfg {
    static constexpr int kStages = (kAccs == 1) ? 6 : 4;
    static constexpr int kBBytes = kAccs * (kHalfN / 64) * kBBoxBytes;    // this CTA's 128 columns of B per accumulator
    static constexpr int kStageBytes = kABytes + kBBytes;                  // 32 KB or 48 KB
    static constexpr int kDataBytes = kStages * kStageBytes;
    static constexpr int kSmemBytes = kDataBytes + kBarBytes;
    static constexpr int kTileCols = kAccs * kTileN;
    static_assert(kStages <= kMaxStages, "barrier arrays");
    static_assert(kSmemBytes <= 232448, "shared memory budget");
};

// Same layout in both CTAs.  L: only the leader's copy is waited on.  B: each CTA waits on its own copy.
struct Barriers {
    uint64_t full[kMaxStages];    // L  A and B of both CTAs landed in this ring slot
    uint64_t empty[kMaxStages];   // B  ring slot consumed (tcgen05.commit to both CTAs)
    uint64_t acc_full[2];      // B  accumulator complete (tcgen05.commit to both CTAs)
    uint64_t acc_empty[2];     // L  both epilogues have read the accumulator (2 x kEpiWarps arrivals)
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= kBarBytes, "barrier block");

__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* status_word) {
    return bounded_wait_on<false>(bar, parity, &bars->abort_flag, status_word);
}

// Tile t of the pair's round-robin sequence: first n_wide tiles of 256 columns, then narrow tiles of 128 columns
// (two per 256 x 256 tile of the grid).  Column tiles are the fast coordinate, so the pairs that run together
// share a few row panels of A and all column panels of B in L2.
template <int kAccs>
__device__ __forceinline__ void tile_origin(const GemmRowsumParams& p, int t, int& row0, int& col0, int& width) {
    int g = t, half = 0;
    width = Cfg<kAccs>::kTileCols;
    if (kAccs == 1 && t >= p.n_wide) {
        const int u = t - p.n_wide;
        g = p.n_wide + (u >> 1);
        half = u & 1;
        width = kHalfN;
    }
    const int tm = g / p.tiles_n;
    row0 = tm * 2 * kTileM;
    col0 = (g - tm * p.tiles_n) * Cfg<kAccs>::kTileCols + half * kHalfN;
}

// ------------------------------------------------------------------------------------------------
// producer: TMA (this CTA's 128 rows of A and 128 columns of B for every K step)
// ------------------------------------------------------------------------------------------------
template <int kAccs>
__device__ __forceinline__ void producer_role(const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const GemmRowsumParams& p,
                                              Barriers* bars, uint32_t ring_smem, uint32_t rank) {
    using C = Cfg<kAccs>;
    ptx::prefetch_tensormap(tmap_a);
    ptx::prefetch_tensormap(tmap_b);
    int ps = 0;
    uint32_t pph = 0;
    const int n_pairs = (int)(gridDim.x >> 1);
    const int nk = (p.K + kTileK - 1) / kTileK;
    for (int t = (int)(blockIdx.x >> 1); t < p.n_tiles; t += n_pairs) {
        int row0, col0, width;
        tile_origin<kAccs>(p, t, row0, col0, width);
        row0 += (int)rank * kTileM;
        const bool narrow = width == kHalfN;                                // one box of B per CTA instead of two
        col0 += (int)rank * (narrow ? kHalfN / 2 : kHalfN);
        const uint32_t tx = 2u * (uint32_t)(narrow ? kABytes + kBBoxBytes : C::kStageBytes);   // the bytes of both CTAs
        for (int ks = 0; ks < nk; ++ks) {
            if (!bounded_wait(ptx::smem_u32(&bars->empty[ps]), pph ^ 1u, bars, p.status_word)) return;
            const uint32_t bar = ptx::smem_u32(&bars->full[ps]);
            const uint32_t dst = ring_smem + ps * C::kStageBytes;
            if (rank == 0) ptx::mbar_arrive_expect_tx(bar, tx);
            ptx::tma_load_4d_pair(dst, tmap_a, bar, ks * kTileK, row0, 0, 0);
            // Accumulator a covers columns [256 a, 256 a + 256) of the tile; this CTA holds 128 of them as two boxes.
#pragma unroll
            for (int a = 0; a < kAccs; ++a) {
                ptx::tma_load_4d_pair(dst + kABytes + (2 * a) * kBBoxBytes, tmap_b, bar, col0 + a * kTileN, ks * kTileK, 0, 0);
                if (!narrow)
                    ptx::tma_load_4d_pair(dst + kABytes + (2 * a + 1) * kBBoxBytes, tmap_b, bar, col0 + a * kTileN + 64, ks * kTileK, 0, 0);
            }
            if (++ps == C::kStages) { ps = 0; pph ^= 1u; }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// MMA issuer (one thread of the leader CTA)
// ------------------------------------------------------------------------------------------------
template <int kAccs>
__device__ __forceinline__ void mma_role(const GemmRowsumParams& p, Barriers* bars, uint32_t tmem, uint32_t ring_smem) {
    using C = Cfg<kAccs>;
    constexpr uint32_t kIdescWide = instr_desc(2 * kTileM, kTileN, true);
    constexpr uint32_t kIdescNarrow = instr_desc(2 * kTileM, kHalfN, true);
    // Descriptor halves (128-byte swizzle, SBO = 1024 B, sm_100 version bit): hi is constant, lo = (address >> 4) |
    // (LBO >> 4) << 16 advances by compile-time constants inside a stage.
    constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
    constexpr uint32_t kLoA = 1u << 16;                                    // LBO unused for a K-major operand
    constexpr uint32_t kLoB = (uint32_t)(kBBoxBytes >> 4) << 16;           // LBO between 64-column blocks of B
    const uint32_t ring_lo = (ring_smem & 0x3FFFFu) >> 4;
    const uint32_t bar_full = ptx::smem_u32(&bars->full[0]);
    const uint32_t bar_empty = ptx::smem_u32(&bars->empty[0]);

    int cs = 0;
    uint32_t cph = 0;
    const int n_pairs = (int)(gridDim.x >> 1);
    const int nk = (p.K + kTileK - 1) / kTileK;
    uint32_t it = 0;                                 // tiles of this pair so far
    for (int t = (int)(blockIdx.x >> 1); t < p.n_tiles; t += n_pairs, ++it) {
        const uint32_t idesc = (kAccs == 2 || t < p.n_wide) ? kIdescWide : kIdescNarrow;
        for (int ks = 0; ks < nk; ++ks) {
            if (!bounded_wait(bar_full + cs * 8, cph, bars, p.status_word)) return;
            ptx::tc_fence_after_sync();
            const uint32_t a_lo = (ring_lo + (uint32_t)cs * (C::kStageBytes >> 4)) | kLoA;
#pragma unroll
            for (int a = 0; a < kAccs; ++a) {
                // Accumulator buffer and how many times it was used before: one tile per buffer in turn, or both
                // buffers in every tile.
                const uint32_t buf = (kAccs == 1) ? (it & 1u) : (uint32_t)a;
                const uint32_t use = (kAccs == 1) ? (it >> 1) : it;
                if (ks == 0) {
                    // The epilogues of both CTAs must have read what this accumulator held before.
                    if (use >= 1u && !bounded_wait(ptx::smem_u32(&bars->acc_empty[buf]), (use - 1u) & 1u, bars, p.status_word)) return;
                    ptx::tc_fence_after_sync();
                }
                const uint32_t d = tmem + buf * kTileN;
                const uint32_t b_lo = (ring_lo + (uint32_t)cs * (C::kStageBytes >> 4) + ((kABytes + 2 * a * kBBoxBytes) >> 4)) | kLoB;
#pragma unroll
                for (int kk = 0; kk < kTileK / 16; ++kk)
                    ptx::mma_ss_pair(d, a_lo + (uint32_t)((kk * 32) >> 4), kDescHi, b_lo + (uint32_t)((kk * 2048) >> 4), kDescHi, idesc,
                                     (ks > 0 || kk > 0) ? 1u : 0u);
                if (ks == nk - 1) ptx::tc_commit_pair(ptx::smem_u32(&bars->acc_full[buf]));
            }
            ptx::tc_commit_pair(bar_empty + cs * 8);
            if (++cs == C::kStages) { cs = 0; cph ^= 1u; }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// epilogue: one thread per row of the CTA's half tile
// ------------------------------------------------------------------------------------------------
template <int kAccs>
__device__ __forceinline__ void epilogue_role(const GemmRowsumParams& p, Barriers* bars, uint32_t tmem, uint32_t rank) {
    const uint32_t quarter = (uint32_t)(threadIdx.x >> 5) & 3u;            // TMEM lanes this warp may touch
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t tm = tmem + ((quarter * 32u) << 16);
    const uint32_t empty_on_leader[2] = {ptx::mapa(ptx::smem_u32(&bars->acc_empty[0]), 0),
                                         ptx::mapa(ptx::smem_u32(&bars->acc_empty[1]), 0)};
    const int n_pairs = (int)(gridDim.x >> 1);
    uint32_t it = 0;
    for (int t = (int)(blockIdx.x >> 1); t < p.n_tiles; t += n_pairs, ++it) {
        int row0, col0, width;
        tile_origin<kAccs>(p, t, row0, col0, width);
        const int n_chunks = (width < kTileN ? width : kTileN) / 32;       // per accumulator
        const int row = row0 + (int)rank * kTileM + (int)(quarter * 32u + lane);
        const bool row_ok = row < p.M;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
        for (int a = 0; a < kAccs; ++a) {
            const uint32_t buf = (kAccs == 1) ? (it & 1u) : (uint32_t)a;
            const uint32_t use = (kAccs == 1) ? (it >> 1) : it;
            const int acol0 = col0 + a * kTileN;
            if (!bounded_wait(ptx::smem_u32(&bars->acc_full[buf]), use & 1u, bars, p.status_word)) return;
            ptx::tc_fence_after_sync();

            char* crow = p.c ? reinterpret_cast<char*>(p.c) + ((long long)row * p.ldc + acol0) * 2 : nullptr;
            uint32_t acc[2][32];
            ptx::tmem_ld_32x32(tm + buf * kTileN, acc[0]);
#pragma unroll
            for (int c = 0; c < kTileN / 32; ++c) {
                if (c >= n_chunks) break;                                   // narrow tile (warp-uniform)
                uint32_t (&cur)[32] = acc[c & 1];
                ptx::tmem_wait_ld_regs(cur);
                if (c + 1 < n_chunks) {
                    ptx::tmem_ld_32x32(tm + buf * kTileN + (c + 1) * 32, acc[(c + 1) & 1]);   // overlaps this chunk's arithmetic
                } else {
                    // The whole accumulator is in registers: the MMA thread may use it for a later tile.
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster_relaxed(empty_on_leader[buf]);
                }
                // Row sum over the unrounded accumulators (columns >= N hold exact zeros).
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    s0 += __uint_as_float(cur[i]);
                    s1 += __uint_as_float(cur[i + 1]);
                    s2 += __uint_as_float(cur[i + 2]);
                    s3 += __uint_as_float(cur[i + 3]);
                }
                if (crow && row_ok) {
                    uint4* dst = reinterpret_cast<uint4*>(crow + c * 64);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (acol0 + c * 32 + i * 8 < p.N) {                 // N is a multiple of 8
                            uint4 w;
                            w.x = ptx::pack_bf16x2(__uint_as_float(cur[8 * i]), __uint_as_float(cur[8 * i + 1]));
                            w.y = ptx::pack_bf16x2(__uint_as_float(cur[8 * i + 2]), __uint_as_float(cur[8 * i + 3]));
                            w.z = ptx::pack_bf16x2(__uint_as_float(cur[8 * i + 4]), __uint_as_float(cur[8 * i + 5]));
                            w.w = ptx::pack_bf16x2(__uint_as_float(cur[8 * i + 6]), __uint_as_float(cur[8 * i + 7]));
                            dst[i] = w;
                        }
                    }
                }
            }
        }
        if (row_ok) atomicAdd(p.rowsum + row, (s0 + s1) + (s2 + s3));
    }
}

// ------------------------------------------------------------------------------------------------
// kernel (cluster of two CTAs)
// ------------------------------------------------------------------------------------------------
template <int kAccs>
__global__ void __launch_bounds__(kThreads, 1)
gemm_rowsum_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                        const __grid_constant__ GemmRowsumParams p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = ptx::smem_u32(smem);
    const uint32_t rank = ptx::cluster_ctarank();
    // The swizzled tiles need a 1024-byte aligned base.  Both CTAs see the same offset, so both leave together if
    // that ever failed to hold.
    if ((base & 1023u) != 0u) {
        if (threadIdx.x == 0 && p.status_word) atomicExch(p.status_word, (int)ATTN_ERR_ALIGN);
        return;
    }
    Barriers* bars = reinterpret_cast<Barriers*>(smem + Cfg<kAccs>::kDataBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(ptx::smem_u32(&bars->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(ptx::smem_u32(&bars->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&bars->acc_empty[b]), 2 * kEpiWarps);
        }
        bars->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0) {
        ptx::tmem_alloc_pair<kTmemCols>(ptx::smem_u32(&bars->tmem_base));
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    ptx::cluster_sync_all();          // barriers of both CTAs are initialised before anyone signals across
    ptx::tc_fence_after_sync();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

    if (warp >= kFirstEpiWarp) {
        epilogue_role<kAccs>(p, bars, tmem, rank);
    } else {
        if (warp == 0) {
            if (lane == 0) producer_role<kAccs>(&tmap_a, &tmap_b, p, bars, base, rank);
        } else {
            if (lane == 0 && rank == 0) mma_role<kAccs>(p, bars, tmem, base);
        }
        __syncwarp();
    }

    // Common exit: both CTAs meet before either gives back shared memory or TMEM that the other may still
    // signal into.  After an abort, give copies and MMAs still in flight time to land first.
    if (*reinterpret_cast<volatile int*>(&bars->abort_flag)) __nanosleep(1000000);
    ptx::tc_fence_before_sync();
    ptx::cluster_sync_all();
    if (warp == 0) ptx::tmem_dealloc_pair<kTmemCols>(tmem);
}

}  // namespace

namespace {

// Sets the kernel's shared-memory attribute and asks how many clusters of two fit on the device at once (once per
// device and kernel).  Persistent pairs take tiles round-robin, so the grid must not exceed what is resident at once
// (a GPC with an odd number of free SMs leaves one of them without a partner).
template <int kAccs>
int prepare(int dev, cudaLaunchConfig_t& cfg, int& max_pairs_out) {
    static std::atomic<bool> attr_set[64];      // host threads may race on the first call: both compute the same values
    static std::atomic<int> max_pairs[64];
    auto kernel = gemm_rowsum_pair_kernel<kAccs>;
    cfg.dynamicSmemBytes = Cfg<kAccs>::kSmemBytes;
    if (!attr_set[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<kAccs>::kSmemBytes) != cudaSuccess)
            return ATTN_ERR_CUDA;
        int sms = 0, n = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2) return ATTN_ERR_CUDA;
        cfg.gridDim = dim3((unsigned)(sms / 2 * 2), 1, 1);
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n < 1) return ATTN_ERR_CUDA;
        max_pairs[dev].store(n < sms / 2 ? n : sms / 2, std::memory_order_relaxed);
        attr_set[dev].store(true, std::memory_order_release);
    }
    max_pairs_out = max_pairs[dev].load(std::memory_order_relaxed);
    return ATTN_OK;
}

}  // namespace

int launch_gemm_rowsum_bf16(GemmRowsumParams p, cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ATTN_ERR_CUDA;
    if (dev < 0 || dev >= 64) return ATTN_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // A as [1, 1, M, K] with boxes of 128 rows x 64 k; B as [1, 1, K, N] with boxes of 64 k x 64 columns.
    CUtensorMap ma, mb;
    const long long sa[3] = {(long long)p.M * p.lda, (long long)p.M * p.lda, p.lda};
    const long long sb[3] = {(long long)p.K * p.ldb, (long long)p.K * p.ldb, p.ldb};
    if (!make_map(&ma, p.a, 1, 1, p.M, p.K, sa, kTileM, kTileK) || !make_map(&mb, p.b, 1, 1, p.K, p.N, sb, kTileK, 64))
        return ATTN_ERR_CUDA;
    p.tiles_m = (p.M + 2 * kTileM - 1) / (2 * kTileM);
    const char* mode = std::getenv("B200ATTN_GEMM_TILES");   // wide / narrow / big: overrides the choice (for measurements)

    // 256 x 512 tiles when the main loop is long enough to pay for their exposed epilogue and there are enough of
    // them for every pair.
    int P2 = 0;
    if (int rc = prepare<2>(dev, cfg, P2)) return rc;
    const long long big_tiles = (long long)p.tiles_m * ((p.N + 2 * kTileN - 1) / (2 * kTileN));
    bool big = p.K >= 2048 && big_tiles >= P2;
    if (mode) big = mode[0] == 'b';
    if (big) {
        p.tiles_n = (p.N + 2 * kTileN - 1) / (2 * kTileN);
        if (big_tiles > 0x3fffffffLL) return ATTN_ERR_SHAPE;
        p.n_wide = p.n_tiles = (int)big_tiles;
        const long long pairs = big_tiles < P2 ? big_tiles : P2;
        cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
        if (cudaMemsetAsync(p.rowsum, 0, (size_t)p.M * sizeof(float), stream) != cudaSuccess) return ATTN_ERR_CUDA;
        return cudaLaunchKernelEx(&cfg, gemm_rowsum_pair_kernel<2>, ma, mb, p) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
    }

    int P1 = 0;
    if (int rc = prepare<1>(dev, cfg, P1)) return rc;
    p.tiles_n = (p.N + kTileN - 1) / kTileN;
    const long long tiles = (long long)p.tiles_m * p.tiles_n;
    if (tiles > 0x3fffffffLL) return ATTN_ERR_SHAPE;
    // The tiles of a last round that would occupy at most half of the pairs are split into 256 x 128 halves.
    const long long rem = tiles % P1;
    bool split = rem > 0 && 2 * rem <= P1;
    long long n_split = rem;
    if (mode && mode[0] == 'w') split = false;
    if (mode && mode[0] == 'n') { split = true; n_split = tiles; }
    p.n_wide = (int)(split ? tiles - n_split : tiles);
    p.n_tiles = (int)(split ? tiles + n_split : tiles);
    const long long pairs = p.n_tiles < P1 ? p.n_tiles : P1;
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    // The row sums are cleared on the caller's stream only now, after everything that can fail on the host.
    if (cudaMemsetAsync(p.rowsum, 0, (size_t)p.M * sizeof(float), stream) != cudaSuccess) return ATTN_ERR_CUDA;
    return cudaLaunchKernelEx(&cfg, gemm_rowsum_pair_kernel<1>, ma, mb, p) == cudaSuccess ? ATTN_OK : ATTN_ERR_CUDA;
}

}  // namespace b200attn
