// fp32 attention forward on the FMA pipe: the path for fp32 inputs.
//
// tcgen05 kind::tf32 rounds operands to 10 mantissa bits, which cannot meet a 1e-5
// absolute bar, so fp32 inputs are contracted with plain FFMA.  A CTA of eight warps
// owns eight consecutive query rows of one (batch, head); one warp owns one row.  The
// CTA walks the keys that any of its rows can see, 32 keys at a time; each chunk of K
// and V rows is brought into shared memory once for all eight rows (cp.async, three
// stages: the next two chunks are in flight while the current one is used):
//   phase 1: lane l computes the score of key j0 + l (q row and K chunk in shared
//            memory), applies softcap / linear bias (Appendix A.1), and the warp keeps
//            an online softmax (running max, running sum) or evaluates the sigmoid /
//            ReLU normaliser (Appendix A.3);
//   phase 2: lanes switch to owning output columns and accumulate p_j * V[j, :].
// Chunks outside the CTA's key range are never touched (masked tiles skipped; Appendix
// A.2); inside a chunk every row applies its own visibility: an invisible key gets the
// weight 0 and still goes through the (branch-free, fully unrolled) accumulation, which is
// why staged rows past Sk are zero-filled.  The kernel is compiled per number of 32-column
// groups of the head dimension.
#include "attn_params.cuh"
#include "sm100_sync.cuh"

namespace b200attn {

constexpr int kSimtWarps = 8;           // query rows per CTA
constexpr int kSimtMaxD = 256;
constexpr int kSimtChunk = 32;          // keys per chunk
constexpr int kSimtStages = 3;         // K/V chunks in shared memory: one in use, two in flight
constexpr int kSimtPad = 4;             // floats of padding per staged row: a warp's float4 reads of 32 rows hit all banks

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ void cp_async16(float* dst_smem, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// Waits until at most kSimtStages - 2 of the most recently committed groups are still in flight.
__device__ __forceinline__ void cp_async_wait_oldest() { asm volatile("cp.async.wait_group %0;" ::"n"(kSimtStages - 2) : "memory"); }

// Dynamic shared memory: q rows [kSimtWarps][D], then kSimtStages stages of {K chunk, V chunk}, each [32][D + pad].
__host__ __device__ inline size_t simt_smem_bytes(int D) {
    return sizeof(float) * ((size_t)kSimtWarps * D + (size_t)kSimtStages * 2u * kSimtChunk * (D + kSimtPad));
}

template <int kT>   // 32-column groups of the head dimension: 32 (kT - 1) < D <= 32 kT
__global__ void __launch_bounds__(kSimtWarps * 32)
attn_fwd_fp32_kernel(const AttnParams p) {
    extern __shared__ __align__(16) float simt_smem[];
    const int D = p.D, ld = D + kSimtPad;
    float* q_sm = simt_smem;                                   // [kSimtWarps][D]
    float* kv_sm = simt_smem + kSimtWarps * D;                 // [kSimtStages][K | V][32][ld]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (blockIdx.x == 0 && warp == 0 && (p.mask_flags & kMaskDocument))
        tc::check_offsets_warp(p.cu, p.num_docs, p.Sq, p.status_word);

    const int nrb = (p.Sq + kSimtWarps - 1) / kSimtWarps;      // row blocks per (batch, head)
    const int rb = blockIdx.x % nrb;
    const int bh = blockIdx.x / nrb;
    const int h = bh % p.Hq, b = bh / p.Hq;
    const int g = h / p.group;
    const int r0 = rb * kSimtWarps;
    const int i = r0 + warp;
    const bool row_ok = i < p.Sq;
    const int ic = row_ok ? i : p.Sq - 1;                      // rows past Sq follow the last row and store nothing

    const float* kbase = (const float*)p.k + (long long)b * p.ks[0] + (long long)g * p.ks[1];
    const float* vbase = (const float*)p.v + (long long)b * p.vs[0] + (long long)g * p.vs[1];
    {
        const float* qrow = (const float*)p.q + (long long)b * p.qs[0] + (long long)h * p.qs[1] + (long long)ic * p.qs[2];
        for (int d = lane; d < D; d += 32) q_sm[warp * D + d] = qrow[d];
    }

    const RowInterval iv = row_interval(p, ic);
    const int ip = ic + p.Sk - p.Sq;
    const float slope = p.slopes ? __ldg(p.slopes + h) : 0.f;
    const bool softmax = (p.normalizer == kNormSoftmax);

    // The CTA's chunks: those of the global tokens [0, pre_max) (Appendix A.2, Global Sliding Window and Share
    // Question mask) and those of [lo_min, hi_max]; one run of chunks when the two meet, so that no chunk comes
    // twice.  Every warp computes the same bounds.
    const TileBounds tb = tile_bounds(p, r0, kSimtWarps);
    int first_chunk[2] = {0, 0}, n_chunks[2] = {0, 0};
    if (tb.pre_max > 0) n_chunks[0] = (tb.pre_max - 1) / kSimtChunk + 1;
    if (tb.hi_max >= 0 && tb.lo_min <= tb.hi_max) {
        first_chunk[1] = tb.lo_min / kSimtChunk;
        n_chunks[1] = tb.hi_max / kSimtChunk - first_chunk[1] + 1;
        if (first_chunk[1] <= n_chunks[0]) {                   // the runs meet or overlap
            n_chunks[1] = max(first_chunk[1] + n_chunks[1], n_chunks[0]);
            first_chunk[1] = 0;
            n_chunks[0] = 0;
        }
    }
    const int total_chunks = n_chunks[0] + n_chunks[1];
    auto chunk_key0 = [&](int c) { return (c < n_chunks[0] ? c : first_chunk[1] + (c - n_chunks[0])) * kSimtChunk; };

    // Cooperative copy of one K / V chunk; rows past Sk are zero-filled (they get the weight 0, which must not meet
    // stale non-finite bits).
    const int f4_per_row = D / 4;
    auto load_chunk = [&](int c) {
        if (c >= total_chunks) { cp_async_commit(); return; }   // an empty group keeps the group count in step
        const int j0 = chunk_key0(c);
        float* ks = kv_sm + (size_t)(c % kSimtStages) * 2 * kSimtChunk * ld;
        float* vs = ks + kSimtChunk * ld;
        for (int idx = threadIdx.x; idx < kSimtChunk * f4_per_row; idx += kSimtWarps * 32) {
            const int r = idx / f4_per_row, c4 = idx - r * f4_per_row;
            const int j = j0 + r;
            if (j < p.Sk) {
                cp_async16(ks + r * ld + c4 * 4, kbase + (long long)j * p.ks[2] + c4 * 4);
                cp_async16(vs + r * ld + c4 * 4, vbase + (long long)j * p.vs[2] + c4 * 4);
            } else {
                *reinterpret_cast<float4*>(ks + r * ld + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4*>(vs + r * ld + c4 * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        cp_async_commit();
    };

    float acc[kT];
#pragma unroll
    for (int t = 0; t < kT; ++t) acc[t] = 0.f;
    float m = -INFINITY, l = 0.f;

#pragma unroll
    for (int c = 0; c < kSimtStages - 1; ++c) load_chunk(c);
    for (int c = 0; c < total_chunks; ++c) {
        cp_async_wait_oldest();
        __syncthreads();                                       // chunk c has landed; everyone is done with chunk c - 1
        load_chunk(c + kSimtStages - 1);                       // into the stage that chunk c - 1 used

        const int j0 = chunk_key0(c);
        const float* ks = kv_sm + (size_t)(c % kSimtStages) * 2 * kSimtChunk * ld;
        const float* vs = ks + kSimtChunk * ld;
        const int j = j0 + lane;
        const bool valid = (j < iv.pre) || (j >= iv.lo && j <= iv.hi);
        const unsigned vis = __ballot_sync(0xffffffffu, valid);
        if (vis == 0u) continue;                               // nothing of this chunk is visible to this row

        // Score of key j0 + lane: four independent partial sums over the head dimension.
        float s;
        {
            const float4* kr = (const float4*)(ks + lane * ld);
            const float4* q4 = (const float4*)(q_sm + warp * D);
            float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
            for (int d4 = 0; d4 < 8 * kT; ++d4) {
                if (d4 < f4_per_row) {
                    const float4 kk = kr[d4];
                    const float4 qq = q4[d4];
                    d0 = fmaf(qq.x, kk.x, d0);
                    d1 = fmaf(qq.y, kk.y, d1);
                    d2 = fmaf(qq.z, kk.z, d2);
                    d3 = fmaf(qq.w, kk.w, d3);
                }
            }
            s = ((d0 + d1) + (d2 + d3)) * p.scale;
            if (p.softcap > 0.f) s = p.softcap * tanhf(s / p.softcap);
            s = fmaf(slope, (float)(ip - j), s);
            if (!valid) s = -INFINITY;
        }
        float pj;
        if (softmax) {
            const float m_new = fmaxf(m, warp_max(s));          // finite: the chunk holds a visible key
            const float alpha = (m == -INFINITY) ? 0.f : expf(m - m_new);
            pj = valid ? expf(s - m_new) : 0.f;
            l = l * alpha + warp_sum(pj);
#pragma unroll
            for (int t = 0; t < kT; ++t) acc[t] *= alpha;
            m = m_new;
        } else if (p.normalizer == kNormSigmoid) {
            pj = valid ? p.out_scale / (1.f + expf(-(s + p.sigmoid_bias))) : 0.f;
        } else {                                                // ReLU (Appendix A.3)
            pj = valid ? p.out_scale * fmaxf(s, 0.f) : 0.f;
        }
        // O += p_j V_j for all 32 keys of the chunk (weight 0 for the invisible ones).
#pragma unroll
        for (int jj = 0; jj < kSimtChunk; ++jj) {
            const float pb = __shfl_sync(0xffffffffu, pj, jj);
            const float* vr = vs + jj * ld;
#pragma unroll
            for (int t = 0; t < kT; ++t) {
                const int d = lane + 32 * t;
                if (t < kT - 1 || d < D) acc[t] = fmaf(pb, vr[d], acc[t]);
            }
        }
    }

    if (!row_ok) return;
    float* orow = (float*)p.o + (long long)b * p.os[0] + (long long)h * p.os[1] + (long long)i * p.os[2];
    const float inv = softmax ? (l > 0.f ? 1.f / l : 0.f) : 1.f;
#pragma unroll
    for (int t = 0; t < kT; ++t) {
        const int d = lane + 32 * t;
        if (d < D) orow[d] = acc[t] * inv;
    }
    if (softmax && p.lse && lane == 0)
        p.lse[((long long)b * p.Hq + h) * p.Sq + i] = (l > 0.f) ? m + logf(l) : -INFINITY;
}

namespace {

template <int kT>
cudaError_t launch_t(const AttnParams& p, unsigned blocks, cudaStream_t stream) {
    // The opt-in shared-memory size is a per-device function attribute: set it once per device.
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(attn_fwd_fp32_kernel<kT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)simt_smem_bytes(32 * kT));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    attn_fwd_fp32_kernel<kT><<<blocks, kSimtWarps * 32, simt_smem_bytes(p.D), stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_fwd_fp32(const AttnParams& p, cudaStream_t stream) {
    const long long nrb = (p.Sq + kSimtWarps - 1) / kSimtWarps;
    const long long blocks = nrb * p.B * p.Hq;
    if (blocks > 0x7fffffffLL || p.D < 1 || p.D > kSimtMaxD) return cudaErrorInvalidConfiguration;
    switch ((p.D + 31) / 32) {
        case 1: return launch_t<1>(p, (unsigned)blocks, stream);
        case 2: return launch_t<2>(p, (unsigned)blocks, stream);
        case 3: return launch_t<3>(p, (unsigned)blocks, stream);
        case 4: return launch_t<4>(p, (unsigned)blocks, stream);
        case 5: return launch_t<5>(p, (unsigned)blocks, stream);
        case 6: return launch_t<6>(p, (unsigned)blocks, stream);
        case 7: return launch_t<7>(p, (unsigned)blocks, stream);
        default: return launch_t<8>(p, (unsigned)blocks, stream);
    }
}

}  // namespace b200attn
