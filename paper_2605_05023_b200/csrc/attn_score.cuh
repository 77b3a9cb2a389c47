// Score modifier of Appendix A.1 on 32 score columns held in registers, shared by the tensor-core kernels:
//   softcap   s -> C * tanh(scale * s / C)      (then, in log2 units, times log2 e)
//   bias      s -> s + slope_h * (i' - j)
// Everything is produced in log2 units (scores are later fed to ex2).
#pragma once
#include "sm100_ptx.cuh"

namespace b200attn {

struct ScoreConsts {
    float cs;          // scale * log2(e): raw score -> log2 units (no softcap)
    float slope2;      // slope_h * log2(e), 0 when the head has no bias
    float cap_in;      // scale / C   (0 when softcap is off)
    float cap_out;     // C * log2(e)
    float k0, k1, k2, k3;   // C*log2(e) * tanh(c s) ~= s * (k0 + k1 z + k2 z^2 + k3 z^3), z = s^2, c = cap_in, |c s| <= 0.5
    float z_limit;     // the polynomial holds while s^2 <= z_limit = (0.5 / cap_in)^2
    float l0, l1;      // the same with a + b z, for |c s| <= 0.2 (relative error 3e-5)
    float zl_limit;    // (0.2 / cap_in)^2
    bool softcap, has_bias;
};

// Coefficients of the softcap polynomial as register pairs.  identity: {1, 0, 0, 0}, which makes the polynomial
// step return its input unchanged (second pass over a tile whose scores were capped exactly, see score_chunk32_tile).
struct CapPoly {
    uint64_t k0, k1, k2, k3;
};
__device__ __forceinline__ CapPoly cap_poly(const ScoreConsts& sc, bool identity) {
    CapPoly k;
    k.k0 = identity ? ptx::pack2(1.0f, 1.0f) : ptx::pack2(sc.k0, sc.k0);
    k.k1 = identity ? 0ull : ptx::pack2(sc.k1, sc.k1);
    k.k2 = identity ? 0ull : ptx::pack2(sc.k2, sc.k2);
    k.k3 = identity ? 0ull : ptx::pack2(sc.k3, sc.k3);
    return k;
}

// tanh(x) / x on |x| <= 0.5 as a cubic in x^2 (minimax, relative error 5.4e-7), with the input and output scales
// folded into the coefficients.
__device__ __forceinline__ ScoreConsts make_score_consts(float scale, float softcap, float slope) {
    constexpr float kL2e = 1.4426950408889634f;
    ScoreConsts sc;
    sc.cs = scale * kL2e;
    sc.slope2 = slope * kL2e;
    sc.has_bias = slope != 0.f;
    sc.softcap = softcap > 0.f;
    sc.cap_in = sc.softcap ? scale / softcap : 0.f;
    sc.cap_out = softcap * kL2e;
    const float c = sc.cap_in, c2 = c * c, a = sc.cap_out * c;
    sc.k0 = a * 0.9999994557706542f;
    sc.k1 = a * c2 * -0.3332631793391532f;
    sc.k2 = a * c2 * c2 * 0.13190296581692276f;
    sc.k3 = a * c2 * c2 * c2 * -0.04440222555537668f;
    sc.z_limit = sc.softcap ? 0.25f / c2 : INFINITY;
    sc.l0 = a * 0.9999733f;
    sc.l1 = a * c2 * -0.3280f;
    sc.zl_limit = sc.softcap ? 0.04f / c2 : INFINITY;
    return sc;
}

// tanh for any x through the exponential (two MUFU operations).
__device__ __forceinline__ float tanh_by_exp(float x) {
    const float e = ptx::ex2_approx(fabsf(x) * (2.0f * 1.4426950408889634f));   // e^{2|x|}
    const float t = 1.0f - 2.0f * ptx::rcp_approx(1.0f + e);
    return copysignf(t, x);
}

// y[0..32): raw scores in, modified scores (log2 units) out.  rowoff = i' - (key index of column 0 of the chunk).
// The polynomial tanh holds while |scale * s / C| <= 0.5 for every score of the warp's chunk; otherwise the whole
// warp takes the exponential form for this chunk (warp-uniform choice, rare on ordinary data).
// Must be called by all 32 lanes of the warp.  Each case is its own straight-line loop so that the 16 pairs
// of a chunk can be interleaved by the scheduler.
// kMaySoftcap = false compiles the softcap branch out (the bias-only kernel instances).
template <bool kMaySoftcap>
__device__ __forceinline__ void score_chunk32(uint32_t* y, const ScoreConsts& sc, float rowoff) {
    if (kMaySoftcap && sc.softcap) {
        float ax = 0.f;
#pragma unroll
        for (int i = 0; i < 32; i += 2) ax = ptx::max3(ax, fabsf(__uint_as_float(y[i])), fabsf(__uint_as_float(y[i + 1])));
        if (__any_sync(0xffffffffu, ax * sc.cap_in > 0.5f)) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                y[i] = __float_as_uint(sc.cap_out * tanh_by_exp(__uint_as_float(y[i]) * sc.cap_in));
        } else {
            const uint64_t k0 = ptx::pack2(sc.k0, sc.k0), k1 = ptx::pack2(sc.k1, sc.k1), k2 = ptx::pack2(sc.k2, sc.k2),
                           k3 = ptx::pack2(sc.k3, sc.k3);
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const uint64_t s2 = ptx::pack2(__uint_as_float(y[i]), __uint_as_float(y[i + 1]));
                const uint64_t z = ptx::mul2(s2, s2);
                uint64_t r = ptx::fma2(k3, z, k2);
                r = ptx::fma2(r, z, k1);
                r = ptx::fma2(r, z, k0);
                float s0, s1;
                ptx::unpack2(ptx::mul2(r, s2), s0, s1);
                y[i] = __float_as_uint(s0);
                y[i + 1] = __float_as_uint(s1);
            }
        }
        if (sc.has_bias) {
#pragma unroll
            for (int i = 0; i < 32; ++i)      // + slope * (i' - j): the distance is formed exactly, then scaled
                y[i] = __float_as_uint(fmaf(sc.slope2, rowoff - (float)i, __uint_as_float(y[i])));
        }
    } else if (!kMaySoftcap || sc.has_bias) {     // the bias-only instances always carry slopes
        const uint64_t cs2 = ptx::pack2(sc.cs, sc.cs), slope22 = ptx::pack2(sc.slope2, sc.slope2);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const uint64_t s2 = ptx::pack2(__uint_as_float(y[i]), __uint_as_float(y[i + 1]));
            const uint64_t dist = ptx::pack2(rowoff - (float)i, rowoff - (float)(i + 1));
            float s0, s1;
            ptx::unpack2(ptx::fma2(slope22, dist, ptx::mul2(s2, cs2)), s0, s1);
            y[i] = __float_as_uint(s0);
            y[i + 1] = __float_as_uint(s1);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = __float_as_uint(__uint_as_float(y[i]) * sc.cs);
    }
}

// ---- The softmax instances take the rare exponential form out of their key loop -------------------------------
// (With the per-chunk choice above, the four unrolled copies of the exponential form sit inside the loop body and
// every chunk ends in a warp vote: without them the softcap instances of the ping-pong kernel run 14 % faster.
// The sigmoid and ReLU instances are slower with this form and keep the one above.)
// A key tile is first capped with a + b s^2 (softcap_lin_chunk32: scores up to 0.2 of the cap); the largest
// s^2 of the warp's tile, collected on the way, decides once per tile whether that was enough; if not, the pass is
// repeated with the cubic in s^2 (up to half the cap) or on scores capped exactly.
//
// Softcap of large scores, exactly: the 32-lane x (32 * nchunks)-column block of raw scores at TMEM address taddr
// is replaced in place by C * log2(e) * tanh(scale * s / C).  Called by all 32 lanes of a warp.
static __device__ __noinline__ void softcap_exact_in_tmem(uint32_t taddr, int nchunks, float cap_in, float cap_out) {
#pragma unroll 1
    for (int c = 0; c < nchunks; ++c) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(taddr + c * 32, v);
        ptx::tmem_wait_ld_regs(v);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(cap_out * tanh_by_exp(__uint_as_float(v[i]) * cap_in));
        ptx::tmem_st_32x32(taddr + c * 32, v);
    }
    ptx::tmem_wait_st();
}

// The pieces of the softcap score on one chunk.  Polynomial with the item's own coefficients; zmax collects the
// largest s^2 seen (the caller compares it with sc.z_limit once per tile and caps exactly where it is exceeded).
__device__ __forceinline__ void softcap_poly_chunk32(uint32_t* y, const ScoreConsts& sc, float& zmax) {
    const uint64_t k0 = ptx::pack2(sc.k0, sc.k0), k1 = ptx::pack2(sc.k1, sc.k1), k2 = ptx::pack2(sc.k2, sc.k2),
                   k3 = ptx::pack2(sc.k3, sc.k3);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const uint64_t s2 = ptx::pack2(__uint_as_float(y[i]), __uint_as_float(y[i + 1]));
        const uint64_t z = ptx::mul2(s2, s2);
        float z0, z1;
        ptx::unpack2(z, z0, z1);
        zmax = ptx::max3(zmax, z0, z1);
        uint64_t r = ptx::fma2(k3, z, k2);
        r = ptx::fma2(r, z, k1);
        r = ptx::fma2(r, z, k0);
        float s0, s1;
        ptx::unpack2(ptx::mul2(r, s2), s0, s1);
        y[i] = __float_as_uint(s0);
        y[i + 1] = __float_as_uint(s1);
    }
}
// tanh(x) / x as a + b x^2, for the common case of scores well inside the cap: two FMAs less per pair of scores than
// the cubic, for |x| <= 0.2 (economised from the series on x^2 in [0, 0.04]: relative error 3e-5, which is 3e-4 of a
// score unit at the edge of the range).
__device__ __forceinline__ void softcap_lin_chunk32(uint32_t* y, const ScoreConsts& sc, float& zmax) {
    const uint64_t l0 = ptx::pack2(sc.l0, sc.l0), l1 = ptx::pack2(sc.l1, sc.l1);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const uint64_t s2 = ptx::pack2(__uint_as_float(y[i]), __uint_as_float(y[i + 1]));
        const uint64_t z = ptx::mul2(s2, s2);
        float z0, z1;
        ptx::unpack2(z, z0, z1);
        zmax = ptx::max3(zmax, z0, z1);
        float s0, s1;
        ptx::unpack2(ptx::mul2(ptx::fma2(l1, z, l0), s2), s0, s1);
        y[i] = __float_as_uint(s0);
        y[i + 1] = __float_as_uint(s1);
    }
}
// Exponential form, any magnitude (raw scores in).
__device__ __forceinline__ void softcap_exact_chunk32(uint32_t* y, const ScoreConsts& sc) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = __float_as_uint(sc.cap_out * tanh_by_exp(__uint_as_float(y[i]) * sc.cap_in));
}
// + slope * (i' - j): the distance is formed exactly, then scaled.
__device__ __forceinline__ void bias_add_chunk32(uint32_t* y, const ScoreConsts& sc, float rowoff) {
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = __float_as_uint(fmaf(sc.slope2, rowoff - (float)i, __uint_as_float(y[i])));
}

// Softcap (always on in the instances that call this) and bias of one chunk, the softcap as a + b s^2; zmax as
// in softcap_lin_chunk32.  The first pass over a tile.
__device__ __forceinline__ void score_chunk32_lin(uint32_t* y, const ScoreConsts& sc, float rowoff, float& zmax) {
    softcap_lin_chunk32(y, sc, zmax);
    if (sc.has_bias) bias_add_chunk32(y, sc, rowoff);
}

// Softcap (always on in the instances that call this) and bias of one chunk, the softcap as the polynomial with the
// coefficients `poly`; zmax collects the largest s^2 seen, and the caller compares it with sc.z_limit once per tile:
// if any score of the warp's tile lies beyond, it has the tile capped exactly in TMEM (softcap_exact_in_tmem) and
// runs its pass again with the identity coefficients.
__device__ __forceinline__ void score_chunk32_tile(uint32_t* y, const ScoreConsts& sc, float rowoff, const CapPoly& poly, float& zmax) {
    {
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
            const uint64_t s2 = ptx::pack2(__uint_as_float(y[i]), __uint_as_float(y[i + 1]));
            const uint64_t z = ptx::mul2(s2, s2);
            float z0, z1;
            ptx::unpack2(z, z0, z1);
            zmax = ptx::max3(zmax, z0, z1);
            uint64_t r = ptx::fma2(poly.k3, z, poly.k2);
            r = ptx::fma2(r, z, poly.k1);
            r = ptx::fma2(r, z, poly.k0);
            float s0, s1;
            ptx::unpack2(ptx::mul2(r, s2), s0, s1);
            y[i] = __float_as_uint(s0);
            y[i + 1] = __float_as_uint(s1);
        }
        if (sc.has_bias) bias_add_chunk32(y, sc, rowoff);
    }
}

}  // namespace b200attn
