// Host side of the C ABI declared in include/attn.h: argument validation, parameter block, kernel selection,
// and the cache of encoded TMA tensor maps.  Nothing here computes; every step of the path runs in the kernels
// of attn_simt_fp32.cu (fp32 inputs) and attn_tc_pingpong*.cu / attn_tc_pair.cu / attn_tc_split.cu (bf16 inputs,
// tcgen05).
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "../../include/attn.h"
#include "attn_params.cuh"
#include "attn_tc_common.cuh"

namespace b200attn {
cudaError_t launch_attn_fwd_fp32(const AttnParams& p, cudaStream_t stream);
// Returns ATTN_OK, ATTN_ERR_UNSUPPORTED or ATTN_ERR_CUDA; *launches receives the number of
// kernels enqueued.
int launch_attn_fwd_bf16(const AttnParams& p, cudaStream_t stream, int* launches);
}  // namespace b200attn

namespace b200attn {
namespace tc {

// Encoded tensor maps are pure functions of (address, shape, strides, box): they are kept in a small direct-mapped
// table so that a call on tensors seen before skips the driver's encoder.  One mutex guards the table; an entry is
// never stale (the same key always encodes to the same 128 bytes), attn_clear_cache() merely empties it.
namespace {
constexpr int kMapCacheSlots = 256;
struct MapSlot { bool used; MapKey key; CUtensorMap map; };
MapSlot g_map_cache[kMapCacheSlots];
std::mutex g_map_mutex;
std::atomic<long long> g_map_hits{0};

bool same_key(const MapKey& a, const MapKey& b) {
    return a.ptr == b.ptr && a.B == b.B && a.H == b.H && a.S == b.S && a.D == b.D && a.st[0] == b.st[0] &&
           a.st[1] == b.st[1] && a.st[2] == b.st[2] && a.box_rows == b.box_rows && a.box_cols == b.box_cols &&
           a.swizzle_bytes == b.swizzle_bytes;
}
size_t slot_of(const MapKey& k) {
    uint64_t h = reinterpret_cast<uintptr_t>(k.ptr) * 0x9E3779B97F4A7C15ull;
    h ^= ((uint64_t)k.S << 32) ^ ((uint64_t)k.H << 16) ^ ((uint64_t)k.B << 8) ^ (uint64_t)k.D ^ ((uint64_t)k.box_rows << 48) ^
         ((uint64_t)k.box_cols << 56) ^ ((uint64_t)k.st[2] * 0xC2B2AE3D27D4EB4Full);
    return (size_t)((h >> 29) % kMapCacheSlots);
}
}  // namespace

bool cached_map(CUtensorMap* out, const MapKey& key) {
    MapSlot& slot = g_map_cache[slot_of(key)];
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        if (slot.used && same_key(slot.key, key)) {
            *out = slot.map;
            g_map_hits.fetch_add(1, std::memory_order_relaxed);
            return true;
        }
    }
    if (!encode_map(out, key)) return false;
    std::lock_guard<std::mutex> lock(g_map_mutex);
    slot.used = true;
    slot.key = key;
    slot.map = *out;
    return true;
}

void clear_map_cache() {
    std::lock_guard<std::mutex> lock(g_map_mutex);
    for (MapSlot& s : g_map_cache) s.used = false;
}

long long map_cache_hits() { return g_map_hits.load(std::memory_order_relaxed); }

}  // namespace tc
}  // namespace b200attn

namespace {

std::atomic<long long> g_launches{0};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Fills element strides (batch, head, row); all-zero input means contiguous [B,H,S,D].
// Returns false if a given stride set is not usable.
bool resolve_strides(const int64_t in[3], long long out[3], int H, int S, int D, size_t elem) {
    if (in[0] == 0 && in[1] == 0 && in[2] == 0) {
        out[2] = D;
        out[1] = (long long)S * D;
        out[0] = (long long)H * S * D;
        return true;
    }
    for (int a = 0; a < 3; ++a) {
        if (in[a] <= 0) return false;
        out[a] = in[a];
    }
    if (out[2] < D) return false;
    for (int a = 0; a < 3; ++a)
        if ((out[a] * (long long)elem) % 16 != 0) return false;
    return true;
}


// Every argument check of attn_fwd, made before any CUDA call; fills the kernels' parameter block.
int check_and_fill(const void* q, const void* k, const void* v, void* o, float* lse,
                   int B, int Hq, int Hkv, int Sq, int Sk, int D,
                   const attn_variant_desc* desc, b200attn::AttnParams* out) {
    using namespace b200attn;
    if (!q || !k || !v || !o || !desc) return ATTN_ERR_NULL;
    if (desc->struct_size != sizeof(attn_variant_desc)) return ATTN_ERR_DESC;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return ATTN_ERR_SHAPE;
    if (Hq % Hkv != 0) return ATTN_ERR_SHAPE;
    if (desc->dtype != ATTN_BF16 && desc->dtype != ATTN_FP32) return ATTN_ERR_DESC;
    if (desc->o_dtype != ATTN_BF16 && desc->o_dtype != ATTN_FP32) return ATTN_ERR_DESC;
    if (desc->normalizer > ATTN_NORM_RELU) return ATTN_ERR_DESC;
    if (desc->mask_flags & ~(ATTN_MASK_CAUSAL | ATTN_MASK_WINDOW | ATTN_MASK_DOCUMENT | ATTN_MASK_PREFIX |
                             ATTN_MASK_TEST_QUERY | ATTN_MASK_GLOBAL))
        return ATTN_ERR_DESC;
    if ((desc->mask_flags & ATTN_MASK_GLOBAL) && desc->global_len < 0) return ATTN_ERR_DESC;
    if ((desc->mask_flags & ATTN_MASK_PREFIX) && (!(desc->mask_flags & ATTN_MASK_CAUSAL) || desc->prefix_len < 0))
        return ATTN_ERR_DESC;
    if ((desc->mask_flags & ATTN_MASK_TEST_QUERY) &&
        (!(desc->mask_flags & ATTN_MASK_DOCUMENT) || desc->test_query_start < 0))
        return ATTN_ERR_DESC;
    if (!(desc->scale >= 0.f) || !std::isfinite(desc->scale)) return ATTN_ERR_DESC;
    if (!(desc->softcap >= 0.f) || !std::isfinite(desc->softcap)) return ATTN_ERR_DESC;
    if (!std::isfinite(desc->sigmoid_bias) || !std::isfinite(desc->out_scale)) return ATTN_ERR_DESC;
    if (desc->mask_flags & ATTN_MASK_DOCUMENT) {
        if (!desc->cu_seqlens || desc->num_docs <= 0) return ATTN_ERR_DESC;
        if (B != 1 || Sq != Sk) return ATTN_ERR_SHAPE;
    }
    if (desc->dtype == ATTN_FP32) {
        if (desc->o_dtype != ATTN_FP32) return ATTN_ERR_UNSUPPORTED;
        if (D > 256 || D % 4 != 0) return ATTN_ERR_UNSUPPORTED;
    } else {
        if (D != 64 && D != 128 && D != 256) return ATTN_ERR_UNSUPPORTED;
    }
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return ATTN_ERR_ALIGN;
    if ((desc->bias_slopes && (reinterpret_cast<uintptr_t>(desc->bias_slopes) & 3u)) ||
        (desc->cu_seqlens && (reinterpret_cast<uintptr_t>(desc->cu_seqlens) & 3u)) ||
        (desc->status_word && (reinterpret_cast<uintptr_t>(desc->status_word) & 3u)) ||
        (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)))
        return ATTN_ERR_ALIGN;

    AttnParams p;
    std::memset(&p, 0, sizeof(p));
    const size_t in_elem = desc->dtype == ATTN_FP32 ? 4 : 2;
    const size_t out_elem = desc->o_dtype == ATTN_FP32 ? 4 : 2;
    if (!resolve_strides(desc->q_strides, p.qs, Hq, Sq, D, in_elem) ||
        !resolve_strides(desc->k_strides, p.ks, Hkv, Sk, D, in_elem) ||
        !resolve_strides(desc->v_strides, p.vs, Hkv, Sk, D, in_elem) ||
        !resolve_strides(desc->o_strides, p.os, Hq, Sq, D, out_elem))
        return ATTN_ERR_ALIGN;
    p.q = q; p.k = k; p.v = v; p.o = o; p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Sk = Sk; p.D = D;
    p.group = Hq / Hkv;
    p.scale = desc->scale > 0.f ? desc->scale : (float)(1.0 / std::sqrt((double)D));
    p.softcap = desc->softcap;
    p.slopes = desc->bias_slopes;
    p.sigmoid_bias = desc->sigmoid_bias;
    p.out_scale = desc->out_scale != 0.f ? desc->out_scale : 1.f;
    p.mask_flags = desc->mask_flags;
    // Window widths beyond the problem size behave as unbounded; clamping keeps i' +/- w in int range.
    const int wmax = Sq + Sk;
    p.window_left = desc->window_left < 0 ? -1 : (desc->window_left > wmax ? wmax : desc->window_left);
    p.window_right = desc->window_right < 0 ? -1 : (desc->window_right > wmax ? wmax : desc->window_right);
    p.cu = desc->cu_seqlens;
    p.num_docs = desc->num_docs;
    // Outside their flags the two relaxations are neutral: no prefix, test query beyond the last row.
    p.prefix_len = (desc->mask_flags & ATTN_MASK_PREFIX) ? (desc->prefix_len > Sk ? Sk : desc->prefix_len) : 0;
    p.test_query_start = (desc->mask_flags & ATTN_MASK_TEST_QUERY) ? (desc->test_query_start > Sq ? Sq : desc->test_query_start) : Sq;
    p.global_len = (desc->mask_flags & ATTN_MASK_GLOBAL) ? (desc->global_len > Sk ? Sk : desc->global_len) : 0;
    p.normalizer = (int)desc->normalizer;
    p.o_fp32 = desc->o_dtype == ATTN_FP32;
    p.status_word = desc->status_word;
    *out = p;
    return ATTN_OK;
}


// Kernel selection and launch for a checked parameter block.
int launch_checked(const b200attn::AttnParams& p, uint32_t dtype, cudaStream_t st) {
    using namespace b200attn;
    if (dtype == ATTN_FP32) {
        if (launch_attn_fwd_fp32(p, st) != cudaSuccess) return ATTN_ERR_CUDA;
        g_launches.fetch_add(1);
        return ATTN_OK;
    }
    int launches = 0;
    const int rc = launch_attn_fwd_bf16(p, st, &launches);
    g_launches.fetch_add(launches);
    return rc;
}

}  // namespace

extern "C" {

const char* attn_status_string(int status) {
    switch (status) {
        case ATTN_OK: return "ok";
        case ATTN_ERR_NULL: return "a required pointer is NULL";
        case ATTN_ERR_SHAPE: return "invalid shape";
        case ATTN_ERR_UNSUPPORTED: return "unsupported dtype, head dimension or combination";
        case ATTN_ERR_ALIGN: return "pointer or stride is not 16-byte aligned";
        case ATTN_ERR_DESC: return "malformed variant descriptor";
        case ATTN_ERR_CUDA: return "a CUDA call failed";
        case ATTN_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

int attn_version(void) { return 100; }

int64_t attn_launch_count(void) { return g_launches.load(); }

int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int Hq, int Hkv, int Sq, int Sk, int D,
             const attn_variant_desc* desc, void* stream) {
    b200attn::AttnParams p;
    if (const int rc = check_and_fill(q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, desc, &p)) return rc;
    return launch_checked(p, desc->dtype, reinterpret_cast<cudaStream_t>(stream));
}

int attn_clear_cache(void) {
    b200attn::tc::clear_map_cache();
    return ATTN_OK;
}

int64_t attn_cache_hits(void) { return b200attn::tc::map_cache_hits(); }

namespace {
size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }
struct HostLayout { size_t q, k, v, o, lse, total, qb, kvb, ob, lseb; };
bool host_layout(int B, int Hq, int Hkv, int Sq, int Sk, int D, const attn_variant_desc* desc, HostLayout* L) {
    if (!desc || B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return false;
    const size_t ein = desc->dtype == ATTN_FP32 ? 4 : 2, eout = desc->o_dtype == ATTN_FP32 ? 4 : 2;
    L->qb = (size_t)B * Hq * Sq * D * ein;
    L->kvb = (size_t)B * Hkv * Sk * D * ein;
    L->ob = (size_t)B * Hq * Sq * D * eout;
    L->lseb = (size_t)B * Hq * Sq * 4;
    L->q = 0;
    L->k = L->q + round256(L->qb);
    L->v = L->k + round256(L->kvb);
    L->o = L->v + round256(L->kvb);
    L->lse = L->o + round256(L->ob);
    L->total = L->lse + round256(L->lseb);
    return true;
}
}  // namespace

size_t attn_host_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, const attn_variant_desc* desc) {
    HostLayout L;
    return host_layout(B, Hq, Hkv, Sq, Sk, D, desc, &L) ? L.total : 0;
}

int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host,
                  int B, int Hq, int Hkv, int Sq, int Sk, int D,
                  const attn_variant_desc* desc, void* workspace, size_t workspace_bytes, void* stream) {
    if (!q_host || !k_host || !v_host || !o_host || !desc || !workspace) return ATTN_ERR_NULL;
    if (desc->struct_size != sizeof(attn_variant_desc)) return ATTN_ERR_DESC;
    for (int a = 0; a < 3; ++a)
        if (desc->q_strides[a] || desc->k_strides[a] || desc->v_strides[a] || desc->o_strides[a]) return ATTN_ERR_DESC;
    HostLayout L;
    if (!host_layout(B, Hq, Hkv, Sq, Sk, D, desc, &L)) return ATTN_ERR_SHAPE;
    if (workspace_bytes < L.total) return ATTN_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ATTN_ERR_ALIGN;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const bool want_lse = lse_host && desc->normalizer == ATTN_NORM_SOFTMAX;
    // Every argument check runs before the first copy is enqueued: on an argument error nothing reaches the stream.
    b200attn::AttnParams p;
    if (const int rc = check_and_fill(ws + L.q, ws + L.k, ws + L.v, ws + L.o, want_lse ? reinterpret_cast<float*>(ws + L.lse) : nullptr,
                                      B, Hq, Hkv, Sq, Sk, D, desc, &p))
        return rc;
    if (cudaMemcpyAsync(ws + L.q, q_host, L.qb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ws + L.k, k_host, L.kvb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ws + L.v, v_host, L.kvb, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return ATTN_ERR_CUDA;
    const int rc = launch_checked(p, desc->dtype, st);
    if (rc != ATTN_OK) return rc;
    if (cudaMemcpyAsync(o_host, ws + L.o, L.ob, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ATTN_ERR_CUDA;
    if (want_lse && cudaMemcpyAsync(lse_host, ws + L.lse, L.lseb, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ATTN_ERR_CUDA;
    return ATTN_OK;
}

}  // extern "C"
