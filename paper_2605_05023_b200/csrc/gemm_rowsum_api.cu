// C ABI of the GEMM + row-sum operator (include/gemm_rowsum.h): argument validation, which runs before any
// CUDA call, then the launch.  No CPU path: without a GPU the CUDA calls fail and the status says so.
#include <atomic>
#include <cstdint>

#include "../../include/attn.h"
#include "../../include/gemm_rowsum.h"
#include "gemm_rowsum_params.cuh"

namespace {

std::atomic<int64_t> g_gemm_launches{0};

struct HostLayout {
    size_t a, b, c, r, total, ab, bb, cb, rb;
};

bool host_layout(int M, int N, int K, HostLayout* L) {
    if (M <= 0 || N <= 0 || K <= 0) return false;
    auto up = [](size_t x) { return (x + 255u) & ~(size_t)255u; };
    L->ab = (size_t)M * K * 2;
    L->bb = (size_t)K * N * 2;
    L->cb = (size_t)M * N * 2;
    L->rb = (size_t)M * 4;
    L->a = 0;
    L->b = L->a + up(L->ab);
    L->c = L->b + up(L->bb);
    L->r = L->c + up(L->cb);
    L->total = L->r + up(L->rb);
    return true;
}

// Every argument check of gemm_rowsum, made before any CUDA call; fills the launch parameters.
int check_and_fill(const void* a, const void* b, void* c, float* rowsum, int M, int N, int K,
                   const gemm_rowsum_desc* desc, b200attn::GemmRowsumParams* out) {
    if (!a || !b || !rowsum) return ATTN_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0) return ATTN_ERR_SHAPE;
    if (desc && (desc->struct_size != sizeof(gemm_rowsum_desc) || desc->reserved != 0)) return ATTN_ERR_DESC;
    b200attn::GemmRowsumParams p = {};
    p.a = a; p.b = b; p.c = c; p.rowsum = rowsum;
    p.M = M; p.N = N; p.K = K;
    p.lda = (desc && desc->lda) ? desc->lda : K;
    p.ldb = (desc && desc->ldb) ? desc->ldb : N;
    p.ldc = (desc && desc->ldc) ? desc->ldc : N;
    p.status_word = desc ? desc->status_word : nullptr;
    if (p.lda < K || p.ldb < N || p.ldc < N) return ATTN_ERR_SHAPE;
    // TMA and the 16-byte stores: 16-byte aligned bases, row strides that are multiples of 16 bytes, and N a
    // multiple of 8 so that a row of C ends on a 16-byte boundary.
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b) | reinterpret_cast<uintptr_t>(c)) & 15u) return ATTN_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(rowsum) & 3u) return ATTN_ERR_ALIGN;
    if ((p.lda | p.ldb | p.ldc) & 7 || (N & 7)) return ATTN_ERR_ALIGN;
    *out = p;
    return ATTN_OK;
}

}  // namespace

extern "C" {

int gemm_rowsum(const void* a, const void* b, void* c, float* rowsum, int M, int N, int K,
                const gemm_rowsum_desc* desc, void* stream) {
    b200attn::GemmRowsumParams p;
    if (const int rc = check_and_fill(a, b, c, rowsum, M, N, K, desc, &p)) return rc;
    const int rc = b200attn::launch_gemm_rowsum_bf16(p, reinterpret_cast<cudaStream_t>(stream));
    if (rc == ATTN_OK) g_gemm_launches.fetch_add(1, std::memory_order_relaxed);
    return rc;
}

size_t gemm_rowsum_host_workspace_bytes(int M, int N, int K) {
    HostLayout L;
    return host_layout(M, N, K, &L) ? L.total : 0;
}

int gemm_rowsum_host(const void* a_host, const void* b_host, void* c_host, float* rowsum_host, int M, int N, int K,
                     const gemm_rowsum_desc* desc, void* workspace, size_t workspace_bytes, void* stream) {
    if (!a_host || !b_host || !rowsum_host || !workspace) return ATTN_ERR_NULL;
    if (desc && (desc->struct_size != sizeof(gemm_rowsum_desc) || desc->reserved != 0)) return ATTN_ERR_DESC;
    if (desc && (desc->lda || desc->ldb || desc->ldc)) return ATTN_ERR_DESC;
    HostLayout L;
    if (!host_layout(M, N, K, &L)) return ATTN_ERR_SHAPE;
    if (workspace_bytes < L.total) return ATTN_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return ATTN_ERR_ALIGN;
    char* ws = static_cast<char*>(workspace);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // Every argument check runs before the first copy is enqueued: on an argument error nothing reaches the stream.
    b200attn::GemmRowsumParams p;
    if (const int rc = check_and_fill(ws + L.a, ws + L.b, c_host ? ws + L.c : nullptr, reinterpret_cast<float*>(ws + L.r), M, N, K,
                                      desc, &p))
        return rc;
    if (cudaMemcpyAsync(ws + L.a, a_host, L.ab, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ws + L.b, b_host, L.bb, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return ATTN_ERR_CUDA;
    const int rc = b200attn::launch_gemm_rowsum_bf16(p, st);
    if (rc != ATTN_OK) return rc;
    g_gemm_launches.fetch_add(1, std::memory_order_relaxed);
    if (c_host && cudaMemcpyAsync(c_host, ws + L.c, L.cb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ATTN_ERR_CUDA;
    if (cudaMemcpyAsync(rowsum_host, ws + L.r, L.rb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return ATTN_ERR_CUDA;
    return ATTN_OK;
}

int64_t gemm_rowsum_launch_count(void) { return g_gemm_launches.load(std::memory_order_relaxed); }

}  // extern "C"
