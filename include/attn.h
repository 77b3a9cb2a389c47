/*
 * attn.h -- C ABI of the B200 (sm_100a) fused attention-forward library.
 *
 * One call computes, for every batch b, query head h and query row i,
 *
 *     O[b,h,i,:] = sum_j  Norm( Mask( Score( scale * q_i . k_j ) ) )_ij * V[b,g,j,:]
 *
 * i.e. Eq. 2 of the CuBridge paper (Sec. 2.2; restated in Appendix A), of which Eq. 1
 * (softmax attention) is the special case with no score modifier and no mask:
 *   Score  (Appendix A.1)  softcap C*tanh(s/C), then a linear position bias
 *                          slope_h*(i' - j) (the paper's "relative position" variant is
 *                          slope = +1; ALiBi is slope_h = -m_h);
 *   Mask   (Appendix A.2)  causal clause j <= i', sliding-window clause
 *                          i' - window_left <= j <= i' + window_right, and the document
 *                          clause D_i = D_j of the causal blockwise mask, given as
 *                          cumulative offsets of packed documents.  Masks compose by AND;
 *                          a masked score is -inf and contributes nothing.  Three
 *                          relaxations give the paper's other masks: a PrefixLM prefix
 *                          (relaxes the causal clause), the test-query rows of the causal
 *                          blockwise mask (relax the document clause) and global tokens
 *                          (Global Sliding Window, Share Question mask; relax the window
 *                          and document clauses);
 *   Norm   (Eq. 1 / Appendix A.3)  row softmax, or out_scale*sigmoid(s + b) or
 *                          out_scale*max(s, 0) without row normalisation ((1/L)*Sigmoid(S)
 *                          is b = 0, out_scale = 1/L; (1/L)*ReLU(S) is out_scale = 1/L).
 * i' = i + (Sk - Sq) aligns the last query with the last key.  Query head h reads
 * key/value head g = h / (Hq / Hkv) (grouped-query attention).  Indices are 0-based.
 *
 * Fully masked key tiles are skipped and element-wise mask tests run only on tiles that
 * straddle a mask edge (the loop splitting of Sec. 3.4, "Performance-Aware
 * Transformation").
 *
 * Conventions
 *   - q, k, v, o, lse and every pointer inside the descriptor are DEVICE pointers owned by
 *     the caller; the descriptor itself is HOST memory, read during the call only.
 *   - The call enqueues work on `stream` and returns; it never synchronises, never prints
 *     and never aborts.  Device arrays must stay valid until the stream work is done.
 *   - Any failure is a non-zero attn_status return; every argument check runs before the first CUDA call, so an
 *     argument error leaves nothing on the stream (attn_fwd_host included: no copy is enqueued either).
 *   - Thread safety: every entry point may be called from several host threads at once, on the same or on
 *     different devices (the per-device set-up of the first call and the tensor-map cache are guarded); calls
 *     that share a stream are ordered by CUDA as usual.
 *   - Layout: q, o are [B, Hq, Sq, D]; k, v are [B, Hkv, Sk, D]; lse is [B, Hq, Sq] fp32,
 *     contiguous.  Strides (in elements, for batch / head / row) may be given in the
 *     descriptor; all-zero means contiguous.  The innermost dimension is always dense.
 */
#ifndef B200_ATTN_H_
#define B200_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum attn_status {
    ATTN_OK = 0,
    ATTN_ERR_NULL = 1,         /* a required pointer is NULL */
    ATTN_ERR_SHAPE = 2,        /* non-positive size, Hq % Hkv != 0, document mask with B != 1 or Sq != Sk */
    ATTN_ERR_UNSUPPORTED = 3,  /* dtype / head dimension / combination not built */
    ATTN_ERR_ALIGN = 4,        /* base pointer or stride not 16-byte aligned */
    ATTN_ERR_DESC = 5,         /* malformed descriptor (struct_size, enum values, missing arrays) */
    ATTN_ERR_CUDA = 6,         /* a CUDA runtime / driver call failed */
    ATTN_ERR_TIMEOUT = 7       /* device side only: a bounded wait inside the kernel gave up */
} attn_status;

enum { ATTN_BF16 = 0, ATTN_FP32 = 1 };                      /* element types */
enum { ATTN_NORM_SOFTMAX = 0, ATTN_NORM_SIGMOID = 1, ATTN_NORM_RELU = 2 };   /* Norm of Eq. 2 (Appendix A.3) */
/* Mask clauses of Appendix A.2, combined by AND.  ATTN_MASK_PREFIX relaxes the causal clause (PrefixLM:
 * keys j < prefix_len are visible to every row) and needs ATTN_MASK_CAUSAL; ATTN_MASK_TEST_QUERY relaxes
 * the document clause (causal blockwise mask: rows i >= test_query_start see keys of every document) and
 * needs ATTN_MASK_DOCUMENT.  ATTN_MASK_GLOBAL makes the first global_len positions global tokens: a key j <
 * global_len, and every key for a query row at position i' < global_len, passes the window and document
 * clauses (Global Sliding Window: "i in G or j in G"; Share Question mask: documents = prompt and responses,
 * global_len = prompt length, with the causal clause).  With ATTN_MASK_GLOBAL a row sees up to two key
 * intervals (the global keys and its own window / document). */
enum { ATTN_MASK_CAUSAL = 1u, ATTN_MASK_WINDOW = 2u, ATTN_MASK_DOCUMENT = 4u, ATTN_MASK_PREFIX = 8u,
       ATTN_MASK_TEST_QUERY = 16u, ATTN_MASK_GLOBAL = 32u };

typedef struct attn_variant_desc {
    uint32_t struct_size;      /* sizeof(attn_variant_desc) */
    uint32_t dtype;            /* element type of q, k, v */
    uint32_t o_dtype;          /* element type of o: equal to dtype, or ATTN_FP32 with bf16 inputs */
    uint32_t normalizer;       /* ATTN_NORM_* */
    uint32_t mask_flags;       /* OR of ATTN_MASK_* */
    int32_t  window_left;      /* with ATTN_MASK_WINDOW: j >= i' - window_left ; < 0 = unbounded */
    int32_t  window_right;     /* with ATTN_MASK_WINDOW: j <= i' + window_right ; < 0 = unbounded */
    float    scale;            /* multiplies q.k ; 0 means 1/sqrt(D) (Eq. 1) */
    float    softcap;          /* C of Appendix A.1 ; 0 = off */
    const float*   bias_slopes;/* device [Hq] or NULL: score += bias_slopes[h] * (i' - j) */
    float    sigmoid_bias;     /* b in out_scale * sigmoid(s + b) */
    float    out_scale;        /* 0 means 1 ; sigmoid normaliser: out_scale * sigmoid(s + b); ReLU normaliser:
                                  out_scale * max(s, 0) (the paper's 1/L) */
    const int32_t* cu_seqlens; /* device [num_docs + 1], cu[0] = 0, cu[num_docs] = Sq = Sk, non-decreasing;
                                  required with ATTN_MASK_DOCUMENT */
    int32_t  num_docs;
    int32_t  prefix_len;       /* with ATTN_MASK_PREFIX: L_p >= 0 */
    int32_t  test_query_start; /* with ATTN_MASK_TEST_QUERY: L_q >= 0 */
    int32_t  global_len;       /* with ATTN_MASK_GLOBAL: number of global tokens >= 0 */
    int64_t  q_strides[3];     /* elements: batch, head, row ; all zero = contiguous */
    int64_t  k_strides[3];
    int64_t  v_strides[3];
    int64_t  o_strides[3];
    int32_t* status_word;      /* optional device int32, zeroed by the caller (the library never clears it): a kernel
                                  that gives up a bounded wait stores ATTN_ERR_TIMEOUT here; a cu_seqlens table that
                                  does not start at 0, end at Sq or that decreases somewhere is reported as
                                  ATTN_ERR_DESC (the kernel stays memory safe and the output is unspecified); with
                                  the sigmoid normaliser at D = 128 and D = 256 (CTA-pair kernel) V is converted to
                                  fp16 on chip, and a |v| of 65536 or more (or a non-finite v) is reported as
                                  ATTN_ERR_UNSUPPORTED (output unspecified) */
} attn_variant_desc;

/*
 * attn_fwd -- the fused forward pass described at the top of this file (Eq. 1, Eq. 2,
 * Appendix A.1-A.3).
 *
 *   q, k, v  device, read only.      o  device, written for every row i < Sq.
 *   lse      device fp32 [B,Hq,Sq] or NULL.  Softmax: natural log of the row's sum of
 *            exp(modified, masked score); -inf for a row with no visible key (whose O row
 *            is 0).  Ignored (not written) for the sigmoid and ReLU normalisers.
 *   desc     host; see attn_variant_desc.
 *   stream   cudaStream_t (NULL = default stream).
 *
 * Supported: bf16 inputs with D in {64, 128, 256} (tcgen05 tensor-core kernel; o in bf16
 * or fp32), fp32 inputs with D <= 256 and D % 4 == 0 (fp32 FMA kernel; o in fp32).  Base
 * pointers 16-byte aligned; strides multiples of 16 bytes.  With ATTN_MASK_DOCUMENT:
 * B == 1 and Sq == Sk.
 *
 * The first call on a device loads the kernels and sets their shared-memory attribute.
 * Returns ATTN_OK or an attn_status; on an argument error nothing was launched.
 */
int attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
             int B, int Hq, int Hkv, int Sq, int Sk, int D,
             const attn_variant_desc* desc, void* stream);

/*
 * attn_fwd_host -- the same forward pass (Eq. 1, Eq. 2, Appendix A.1-A.3) for callers whose
 * tensors live in HOST memory (pinned memory makes the copies asynchronous).  It stages
 * q, k, v into `workspace` with cudaMemcpyAsync on `stream`, runs attn_fwd there and copies
 * o (and lse, if not NULL) back, all enqueued on `stream`; nothing is allocated.
 *
 *   q_host, k_host, v_host, o_host, lse_host   HOST pointers, contiguous [B,H,S,D] / [B,Hq,Sq].
 *   desc        as for attn_fwd, but the four stride arrays must be all zero; the device arrays
 *               it names (bias_slopes, cu_seqlens, status_word) stay DEVICE pointers.
 *   workspace   DEVICE pointer, 256-byte aligned, at least attn_host_workspace_bytes(...) bytes,
 *               owned by the caller and reusable across calls on the same stream.
 *
 * Returns ATTN_OK or an attn_status (ATTN_ERR_SHAPE if the workspace is too small); the host
 * output is complete once the stream work has finished.
 */
int attn_fwd_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host,
                  int B, int Hq, int Hkv, int Sq, int Sk, int D,
                  const attn_variant_desc* desc, void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of device workspace attn_fwd_host needs for these sizes (0 on invalid arguments). */
size_t attn_host_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, const attn_variant_desc* desc);

/* Text for an attn_status (static storage; never NULL). */
const char* attn_status_string(int status);

/* Library version: major * 10000 + minor * 100 + patch. */
int attn_version(void);

/* Number of kernel launches attn_fwd has issued in this process (for benchmarks). */
int64_t attn_launch_count(void);

/*
 * attn_clear_cache -- empties the library's cache of encoded TMA tensor maps (host memory only).  The tensor-core
 * kernels read Q, K and V tiles (Eq. 1) through tensor maps, which are pure functions of (base address, shape,
 * strides, box); a call on tensors seen before reuses the cached encoding.  An entry is never stale, so clearing
 * is never needed for correctness; it returns the table to its initial state.  Always ATTN_OK.
 */
int attn_clear_cache(void);

/* Number of tensor-map look-ups served from that cache in this process (for tests and benchmarks). */
int64_t attn_cache_hits(void);

/*
 * attn_selftest_timeout -- exercises the failure path of the kernels' bounded waits without a fault: launches
 * a one-CTA kernel in which one thread waits, for at most limit_ns, on an mbarrier that nothing arrives on (the
 * kernels that compute Eq. 1 / Eq. 2 link their roles with such barriers).  When the limit passes it stores
 * ATTN_ERR_TIMEOUT in *status_word and raises the CTA's abort flag; a second thread waiting on the same barrier
 * with the kernels' full limit sees the flag and returns at once (it stores 2 in *second_waiter, if given);
 * the kernel ends normally and the context stays usable.
 *
 *   status_word    device int32, zeroed by the caller.       second_waiter   device int32 or NULL.
 *   limit_ns       1 .. 100 000 000 (0.1 s); outside: ATTN_ERR_DESC, nothing launched.
 */
int attn_selftest_timeout(int32_t* status_word, uint64_t limit_ns, int32_t* second_waiter, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* B200_ATTN_H_ */
