// Ping-pong attention kernel (attn_tc_pingpong.cuh): the instances for masks whose rows see one key interval and
// whose output is stored by the threads themselves (work items of 256 rows of one head, or fp32 output), and the
// choice among all tensor-core kernels.  The instances for global-token masks and for TMA-stored output are compiled
// in files of their own (attn_tc_pingpong_global.cu, attn_tc_pingpong_tmaout.cu) so that they build in parallel.
#include "attn_tc_pingpong.cuh"

namespace b200attn {

int launch_attn_fwd_bf16_split(const AttnParams& p, cudaStream_t stream);          // attn_tc_split.cu
int launch_attn_fwd_bf16_pair(const AttnParams& p, cudaStream_t stream);           // attn_tc_pair.cu
int launch_attn_fwd_bf16_pingpong_global(const AttnParams& p, cudaStream_t stream);   // attn_tc_pingpong_global.cu
int launch_attn_fwd_bf16_pingpong_tmaout(const AttnParams& p, cudaStream_t stream);   // attn_tc_pingpong_tmaout.cu

namespace {
// Masks with global tokens get their own instances, so that the others carry none of the two-piece walk; work items
// of two heads x 128 rows (even GQA group) with bf16 output get the instances whose epilogue goes through TMA stores.
// A causal blockwise mask whose test-query blocks should open the work order (few heads per L2 section: see
// leading_blocks) runs on the global-token instances as well: they are the ones that decode such an order, and without
// global tokens they compute the same thing (their steps are ~3 % slower; the order gains far more there).
int launch_pingpong(const AttnParams& p, cudaStream_t stream) {
    if (p.mask_flags & kMaskGlobal) return launch_attn_fwd_bf16_pingpong_global(p, stream);
    if ((p.mask_flags & kMaskTestQuery) && planned_leading_blocks(p) > 0) return launch_attn_fwd_bf16_pingpong_global(p, stream);
    if (p.group % 2 == 0 && !p.o_fp32) return launch_attn_fwd_bf16_pingpong_tmaout(p, stream);
    switch (p.D) {
        case 64: return launch_for_mask<64, 2, false, false>(p, stream);
        case 128: return launch_for_mask<128, 2, false, false>(p, stream);
        default: return ATTN_ERR_UNSUPPORTED;
    }
}
}  // namespace

// Kernel choice.  D = 64, 128: two query tiles per work item ping-pong on one SM (this file).  D = 256: CTA pairs
// (attn_tc_pair.cu), which halve the K / V traffic from L2.  The sigmoid normaliser at D = 128 runs on the CTA-pair
// kernel too: its one-pass fp16 form of P V (with V converted on chip) beats the bf16 hi + lo pair of this file by
// 15 to 40 % on the paper-shaped sweep.  B200ATTN_FORCE_SPLIT=1 / B200ATTN_FORCE_PAIR=1 in the
// environment route every head dimension they support to the one-tile kernel (attn_tc_split.cu) or to the
// CTA-pair kernel; the tests use them to cover those kernels at the other head dimensions.
int launch_attn_fwd_bf16(const AttnParams& p, cudaStream_t stream, int* launches) {
    *launches = 0;
    static const bool force_split = []() { const char* e = getenv("B200ATTN_FORCE_SPLIT"); return e && e[0] == '1'; }();
    static const bool force_pair = []() { const char* e = getenv("B200ATTN_FORCE_PAIR"); return e && e[0] == '1'; }();
    int rc;
    const bool global = (p.mask_flags & kMaskGlobal) != 0;
    if (force_split || (global && (p.D == 256 || force_pair))) {   // two key pieces per row: not on the CTA-pair kernel
        rc = launch_attn_fwd_bf16_split(p, stream);
    } else if (p.D == 256 || (p.D == 128 && !global && (force_pair || p.normalizer == kNormSigmoid))) {
        rc = launch_attn_fwd_bf16_pair(p, stream);
    } else {
        rc = launch_pingpong(p, stream);
    }
    if (rc == ATTN_OK) *launches = 1;
    return rc;
}

}  // namespace b200attn
