// Ping-pong attention kernel (attn_tc_pingpong.cuh): the instances for masks with global tokens (Appendix A.2: Global
// Sliding Window, Share Question mask), in which a row sees two key pieces and the key-tile list of a work item is
// walked by position.
#include "attn_tc_pingpong.cuh"

namespace b200attn {

int launch_attn_fwd_bf16_pingpong_global(const AttnParams& p, cudaStream_t stream) {
    switch (p.D) {
        case 64: return launch_for_mask<64, 2, true, false>(p, stream);
        case 128: return launch_for_mask<128, 2, true, false>(p, stream);
        default: return ATTN_ERR_UNSUPPORTED;
    }
}

}  // namespace b200attn
