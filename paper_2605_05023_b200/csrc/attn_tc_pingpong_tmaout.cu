// Ping-pong attention kernel (attn_tc_pingpong.cuh): the instances for work items of two heads x 128 rows (even GQA
// group) with bf16 output, whose epilogue goes through per-warp shared-memory boxes and TMA tile stores.
#include "attn_tc_pingpong.cuh"

namespace b200attn {

int launch_attn_fwd_bf16_pingpong_tmaout(const AttnParams& p, cudaStream_t stream) {
    switch (p.D) {
        case 64: return launch_for_mask<64, 2, false, true>(p, stream);
        case 128: return launch_for_mask<128, 2, false, true>(p, stream);
        default: return ATTN_ERR_UNSUPPORTED;
    }
}

}  // namespace b200attn
