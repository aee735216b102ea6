// Window attention kernels (N <= 64) of the IPTQ_SM_LOG2 Softmax variant (both head dimensions, every flag combination).
#include "attention_window.cuh"

namespace iptq {

int window_launch_variant3(int dh, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                           const AttnParams& p, int smem_bytes, cudaStream_t st)
{
    if (dh == 64) return launch_window_attn<64, IPTQ_SM_LOG2>(mq, mk, mv, p, smem_bytes, st);
    return launch_window_attn<32, IPTQ_SM_LOG2>(mq, mk, mv, p, smem_bytes, st);
}

}  // namespace iptq
