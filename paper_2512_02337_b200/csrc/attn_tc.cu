// Tensor-core (tcgen05 / TMEM / TMA) verification attention for bfloat16, d = 128, 64-token pages.
#include "common.cuh"

namespace specpv {

bool attention_tc_supported(const AttnArgs& a) {
    (void)a;
    return false;
}

specpv_status launch_attention_tc(const AttnArgs& a, cudaStream_t stream) {
    (void)a;
    (void)stream;
    return SPECPV_ERR_UNSUPPORTED;
}

}  // namespace specpv
