// Tensor-core (tcgen05) kernel of the channel-compacted FFN -- placeholder until the
// kernel lands: reports "not supported" so that the plain-ALU kernel takes every shape.
#include "common.cuh"
#include "ffn_plan.cuh"

bool ffn_tc_supported(const sentry_ffn_desc&) { return false; }
int ffn_tc_kc_pad(int k_c) { return (k_c + 127) / 128 * 128; }
int launch_ffn_tc(sentry_ctx*, const FfnArgs&, const FfnPlan&, void*, void*, int, int, cudaStream_t) {
    return SENTRY_ERR_UNSUPPORTED;
}
