#include "umma_engine.cuh"
namespace mg {
int umma_supported(const mgrit_gru_cfg*) { return MGRIT_UNSUPPORTED; }
void umma_plan_fwd(const mgrit_gru_cfg*, const int*, int, char*, size_t*, UmmaFwdWs*) {}
void umma_plan_adj(const mgrit_gru_cfg*, const int*, int, char*, size_t*, UmmaAdjWs*) {}
int umma_prepare_fwd(const mgrit_gru_cfg*, const gru_params*, const float*, float*, UmmaFwdWs*, cudaStream_t) { return MGRIT_UNSUPPORTED; }
int umma_prepare_adj(const mgrit_gru_cfg*, const gru_params*, UmmaAdjWs*, cudaStream_t) { return MGRIT_UNSUPPORTED; }
void umma_fwd_step(const FwdStepArgs&, UmmaFwdWs*, cudaStream_t) {}
void umma_linearise(const LinArgs&, UmmaAdjWs*, cudaStream_t) {}
void umma_adj_step(const AdjStepArgs&, UmmaAdjWs*, cudaStream_t) {}
int umma_gradients(const mgrit_gru_cfg*, const gru_params*, const float*, const float*, const float*, const float*, const float*,
                   const float*, const float*, const float*, float*, const gru_grads*, UmmaAdjWs*, cudaStream_t) { return MGRIT_UNSUPPORTED; }
int umma_device_status() { return 0; }
}
