// Interface of the tensor-core (tcgen05 / TMA, bf16 operands, fp32 accumulation) engine.
#pragma once
#include "common.cuh"

namespace mg {

struct UmmaFwdWs {
  __nv_bfloat16* W_hh;   // [3H,H]
  __nv_bfloat16* W_ih;   // [3H,I]
  __nv_bfloat16* xb;     // [T*B,I]
  __nv_bfloat16* Apack;  // [maxM,H]  A operand of one step (rows gathered from the level state)
  size_t maxM;
};

struct UmmaAdjWs {
  __nv_bfloat16* W_hh;    // [3H,H]   (linearisation)
  __nv_bfloat16* W_hhT;   // [H,3H]   (adjoint step: B operand, K = 3H contiguous)
  __nv_bfloat16* W_ihT;   // [I,3H]   (dx = dA_i W_ih)
  __nv_bfloat16* Apack;   // [maxM,3H]
  size_t apack_elems;     // its size in elements
  __nv_bfloat16* dAh;     // [T*B,3H]  gradient-pass operand [cr|cz|cn]*lambda
  __nv_bfloat16* dAi;     // [T*B,3H]  gradient-pass operand [cr|cz|cn']*lambda
  __nv_bfloat16* xb;      // [T*B,I]   bf16 copy of the layer input
  __nv_bfloat16* hb0;     // [(T+1)*B,H] bf16 copy of [h_0; h]: row (t,b) is h_{t-1} of step t
  __nv_bfloat16* hb;      // = hb0 + B*H: the given states
  size_t maxM;
};

int umma_supported(const mgrit_gru_cfg* c);
void umma_plan_fwd(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, UmmaFwdWs* o);
void umma_plan_adj(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, UmmaAdjWs* o);
int umma_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, UmmaFwdWs* w, cudaStream_t s);
int umma_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, const float* h0, const float* h, UmmaAdjWs* w, bool have_hb,
                     cudaStream_t s);
void umma_convert(const float* src, __nv_bfloat16* dst, i64 n, cudaStream_t s);
int umma_project_rows(const float* X, __nv_bfloat16* xb, const __nv_bfloat16* Wb, const float* bias, float* out, int M, int K, int H3,
                      cudaStream_t s);
int umma_adj_dx(const AdjStepArgs& a, const __nv_bfloat16* W_ihT, int C, float* out, UmmaAdjWs* w, cudaStream_t s);
int umma_fwd_step(const FwdStepArgs& a, UmmaFwdWs* w, cudaStream_t s);
int umma_linearise(const LinArgs& a, UmmaAdjWs* w, cudaStream_t s);
int umma_adj_step(const AdjStepArgs& a, UmmaAdjWs* w, cudaStream_t s);
int umma_gradients(const mgrit_gru_cfg* c, const gru_params* p, const float* x, const float* h0, const float* h,
                   const float* lam, i64 lam_ts, const __nv_bfloat16* cr, const __nv_bfloat16* cz, const __nv_bfloat16* cn,
                   const __nv_bfloat16* cnp, float* dx,
                   const gru_grads* g, UmmaAdjWs* w, bool have_xb, cudaStream_t s);
// the three step functions return MGRIT_OK or MGRIT_CUDA_ERROR (a tensor map could not be encoded, a launch failed)
int umma_device_status();
int umma_clear_device_status();

}  // namespace mg
