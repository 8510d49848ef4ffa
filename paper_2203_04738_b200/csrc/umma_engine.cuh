// Interface of the tensor-core (tcgen05 / TMA, bf16 operands, fp32 accumulation) engine.
#pragma once
#include "common.cuh"

namespace mg {

struct UmmaFwdWs {
  __nv_bfloat16* W_hh;   // [3H,H]
  __nv_bfloat16* W_ih;   // [3H,I]
  __nv_bfloat16* xb;     // [T*B,I]
  __nv_bfloat16* Apack;  // [maxM,H]  A operand of one step (rows gathered from the level state)
  __nv_bfloat16* gib;    // [T*B,3H]  bf16 copy of the input projection, written by the projection's epilogue
  size_t maxM;
};

struct UmmaAdjWs {
  __nv_bfloat16* W_hh;    // [3H,H]   (linearisation)
  __nv_bfloat16* W_hhT;   // [H,3H]   (adjoint step: B operand, K = 3H contiguous)
  __nv_bfloat16* W_ihT;   // [I,3H]   (dx = dA_i W_ih)
  __nv_bfloat16* Apack;   // [maxM,3H]
  size_t apack_elems;     // its size in elements
  __nv_bfloat16* dA4;     // [T*B,4H]  gradient-pass operands [cr|cz|cn|cn']*lambda (recurrent weights: blocks 0-2; input side: 0, 1, 3)
  __nv_bfloat16* xb;      // [T*B,I]   bf16 copy of the layer input
  __nv_bfloat16* hb0;     // [(T+1)*B,H] bf16 copy of [h_0; h]: row (t,b) is h_{t-1} of step t
  __nv_bfloat16* hb;      // = hb0 + B*H: the given states
  const __nv_bfloat16* gib;  // bf16 copy of the input projection left by the forward call, or nullptr
  size_t maxM;
};

// TF32 operand modes (same GEMM kernel, `.kind::tf32`): operands are fp32 arrays of tf32 values, split in S = 3 parts
// along the reduction (MGRIT_OPERANDS_TF32) or rounded once (S = 1, MGRIT_OPERANDS_TF32_1PASS)
struct Tf32Ws {
  int S;
  int ng;         // gate blocks of the weights: 3 (GRU) or 4 (LSTM); "3H" below reads ng*H
  float* W_hh;    // [3H, S*H]   B side of the forward product
  float* W_ih;    // [3H, S*I]   forward call only
  float* W_hhT;   // [H, S*3H]   adjoint call: B side of the adjoint step
  float* W_ihT;   // [I, S*3H]   adjoint call: B side of dx = dA_i W_ih
  float* Apack;   // A side of the current product
  size_t apack_elems;
  float* dAT;     // [3H, S*T*B] gradient pass: dA^T
  float* RT;      // [max(H,I), S*T*B]: h_prev^T or x^T
  float* split_scratch;   // partial products of a split reduction
};
int tf32_supported(const mgrit_gru_cfg* c);
void tf32_plan_fwd(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, Tf32Ws* o, int ng = 3);
void tf32_plan_adj(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, Tf32Ws* o, int ng = 3);
// Implicit LSTM steps on the same products (raw results, contiguous [M, H], as the fp32 engine's)
int tf32_lstm_fwd_step(const LstmFwdArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_lstm_linearise(const LstmLinArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_lstm_adj_step(const LstmAdjArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, Tf32Ws* w, cudaStream_t s);
int tf32_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, Tf32Ws* w, cudaStream_t s);
int tf32_fwd_step(const FwdStepArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_linearise(const LinArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_adj_step(const AdjStepArgs& a, Tf32Ws* w, cudaStream_t s);
int tf32_wgrad(const float* dA, int M, int H3, const float* first, int Bfirst, const float* rest, int C, float* dW, Tf32Ws* w,
               cudaStream_t s);
int tf32_dgrad(const float* dA, int M, int H3, int C, float* dx, Tf32Ws* w, cudaStream_t s);

// Implicit LSTM with bf16 operands: the plain GEMM with four-gate tiles, fp32 states and fp32 coefficients
struct LstmBfWs {
  __nv_bfloat16 *W_hh, *W_ih;     // [4H,H], [4H,I]
  __nv_bfloat16 *W_hhT, *W_ihT;   // [H,4H], [I,4H]   (adjoint call)
  __nv_bfloat16* Apack;           // A side of the current product
  size_t apack_elems;
  __nv_bfloat16 *xb, *hb0, *dAb;  // [T*B,I]; [(T+1)*B,H] = [h_0; h]; [T*B,4H]   (gradient pass)
  float* scratch; size_t scratch_bytes;   // partial products of the split weight-gradient reductions
};
void lstmbf_plan_fwd(const mgrit_gru_cfg* c, size_t max_rows, char* base, size_t* off, LstmBfWs* o);
void lstmbf_plan_adj(const mgrit_gru_cfg* c, size_t max_rows, char* base, size_t* off, LstmBfWs* o);
int lstmbf_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, LstmBfWs* w, cudaStream_t s);
int lstmbf_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, LstmBfWs* w, cudaStream_t s);
int lstmbf_fwd_step(const LstmFwdArgs& a, LstmBfWs* w, cudaStream_t s);
int lstmbf_linearise(const LstmLinArgs& a, LstmBfWs* w, cudaStream_t s);
int lstmbf_adj_step(const LstmAdjArgs& a, LstmBfWs* w, cudaStream_t s);
// dW_hh, dW_ih (and dx) from dA[T*B,4H] fp32; hidden states h0 [B,H] and hk [T,B,H] fp32
int lstmbf_gradients(const mgrit_gru_cfg* c, const float* lc, const float* lh, i64 lam_ts, const float* p, const __nv_bfloat16* ci,
                     const __nv_bfloat16* cf, const __nv_bfloat16* cg, const __nv_bfloat16* co, const float* x, const float* h0,
                     const float* h_rows, i64 h_ts, const gru_grads* g, float* dx, LstmBfWs* w, cudaStream_t s);

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
// all steps of a relaxation sweep in one launch of the fused kernel (needs the bf16 state copies and 128 % B == 0);
// MGRIT_UNSUPPORTED = not available for this shape (the caller launches the steps one by one)
int umma_fwd_sweep(const FwdSweepArgs& a, UmmaFwdWs* w, cudaStream_t s);
int umma_linearise(const LinArgs& a, UmmaAdjWs* w, cudaStream_t s);
int umma_adj_step(const AdjStepArgs& a, UmmaAdjWs* w, cudaStream_t s);
int umma_gradients(const mgrit_gru_cfg* c, const gru_params* p, const float* x, const float* h0, const float* h,
                   const float* lam, i64 lam_ts, const __nv_bfloat16* cr, const __nv_bfloat16* cz, const __nv_bfloat16* cn,
                   const __nv_bfloat16* cnp, float* dx,
                   const gru_grads* g, UmmaAdjWs* w, bool have_xb, cudaStream_t s);
// the three step functions return MGRIT_OK or MGRIT_CUDA_ERROR (a tensor map could not be encoded, a launch failed)
int umma_device_status();
int umma_selftest_wait(int limit_ms, cudaStream_t s);
int umma_clear_device_status();

}  // namespace mg
