// Interface of the persistent kernels for chains of dependent steps with few rows.
#pragma once
#include "common.cuh"

namespace mg {

// u_j = Phi_gamma(gi_j, u_{j-1}) + g_j,  j = 1..nsteps   (slot-major state [nsteps+1][B][H], slot 0 given)
struct SerialFwdArgs {
  int B, H, nsteps;
  float* u;                      // level state; slots 1..nsteps are written
  __nv_bfloat16* ub;             // [2][B][H] scratch: bf16 copy of the newest state
  const float* gi; i64 gi_step;  // projection rows of step 1 (+ (j-1)*gi_step for step j), row b at + b*3H
  const __nv_bfloat16* gi_b;     // the projection as bf16 (same indexing as gi), or nullptr; when given, gi is not read
  int gi_as_bf16;                // 1: round every projection value to bf16 after loading it, so that the chain sees the same
                                 // values as the relaxation kernels of the other levels, which stage the projection's bf16 copy
  const float* g;                // [nsteps+1][B][H] additive term, or nullptr
  const __nv_bfloat16* W;        // [3H][H]
  const float* b_hh;
  float gamma; int cell;
  unsigned* bar;                 // [ceil(B/16)] barrier counters (scratch)
  uint4* xw; size_t xw_bytes;    // exchange words of the flag-in-data hand-over (scratch, serial_xw_bytes()), or nullptr
};

// mu_s = a_s*mu_{s-1} + ([cr_s|cz_s|cn_s]*mu_{s-1}) W_hh + g_s,  s = 1..nsteps
struct SerialAdjArgs {
  int B, H, nsteps;
  float* mu;                     // [nsteps+1][B][H], slot 0 given
  __nv_bfloat16* dAb;            // [2][B][3H] scratch
  const float* a;                // coefficient rows of step 1; step s at + (s-1)*coef_step
  const __nv_bfloat16 *cr, *cz, *cn;
  i64 coef_step;
  const float* g;                // [nsteps+1][B][H] or nullptr
  const __nv_bfloat16* WT;       // [H][3H] = W_hh^T
  unsigned* bar;
  uint4* xw; size_t xw_bytes;    // as in SerialFwdArgs (three gate blocks per producer)
};

// The same chains in fp32 arithmetic (FFMA, precise gate math) for the fp32 and tf32 operand modes: fp32 weights in
// shared memory, the fp32 state itself crosses CTAs (counter barrier + reload).
struct Serial32FwdArgs {
  int B, H, nsteps;
  float* u;                      // level state; slots 1..nsteps are written
  const float* gi; i64 gi_step;
  const float* g;
  const float* W;                // [3H][H] fp32
  const float* b_hh;
  float gamma; int cell;
  unsigned* bar;                 // [ceil(B/16)] barrier counters (scratch)
};
struct Serial32AdjArgs {
  int B, H, nsteps;
  float* mu;
  float* dA;                     // [2][B][3H] scratch: [cr|cz|cn] of the next step times the newest mu
  const float *a, *cr, *cz, *cn; // coefficient rows of step 1; step s at + (s-1)*coef_step
  i64 coef_step;
  const float* g;
  const float* W;                // [3H][H] fp32 (W_hh as given)
  unsigned* bar;
};
bool serial32_fwd_solve(const Serial32FwdArgs& a, cudaStream_t s);
bool serial32_adj_solve(const Serial32AdjArgs& a, cudaStream_t s);

// bytes of exchange words for a chain over B rows of H units carrying `gates` values per (row, unit)
size_t serial_xw_bytes(int B, int H, int gates);

bool serial_fwd_supported(int B, int H);
bool serial_adj_supported(int B, int H);
// false: shape not supported or the cooperative launch failed (the caller then advances step by step)
bool serial_fwd_solve(const SerialFwdArgs& a, cudaStream_t s);
bool serial_adj_solve(const SerialAdjArgs& a, cudaStream_t s);
// Implicit LSTM chains, bf16 operands.  A state slot is (c, h): arrays [nsteps+1][2][B][H], slot 0 given.
//   forward:  (c, h)_j = Phi_gamma(gi_j, (c, h)_{j-1}) + g_j
//   adjoint:  dc = Lc + p*Lh;  (Lc, Lh)_s = (a*dc, [ci*dc | cf*dc | cg*dc | co*Lh] W_hh) + g_s   (coefficients of step s)
struct LstmChainFwdArgs {
  int B, H, nsteps;
  float* u;
  const float* gi; i64 gi_step;  // projection rows of step 1 (+ (j-1)*gi_step for step j), row b at + b*4H
  const float* g;                // [nsteps+1][2][B][H] additive term, or nullptr
  const __nv_bfloat16* W;        // [4H][H]
  const float* b_hh;
  float gamma; int cell;
  uint4* xw; size_t xw_bytes;    // exchange words, serial_xw_bytes(B, H, 1)
};
struct LstmChainAdjArgs {
  int B, H, nsteps;
  float* mu;
  const float *a, *p;                       // coefficient rows of step 1; step s at + (s-1)*coef_step
  const __nv_bfloat16 *ci, *cf, *cg, *co;   // the four gate coefficients (bf16), same indexing
  i64 coef_step;
  const float* g;
  const __nv_bfloat16* WT;       // [H][4H] = W_hh^T
  uint4* xw; size_t xw_bytes;    // exchange words, serial_xw_bytes(B, H, 4)
};
// false: shape not supported (forward: H % 128 != 0; adjoint: H not in {128, 256, 512, 1024}; too many CTAs for one wave)
// or the cooperative launch failed: the caller then advances step by step
bool lstm_chain_fwd_solve(const LstmChainFwdArgs& a, cudaStream_t s);
bool lstm_chain_adj_solve(const LstmChainAdjArgs& a, cudaStream_t s);
int serial_device_status();
int serial_clear_device_status();

}  // namespace mg
