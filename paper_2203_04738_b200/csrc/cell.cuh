// Device arithmetic of one GRU cell evaluation and of its transposed Jacobian.
//
// FAST = false: precise expf/tanhf/division, used by the fp32 operand mode.
// FAST = true : MUFU approximations (tanh.approx, rcp.approx; absolute error about 5e-4 on a gate),
//               used by the bf16 operand mode, whose operand rounding is coarser than that.  At
//               H = 1024 the gate arithmetic of a tile costs as many issue slots as its tensor-core
//               main loop, so the instruction count per element matters.
#pragma once
#include "common.cuh"

namespace mg {

__device__ __forceinline__ float tanh_approx(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <bool FAST> __device__ __forceinline__ float sigmoid_t(float x) {
  if (FAST) return fmaf(tanh_approx(0.5f * x), 0.5f, 0.5f);
  return 1.0f / (1.0f + __expf(-x));
}
template <bool FAST> __device__ __forceinline__ float tanh_t(float x) { return FAST ? tanh_approx(x) : tanhf(x); }
template <bool FAST> __device__ __forceinline__ float inv_t(float x) { return FAST ? rcp_approx(x) : 1.0f / x; }

// Phi_gamma(x_t, h_{t-1}) given the pre-activations: gi_* = W_i* x + b_i*, gh_* = W_h* h + b_h*.
// classic  (Eq. "gru-classic"): h + gamma(1-z)(n - h)
// implicit (Eq. "gru-imap")   : (h + gamma(1-z) n) / (1 + gamma(1-z))
template <bool FAST = false>
__device__ __forceinline__ float cell_forward(float gir, float giz, float gin, float ghr, float ghz, float ghn,
                                              float hp, float gamma, int cell) {
  float r = sigmoid_t<FAST>(gir + ghr);
  float z = sigmoid_t<FAST>(giz + ghz);
  float n = tanh_t<FAST>(fmaf(r, ghn, gin));
  float q = gamma * (1.0f - z);
  return cell == MGRIT_CELL_IMPLICIT ? fmaf(q, n, hp) * inv_t<FAST>(1.0f + q) : fmaf(q, n - hp, hp);
}

struct CellLin { float a, cr, cz, cn, cnp; };

// Entries of the transposed Jacobian of one step: lambda_prev = a*lam + [cr*lam|cz*lam|cn*lam] W_hh,
// d(gi) = [cr*lam|cz*lam|cnp*lam].
template <bool FAST = false>
__device__ __forceinline__ CellLin cell_linearise(float gir, float giz, float gin, float ghr, float ghz, float ghn,
                                                  float hp, float gamma, int cell) {
  float r = sigmoid_t<FAST>(gir + ghr);
  float z = sigmoid_t<FAST>(giz + ghz);
  float n = tanh_t<FAST>(fmaf(r, ghn, gin));
  float q = gamma * (1.0f - z);
  float a, dn, dz;
  if (cell == MGRIT_CELL_IMPLICIT) {
    float inv = inv_t<FAST>(1.0f + q);
    a = inv; dn = q * inv; dz = -gamma * (n - hp) * inv * inv;
  } else {
    a = 1.0f - q; dn = q; dz = -gamma * (n - hp);
  }
  CellLin o;
  o.a = a;
  o.cnp = dn * (1.0f - n * n);
  o.cn = o.cnp * r;
  o.cr = o.cnp * ghn * r * (1.0f - r);
  o.cz = dz * z * (1.0f - z);
  return o;
}

// ---- Implicit LSTM: the cell state is an Euler step of c' = -(1-f) c + i g with step gamma, decay term implicit
// (implicit) or explicit (classic; gamma = 1 is the textbook LSTM); h = o tanh(c) is re-evaluated from the new c.
// Pre-activations: gi_* = W_i* x + b_i*, gh_* = W_h* h + b_h*, gate order i | f | g | o.
struct LstmOut { float c, h; };
template <bool FAST = false>
__device__ __forceinline__ LstmOut lstm_forward(float gii, float gif, float gig, float gio, float ghi, float ghf, float ghg, float gho,
                                                float cp, float gamma, int cell) {
  float i = sigmoid_t<FAST>(gii + ghi), f = sigmoid_t<FAST>(gif + ghf), g = tanh_t<FAST>(gig + ghg), o = sigmoid_t<FAST>(gio + gho);
  float q = gamma * (1.0f - f);
  LstmOut r;
  r.c = cell == MGRIT_CELL_IMPLICIT ? fmaf(gamma * i, g, cp) * inv_t<FAST>(1.0f + q) : fmaf(gamma * i, g, cp - q * cp);
  r.h = o * tanh_t<FAST>(r.c);
  return r;
}

// Transposed Jacobian of one LSTM step: with (L_c, L_h) the sensitivities of the outputs,
//   dc = L_c + p*L_h;  d(pre-activations) = [ci*dc | cf*dc | cg*dc | co*L_h];  L_c_in = a*dc;  L_h_in = d(pre) W_hh
struct LstmLin { float a, p, ci, cf, cg, co; };
template <bool FAST = false>
__device__ __forceinline__ LstmLin lstm_linearise(float gii, float gif, float gig, float gio, float ghi, float ghf, float ghg, float gho,
                                                  float cp, float gamma, int cell) {
  float i = sigmoid_t<FAST>(gii + ghi), f = sigmoid_t<FAST>(gif + ghf), g = tanh_t<FAST>(gig + ghg), o = sigmoid_t<FAST>(gio + gho);
  float q = gamma * (1.0f - f);
  float c, a, dci, dcg, dcf;
  if (cell == MGRIT_CELL_IMPLICIT) {
    float inv = inv_t<FAST>(1.0f + q);
    c = fmaf(gamma * i, g, cp) * inv;
    a = inv; dci = gamma * g * inv; dcg = gamma * i * inv; dcf = gamma * c * inv;
  } else {
    c = fmaf(gamma * i, g, cp - q * cp);
    a = 1.0f - q; dci = gamma * g; dcg = gamma * i; dcf = gamma * cp;
  }
  float th = tanh_t<FAST>(c);
  LstmLin r;
  r.a = a; r.p = o * (1.0f - th * th);
  r.ci = dci * i * (1.0f - i); r.cf = dcf * f * (1.0f - f); r.cg = dcg * (1.0f - g * g); r.co = th * o * (1.0f - o);
  return r;
}

}  // namespace mg
