// Device arithmetic of one GRU cell evaluation and of its transposed Jacobian.
#pragma once
#include "common.cuh"

namespace mg {

__device__ __forceinline__ float sigmoid_f(float x) { return 1.0f / (1.0f + __expf(-x)); }

// Phi_gamma(x_t, h_{t-1}) given the pre-activations: gi_* = W_i* x + b_i*, gh_* = W_h* h + b_h*.
// classic  (Eq. "gru-classic"): h + gamma(1-z)(n - h)
// implicit (Eq. "gru-imap")   : (h + gamma(1-z) n) / (1 + gamma(1-z))
__device__ __forceinline__ float cell_forward(float gir, float giz, float gin, float ghr, float ghz, float ghn,
                                              float hp, float gamma, int cell) {
  float r = sigmoid_f(gir + ghr);
  float z = sigmoid_f(giz + ghz);
  float n = tanhf(gin + r * ghn);
  float q = gamma * (1.0f - z);
  return cell == MGRIT_CELL_IMPLICIT ? (hp + q * n) / (1.0f + q) : hp + q * (n - hp);
}

struct CellLin { float a, cr, cz, cn, cnp; };

// Entries of the transposed Jacobian of one step: lambda_prev = a*lam + [cr*lam|cz*lam|cn*lam] W_hh,
// d(gi) = [cr*lam|cz*lam|cnp*lam].
__device__ __forceinline__ CellLin cell_linearise(float gir, float giz, float gin, float ghr, float ghz, float ghn,
                                                  float hp, float gamma, int cell) {
  float r = sigmoid_f(gir + ghr);
  float z = sigmoid_f(giz + ghz);
  float n = tanhf(gin + r * ghn);
  float q = gamma * (1.0f - z);
  float a, dn, dz;
  if (cell == MGRIT_CELL_IMPLICIT) {
    float inv = 1.0f / (1.0f + q);
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

}  // namespace mg
