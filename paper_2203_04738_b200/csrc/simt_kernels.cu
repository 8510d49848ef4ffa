// fp32 FFMA engine: one tiled GEMM skeleton with operand-loader and epilogue functors.
// Used when cfg.operands == MGRIT_OPERANDS_FP32 (the precision mode whose results must agree
// with the fp64 oracle to 1e-4), and for shapes the tensor-core engine does not cover.
#include "cell.cuh"

namespace mg {

namespace {

constexpr int BM = 32, BN = 32, BK = 32, NT = 256;

// C[m, (g, n)] = sum_k A(m, k) * B(g, n, k);  epi(m, n, acc[NG]).
// AKC / BKC: the loader's fastest index is k (operand stored K-contiguous) or the row/column.
template <int NG, bool AKC, bool BKC, class AL, class BL, class Epi>
__global__ void __launch_bounds__(NT) simt_gemm_kernel(int M, int N, int K, AL al, BL bl, Epi epi) {
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[NG][BK][BN + 1];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  const int ty = tid / 16, tx = tid % 16;
  float acc[NG][2][2];
#pragma unroll
  for (int g = 0; g < NG; ++g) { acc[g][0][0] = acc[g][0][1] = acc[g][1][0] = acc[g][1][1] = 0.f; }

  for (int k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int e = tid; e < BM * BK; e += NT) {
      int r, k;
      if (AKC) { r = e / BK; k = e % BK; } else { r = e % BM; k = e / BM; }
      int gr = m0 + r, gk = k0 + k;
      As[k][r] = (gr < M && gk < K) ? al(gr, gk) : 0.f;
    }
#pragma unroll
    for (int g = 0; g < NG; ++g) {
#pragma unroll
      for (int e = tid; e < BN * BK; e += NT) {
        int c, k;
        if (BKC) { c = e / BK; k = e % BK; } else { c = e % BN; k = e / BN; }
        int gc = n0 + c, gk = k0 + k;
        Bs[g][k][c] = (gc < N && gk < K) ? bl(g, gc, gk) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < BK; ++k) {
      float a0 = As[k][ty], a1 = As[k][ty + 16];
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        float b0 = Bs[g][k][tx], b1 = Bs[g][k][tx + 16];
        acc[g][0][0] = fmaf(a0, b0, acc[g][0][0]);
        acc[g][0][1] = fmaf(a0, b1, acc[g][0][1]);
        acc[g][1][0] = fmaf(a1, b0, acc[g][1][0]);
        acc[g][1][1] = fmaf(a1, b1, acc[g][1][1]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      int row = m0 + ty + 16 * i, col = n0 + tx + 16 * j;
      if (row < M && col < N) {
        float v[NG];
#pragma unroll
        for (int g = 0; g < NG; ++g) v[g] = acc[g][i][j];
        epi(row, col, v);
      }
    }
}

template <int NG, bool AKC, bool BKC, class AL, class BL, class Epi>
void launch(int kc, int M, int N, int K, AL al, BL bl, Epi epi, cudaStream_t s) {
  if (M <= 0 || N <= 0) return;
  dim3 grid((M + BM - 1) / BM, (N + BN - 1) / BN);
  prof_begin(kc, 2.0 * M * N * NG * K, s);
  simt_gemm_kernel<NG, AKC, BKC><<<grid, NT, 0, s>>>(M, N, K, al, bl, epi);
  prof_end(s);
  count_launch();
}

// ---------------------------------------------------------------- loaders
struct DenseA {  // A[m,k] = p[m*ld + k]
  const float* p; i64 ld;
  __device__ float operator()(int m, int k) const { return p[(i64)m * ld + k]; }
};
struct DenseAT {  // A[m,k] = p[k*ld + m]
  const float* p; i64 ld;
  __device__ float operator()(int m, int k) const { return p[(i64)k * ld + m]; }
};
struct StridedRowsA {  // rows (k_, b): p + k_*ks + b*H
  const float* p; i64 ks; int B, H;
  __device__ float operator()(int m, int k) const { return p[(i64)(m / B) * ks + (i64)(m % B) * H + k]; }
};
struct GateW {  // B(g, n, k) = W[(g*H + n)*ld + k]
  const float* W; int H; i64 ld;
  __device__ float operator()(int g, int n, int k) const { return W[((i64)g * H + n) * ld + k]; }
};
struct DenseB {  // B(0, n, k) = W[n*ld + k]
  const float* W; i64 ld;
  __device__ float operator()(int, int n, int k) const { return W[(i64)n * ld + k]; }
};
struct DenseBT {  // B(0, n, k) = W[k*ld + n]
  const float* W; i64 ld;
  __device__ float operator()(int, int n, int k) const { return W[(i64)k * ld + n]; }
};
struct FirstRestBT {  // B(0, n, k=m): m < nfirst ? first[m*C + n] : rest[(m - nfirst)*C + n]
  const float* first; int nfirst; const float* rest; int C;
  __device__ float operator()(int, int n, int k) const {
    return k < nfirst ? first[(i64)k * C + n] : rest[(i64)(k - nfirst) * C + n];
  }
};
struct LinA {  // state entering forward step j = m/B + 1 of a level: h at fine time t0 + stride*(j-1)
  const float* h0; const float* h; i64 stride_t, t0; int B, H;
  __device__ float operator()(int m, int k) const {
    int j1 = m / B, b = m % B;
    const i64 t = t0 + (i64)j1 * stride_t;
    return t == 0 ? h0[(i64)b * H + k] : h[(t - 1) * B * H + (i64)b * H + k];
  }
};
struct AdjA {  // A[m, g*H + i] = c_g[m, i] * lam[m, i]
  const float* lin; i64 lin_ks; const float *cr, *cz, *cn; i64 coef_ks; int B, H;
  __device__ float operator()(int m, int k) const {
    int kk = m / B, b = m % B, g = k / H, i = k - g * H;
    const float* c = g == 0 ? cr : (g == 1 ? cz : cn);
    return c[(i64)kk * coef_ks + (i64)b * H + i] * lin[(i64)kk * lin_ks + (i64)b * H + i];
  }
};

// ---------------------------------------------------------------- epilogues
struct BiasEpi {
  float* out; i64 ld; const float* bias;
  __device__ void operator()(int m, int n, const float* v) const { out[(i64)m * ld + n] = v[0] + bias[n]; }
};
struct StoreEpi {
  float* out; i64 ld;
  __device__ void operator()(int m, int n, const float* v) const { out[(i64)m * ld + n] = v[0]; }
};
struct FwdEpi {
  FwdStepArgs a;
  __device__ void operator()(int m, int n, const float* v) const {
    int k = m / a.B, b = m % a.B;
    const float* gi = a.gi + (i64)k * a.gi_ks + (i64)b * 3 * a.H;
    float hp = a.hin[(i64)k * a.hin_ks + (i64)b * a.H + n];
    float phi = cell_forward(gi[n], gi[a.H + n], gi[2 * a.H + n], v[0] + a.b_hh[n], v[1] + a.b_hh[a.H + n],
                             v[2] + a.b_hh[2 * a.H + n], hp, a.gamma, a.cell);
    float* o = a.hout + (i64)k * a.hout_ks + (i64)b * a.H + n;
    if (a.mode == 0) {
      if (a.gadd) phi += a.gadd[(i64)k * a.gadd_ks + (i64)b * a.H + n];
      *o = phi;
    } else {
      *o = *o - phi;
    }
  }
};
struct LinEpi {
  LinArgs a;
  __device__ void operator()(int m, int n, const float* v) const {
    int j1 = m / a.B, b = m % a.B;
    const i64 t = a.t0 + (i64)j1 * a.stride_t;        // fine time the step leaves from
    const float* gi = a.gi + ((t + a.stride_t - 1) * a.B + b) * 3 * a.H;
    float hp = t == 0 ? a.h0[(i64)b * a.H + n] : a.h[((t - 1) * a.B + b) * a.H + n];
    CellLin c = cell_linearise(gi[n], gi[a.H + n], gi[2 * a.H + n], v[0] + a.b_hh[n], v[1] + a.b_hh[a.H + n],
                               v[2] + a.b_hh[2 * a.H + n], hp, a.gamma, a.cell);
    i64 o = (i64)m * a.H + n;
    a.a[o] = c.a; a.cr[o] = c.cr; a.cz[o] = c.cz; a.cn[o] = c.cn;
    if (a.cnp) a.cnp[o] = c.cnp;
  }
};
struct AdjEpi {
  AdjStepArgs a;
  __device__ void operator()(int m, int n, const float* v) const {
    int k = m / a.B, b = m % a.B;
    float lam = a.lin[(i64)k * a.lin_ks + (i64)b * a.H + n];
    float val = a.a[(i64)k * a.coef_ks + (i64)b * a.H + n] * lam + v[0];
    float* o = a.lout + (i64)k * a.lout_ks + (i64)b * a.H + n;
    if (a.mode == 0) {
      if (a.gadd) val += a.gadd[(i64)k * a.gadd_ks + (i64)b * a.H + n];
      *o = val;
    } else {
      *o = *o - val;
    }
  }
};

// ---------------------------------------------------------------- Implicit LSTM (four gates)
struct LstmFwdEpi {
  LstmFwdArgs a;
  __device__ void operator()(int m, int n, const float* v) const {
    int k = m / a.B, b = m % a.B;
    const float* gi = a.gi + (i64)k * a.gi_ks + (i64)b * 4 * a.H;
    float cp = a.cin[(i64)k * a.in_ks + (i64)b * a.H + n];
    LstmOut o = lstm_forward(gi[n], gi[a.H + n], gi[2 * a.H + n], gi[3 * a.H + n], v[0] + a.b_hh[n], v[1] + a.b_hh[a.H + n],
                             v[2] + a.b_hh[2 * a.H + n], v[3] + a.b_hh[3 * a.H + n], cp, a.gamma, a.cell);
    a.cout[(i64)m * a.H + n] = o.c;
    a.hout[(i64)m * a.H + n] = o.h;
  }
};
struct LstmLinA {   // hidden state entering step j = m/B + 1: h at fine time t0 + stride*(j-1)
  const float* h0; const float* h; i64 ts, stride_t, t0; int B, H;
  __device__ float operator()(int m, int k) const {
    int j1 = m / B, b = m % B;
    const i64 t = t0 + (i64)j1 * stride_t;
    return t == 0 ? h0[(i64)b * H + k] : h[(t - 1) * ts + (i64)b * H + k];
  }
};
struct LstmLinEpi {
  LstmLinArgs a;
  __device__ void operator()(int m, int n, const float* v) const {
    int j1 = m / a.B, b = m % a.B;
    const i64 t = a.t0 + (i64)j1 * a.stride_t;
    const float* gi = a.gi + ((t + a.stride_t - 1) * a.B + b) * 4 * a.H;
    float cp = t == 0 ? a.c0[(i64)b * a.H + n] : a.c[(t - 1) * a.ts + (i64)b * a.H + n];
    LstmLin L = lstm_linearise(gi[n], gi[a.H + n], gi[2 * a.H + n], gi[3 * a.H + n], v[0] + a.b_hh[n], v[1] + a.b_hh[a.H + n],
                               v[2] + a.b_hh[2 * a.H + n], v[3] + a.b_hh[3 * a.H + n], cp, a.gamma, a.cell);
    i64 o = (i64)m * a.H + n;
    a.a[o] = L.a; a.p[o] = L.p; a.ci[o] = L.ci; a.cf[o] = L.cf; a.cg[o] = L.cg; a.co[o] = L.co;
  }
};
struct LstmAdjA {   // A[m, g*H + i] = coefficient_g * (g < 3 ? Lc + p*Lh : Lh)
  LstmAdjArgs a;
  __device__ float operator()(int m, int k) const {
    int kk = m / a.B, b = m % a.B, g = k / a.H, i = k - g * a.H;
    i64 ci = (i64)kk * a.coef_ks + (i64)b * a.H + i, li = (i64)kk * a.in_ks + (i64)b * a.H + i;
    float lh = a.lh[li];
    if (g == 3) return a.co[ci] * lh;
    float dc = a.lc[li] + a.p[ci] * lh;
    return (g == 0 ? a.ci[ci] : (g == 1 ? a.cf[ci] : a.cg[ci])) * dc;
  }
};
__global__ void __launch_bounds__(256) lstm_adj_c_kernel(LstmAdjArgs a) {
  i64 total = (i64)a.M * a.H;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / a.H; int i = (int)(e % a.H);
    i64 kk = m / a.B; int b = (int)(m % a.B);
    i64 ci = kk * a.coef_ks + (i64)b * a.H + i, li = kk * a.in_ks + (i64)b * a.H + i;
    a.lc_out[e] = a.a[ci] * (a.lc[li] + a.p[ci] * a.lh[li]);
  }
}
__global__ void __launch_bounds__(256) lstm_form_dA_kernel(const float* __restrict__ lc, const float* __restrict__ lh, i64 lam_ts, int B,
                                                           const float* __restrict__ p, const float* __restrict__ ci,
                                                           const float* __restrict__ cf, const float* __restrict__ cg,
                                                           const float* __restrict__ co, float* __restrict__ dA, i64 M, int H) {
  i64 total = M * H;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / H; int i = (int)(e % H);
    i64 t = m / B; int b = (int)(m % B);
    i64 li = t * lam_ts + (i64)b * H + i;
    float h = lh[li], dc = lc[li] + p[e] * h;
    float* d = dA + m * 4 * H + i;
    d[0] = ci[e] * dc; d[H] = cf[e] * dc; d[2 * H] = cg[e] * dc; d[3 * H] = co[e] * h;
  }
}

}  // namespace

void simt_lstm_fwd_step(const LstmFwdArgs& a, cudaStream_t s) {
  launch<4, true, true>(KC_FWD_STEP, a.M, a.H, a.H, StridedRowsA{a.hin, a.in_ks, a.B, a.H}, GateW{a.W_hh, a.H, a.H}, LstmFwdEpi{a}, s);
}
void simt_lstm_linearise(const LstmLinArgs& a, cudaStream_t s) {
  launch<4, true, true>(KC_LINEARISE, a.M, a.H, a.H, LstmLinA{a.h0, a.h, a.ts, a.stride_t, a.t0, a.B, a.H}, GateW{a.W_hh, a.H, a.H},
                        LstmLinEpi{a}, s);
}
void simt_lstm_adj_step(const LstmAdjArgs& a, cudaStream_t s) {
  i64 items = (i64)a.M * a.H;
  int grid = (int)((items + 255) / 256 < 1184 ? (items + 255) / 256 : 1184);
  lstm_adj_c_kernel<<<grid < 1 ? 1 : grid, 256, 0, s>>>(a);
  count_launch();
  launch<1, true, false>(KC_ADJ_STEP, a.M, a.H, 4 * a.H, LstmAdjA{a}, DenseBT{a.W_hh, a.H}, StoreEpi{a.lh_out, a.H}, s);
}
void simt_lstm_form_dA(const float* lc, const float* lh, i64 lam_ts, int B, const float* p, const float* ci, const float* cf,
                       const float* cg, const float* co, float* dA, i64 M, int H, cudaStream_t s) {
  i64 items = M * H;
  int grid = (int)((items + 255) / 256 < 1184 ? (items + 255) / 256 : 1184);
  lstm_form_dA_kernel<<<grid < 1 ? 1 : grid, 256, 0, s>>>(lc, lh, lam_ts, B, p, ci, cf, cg, co, dA, M, H);
  count_launch();
}

void simt_project(const float* x, const float* W_ih, const float* b_ih, float* gi, int M, int I, int H3, cudaStream_t s) {
  launch<1, true, true>(KC_PROJ, M, H3, I, DenseA{x, I}, DenseB{W_ih, I}, BiasEpi{gi, H3, b_ih}, s);
}

void simt_fwd_step(const FwdStepArgs& a, cudaStream_t s) {
  launch<3, true, true>(KC_FWD_STEP, a.M, a.H, a.H, StridedRowsA{a.hin, a.hin_ks, a.B, a.H}, GateW{a.W_hh, a.H, a.H}, FwdEpi{a}, s);
}

void simt_linearise(const LinArgs& a, cudaStream_t s) {
  launch<3, true, true>(KC_LINEARISE, a.M, a.H, a.H, LinA{a.h0, a.h, a.stride_t, a.t0, a.B, a.H}, GateW{a.W_hh, a.H, a.H}, LinEpi{a}, s);
}

void simt_adj_step(const AdjStepArgs& a, cudaStream_t s) {
  launch<1, true, false>(KC_ADJ_STEP, a.M, a.H, 3 * a.H, AdjA{a.lin, a.lin_ks, a.cr, a.cz, a.cn, a.coef_ks, a.B, a.H},
                         DenseBT{a.W_hh, a.H}, AdjEpi{a}, s);
}

void simt_wgrad(const float* dA, int M, int H3, const float* first, int Bfirst, const float* rest, int C, float* dW,
                cudaStream_t s) {
  launch<1, false, false>(KC_WGRAD, H3, C, M, DenseAT{dA, H3}, FirstRestBT{first, Bfirst, rest, C}, StoreEpi{dW, C}, s);
}

void simt_adj_dx(const AdjStepArgs& a, const float* W_ih, int C, float* out, cudaStream_t s) {
  launch<1, true, false>(KC_ADJ_STEP, a.M, C, 3 * a.H, AdjA{a.lin, a.lin_ks, a.cr, a.cz, a.cn, a.coef_ks, a.B, a.H}, DenseBT{W_ih, C},
                         StoreEpi{out, C}, s);
}

void simt_dgrad(const float* dA, int M, int H3, const float* W, int C, float* dx, cudaStream_t s) {
  launch<1, true, false>(KC_WGRAD, M, C, H3, DenseA{dA, H3}, DenseBT{W, C}, StoreEpi{dx, C}, s);
}

}  // namespace mg
