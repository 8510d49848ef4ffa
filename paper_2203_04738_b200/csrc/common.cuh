// Shared declarations of the library's translation units (host launchers and argument structs).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include <atomic>
#include <stdint.h>
#include <stddef.h>

#include "../../include/mgrit_gru.h"

namespace mg {

typedef long long i64;

// Every launch goes through this counter (reported by mgrit_gru_kernel_launches()).
extern std::atomic<unsigned long long> g_kernel_launches;
inline void count_launch(int n = 1) { g_kernel_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// Host-side caches that depend on the device (addresses of __device__ variables, function attributes, SM
// count) are kept per device ordinal and filled on the first call made with that device current.
constexpr int kMaxDevices = 64;
// ordinal of the current device, or -1 (no device / more than kMaxDevices)
inline int current_device_slot() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}
// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per (kernel instantiation, device); `done` is the
// instantiation's own per-device flag array
template <class K>
inline bool set_smem_once(K kern, int bytes, bool (&done)[kMaxDevices]) {
  const int dev = current_device_slot();
  if (dev < 0) return false;
  if (done[dev]) return true;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done[dev] = true;
  return true;
}

// Programmatic dependent launch: a kernel launched through launch_pdl() may become resident (and run its
// prologue: barrier set-up, TMEM allocation, descriptor prefetch) while its predecessor in the stream is
// still running.  Such a kernel calls pdl_wait() in EVERY thread before its first access to global memory
// (the wait returns once the predecessor has completed and its writes are visible), then pdl_trigger() to
// let its own successor start the same way.  At most two kernels overlap, and never their memory traffic.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// cluster_x > 1 launches thread-block clusters of that many CTAs along x (the grid must be a multiple).
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl_cluster(void (*kern)(KArgs...), int cluster_x, dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                      Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  if (cluster_x > 1) {
    at[1].id = cudaLaunchAttributeClusterDimension;
    at[1].val.clusterDim.x = (unsigned)cluster_x; at[1].val.clusterDim.y = 1; at[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  return launch_pdl_cluster(kern, 1, grid, block, smem, s, static_cast<Args&&>(args)...);
}
#endif

// Optional per-launch timing of the GEMM-shaped kernels (CUDA events on the launching stream).
enum KernelClass { KC_PROJ = 0, KC_FWD_STEP, KC_LINEARISE, KC_ADJ_STEP, KC_WGRAD, KC_FWD_SERIAL, KC_ADJ_SERIAL, KC_COUNT };
extern bool g_prof_on;
// prof_begin/prof_end bracket one record; records do not nest: a begin issued while a record is open (a GEMM
// launcher called from a function that times itself together with its operand-forming kernels) is ignored
// together with its matching end.
void prof_begin(int kc, double flops, cudaStream_t s);
void prof_end(cudaStream_t s);
struct ProfScope {
  cudaStream_t s;
  ProfScope(int kc, double flops, cudaStream_t st) : s(st) { prof_begin(kc, flops, st); }
  ~ProfScope() { prof_end(s); }
};

// ---- one forward cell evaluation for M = nk*B rows (Eq. "gru" + Eq. "gru-classic"/"gru-imap") ----
// Row m = (k, b): k = m / B, b = m % B.  All *_ks are strides per k in ELEMENTS (may be negative).
struct FwdStepArgs {
  int M, B, H;
  const float* hin;  i64 hin_ks;    // previous state rows      hin  + k*hin_ks  + b*H
  float* hout;       i64 hout_ks;   // result rows              hout + k*hout_ks + b*H
  const __nv_bfloat16* hin_b;       // bf16 copy of the previous state rows (same indexing) or nullptr
  __nv_bfloat16* hout_b;            // where to write the bf16 copy of the result (same indexing) or nullptr
  const float* gi;   i64 gi_ks;     // input projection rows    gi   + k*gi_ks   + b*3H
  const __nv_bfloat16* gi_b;        // bf16 copy of those rows (same indexing) or nullptr: what the fused tensor-core kernel stages
  const float* gadd; i64 gadd_ks;   // optional FAS term rows (same shape as hout) or nullptr
  const float* W_hh;                // [3H,H] fp32
  const float* b_hh;                // [3H]
  float gamma;                      // time step of the level: cf^l * dt
  int cell;                         // MGRIT_CELL_*
  int mode;                         // 0: hout = Phi + gadd ; 1: hout = hout - Phi   (FAS right-hand side)
};

// ---- a relaxation sweep: n dependent forward steps of one level over the same nk intervals, in ONE launch ----
// Slots of the level: point j = k*cf + s (interval k, slot s).  A step starts from slot coordinate in_s of every
// interval and arrives at target coordinate tgt_s, counted from slot 1 (tgt_s = cf - 1 is the C-point that closes
// the interval); its result goes to rows out + k*out_ks + b*H (and their bf16 copy).
struct FwdSweepStep {
  int in_s, tgt_s;
  float* out; i64 out_ks; __nv_bfloat16* out_b;
  int dep;       // 0: first step; 1: follows a step on the same intervals; 2: follows a step that advanced the C-points
                 // (reads what the neighbouring interval wrote); 3: advances the C-points (must not overtake their readers)
};
constexpr int kMaxFwdSweepSteps = 20;
struct FwdSweepArgs {
  int B, H, nk, cf, n;
  const float* U; const __nv_bfloat16* Ub;   // level state and its bf16 copy, from slot 0
  const float* gi; i64 gi_ss, gi_ks;         // input projection of target coordinate 0 of interval 0; element strides per slot / interval
  const __nv_bfloat16* gi_b;                 // its bf16 copy (same indexing) or nullptr
  const float* g;                            // FAS term of target coordinate 0 of interval 0 (slots like U), or nullptr
  const float* b_hh; float gamma; int cell;
  int* ctr;                                  // n * ceil(nk*B / 128) zeroed ints
  FwdSweepStep st[kMaxFwdSweepSteps];
};

// ---- adjoint coefficients of every step of one level (discrete adjoint of the cell) ----
// Row m = (j-1, b) for the level's forward steps j = 1..N_l; step j leaves fine time t0 + stride_t*(j-1) and arrives
// at t0 + stride_t*j with that time's input.  Outputs are [N_l*B, H] each.
struct LinArgs {
  int M, B, H;
  const float* h0;                  // [B,H]   state at fine time 0
  const float* h;                   // [T,B,H] fine states (h[k] = h_{k+1})
  i64 stride_t;                     // fine steps per level step: cf^l
  i64 t0;                           // fine time the level's first step leaves from (0 unless T is ragged)
  const float* gi;                  // [T,B,3H]
  const __nv_bfloat16* gi_b;        // its bf16 copy or nullptr (fused tensor-core kernel only)
  const float* W_hh; const float* b_hh;
  float gamma; int cell;
  float *a, *cr, *cz, *cn, *cnp;    // cnp may be nullptr (only level 0 needs it)
  // The tensor-core engine keeps the four gate coefficients in bf16 (they only ever enter bf16 operands;
  // `a`, which multiplies the carried sensitivity in fp32, stays fp32): it writes these and ignores the fp32 ones.
  __nv_bfloat16 *crb, *czb, *cnb, *cnpb;
};

// ---- one adjoint step for M = nk*B rows:  out = a*lam + [cr*lam | cz*lam | cn*lam] W_hh (+ gadd) ----
struct AdjStepArgs {
  int M, B, H;
  const float* lin;  i64 lin_ks;    // incoming sensitivity rows
  float* lout;       i64 lout_ks;
  const float* gadd; i64 gadd_ks;   // optional source / FAS term, same shape as lout
  const float *a, *cr, *cz, *cn; i64 coef_ks;   // coefficient rows (+k*coef_ks + b*H), already offset to k = 0
  const __nv_bfloat16 *crb, *czb, *cnb;         // the same rows in bf16 (tensor-core engine; same indexing)
  const float* W_hh;                // [3H,H] fp32
  int mode;                         // as FwdStepArgs
};

// ---- Implicit LSTM steps (state of a point = (c, h), 4H gate rows i | f | g | o); rows m = (k, b) as above ----
// Level-array update formed by the step kernel itself (tensor-core engines): the raw result of row (k, b) goes to
// out + k*out_ks + b*H (cell part; hidden part at + part) as raw + g (mode 0; g optional, same indexing with g_ks) or as
// (previous content) - raw (mode 1, FAS right-hand side).  out == nullptr: the raw results go to the contiguous
// [M, H] arrays of the step instead and the caller combines them.
struct LstmUpdate { float* out; i64 out_ks; const float* g; i64 g_ks; i64 part; int mode; };
struct LstmFwdArgs {
  int M, B, H;
  const float* cin; const float* hin; i64 in_ks;    // previous cell / hidden state rows (+ k*in_ks + b*H)
  float* cout; float* hout;                         // raw new states, contiguous [M, H] each
  const float* gi; i64 gi_ks;                       // input projection rows (+ k*gi_ks + b*4H)
  const float* W_hh; const float* b_hh;             // [4H, H], [4H]
  float gamma; int cell;
  LstmUpdate up;
};
// coefficients of every step of one level: step j = 1..N leaves fine time t0 + stride_t*(j-1); the given states are
// c/h[t] at c + (t-1)*ts / h + (t-1)*ts for t >= 1 and c0/h0 for t = 0; outputs [N*B, H] each
struct LstmLinArgs {
  int M, B, H;
  const float *c0, *h0, *c, *h; i64 ts;
  i64 stride_t, t0;
  const float* gi;                                  // [T, B, 4H]
  const float* W_hh; const float* b_hh; float gamma; int cell;
  float *a, *p, *ci, *cf, *cg, *co;
  __nv_bfloat16 *cib, *cfb, *cgb, *cob;             // bf16 engine: the four gate coefficients as bf16 instead (ci..co unused)
};
// one adjoint step: dc = Lc + p*Lh; lc_out = a*dc; lh_out = [ci*dc | cf*dc | cg*dc | co*Lh] W_hh   (raw, contiguous [M, H] each)
struct LstmAdjArgs {
  int M, B, H;
  const float* lc; const float* lh; i64 in_ks;      // incoming sensitivities rows
  float* lc_out; float* lh_out;
  const float *a, *p, *ci, *cf, *cg, *co; i64 coef_ks;
  const __nv_bfloat16 *cib, *cfb, *cgb, *cob;       // bf16 engine: the four gate coefficients as bf16 instead (ci..co unused)
  const float* W_hh;
  LstmUpdate up;
};
void simt_lstm_fwd_step(const LstmFwdArgs& a, cudaStream_t s);
void simt_lstm_linearise(const LstmLinArgs& a, cudaStream_t s);
void simt_lstm_adj_step(const LstmAdjArgs& a, cudaStream_t s);
// dA[m, :] = [ci*dc | cf*dc | cg*dc | co*Lh] for M contiguous rows (gradient pass); lam rows (c, h) at lc/lh + m-row stride lam_ks per time
void simt_lstm_form_dA(const float* lc, const float* lh, i64 lam_ts, int B, const float* p, const float* ci, const float* cf,
                       const float* cg, const float* co, float* dA, i64 M, int H, cudaStream_t s);

// SIMT (fp32 FFMA) engine
void simt_project(const float* x, const float* W_ih, const float* b_ih, float* gi, int M, int I, int H3, cudaStream_t s);
void simt_fwd_step(const FwdStepArgs& a, cudaStream_t s);
void simt_linearise(const LinArgs& a, cudaStream_t s);
void simt_adj_step(const AdjStepArgs& a, cudaStream_t s);
// dW[n3, c] = sum_m dA[m, n3] * R[m, c],  R rows: m < B ? first[m] : rest[m-B]   (first may be nullptr with B = 0)
void simt_wgrad(const float* dA, int M, int H3, const float* first, int Bfirst, const float* rest, int C, float* dW, cudaStream_t s);
// dx[m, c] = sum_n3 dA[m, n3] * W[n3, c]
void simt_dgrad(const float* dA, int M, int H3, const float* W, int C, float* dx, cudaStream_t s);
// out[m, c] = sum_{g,i} (c_g * lam)[m, i] W_ih[g*H + i, c]: what the step described by `a` (its cn slot holding c_n') sends to
// the input of its cell, contiguous rows [M, C]
void simt_adj_dx(const AdjStepArgs& a, const float* W_ih, int C, float* out, cudaStream_t s);

// streaming kernels
// r = uC - v at the C-points, sum of squares into *acc (double, device), copy of the C-point state
// to the coarse level:   uc[k] = uf[cf*k],  k = 1..nc   (rows of rowlen = B*H floats)
// ucb / ufb: optional bf16 copies of the written rows (same indexing), nullptr to skip
void stream_restrict_residual(const float* uf, int cf, const float* v, float* uc, __nv_bfloat16* ucb, int nc, i64 rowlen, double* acc, cudaStream_t s);
void stream_correct(float* uf, __nv_bfloat16* ufb, int cf, const float* uc, int nc, i64 rowlen, cudaStream_t s);
// dst[k] = src[k*src_ks], k = 0..nk-1, rows of rowlen floats (src_ks in elements, may be negative)
void stream_gather_rows(float* dst, i64 dst_ks, const float* src, i64 src_ks, int nk, i64 rowlen, cudaStream_t s);
void stream_add_rows(float* dst, const float* src, i64 n, cudaStream_t s);
// tmp[M, H] contiguous (rows (k, b)) -> dst rows at dst + k*dst_ks + b*H: mode 0 dst = tmp (+ g rows, same indexing with g_ks),
// mode 1 dst = dst - tmp
void stream_combine_rows(const float* tmp, const float* g, i64 g_ks, float* dst, i64 dst_ks, int B, int H, i64 M, int mode, cudaStream_t s);
// dA_h = [cr*lam | cz*lam | cn*lam], dA_i = [cr*lam | cz*lam | cnp*lam]  for M rows of H
void stream_form_dA(const float* lam, const float* cr, const float* cz, const float* cn, const float* cnp,
                    float* dA_h, float* dA_i, i64 M, int H, cudaStream_t s);
void stream_colsum(const float* A, i64 M, int N, float* out, cudaStream_t s);
void stream_sqrt_to_float(const double* acc, float* out, int n, cudaStream_t s);
void stream_xent(int B, int H, int C, const float* hT, const float* Wc, const float* bc, const int32_t* labels,
                 float* loss, float* dhT, float* dWc, float* dbc, float* dlogits, cudaStream_t s);
void stream_sgd(float* p, const float* g, size_t n, float lr, cudaStream_t s);
void stream_adam(float* p, const float* g, float* m, float* v, size_t n, float lr, float b1, float b2, float eps, int step,
                 cudaStream_t s);

}  // namespace mg
