// C ABI, argument validation, workspace layout and the host side of the multigrid cycle.
// The cycle logic is written once over an abstract "step" and instantiated for the forward
// recurrence and for its adjoint; every step, transfer and reduction is a kernel launch.
#include <limits.h>
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <vector>

#include "common.cuh"
#include "serial_engine.cuh"
#include "umma_engine.cuh"

namespace mg {

std::atomic<unsigned long long> g_kernel_launches{0};
bool g_prof_on = false;

namespace {
struct ProfRec { int kc; double flops; cudaEvent_t e0, e1; };
std::vector<ProfRec> g_prof_recs;
std::vector<cudaEvent_t> g_prof_pool;
cudaEvent_t prof_event() {
  cudaEvent_t e = nullptr;
  if (!g_prof_pool.empty()) { e = g_prof_pool.back(); g_prof_pool.pop_back(); }
  else cudaEventCreate(&e);
  return e;
}
}  // namespace

static int g_prof_depth = 0;
void prof_begin(int kc, double flops, cudaStream_t s) {
  if (!g_prof_on) return;
  if (g_prof_depth++ > 0) return;     // inside an open record
  ProfRec r{kc, flops, prof_event(), prof_event()};
  cudaEventRecord(r.e0, s);
  g_prof_recs.push_back(r);
}
void prof_end(cudaStream_t s) {
  if (!g_prof_on || g_prof_depth == 0) return;
  if (--g_prof_depth > 0 || g_prof_recs.empty()) return;
  cudaEventRecord(g_prof_recs.back().e1, s);
}

namespace {

constexpr int kMaxLevels = 16;

struct Ws {  // bump allocator over the caller's workspace; base == nullptr only counts bytes
  char* base; size_t size; size_t off;
  template <class T> T* take(size_t n) {
    size_t bytes = (n * sizeof(T) + 255) & ~(size_t)255;
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += bytes;
    return p;
  }
  bool fits() const { return base == nullptr || off <= size; }
};

struct Hier {
  int L; int N[kMaxLevels]; i64 stride_t[kMaxLevels]; float gamma[kMaxLevels];
  i64 rem[kMaxLevels];   // T - stride_t * N: fine steps before the first reversed (adjoint) point of the level; 0 unless T is ragged
};

// every data pointer must be 32-byte aligned (nullptr passes: optional arguments are checked for presence elsewhere)
template <class... P>
bool aligned32(P... ptrs) {
  uintptr_t m = 0;
  ((m |= (uintptr_t)(const void*)ptrs), ...);
  return (m & 31u) == 0;
}

inline bool is_tf32(const mgrit_gru_cfg* c) { return c->operands == MGRIT_OPERANDS_TF32 || c->operands == MGRIT_OPERANDS_TF32_1PASS; }

int check_cfg(const mgrit_gru_cfg* c, Hier* hr) {
  if (!c) return MGRIT_INVALID_ARG;
  if (c->T <= 0 || c->B <= 0 || c->I <= 0 || c->H <= 0 || c->levels < 1 || c->levels > kMaxLevels) return MGRIT_INVALID_ARG;
  if (c->levels > 1 && (c->cf < 2 || c->iters < 0)) return MGRIT_INVALID_ARG;
  if (c->cell != MGRIT_CELL_CLASSIC && c->cell != MGRIT_CELL_IMPLICIT) return MGRIT_INVALID_ARG;
  if (c->relax_fine < MGRIT_RELAX_F || c->relax_fine > MGRIT_RELAX_MAX) return MGRIT_INVALID_ARG;
  if (c->relax_coarse < MGRIT_RELAX_F || c->relax_coarse > MGRIT_RELAX_MAX) return MGRIT_INVALID_ARG;
  if (c->operands < MGRIT_OPERANDS_FP32 || c->operands > MGRIT_OPERANDS_TF32_1PASS) return MGRIT_INVALID_ARG;
  if (!(c->dt > 0.f)) return MGRIT_INVALID_ARG;
  if (c->H % 8 != 0 || c->I % 8 != 0) return MGRIT_UNSUPPORTED;
  // row counts (T+1)*B, widths and grid sizes are 32-bit inside the kernels; element offsets are 64-bit
  if (((i64)c->T + 1) * c->B > (i64)INT_MAX - 1024 || (i64)3 * c->H > INT_MAX / 4 || c->I > INT_MAX / 4) return MGRIT_UNSUPPORTED;
  i64 m = 1;
  hr->L = c->levels;
  const bool ragged = (c->flags & MGRIT_FLAG_RAGGED_T) != 0;
  for (int l = 0; l < c->levels; ++l) {
    // ragged: the C-points of a level are its points 0, cf, 2 cf, ...; N_{l+1} = floor(N_l / cf) = floor(T / cf^(l+1))
    if (!ragged && c->T % m != 0) return MGRIT_NOT_DIVISIBLE;
    hr->N[l] = (int)(c->T / m);
    hr->stride_t[l] = m;
    hr->gamma[l] = (float)m * c->dt;
    hr->rem[l] = c->T - m * hr->N[l];
    if (l + 1 < c->levels) {
      m *= c->cf;
      if (m > c->T) return MGRIT_NOT_DIVISIBLE;
    }
  }
  if (c->operands == MGRIT_OPERANDS_BF16) {
    int rc = umma_supported(c);
    if (rc != MGRIT_OK) return rc;
  }
  if (is_tf32(c)) {
    int rc = tf32_supported(c);
    if (rc != MGRIT_OK) return rc;
  }
  return MGRIT_OK;
}

// With MGRIT_FLAG_GI_CARRIES_COPIES the caller's gi buffer is followed by the bf16 copies that the forward call makes
// anyway and the adjoint call needs again: x as [T*B, I] and the level-0 state [h_0; h] as [(T+1)*B, H].
struct GiTail { __nv_bfloat16* xb; __nv_bfloat16* hb0; __nv_bfloat16* gib; size_t total_bytes; };
GiTail gi_tail(const mgrit_gru_cfg* c, float* gi) {
  const size_t TB = (size_t)c->T * c->B;
  size_t off = (TB * 3 * c->H * sizeof(float) + 255) & ~(size_t)255;
  GiTail t;
  t.xb = gi ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(gi) + off) : nullptr;
  off += (TB * c->I * sizeof(__nv_bfloat16) + 255) & ~(size_t)255;
  t.hb0 = gi ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(gi) + off) : nullptr;
  off += ((TB + c->B) * c->H * sizeof(__nv_bfloat16) + 255) & ~(size_t)255;
  t.gib = gi ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<char*>(gi) + off) : nullptr;      // the projection itself as bf16
  off += (TB * 3 * c->H * sizeof(__nv_bfloat16) + 255) & ~(size_t)255;
  t.total_bytes = off;
  return t;
}
// the copies exist when the tensor-core engine keeps bf16 shadows of the level states (B divides 128) in an MGRIT solve
bool carries_copies(const mgrit_gru_cfg* c, bool serial) {
  return !serial && (c->flags & MGRIT_FLAG_GI_CARRIES_COPIES) && c->operands == MGRIT_OPERANDS_BF16 && 128 % c->B == 0 && c->levels > 1;
}

// MGRIT_GRU_GI_BF16=0 in the environment keeps the fused kernels on the fp32 input projection (A/B measurements).
bool gi_bf16_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_GI_BF16"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

struct FwdWs {
  float* U[kMaxLevels]; float* G[kMaxLevels]; double* res_acc; UmmaFwdWs um; Tf32Ws tf;
  __nv_bfloat16* chain_ub; unsigned* chain_bar; uint4* chain_xw; size_t chain_xw_bytes;   // scratch of the persistent serial-chain kernel
  __nv_bfloat16* Ub[kMaxLevels];                  // bf16 copies of the level states (tensor-core A operands)
  int* sweep_ctr; size_t sweep_ctr_n, sweep_ctr_used;   // progress counters of the multi-step relaxation launches (zeroed per call)
};
struct AdjWs {
  float* U[kMaxLevels]; float* G[kMaxLevels];
  float *a[kMaxLevels], *cr[kMaxLevels], *cz[kMaxLevels], *cn[kMaxLevels], *cnp;   // gate coefficients: fp32 engine
  __nv_bfloat16 *crb[kMaxLevels], *czb[kMaxLevels], *cnb[kMaxLevels], *cnpb;       // ... tensor-core engine (bf16)
  float *dA_h, *dA_i, *lam_tmp; double* res_acc; UmmaAdjWs um; Tf32Ws tf;
  __nv_bfloat16* chain_dAb; unsigned* chain_bar; uint4* chain_xw; size_t chain_xw_bytes;
  float* chain_dA32;        // fp32 chain: [2][B][3H] operand exchange
};

void plan_fwd(const mgrit_gru_cfg* c, const Hier& hr, Ws& w, FwdWs* o) {
  size_t BH = (size_t)c->B * c->H;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * BH);
    o->G[l] = l == 0 ? nullptr : w.take<float>((size_t)(hr.N[l] + 1) * BH);
  }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  o->chain_ub = nullptr; o->chain_bar = nullptr; o->chain_xw = nullptr; o->chain_xw_bytes = 0;
  o->sweep_ctr = nullptr; o->sweep_ctr_n = o->sweep_ctr_used = 0;
  for (int l = 0; l < kMaxLevels; ++l) o->Ub[l] = nullptr;
  if (c->operands == MGRIT_OPERANDS_BF16) {
    umma_plan_fwd(c, hr.N, hr.L, w.base, &w.off, &o->um);
    for (int l = 0; l < hr.L; ++l) o->Ub[l] = w.take<__nv_bfloat16>((size_t)(hr.N[l] + 1) * BH);
    o->chain_ub = w.take<__nv_bfloat16>(2 * BH);
    o->chain_bar = w.take<unsigned>(((size_t)c->B / 16 + 1) * ((size_t)c->H / 8) + 64);
    o->chain_xw_bytes = serial_xw_bytes(c->B, c->H, 1);
    o->chain_xw = reinterpret_cast<uint4*>(w.take<char>(o->chain_xw_bytes));
    o->sweep_ctr_n = 1 << 16;
    o->sweep_ctr = w.take<int>(o->sweep_ctr_n);
  } else {
    o->chain_bar = w.take<unsigned>((size_t)c->B / 16 + 64);
  }
  if (is_tf32(c)) tf32_plan_fwd(c, hr.N, hr.L, w.base, &w.off, &o->tf);
}

void plan_adj(const mgrit_gru_cfg* c, const Hier& hr, Ws& w, AdjWs* o) {
  size_t BH = (size_t)c->B * c->H;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * BH);
    o->G[l] = w.take<float>((size_t)(hr.N[l] + 1) * BH);
    o->a[l] = w.take<float>((size_t)hr.N[l] * BH);
    if (c->operands == MGRIT_OPERANDS_BF16) {
      o->cr[l] = o->cz[l] = o->cn[l] = nullptr;
      o->crb[l] = w.take<__nv_bfloat16>((size_t)hr.N[l] * BH);
      o->czb[l] = w.take<__nv_bfloat16>((size_t)hr.N[l] * BH);
      o->cnb[l] = w.take<__nv_bfloat16>((size_t)hr.N[l] * BH);
    } else {
      o->crb[l] = o->czb[l] = o->cnb[l] = nullptr;
      o->cr[l] = w.take<float>((size_t)hr.N[l] * BH);
      o->cz[l] = w.take<float>((size_t)hr.N[l] * BH);
      o->cn[l] = w.take<float>((size_t)hr.N[l] * BH);
    }
  }
  if (c->operands == MGRIT_OPERANDS_BF16) { o->cnp = nullptr; o->cnpb = w.take<__nv_bfloat16>((size_t)hr.N[0] * BH); }
  else { o->cnpb = nullptr; o->cnp = w.take<float>((size_t)hr.N[0] * BH); }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  if (c->operands == MGRIT_OPERANDS_BF16) {
    o->dA_h = o->dA_i = o->lam_tmp = nullptr;
    umma_plan_adj(c, hr.N, hr.L, w.base, &w.off, &o->um);
    o->chain_dA32 = nullptr;
    o->chain_dAb = w.take<__nv_bfloat16>(6 * BH);
    o->chain_bar = w.take<unsigned>(((size_t)c->B / 16 + 1) * ((size_t)c->H / 8) + 64);
    o->chain_xw_bytes = serial_xw_bytes(c->B, c->H, 3);
    o->chain_xw = reinterpret_cast<uint4*>(w.take<char>(o->chain_xw_bytes));
  } else {
    o->chain_dAb = nullptr; o->chain_xw = nullptr; o->chain_xw_bytes = 0;
    o->chain_bar = w.take<unsigned>((size_t)c->B / 16 + 64);
    o->chain_dA32 = w.take<float>(6 * BH);
    o->dA_h = w.take<float>((size_t)c->T * BH * 3);
    o->dA_i = w.take<float>((size_t)c->T * BH * 3);
    o->lam_tmp = w.take<float>((size_t)c->T * BH);     // lambda in forward order when the caller wants no dh
  }
  if (is_tf32(c)) tf32_plan_adj(c, hr.N, hr.L, w.base, &w.off, &o->tf);
}

// One launch of "advance nk*B rows by one step of level l".
struct StepDesc {
  int l, nk;
  int in_slot, in_stride;                 // source slots in U[l]
  float* out; int out_slot, out_stride;   // destination array (slot-major [.,B,H]) and slots
  const float* gadd; int gadd_slot, gadd_stride;
  int tgt_slot, tgt_stride;               // level-l point the step arrives at (selects input / coefficients)
  int mode;
};

// The multigrid cycle (Algorithm "MGProp" with the recursive coarse solve of the remark
// "Beyond Two-Level"), FAS form: level l solves u_j = step_l(u_{j-1}) + g_j.
struct Cycle {
  const mgrit_gru_cfg* c; Hier hr; cudaStream_t s;
  float** U; float** G; double* res_acc; int cycle_idx = 0;
  __nv_bfloat16** Ub = nullptr;   // optional bf16 copies of U (kept in step with every writer)
  size_t BH;
  int rc = MGRIT_OK;              // first failure of a launch (a step that cannot be prepared or launched)
  virtual int launch_step(const StepDesc& d) = 0;
  void step(const StepDesc& d) {
    if (rc != MGRIT_OK) return;   // after a failure nothing more is enqueued: outputs are undefined
    rc = launch_step(d);
  }
  // all N_l dependent steps of level l in one persistent launch; false = not available here
  virtual bool chain(int l) { (void)l; return false; }
  // A relaxation sweep of level l in one launch: kinds[i] = s in 1..cf-1: F-step to slot s of every interval;
  // cf: C-step; cf + 1: the step that evaluates v at the C-points into G[l+1].  false = not available here.
  virtual bool launch_sweep(int l, const int* kinds, int n) { (void)l; (void)kinds; (void)n; return false; }
  // F (CF)^relax (the opening F optional), optionally followed by the evaluation of v at the C-points
  bool relax_sweep(int l, bool first_f, int relax, bool with_v) {
    if (rc != MGRIT_OK) return true;
    int kinds[64], n = 0;
    const int cf = c->cf;
    if ((cf - 1) * (relax + 1) + relax + 1 > 64) return false;
    if (first_f) for (int sI = 1; sI < cf; ++sI) kinds[n++] = sI;
    for (int r = 0; r < relax; ++r) { kinds[n++] = cf; for (int sI = 1; sI < cf; ++sI) kinds[n++] = sI; }
    if (with_v) kinds[n++] = cf + 1;
    if (n < 2) return false;
    return launch_sweep(l, kinds, n);
  }
  virtual ~Cycle() {}

  // F-relaxation: from every C-point the cf - 1 F-points of its interval, one dependent step per launch over all
  // intervals; a ragged level has one more, shorter interval of N % cf F-points behind its last C-point.
  void frelax(int l) {
    int cf = c->cf, nki = hr.N[l] / cf, tail = hr.N[l] % cf;
    for (int sI = 1; sI < cf; ++sI)
      step(StepDesc{l, nki + (sI <= tail ? 1 : 0), sI - 1, cf, U[l], sI, cf, G[l], sI, cf, sI, cf, 0});
  }
  void crelax(int l) {
    int cf = c->cf, nki = hr.N[l] / cf;
    step(StepDesc{l, nki, cf - 1, cf, U[l], cf, cf, G[l], cf, cf, cf, cf, 0});
  }
  // One cycle from level l down.  skip_first_f: the state of level l was F-relaxed last and no C-point has changed
  // since, so the opening F-relaxation would reproduce it bit for bit.  record: store the level-0 residual norm.
  void cycle(int l, bool skip_first_f, bool record) {
    int cf = c->cf, N = hr.N[l];
    if (l == hr.L - 1) {  // coarsest level: serial propagation
      if (chain(l)) return;
      for (int j = 1; j <= N; ++j) step(StepDesc{l, 1, j - 1, 1, U[l], j, 1, G[l], j, 1, j, 1, 0});
      return;
    }
    int relax = l == 0 ? c->relax_fine : c->relax_coarse;       // n: F (CF)^n
    int nc = hr.N[l + 1];
    if (!relax_sweep(l, !skip_first_f, relax, true)) {
      if (!skip_first_f) frelax(l);
      for (int n = 0; n < relax; ++n) { crelax(l); frelax(l); }
      // v_k = step_l(u_{cf k - 1}) + g_{cf k}  ->  G[l+1][k]
      step(StepDesc{l, nc, cf - 1, cf, G[l + 1], 1, 1, G[l], cf, cf, cf, cf, 0});
    }
    // r_k = u_{cf k} - v_k ; U'_k = u_{cf k}
    stream_restrict_residual(U[l], cf, G[l + 1], U[l + 1], Ub ? Ub[l + 1] : nullptr, nc, (i64)BH,
                             (l == 0 && record) ? res_acc + cycle_idx : nullptr, s);
    // G_k = v_k - step_{l+1}(U'_{k-1})
    step(StepDesc{l + 1, nc, 0, 1, G[l + 1], 1, 1, nullptr, 0, 0, 1, 1, 1});
    cycle(l + 1, false, false);
    stream_correct(U[l], Ub ? Ub[l] : nullptr, cf, U[l + 1], nc, (i64)BH, s);
    if (!relax_sweep(l, true, 0, false)) frelax(l);
    // F-cycle: one more V-cycle from this level down on the corrected state (on the last two levels: a second
    // V-cycle).  Its opening F-relaxation would repeat the one just done.
    if ((c->flags & MGRIT_FLAG_F_CYCLE) && fcycle_leg) {
      const bool saved = fcycle_leg;
      fcycle_leg = false;
      cycle(l, true, false);
      fcycle_leg = saved;
    }
  }
  bool fcycle_leg = true;     // false while a trailing V-cycle of an F-cycle runs (it does not spawn further ones)
  int solve() {
    if (hr.L == 1) { cycle(0, false, false); return rc; }
    cudaMemsetAsync(res_acc, 0, sizeof(double) * (size_t)(c->iters > 0 ? c->iters : 1), s);
    for (cycle_idx = 0; cycle_idx < c->iters && rc == MGRIT_OK; ++cycle_idx) {
      // the previous cycle ended with an F-relaxation of level 0: the caller may ask not to repeat it
      const bool dup = cycle_idx > 0 && (c->flags & MGRIT_FLAG_SKIP_DUPLICATE_FRELAX);
      cycle(0, dup, true);
    }
    return rc;
  }
};

struct FwdCycle : Cycle {
  const gru_params* p; const float* gi; UmmaFwdWs* um; FwdWs* fw;
  const __nv_bfloat16* gib = nullptr;   // bf16 copy of gi: what every kernel of the solve reads when the state copies exist
  bool gi_f32 = true;                   // false: the fp32 projection was not written (MGRIT_FLAG_GI_F32_UNUSED); gib is set

  bool chain(int l) override {
    if (c->operands != MGRIT_OPERANDS_BF16) {     // fp32 and tf32 modes: the chain in FFMA arithmetic
      if (!fw->chain_bar) return false;
      Serial32FwdArgs a;
      a.B = c->B; a.H = c->H; a.nsteps = hr.N[l]; a.u = U[l];
      const i64 st = hr.stride_t[l];
      a.gi = gi + (st - 1) * (i64)BH * 3; a.gi_step = st * (i64)BH * 3;
      a.g = G[l]; a.W = p->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c->cell; a.bar = fw->chain_bar;
      return serial32_fwd_solve(a, s);
    }
    if (!fw->chain_ub) return false;
    SerialFwdArgs a{};
    a.B = c->B; a.H = c->H; a.nsteps = hr.N[l];
    a.u = U[l]; a.ub = fw->chain_ub;
    i64 st = hr.stride_t[l];
    a.gi = gi + (st - 1) * (i64)BH * 3; a.gi_step = st * (i64)BH * 3;
    // (the plain serial sweep has no other level to stay consistent with: it uses the fp32 projection as it is)
    a.gi_as_bf16 = (gib && hr.L > 1) ? 1 : 0;
    if (!gi_f32) { a.gi_b = gib + (st - 1) * (i64)BH * 3; a.gi = nullptr; }
    a.g = G[l]; a.W = um->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c->cell; a.bar = fw->chain_bar;
    a.xw = fw->chain_xw; a.xw_bytes = fw->chain_xw_bytes;
    return serial_fwd_solve(a, s);
  }
  bool launch_sweep(int l, const int* kinds, int n) override {
    const int cf = c->cf;
    if (c->operands != MGRIT_OPERANDS_BF16 || !Ub || hr.N[l] % cf != 0 || n > kMaxFwdSweepSteps) return false;
    FwdSweepArgs a{};
    a.B = c->B; a.H = c->H; a.nk = hr.N[l] / cf; a.cf = cf; a.n = n;
    const size_t need = (size_t)n * (((size_t)a.nk * c->B + 127) / 128);
    if (!fw->sweep_ctr || fw->sweep_ctr_used + need > fw->sweep_ctr_n) return false;
    a.U = U[l]; a.Ub = Ub[l];
    const i64 st = hr.stride_t[l];
    a.gi = gi + (st - 1) * (i64)BH * 3; a.gi_ss = st * (i64)BH * 3; a.gi_ks = st * cf * (i64)BH * 3;
    a.gi_b = gib ? gib + (st - 1) * (i64)BH * 3 : nullptr;
    a.g = G[l] ? G[l] + BH : nullptr;
    a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c->cell;
    a.ctr = fw->sweep_ctr + fw->sweep_ctr_used;
    for (int i = 0; i < n; ++i) {
      FwdSweepStep& q = a.st[i];
      const int kd = kinds[i], prev = i ? kinds[i - 1] : 0;
      if (kd < cf) {             // F-step to slot kd
        q.in_s = kd - 1; q.tgt_s = kd - 1;
        q.out = U[l] + (size_t)kd * BH; q.out_ks = (i64)cf * BH; q.out_b = Ub[l] + (size_t)kd * BH;
        q.dep = prev == cf ? 2 : 1;
      } else if (kd == cf) {     // C-step: slot cf of interval k = slot 0 of interval k + 1
        q.in_s = cf - 1; q.tgt_s = cf - 1;
        q.out = U[l] + (size_t)cf * BH; q.out_ks = (i64)cf * BH; q.out_b = Ub[l] + (size_t)cf * BH;
        q.dep = 3;
      } else {                   // v at the C-points, into the coarse level's G
        q.in_s = cf - 1; q.tgt_s = cf - 1;
        q.out = G[l + 1] + BH; q.out_ks = (i64)BH; q.out_b = nullptr;
        q.dep = 1;
      }
    }
    const int r = umma_fwd_sweep(a, um, s);
    if (r == MGRIT_UNSUPPORTED) return false;
    fw->sweep_ctr_used += need;
    if (r != MGRIT_OK) rc = r;
    return true;
  }
  int launch_step(const StepDesc& d) override {
    FwdStepArgs a{};
    a.M = d.nk * c->B; a.B = c->B; a.H = c->H;
    a.hin = U[d.l] + (size_t)d.in_slot * BH; a.hin_ks = (i64)d.in_stride * BH;
    a.hout = d.out + (size_t)d.out_slot * BH; a.hout_ks = (i64)d.out_stride * BH;
    a.hin_b = Ub ? Ub[d.l] + (size_t)d.in_slot * BH : nullptr;
    a.hout_b = (Ub && d.out == U[d.l]) ? Ub[d.l] + (size_t)d.out_slot * BH : nullptr;
    i64 st = hr.stride_t[d.l];
    a.gi = gi + ((i64)st * d.tgt_slot - 1) * (i64)BH * 3; a.gi_ks = st * d.tgt_stride * (i64)BH * 3;
    a.gi_b = gib ? gib + ((i64)st * d.tgt_slot - 1) * (i64)BH * 3 : nullptr;
    a.gadd = d.gadd ? d.gadd + (size_t)d.gadd_slot * BH : nullptr; a.gadd_ks = (i64)d.gadd_stride * BH;
    a.W_hh = p->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[d.l]; a.cell = c->cell; a.mode = d.mode;
    if (c->operands == MGRIT_OPERANDS_BF16) return umma_fwd_step(a, um, s);
    if (is_tf32(c)) return tf32_fwd_step(a, &fw->tf, s);
    simt_fwd_step(a, s);
    return MGRIT_OK;
  }
};

struct AdjCycle : Cycle {
  const gru_params* p; AdjWs* w;
  bool chain(int l) override {
    if (c->operands != MGRIT_OPERANDS_BF16) {
      if (!w->chain_bar || !w->chain_dA32) return false;
      Serial32AdjArgs a;
      a.B = c->B; a.H = c->H; a.nsteps = hr.N[l]; a.mu = U[l]; a.dA = w->chain_dA32;
      const i64 row0 = (i64)(hr.N[l] - 1) * BH;    // step s = 1 applies forward step N_l, stored at row N_l - 1
      a.a = w->a[l] + row0; a.cr = w->cr[l] + row0; a.cz = w->cz[l] + row0; a.cn = w->cn[l] + row0;
      a.coef_step = -(i64)BH;
      a.g = G[l]; a.W = p->W_hh; a.bar = w->chain_bar;
      return serial32_adj_solve(a, s);
    }
    if (!w->chain_dAb) return false;
    SerialAdjArgs a;
    a.B = c->B; a.H = c->H; a.nsteps = hr.N[l];
    a.mu = U[l]; a.dAb = w->chain_dAb;
    i64 row0 = (i64)(hr.N[l] - 1) * BH;        // step s = 1 applies forward step N_l, stored at row N_l - 1
    a.a = w->a[l] + row0; a.cr = w->crb[l] + row0; a.cz = w->czb[l] + row0; a.cn = w->cnb[l] + row0;
    a.coef_step = -(i64)BH;
    a.g = G[l]; a.WT = w->um.W_hhT; a.bar = w->chain_bar;
    a.xw = w->chain_xw; a.xw_bytes = w->chain_xw_bytes;
    return serial_adj_solve(a, s);
  }
  int launch_step(const StepDesc& d) override {
    AdjStepArgs a;
    a.M = d.nk * c->B; a.B = c->B; a.H = c->H;
    a.lin = U[d.l] + (size_t)d.in_slot * BH; a.lin_ks = (i64)d.in_stride * BH;
    a.lout = d.out + (size_t)d.out_slot * BH; a.lout_ks = (i64)d.out_stride * BH;
    a.gadd = d.gadd ? d.gadd + (size_t)d.gadd_slot * BH : nullptr; a.gadd_ks = (i64)d.gadd_stride * BH;
    // the step arriving at reversed point s applies forward step j = N_l - s + 1, stored at row N_l - s
    i64 row0 = (i64)(hr.N[d.l] - d.tgt_slot) * BH;
    a.a = w->a[d.l] + row0;
    if (c->operands == MGRIT_OPERANDS_BF16) {
      a.cr = a.cz = a.cn = nullptr;
      a.crb = w->crb[d.l] + row0; a.czb = w->czb[d.l] + row0; a.cnb = w->cnb[d.l] + row0;
    } else {
      a.crb = a.czb = a.cnb = nullptr;
      a.cr = w->cr[d.l] + row0; a.cz = w->cz[d.l] + row0; a.cn = w->cn[d.l] + row0;
    }
    a.coef_ks = -(i64)d.tgt_stride * BH;
    a.W_hh = p->W_hh; a.mode = d.mode;
    if (c->operands == MGRIT_OPERANDS_BF16) return umma_adj_step(a, &w->um, s);
    if (is_tf32(c)) return tf32_adj_step(a, &w->tf, s);
    simt_adj_step(a, s);
    return MGRIT_OK;
  }
};

// Zero initial guess of a level-0 array [T + 1 slots of `slot` elements] behind its fixed slot 0.  In a multigrid solve
// with at least one cycle only the C-points are read before they are written (the first F-relaxation fills every
// F-point from them), so only those slots are cleared: 1 / cf of the memory traffic.
template <class T>
void zero_guess(T* U0, const mgrit_gru_cfg& c, const Hier& hr, size_t slot, cudaStream_t s) {
  if (hr.L > 1 && c.iters > 0 && c.cf > 1 && c.T / c.cf > 0) {
    cudaMemset2DAsync(U0 + (size_t)c.cf * slot, (size_t)c.cf * slot * sizeof(T), 0, slot * sizeof(T), (size_t)(c.T / c.cf), s);
  } else {
    cudaMemsetAsync(U0 + slot, 0, sizeof(T) * (size_t)c.T * slot, s);
  }
}

int finish(cudaStream_t s, bool sync) {
  if (sync && cudaStreamSynchronize(s) != cudaSuccess) return MGRIT_CUDA_ERROR;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { fprintf(stderr, "mgrit_gru: CUDA error: %s\n", cudaGetErrorString(e)); return MGRIT_CUDA_ERROR; }
  if (sync && (umma_device_status() != 0 || serial_device_status() != 0)) return MGRIT_DEVICE_TIMEOUT;
  return MGRIT_OK;
}

int fetch_resnorm(const double* acc, float* resnorm, int iters, cudaStream_t s) {
  double tmp[64];
  for (int base = 0; base < iters; base += 64) {
    int n = iters - base < 64 ? iters - base : 64;
    if (cudaMemcpyAsync(tmp, acc + base, sizeof(double) * n, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MGRIT_CUDA_ERROR;
    if (cudaStreamSynchronize(s) != cudaSuccess) return MGRIT_CUDA_ERROR;
    for (int i = 0; i < n; ++i) resnorm[base + i] = (float)sqrt(tmp[i]);
  }
  return MGRIT_OK;
}

int forward_impl(const mgrit_gru_cfg* cfg_in, bool serial, const gru_params* p, const float* x, const float* h0, float* gi,
                 float* h, float* resnorm, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!cfg_in || !p || !x || !h0 || !gi || !h || !ws || !p->W_ih || !p->W_hh || !p->b_ih || !p->b_hh) return MGRIT_INVALID_ARG;
  if (!aligned32(x, h0, gi, h, ws, p->W_ih, p->W_hh, p->b_ih, p->b_hh)) return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg_in;
  if (serial) { c.levels = 1; c.iters = 1; c.cf = 2; }
  Hier hr;
  int rc = check_cfg(&c, &hr);
  if (rc) return rc;
  Ws w{(char*)ws, ws_bytes, 0};
  FwdWs fw;
  plan_fwd(&c, hr, w, &fw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  size_t BH = (size_t)c.B * c.H;
  // the caller's array has a leading slot for h_0: the level-0 unknowns live there and nothing is copied at the end
  const bool h_in_place = (c.flags & MGRIT_FLAG_H_LEADS_WITH_H0) != 0;
  if (h_in_place) fw.U[0] = h;
  if (carries_copies(&c, serial)) {      // make the copies where the adjoint call will look for them
    GiTail t = gi_tail(&c, gi);
    fw.um.xb = t.xb;
    fw.Ub[0] = t.hb0;
    fw.um.gib = t.gib;
  }
  if (!gi_bf16_enabled()) fw.um.gib = nullptr;
  // the caller does not read the fp32 projection and every kernel of this solve reads its bf16 copy: do not write it
  const bool gi_f32 = !((c.flags & MGRIT_FLAG_GI_F32_UNUSED) && carries_copies(&c, serial) && fw.um.gib);

  if (c.operands == MGRIT_OPERANDS_BF16) {
    rc = umma_prepare_fwd(&c, p, x, gi_f32 ? gi : nullptr, &fw.um, s);
    if (rc) return rc;
  } else if (is_tf32(&c)) {
    rc = tf32_prepare_fwd(&c, p, x, gi, &fw.tf, s);
    if (rc) return rc;
  } else {
    simt_project(x, p->W_ih, p->b_ih, gi, c.T * c.B, c.I, 3 * c.H, s);
  }
  zero_guess(fw.U[0], c, hr, BH, s);
  for (int l = 0; l < hr.L; ++l) cudaMemcpyAsync(fw.U[l], h0, sizeof(float) * BH, cudaMemcpyDeviceToDevice, s);
  const bool shadows = c.operands == MGRIT_OPERANDS_BF16 && 128 % c.B == 0;
  if (shadows && fw.sweep_ctr) cudaMemsetAsync(fw.sweep_ctr, 0, sizeof(int) * fw.sweep_ctr_n, s);
  if (shadows) {
    zero_guess(fw.Ub[0], c, hr, BH, s);
    for (int l = 0; l < hr.L; ++l) umma_convert(h0, fw.Ub[l], (i64)BH, s);
  }

  FwdCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = fw.U; cy.G = fw.G; cy.res_acc = fw.res_acc; cy.BH = BH;
  cy.p = p; cy.gi = gi; cy.um = &fw.um; cy.fw = &fw;
  cy.Ub = shadows ? fw.Ub : nullptr;
  cy.gib = shadows ? fw.um.gib : nullptr;
  cy.gi_f32 = gi_f32;
  rc = cy.solve();
  if (rc) return rc;
  if (!h_in_place) cudaMemcpyAsync(h, fw.U[0] + BH, sizeof(float) * (size_t)c.T * BH, cudaMemcpyDeviceToDevice, s);
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(fw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}

int adjoint_impl(const mgrit_gru_cfg* cfg_in, bool serial, const gru_params* p, const float* x, const float* h0,
                 const float* gi, const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0, float* dx,
                 const gru_grads* g, float* resnorm, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!cfg_in || !p || !x || !h0 || !gi || !h || !dh0 || !g || !ws) return MGRIT_INVALID_ARG;
  if (!dh_seed && !dhT) return MGRIT_INVALID_ARG;
  if (!p->W_ih || !p->W_hh || !p->b_ih || !p->b_hh || !g->dW_ih || !g->dW_hh || !g->db_ih || !g->db_hh) return MGRIT_INVALID_ARG;
  if (!aligned32(x, h0, gi, h, dh_seed, dhT, dh, dh0, dx, ws, p->W_ih, p->W_hh, p->b_ih, p->b_hh, g->dW_ih, g->dW_hh, g->db_ih, g->db_hh))
    return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg_in;
  if (serial) { c.levels = 1; c.iters = 1; c.cf = 2; }
  Hier hr;
  int rc = check_cfg(&c, &hr);
  if (rc) return rc;
  Ws w{(char*)ws, ws_bytes, 0};
  AdjWs aw;
  plan_adj(&c, hr, w, &aw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  size_t BH = (size_t)c.B * c.H;
  const int T = c.T;
  const bool bf16 = c.operands == MGRIT_OPERANDS_BF16;

  const bool copies = carries_copies(&c, serial);
  if (copies) {                           // bf16 x and [h_0; h] were left behind the projection by the forward call
    GiTail t = gi_tail(&c, const_cast<float*>(gi));
    aw.um.xb = t.xb;
    aw.um.hb0 = t.hb0;
    aw.um.hb = t.hb0 + BH;
    aw.um.gib = gi_bf16_enabled() ? t.gib : nullptr;
  }
  if (bf16) {
    rc = umma_prepare_adj(&c, p, h0, h, &aw.um, copies, s);
    if (rc) return rc;
  }
  const bool tf32 = is_tf32(&c);
  if (tf32) {
    rc = tf32_prepare_adj(&c, p, &aw.tf, s);
    if (rc) return rc;
  }
  // adjoint coefficients of every level's steps at the given states (restricted by injection)
  for (int l = 0; l < hr.L; ++l) {
    LinArgs a{};
    a.M = hr.N[l] * c.B; a.B = c.B; a.H = c.H; a.h0 = h0; a.h = h; a.stride_t = hr.stride_t[l]; a.gi = gi;
    a.t0 = hr.rem[l];     // the level's reversed grid is anchored at T: its forward steps arrive at t0 + stride * j
    a.W_hh = p->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c.cell;
    a.a = aw.a[l]; a.cr = aw.cr[l]; a.cz = aw.cz[l]; a.cn = aw.cn[l]; a.cnp = l == 0 ? aw.cnp : nullptr;
    a.crb = aw.crb[l]; a.czb = aw.czb[l]; a.cnb = aw.cnb[l]; a.cnpb = l == 0 ? aw.cnpb : nullptr;
    a.gi_b = (bf16 && copies) ? aw.um.gib : nullptr;
    if (bf16) {
      rc = umma_linearise(a, &aw.um, s);
      if (rc) return rc;
    } else if (tf32) {
      rc = tf32_linearise(a, &aw.tf, s);
      if (rc) return rc;
    } else {
      simt_linearise(a, s);
    }
  }
  // mu_0 = lambda_T; zero initial guess elsewhere; fine-level source = reversed dh_seed
  zero_guess(aw.U[0], c, hr, BH, s);        // (slot 0 is set below)
  if (dh_seed) {
    cudaMemcpyAsync(aw.U[0], dh_seed + (size_t)(T - 1) * BH, sizeof(float) * BH, cudaMemcpyDeviceToDevice, s);
    if (dhT) stream_add_rows(aw.U[0], dhT, (i64)BH, s);
    cudaMemsetAsync(aw.G[0], 0, sizeof(float) * BH, s);
    cudaMemsetAsync(aw.G[0] + (size_t)T * BH, 0, sizeof(float) * BH, s);
    if (T > 1) stream_gather_rows(aw.G[0] + BH, (i64)BH, dh_seed + (size_t)(T - 2) * BH, -(i64)BH, T - 1, (i64)BH, s);
  } else {
    cudaMemcpyAsync(aw.U[0], dhT, sizeof(float) * BH, cudaMemcpyDeviceToDevice, s);
  }
  for (int l = 1; l < hr.L; ++l) cudaMemcpyAsync(aw.U[l], aw.U[0], sizeof(float) * BH, cudaMemcpyDeviceToDevice, s);

  float* Gl[kMaxLevels];
  for (int l = 0; l < hr.L; ++l) Gl[l] = aw.G[l];
  if (!dh_seed) Gl[0] = nullptr;
  AdjCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = aw.U; cy.G = Gl; cy.res_acc = aw.res_acc; cy.BH = BH;
  cy.p = p; cy.w = &aw;
  rc = cy.solve();
  if (rc) return rc;

  // dh[k] = lambda_{k+1} = mu_{T-1-k} (optional output);  dh0 = lambda_0 = mu_T
  if (dh) stream_gather_rows(dh, (i64)BH, aw.U[0] + (size_t)(T - 1) * BH, -(i64)BH, T, (i64)BH, s);
  cudaMemcpyAsync(dh0, aw.U[0] + (size_t)T * BH, sizeof(float) * BH, cudaMemcpyDeviceToDevice, s);

  // gradient pass g = w * dh/dTheta over all fine steps at once
  if (bf16) {
    // lambda_{t+1} for t = 0..T-1 is read in place from the reversed unknowns (row stride -B*H)
    rc = umma_gradients(&c, p, x, h0, h, aw.U[0] + (size_t)(T - 1) * BH, -(i64)BH, aw.crb[0], aw.czb[0], aw.cnb[0], aw.cnpb, dx, g,
                        &aw.um, copies, s);
    if (rc) return rc;
  } else {
    i64 M = (i64)T * c.B;
    const float* lam = dh;
    if (!lam) {   // no dh output requested: gather lambda in forward order into workspace scratch
      lam = aw.lam_tmp;
      stream_gather_rows(aw.lam_tmp, (i64)BH, aw.U[0] + (size_t)(T - 1) * BH, -(i64)BH, T, (i64)BH, s);
    }
    stream_form_dA(lam, aw.cr[0], aw.cz[0], aw.cn[0], aw.cnp, aw.dA_h, aw.dA_i, M, c.H, s);
    if (tf32) {
      rc = tf32_wgrad(aw.dA_h, (int)M, 3 * c.H, h0, c.B, h, c.H, g->dW_hh, &aw.tf, s);
      if (!rc) rc = tf32_wgrad(aw.dA_i, (int)M, 3 * c.H, nullptr, 0, x, c.I, g->dW_ih, &aw.tf, s);
      if (rc) return rc;
    } else {
      simt_wgrad(aw.dA_h, (int)M, 3 * c.H, h0, c.B, h, c.H, g->dW_hh, s);
      simt_wgrad(aw.dA_i, (int)M, 3 * c.H, nullptr, 0, x, c.I, g->dW_ih, s);
    }
    stream_colsum(aw.dA_h, M, 3 * c.H, g->db_hh, s);
    stream_colsum(aw.dA_i, M, 3 * c.H, g->db_ih, s);
    if (dx) {
      if (tf32) { rc = tf32_dgrad(aw.dA_i, (int)M, 3 * c.H, c.I, dx, &aw.tf, s); if (rc) return rc; }
      else simt_dgrad(aw.dA_i, (int)M, 3 * c.H, p->W_ih, c.I, dx, s);
    }
  }
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(aw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}


// ======================================================================================================
// Stacked layers in one state: the state of a time point is the stack of all layers' hidden states, layer k's input
// at a step is layer k-1's NEW state of the same step, and ONE multigrid cycle advances the whole stack.  Level
// arrays are [N_l + 1][n_layers][B][H]; the cycle logic (Cycle) is the same, a "step" becomes a short sequence of
// launches per layer: cell step on the raw result, FAS combination, input projection for the layer above.
constexpr int kMaxStack = 8;

size_t stack_max_rows(const mgrit_gru_cfg* c, const Hier& hr) {
  size_t m = (size_t)c->B;
  for (int l = 0; l + 1 < hr.L; ++l) {
    size_t r = (size_t)((hr.N[l] + c->cf - 1) / c->cf) * c->B;
    if (r > m) m = r;
  }
  return m;
}

struct StackFwdWs {
  float* U[kMaxLevels]; float* G[kMaxLevels]; double* res_acc;
  float* tmpPhi; float* gi_tmp; size_t maxM;
  UmmaFwdWs um[kMaxStack];
};

mgrit_gru_cfg layer_cfg(const mgrit_gru_cfg& c, int k) {
  mgrit_gru_cfg ck = c;
  if (k > 0) ck.I = c.H;
  return ck;
}

void plan_stack_fwd(const mgrit_gru_cfg* c, int nl, const Hier& hr, Ws& w, StackFwdWs* o) {
  const size_t slot = (size_t)nl * c->B * c->H;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
    o->G[l] = l == 0 ? nullptr : w.take<float>((size_t)(hr.N[l] + 1) * slot);
  }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  o->maxM = stack_max_rows(c, hr);
  o->tmpPhi = w.take<float>(o->maxM * c->H);
  o->gi_tmp = w.take<float>(o->maxM * 3 * c->H);
  if (c->operands == MGRIT_OPERANDS_BF16)
    for (int k = 0; k < nl; ++k) {
      mgrit_gru_cfg ck = layer_cfg(*c, k);
      umma_plan_fwd(&ck, hr.N, hr.L, w.base, &w.off, &o->um[k]);
    }
}

struct StackFwdCycle : Cycle {
  int nl; const gru_params* p; const float* gi0; StackFwdWs* fw;
  int launch_step(const StepDesc& d) override {
    const size_t bh = (size_t)c->B * c->H, slot = (size_t)nl * bh;
    const int M = d.nk * c->B;
    const bool bf16 = c->operands == MGRIT_OPERANDS_BF16;
    const i64 st = hr.stride_t[d.l];
    for (int k = 0; k < nl; ++k) {
      FwdStepArgs a{};
      a.M = M; a.B = c->B; a.H = c->H;
      a.hin = U[d.l] + ((size_t)d.in_slot * nl + k) * bh; a.hin_ks = (i64)d.in_stride * slot;
      a.hout = fw->tmpPhi; a.hout_ks = (i64)bh;            // the raw step result, rows (k, b) contiguous
      a.hin_b = nullptr; a.hout_b = nullptr;
      if (k == 0) { a.gi = gi0 + ((i64)st * d.tgt_slot - 1) * (i64)bh * 3; a.gi_ks = st * d.tgt_stride * (i64)bh * 3; }
      else { a.gi = fw->gi_tmp; a.gi_ks = (i64)bh * 3; }
      a.gadd = nullptr; a.gadd_ks = 0;
      a.W_hh = p[k].W_hh; a.b_hh = p[k].b_hh; a.gamma = hr.gamma[d.l]; a.cell = c->cell; a.mode = 0;
      if (bf16) { int r = umma_fwd_step(a, &fw->um[k], s); if (r) return r; }
      else simt_fwd_step(a, s);
      // level unknown = raw result + FAS term (mode 0), or right-hand side -= raw result (mode 1)
      const float* g = d.gadd ? d.gadd + ((size_t)d.gadd_slot * nl + k) * bh : nullptr;
      stream_combine_rows(fw->tmpPhi, g, (i64)d.gadd_stride * slot, d.out + ((size_t)d.out_slot * nl + k) * bh, (i64)d.out_stride * slot,
                          c->B, c->H, (i64)M, d.mode, s);
      if (k + 1 < nl) {   // input projection of the layer above: its input is this layer's raw new state
        if (bf16) {
          int r = umma_project_rows(fw->tmpPhi, fw->um[k + 1].xb, fw->um[k + 1].W_ih, p[k + 1].b_ih, fw->gi_tmp, M, c->H, 3 * c->H, s);
          if (r) return r;
        } else {
          simt_project(fw->tmpPhi, p[k + 1].W_ih, p[k + 1].b_ih, fw->gi_tmp, M, c->H, 3 * c->H, s);
        }
      }
    }
    return MGRIT_OK;
  }
};

bool stack_args_ok(const mgrit_gru_cfg* c, int nl, const gru_params* p) {
  if (!c || !p || nl < 1 || nl > kMaxStack) return false;
  for (int k = 0; k < nl; ++k)
    if (!p[k].W_ih || !p[k].W_hh || !p[k].b_ih || !p[k].b_hh || !aligned32(p[k].W_ih, p[k].W_hh, p[k].b_ih, p[k].b_hh)) return false;
  return true;
}

int stack_forward_impl(const mgrit_gru_cfg* cfg, int nl, const gru_params* p, const float* x, const float* h0, float* gi0, float* h,
                       float* resnorm, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!stack_args_ok(cfg, nl, p) || !x || !h0 || !gi0 || !h || !ws) return MGRIT_INVALID_ARG;
  if (!aligned32(x, h0, gi0, h, ws)) return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg;
  Hier hr;
  int rc = check_cfg(&c, &hr);
  if (rc) return rc;
  if (is_tf32(&c)) return MGRIT_UNSUPPORTED;      // the stacked solve runs on the fp32 or the bf16 engine
  if (nl > 1) { mgrit_gru_cfg c1 = layer_cfg(c, 1); Hier h1; rc = check_cfg(&c1, &h1); if (rc) return rc; }
  Ws w{(char*)ws, ws_bytes, 0};
  StackFwdWs fw;
  plan_stack_fwd(&c, nl, hr, w, &fw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  const size_t bh = (size_t)c.B * c.H, slot = (size_t)nl * bh;
  if (c.operands == MGRIT_OPERANDS_BF16) {
    rc = umma_prepare_fwd(&c, &p[0], x, gi0, &fw.um[0], s);
    if (rc) return rc;
    for (int k = 1; k < nl; ++k) {
      umma_convert(p[k].W_hh, fw.um[k].W_hh, (i64)3 * c.H * c.H, s);
      umma_convert(p[k].W_ih, fw.um[k].W_ih, (i64)3 * c.H * c.H, s);
    }
  } else {
    simt_project(x, p[0].W_ih, p[0].b_ih, gi0, c.T * c.B, c.I, 3 * c.H, s);
  }
  cudaMemsetAsync(fw.U[0] + slot, 0, sizeof(float) * (size_t)c.T * slot, s);
  for (int l = 0; l < hr.L; ++l) cudaMemcpyAsync(fw.U[l], h0, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
  StackFwdCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = fw.U; cy.G = fw.G; cy.res_acc = fw.res_acc; cy.BH = slot;
  cy.nl = nl; cy.p = p; cy.gi0 = gi0; cy.fw = &fw;
  rc = cy.solve();
  if (rc) return rc;
  cudaMemcpyAsync(h, fw.U[0] + slot, sizeof(float) * (size_t)c.T * slot, cudaMemcpyDeviceToDevice, s);
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(fw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}

struct StackLayerAdj {
  float *a[kMaxLevels], *cr[kMaxLevels], *cz[kMaxLevels], *cn[kMaxLevels], *cnp[kMaxLevels];                 // fp32 engine
  __nv_bfloat16 *crb[kMaxLevels], *czb[kMaxLevels], *cnb[kMaxLevels], *cnpb[kMaxLevels];                     // tensor-core engine
  float* hk;                 // this layer's given states [T, B, H], contiguous
  float* gik;                // layers >= 1: input projection of the layer below's given states [T, B, 3H]
  __nv_bfloat16* Wihb;       // layers >= 1, tensor-core engine: W_ih as bf16 [3H, H]
  UmmaAdjWs um;
};
struct StackAdjWs {
  float* U[kMaxLevels]; float* G[kMaxLevels]; double* res_acc;
  float *tmpLin, *tmpDx, *lamk, *dxk, *dA_h, *dA_i; size_t maxM;
  StackLayerAdj L[kMaxStack];
};

void plan_stack_adj(const mgrit_gru_cfg* c, int nl, const Hier& hr, Ws& w, StackAdjWs* o) {
  const size_t bh = (size_t)c->B * c->H, slot = (size_t)nl * bh, TB = (size_t)c->T * c->B;
  const bool bf16 = c->operands == MGRIT_OPERANDS_BF16;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
    o->G[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
  }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  o->maxM = stack_max_rows(c, hr);
  o->tmpLin = w.take<float>(o->maxM * c->H);
  o->tmpDx = w.take<float>(o->maxM * c->H);
  o->lamk = w.take<float>(TB * c->H);
  o->dxk = w.take<float>(TB * c->H);
  if (bf16) { o->dA_h = o->dA_i = nullptr; }
  else { o->dA_h = w.take<float>(TB * 3 * c->H); o->dA_i = w.take<float>(TB * 3 * c->H); }
  for (int k = 0; k < nl; ++k) {
    StackLayerAdj& L = o->L[k];
    for (int l = 0; l < hr.L; ++l) {
      const size_t n = (size_t)hr.N[l] * bh;
      L.a[l] = w.take<float>(n);
      if (bf16) {
        L.cr[l] = L.cz[l] = L.cn[l] = L.cnp[l] = nullptr;
        L.crb[l] = w.take<__nv_bfloat16>(n); L.czb[l] = w.take<__nv_bfloat16>(n);
        L.cnb[l] = w.take<__nv_bfloat16>(n); L.cnpb[l] = w.take<__nv_bfloat16>(n);
      } else {
        L.crb[l] = L.czb[l] = L.cnb[l] = L.cnpb[l] = nullptr;
        L.cr[l] = w.take<float>(n); L.cz[l] = w.take<float>(n); L.cn[l] = w.take<float>(n); L.cnp[l] = w.take<float>(n);
      }
    }
    L.hk = w.take<float>(TB * c->H);
    L.gik = k > 0 ? w.take<float>(TB * 3 * c->H) : nullptr;
    L.Wihb = (bf16 && k > 0) ? w.take<__nv_bfloat16>((size_t)3 * c->H * c->H) : nullptr;
    if (bf16) { mgrit_gru_cfg ck = layer_cfg(*c, k); umma_plan_adj(&ck, hr.N, hr.L, w.base, &w.off, &L.um); }
  }
}

struct StackAdjCycle : Cycle {
  int nl; const gru_params* p; StackAdjWs* w;
  int launch_step(const StepDesc& d) override {
    const size_t bh = (size_t)c->B * c->H, slot = (size_t)nl * bh;
    const int M = d.nk * c->B;
    const bool bf16 = c->operands == MGRIT_OPERANDS_BF16;
    // the step arriving at reversed point s applies the level's forward step stored at coefficient row N_l - s
    const i64 row0 = (i64)(hr.N[d.l] - d.tgt_slot) * (i64)bh, coef_ks = -(i64)d.tgt_stride * (i64)bh;
    for (int k = nl - 1; k >= 0; --k) {       // top layer first: what it sends to its input joins the layer below
      StackLayerAdj& L = w->L[k];
      AdjStepArgs a;
      a.M = M; a.B = c->B; a.H = c->H;
      if (k == nl - 1) { a.lin = U[d.l] + ((size_t)d.in_slot * nl + k) * bh; a.lin_ks = (i64)d.in_stride * slot; }
      else { a.lin = w->tmpLin; a.lin_ks = (i64)bh; }
      a.lout = d.out + ((size_t)d.out_slot * nl + k) * bh; a.lout_ks = (i64)d.out_stride * slot;
      a.gadd = d.gadd ? d.gadd + ((size_t)d.gadd_slot * nl + k) * bh : nullptr; a.gadd_ks = (i64)d.gadd_stride * slot;
      a.a = L.a[d.l] + row0; a.coef_ks = coef_ks; a.W_hh = p[k].W_hh; a.mode = d.mode;
      if (bf16) { a.cr = a.cz = a.cn = nullptr; a.crb = L.crb[d.l] + row0; a.czb = L.czb[d.l] + row0; a.cnb = L.cnb[d.l] + row0; }
      else { a.crb = a.czb = a.cnb = nullptr; a.cr = L.cr[d.l] + row0; a.cz = L.cz[d.l] + row0; a.cn = L.cn[d.l] + row0; }
      if (bf16) { int r = umma_adj_step(a, &L.um, s); if (r) return r; }
      else simt_adj_step(a, s);
      if (k > 0) {
        // total output sensitivity of the layer below = its own entry of the incoming unknown + [c_r|c_z|c_n'] * lin W_ih
        AdjStepArgs b = a;
        if (bf16) { b.cnb = L.cnpb[d.l] + row0; int r = umma_adj_dx(b, L.um.W_ihT, c->H, w->tmpDx, &L.um, s); if (r) return r; }
        else { b.cn = L.cnp[d.l] + row0; simt_adj_dx(b, p[k].W_ih, c->H, w->tmpDx, s); }
        stream_gather_rows(w->tmpLin, (i64)bh, U[d.l] + ((size_t)d.in_slot * nl + (k - 1)) * bh, (i64)d.in_stride * slot, d.nk, (i64)bh, s);
        stream_add_rows(w->tmpLin, w->tmpDx, (i64)M * c->H, s);
      }
    }
    return MGRIT_OK;
  }
};

// time-parallel gradient pass of one layer given its total output sensitivities lam[T, B, H] (forward order, contiguous)
int stack_layer_gradients(const mgrit_gru_cfg& ck, const gru_params* pk, const float* xk, const float* h0k, StackLayerAdj& L,
                          StackAdjWs& w, float* dx, const gru_grads* g, cudaStream_t s) {
  const i64 bh = (i64)ck.B * ck.H, M = (i64)ck.T * ck.B;
  if (ck.operands == MGRIT_OPERANDS_BF16)
    return umma_gradients(&ck, pk, xk, h0k, L.hk, w.lamk, bh, L.crb[0], L.czb[0], L.cnb[0], L.cnpb[0], dx, g, &L.um, false, s);
  stream_form_dA(w.lamk, L.cr[0], L.cz[0], L.cn[0], L.cnp[0], w.dA_h, w.dA_i, M, ck.H, s);
  simt_wgrad(w.dA_h, (int)M, 3 * ck.H, h0k, ck.B, L.hk, ck.H, g->dW_hh, s);
  simt_wgrad(w.dA_i, (int)M, 3 * ck.H, nullptr, 0, xk, ck.I, g->dW_ih, s);
  stream_colsum(w.dA_h, M, 3 * ck.H, g->db_hh, s);
  stream_colsum(w.dA_i, M, 3 * ck.H, g->db_ih, s);
  if (dx) simt_dgrad(w.dA_i, (int)M, 3 * ck.H, pk->W_ih, ck.I, dx, s);
  return MGRIT_OK;
}

int stack_adjoint_impl(const mgrit_gru_cfg* cfg, int nl, const gru_params* p, const float* x, const float* h0, const float* gi0,
                       const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0, float* dx, const gru_grads* g,
                       float* resnorm, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!stack_args_ok(cfg, nl, p) || !x || !h0 || !gi0 || !h || !dh0 || !g || !ws) return MGRIT_INVALID_ARG;
  if (!dh_seed && !dhT) return MGRIT_INVALID_ARG;
  if (!aligned32(x, h0, gi0, h, dh_seed, dhT, dh, dh0, dx, ws)) return MGRIT_INVALID_ARG;
  for (int k = 0; k < nl; ++k)
    if (!g[k].dW_ih || !g[k].dW_hh || !g[k].db_ih || !g[k].db_hh || !aligned32(g[k].dW_ih, g[k].dW_hh, g[k].db_ih, g[k].db_hh))
      return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg;
  Hier hr;
  int rc = check_cfg(&c, &hr);
  if (rc) return rc;
  if (is_tf32(&c)) return MGRIT_UNSUPPORTED;      // the stacked solve runs on the fp32 or the bf16 engine
  if (nl > 1) { mgrit_gru_cfg c1 = layer_cfg(c, 1); Hier h1; rc = check_cfg(&c1, &h1); if (rc) return rc; }
  Ws w{(char*)ws, ws_bytes, 0};
  StackAdjWs aw;
  plan_stack_adj(&c, nl, hr, w, &aw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  const size_t bh = (size_t)c.B * c.H, slot = (size_t)nl * bh;
  const int T = c.T;
  const bool bf16 = c.operands == MGRIT_OPERANDS_BF16;

  // every layer's given states as their own [T, B, H] array; input projections of the layers above the first
  for (int k = 0; k < nl; ++k) stream_gather_rows(aw.L[k].hk, (i64)bh, h + (size_t)k * bh, (i64)slot, T, (i64)bh, s);
  for (int k = 0; k < nl; ++k) {
    StackLayerAdj& L = aw.L[k];
    mgrit_gru_cfg ck = layer_cfg(c, k);
    if (bf16) {
      rc = umma_prepare_adj(&ck, &p[k], h0 + (size_t)k * bh, L.hk, &L.um, false, s);
      if (rc) return rc;
    }
    if (k > 0) {
      if (bf16) {
        umma_convert(p[k].W_ih, L.Wihb, (i64)3 * c.H * c.H, s);
        rc = umma_project_rows(aw.L[k - 1].hk, L.um.xb, L.Wihb, p[k].b_ih, L.gik, T * c.B, c.H, 3 * c.H, s);
        if (rc) return rc;
      } else {
        simt_project(aw.L[k - 1].hk, p[k].W_ih, p[k].b_ih, L.gik, T * c.B, c.H, 3 * c.H, s);
      }
    }
    for (int l = 0; l < hr.L; ++l) {
      LinArgs a{};
      a.M = hr.N[l] * c.B; a.B = c.B; a.H = c.H; a.h0 = h0 + (size_t)k * bh; a.h = L.hk; a.stride_t = hr.stride_t[l];
      a.t0 = hr.rem[l]; a.gi = k == 0 ? gi0 : L.gik;
      a.W_hh = p[k].W_hh; a.b_hh = p[k].b_hh; a.gamma = hr.gamma[l]; a.cell = c.cell;
      a.a = L.a[l]; a.cr = L.cr[l]; a.cz = L.cz[l]; a.cn = L.cn[l]; a.cnp = L.cnp[l];
      a.crb = L.crb[l]; a.czb = L.czb[l]; a.cnb = L.cnb[l]; a.cnpb = L.cnpb[l];
      if (bf16) { rc = umma_linearise(a, &L.um, s); if (rc) return rc; }
      else simt_linearise(a, s);
    }
  }
  // mu_0 = lambda_T (all layers); zero initial guess elsewhere; fine-level source = reversed dh_seed
  cudaMemsetAsync(aw.U[0], 0, sizeof(float) * (size_t)(T + 1) * slot, s);
  cudaMemsetAsync(aw.G[0], 0, sizeof(float) * (size_t)(T + 1) * slot, s);
  if (dh_seed) {
    cudaMemcpyAsync(aw.U[0], dh_seed + (size_t)(T - 1) * slot, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
    if (T > 1) stream_gather_rows(aw.G[0] + slot, (i64)slot, dh_seed + (size_t)(T - 2) * slot, -(i64)slot, T - 1, (i64)slot, s);
  }
  if (dhT) stream_add_rows(aw.U[0] + (size_t)(nl - 1) * bh, dhT, (i64)bh, s);       // loss on the top layer's last state
  for (int l = 1; l < hr.L; ++l) cudaMemcpyAsync(aw.U[l], aw.U[0], sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);

  StackAdjCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = aw.U; cy.G = aw.G; cy.res_acc = aw.res_acc; cy.BH = slot;
  cy.nl = nl; cy.p = p; cy.w = &aw;
  rc = cy.solve();
  if (rc) return rc;

  if (dh) stream_gather_rows(dh, (i64)slot, aw.U[0] + (size_t)(T - 1) * slot, -(i64)slot, T, (i64)slot, s);
  cudaMemcpyAsync(dh0, aw.U[0] + (size_t)T * slot, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);

  // gradient pass, top layer first: a layer's total output sensitivity is its entry of the unknown plus what the layer
  // above sends to its input (that layer's input gradient)
  for (int k = nl - 1; k >= 0; --k) {
    stream_gather_rows(aw.lamk, (i64)bh, aw.U[0] + (size_t)(T - 1) * slot + (size_t)k * bh, -(i64)slot, T, (i64)bh, s);
    if (k < nl - 1) stream_add_rows(aw.lamk, aw.dxk, (i64)T * (i64)bh, s);
    mgrit_gru_cfg ck = layer_cfg(c, k);
    rc = stack_layer_gradients(ck, &p[k], k == 0 ? x : aw.L[k - 1].hk, h0 + (size_t)k * bh, aw.L[k], aw, k > 0 ? aw.dxk : dx, &g[k], s);
    if (rc) return rc;
  }
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(aw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}


// ======================================================================================================
// Implicit LSTM: the state of a time point is (c, h); level arrays are [N_l + 1][2][B][H] (part 0 = c, part 1 = h) and
// the same Cycle drives them.  fp32 engine only (four-gate FFMA products).
struct LstmFwdWs {
  float* U[kMaxLevels]; float* G[kMaxLevels]; double* res_acc; float *tmpC, *tmpH; size_t maxM; Tf32Ws tf; LstmBfWs bf;
  uint4* chain_xw; size_t chain_xw_bytes;      // exchange words of the persistent chain kernel (bf16 operands)
};
struct LstmAdjWs {
  float* U[kMaxLevels]; float* G[kMaxLevels]; double* res_acc;
  float *a[kMaxLevels], *p[kMaxLevels], *ci[kMaxLevels], *cf[kMaxLevels], *cg[kMaxLevels], *co[kMaxLevels];
  __nv_bfloat16 *cib[kMaxLevels], *cfb[kMaxLevels], *cgb[kMaxLevels], *cob[kMaxLevels];    // bf16 operands: the gate coefficients as bf16 instead
  float *tmpC, *tmpH, *hk, *dA; size_t maxM; Tf32Ws tf; LstmBfWs bf;
  uint4* chain_xw; size_t chain_xw_bytes;
};

void plan_lstm_fwd(const mgrit_gru_cfg* c, const Hier& hr, Ws& w, LstmFwdWs* o) {
  const size_t slot = (size_t)2 * c->B * c->H;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
    o->G[l] = l == 0 ? nullptr : w.take<float>((size_t)(hr.N[l] + 1) * slot);
  }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  o->maxM = stack_max_rows(c, hr);
  o->tmpC = w.take<float>(o->maxM * c->H);
  o->tmpH = w.take<float>(o->maxM * c->H);
  if (is_tf32(c)) tf32_plan_fwd(c, hr.N, hr.L, w.base, &w.off, &o->tf, 4);
  if (c->operands == MGRIT_OPERANDS_BF16) lstmbf_plan_fwd(c, o->maxM, w.base, &w.off, &o->bf);
  o->chain_xw = nullptr; o->chain_xw_bytes = 0;
  if (c->operands == MGRIT_OPERANDS_BF16 && c->H % 128 == 0) {
    o->chain_xw_bytes = serial_xw_bytes(c->B, c->H, 1);
    o->chain_xw = reinterpret_cast<uint4*>(w.take<char>(o->chain_xw_bytes));
  }
}

void plan_lstm_adj(const mgrit_gru_cfg* c, const Hier& hr, Ws& w, LstmAdjWs* o) {
  const size_t bh = (size_t)c->B * c->H, slot = 2 * bh, TB = (size_t)c->T * c->B;
  for (int l = 0; l < hr.L; ++l) {
    o->U[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
    o->G[l] = w.take<float>((size_t)(hr.N[l] + 1) * slot);
    const size_t n = (size_t)hr.N[l] * bh;
    o->a[l] = w.take<float>(n); o->p[l] = w.take<float>(n);
    if (c->operands == MGRIT_OPERANDS_BF16) {
      o->ci[l] = o->cf[l] = o->cg[l] = o->co[l] = nullptr;
      o->cib[l] = w.take<__nv_bfloat16>(n); o->cfb[l] = w.take<__nv_bfloat16>(n);
      o->cgb[l] = w.take<__nv_bfloat16>(n); o->cob[l] = w.take<__nv_bfloat16>(n);
    } else {
      o->ci[l] = w.take<float>(n); o->cf[l] = w.take<float>(n); o->cg[l] = w.take<float>(n); o->co[l] = w.take<float>(n);
      o->cib[l] = o->cfb[l] = o->cgb[l] = o->cob[l] = nullptr;
    }
  }
  o->res_acc = w.take<double>((size_t)(c->iters > 0 ? c->iters : 1));
  o->maxM = stack_max_rows(c, hr);
  o->tmpC = w.take<float>(o->maxM * c->H);
  o->tmpH = w.take<float>(o->maxM * c->H);
  o->hk = w.take<float>(TB * c->H);
  o->dA = w.take<float>(TB * 4 * c->H);
  if (is_tf32(c)) tf32_plan_adj(c, hr.N, hr.L, w.base, &w.off, &o->tf, 4);
  if (c->operands == MGRIT_OPERANDS_BF16) lstmbf_plan_adj(c, o->maxM, w.base, &w.off, &o->bf);
  o->chain_xw = nullptr; o->chain_xw_bytes = 0;
  if (c->operands == MGRIT_OPERANDS_BF16 && c->H % 128 == 0) {
    o->chain_xw_bytes = serial_xw_bytes(c->B, c->H, 4);
    o->chain_xw = reinterpret_cast<uint4*>(w.take<char>(o->chain_xw_bytes));
  }
}

struct LstmFwdCycle : Cycle {
  const gru_params* p; const float* gi; LstmFwdWs* fw;
  bool chain(int l) override {
    if (c->operands != MGRIT_OPERANDS_BF16 || !fw->chain_xw) return false;
    const i64 bh = (i64)c->B * c->H, st = hr.stride_t[l];
    LstmChainFwdArgs a{};
    a.B = c->B; a.H = c->H; a.nsteps = hr.N[l]; a.u = U[l];
    a.gi = gi + (st - 1) * bh * 4; a.gi_step = st * bh * 4;
    a.g = G[l]; a.W = fw->bf.W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c->cell;
    a.xw = fw->chain_xw; a.xw_bytes = fw->chain_xw_bytes;
    return lstm_chain_fwd_solve(a, s);
  }
  int launch_step(const StepDesc& d) override {
    const size_t bh = (size_t)c->B * c->H, slot = 2 * bh;
    const i64 st = hr.stride_t[d.l];
    LstmFwdArgs a;
    a.M = d.nk * c->B; a.B = c->B; a.H = c->H;
    a.cin = U[d.l] + (size_t)d.in_slot * slot; a.hin = a.cin + bh; a.in_ks = (i64)d.in_stride * slot;
    a.cout = fw->tmpC; a.hout = fw->tmpH;
    a.gi = gi + ((i64)st * d.tgt_slot - 1) * (i64)bh * 4; a.gi_ks = st * d.tgt_stride * (i64)bh * 4;
    a.W_hh = p->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[d.l]; a.cell = c->cell;
    // the tensor-core engines write the level array from their epilogue; the FFMA engine leaves raw results to combine
    const bool fused = c->operands != MGRIT_OPERANDS_FP32;
    a.up = LstmUpdate{};
    if (fused)
      a.up = LstmUpdate{d.out + (size_t)d.out_slot * slot, (i64)d.out_stride * (i64)slot, d.gadd ? d.gadd + (size_t)d.gadd_slot * slot : nullptr,
                        (i64)d.gadd_stride * (i64)slot, (i64)bh, d.mode};
    if (is_tf32(c)) { int r = tf32_lstm_fwd_step(a, &fw->tf, s); if (r) return r; }
    else if (c->operands == MGRIT_OPERANDS_BF16) { int r = lstmbf_fwd_step(a, &fw->bf, s); if (r) return r; }
    else simt_lstm_fwd_step(a, s);
    for (int part = 0; part < 2 && !fused; ++part) {
      const float* g = d.gadd ? d.gadd + (size_t)d.gadd_slot * slot + part * bh : nullptr;
      stream_combine_rows(part == 0 ? fw->tmpC : fw->tmpH, g, (i64)d.gadd_stride * slot, d.out + (size_t)d.out_slot * slot + part * bh,
                          (i64)d.out_stride * slot, c->B, c->H, (i64)a.M, d.mode, s);
    }
    return MGRIT_OK;
  }
};

struct LstmAdjCycle : Cycle {
  const gru_params* p; LstmAdjWs* w;
  bool chain(int l) override {
    if (c->operands != MGRIT_OPERANDS_BF16 || !w->chain_xw) return false;
    const i64 bh = (i64)c->B * c->H;
    const i64 row0 = (i64)(hr.N[l] - 1) * bh;     // step s = 1 applies forward step N_l, stored at row N_l - 1
    LstmChainAdjArgs a{};
    a.B = c->B; a.H = c->H; a.nsteps = hr.N[l]; a.mu = U[l];
    a.a = w->a[l] + row0; a.p = w->p[l] + row0; a.ci = w->cib[l] + row0; a.cf = w->cfb[l] + row0; a.cg = w->cgb[l] + row0;
    a.co = w->cob[l] + row0; a.coef_step = -bh;
    a.g = G[l]; a.WT = w->bf.W_hhT;
    a.xw = w->chain_xw; a.xw_bytes = w->chain_xw_bytes;
    return lstm_chain_adj_solve(a, s);
  }
  int launch_step(const StepDesc& d) override {
    const size_t bh = (size_t)c->B * c->H, slot = 2 * bh;
    const i64 row0 = (i64)(hr.N[d.l] - d.tgt_slot) * (i64)bh;
    LstmAdjArgs a;
    a.M = d.nk * c->B; a.B = c->B; a.H = c->H;
    a.lc = U[d.l] + (size_t)d.in_slot * slot; a.lh = a.lc + bh; a.in_ks = (i64)d.in_stride * slot;
    a.lc_out = w->tmpC; a.lh_out = w->tmpH;
    a.a = w->a[d.l] + row0; a.p = w->p[d.l] + row0; a.coef_ks = -(i64)d.tgt_stride * (i64)bh;
    const bool cb = w->cib[d.l] != nullptr;      // (the four gate coefficients: bf16 arrays on the bf16 engine, fp32 arrays otherwise)
    a.ci = cb ? nullptr : w->ci[d.l] + row0; a.cf = cb ? nullptr : w->cf[d.l] + row0;
    a.cg = cb ? nullptr : w->cg[d.l] + row0; a.co = cb ? nullptr : w->co[d.l] + row0;
    a.cib = cb ? w->cib[d.l] + row0 : nullptr; a.cfb = cb ? w->cfb[d.l] + row0 : nullptr;
    a.cgb = cb ? w->cgb[d.l] + row0 : nullptr; a.cob = cb ? w->cob[d.l] + row0 : nullptr;
    a.W_hh = p->W_hh;
    const bool fused = c->operands != MGRIT_OPERANDS_FP32;
    a.up = LstmUpdate{};
    if (fused)
      a.up = LstmUpdate{d.out + (size_t)d.out_slot * slot, (i64)d.out_stride * (i64)slot, d.gadd ? d.gadd + (size_t)d.gadd_slot * slot : nullptr,
                        (i64)d.gadd_stride * (i64)slot, (i64)bh, d.mode};
    if (is_tf32(c)) { int r = tf32_lstm_adj_step(a, &w->tf, s); if (r) return r; }
    else if (c->operands == MGRIT_OPERANDS_BF16) { int r = lstmbf_adj_step(a, &w->bf, s); if (r) return r; }
    else simt_lstm_adj_step(a, s);
    for (int part = 0; part < 2 && !fused; ++part) {
      const float* g = d.gadd ? d.gadd + (size_t)d.gadd_slot * slot + part * bh : nullptr;
      stream_combine_rows(part == 0 ? w->tmpC : w->tmpH, g, (i64)d.gadd_stride * slot, d.out + (size_t)d.out_slot * slot + part * bh,
                          (i64)d.out_stride * slot, c->B, c->H, (i64)a.M, d.mode, s);
    }
    return MGRIT_OK;
  }
};

int lstm_check(const mgrit_gru_cfg* cfg, Hier* hr) {
  if (!cfg) return MGRIT_INVALID_ARG;
  return check_cfg(cfg, hr);        // (bf16 and tf32 operands: check_cfg applies the tensor-core engines' shape limits)
}

int lstm_forward_impl(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, float* gi, float* u,
                      float* resnorm, void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!cfg || !p || !x || !u0 || !gi || !u || !ws || !p->W_ih || !p->W_hh || !p->b_ih || !p->b_hh) return MGRIT_INVALID_ARG;
  if (!aligned32(x, u0, gi, u, ws, p->W_ih, p->W_hh, p->b_ih, p->b_hh)) return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg;
  Hier hr;
  int rc = lstm_check(&c, &hr);
  if (rc) return rc;
  Ws w{(char*)ws, ws_bytes, 0};
  LstmFwdWs fw;
  plan_lstm_fwd(&c, hr, w, &fw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  const size_t slot = (size_t)2 * c.B * c.H;
  if (is_tf32(&c)) { rc = tf32_prepare_fwd(&c, p, x, gi, &fw.tf, s); if (rc) return rc; }
  else if (c.operands == MGRIT_OPERANDS_BF16) { rc = lstmbf_prepare_fwd(&c, p, x, gi, &fw.bf, s); if (rc) return rc; }
  else simt_project(x, p->W_ih, p->b_ih, gi, c.T * c.B, c.I, 4 * c.H, s);
  cudaMemsetAsync(fw.U[0] + slot, 0, sizeof(float) * (size_t)c.T * slot, s);
  for (int l = 0; l < hr.L; ++l) cudaMemcpyAsync(fw.U[l], u0, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
  LstmFwdCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = fw.U; cy.G = fw.G; cy.res_acc = fw.res_acc; cy.BH = slot;
  cy.p = p; cy.gi = gi; cy.fw = &fw;
  rc = cy.solve();
  if (rc) return rc;
  cudaMemcpyAsync(u, fw.U[0] + slot, sizeof(float) * (size_t)c.T * slot, cudaMemcpyDeviceToDevice, s);
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(fw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}

int lstm_adjoint_impl(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, const float* gi, const float* u,
                      const float* du_seed, const float* dhT, float* du, float* du0, float* dx, const gru_grads* g, float* resnorm,
                      void* ws, size_t ws_bytes, cudaStream_t s) {
  if (!cfg || !p || !x || !u0 || !gi || !u || !du0 || !g || !ws) return MGRIT_INVALID_ARG;
  if (!du_seed && !dhT) return MGRIT_INVALID_ARG;
  if (!p->W_ih || !p->W_hh || !p->b_ih || !p->b_hh || !g->dW_ih || !g->dW_hh || !g->db_ih || !g->db_hh) return MGRIT_INVALID_ARG;
  if (!aligned32(x, u0, gi, u, du_seed, dhT, du, du0, dx, ws, p->W_ih, p->W_hh, p->b_ih, p->b_hh, g->dW_ih, g->dW_hh, g->db_ih, g->db_hh))
    return MGRIT_INVALID_ARG;
  mgrit_gru_cfg c = *cfg;
  Hier hr;
  int rc = lstm_check(&c, &hr);
  if (rc) return rc;
  Ws w{(char*)ws, ws_bytes, 0};
  LstmAdjWs aw;
  plan_lstm_adj(&c, hr, w, &aw);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  const size_t bh = (size_t)c.B * c.H, slot = 2 * bh;
  const int T = c.T;
  const bool tf32 = is_tf32(&c), bf = c.operands == MGRIT_OPERANDS_BF16;
  if (tf32) { rc = tf32_prepare_adj(&c, p, &aw.tf, s); if (rc) return rc; }
  if (bf) { rc = lstmbf_prepare_adj(&c, p, &aw.bf, s); if (rc) return rc; }
  for (int l = 0; l < hr.L; ++l) {
    LstmLinArgs a;
    a.M = hr.N[l] * c.B; a.B = c.B; a.H = c.H; a.c0 = u0; a.h0 = u0 + bh; a.c = u; a.h = u + bh; a.ts = (i64)slot;
    a.stride_t = hr.stride_t[l]; a.t0 = hr.rem[l]; a.gi = gi; a.W_hh = p->W_hh; a.b_hh = p->b_hh; a.gamma = hr.gamma[l]; a.cell = c.cell;
    a.a = aw.a[l]; a.p = aw.p[l]; a.ci = aw.ci[l]; a.cf = aw.cf[l]; a.cg = aw.cg[l]; a.co = aw.co[l];
    a.cib = aw.cib[l]; a.cfb = aw.cfb[l]; a.cgb = aw.cgb[l]; a.cob = aw.cob[l];
    if (tf32) { rc = tf32_lstm_linearise(a, &aw.tf, s); if (rc) return rc; }
    else if (bf) { rc = lstmbf_linearise(a, &aw.bf, s); if (rc) return rc; }
    else simt_lstm_linearise(a, s);
  }
  cudaMemsetAsync(aw.U[0], 0, sizeof(float) * (size_t)(T + 1) * slot, s);
  cudaMemsetAsync(aw.G[0], 0, sizeof(float) * (size_t)(T + 1) * slot, s);
  if (du_seed) {
    cudaMemcpyAsync(aw.U[0], du_seed + (size_t)(T - 1) * slot, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
    if (T > 1) stream_gather_rows(aw.G[0] + slot, (i64)slot, du_seed + (size_t)(T - 2) * slot, -(i64)slot, T - 1, (i64)slot, s);
  }
  if (dhT) stream_add_rows(aw.U[0] + bh, dhT, (i64)bh, s);      // loss on the last hidden state
  for (int l = 1; l < hr.L; ++l) cudaMemcpyAsync(aw.U[l], aw.U[0], sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
  LstmAdjCycle cy;
  cy.c = &c; cy.hr = hr; cy.s = s; cy.U = aw.U; cy.G = aw.G; cy.res_acc = aw.res_acc; cy.BH = slot;
  cy.p = p; cy.w = &aw;
  rc = cy.solve();
  if (rc) return rc;
  if (du) stream_gather_rows(du, (i64)slot, aw.U[0] + (size_t)(T - 1) * slot, -(i64)slot, T, (i64)slot, s);
  cudaMemcpyAsync(du0, aw.U[0] + (size_t)T * slot, sizeof(float) * slot, cudaMemcpyDeviceToDevice, s);
  // gradient pass over all fine steps at once: dA_t from the step-output sensitivities (read in place, reversed in time)
  const i64 M = (i64)T * c.B;
  const float* lam_c = aw.U[0] + (size_t)(T - 1) * slot;
  if (bf) {
    // bf16 operands: dA is formed as bf16 together with the bias sums, the hidden states are packed straight from u
    rc = lstmbf_gradients(&c, lam_c, lam_c + bh, -(i64)slot, aw.p[0], aw.cib[0], aw.cfb[0], aw.cgb[0], aw.cob[0], x, u0 + bh, u + bh, (i64)slot, g,
                          dx, &aw.bf, s);
    if (rc) return rc;
  } else {
    simt_lstm_form_dA(lam_c, lam_c + bh, -(i64)slot, c.B, aw.p[0], aw.ci[0], aw.cf[0], aw.cg[0], aw.co[0], aw.dA, M, c.H, s);
    stream_gather_rows(aw.hk, (i64)bh, u + bh, (i64)slot, T, (i64)bh, s);        // hidden states as their own [T, B, H] array
    if (tf32) {
      rc = tf32_wgrad(aw.dA, (int)M, 4 * c.H, u0 + bh, c.B, aw.hk, c.H, g->dW_hh, &aw.tf, s);
      if (!rc) rc = tf32_wgrad(aw.dA, (int)M, 4 * c.H, nullptr, 0, x, c.I, g->dW_ih, &aw.tf, s);
      if (rc) return rc;
    } else {
      simt_wgrad(aw.dA, (int)M, 4 * c.H, u0 + bh, c.B, aw.hk, c.H, g->dW_hh, s);
      simt_wgrad(aw.dA, (int)M, 4 * c.H, nullptr, 0, x, c.I, g->dW_ih, s);
    }
    stream_colsum(aw.dA, M, 4 * c.H, g->db_hh, s);
    cudaMemcpyAsync(g->db_ih, g->db_hh, sizeof(float) * 4 * c.H, cudaMemcpyDeviceToDevice, s);
    if (dx) {
      if (tf32) { rc = tf32_dgrad(aw.dA, (int)M, 4 * c.H, c.I, dx, &aw.tf, s); if (rc) return rc; }
      else simt_dgrad(aw.dA, (int)M, 4 * c.H, p->W_ih, c.I, dx, s);
    }
  }
  if (resnorm && hr.L > 1 && c.iters > 0) {
    rc = fetch_resnorm(aw.res_acc, resnorm, c.iters, s);
    if (rc) return rc;
    return finish(s, true);
  }
  return finish(s, false);
}

}  // namespace
}  // namespace mg

using namespace mg;

extern "C" {

int mgrit_gru_workspace_bytes(const mgrit_gru_cfg* cfg, size_t* fwd_bytes, size_t* adj_bytes) {
  Hier hr;
  int rc = check_cfg(cfg, &hr);
  if (rc) return rc;
  // the serial entry points run the same cfg with levels = 1: take the larger of the two plans
  mgrit_gru_cfg c1 = *cfg; c1.levels = 1; c1.iters = 1; c1.cf = 2;
  Hier h1;
  rc = check_cfg(&c1, &h1);
  if (rc) return rc;
  if (fwd_bytes) {
    Ws w{nullptr, 0, 0}; FwdWs f; plan_fwd(cfg, hr, w, &f);
    Ws w1{nullptr, 0, 0}; FwdWs f1; plan_fwd(&c1, h1, w1, &f1);
    *fwd_bytes = (w.off > w1.off ? w.off : w1.off) + 256;
  }
  if (adj_bytes) {
    Ws w{nullptr, 0, 0}; AdjWs a; plan_adj(cfg, hr, w, &a);
    Ws w1{nullptr, 0, 0}; AdjWs a1; plan_adj(&c1, h1, w1, &a1);
    *adj_bytes = (w.off > w1.off ? w.off : w1.off) + 256;
  }
  return MGRIT_OK;
}

int gru_step_rows(const mgrit_gru_cfg* cfg, const gru_params* p, int32_t n, float gamma, const float* gi_rows, const float* u_prev,
                  float* out, mgrit_stream_t stream) {
  if (!cfg || !p || !p->W_hh || !p->b_hh || !gi_rows || !u_prev || !out || n < 0) return MGRIT_INVALID_ARG;
  if (cfg->B <= 0 || cfg->H <= 0 || cfg->H % 8 != 0 || !(gamma > 0.f)) return MGRIT_INVALID_ARG;
  if (cfg->cell != MGRIT_CELL_CLASSIC && cfg->cell != MGRIT_CELL_IMPLICIT) return MGRIT_INVALID_ARG;
  if (!aligned32(gi_rows, u_prev, out, p->W_hh, p->b_hh)) return MGRIT_INVALID_ARG;
  if ((i64)n * cfg->B > (i64)INT_MAX - 1024) return MGRIT_UNSUPPORTED;
  if (n == 0) return MGRIT_OK;
  cudaStream_t s = (cudaStream_t)stream;
  const i64 BH = (i64)cfg->B * cfg->H;
  FwdStepArgs a{};
  a.M = n * cfg->B; a.B = cfg->B; a.H = cfg->H;
  a.hin = u_prev; a.hin_ks = BH; a.hout = out; a.hout_ks = BH;
  a.gi = gi_rows; a.gi_ks = 3 * BH;
  a.W_hh = p->W_hh; a.b_hh = p->b_hh; a.gamma = gamma; a.cell = cfg->cell; a.mode = 0;
  simt_fwd_step(a, s);
  return finish(s, false);
}

int gru_adjoint_step_rows(const mgrit_gru_cfg* cfg, const gru_params* p, int32_t n, float gamma, const float* gi_rows,
                          const float* h_lin, const float* mu, float* out, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  if (!cfg || !p || !p->W_hh || !p->b_hh || !gi_rows || !h_lin || !mu || !out || n < 0) return MGRIT_INVALID_ARG;
  if (cfg->B <= 0 || cfg->H <= 0 || cfg->H % 8 != 0 || !(gamma > 0.f)) return MGRIT_INVALID_ARG;
  if (cfg->cell != MGRIT_CELL_CLASSIC && cfg->cell != MGRIT_CELL_IMPLICIT) return MGRIT_INVALID_ARG;
  if (!aligned32(gi_rows, h_lin, mu, out, ws, p->W_hh, p->b_hh)) return MGRIT_INVALID_ARG;
  if ((i64)n * cfg->B > (i64)INT_MAX - 1024) return MGRIT_UNSUPPORTED;
  if (n == 0) return MGRIT_OK;
  const i64 BH = (i64)cfg->B * cfg->H;
  const size_t rows = (size_t)n * BH;
  if (!ws) return MGRIT_INVALID_ARG;
  Ws w{(char*)ws, ws_bytes, 0};
  float* ca = w.take<float>(rows); float* cr = w.take<float>(rows); float* cz = w.take<float>(rows);
  float* cn = w.take<float>(rows); float* cnp = w.take<float>(rows);
  if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
  cudaStream_t s = (cudaStream_t)stream;
  // coefficients of the n*B steps: row (j, b) leaves the state h_lin[j] with the input projection gi_rows[j]
  // (the level layout of the linearisation with unit stride: step j + 1 leaves fine time 1 + j)
  LinArgs l{};
  l.M = n * cfg->B; l.B = cfg->B; l.H = cfg->H; l.h0 = h_lin; l.h = h_lin; l.stride_t = 1; l.t0 = 1;
  l.gi = gi_rows - 3 * BH;      // its row t + stride - 1 = j + 1 is gi_rows[j]; row 0 is never read
  l.W_hh = p->W_hh; l.b_hh = p->b_hh; l.gamma = gamma; l.cell = cfg->cell;
  l.a = ca; l.cr = cr; l.cz = cz; l.cn = cn; l.cnp = cnp;
  simt_linearise(l, s);
  AdjStepArgs a{};
  a.M = n * cfg->B; a.B = cfg->B; a.H = cfg->H;
  a.lin = mu; a.lin_ks = BH; a.lout = out; a.lout_ks = BH;
  a.a = ca; a.cr = cr; a.cz = cz; a.cn = cn; a.coef_ks = BH;
  a.W_hh = p->W_hh; a.mode = 0;
  simt_adj_step(a, s);
  return finish(s, false);
}

size_t mgrit_gru_gi_bytes(const mgrit_gru_cfg* cfg) {
  Hier hr;
  if (check_cfg(cfg, &hr) != MGRIT_OK) return 0;
  const size_t plain = (size_t)cfg->T * cfg->B * 3 * cfg->H * sizeof(float);
  return (cfg->flags & MGRIT_FLAG_GI_CARRIES_COPIES) ? gi_tail(cfg, nullptr).total_bytes : plain;
}

int gru_input_projection(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, float* gi, void* ws, size_t ws_bytes,
                         mgrit_stream_t stream) {
  if (!cfg || !p || !x || !gi || !p->W_ih || !p->b_ih) return MGRIT_INVALID_ARG;
  if (!aligned32(x, gi, ws, p->W_ih, p->b_ih)) return MGRIT_INVALID_ARG;
  Hier hr;
  int rc = check_cfg(cfg, &hr);
  if (rc) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  if (cfg->operands == MGRIT_OPERANDS_BF16) {
    if (!ws) return MGRIT_INVALID_ARG;
    Ws w{(char*)ws, ws_bytes, 0};
    FwdWs fw;
    plan_fwd(cfg, hr, w, &fw);
    if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
    rc = umma_prepare_fwd(cfg, p, x, gi, &fw.um, s);
    if (rc) return rc;
  } else if (is_tf32(cfg)) {
    if (!ws) return MGRIT_INVALID_ARG;
    Ws w{(char*)ws, ws_bytes, 0};
    FwdWs fw;
    plan_fwd(cfg, hr, w, &fw);
    if (!w.fits()) return MGRIT_WORKSPACE_TOO_SMALL;
    rc = tf32_prepare_fwd(cfg, p, x, gi, &fw.tf, s);
    if (rc) return rc;
  } else {
    simt_project(x, p->W_ih, p->b_ih, gi, cfg->T * cfg->B, cfg->I, 3 * cfg->H, s);
  }
  return finish(s, false);
}

int mgrit_gru_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0, float* gi, float* h,
                      float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return forward_impl(cfg, false, p, x, h0, gi, h, resnorm, ws, ws_bytes, (cudaStream_t)stream);
}

int gru_serial_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0, float* gi, float* h,
                       void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return forward_impl(cfg, true, p, x, h0, gi, h, nullptr, ws, ws_bytes, (cudaStream_t)stream);
}

int mgrit_gru_adjoint(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0, const float* gi,
                      const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0, float* dx,
                      const gru_grads* grads, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return adjoint_impl(cfg, false, p, x, h0, gi, h, dh_seed, dhT, dh, dh0, dx, grads, resnorm, ws, ws_bytes, (cudaStream_t)stream);
}

int gru_serial_backward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0, const float* gi,
                        const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0, float* dx,
                        const gru_grads* grads, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return adjoint_impl(cfg, true, p, x, h0, gi, h, dh_seed, dhT, dh, dh0, dx, grads, nullptr, ws, ws_bytes, (cudaStream_t)stream);
}

int mgrit_gru_stack_workspace_bytes(const mgrit_gru_cfg* cfg, int32_t n_layers, size_t* fwd_bytes, size_t* adj_bytes) {
  Hier hr;
  int rc = check_cfg(cfg, &hr);
  if (rc) return rc;
  if (n_layers < 1 || n_layers > kMaxStack) return MGRIT_INVALID_ARG;
  if (is_tf32(cfg)) return MGRIT_UNSUPPORTED;
  if (n_layers > 1) { mgrit_gru_cfg c1 = layer_cfg(*cfg, 1); Hier h1; rc = check_cfg(&c1, &h1); if (rc) return rc; }
  if (fwd_bytes) { Ws w{nullptr, 0, 0}; StackFwdWs f; plan_stack_fwd(cfg, n_layers, hr, w, &f); *fwd_bytes = w.off + 256; }
  if (adj_bytes) { Ws w{nullptr, 0, 0}; StackAdjWs a; plan_stack_adj(cfg, n_layers, hr, w, &a); *adj_bytes = w.off + 256; }
  return MGRIT_OK;
}

int mgrit_gru_stack_forward(const mgrit_gru_cfg* cfg, int32_t n_layers, const gru_params* layers, const float* x, const float* h0,
                            float* gi0, float* h, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return stack_forward_impl(cfg, n_layers, layers, x, h0, gi0, h, resnorm, ws, ws_bytes, (cudaStream_t)stream);
}

int mgrit_gru_stack_adjoint(const mgrit_gru_cfg* cfg, int32_t n_layers, const gru_params* layers, const float* x, const float* h0,
                            const float* gi0, const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0, float* dx,
                            const gru_grads* grads, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return stack_adjoint_impl(cfg, n_layers, layers, x, h0, gi0, h, dh_seed, dhT, dh, dh0, dx, grads, resnorm, ws, ws_bytes,
                            (cudaStream_t)stream);
}

int mgrit_lstm_workspace_bytes(const mgrit_gru_cfg* cfg, size_t* fwd_bytes, size_t* adj_bytes) {
  Hier hr;
  int rc = lstm_check(cfg, &hr);
  if (rc) return rc;
  if (fwd_bytes) { Ws w{nullptr, 0, 0}; LstmFwdWs f; plan_lstm_fwd(cfg, hr, w, &f); *fwd_bytes = w.off + 256; }
  if (adj_bytes) { Ws w{nullptr, 0, 0}; LstmAdjWs a; plan_lstm_adj(cfg, hr, w, &a); *adj_bytes = w.off + 256; }
  return MGRIT_OK;
}

int mgrit_lstm_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, float* gi, float* u,
                       float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return lstm_forward_impl(cfg, p, x, u0, gi, u, resnorm, ws, ws_bytes, (cudaStream_t)stream);
}

int mgrit_lstm_adjoint(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, const float* gi,
                       const float* u, const float* du_seed, const float* dhT, float* du, float* du0, float* dx,
                       const gru_grads* grads, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  return lstm_adjoint_impl(cfg, p, x, u0, gi, u, du_seed, dhT, du, du0, dx, grads, resnorm, ws, ws_bytes, (cudaStream_t)stream);
}

size_t xent_head_workspace_bytes(int32_t B, int32_t C) {
  if (B <= 0 || C <= 0) return 0;
  return ((((size_t)B * C + (size_t)B) * sizeof(float)) + 255) & ~(size_t)255;     // dlogits [B, C] + per-row loss terms [B]
}

int xent_head_fwd_bwd(int32_t B, int32_t H, int32_t C, const float* hT, const float* Wc, const float* bc, const int32_t* labels,
                      float* loss, float* dhT, float* dWc, float* dbc, void* ws, size_t ws_bytes, mgrit_stream_t stream) {
  if (B <= 0 || H <= 0 || C <= 0 || !hT || !Wc || !bc || !labels || !loss || !dhT || !dWc || !dbc || !ws) return MGRIT_INVALID_ARG;
  if (C > 8192) return MGRIT_UNSUPPORTED;
  if (ws_bytes < xent_head_workspace_bytes(B, C)) return MGRIT_WORKSPACE_TOO_SMALL;
  stream_xent(B, H, C, hT, Wc, bc, labels, loss, dhT, dWc, dbc, (float*)ws, (cudaStream_t)stream);
  return finish((cudaStream_t)stream, false);
}

int sgd_update(float* p, const float* g, size_t n, float lr, mgrit_stream_t stream) {
  if (!p || !g) return MGRIT_INVALID_ARG;
  if (n == 0) return MGRIT_OK;
  if (((uintptr_t)p | (uintptr_t)g) & 15) return MGRIT_INVALID_ARG;
  stream_sgd(p, g, n, lr, (cudaStream_t)stream);
  return finish((cudaStream_t)stream, false);
}

int adam_update(float* p, const float* g, float* m, float* v, size_t n, float lr, float beta1, float beta2, float eps, int32_t step,
                mgrit_stream_t stream) {
  if (!p || !g || !m || !v || step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f))
    return MGRIT_INVALID_ARG;
  if (n == 0) return MGRIT_OK;
  stream_adam(p, g, m, v, n, lr, beta1, beta2, eps, step, (cudaStream_t)stream);
  return finish((cudaStream_t)stream, false);
}

int mgrit_gru_last_device_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return MGRIT_CUDA_ERROR;
  return (umma_device_status() != 0 || serial_device_status() != 0) ? MGRIT_DEVICE_TIMEOUT : MGRIT_OK;
}

int mgrit_gru_clear_device_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return MGRIT_CUDA_ERROR;
  return (umma_clear_device_status() == 0 && serial_clear_device_status() == 0) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int mgrit_gru_selftest_bounded_wait(int32_t limit_ms, mgrit_stream_t stream) { return umma_selftest_wait(limit_ms, (cudaStream_t)stream); }

unsigned long long mgrit_gru_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

int mgrit_gru_profile_enable(int on) {
  for (auto& r : g_prof_recs) { g_prof_pool.push_back(r.e0); g_prof_pool.push_back(r.e1); }
  g_prof_recs.clear();
  g_prof_depth = 0;
  g_prof_on = on != 0;
  return MGRIT_OK;
}

int mgrit_gru_profile_records(double* ms, double* flops, int32_t* kernel_class, size_t cap, size_t* n) {
  if (!n) return MGRIT_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return MGRIT_CUDA_ERROR;
  *n = g_prof_recs.size();
  for (size_t i = 0; i < g_prof_recs.size() && i < cap; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_prof_recs[i].e0, g_prof_recs[i].e1) != cudaSuccess) return MGRIT_CUDA_ERROR;
    if (ms) ms[i] = t;
    if (flops) flops[i] = g_prof_recs[i].flops;
    if (kernel_class) kernel_class[i] = g_prof_recs[i].kc;
  }
  return MGRIT_OK;
}

int mgrit_gru_profile_read(int kernel_class, double* total_ms, unsigned long long* launches, double* flops) {
  if (kernel_class < 0 || kernel_class >= KC_COUNT) return MGRIT_INVALID_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return MGRIT_CUDA_ERROR;
  double ms = 0, fl = 0; unsigned long long n = 0;
  for (auto& r : g_prof_recs) {
    if (r.kc != kernel_class) continue;
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess) return MGRIT_CUDA_ERROR;
    ms += t; fl += r.flops; ++n;
  }
  if (total_ms) *total_ms = ms;
  if (launches) *launches = n;
  if (flops) *flops = fl;
  return MGRIT_OK;
}

const char* mgrit_gru_strerror(int code) {
  switch (code) {
    case MGRIT_OK: return "ok";
    case MGRIT_INVALID_ARG: return "invalid argument";
    case MGRIT_NOT_DIVISIBLE: return "T is not divisible by cf^(levels-1)";
    case MGRIT_WORKSPACE_TOO_SMALL: return "workspace too small";
    case MGRIT_UNSUPPORTED: return "shape not supported (operand mode limits, C > 8192 in the loss head, or sizes beyond 32-bit row counts)";
    case MGRIT_CUDA_ERROR: return "CUDA error";
    case MGRIT_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case MGRIT_SCRATCH_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point (B*(C+1) <= 65536)";
    default: return "unknown error";
  }
}

}  // extern "C"
