/* mgrit_gru.h -- C ABI of the B200 (sm_100a) MGRIT solver for the GRU hidden-state recurrence.
 *
 * The library implements, as CUDA kernels only (there is no CPU fallback), the parallel-in-time
 * training path of "Parallel Training of GRU Networks with a Multi-Grid Solver for Long
 * Sequences": the input projection, the multigrid-reduction-in-time (MGRIT) cycle for the
 * forward recurrence h_t = Phi(x_t, h_{t-1}) and for its adjoint, the time-parallel weight
 * gradients, a classifier/loss head, the SGD update, and the exact serial sweep it converges to.
 *
 * Conventions
 *  - Every data pointer is a DEVICE pointer owned by the caller, 32-byte aligned (the kernels move whole
 *    32-byte sectors per thread; a misaligned pointer is rejected with MGRIT_INVALID_ARG), fp32, row-major,
 *    time-major: x[T,B,I], gi[T,B,3H], h[T,B,H]; h[k] is the paper's h_{k+1}, h_0 is passed
 *    separately.  Gate order along 3H is r | z | n (Eq. "gru").
 *  - cfg, resnorm and the size outputs are HOST pointers.
 *  - The library never allocates or frees device memory: scratch is a caller-provided workspace
 *    (device, 256-byte aligned) of at least the size reported by mgrit_gru_workspace_bytes().
 *  - Calls enqueue work on `stream` and return without synchronising, except that a non-NULL
 *    `resnorm` makes the call synchronise the stream before it returns.
 *  - Return value: MGRIT_OK (0) or a negative error code; outputs are undefined after an error.
 *    Nothing aborts the process.  Device-side waits are bounded: a wait that runs out makes the
 *    next synchronising call (or mgrit_gru_last_device_status) report MGRIT_DEVICE_TIMEOUT.
 *  - A call works on the device that is current when it is made (no sharding, no collectives); a process may use
 *    the library on several devices, each with its own workspaces.  Calls that share a workspace must not overlap
 *    on the GPU.  The library is NOT thread-safe: calls made from several host threads must be serialised by the
 *    caller (the launch counter is atomic; the profiling records and the first-use set-up of a device are not).
 *  - Sizes: (T + 1) * B must stay below 2^31 - 1024 (row counts are 32-bit inside the kernels; element offsets
 *    are 64-bit); larger problems are rejected with MGRIT_UNSUPPORTED.
 */
#ifndef MGRIT_GRU_H_
#define MGRIT_GRU_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* mgrit_stream_t; /* a cudaStream_t */

enum {
  MGRIT_OK = 0,
  MGRIT_INVALID_ARG = -1,        /* NULL pointer, non-positive size, unknown enum value */
  MGRIT_NOT_DIVISIBLE = -2,      /* T is not a multiple of cf^(levels-1) */
  MGRIT_WORKSPACE_TOO_SMALL = -3,
  MGRIT_UNSUPPORTED = -4,        /* shape outside what the selected operand mode supports, or beyond 32-bit row counts */
  MGRIT_CUDA_ERROR = -5,         /* a CUDA runtime/driver call failed: a launch, or the preparation of one (tensor-map
                                    encoding); nothing further is enqueued by that call and its outputs are undefined */
  MGRIT_DEVICE_TIMEOUT = -6,     /* a bounded device-side wait ran out */
  MGRIT_SCRATCH_LIMIT = -7       /* problem larger than the built-in scratch of a no-allocation entry point */
};

enum { MGRIT_CELL_CLASSIC = 0, MGRIT_CELL_IMPLICIT = 1 };
/* relaxation = n means F (CF)^n: F-relaxation followed by n C- and F-sweeps (Eq. "fcf-relax" is n = 1) */
enum { MGRIT_RELAX_F = 0, MGRIT_RELAX_FCF = 1, MGRIT_RELAX_FCFCF = 2, MGRIT_RELAX_MAX = 8 };
enum { MGRIT_OPERANDS_FP32 = 0, MGRIT_OPERANDS_TF32 = 1, MGRIT_OPERANDS_BF16 = 2, MGRIT_OPERANDS_TF32_1PASS = 3 };
enum {
  MGRIT_FLAG_SKIP_DUPLICATE_FRELAX = 1,
  /* F-cycles instead of V-cycles: when the correction of a level has been spread by its final F-relaxation, one
   * more V-cycle is run from that level down (on the last two levels: two V-cycles).  The paper's Algorithm
   * "MGProp" with the recursion of remark "Beyond Two-Level" is the V-cycle; the F-cycle is the usual multigrid
   * variant of it.  resnorm keeps one entry per cycle: the level-0 residual of the cycle's first visit. */
  MGRIT_FLAG_F_CYCLE = 2,
  /* Accept any T >= cf^(levels-1): the C-points of a level are its points 0, cf, 2 cf, ...; what follows the last
   * one is a shorter last interval of F-points, so N_{l+1} = floor(N_l / cf).  The forward grids are anchored at
   * t = 0, the adjoint's reversed grids at t = T (the paper always uses T = 128 = a multiple of cf^(levels-1)). */
  MGRIT_FLAG_RAGGED_T = 4,
  /* The gi buffer of mgrit_gru_forward / mgrit_gru_adjoint has mgrit_gru_gi_bytes(cfg) bytes: the projection
   * gi[T,B,3H] followed by room for the bf16 copies of x, of [h_0; h] and of gi itself that the forward call makes
   * anyway in the bf16 operand mode; the adjoint call, given the same buffer (and the h that forward call returned),
   * reads them instead of converting x and h again, and linearises at the bf16 copy of gi (the values the forward
   * solve used) instead of the fp32 one.  Set it in the cfg of BOTH calls.  Ignored (and harmless) where no such
   * copies exist: fp32 operands, B not dividing 128, levels == 1, the serial entry points. */
  MGRIT_FLAG_GI_CARRIES_COPIES = 8,
  /* The caller never reads the fp32 values of gi: where the copies of MGRIT_FLAG_GI_CARRIES_COPIES exist (that flag
   * set, bf16 operands, B dividing 128, levels > 1) the forward call then writes only the bf16 copy of the
   * projection -- every kernel of the solve and of the adjoint reads that copy anyway -- and leaves the T*B*3H floats
   * at the start of the buffer untouched (0.8 GB of stores per layer of the default workload).  All outputs are
   * bit-identical with and without it.  Set it in the cfg of BOTH calls; ignored where the copies do not exist. */
  MGRIT_FLAG_GI_F32_UNUSED = 16,
  /* mgrit_gru_forward / gru_serial_forward only: h points to T + 1 slots [T+1,B,H] instead of T.  The call writes h_0
   * to slot 0 and h_t to slot t: the level-0 unknowns of the solve live in the caller's array itself and the copy of
   * T*B*H floats that otherwise ends the call is saved (same bits).  The adjoint calls take h + B*H as their h. */
  MGRIT_FLAG_H_LEADS_WITH_H0 = 32
};

/* Problem and cycle description (Algorithm "MGProp", remark "Beyond Two-Level", Section
 * "Coarse Grid Propagators").  Level l has N_l = T / cf^l points and time step cf^l * dt. */
typedef struct {
  int32_t T, B, I, H;   /* sequence length, batch, input width, hidden width; H % 8 == 0, I % 8 == 0 */
  int32_t cf;           /* coarsening factor c_f >= 2 */
  int32_t levels;       /* >= 1; 1 = plain serial sweep; needs T % cf^(levels-1) == 0 unless MGRIT_FLAG_RAGGED_T */
  int32_t iters;        /* number of MGRIT cycles (ForwardIters / BackwardIters of Algorithm "MGRITTraining") */
  int32_t cell;         /* MGRIT_CELL_CLASSIC: Eq. "gru-classic"; MGRIT_CELL_IMPLICIT: Eq. "gru-imap"; same on all levels */
  int32_t relax_fine;   /* relaxation on level 0: MGRIT_RELAX_F, MGRIT_RELAX_FCF (Eq. "fcf-relax"), MGRIT_RELAX_FCFCF, ... */
  int32_t relax_coarse; /* relaxation on levels 1 .. levels-2 */
  int32_t operands;     /* MGRIT_OPERANDS_FP32: FFMA everywhere; MGRIT_OPERANDS_BF16: bf16 tensor-core
                           operands with fp32 accumulation; states, gates and gradients stay fp32 (the
                           adjoint's gate coefficients, which only ever enter such operands, are kept
                           in bf16 inside the workspace); MGRIT_OPERANDS_TF32: every product on the tensor
                           cores as a three-term split of tf32 operands (x_hi w_hi + x_lo w_hi + x_hi w_lo),
                           fp32 accumulation and fp32 everything else: meets the fp32 tolerances;
                           MGRIT_OPERANDS_TF32_1PASS: operands rounded to tf32 once (10 mantissa bits).
                           The tf32 modes need H % 64 == 0, I % 16 == 0, (T*B) % 4 == 0 and serve the
                           mgrit_gru_* / gru_serial_* / gru_input_projection calls of one layer and the
                           mgrit_lstm_* calls (not the stacked-state calls). */
  int32_t flags;        /* OR of MGRIT_FLAG_*.  MGRIT_FLAG_SKIP_DUPLICATE_FRELAX: a cycle after the first starts
                           from C-points whose F-points the previous cycle's final F-relaxation already filled;
                           skip re-doing it (results are identical) */
  float dt;             /* fine time step (1.0 in every experiment of the paper) */
} mgrit_gru_cfg;

/* GRU parameters of Eq. "gru", PyTorch layout: rows r | z | n. */
typedef struct {
  const float* W_ih; /* [3H, I] */
  const float* W_hh; /* [3H, H] */
  const float* b_ih; /* [3H] */
  const float* b_hh; /* [3H] */
} gru_params;

/* Parameter gradients; overwritten, not accumulated. */
typedef struct {
  float* dW_ih; /* [3H, I] */
  float* dW_hh; /* [3H, H] */
  float* db_ih; /* [3H] */
  float* db_hh; /* [3H] */
} gru_grads;

/* Workspace sizes in bytes for this cfg.  fwd_bytes serves gru_input_projection,
 * mgrit_gru_forward and gru_serial_forward; adj_bytes serves mgrit_gru_adjoint and
 * gru_serial_backward.  Either output may be NULL. */
int mgrit_gru_workspace_bytes(const mgrit_gru_cfg* cfg, size_t* fwd_bytes, size_t* adj_bytes);

/* Building blocks of a time-sharded solve (Fig. "Parallel distribution of work in parallel-in-time training": every
 * device owns a contiguous piece of the time axis and advances its own points): one cell evaluation, or its adjoint,
 * for n*B independent rows given as contiguous arrays.  fp32 engine (FFMA) whatever cfg->operands says; cfg supplies
 * B, H and the cell.
 *   gru_step_rows:          out[n,B,H] = Phi_gamma(gi_rows[n,B,3H], u_prev[n,B,H])               (Eq. "gru", "gru-imap")
 *   gru_adjoint_step_rows:  out[n,B,H] = (dPhi_gamma/dh at (gi_rows, h_lin))^T mu[n,B,H]         (discrete adjoint of it)
 * ws: gru_adjoint_step_rows needs 5*n*B*H floats of device workspace (ws_bytes checked); gru_step_rows none.
 * Asynchronous on `stream`; all pointers device, 32-byte aligned. */
int gru_step_rows(const mgrit_gru_cfg* cfg, const gru_params* p, int32_t n, float gamma, const float* gi_rows, const float* u_prev,
                  float* out, mgrit_stream_t stream);
int gru_adjoint_step_rows(const mgrit_gru_cfg* cfg, const gru_params* p, int32_t n, float gamma, const float* gi_rows,
                          const float* h_lin, const float* mu, float* out, void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Size in bytes of the gi buffer for this cfg: T*B*3H floats, more with MGRIT_FLAG_GI_CARRIES_COPIES (0 for a bad cfg). */
size_t mgrit_gru_gi_bytes(const mgrit_gru_cfg* cfg);

/* gi[t] = W_ih x_t + b_ih for all t (input half of Eq. "gru"); computed once on the fine grid
 * and reused by every level and by the adjoint.  x[T,B,I] -> gi[T,B,3H]. */
int gru_input_projection(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, float* gi,
                         void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Forward propagation by cfg->iters MGRIT cycles from the zero initial guess (Algorithm
 * "MGRITTraining", forward block; Algorithm "MGProp"): relaxation, residual restriction,
 * FAS coarse equation, recursive / serial coarse solve, correction, final F-relaxation.
 *   x[T,B,I], h0[B,H]  -> gi[T,B,3H] (written: the projection, kept for the adjoint), h[T,B,H].
 *   resnorm: HOST array of cfg->iters floats or NULL; entry i = 2-norm of the level-0 C-point
 *   residual measured in cycle i after its pre-relaxation.  levels == 1 runs the serial sweep. */
int mgrit_gru_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0,
                      float* gi, float* h, float* resnorm, void* ws, size_t ws_bytes,
                      mgrit_stream_t stream);

/* Backward propagation by cfg->iters MGRIT cycles on the adjoint recurrence, time reversed
 * (Algorithm "MGRITTraining", backward block; Appendix "Training With MGRIT"), linearised at the
 * GIVEN states h (the possibly inexact forward result), followed by the time-parallel gradient
 * pass g_i = w_i dh_i/dTheta.
 *   dh_seed[T,B,H] or NULL: direct loss derivative w.r.t. every h_t (stacked layers);
 *   dhT[B,H] or NULL: direct loss derivative w.r.t. h_T, added to dh_seed[T-1]; one of the two
 *   must be given.  Outputs: dh[T,B,H] total dL/dh_t or NULL (a training step only needs dx and the gradients),
 *   dh0[B,H], dx[T,B,I] or NULL, grads.
 *   gi is the projection written by the forward call for the same x and parameters. */
int mgrit_gru_adjoint(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0,
                      const float* gi, const float* h, const float* dh_seed, const float* dhT,
                      float* dh, float* dh0, float* dx, const gru_grads* grads, float* resnorm,
                      void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Exact serial sweep h_t = Phi_dt(x_t, h_{t-1}), t = 1..T (the solution of Eq. "fine-res"), with
 * the same cell as level 0 of the MGRIT solve; also writes gi. cf/levels/iters are ignored. */
int gru_serial_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0,
                       float* gi, float* h, void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Exact back-propagation through time for the serial sweep; arguments as mgrit_gru_adjoint. */
int gru_serial_backward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* h0,
                        const float* gi, const float* h, const float* dh_seed, const float* dhT,
                        float* dh, float* dh0, float* dx, const gru_grads* grads,
                        void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Stacked layers in ONE state (tables of training parameters: "Num. Layers 2"): the state of a time point is the
 * stack of all layers' hidden states, layer k's input at a step is layer k-1's new state of the same step (layer 0
 * reads x), and one MGRIT cycle (Algorithm "MGProp") advances the whole stack; on level l every layer uses the cell
 * with time step cf^l.  With levels == 1 this is the serial sweep of the stacked network (the usual multi-layer GRU
 * for the classic cell and dt = 1).  The alternative -- one MGRIT solve per layer, the layer below solved first --
 * is composed from mgrit_gru_forward / mgrit_gru_adjoint by the caller.
 *   cfg->I is the input width of layer 0; layers >= 1 have input width H.  n_layers <= 8.
 *   layers: HOST array of n_layers gru_params (device pointers inside).  h0[n_layers,B,H]; h[T,n_layers,B,H];
 *   gi0[T,B,3H]: projection of x for layer 0 (written by the forward call, read by the adjoint call).
 *   Adjoint: linearised at the GIVEN states; on coarse levels the input of layer k >= 1 is the layer below's given
 *   state at the step's arrival time (restriction by injection for inputs as for states).
 *   dh_seed[T,n_layers,B,H] or NULL; dhT[B,H] or NULL: loss derivative w.r.t. the TOP layer's last state; dh (optional)
 *   and dh0 have the shapes of h and h0: the sensitivities of the states as step outputs; dx[T,B,I] or NULL;
 *   grads: HOST array of n_layers gru_grads.  The coarsest level is advanced step by step (no persistent chain). */
int mgrit_gru_stack_workspace_bytes(const mgrit_gru_cfg* cfg, int32_t n_layers, size_t* fwd_bytes, size_t* adj_bytes);
int mgrit_gru_stack_forward(const mgrit_gru_cfg* cfg, int32_t n_layers, const gru_params* layers, const float* x, const float* h0,
                            float* gi0, float* h, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream);
int mgrit_gru_stack_adjoint(const mgrit_gru_cfg* cfg, int32_t n_layers, const gru_params* layers, const float* x, const float* h0,
                            const float* gi0, const float* h, const float* dh_seed, const float* dhT, float* dh, float* dh0,
                            float* dx, const gru_grads* grads, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Implicit LSTM (the paper's conclusion names the LSTM as a cell the same implicit treatment applies to).  Reading:
 * the cell state is a unit-step forward-Euler update of c' = -(1-f) c + i g, as Eq. "gru-classic" reads the GRU, and
 * the stiff decay term is taken implicitly as in Eq. "gru-implicit": (1 + gamma (1-f)) c_t = c_{t-1} + gamma i g;
 * h_t = o tanh(c_t) is re-evaluated from the new cell state.  cfg->cell selects this (MGRIT_CELL_IMPLICIT) or the
 * explicit update (MGRIT_CELL_CLASSIC: with dt = 1 the textbook LSTM); level l uses gamma = cf^l dt.
 *   Parameters: gru_params with W_ih[4H,I], W_hh[4H,H], b_ih[4H], b_hh[4H], gate order i | f | g | o.
 *   The state of a time point is (c, h): u0[2,B,H], u[T,2,B,H], du_seed / du likewise; gi[T,B,4H].
 *   dhT[B,H]: loss derivative w.r.t. the last HIDDEN state.  grads: one gru_grads with the 4H-row shapes.
 *   Everything else (cycles, relaxation, flags, resnorm, levels == 1 = serial sweep / exact BPTT) as for the GRU calls.
 *   Operand modes: MGRIT_OPERANDS_FP32 (FFMA), the tf32 modes and MGRIT_OPERANDS_BF16 (tcgen05 products on four-gate
 *   tiles of 64 hidden units; same shape limits and tolerances as for the GRU). */
int mgrit_lstm_workspace_bytes(const mgrit_gru_cfg* cfg, size_t* fwd_bytes, size_t* adj_bytes);
int mgrit_lstm_forward(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, float* gi, float* u,
                       float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream);
int mgrit_lstm_adjoint(const mgrit_gru_cfg* cfg, const gru_params* p, const float* x, const float* u0, const float* gi,
                       const float* u, const float* du_seed, const float* dhT, float* du, float* du0, float* dx,
                       const gru_grads* grads, float* resnorm, void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* Classifier head on h_T with mean softmax cross-entropy (the loss whose gradient seeds the
 * backward block: w_T = grad_{h_T} L).  hT[B,H], Wc[C,H], bc[C], labels[B] (int32, device)
 * -> loss[1] (device), dhT[B,H], dWc[C,H], dbc[C].  ws: device scratch of at least
 * xent_head_workspace_bytes(B, C) bytes.  C <= 8192 (the logits of a row are kept in shared memory), otherwise
 * MGRIT_UNSUPPORTED.  A label outside [0, C) marks a row without a target: it contributes nothing to the loss and
 * has no one-hot term (the mean still divides by B).  All sums run in a fixed order: results repeat bit for bit. */
size_t xent_head_workspace_bytes(int32_t B, int32_t C);
int xent_head_fwd_bwd(int32_t B, int32_t H, int32_t C, const float* hT, const float* Wc, const float* bc,
                      const int32_t* labels, float* loss, float* dhT, float* dWc, float* dbc,
                      void* ws, size_t ws_bytes, mgrit_stream_t stream);

/* The same classifier head for callers that cannot allocate device memory (the paper has no
 * counterpart; this exists for hosts of the library).  Typical cases: a process whose own memory
 * arena already owns all of the GPU's memory, so that cudaMalloc fails or would fragment it, and
 * latency-critical loops that must stay clear of the driver's allocator, which takes a global lock
 * and may synchronise the device.  Instead of a workspace argument the [B, C] intermediate (loss
 * derivative w.r.t. the logits) is kept in a fixed 256 KiB array that is part of the library image:
 * every GPU that loads the library holds it until the process exits.
 *   Limit: B * (C + 1) <= 65536 (the derivatives and one loss term per row), otherwise MGRIT_SCRATCH_LIMIT is
 *   returned and nothing is launched; C <= 8192 as for xent_head_fwd_bwd (MGRIT_UNSUPPORTED).
 *   The call performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   The first call on each device looks up the array's device address (once per device, with that
 *   device current); make that first call before any stream capture is started on the device.
 *   All calls share the one array, which keeps the previous call's contents; nothing in it needs to be
 *   cleared between calls (each call overwrites the B * (C + 1) entries it reads).  Two calls that overlap on
 *   the GPU (different streams, or different host threads) race on it: serialise them.
 *   Inputs, outputs and results are exactly those of xent_head_fwd_bwd. */
int xent_head_fwd_bwd_noalloc(int32_t B, int32_t H, int32_t C, const float* hT, const float* Wc, const float* bc,
                              const int32_t* labels, float* loss, float* dhT, float* dWc, float* dbc,
                              mgrit_stream_t stream);

/* Theta <- Theta - lr * g (last line of Algorithm "MGRITTraining"); n fp32 elements. */
int sgd_update(float* p, const float* g, size_t n, float lr, mgrit_stream_t stream);

/* Adam step with bias correction, the optimiser of the paper's experiments (Section "Training with MGRIT";
 * tables of training parameters: Adam, learning rate 0.001).  Same update as the usual Adam without weight
 * decay:  m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;  p <- p - lr/(1-b1^t) * m / (sqrt(v)/sqrt(1-b2^t) + eps).
 * p, g, m, v: n fp32 elements each (device; m and v are the caller-owned moment buffers, zero before step 1);
 * step = t >= 1. */
int adam_update(float* p, const float* g, float* m, float* v, size_t n, float lr, float beta1, float beta2, float eps,
                int32_t step, mgrit_stream_t stream);

/* Status of the bounded device-side waits on the current device since the library was loaded or the status was
 * last cleared: MGRIT_OK, or MGRIT_DEVICE_TIMEOUT when one ran out.  Synchronises the device.
 * The status words are sticky: once a wait has run out, every later persistent kernel on that device sees the
 * non-zero word and leaves early (its results are then incomplete), until mgrit_gru_clear_device_status() is
 * called.  Asynchronous calls cannot report the condition themselves; after MGRIT_DEVICE_TIMEOUT discard the
 * results computed since the last MGRIT_OK status, clear the status and repeat the work. */
int mgrit_gru_last_device_status(void);
/* Synchronises the current device and resets its status words to zero. */
int mgrit_gru_clear_device_status(void);

/* Self-test of the bounded device-side waits (no counterpart in the paper): launches one warp that waits, with the
 * library's own wait routine and a limit of limit_ms (1..1000) instead of the 2 s of the real kernels, on a barrier
 * that nothing signals.  The wait runs out, the kernel records it in the status word and returns normally; afterwards
 * mgrit_gru_last_device_status() reports MGRIT_DEVICE_TIMEOUT until mgrit_gru_clear_device_status() is called.
 * Asynchronous on `stream`. */
int mgrit_gru_selftest_bounded_wait(int32_t limit_ms, mgrit_stream_t stream);

/* Number of kernels this library has launched since it was loaded (all streams). */
unsigned long long mgrit_gru_kernel_launches(void);

/* Measurement aid (no counterpart in the paper): while enabled, every launch of a GEMM-shaped
 * kernel is bracketed by CUDA events on its stream.  mgrit_gru_profile_enable(1) clears earlier
 * records and starts recording, (0) stops.  mgrit_gru_profile_read synchronises the device and
 * returns, for one kernel class, the summed launch durations (ms), the number of launches and
 * their algorithmic flops (2*M*N*K).  Classes: 0 input projection, 1 forward relaxation step,
 * 2 adjoint linearisation, 3 adjoint relaxation step, 4 weight/input gradient GEMMs, 5 / 6 forward /
 * adjoint persistent serial chain (all dependent steps of the coarsest level in one launch). */
int mgrit_gru_profile_enable(int on);
int mgrit_gru_profile_read(int kernel_class, double* total_ms, unsigned long long* launches, double* flops);
/* The individual records in launch order: duration (ms), algorithmic flops and class of each
 * recorded launch; writes min(cap, *n) entries and the total count to *n (HOST arrays). */
int mgrit_gru_profile_records(double* ms, double* flops, int32_t* kernel_class, size_t cap, size_t* n);

const char* mgrit_gru_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* MGRIT_GRU_H_ */
