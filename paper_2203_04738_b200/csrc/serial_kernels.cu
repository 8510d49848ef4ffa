// Persistent kernels for chains of DEPENDENT steps with few rows (the serial coarsest-level solve of
// the multigrid cycle and the exact serial sweep; forward and adjoint).  One launch advances all
// steps: every CTA keeps its slice of the recurrent weight matrix in shared memory for the whole
// chain, the state crosses CTAs through L2 once per step as a bf16 operand copy, and the steps are
// separated by a grid barrier with a bounded wait.  16 batch rows per CTA row group (row groups never
// interact), bf16 mma.sync m16n8k16 with fp32 accumulation, K split over the 8 warps of a CTA.
//
// A wait that runs out writes a non-zero code to the status word; every CTA that sees a non-zero
// status leaves at its next barrier, so the launch always terminates.
#include <stdlib.h>

#include "cell.cuh"
#include "serial_engine.cuh"

namespace mg {

namespace {

typedef __nv_bfloat16 bf16;
constexpr int kThreads = 256, kWarps = 8, kRows = 16;
constexpr uint64_t kWaitLimitNs = 2000000000ull;

__device__ int g_serial_status = 0;
int* g_serial_status_ptrs[kMaxDevices] = {nullptr};   // its address on each device

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// All CTAs that share `ctr` have finished the step whose arrival count is `target`.
__device__ __forceinline__ bool grid_barrier(unsigned* ctr, unsigned target, int* status, int* ok_smem) {
  __syncthreads();
  if (threadIdx.x == 0) {
    // release: the CTA's stores (ordered before this thread by the barrier above) become visible before the count
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
    int ok = 1;
    unsigned spins = 0;
    uint64_t t0 = 0;
    while (ld_acquire(ctr) < target) {
      if ((++spins & 127u) == 0) {
        if (t0 == 0) t0 = global_ns();
        if (ld_relaxed(status) != 0) { ok = 0; break; }
        if (global_ns() - t0 > kWaitLimitNs) { atomicCAS(status, 0, 5); ok = 0; break; }
      }
    }
    *ok_smem = ok;      // the acquire load above orders the reloads that follow the barrier below
  }
  __syncthreads();
  return *ok_smem != 0;
}

// 16-byte asynchronous copy global (through L2, not L1) -> shared: no register staging, so a thread keeps all
// of its copies of a reload in flight at once instead of a few dependent load/store pairs.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// ---- exchange of the new state between CTAs with the "ready" flag inside the data --------------------------------
// A 16-byte word carries six bf16 values and the number of the step that produced them; it is written by ONE
// 16-byte store of one thread (a single transaction inside one 32-byte sector), so a reader that sees the step
// number sees the six values too.  Readers poll the words they need directly: one trip to L2 once the data is
// there, instead of an arrival counter, a poll of that counter and a reload.  Two buffers alternate by step
// parity: a CTA writes step j + 2 only after it has read all of step j + 1, which nobody could produce before
// reading all of step j.  The host clears the words before every launch (step numbers start at 1).
constexpr int kValsPerWord = 6;
__device__ __forceinline__ uint4 ld_word(const uint4* p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_word(uint4* p, uint4 v) {
  asm volatile("st.volatile.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// Words of one producer block of `nvals` bf16 values (a multiple of 2) staged in shared memory -> global, tagged `step`.
__device__ __forceinline__ void publish_block(const bf16* stage, int nvals, uint4* dst, unsigned step) {
  const int nwords = (nvals + kValsPerWord - 1) / kValsPerWord;
  for (int w = threadIdx.x; w < nwords; w += kThreads) {
    const uint32_t* s32 = reinterpret_cast<const uint32_t*>(stage) + 3 * w;      // values 6w .. 6w+5 as three pairs
    uint4 v;
    v.x = 6 * w < nvals ? s32[0] : 0u;
    v.y = 6 * w + 2 < nvals ? s32[1] : 0u;
    v.z = 6 * w + 4 < nvals ? s32[2] : 0u;
    v.w = step;
    st_word(dst + w, v);
  }
}
// All producers' blocks of step `step` -> the CTA's operand rows in shared memory.  A block holds GATES x 16 x UNC
// values in the order [gate][row][unit]; value (g, r, i) of producer x goes to As[r][g*H + x*UNC + i].
// Every round a thread issues the loads of all its words that are still missing together and then looks at what
// came back, so a round costs one trip to L2 however many words are outstanding.
template <int UNC, int GATES>
__device__ __forceinline__ bool gather_blocks(const uint4* src, int nprod, unsigned step, bf16* As, int ldk, int H, int* status) {
  constexpr int kBlockVals = GATES * kRows * UNC, kBlockWords = (kBlockVals + kValsPerWord - 1) / kValsPerWord;
  constexpr int kBatch = GATES == 1 ? 12 : 16;
  const int total = nprod * kBlockWords;
  for (int base = threadIdx.x; base < total; base += kThreads * kBatch) {
    unsigned pending = 0;
#pragma unroll
    for (int q = 0; q < kBatch; ++q)
      if (base + q * kThreads < total) pending |= 1u << q;
    unsigned rounds = 0;
    uint64_t t0 = 0;
    while (pending) {
      uint4 v[kBatch];
#pragma unroll
      for (int q = 0; q < kBatch; ++q)
        if (pending & (1u << q)) v[q] = ld_word(src + base + q * kThreads);
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        if ((pending & (1u << q)) && v[q].w == step) {
          pending &= ~(1u << q);
          const int e = base + q * kThreads, x = e / kBlockWords, w = e % kBlockWords;
          const uint32_t d[3] = {v[q].x, v[q].y, v[q].z};
#pragma unroll
          for (int t = 0; t < 3; ++t) {
            const int vv = kValsPerWord * w + 2 * t;
            if (vv < kBlockVals) {
              const int g = vv / (kRows * UNC), r = (vv / UNC) % kRows, i = vv % UNC;
              *reinterpret_cast<uint32_t*>(As + r * ldk + g * H + x * UNC + i) = d[t];
            }
          }
        }
      }
      if (pending && (++rounds & 31u) == 0) {      // bounded: give up once the status word is set or after the limit
        if (t0 == 0) t0 = global_ns();
        if (ld_relaxed(status) != 0) return false;
        if (global_ns() - t0 > kWaitLimitNs) { atomicCAS(status, 0, 6); return false; }
      }
    }
  }
  return true;
}

__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// acc[nt] += As[16, kbeg:kend] * Ws[nt*8 .. nt*8+8, kbeg:kend]^T   (both K-contiguous, row pitch ldk)
template <int NT>
__device__ __forceinline__ void warp_gemm(const bf16* As, const bf16* Ws, int ldk, int kbeg, int kend, float (*acc)[4]) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  for (int k0 = kbeg; k0 < kend; k0 += 16) {
    uint32_t a[4];
    a[0] = *reinterpret_cast<const uint32_t*>(As + g * ldk + k0 + 2 * t);
    a[1] = *reinterpret_cast<const uint32_t*>(As + (g + 8) * ldk + k0 + 2 * t);
    a[2] = *reinterpret_cast<const uint32_t*>(As + g * ldk + k0 + 2 * t + 8);
    a[3] = *reinterpret_cast<const uint32_t*>(As + (g + 8) * ldk + k0 + 2 * t + 8);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const bf16* wr = Ws + (nt * 8 + g) * ldk + k0 + 2 * t;
      mma16816(acc[nt], a, *reinterpret_cast<const uint32_t*>(wr), *reinterpret_cast<const uint32_t*>(wr + 8));
    }
  }
}

// The same product with the B fragments (the CTA's weight slice, constant for the whole chain) held in registers:
// w[ks][nt] = the two words a lane feeds to the product of k-step ks and column tile nt.  Same instructions in the same
// order as warp_gemm, so the results are bit-identical; the shared-memory reads of the weights disappear.
template <int NT, int KS>
__device__ __forceinline__ void load_wregs(const bf16* Ws, int ldk, int kbeg, uint32_t (&w)[KS][NT][2]) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const bf16* wr = Ws + (nt * 8 + g) * ldk + kbeg + 16 * ks + 2 * t;
      w[ks][nt][0] = *reinterpret_cast<const uint32_t*>(wr);
      w[ks][nt][1] = *reinterpret_cast<const uint32_t*>(wr + 8);
    }
}
template <int NT, int KS>
__device__ __forceinline__ void warp_gemm_regs(const bf16* As, int ldk, int kbeg, const uint32_t (&w)[KS][NT][2], float (*acc)[4]) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int ks = 0; ks < KS; ++ks) {
    const int k0 = kbeg + 16 * ks;
    uint32_t a[4];
    a[0] = *reinterpret_cast<const uint32_t*>(As + g * ldk + k0 + 2 * t);
    a[1] = *reinterpret_cast<const uint32_t*>(As + (g + 8) * ldk + k0 + 2 * t);
    a[2] = *reinterpret_cast<const uint32_t*>(As + g * ldk + k0 + 2 * t + 8);
    a[3] = *reinterpret_cast<const uint32_t*>(As + (g + 8) * ldk + k0 + 2 * t + 8);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) mma16816(acc[nt], a, w[ks][nt][0], w[ks][nt][1]);
  }
}

// warp partial sums -> red[warp][row][col]   (col < NT*8)
template <int NT>
__device__ __forceinline__ void store_partials(float* red, float (*acc)[4]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  constexpr int NC = NT * 8;
  float* base = red + warp * kRows * NC;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    base[g * NC + nt * 8 + 2 * t] = acc[nt][0];
    base[g * NC + nt * 8 + 2 * t + 1] = acc[nt][1];
    base[(g + 8) * NC + nt * 8 + 2 * t] = acc[nt][2];
    base[(g + 8) * NC + nt * 8 + 2 * t + 1] = acc[nt][3];
  }
}
template <int NC>
__device__ __forceinline__ float sum_partials(const float* red, int row, int col) {
  float s = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) s += red[(w * kRows + row) * NC + col];
  return s;
}

// A projection value as the chain's prefetch loads it and as the cell uses it.  Nothing may depend on the load before the
// exchange (a dependent instruction would wait for DRAM there), so a bf16 source is kept as its raw 16 bits in the
// register and widened only at the use; an fp32 source is rounded to bf16 at the use when the solve's other levels read
// the bf16 copy.
__device__ __forceinline__ float ld_gi(const SerialFwdArgs& a, i64 idx) {
  if (a.gi_b) return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(a.gi_b)[idx]);
  return a.gi[idx];
}
__device__ __forceinline__ float use_gi(const SerialFwdArgs& a, float raw) {
  if (a.gi_b) return __uint_as_float(__float_as_uint(raw) << 16);
  return a.gi_as_bf16 ? bf16_round(raw) : raw;
}

// ------------------------------------------------------------------------------------------------
// forward chain:  u_j = Phi_gamma(gi_j, u_{j-1}) + g_j ,  j = 1..nsteps
// KS > 0: the weight fragments live in registers (KS = k-steps of 16 per warp = H / 128; see warp_gemm_regs).
template <int UNC, bool LL, int KS = 0>
__global__ void __launch_bounds__(kThreads, 1) serial_fwd_kernel(SerialFwdArgs a, int* status) {
  constexpr int NW = 3 * UNC, NT = NW / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  constexpr int kBlockVals = kRows * UNC, kBlockWords = (kBlockVals + kValsPerWord - 1) / kValsPerWord;
  __shared__ __align__(16) bf16 xstage[kRows * 32];
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, ldk = H + 8;
  bf16* Ws = reinterpret_cast<bf16*>(smem);                 // [NW][ldk]
  bf16* As = Ws + NW * ldk;                                 // [16][ldk]
  float* red = reinterpret_cast<float*>(As + kRows * ldk);  // [8][16][NW]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const unsigned ncta_rg = gridDim.x;
  const i64 BH = (i64)a.B * H;

  // weights of this CTA's units (rows gate*H + u0 + i), resident for the whole chain
  for (int e = tid; e < NW * (H / 8); e += kThreads) {
    int r = e / (H / 8), c = e % (H / 8);
    int gate = r / UNC, i = r % UNC;
    *reinterpret_cast<uint4*>(Ws + r * ldk + c * 8) =
        __ldg(reinterpret_cast<const uint4*>(a.W + ((i64)gate * H + u0 + i) * H + c * 8));
  }
  // rows beyond the batch stay zero
  for (int e = tid; e < kRows * ldk / 2; e += kThreads) reinterpret_cast<uint32_t*>(As)[e] = 0u;
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  // step 1 reads the fp32 initial state
  for (int e = tid; e < nrows * (H / 4); e += kThreads) {
    int r = e / (H / 4), c = e % (H / 4);
    float4 v = __ldcg(reinterpret_cast<const float4*>(a.u + (i64)(row0 + r) * H + c * 4));
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 o; o.x = *reinterpret_cast<uint32_t*>(&lo); o.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(As + r * ldk + c * 4) = o;
  }
  // outputs owned by this thread: (row, unit) pairs; previous value carried in registers
  float hp[OPT], pgr[OPT], pgz[OPT], pgn[OPT], pg[OPT];
  float br[OPT], bz[OPT], bn[OPT];
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    hp[o] = v ? __ldcg(a.u + (i64)(row0 + r) * H + u0 + i) : 0.f;
    br[o] = a.b_hh[u0 + i]; bz[o] = a.b_hh[H + u0 + i]; bn[o] = a.b_hh[2 * H + u0 + i];
    const i64 go = (i64)(row0 + r) * 3 * H + u0 + i;
    pgr[o] = v ? ld_gi(a, go) : 0.f; pgz[o] = v ? ld_gi(a, go + H) : 0.f; pgn[o] = v ? ld_gi(a, go + 2 * H) : 0.f;
    pg[o] = (v && a.g) ? a.g[BH + (i64)(row0 + r) * H + u0 + i] : 0.f;
  }
  __syncthreads();

  const int kw = H / kWarps;
  uint32_t wreg[KS > 0 ? KS : 1][NT][2];
  if (KS > 0) load_wregs<NT, (KS > 0 ? KS : 1)>(Ws, ldk, warp * kw, wreg);
  for (int j = 1; j <= a.nsteps; ++j) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    if (KS > 0) warp_gemm_regs<NT, (KS > 0 ? KS : 1)>(As, ldk, warp * kw, wreg, acc);
    else warp_gemm<NT>(As, Ws, ldk, warp * kw, (warp + 1) * kw, acc);
    store_partials<NT>(red, acc);
    __syncthreads();
    bf16* ub = a.ub + (i64)(j & 1) * BH;
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      float val = 0.f;
      if (idx < kRows * UNC && r < nrows) {
        float ghr = sum_partials<NW>(red, r, i) + br[o];
        float ghz = sum_partials<NW>(red, r, UNC + i) + bz[o];
        float ghn = sum_partials<NW>(red, r, 2 * UNC + i) + bn[o];
        const float gir = use_gi(a, pgr[o]), giz = use_gi(a, pgz[o]), gin = use_gi(a, pgn[o]);
        val = cell_forward<true>(gir, giz, gin, ghr, ghz, ghn, hp[o], a.gamma, a.cell) + pg[o];
        hp[o] = val;
        i64 off = (i64)(row0 + r) * H + u0 + i;
        a.u[(i64)j * BH + off] = val;
        if (!LL) ub[off] = __float2bfloat16(val);
      }
      if (LL && idx < kRows * UNC) xstage[idx] = __float2bfloat16(val);      // rows beyond the batch travel as zeros
    }
    if (j == a.nsteps) break;
    if (LL) {
      __syncthreads();
      publish_block(xstage, kBlockVals, a.xw + ((i64)(rg * 2 + (j & 1)) * gridDim.x + blockIdx.x) * kBlockWords, (unsigned)j);
    }
    // operands of the next step that do not depend on other CTAs
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        const i64 go = (i64)j * a.gi_step + (i64)(row0 + r) * 3 * H + u0 + i;
        // (loaded now, rounded where they are used: an instruction that depends on these loads here would wait for them
        // in front of the exchange)
        pgr[o] = ld_gi(a, go); pgz[o] = ld_gi(a, go + H); pgn[o] = ld_gi(a, go + 2 * H);
        if (a.g) pg[o] = a.g[(i64)(j + 1) * BH + (i64)(row0 + r) * H + u0 + i];
      }
    }
    if (LL) {
      // the full new state of this row group, as the bf16 A operand: every producer's words, polled in place
      const bool ok = gather_blocks<UNC, 1>(a.xw + (i64)(rg * 2 + (j & 1)) * gridDim.x * kBlockWords, (int)gridDim.x, (unsigned)j, As, ldk,
                                            H, status);
      if (!ok) ok_smem = 0;
      __syncthreads();
      if (ok_smem == 0) return;
    } else {
      if (!grid_barrier(a.bar + rg, (unsigned)j * ncta_rg, status, &ok_smem)) return;
      // the full new state of this row group, as the bf16 A operand
      for (int e = tid; e < nrows * (H / 8); e += kThreads) {
        int r = e / (H / 8), c = e % (H / 8);
        cp_async16(As + r * ldk + c * 8, ub + (i64)(row0 + r) * H + c * 8);
      }
      cp_async_wait_all();
      __syncthreads();
    }
  }
}

// ------------------------------------------------------------------------------------------------
// adjoint chain:  mu_s = a_s * mu_{s-1} + [cr_s|cz_s|cn_s]*mu_{s-1} W_hh + g_s ,  s = 1..nsteps
// The bf16 operand copy carries dA_{s+1} = [cr|cz|cn]_{s+1} * mu_s, formed by the CTA that produced mu_s.
template <int UNC, bool LL, int KS = 0>     // KS > 0: weight fragments in registers, KS = 3H / 128
__global__ void __launch_bounds__(kThreads, 1) serial_adj_kernel(SerialAdjArgs a, int* status) {
  constexpr int NT = UNC / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  constexpr int kBlockVals = 3 * kRows * UNC, kBlockWords = (kBlockVals + kValsPerWord - 1) / kValsPerWord;
  __shared__ __align__(16) bf16 xstage[3 * kRows * 32];
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, K = 3 * H, ldk = K + 8;
  bf16* Ws = reinterpret_cast<bf16*>(smem);                 // [UNC][ldk]   rows of W_hh^T
  bf16* As = Ws + UNC * ldk;                                // [16][ldk]
  float* red = reinterpret_cast<float*>(As + kRows * ldk);  // [8][16][UNC]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const unsigned ncta_rg = gridDim.x;
  const i64 BH = (i64)a.B * H;

  for (int e = tid; e < UNC * (K / 8); e += kThreads) {
    int r = e / (K / 8), c = e % (K / 8);
    *reinterpret_cast<uint4*>(Ws + r * ldk + c * 8) = __ldg(reinterpret_cast<const uint4*>(a.WT + (i64)(u0 + r) * K + c * 8));
  }
  for (int e = tid; e < kRows * ldk / 2; e += kThreads) reinterpret_cast<uint32_t*>(As)[e] = 0u;
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  // step 1: dA_1 = c_1 * mu_0 for all 3H columns of this row group
  for (int e = tid; e < nrows * H; e += kThreads) {
    int r = e / H, i = e % H;
    i64 off = (i64)(row0 + r) * H + i;
    float m = __ldcg(a.mu + off);
    As[r * ldk + i] = __float2bfloat16(__bfloat162float(a.cr[off]) * m);
    As[r * ldk + H + i] = __float2bfloat16(__bfloat162float(a.cz[off]) * m);
    As[r * ldk + 2 * H + i] = __float2bfloat16(__bfloat162float(a.cn[off]) * m);
  }
  float mp[OPT], pa[OPT], pg[OPT];
  bf16 ncr[OPT], ncz[OPT], ncn[OPT];   // kept raw: converting at the load would wait for it before the barrier
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    i64 off = (i64)(row0 + r) * H + u0 + i;
    mp[o] = v ? __ldcg(a.mu + off) : 0.f;
    pa[o] = v ? a.a[off] : 0.f;
    pg[o] = (v && a.g) ? a.g[BH + off] : 0.f;
    bool more = v && a.nsteps > 1;
    const bf16 zero = __float2bfloat16(0.f);
    ncr[o] = more ? a.cr[a.coef_step + off] : zero;
    ncz[o] = more ? a.cz[a.coef_step + off] : zero;
    ncn[o] = more ? a.cn[a.coef_step + off] : zero;
  }
  __syncthreads();

  const int kw = K / kWarps;
  uint32_t wreg[KS > 0 ? KS : 1][NT][2];
  if (KS > 0) load_wregs<NT, (KS > 0 ? KS : 1)>(Ws, ldk, warp * kw, wreg);
  for (int s = 1; s <= a.nsteps; ++s) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    if (KS > 0) warp_gemm_regs<NT, (KS > 0 ? KS : 1)>(As, ldk, warp * kw, wreg, acc);
    else warp_gemm<NT>(As, Ws, ldk, warp * kw, (warp + 1) * kw, acc);
    store_partials<NT>(red, acc);
    __syncthreads();
    bf16* dAb = a.dAb + (i64)(s & 1) * 3 * BH;
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      float val = 0.f;
      const bool live = idx < kRows * UNC && r < nrows;
      if (live) {
        val = pa[o] * mp[o] + sum_partials<UNC>(red, r, i) + pg[o];
        mp[o] = val;
        i64 off = (i64)(row0 + r) * H + u0 + i;
        a.mu[(i64)s * BH + off] = val;
        if (!LL && s < a.nsteps) {
          bf16* d = dAb + (i64)(row0 + r) * K + u0 + i;
          d[0] = __float2bfloat16(__bfloat162float(ncr[o]) * val);
          d[H] = __float2bfloat16(__bfloat162float(ncz[o]) * val);
          d[2 * H] = __float2bfloat16(__bfloat162float(ncn[o]) * val);
        }
      }
      if (LL && idx < kRows * UNC) {     // block order [gate][row][unit]; rows beyond the batch travel as zeros
        xstage[idx] = __float2bfloat16(live ? __bfloat162float(ncr[o]) * val : 0.f);
        xstage[kRows * UNC + idx] = __float2bfloat16(live ? __bfloat162float(ncz[o]) * val : 0.f);
        xstage[2 * kRows * UNC + idx] = __float2bfloat16(live ? __bfloat162float(ncn[o]) * val : 0.f);
      }
    }
    if (s == a.nsteps) break;
    if (LL) {
      __syncthreads();
      publish_block(xstage, kBlockVals, a.xw + ((i64)(rg * 2 + (s & 1)) * gridDim.x + blockIdx.x) * kBlockWords, (unsigned)s);
    }
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        i64 off = (i64)(row0 + r) * H + u0 + i;
        pa[o] = a.a[(i64)s * a.coef_step + off];
        if (a.g) pg[o] = a.g[(i64)(s + 1) * BH + off];
        if (s + 1 < a.nsteps) {
          i64 co = (i64)(s + 1) * a.coef_step + off;
          ncr[o] = a.cr[co]; ncz[o] = a.cz[co]; ncn[o] = a.cn[co];
        }
      }
    }
    if (LL) {
      const bool ok = gather_blocks<UNC, 3>(a.xw + (i64)(rg * 2 + (s & 1)) * gridDim.x * kBlockWords, (int)gridDim.x, (unsigned)s, As, ldk,
                                            H, status);
      if (!ok) ok_smem = 0;
      __syncthreads();
      if (ok_smem == 0) return;
    } else {
      if (!grid_barrier(a.bar + rg, (unsigned)s * ncta_rg, status, &ok_smem)) return;
      for (int e = tid; e < nrows * (K / 8); e += kThreads) {
        int r = e / (K / 8), c = e % (K / 8);
        cp_async16(As + r * ldk + c * 8, dAb + (i64)(row0 + r) * K + c * 8);
      }
      cp_async_wait_all();
      __syncthreads();
    }
  }
}

// ================================================================================================
// Implicit LSTM chains (bf16 operands, flag-in-data exchange).  The structure is that of the GRU chains above; a
// time point's state is (c, h): the cell state never leaves the thread that owns its (row, unit), only h crosses CTAs.
//
// forward:  gates from gi_j and h_{j-1} W_hh^T (four gate rows per unit in shared memory), (c, h)_j = cell + g_j
template <int UNC>
__global__ void __launch_bounds__(kThreads, 1) lstm_fwd_chain_kernel(LstmChainFwdArgs a, int* status) {
  constexpr int NW = 4 * UNC, NT = NW / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  constexpr int kBlockVals = kRows * UNC, kBlockWords = (kBlockVals + kValsPerWord - 1) / kValsPerWord;
  __shared__ __align__(16) bf16 xstage[kRows * 32];
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, ldk = H + 8;
  bf16* Ws = reinterpret_cast<bf16*>(smem);                 // [NW][ldk]
  bf16* As = Ws + NW * ldk;                                 // [16][ldk]
  float* red = reinterpret_cast<float*>(As + kRows * ldk);  // [8][16][NW]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const i64 BH = (i64)a.B * H, slot = 2 * BH;

  for (int e = tid; e < NW * (H / 8); e += kThreads) {      // weight rows gate*H + u0 + i, resident for the whole chain
    int r = e / (H / 8), c = e % (H / 8);
    int gate = r / UNC, i = r % UNC;
    *reinterpret_cast<uint4*>(Ws + r * ldk + c * 8) =
        __ldg(reinterpret_cast<const uint4*>(a.W + ((i64)gate * H + u0 + i) * H + c * 8));
  }
  for (int e = tid; e < kRows * ldk / 2; e += kThreads) reinterpret_cast<uint32_t*>(As)[e] = 0u;     // rows beyond the batch stay zero
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  for (int e = tid; e < nrows * (H / 4); e += kThreads) {   // step 1 reads the fp32 initial hidden state
    int r = e / (H / 4), c = e % (H / 4);
    float4 v = __ldcg(reinterpret_cast<const float4*>(a.u + BH + (i64)(row0 + r) * H + c * 4));
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 o; o.x = *reinterpret_cast<uint32_t*>(&lo); o.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(As + r * ldk + c * 4) = o;
  }
  float cp[OPT], pgi[OPT][4], bia[OPT][4], pgc[OPT], pgh[OPT];
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    const i64 off = (i64)(row0 + r) * H + u0 + i;
    cp[o] = v ? __ldcg(a.u + off) : 0.f;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      bia[o][g] = a.b_hh[g * H + u0 + i];
      pgi[o][g] = v ? a.gi[(i64)(row0 + r) * 4 * H + g * H + u0 + i] : 0.f;
    }
    pgc[o] = (v && a.g) ? a.g[slot + off] : 0.f;
    pgh[o] = (v && a.g) ? a.g[slot + BH + off] : 0.f;
  }
  __syncthreads();

  const int kw = H / kWarps;
  for (int j = 1; j <= a.nsteps; ++j) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    warp_gemm<NT>(As, Ws, ldk, warp * kw, (warp + 1) * kw, acc);
    store_partials<NT>(red, acc);
    __syncthreads();
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      float hv = 0.f;
      if (idx < kRows * UNC && r < nrows) {
        float gh[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) gh[g] = sum_partials<NW>(red, r, g * UNC + i) + bia[o][g];
        LstmOut q = lstm_forward<true>(pgi[o][0], pgi[o][1], pgi[o][2], pgi[o][3], gh[0], gh[1], gh[2], gh[3], cp[o], a.gamma, a.cell);
        const float cv = q.c + pgc[o];
        hv = q.h + pgh[o];
        cp[o] = cv;
        const i64 off = (i64)(row0 + r) * H + u0 + i;
        a.u[(i64)j * slot + off] = cv;
        a.u[(i64)j * slot + BH + off] = hv;
      }
      if (idx < kRows * UNC) xstage[idx] = __float2bfloat16(hv);      // rows beyond the batch travel as zeros
    }
    if (j == a.nsteps) break;
    __syncthreads();
    publish_block(xstage, kBlockVals, a.xw + ((i64)(rg * 2 + (j & 1)) * gridDim.x + blockIdx.x) * kBlockWords, (unsigned)j);
    // operands of the next step that do not depend on other CTAs (nothing may depend on these loads before the exchange)
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        const float* gi = a.gi + (i64)j * a.gi_step + (i64)(row0 + r) * 4 * H + u0 + i;
#pragma unroll
        for (int g = 0; g < 4; ++g) pgi[o][g] = gi[g * H];
        if (a.g) {
          const i64 off = (i64)(j + 1) * slot + (i64)(row0 + r) * H + u0 + i;
          pgc[o] = a.g[off]; pgh[o] = a.g[off + BH];
        }
      }
    }
    const bool ok = gather_blocks<UNC, 1>(a.xw + (i64)(rg * 2 + (j & 1)) * gridDim.x * kBlockWords, (int)gridDim.x, (unsigned)j, As, ldk, H,
                                          status);
    if (!ok) ok_smem = 0;
    __syncthreads();
    if (ok_smem == 0) return;
  }
}

// adjoint:  the CTA owns UNC output units (columns of W_hh) over all K = 4H reduction indices.  Its slice of W_hh^T
// (UNC x 4H bf16, up to 128 KB) does not fit shared memory next to the 16 x 4H operand rows, so it lives in REGISTERS
// for the whole chain: warp w reduces k in [w*K/8, (w+1)*K/8) and a lane keeps exactly the B fragments of its
// m16n8k16 products there (KS k-steps x UNC/8 column tiles x 2 words; 128 registers at H = 1024, UNC = 16).
// The bf16 operand [ci*dc | cf*dc | cg*dc | co*Lh] of the NEXT step is formed by the CTA that produced (Lc, Lh).
template <int UNC, int KS>
__global__ void __launch_bounds__(kThreads, 1) lstm_adj_chain_kernel(LstmChainAdjArgs a, int* status) {
  constexpr int NT = UNC / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  constexpr int kBlockVals = 4 * kRows * UNC, kBlockWords = (kBlockVals + kValsPerWord - 1) / kValsPerWord;
  __shared__ __align__(16) bf16 xstage[4 * kRows * 16];
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, K = 4 * H, ldk = K + 8;
  bf16* As = reinterpret_cast<bf16*>(smem);                 // [16][ldk]
  float* red = reinterpret_cast<float*>(As + kRows * ldk);  // [8][16][UNC]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, lg = lane >> 2, lt = lane & 3;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const i64 BH = (i64)a.B * H, slot = 2 * BH;
  const int kbeg = warp * (K / kWarps);                     // K / 8 = 16 KS

  uint32_t wreg[KS][NT][2];
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const bf16* wp = a.WT + (i64)(u0 + nt * 8 + lg) * K + kbeg + 16 * ks + 2 * lt;
      wreg[ks][nt][0] = __ldg(reinterpret_cast<const uint32_t*>(wp));
      wreg[ks][nt][1] = __ldg(reinterpret_cast<const uint32_t*>(wp + 8));
    }
  for (int e = tid; e < kRows * ldk / 2; e += kThreads) reinterpret_cast<uint32_t*>(As)[e] = 0u;
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  // step 1: operand from the given sensitivities (slot 0) and the coefficients of step 1, all 4H columns of this row group
  for (int e = tid; e < nrows * H; e += kThreads) {
    int r = e / H, i = e % H;
    const i64 off = (i64)(row0 + r) * H + i;
    const float lh = __ldcg(a.mu + BH + off), dc = __ldcg(a.mu + off) + a.p[off] * lh;
    As[r * ldk + i] = __float2bfloat16(__bfloat162float(a.ci[off]) * dc);
    As[r * ldk + H + i] = __float2bfloat16(__bfloat162float(a.cf[off]) * dc);
    As[r * ldk + 2 * H + i] = __float2bfloat16(__bfloat162float(a.cg[off]) * dc);
    As[r * ldk + 3 * H + i] = __float2bfloat16(__bfloat162float(a.co[off]) * lh);
  }
  // per owned (row, unit): dc of the step in flight, its a and source terms; the coefficients of the step after it
  // (the bf16 gate coefficients stay raw in their registers until they are used: a conversion behind the load would wait
  // for it in front of the exchange)
  float dcur[OPT], pa[OPT], pgc[OPT], pgh[OPT], np_[OPT];
  bf16 nci[OPT], ncf[OPT], ncg[OPT], nco[OPT];
  const bf16 bzero = __float2bfloat16(0.f);
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    const i64 off = (i64)(row0 + r) * H + u0 + i;
    dcur[o] = v ? __ldcg(a.mu + off) + a.p[off] * __ldcg(a.mu + BH + off) : 0.f;
    pa[o] = v ? a.a[off] : 0.f;
    pgc[o] = (v && a.g) ? a.g[slot + off] : 0.f;
    pgh[o] = (v && a.g) ? a.g[slot + BH + off] : 0.f;
    const bool more = v && a.nsteps > 1;
    const i64 co = a.coef_step + off;
    np_[o] = more ? a.p[co] : 0.f; nci[o] = more ? a.ci[co] : bzero; ncf[o] = more ? a.cf[co] : bzero;
    ncg[o] = more ? a.cg[co] : bzero; nco[o] = more ? a.co[co] : bzero;
  }
  __syncthreads();

  for (int s = 1; s <= a.nsteps; ++s) {
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int k0 = kbeg + 16 * ks;
      uint32_t af[4];
      af[0] = *reinterpret_cast<const uint32_t*>(As + lg * ldk + k0 + 2 * lt);
      af[1] = *reinterpret_cast<const uint32_t*>(As + (lg + 8) * ldk + k0 + 2 * lt);
      af[2] = *reinterpret_cast<const uint32_t*>(As + lg * ldk + k0 + 2 * lt + 8);
      af[3] = *reinterpret_cast<const uint32_t*>(As + (lg + 8) * ldk + k0 + 2 * lt + 8);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) mma16816(acc[nt], af, wreg[ks][nt][0], wreg[ks][nt][1]);
    }
    store_partials<NT>(red, acc);
    __syncthreads();
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      const bool live = idx < kRows * UNC && r < nrows;
      float x4[4] = {0.f, 0.f, 0.f, 0.f};
      if (live) {
        const float lc = pa[o] * dcur[o] + pgc[o];
        const float lh = sum_partials<UNC>(red, r, i) + pgh[o];
        const i64 off = (i64)(row0 + r) * H + u0 + i;
        a.mu[(i64)s * slot + off] = lc;
        a.mu[(i64)s * slot + BH + off] = lh;
        const float dn = lc + np_[o] * lh;      // the next step's dc (its coefficients are zero behind the last step)
        dcur[o] = dn;
        x4[0] = __bfloat162float(nci[o]) * dn; x4[1] = __bfloat162float(ncf[o]) * dn; x4[2] = __bfloat162float(ncg[o]) * dn;
        x4[3] = __bfloat162float(nco[o]) * lh;
      }
      if (idx < kRows * UNC) {                  // block order [gate][row][unit]; rows beyond the batch travel as zeros
#pragma unroll
        for (int g = 0; g < 4; ++g) xstage[g * kRows * UNC + idx] = __float2bfloat16(x4[g]);
      }
    }
    if (s == a.nsteps) break;
    __syncthreads();
    publish_block(xstage, kBlockVals, a.xw + ((i64)(rg * 2 + (s & 1)) * gridDim.x + blockIdx.x) * kBlockWords, (unsigned)s);
#pragma unroll
    for (int o = 0; o < OPT; ++o) {             // operands of the steps to come that do not depend on other CTAs
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        const i64 off = (i64)(row0 + r) * H + u0 + i;
        pa[o] = a.a[(i64)s * a.coef_step + off];
        if (a.g) { pgc[o] = a.g[(i64)(s + 1) * slot + off]; pgh[o] = a.g[(i64)(s + 1) * slot + BH + off]; }
        if (s + 1 < a.nsteps) {
          const i64 co = (i64)(s + 1) * a.coef_step + off;
          np_[o] = a.p[co]; nci[o] = a.ci[co]; ncf[o] = a.cf[co]; ncg[o] = a.cg[co]; nco[o] = a.co[co];
        } else {
          np_[o] = 0.f; nci[o] = ncf[o] = ncg[o] = nco[o] = bzero;
        }
      }
    }
    const bool ok = gather_blocks<UNC, 4>(a.xw + (i64)(rg * 2 + (s & 1)) * gridDim.x * kBlockWords, (int)gridDim.x, (unsigned)s, As, ldk, H,
                                          status);
    if (!ok) ok_smem = 0;
    __syncthreads();
    if (ok_smem == 0) return;
  }
}

// ================================================================================================
// fp32 chains: the same two recurrences in FFMA arithmetic with precise gate math.  K is split over the 8 warps; a
// lane owns 4 rows x CPL columns of the 16 x (8 CPL) outputs (the 8 lanes of a quarter warp read the same A words --
// a broadcast -- and W rows 3 CPL (H + 4) floats apart: conflict-free 16-byte loads).
template <int CPL>
__device__ __forceinline__ void warp_gemm32(const float* As, const float* Ws, int ldk, int kbeg, int kend, float (*acc)[CPL]) {
  const int lane = threadIdx.x & 31, rq = lane >> 3, cq = lane & 7;
  const float* ar = As + (rq * 4) * ldk;
  const float* wr = Ws + (cq * CPL) * ldk;
  for (int k = kbeg; k < kend; k += 4) {
    float4 av[4], wv[CPL];
#pragma unroll
    for (int r = 0; r < 4; ++r) av[r] = *reinterpret_cast<const float4*>(ar + r * ldk + k);
#pragma unroll
    for (int c = 0; c < CPL; ++c) wv[c] = *reinterpret_cast<const float4*>(wr + c * ldk + k);
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < CPL; ++c)
        acc[r][c] = fmaf(av[r].x, wv[c].x, fmaf(av[r].y, wv[c].y, fmaf(av[r].z, wv[c].z, fmaf(av[r].w, wv[c].w, acc[r][c]))));
  }
}
// warp partial sums -> red[warp][row][col]   (col < 8 CPL)
template <int CPL>
__device__ __forceinline__ void store_partials32(float* red, float (*acc)[CPL]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, rq = lane >> 3, cq = lane & 7;
  constexpr int NC = 8 * CPL;
  float* base = red + warp * kRows * NC;
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < CPL; ++c) base[(rq * 4 + r) * NC + cq * CPL + c] = acc[r][c];
}

// forward:  u_j = Phi_gamma(gi_j, u_{j-1}) + g_j ;  the CTA owns UNC hidden units (3 UNC weight rows)
template <int UNC>
__global__ void __launch_bounds__(kThreads, 1) serial32_fwd_kernel(Serial32FwdArgs a, int* status) {
  constexpr int NW = 3 * UNC, CPL = NW / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, ldk = H + 4;
  float* Ws = reinterpret_cast<float*>(smem);   // [NW][ldk]
  float* As = Ws + NW * ldk;                    // [16][ldk]
  float* red = As + kRows * ldk;                // [8][16][NW]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const unsigned ncta_rg = gridDim.x;
  const i64 BH = (i64)a.B * H;

  for (int e = tid; e < NW * (H / 4); e += kThreads) {
    int r = e / (H / 4), c = e % (H / 4);
    int gate = r / UNC, i = r % UNC;
    *reinterpret_cast<float4*>(Ws + r * ldk + c * 4) = __ldg(reinterpret_cast<const float4*>(a.W + ((i64)gate * H + u0 + i) * H + c * 4));
  }
  for (int e = tid; e < kRows * ldk; e += kThreads) As[e] = 0.f;     // rows beyond the batch stay zero
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  for (int e = tid; e < nrows * (H / 4); e += kThreads) {
    int r = e / (H / 4), c = e % (H / 4);
    *reinterpret_cast<float4*>(As + r * ldk + c * 4) = __ldcg(reinterpret_cast<const float4*>(a.u + (i64)(row0 + r) * H + c * 4));
  }
  float hp[OPT], pgr[OPT], pgz[OPT], pgn[OPT], pg[OPT], br[OPT], bz[OPT], bn[OPT];
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    hp[o] = v ? __ldcg(a.u + (i64)(row0 + r) * H + u0 + i) : 0.f;
    br[o] = a.b_hh[u0 + i]; bz[o] = a.b_hh[H + u0 + i]; bn[o] = a.b_hh[2 * H + u0 + i];
    const float* gi = a.gi + (i64)(row0 + r) * 3 * H + u0 + i;
    pgr[o] = v ? gi[0] : 0.f; pgz[o] = v ? gi[H] : 0.f; pgn[o] = v ? gi[2 * H] : 0.f;
    pg[o] = (v && a.g) ? a.g[BH + (i64)(row0 + r) * H + u0 + i] : 0.f;
  }
  __syncthreads();

  const int kw = H / kWarps;
  for (int j = 1; j <= a.nsteps; ++j) {
    float acc[4][CPL];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < CPL; ++c) acc[r][c] = 0.f;
    warp_gemm32<CPL>(As, Ws, ldk, warp * kw, (warp + 1) * kw, acc);
    store_partials32<CPL>(red, acc);
    __syncthreads();
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        float ghr = sum_partials<NW>(red, r, i) + br[o];
        float ghz = sum_partials<NW>(red, r, UNC + i) + bz[o];
        float ghn = sum_partials<NW>(red, r, 2 * UNC + i) + bn[o];
        float val = cell_forward<false>(pgr[o], pgz[o], pgn[o], ghr, ghz, ghn, hp[o], a.gamma, a.cell) + pg[o];
        hp[o] = val;
        a.u[(i64)j * BH + (i64)(row0 + r) * H + u0 + i] = val;
      }
    }
    if (j == a.nsteps) break;
#pragma unroll
    for (int o = 0; o < OPT; ++o) {   // operands of the next step that do not depend on other CTAs
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        const float* gi = a.gi + (i64)j * a.gi_step + (i64)(row0 + r) * 3 * H + u0 + i;
        pgr[o] = gi[0]; pgz[o] = gi[H]; pgn[o] = gi[2 * H];
        if (a.g) pg[o] = a.g[(i64)(j + 1) * BH + (i64)(row0 + r) * H + u0 + i];
      }
    }
    if (!grid_barrier(a.bar + rg, (unsigned)j * ncta_rg, status, &ok_smem)) return;
    const float* uj = a.u + (i64)j * BH;     // the full new state of this row group
    for (int e = tid; e < nrows * (H / 4); e += kThreads) {
      int r = e / (H / 4), c = e % (H / 4);
      cp_async16(As + r * ldk + c * 4, uj + (i64)(row0 + r) * H + c * 4);
    }
    cp_async_wait_all();
    __syncthreads();
  }
}

// adjoint:  mu_s = a_s mu_{s-1} + ([cr|cz|cn]_s mu_{s-1}) W_hh + g_s ;  the CTA owns UNC output units (columns of W_hh)
template <int UNC>
__global__ void __launch_bounds__(kThreads, 1) serial32_adj_kernel(Serial32AdjArgs a, int* status) {
  constexpr int CPL = UNC / 8, OPT = (kRows * UNC + kThreads - 1) / kThreads;
  extern __shared__ __align__(16) uint8_t smem[];
  const int H = a.H, K = 3 * H, ldk = K + 4;
  float* Ws = reinterpret_cast<float*>(smem);   // [UNC][ldk]: Ws[n][k] = W_hh[k][u0 + n]
  float* As = Ws + UNC * ldk;                   // [16][ldk]
  float* red = As + kRows * ldk;                // [8][16][UNC]
  __shared__ int ok_smem;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int u0 = blockIdx.x * UNC, rg = blockIdx.y, row0 = rg * kRows;
  const int nrows = min(kRows, a.B - row0);
  const unsigned ncta_rg = gridDim.x;
  const i64 BH = (i64)a.B * H;

  for (int e = tid; e < K * UNC; e += kThreads) {
    int k = e / UNC, n = e % UNC;
    Ws[n * ldk + k] = __ldg(a.W + (i64)k * H + u0 + n);
  }
  for (int e = tid; e < kRows * ldk; e += kThreads) As[e] = 0.f;
  if (tid == 0) ok_smem = 1;
  __syncthreads();
  for (int e = tid; e < nrows * H; e += kThreads) {     // step 1: dA_1 = c_1 * mu_0
    int r = e / H, i = e % H;
    i64 off = (i64)(row0 + r) * H + i;
    float m = __ldcg(a.mu + off);
    As[r * ldk + i] = a.cr[off] * m;
    As[r * ldk + H + i] = a.cz[off] * m;
    As[r * ldk + 2 * H + i] = a.cn[off] * m;
  }
  float mp[OPT], pa[OPT], pg[OPT], ncr[OPT], ncz[OPT], ncn[OPT];
#pragma unroll
  for (int o = 0; o < OPT; ++o) {
    int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
    bool v = idx < kRows * UNC && r < nrows;
    i64 off = (i64)(row0 + r) * H + u0 + i;
    mp[o] = v ? __ldcg(a.mu + off) : 0.f;
    pa[o] = v ? a.a[off] : 0.f;
    pg[o] = (v && a.g) ? a.g[BH + off] : 0.f;
    bool more = v && a.nsteps > 1;
    ncr[o] = more ? a.cr[a.coef_step + off] : 0.f;
    ncz[o] = more ? a.cz[a.coef_step + off] : 0.f;
    ncn[o] = more ? a.cn[a.coef_step + off] : 0.f;
  }
  __syncthreads();

  const int kw = K / kWarps;
  for (int s = 1; s <= a.nsteps; ++s) {
    float acc[4][CPL];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < CPL; ++c) acc[r][c] = 0.f;
    warp_gemm32<CPL>(As, Ws, ldk, warp * kw, (warp + 1) * kw, acc);
    store_partials32<CPL>(red, acc);
    __syncthreads();
    float* dA = a.dA + (i64)(s & 1) * 3 * BH;
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        float val = pa[o] * mp[o] + sum_partials<UNC>(red, r, i) + pg[o];
        mp[o] = val;
        i64 off = (i64)(row0 + r) * H + u0 + i;
        a.mu[(i64)s * BH + off] = val;
        if (s < a.nsteps) {
          float* d = dA + (i64)(row0 + r) * K + u0 + i;
          d[0] = ncr[o] * val; d[H] = ncz[o] * val; d[2 * H] = ncn[o] * val;
        }
      }
    }
    if (s == a.nsteps) break;
#pragma unroll
    for (int o = 0; o < OPT; ++o) {
      int idx = tid + o * kThreads, r = idx / UNC, i = idx % UNC;
      if (idx < kRows * UNC && r < nrows) {
        i64 off = (i64)(row0 + r) * H + u0 + i;
        pa[o] = a.a[(i64)s * a.coef_step + off];
        if (a.g) pg[o] = a.g[(i64)(s + 1) * BH + off];
        if (s + 1 < a.nsteps) {
          i64 co = (i64)(s + 1) * a.coef_step + off;
          ncr[o] = a.cr[co]; ncz[o] = a.cz[co]; ncn[o] = a.cn[co];
        }
      }
    }
    if (!grid_barrier(a.bar + rg, (unsigned)s * ncta_rg, status, &ok_smem)) return;
    for (int e = tid; e < nrows * (K / 4); e += kThreads) {
      int r = e / (K / 4), c = e % (K / 4);
      cp_async16(As + r * ldk + c * 4, dA + (i64)(row0 + r) * K + c * 4);
    }
    cp_async_wait_all();
    __syncthreads();
  }
}

int* status_ptr() {     // status word of the current device, nullptr on failure
  const int dev = current_device_slot();
  if (dev < 0) return nullptr;
  if (!g_serial_status_ptrs[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_serial_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    g_serial_status_ptrs[dev] = p;
  }
  return g_serial_status_ptrs[dev];
}

constexpr size_t kSmemLimit = 227 * 1024 - 4096;   // dynamic part: the kernels also hold up to 3 KiB of static shared memory
int g_sm_count[kMaxDevices] = {0};
int sm_count() {
  const int dev = current_device_slot();
  if (dev < 0) return 148;
  if (g_sm_count[dev] == 0) {
    if (cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_sm_count[dev] <= 0) {
      cudaGetLastError();
      g_sm_count[dev] = 148;
    }
  }
  return g_sm_count[dev];
}

size_t fwd_smem(int unc, int H) { return (size_t)(3 * unc + kRows) * (H + 8) * 2 + (size_t)kWarps * kRows * 3 * unc * 4; }
size_t adj_smem(int unc, int H) { return (size_t)(unc + kRows) * (3 * H + 8) * 2 + (size_t)kWarps * kRows * unc * 4; }

// smallest units-per-CTA whose grid is co-resident (one CTA per SM) and whose slice fits shared memory
int pick_unc(int B, int H, bool adj) {
  if (H % 128 != 0) return 0;
  int rgs = (B + kRows - 1) / kRows;
  const int cands[3] = {8, 16, 32};
  for (int c : cands) {
    if (H % c != 0) continue;
    if ((i64)(H / c) * rgs > sm_count()) continue;
    size_t sm = adj ? adj_smem(c, H) : fwd_smem(c, H);
    if (sm > kSmemLimit) continue;
    return c;
  }
  return 0;
}

// MGRIT_GRU_CHAIN_LL=0 in the environment selects the counter barrier + reload instead of the flag-in-data exchange.
bool chain_ll_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_CHAIN_LL"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

template <class Args, class Kern>
bool launch_coop(Kern kern, const Args& a, int unc, size_t smem, bool ll, int gates, cudaStream_t s) {
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
  int rgs = (a.B + kRows - 1) / kRows;
  if (cudaMemsetAsync(a.bar, 0, sizeof(unsigned) * rgs, s) != cudaSuccess) return false;
  if (ll) {   // no word may carry a step number of an earlier launch
    const size_t words = (size_t)rgs * 2 * (a.H / unc) * ((size_t)(gates * kRows * unc + kValsPerWord - 1) / kValsPerWord);
    if (words * sizeof(uint4) > a.xw_bytes) return false;
    if (cudaMemsetAsync(a.xw, 0, words * sizeof(uint4), s) != cudaSuccess) return false;
  }
  Args args = a;
  int* st = status_ptr();
  if (!st) return false;
  void* params[2] = {(void*)&args, (void*)&st};
  dim3 grid(a.H / unc, rgs);
  if (cudaLaunchCooperativeKernel((const void*)kern, grid, dim3(kThreads), params, smem, s) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  count_launch();
  return true;
}

// ---- fp32 chains
size_t fwd32_smem(int unc, int H) { return ((size_t)(3 * unc + kRows) * (H + 4) + (size_t)kWarps * kRows * 3 * unc) * 4; }
size_t adj32_smem(int unc, int H) { return ((size_t)(unc + kRows) * (3 * H + 4) + (size_t)kWarps * kRows * unc) * 4; }
int pick_unc32(int B, int H, bool adj) {
  if (H % 32 != 0) return 0;                   // K split over 8 warps in steps of four
  const int rgs = (B + kRows - 1) / kRows;
  const int cands[2] = {8, 16};
  for (int c : cands) {
    if (H % c != 0) continue;
    if ((i64)(H / c) * rgs > sm_count()) continue;
    if ((adj ? adj32_smem(c, H) : fwd32_smem(c, H)) > kSmemLimit) continue;
    return c;
  }
  return 0;
}
template <class Args, class Kern>
bool launch_coop32(Kern kern, const Args& a, int unc, size_t smem, cudaStream_t s) {
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
  const int rgs = (a.B + kRows - 1) / kRows;
  if (cudaMemsetAsync(a.bar, 0, sizeof(unsigned) * rgs, s) != cudaSuccess) return false;
  Args args = a;
  int* st = status_ptr();
  if (!st) return false;
  void* params[2] = {(void*)&args, (void*)&st};
  if (cudaLaunchCooperativeKernel((const void*)kern, dim3(a.H / unc, rgs), dim3(kThreads), params, smem, s) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  count_launch();
  return true;
}

}  // namespace

size_t serial_xw_bytes(int B, int H, int gates) {
  // the smallest unit slice (8) has the most words: 2 parities x row groups x (H / 8) producers x ceil(gates*16*8 / 6)
  const size_t rgs = (size_t)(B + kRows - 1) / kRows;
  return rgs * 2 * (size_t)(H / 8) * (size_t)((gates * kRows * 8 + kValsPerWord - 1) / kValsPerWord) * sizeof(uint4) + 256;
}

bool serial_fwd_supported(int B, int H) { return pick_unc(B, H, false) != 0; }
bool serial_adj_supported(int B, int H) { return pick_unc(B, H, true) != 0; }

// MGRIT_GRU_CHAIN_WREG=0 in the environment keeps the chains' weight fragments in shared memory (same results).
static bool chain_wreg_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_CHAIN_WREG"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

bool serial_fwd_solve(const SerialFwdArgs& a, cudaStream_t s) {
  int unc = pick_unc(a.B, a.H, false);
  if (unc == 0 || a.nsteps <= 0 || !status_ptr()) return false;
  size_t smem = fwd_smem(unc, a.H);
  prof_begin(KC_FWD_SERIAL, 2.0 * a.B * 3.0 * a.H * a.H * a.nsteps, s);
  const bool ll = chain_ll_enabled() && a.xw != nullptr;
  if (ll && chain_wreg_enabled() && (unc == 8 || unc == 16) && (a.H == 512 || a.H == 1024)) {
    bool okr;
    if (a.H == 1024) okr = unc == 8 ? launch_coop(serial_fwd_kernel<8, true, 8>, a, unc, smem, true, 1, s)
                                    : launch_coop(serial_fwd_kernel<16, true, 8>, a, unc, smem, true, 1, s);
    else okr = unc == 8 ? launch_coop(serial_fwd_kernel<8, true, 4>, a, unc, smem, true, 1, s)
                        : launch_coop(serial_fwd_kernel<16, true, 4>, a, unc, smem, true, 1, s);
    prof_end(s);
    return okr;
  }
  bool ok = ll ? (unc == 8 ? launch_coop(serial_fwd_kernel<8, true>, a, unc, smem, true, 1, s)
                  : unc == 16 ? launch_coop(serial_fwd_kernel<16, true>, a, unc, smem, true, 1, s)
                              : launch_coop(serial_fwd_kernel<32, true>, a, unc, smem, true, 1, s))
               : (unc == 8 ? launch_coop(serial_fwd_kernel<8, false>, a, unc, smem, false, 1, s)
                  : unc == 16 ? launch_coop(serial_fwd_kernel<16, false>, a, unc, smem, false, 1, s)
                              : launch_coop(serial_fwd_kernel<32, false>, a, unc, smem, false, 1, s));
  prof_end(s);
  return ok;
}

bool serial_adj_solve(const SerialAdjArgs& a, cudaStream_t s) {
  int unc = pick_unc(a.B, a.H, true);
  if (unc == 0 || a.nsteps <= 0 || !status_ptr()) return false;
  size_t smem = adj_smem(unc, a.H);
  prof_begin(KC_ADJ_SERIAL, 2.0 * a.B * 3.0 * a.H * a.H * a.nsteps, s);
  const bool ll = chain_ll_enabled() && a.xw != nullptr;
  if (ll && chain_wreg_enabled() && (unc == 8 || unc == 16) && (a.H == 512 || a.H == 1024)) {
    bool okr;
    if (a.H == 1024) okr = unc == 8 ? launch_coop(serial_adj_kernel<8, true, 24>, a, unc, smem, true, 3, s)
                                    : launch_coop(serial_adj_kernel<16, true, 24>, a, unc, smem, true, 3, s);
    else okr = unc == 8 ? launch_coop(serial_adj_kernel<8, true, 12>, a, unc, smem, true, 3, s)
                        : launch_coop(serial_adj_kernel<16, true, 12>, a, unc, smem, true, 3, s);
    prof_end(s);
    return okr;
  }
  bool ok = ll ? (unc == 8 ? launch_coop(serial_adj_kernel<8, true>, a, unc, smem, true, 3, s)
                  : unc == 16 ? launch_coop(serial_adj_kernel<16, true>, a, unc, smem, true, 3, s)
                              : launch_coop(serial_adj_kernel<32, true>, a, unc, smem, true, 3, s))
               : (unc == 8 ? launch_coop(serial_adj_kernel<8, false>, a, unc, smem, false, 3, s)
                  : unc == 16 ? launch_coop(serial_adj_kernel<16, false>, a, unc, smem, false, 3, s)
                              : launch_coop(serial_adj_kernel<32, false>, a, unc, smem, false, 3, s));
  prof_end(s);
  return ok;
}

// ---- Implicit LSTM chains
namespace {
size_t lstm_fwd_smem(int unc, int H) { return (size_t)(4 * unc + kRows) * (H + 8) * 2 + (size_t)kWarps * kRows * 4 * unc * 4; }
size_t lstm_adj_smem(int unc, int H) { return (size_t)kRows * (4 * H + 8) * 2 + (size_t)kWarps * kRows * unc * 4; }
int lstm_pick_unc(int B, int H, bool adj) {
  if (adj ? !(H == 128 || H == 256 || H == 512 || H == 1024) : H % 128 != 0) return 0;
  const int rgs = (B + kRows - 1) / kRows;
  const int cands[3] = {8, 16, 32};
  for (int c : cands) {
    if (H % c != 0 || (adj && c > 16)) continue;
    if ((i64)(H / c) * rgs > sm_count()) continue;
    if ((adj ? lstm_adj_smem(c, H) : lstm_fwd_smem(c, H)) > kSmemLimit) continue;
    return c;
  }
  return 0;
}
template <class Args, class Kern>
bool launch_lstm_chain(Kern kern, const Args& a, int unc, size_t smem, int gates, cudaStream_t s) {
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
  const int rgs = (a.B + kRows - 1) / kRows;
  // no exchange word may carry a step number of an earlier launch
  const size_t words = (size_t)rgs * 2 * (a.H / unc) * ((size_t)(gates * kRows * unc + kValsPerWord - 1) / kValsPerWord);
  if (words * sizeof(uint4) > a.xw_bytes) return false;
  if (cudaMemsetAsync(a.xw, 0, words * sizeof(uint4), s) != cudaSuccess) return false;
  Args args = a;
  int* st = status_ptr();
  if (!st) return false;
  void* params[2] = {(void*)&args, (void*)&st};
  if (cudaLaunchCooperativeKernel((const void*)kern, dim3(a.H / unc, rgs), dim3(kThreads), params, smem, s) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  count_launch();
  return true;
}
template <int UNC>
bool launch_lstm_adj(const LstmChainAdjArgs& a, size_t smem, cudaStream_t s) {
  switch (a.H) {
    case 128: return launch_lstm_chain(lstm_adj_chain_kernel<UNC, 4>, a, UNC, smem, 4, s);
    case 256: return launch_lstm_chain(lstm_adj_chain_kernel<UNC, 8>, a, UNC, smem, 4, s);
    case 512: return launch_lstm_chain(lstm_adj_chain_kernel<UNC, 16>, a, UNC, smem, 4, s);
    case 1024: return launch_lstm_chain(lstm_adj_chain_kernel<UNC, 32>, a, UNC, smem, 4, s);
    default: return false;
  }
}
}  // namespace

bool lstm_chain_fwd_solve(const LstmChainFwdArgs& a, cudaStream_t s) {
  const int unc = chain_ll_enabled() ? lstm_pick_unc(a.B, a.H, false) : 0;
  if (unc == 0 || a.nsteps <= 0 || !a.xw || !status_ptr()) return false;
  const size_t smem = lstm_fwd_smem(unc, a.H);
  prof_begin(KC_FWD_SERIAL, 2.0 * a.B * 4.0 * a.H * a.H * a.nsteps, s);
  const bool ok = unc == 8    ? launch_lstm_chain(lstm_fwd_chain_kernel<8>, a, unc, smem, 1, s)
                  : unc == 16 ? launch_lstm_chain(lstm_fwd_chain_kernel<16>, a, unc, smem, 1, s)
                              : launch_lstm_chain(lstm_fwd_chain_kernel<32>, a, unc, smem, 1, s);
  prof_end(s);
  return ok;
}

bool lstm_chain_adj_solve(const LstmChainAdjArgs& a, cudaStream_t s) {
  const int unc = chain_ll_enabled() ? lstm_pick_unc(a.B, a.H, true) : 0;
  if (unc == 0 || a.nsteps <= 0 || !a.xw || !status_ptr()) return false;
  const size_t smem = lstm_adj_smem(unc, a.H);
  prof_begin(KC_ADJ_SERIAL, 2.0 * a.B * 4.0 * a.H * a.H * a.nsteps, s);
  const bool ok = unc == 8 ? launch_lstm_adj<8>(a, smem, s) : launch_lstm_adj<16>(a, smem, s);
  prof_end(s);
  return ok;
}

// MGRIT_GRU_CHAIN32=0 in the environment advances the fp32 / tf32 modes' coarsest level step by step instead.
static bool chain32_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_CHAIN32"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

bool serial32_fwd_solve(const Serial32FwdArgs& a, cudaStream_t s) {
  const int unc = chain32_enabled() ? pick_unc32(a.B, a.H, false) : 0;
  if (unc == 0 || a.nsteps <= 0 || !a.bar || !status_ptr()) return false;
  const size_t smem = fwd32_smem(unc, a.H);
  prof_begin(KC_FWD_SERIAL, 2.0 * a.B * 3.0 * a.H * a.H * a.nsteps, s);
  const bool ok = unc == 8 ? launch_coop32(serial32_fwd_kernel<8>, a, unc, smem, s) : launch_coop32(serial32_fwd_kernel<16>, a, unc, smem, s);
  prof_end(s);
  return ok;
}

bool serial32_adj_solve(const Serial32AdjArgs& a, cudaStream_t s) {
  const int unc = chain32_enabled() ? pick_unc32(a.B, a.H, true) : 0;
  if (unc == 0 || a.nsteps <= 0 || !a.bar || !a.dA || !status_ptr()) return false;
  const size_t smem = adj32_smem(unc, a.H);
  prof_begin(KC_ADJ_SERIAL, 2.0 * a.B * 3.0 * a.H * a.H * a.nsteps, s);
  const bool ok = unc == 8 ? launch_coop32(serial32_adj_kernel<8>, a, unc, smem, s) : launch_coop32(serial32_adj_kernel<16>, a, unc, smem, s);
  prof_end(s);
  return ok;
}

int serial_device_status() {
  const int dev = current_device_slot();
  if (dev < 0) return -1;
  if (!g_serial_status_ptrs[dev]) return 0;     // no chain kernel has run on this device
  int v = 0;
  if (cudaMemcpy(&v, g_serial_status_ptrs[dev], sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return v;
}

int serial_clear_device_status() {
  const int dev = current_device_slot();
  if (dev < 0) return -1;
  if (!g_serial_status_ptrs[dev]) return 0;
  return cudaMemset(g_serial_status_ptrs[dev], 0, sizeof(int)) == cudaSuccess ? 0 : -1;
}

}  // namespace mg
