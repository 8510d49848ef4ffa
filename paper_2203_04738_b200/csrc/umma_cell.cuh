// Fused "recurrent GEMM + GRU cell" kernel for sm_100a: every operand of the epilogue is staged through
// shared memory by TMA, so that the only latency-exposed global accesses of the epilogue are its stores.
//
//   rows m = (k, b)      k = interval / coarse point, b = batch row, 128 rows per CTA tile = kt k's x B
//   D[m, gate, u] = sum_j hb[m, j] * W_hh[gate*H + u, j]          (tcgen05, bf16 x bf16 -> fp32 in TMEM)
//   forward : out[m, u] = Phi_gamma(gi[m, :, u], D + b_hh, h[m, u]) (+ g[m, u])   or   g - Phi   (mode 1)
//   linearise: a, c_r, c_z, c_n, c_n'[m, u] = transposed-Jacobian coefficients of that step
//
// Two geometries of the same kernel:
//   PAIR = false  one CTA per 128 x (3 x 64) tile, tcgen05.mma.cta_group::1 with N = 192.
//   PAIR = true   clusters of two CTAs (the two SMs of a TPC) share one 256 x (3 x 80) tile:
//                 tcgen05.mma.cta_group::2 with N = 240.  Each CTA stages its own 128 rows of A and HALF of the
//                 weight tile (120 of the 240 gate rows: 31 KiB per k-block instead of 40), so the operand bytes an
//                 SM takes in per flop drop by 40 %.  The width is 80 units because the duration of a pair MMA does
//                 not depend on N (measured on a bare main loop: 256 x N x 16 takes the same 164 cycles for every
//                 N from 128 to 256), so a tile should be as close to 256 columns as three equal gates allow; 240
//                 columns twice fit the 512 columns of tensor memory.  The last unit tile of a row is ragged
//                 (H = 1024: twelve tiles of 80 units and one of 64); its surplus columns are computed on
//                 whatever weight rows follow and never stored.
//   Pair protocol: both CTAs' operand loads complete on the LEADER's (rank 0) full barrier, which expects the
//   bytes of both; the leader's MMA thread issues for the pair and commits each stage to both CTAs' empty barriers
//   and each accumulator to both CTAs' tfull barriers (one commit per destination, no multicast load anywhere);
//   one elected lane per epilogue warp of both CTAs releases the leader's accumulator barrier (remote arrive
//   for rank 1); tensor memory is allocated and freed by the same warp of both CTAs behind cluster barriers.
//
// Warp roles (352 threads): 0 = TMA producer of the A/B ring, 1 = MMA issuer and TMEM owner,
// 2 = TMA producer of the epilogue operands (gi r|z|n, h, g in chunks of 16 hidden units, two
// buffers), 3..10 = epilogue (two warps per TMEM lane quarter, 8 hidden units per thread and chunk).
// The A operand (bf16 copy of the state) and the epilogue operands are addressed through 3-D tensor
// maps {column, batch row, k} whose k-stride is the slot stride of the relaxation, so no gather
// kernel is needed; the epilogue also writes the bf16 copy of the new state for the next step.
// Epilogue tiles use the 64-byte swizzle: rows of 16 floats, 16-byte chunk index XOR ((row >> 1) & 3).
// Every wait on an mbarrier is bounded (2 s): a wait that runs out records a code in the status word and the
// CTA stops issuing work, so both CTAs of a pair reach the closing cluster barrier.
#pragma once
#include "cell.cuh"
#include "umma_gemm_pair.cuh"

namespace mg {
namespace umma {

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// ... whose completion barrier may live in the other CTA of the pair (bar is a shared::cluster address)
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// 4-D maps {column, batch row, slot inside the interval, interval}: the forward kernel addresses the level state, the
// input projection and the additive term by (slot, first interval of the tile), so that ONE launch can run several
// dependent relaxation steps (a sweep) that differ only in the slot coordinate.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// tcgen05.ld is asynchronous: its destination registers are only valid after tcgen05.wait::ld.  The
// results are therefore produced directly in their final registers (no copies that the compiler could
// schedule before the wait), and tmem_ld_wait8 makes every later use depend on the wait.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait8x3(float* a, float* b, float* c) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7]),
                 "+f"(b[0]), "+f"(b[1]), "+f"(b[2]), "+f"(b[3]), "+f"(b[4]), "+f"(b[5]), "+f"(b[6]), "+f"(b[7]),
                 "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]), "+f"(c[4]), "+f"(c[5]), "+f"(c[6]), "+f"(c[7])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait8(float* a) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait8x4(float* a, float* b, float* c, float* d) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]), "+f"(a[4]), "+f"(a[5]), "+f"(a[6]), "+f"(a[7]),
                 "+f"(b[0]), "+f"(b[1]), "+f"(b[2]), "+f"(b[3]), "+f"(b[4]), "+f"(b[5]), "+f"(b[6]), "+f"(b[7]),
                 "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]), "+f"(c[4]), "+f"(c[5]), "+f"(c[6]), "+f"(c[7]),
                 "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]), "+f"(d[4]), "+f"(d[5]), "+f"(d[6]), "+f"(d[7])
               :
               : "memory");
}
// One 32-byte store per thread: a warp's lanes write 32 different rows, and two 16-byte stores per row would
// reach L2 as two half-filled sector writes each.
__device__ __forceinline__ void stg8(float* p, const float* v) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]),
               "f"(v[5]), "f"(v[6]), "f"(v[7])
               : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}
// eight values as bf16 into shared memory: one 16-byte store
__device__ __forceinline__ void sts_bf8(uint32_t addr, const float* v) {
  __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]), p3 = __floats2bfloat162_rn(v[6], v[7]);
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(*reinterpret_cast<uint32_t*>(&p0)),
               "r"(*reinterpret_cast<uint32_t*>(&p1)), "r"(*reinterpret_cast<uint32_t*>(&p2)), "r"(*reinterpret_cast<uint32_t*>(&p3))
               : "memory");
}
// eight bf16 values from shared memory (one 16-byte load) as floats
__device__ __forceinline__ void lds_bf8(uint32_t addr, float* v) {
  uint32_t w[4];
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ float4 lds4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}

struct CellArgs {
  int M, B, H, kt;                                    // kt = 128 / B
  float* hout; i64 hout_ks; __nv_bfloat16* hout_b;    // forward: fp32 rows (k, b) and their bf16 copy (or nullptr)
  float* a;                                           // linearise: row-major [M, H]; a in fp32,
  __nv_bfloat16 *cr, *cz, *cn, *cnp;                  // the gate coefficients in bf16 (cnp may be nullptr)
  const float* b_hh; float gamma; int cell; int mode;
};

// A sweep: up to kMaxSweepSteps dependent forward steps over the same rows (k, b) in one launch.  Work items are
// (step, tile) in step-major order, CTA c takes items c, c + #CTAs, ...; an item of step s > 0 first waits until the
// row tiles of step s - 1 that it reads (and whose earlier readers it must not overtake) are complete: the epilogue
// warps count finished items per (step, row tile) in global memory.  Every dependency points to an earlier item and
// all CTAs of the launch are resident (at most one per SM), so the earliest unfinished item can always proceed;
// the wait is bounded like every other wait here.
constexpr int kMaxSweepSteps = 20;
struct SweepStep {
  float* hout; i64 hout_ks; __nv_bfloat16* hout_b;   // destination rows (k, b): fp32 state and its bf16 copy (or nullptr)
  int in_s;     // slot coordinate of the state the step starts from (maps A and HP)
  int tgt_s;    // slot coordinate of the point it arrives at (maps GI and G)
  int dep;      // row tiles of the previous step that must be complete: 0 none, 1 {mt}, 2 {mt - 1, mt}, 3 {mt, mt + 1}
};
struct SweepArgs {
  int n_steps;
  int* ctr;     // [n_steps][row tiles] zeroed counters (nullptr for a single step)
  SweepStep st[kMaxSweepSteps];
};

// Bounded wait until *ctr >= target (acquire), then order the async proxy (TMA reads) behind what was acquired.
__device__ __forceinline__ bool sweep_wait(const int* ctr, int target, volatile int* abort_flag, int* status, int code) {
  uint64_t t0 = 0;
  uint32_t spins = 0;
  while (true) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) break;
    if ((++spins & 63u) == 0) {
      if (*abort_flag) return false;
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
  asm volatile("fence.proxy.async;" ::: "memory");
  return true;
}

namespace cellk {
constexpr int CH = 16;                  // hidden units per epilogue chunk
constexpr int kThreads = 352;
constexpr int kABytes = BM * BK * 2;
constexpr int kOpBytes = BM * CH * 4;   // one epilogue operand chunk: 128 rows x 16 floats
// The linearisation's four bf16 coefficient arrays leave through shared memory: per chunk four [128 x 16] bf16
// tiles (32-byte swizzle), two buffers, written to global memory by TMA stores.  (Four 16-byte st.global per thread
// and chunk, each touching 32 different rows, cost a third of that kernel's time.)  The forward step's two stores
// per thread and chunk (32 bytes of state, 16 bytes of its bf16 copy) stay direct: staged the same way they cost
// the same 20 us of a 118 us step and one stage of the operand ring; what a store costs here is the number of
// row pieces that reach L2, not the path they take (rows of 128 bytes instead of 64 halve it).
constexpr int kCoefBytes = BM * CH * 2;   // one coefficient chunk: 128 rows x 16 bf16
template <bool PAIR> struct Geo {
  static constexpr int UN = PAIR ? 80 : 64;         // hidden units per tile
  static constexpr int BN = 3 * UN;                 // accumulator columns: r | z | n
  static constexpr int NCH = UN / CH;
  static constexpr int kBox = PAIR ? 40 : 64;       // weight rows per TMA box
  static constexpr int kBBytes = (PAIR ? BN / 2 : BN) * BK * 2;   // weight bytes staged per CTA and k-block
  static constexpr int kStageBytes = kABytes + kBBytes;           // 31 KiB / 40 KiB (multiples of 1 KiB)
};
// GIB: the input projection is staged from its bf16 copy (rows of 32 bytes, 32-byte swizzle) instead of fp32: 10 instead of
// 16 bytes per element of epilogue operands, and a third operand buffer fits.  What hides the latency of those loads is
// the bytes in flight, and shared memory bounds them: a tile needs 128 x UN x (bytes per element) per main-loop time.
template <bool HAS_G, bool LIN = false, bool PAIR = false, bool GIB = false> struct CellCfg {
  using G = Geo<PAIR>;
#ifndef CELL_PAIR_STAGES_PLAIN
#define CELL_PAIR_STAGES_PLAIN 5
#endif
#ifndef CELL_PAIR_STAGES
#define CELL_PAIR_STAGES ((HAS_G || LIN) ? 4 : CELL_PAIR_STAGES_PLAIN)
#endif
#ifndef CELL_PAIR_EBUFS
#define CELL_PAIR_EBUFS 2
#endif
  static constexpr int kStages = PAIR ? CELL_PAIR_STAGES : ((HAS_G || LIN) ? 3 : 4);
#ifndef CELL_GIB_EBUFS
#define CELL_GIB_EBUFS 3
#endif
  static constexpr int kEpiBufs = GIB ? ((PAIR && !HAS_G && !LIN) ? CELL_GIB_EBUFS : (LIN ? 2 : 3)) : (PAIR ? CELL_PAIR_EBUFS : 2);     // epilogue-operand chunks in flight
  static constexpr int kGiBytes = GIB ? BM * CH * 2 : kOpBytes;   // one gate's chunk of the input projection
  static constexpr int kEpiBytes = 3 * kGiBytes + (HAS_G ? 2 : 1) * kOpBytes;   // gi r | z | n, previous state, additive term
  // per buffer: four bf16 coefficient tiles and (with GIB, where shared memory allows it) the fp32 tile of `a`
  static constexpr int kOutBytes = LIN ? 4 * kCoefBytes + (GIB ? kOpBytes : 0) : 0;
  static constexpr int kSmemBytes = kStages * G::kStageBytes + kEpiBufs * kEpiBytes + 2 * kOutBytes + 1024 + 256;
  static_assert(kSmemBytes + 1536 <= 232448, "shared memory budget (dynamic + static <= 227 KiB)");
};
}  // namespace cellk

template <bool LIN, bool HAS_G, bool PAIR, bool GIB = false>
__global__ void __launch_bounds__(cellk::kThreads, 1)
umma_cell_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmGI, const __grid_constant__ CUtensorMap tmHP,
                 const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmCR,
                 const __grid_constant__ CUtensorMap tmCZ, const __grid_constant__ CUtensorMap tmCN,
                 const __grid_constant__ CUtensorMap tmCP, CellArgs p, const __grid_constant__ SweepArgs swp, int* status) {
  using namespace cellk;
  using C = CellCfg<HAS_G, LIN, PAIR, GIB>;
  constexpr int kGi = C::kGiBytes;
  using G = Geo<PAIR>;
  constexpr int UN = G::UN, BN = G::BN, NCH = G::NCH, kStageBytes = G::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t epi_base = tiles_base + C::kStages * kStageBytes;
  const uint32_t out_base = epi_base + C::kEpiBufs * C::kEpiBytes;
  const uint32_t bars = out_base + 2 * C::kOutBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * C::kStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * C::kStages + 2 + a); };
  auto efull_bar = [&](int e) { return bars + 8u * (2 * C::kStages + 4 + e); };
  auto eempty_bar = [&](int e) { return bars + 8u * (2 * C::kStages + 4 + C::kEpiBufs + e); };
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;
  __shared__ uint32_t lds_sink[cellk::kThreads];   // see the operand-buffer release in the epilogue

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int H = p.H;
  // PAIR: a tile is 256 rows; CTA `rank` of the pair owns its rows [128 rank, 128 rank + 128).
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, ncta = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int kTileRows = PAIR ? 2 * BM : BM;
  const int m_tiles = (p.M + kTileRows - 1) / kTileRows, n_tiles = (H + UN - 1) / UN, tiles = m_tiles * n_tiles;
  const int k_blocks = (H + BK - 1) / BK;
  auto row_tile = [&](int t) { return PAIR ? 2 * (t / n_tiles) + (int)rank : t / n_tiles; };
  // forward: items (step, tile); the linearisation is a single step
  const int n_items = LIN ? tiles : tiles * swp.n_steps;
  constexpr int kCtrTarget = PAIR ? 16 : 8;       // epilogue warps that finish one item (both CTAs of a pair)
  // the row tiles of step sg - 1 that item (sg, row tile mtile) depends on are complete (true also when there are none)
  auto deps_ready = [&](int sg, int mtile, int code) {
    if (LIN || sg == 0 || swp.st[sg].dep == 0) return true;
    const int dep = swp.st[sg].dep;
    const int lo = dep == 2 ? mtile - 1 : mtile, hi = dep == 3 ? mtile + 1 : mtile;
    for (int m = lo; m <= hi; ++m) {
      if (m < 0 || m >= m_tiles) continue;
      if (!sweep_wait(swp.ctr + (sg - 1) * m_tiles + m, n_tiles * kCtrTarget, (volatile int*)&abort_flag, status, code)) return false;
    }
    return true;
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < C::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), PAIR ? 16 : 8);      // one elected lane per epilogue warp (of both CTAs)
    }
    for (int e = 0; e < C::kEpiBufs; ++e) { mbar_init(efull_bar(e), 1); mbar_init(eempty_bar(e), 256); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (PAIR) {   // the same warp of both CTAs allocates the same columns in both tensor memories
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;
  pdl_wait();     // everything above touched only shared memory and TMEM
  pdl_trigger();

  if (warp == 0) {
    // ------------------------------------------------------------ A/B producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      for (int w = cta; w < n_items && ok; w += ncta) {
        const int sg = LIN ? 0 : w / tiles, t = w - sg * tiles;
        const int mt = row_tile(t), nt = t % n_tiles;
        const int in_s = LIN ? 0 : swp.st[sg].in_s;
        if (!deps_ready(sg, t / n_tiles, 17)) { ok = false; break; }
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp, status, 11)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          if (PAIR) {
            // The accumulator columns r | z | n (80 each) split into two halves of 120: CTA 0 stages the weight rows
            // of r and of the first 40 units of z, CTA 1 the rest -- six 40-row boxes, three per CTA.
            const uint32_t fullL = mapa_shared(full_bar(stage), 0);
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
            if (LIN) tma_load_3d_pair(a_dst, &tmA, fullL, kb * BK, 0, mt * p.kt);
            else tma_load_4d_pair(a_dst, &tmA, fullL, kb * BK, 0, in_s, mt * p.kt);
#pragma unroll
            for (int j = 0; j < 3; ++j) {
              const int piece = 3 * (int)rank + j;
              tma_load_2d_pair(b_dst + j * (G::kBox * BK * 2), &tmB, fullL, kb * BK, (piece >> 1) * H + nt * UN + (piece & 1) * G::kBox);
            }
          } else {
            mbar_expect_tx(full_bar(stage), kStageBytes);
            if (LIN) tma_load_3d(a_dst, &tmA, full_bar(stage), kb * BK, 0, mt * p.kt);
            else tma_load_4d(a_dst, &tmA, full_bar(stage), kb * BK, 0, in_s, mt * p.kt);
#pragma unroll
            for (int g = 0; g < 3; ++g) tma_load_2d(b_dst + g * (G::kBBytes / 3), &tmB, full_bar(stage), kb * BK, g * H + nt * UN);
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (PAIR: the leader issues for both CTAs)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = PAIR ? instr_desc_bf16_pair(BN) : instr_desc_bf16(BN);
      int stage = 0; uint32_t phase = 0; int it = 0; bool ok = true;
      for (int w = cta; w < n_items && ok; w += ncta, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abortp, status, 12)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp, status, 13)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * kStageBytes;
          const uint64_t adesc = smem_desc_sw128(a_src), bdesc = smem_desc_sw128(a_src + kABytes);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if (PAIR) mma_bf16_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
            else mma_bf16(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          if (PAIR) {   // the stage is free again in both CTAs
            mma_commit_pair(mapa_shared(empty_bar(stage), 0));
            mma_commit_pair(mapa_shared(empty_bar(stage), 1));
          } else {
            mma_commit(empty_bar(stage));
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          if (PAIR) {
            mma_commit_pair(mapa_shared(tfull_bar(as), 0));
            mma_commit_pair(mapa_shared(tfull_bar(as), 1));
          } else {
            mma_commit(tfull_bar(as));
          }
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ epilogue-operand producer
    if (lane == 0) {
      int eb = 0; uint32_t ephase = 0; bool ok = true;
      for (int w = cta; w < n_items && ok; w += ncta) {
        const int sg = LIN ? 0 : w / tiles, t = w - sg * tiles;
        const int mt = row_tile(t), nt = t % n_tiles;
        const int in_s = LIN ? 0 : swp.st[sg].in_s, tgt_s = LIN ? 0 : swp.st[sg].tgt_s;
        if (!deps_ready(sg, t / n_tiles, 18)) { ok = false; break; }
        for (int c = 0; c < NCH; ++c) {
          const int u = nt * UN + c * CH, k0 = mt * p.kt;
          if (u >= H) break;                       // ragged last unit tile: these columns are never stored
          if (!mbar_wait(eempty_bar(eb), ephase ^ 1u, abortp, status, 14)) { ok = false; break; }
          const uint32_t dst = epi_base + eb * C::kEpiBytes;
          mbar_expect_tx(efull_bar(eb), C::kEpiBytes);
          if (LIN) {
            tma_load_3d(dst, &tmGI, efull_bar(eb), u, 0, k0);
            tma_load_3d(dst + kGi, &tmGI, efull_bar(eb), H + u, 0, k0);
            tma_load_3d(dst + 2 * kGi, &tmGI, efull_bar(eb), 2 * H + u, 0, k0);
            tma_load_3d(dst + 3 * kGi, &tmHP, efull_bar(eb), u, 0, k0);
          } else {
            tma_load_4d(dst, &tmGI, efull_bar(eb), u, 0, tgt_s, k0);
            tma_load_4d(dst + kGi, &tmGI, efull_bar(eb), H + u, 0, tgt_s, k0);
            tma_load_4d(dst + 2 * kGi, &tmGI, efull_bar(eb), 2 * H + u, 0, tgt_s, k0);
            tma_load_4d(dst + 3 * kGi, &tmHP, efull_bar(eb), u, 0, in_s, k0);
            if (HAS_G) tma_load_4d(dst + 3 * kGi + kOpBytes, &tmG, efull_bar(eb), u, 0, tgt_s, k0);
          }
          if (++eb == C::kEpiBufs) { eb = 0; ephase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 3..10)
    const int q = warp & 3;              // TMEM lane quarter of this warp
    const int half = (warp - 3) >> 2;    // which 8 of a chunk's 16 hidden units
    const int r = q * 32 + lane;         // row inside the CTA's 128 rows
    const uint32_t sw = (uint32_t)((r >> 1) & 3);
    const uint32_t off0 = (uint32_t)r * 64u + ((((uint32_t)half * 2u) ^ sw) << 4);
    const uint32_t off1 = (uint32_t)r * 64u + ((((uint32_t)half * 2u + 1u) ^ sw) << 4);
    // bf16 coefficient tiles, 32-byte swizzle: rows of 32 bytes, 16-byte piece index XOR ((row >> 2) & 1)
    const uint32_t offb = (uint32_t)r * 32u + ((((uint32_t)half) ^ ((uint32_t)(r >> 2) & 1u)) << 4);
    const bool storer = threadIdx.x == 96;   // the epilogue thread that issues the TMA stores
    int it = 0, eb = 0, ob = 0; uint32_t ephase = 0;
    // A thread whose wait ran out (ok = false) keeps walking the loops without touching data, so that the named
    // barrier of the linearisation's store hand-over still sees all 256 epilogue threads.
    bool ok = true;
    for (int w = cta; w < n_items; w += ncta, ++it) {
      const int sg = LIN ? 0 : w / tiles, t = w - sg * tiles;
      const int mt = row_tile(t), nt = t % n_tiles;
      const int as = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      const int row = mt * BM + r;
      const bool valid = row < p.M;
      const int k = valid ? row / p.B : 0, b = valid ? row % p.B : 0;
      if (ok && !mbar_wait(tfull_bar(as), aphase, abortp, status, 15)) ok = false;
      ok = __all_sync(0xffffffffu, ok);      // warp-uniform: the accumulator loads below are warp-collective
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
      for (int c = 0; c < NCH; ++c) {
        if (nt * UN + c * CH >= H) break;          // ragged last unit tile (uniform over the CTA)
        if (ok && !mbar_wait(efull_bar(eb), ephase, abortp, status, 16)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
        const uint32_t src = epi_base + eb * C::kEpiBytes;
        float gr[8], gz[8], gn[8], hp[8], gg[8];
        if (GIB) {       // eight bf16 values per gate: one 16-byte load each (32-byte rows, 32-byte swizzle)
          lds_bf8(src + offb, gr); lds_bf8(src + kGi + offb, gz); lds_bf8(src + 2 * kGi + offb, gn);
        } else {
          *reinterpret_cast<float4*>(gr) = lds4(src + off0);            *reinterpret_cast<float4*>(gr + 4) = lds4(src + off1);
          *reinterpret_cast<float4*>(gz) = lds4(src + kGi + off0);      *reinterpret_cast<float4*>(gz + 4) = lds4(src + kGi + off1);
          *reinterpret_cast<float4*>(gn) = lds4(src + 2 * kGi + off0);  *reinterpret_cast<float4*>(gn + 4) = lds4(src + 2 * kGi + off1);
        }
        *reinterpret_cast<float4*>(hp) = lds4(src + 3 * kGi + off0);  *reinterpret_cast<float4*>(hp + 4) = lds4(src + 3 * kGi + off1);
        if (HAS_G) {
          *reinterpret_cast<float4*>(gg) = lds4(src + 3 * kGi + kOpBytes + off0); *reinterpret_cast<float4*>(gg + 4) = lds4(src + 3 * kGi + kOpBytes + off1);
        }
        const int cu = c * CH + half * 8;       // first of this thread's 8 units inside the tile
        float ar[8], az[8], an[8];
        tmem_ld8(taddr + cu, ar);
        tmem_ld8(taddr + UN + cu, az);
        tmem_ld8(taddr + 2 * UN + cu, an);
        tmem_ld_wait8x3(ar, az, an);
        // Release the operand buffer as soon as its values are in registers.  An mbarrier.arrive issued right
        // after the ld.shared instructions is NOT ordered behind loads whose results are still in flight (the
        // refilling TMA then overwrote rows that had not been read yet).  So one word that depends on every
        // load's result is stored first: the store cannot issue before the loads have delivered, and the
        // arrive issues after the store.
        {
          uint32_t dep = __float_as_uint(gr[0]) ^ __float_as_uint(gr[4]) ^ __float_as_uint(gz[0]) ^ __float_as_uint(gz[4]) ^
                         __float_as_uint(gn[0]) ^ __float_as_uint(gn[4]) ^ __float_as_uint(hp[0]) ^ __float_as_uint(hp[4]);
          if (HAS_G) dep ^= __float_as_uint(gg[0]) ^ __float_as_uint(gg[4]);
          asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_u32(&lds_sink[threadIdx.x])), "r"(dep) : "memory");
        }
        mbar_arrive(eempty_bar(eb));
        if (++eb == C::kEpiBufs) { eb = 0; ephase ^= 1u; }
        if (valid) {
          const int u = nt * UN + cu;
          float br[8], bz[8], bn[8];
          *reinterpret_cast<float4*>(br) = __ldg(reinterpret_cast<const float4*>(p.b_hh + u));
          *reinterpret_cast<float4*>(br + 4) = __ldg(reinterpret_cast<const float4*>(p.b_hh + u + 4));
          *reinterpret_cast<float4*>(bz) = __ldg(reinterpret_cast<const float4*>(p.b_hh + H + u));
          *reinterpret_cast<float4*>(bz + 4) = __ldg(reinterpret_cast<const float4*>(p.b_hh + H + u + 4));
          *reinterpret_cast<float4*>(bn) = __ldg(reinterpret_cast<const float4*>(p.b_hh + 2 * H + u));
          *reinterpret_cast<float4*>(bn + 4) = __ldg(reinterpret_cast<const float4*>(p.b_hh + 2 * H + u + 4));
          if (!LIN) {
            float o[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              float phi = cell_forward<true>(gr[e], gz[e], gn[e], ar[e] + br[e], az[e] + bz[e], an[e] + bn[e], hp[e], p.gamma, p.cell);
              o[e] = HAS_G ? (p.mode == 1 ? gg[e] - phi : phi + gg[e]) : phi;
            }
            const i64 idx = (i64)k * swp.st[sg].hout_ks + (i64)b * H + u;
            stg8(swp.st[sg].hout + idx, o);
            if (swp.st[sg].hout_b) {
              __nv_bfloat162 p0 = __floats2bfloat162_rn(o[0], o[1]), p1 = __floats2bfloat162_rn(o[2], o[3]);
              __nv_bfloat162 p2 = __floats2bfloat162_rn(o[4], o[5]), p3 = __floats2bfloat162_rn(o[6], o[7]);
              uint4 pk;
              pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
              pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
              *reinterpret_cast<uint4*>(swp.st[sg].hout_b + idx) = pk;
            }
          } else {
            float oa[8], ocr[8], ocz[8], ocn[8], ocp[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              CellLin L = cell_linearise<true>(gr[e], gz[e], gn[e], ar[e] + br[e], az[e] + bz[e], an[e] + bn[e], hp[e], p.gamma, p.cell);
              oa[e] = L.a; ocr[e] = L.cr; ocz[e] = L.cz; ocn[e] = L.cn; ocp[e] = L.cnp;
            }
            const i64 idx = (i64)row * H + u;
            if (GIB) {      // `a` leaves through shared memory like the coefficients (64-byte rows, 64-byte swizzle)
              const uint32_t da = out_base + ob * C::kOutBytes + 4 * kCoefBytes;
              asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(da + off0), "f"(oa[0]), "f"(oa[1]), "f"(oa[2]), "f"(oa[3]) : "memory");
              asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(da + off1), "f"(oa[4]), "f"(oa[5]), "f"(oa[6]), "f"(oa[7]) : "memory");
            } else {
              stg8(p.a + idx, oa);
            }
            const uint32_t dst = out_base + ob * C::kOutBytes + offb;
            sts_bf8(dst, ocr);
            sts_bf8(dst + kCoefBytes, ocz);
            sts_bf8(dst + 2 * kCoefBytes, ocn);
            if (p.cnp) sts_bf8(dst + 3 * kCoefBytes, ocp);
          }
        }
        }  // ok
        if (LIN) {
          // Chunk c's coefficients sit in output buffer ob.  Make them visible to the async proxy; the storing
          // thread first waits until the stores issued one chunk ago have finished READING the other buffer (they
          // had a whole chunk of time), so that after the barrier everybody may overwrite it with chunk c + 1.
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          if (storer) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          asm volatile("bar.sync 1, 256;" ::: "memory");
          if (storer && ok && mt * BM < p.M) {
            const uint32_t srcb = out_base + ob * C::kOutBytes;
            const int u = nt * UN + c * CH, row0 = mt * BM;
            tma_store_2d(&tmCR, srcb, u, row0);
            tma_store_2d(&tmCZ, srcb + kCoefBytes, u, row0);
            tma_store_2d(&tmCN, srcb + 2 * kCoefBytes, u, row0);
            if (p.cnp) tma_store_2d(&tmCP, srcb + 3 * kCoefBytes, u, row0);
            if (GIB) tma_store_2d(&tmG, srcb + 4 * kCoefBytes, u, row0);      // (the linearisation has no additive term: this map is `a`)
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          ob ^= 1;
        }
      }
      if (ok) {
        // every lane's accumulator loads have completed (tcgen05.wait::ld above); one lane releases for the warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (PAIR) mbar_arrive_cluster(mapa_shared(tempty_bar(as), 0));
          else mbar_arrive(tempty_bar(as));
          // sweep: this warp's rows of the item are written (the warp barrier above ordered every lane's stores before
          // this lane; the fence makes them visible before the count)
          if (!LIN && swp.ctr) {
            __threadfence();
            asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(swp.ctr + sg * m_tiles + t / n_tiles) : "memory");
          }
        }
      }
    }
    if (LIN && storer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // coefficients are in global memory before exit
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still signal it
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace umma
}  // namespace mg
