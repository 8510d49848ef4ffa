// Persistent, warp-specialised bf16 GEMM for sm_100a: TMA (cp.async.bulk.tensor) loads into a
// multi-stage shared-memory ring, tcgen05.mma with fp32 accumulators in tensor memory (two
// accumulator buffers, so the epilogue of one tile overlaps the main loop of the next), and a
// functor epilogue that reads the accumulator with tcgen05.ld, one output row per thread.
//
//   D[m, n] = sum_k A[m, k] * B[n, k]      A: [M, K] bf16 row-major, B: [N, K] bf16 row-major
//
// Tile 128 x BN x 64.  With NG = 3 (GRU) or 4 (LSTM) gates the BN = 64 NG accumulator columns are the
// pre-activations of the same 64 hidden units (NG 64-row boxes of the [NG H, K] weight), so the
// epilogue can apply the whole cell without another pass over memory.
//
// Every wait on an mbarrier is bounded: when it runs out the CTA records an error code in the
// status word, stops issuing work, releases its tensor memory and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mg {
namespace umma {

constexpr int BM = 128, BK = 64;
constexpr int kEpiWarps = 8;    // two warps per TMEM lane quarter, each taking half of the tile's columns
constexpr int kThreads = 64 + 32 * kEpiWarps;  // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, rest: epilogue
constexpr uint64_t kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int code,
                                          uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try(bar, parity)) return true;
  uint64_t t0 = global_ns();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if ((++spins & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicCAS(status, 0, code);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 128 bytes, groups
// of 8 rows 1024 bytes apart (stride byte offset), descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused with 128B swizzle, K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}

// Same for an MN-major operand (the matrix is stored [K rows][MN columns]): the stage holds one
// [64 k][64 mn] box (8 KiB, 128-byte rows) per 64 MN elements; leading byte offset = distance between
// those boxes, stride byte offset = distance between groups of 8 k rows.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(8192 >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// ... both MN-major (bits 15 and 16)
__host__ __device__ constexpr uint32_t instr_desc_bf16_mn(int n) { return instr_desc_bf16(n) | (1u << 15) | (1u << 16); }

// D fp32, A and B tf32 (fp32 words whose low 13 mantissa bits the producer has already rounded away), both K-major
__host__ __device__ constexpr uint32_t instr_desc_tf32(int n) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one MMA of .kind::tf32 consumes 8 k (again 32 bytes of a K-major row)
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 consecutive accumulator columns of this thread's row (lane)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

struct GemmShape {
  int M, N, K;          // row pitches must be multiples of 16 bytes (TMA stride rule); any M, N
  int gate_rows;        // NG > 0: row distance between the gate blocks of B (= H); else 0
  int splits;           // split products (MN-major, or an epilogue with kSplitAware): the reduction is cut into `splits`
  int kb_per_split;     // ranges of kb_per_split k-blocks, each (tile, range) is one work item and the epilogue is told
                        // which range it finishes; 0 or 1 = the whole reduction in one item
  int desc;             // 1: row tiles from the last to the first (a producer kernel wrote the A rows in ascending order:
                        // the rows written last are the ones still in L2)
  int a_from, a_add;    // a_add != 0: the A operand skips a column block of its array -- coordinates along the array's
                        // contiguous dimension (K for K-major, M for MN-major operands) at or beyond a_from move up by a_add
};

// An epilogue that can finish one range of a split reduction declares `static constexpr bool kSplitAware = true`
// and takes the range index as a fifth argument.
template <class E, class = void> struct EpiSplitAware { static constexpr bool value = false; };
template <class E> struct EpiSplitAware<E, decltype((void)E::kSplitAware)> { static constexpr bool value = E::kSplitAware; };

template <int BN, int NG>
struct Cfg {
  static constexpr int kStages = NG == 3 ? 5 : (BN <= 64 ? 8 : 4);
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kTmemCols = 512;  // two accumulators of BN <= 256 columns
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment*/ + 256 /*barriers*/;
  static constexpr int kNPerTile = NG > 0 ? BN / NG : BN;  // output columns (hidden units) per tile
};

// Epi: __device__ void operator()(uint32_t tmem_row_addr, int row, int n0, int half) const
//   tmem_row_addr: address of (this thread's lane, first column of the accumulator)
//   row: global output row of this thread (may be >= M: then only the tcgen05.ld's are executed)
//   n0 : first output column (NG > 0: first hidden unit) of the tile
//   half: 0 or 1, the half of the tile's output columns this warp is responsible for
// MNMAJ: D[m, n] = sum_k A[k, m] * B[k, n] with A stored [K, M] and B stored [K, N] (both row-major)
// TF32: the operands are fp32 words holding tf32 values (K-major only); a k-block is 32 of them, again 128 bytes a row
template <int BN, int NG, class Epi, bool MNMAJ = false, bool TF32 = false>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmShape sh, Epi epi,
                 int* status) {
  using C = Cfg<BN, NG>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t bars = tiles_base + C::kStages * C::kStageBytes;   // 8-byte barriers
  // full[s], empty[s], tmem_full[2], tmem_empty[2]
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * C::kStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * C::kStages + 2 + a); };
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (sh.M + BM - 1) / BM;
  const int n_tiles = (sh.N + C::kNPerTile - 1) / C::kNPerTile;
  static_assert(!(MNMAJ && TF32), "tf32 operands are K-major here");
  constexpr int kBK = TF32 ? BK / 2 : BK;                // elements of one 128-byte k-block row
  constexpr bool SPLITK = MNMAJ || EpiSplitAware<Epi>::value;
  const int k_blocks_all = (sh.K + kBK - 1) / kBK;
  const int splits = (SPLITK && sh.splits > 1) ? sh.splits : 1;
  const int mn_tiles = m_tiles * n_tiles;
  const int tiles = mn_tiles * splits;                   // work items
  // k-block range of item t (the whole reduction unless split)
  auto kb_begin = [&](int t) { return splits > 1 ? (t / mn_tiles) * sh.kb_per_split : 0; };
  auto kb_end = [&](int t) {
    if (splits == 1) return k_blocks_all;
    int e = (t / mn_tiles + 1) * sh.kb_per_split;
    return e < k_blocks_all ? e : k_blocks_all;
  };

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < C::kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 32 * kEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)),
                 "r"((uint32_t)C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;
  pdl_wait();     // everything above touched only shared memory and TMEM
  pdl_trigger();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x) {
        const int mq = (t % mn_tiles) / n_tiles, mt = sh.desc ? m_tiles - 1 - mq : mq, nt = t % n_tiles;
        for (int kb = kb_begin(t), kbe = kb_end(t); kb < kbe; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp, status, 1)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * C::kStageBytes;
          const uint32_t b_dst = a_dst + C::kABytes;
          mbar_expect_tx(full_bar(stage), C::kStageBytes);
          if (MNMAJ) {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) {
              int xa = mt * BM + i * 64;
              if (sh.a_add && xa >= sh.a_from) xa += sh.a_add;
              tma_load_2d(a_dst + i * 8192, &tmA, full_bar(stage), xa, kb * BK);
            }
#pragma unroll
            for (int i = 0; i < BN / 64; ++i) tma_load_2d(b_dst + i * 8192, &tmB, full_bar(stage), nt * BN + i * 64, kb * BK);
          } else {
          tma_load_2d(a_dst, &tmA, full_bar(stage), (sh.a_add && kb * kBK >= sh.a_from) ? kb * kBK + sh.a_add : kb * kBK, mt * BM);
          if (NG > 0) {
#pragma unroll
            for (int g = 0; g < NG; ++g)
              tma_load_2d(b_dst + g * (C::kBBytes / (NG > 0 ? NG : 1)), &tmB, full_bar(stage), kb * kBK, g * sh.gate_rows + nt * C::kNPerTile);
          } else {
            tma_load_2d(b_dst, &tmB, full_bar(stage), kb * kBK, nt * BN);
          }
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = TF32 ? instr_desc_tf32(BN) : (MNMAJ ? instr_desc_bf16_mn(BN) : instr_desc_bf16(BN));
      int stage = 0; uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < tiles && ok; t += gridDim.x, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abortp, status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        const int kb0 = kb_begin(t);
        for (int kb = kb0, kbe = kb_end(t); kb < kbe; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp, status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * C::kStageBytes;
          const uint64_t adesc = MNMAJ ? smem_desc_mn_sw128(a_src) : smem_desc_sw128(a_src);
          const uint64_t bdesc = MNMAJ ? smem_desc_mn_sw128(a_src + C::kABytes) : smem_desc_sw128(a_src + C::kABytes);
          // one MMA consumes 16 bf16 (8 tf32) k: 32 bytes along a K-major row, 16 rows of 128 bytes (2048 bytes) when MN-major
          constexpr uint64_t kstep = MNMAJ ? (2048 >> 4) : (32 >> 4);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            if constexpr (TF32) mma_tf32(d_tmem, adesc + kstep * k, bdesc + kstep * k, idesc, ((kb - kb0) | k) != 0 ? 1u : 0u);
            else mma_bf16(d_tmem, adesc + kstep * k, bdesc + kstep * k, idesc, ((kb - kb0) | k) != 0 ? 1u : 0u);
          }
          mma_commit(empty_bar(stage));   // frees the stage when the MMAs have read it
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) mma_commit(tfull_bar(as));  // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;             // TMEM lane quarter this warp may access
    const int half = (warp - 2) >> 2;   // which half of the tile's columns this warp handles
    int it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
      const int mq = (t % mn_tiles) / n_tiles, mt = sh.desc ? m_tiles - 1 - mq : mq, nt = t % n_tiles;
      const int as = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      if (!mbar_wait(tfull_bar(as), aphase, abortp, status, 4)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
      if constexpr (SPLITK) epi(taddr, mt * BM + q * 32 + lane, nt * C::kNPerTile, half, t / mn_tiles);
      else epi(taddr, mt * BM + q * 32 + lane, nt * C::kNPerTile, half);
      tc_fence_before();
      mbar_arrive(tempty_bar(as));
    }
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::kTmemCols) : "memory");
  }
}

}  // namespace umma
}  // namespace mg
