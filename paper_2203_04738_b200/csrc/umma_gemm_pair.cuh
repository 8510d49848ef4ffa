// Plain GEMM D[m, n] = sum_k A[m, k] * B[n, k] as CTA pairs (tcgen05 cta_group::2): two CTAs of a cluster, on the
// two SMs of one TPC, share one 256 x 256 MMA.  Each stages its own 128 rows of A and 128 of the 256 rows of the
// B tile per k-block (32 KiB instead of 48), so the per-SM operand ingest per flop drops by a third.
//
// Protocol (every wait bounded as in the single-CTA kernel):
//  * both CTAs' TMA loads complete on the LEADER's (rank 0) full barrier, which expects the bytes of both;
//  * the leader's MMA thread issues for the pair and commits each stage to both CTAs' empty barriers and each
//    accumulator to both CTAs' tfull barriers (one commit per destination; every TMA load has a single destination CTA);
//  * both CTAs' epilogue warps arrive on the leader's tempty barrier (remote arrive for rank 1);
//  * tensor memory is allocated and freed by the same warp of both CTAs, behind cluster barriers.
#pragma once
#include "umma_gemm.cuh"

namespace mg {
namespace umma {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion barrier may live in the other CTA of the pair (bar is a shared::cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// Instruction descriptor of the pair MMA: M = 256 over the two CTAs, N = n, bf16 K-major operands, fp32 D
__host__ __device__ constexpr uint32_t instr_desc_bf16_pair(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on ONE barrier (a shared::cluster address, in either CTA) once the pair MMAs issued so far are done
__device__ __forceinline__ void mma_commit_pair(uint32_t cluster_bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}

namespace pairk {
constexpr int BN = 256, kStages = 6;
constexpr int kABytes = BM * BK * 2, kBBytes = (BN / 2) * BK * 2, kStageBytes = kABytes + kBBytes;
constexpr int kSmemBytes = kStages * kStageBytes + 1024 + 256;
}  // namespace pairk

template <class Epi>
__global__ void __launch_bounds__(kThreads, 1)
umma_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmShape sh, Epi epi,
                      int* status) {
  using namespace pairk;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t bars = tiles_base + kStages * kStageBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * kStages + 2 + a); };
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int cta = (int)(blockIdx.x >> 1), ncta = (int)(gridDim.x >> 1);
  const int m_tiles = (sh.M + 2 * BM - 1) / (2 * BM);     // a tile is 256 rows; CTA `rank` owns rows [128 rank, +128)
  const int n_tiles = (sh.N + BN - 1) / BN;
  const int tiles = m_tiles * n_tiles;
  const int k_blocks = (sh.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * 32 * kEpiWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // the same warp of both CTAs allocates the same columns in both tensor memories
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_smem)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;
  pdl_wait();
  pdl_trigger();

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      for (int t = cta; t < tiles && ok; t += ncta) {
        const int mq = t / n_tiles, mt = 2 * (sh.desc ? m_tiles - 1 - mq : mq) + (int)rank, nt = t % n_tiles;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp, status, 21)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          const uint32_t fullL = mapa_shared(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
          tma_load_2d_pair(a_dst, &tmA, fullL, (sh.a_add && kb * BK >= sh.a_from) ? kb * BK + sh.a_add : kb * BK, mt * BM);
          tma_load_2d_pair(b_dst, &tmB, fullL, kb * BK, nt * BN + (int)rank * (BN / 2));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc_bf16_pair(BN);
      int stage = 0; uint32_t phase = 0; int it = 0; bool ok = true;
      for (int t = cta; t < tiles && ok; t += ncta, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abortp, status, 22)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp, status, 23)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * kStageBytes;
          const uint64_t adesc = smem_desc_sw128(a_src), bdesc = smem_desc_sw128(a_src + kABytes);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            mma_bf16_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          mma_commit_pair(mapa_shared(empty_bar(stage), 0));   // the stage is free again in both CTAs
          mma_commit_pair(mapa_shared(empty_bar(stage), 1));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          mma_commit_pair(mapa_shared(tfull_bar(as), 0));
          mma_commit_pair(mapa_shared(tfull_bar(as), 1));
        }
      }
    }
  } else {
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    int it = 0;
    for (int t = cta; t < tiles; t += ncta, ++it) {
      const int mq = t / n_tiles, mt = 2 * (sh.desc ? m_tiles - 1 - mq : mq) + (int)rank, nt = t % n_tiles;
      const int as = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      if (!mbar_wait(tfull_bar(as), aphase, abortp, status, 24)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BN);
      epi(taddr, mt * BM + q * 32 + lane, nt * BN, half);
      tc_fence_before();
      mbar_arrive_cluster(mapa_shared(tempty_bar(as), 0));
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves (or frees tensor memory) while the other may still signal it
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace umma
}  // namespace mg
