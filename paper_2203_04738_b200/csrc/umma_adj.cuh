// Adjoint step product with TMA-staged epilogue operands, sm_100a:
//
//   rows m = (k, b)          k = interval / coarse point, b = batch row, 128 rows per CTA = kt k's x B
//   D[m, n]   = sum_j dA[m, j] * W_hhT[n, j]           dA = [c_r | c_z | c_n] * lambda as bf16 [M, 3H] (packed beforehand)
//   out[m, n] = a[m, n] * lambda[m, n] + D[m, n] (+ g[m, n])      or   g - (...)   (mode 1)
//
// The plain GEMM's epilogue read lambda, a and g with one 32-byte global load per thread, row and 8 columns, and the
// product was bound by that epilogue (without those loads a 16384-row step took 117 instead of 153 us).  Here a third
// producer warp stages them by TMA in chunks of 16 columns (64-byte rows, 64-byte swizzle, conflict-free 16-byte
// shared-memory loads), several chunks in flight, exactly as the fused forward kernel does for its operands.
// Coefficient rows are stored in forward time order while the adjoint walks backwards, so their k-stride is negative:
// the tensor map then starts at the lowest address and the k coordinate is reversed (a tile's rows arrive in reversed
// k order; a load may start at a negative coordinate and reads zeros there).
//
// Two geometries as in the other tensor-core kernels: CTA pairs (256 x 256 tiles, cta_group::2) and single CTAs
// (128 x 256).  Warp roles (352 threads): 0 = TMA producer of the A/B ring, 1 = MMA issuer and TMEM owner,
// 2 = TMA producer of the epilogue operands, 3..10 = epilogue.  Every wait on an mbarrier is bounded.
#pragma once
#include "umma_cell.cuh"

namespace mg {
namespace umma {

struct AdjKArgs {
  int M, B, H, kt, nk;                // kt = 128 / B
  float* lout; i64 lout_ks;           // result rows (k, b)
  int a_rev;                          // 1: the coefficient map runs backwards in k (coordinate nk - 1 - k)
  int mode;
};

namespace adjk {
constexpr int ACH = 16, ABN = 256, kAdjThreads = 352;
constexpr int kAdjOpBytes = BM * ACH * 4;
template <bool HAS_G, bool PAIR> struct ACfg {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = (PAIR ? ABN / 2 : ABN) * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;        // 32 KiB / 48 KiB
  static constexpr int kStages = PAIR ? (HAS_G ? 4 : 5) : 3;
  static constexpr int kOps = HAS_G ? 3 : 2;
  static constexpr int kEpiBytes = kOps * kAdjOpBytes;
  static constexpr int kEpiBufs = PAIR ? 3 : (HAS_G ? 3 : 4);
  static constexpr int kSmemBytes = kStages * kStageBytes + kEpiBufs * kEpiBytes + 1024 + 256;
  static_assert(kSmemBytes + 2048 <= 232448, "shared memory budget");
};
}  // namespace adjk

template <bool HAS_G, bool PAIR>
__global__ void __launch_bounds__(adjk::kAdjThreads, 1)
umma_adj_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmL, const __grid_constant__ CUtensorMap tmCa,
                const __grid_constant__ CUtensorMap tmG, AdjKArgs p, int K, int* status) {
  using namespace adjk;
  using C = ACfg<HAS_G, PAIR>;
  constexpr int CHa = ACH, BNa = ABN, kOpB = kAdjOpBytes;
  constexpr int kStageBytes = C::kStageBytes, kABytes = C::kABytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const uint32_t epi_base = tiles_base + C::kStages * kStageBytes;
  const uint32_t bars = epi_base + C::kEpiBufs * C::kEpiBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * C::kStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * C::kStages + 2 + a); };
  auto efull_bar = [&](int e) { return bars + 8u * (2 * C::kStages + 4 + e); };
  auto eempty_bar = [&](int e) { return bars + 8u * (2 * C::kStages + 4 + C::kEpiBufs + e); };
  __shared__ uint32_t tmem_base_smem;
  __shared__ int abort_flag;
  __shared__ uint32_t lds_sink[kAdjThreads];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int H = p.H;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int cta = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, ncta = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int kTileRows = PAIR ? 2 * BM : BM;
  const int m_tiles = (p.M + kTileRows - 1) / kTileRows, n_tiles = (H + BNa - 1) / BNa, tiles = m_tiles * n_tiles;
  const int k_blocks = (K + BK - 1) / BK;
  // Row tiles from the last to the first: the packing kernel writes the operand rows in ascending order and most of the
  // 100 MB of a 16384-row step have left L2 by the time it ends, except the rows written last (and this kernel's
  // results of the first rows are the newest when the next packing kernel starts there).
  auto row_tile = [&](int t) { const int q = m_tiles - 1 - t / n_tiles; return PAIR ? 2 * q + (int)rank : q; };

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
    if (PAIR) {
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
  if (PAIR) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_smem;
  volatile int* abortp = &abort_flag;
  pdl_wait();
  pdl_trigger();

  if (warp == 0) {
    // ------------------------------------------------------------ A/B producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      uint64_t drop_policy;
      asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(drop_policy));
      for (int t = cta; t < tiles && ok; t += ncta) {
        const int mt = row_tile(t), nt = t % n_tiles;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp, status, 31)) { ok = false; break; }
          const uint32_t a_dst = tiles_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          if (PAIR) {
            const uint32_t fullL = mapa_shared(full_bar(stage), 0);
            if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);
            // the packed operand is read once: let it leave L2 first
            asm volatile(
                "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
                ::"r"(a_dst), "l"(&tmA), "r"(fullL), "r"(kb * BK), "r"(mt * BM), "l"(drop_policy)
                : "memory");
            tma_load_2d_pair(b_dst, &tmB, fullL, kb * BK, nt * BNa + (int)rank * (BNa / 2));
          } else {
            mbar_expect_tx(full_bar(stage), kStageBytes);
            tma_load_2d(a_dst, &tmA, full_bar(stage), kb * BK, mt * BM);
            tma_load_2d(b_dst, &tmB, full_bar(stage), kb * BK, nt * BNa);
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (PAIR: the leader issues for both CTAs)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = PAIR ? instr_desc_bf16_pair(BNa) : instr_desc_bf16(BNa);
      int stage = 0; uint32_t phase = 0; int it = 0; bool ok = true;
      for (int t = cta; t < tiles && ok; t += ncta, ++it) {
        const int as = it & 1;
        const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abortp, status, 32)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(as * BNa);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp, status, 33)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = tiles_base + stage * kStageBytes;
          const uint64_t adesc = smem_desc_sw128(a_src), bdesc = smem_desc_sw128(a_src + kABytes);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if (PAIR) mma_bf16_pair(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
            else mma_bf16(d_tmem, adesc + (uint64_t)(k * 2), bdesc + (uint64_t)(k * 2), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          if (PAIR) {
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
      for (int t = cta; t < tiles && ok; t += ncta) {
        const int mt = row_tile(t), nt = t % n_tiles;
        const int k0 = mt * p.kt;
        const int ka = p.a_rev ? p.nk - k0 - p.kt : k0;      // may be negative in the last row tile: those rows read zeros
        for (int c = 0; c < BNa / CHa; ++c) {
          const int n = nt * BNa + c * CHa;
          if (n >= H) break;
          if (!mbar_wait(eempty_bar(eb), ephase ^ 1u, abortp, status, 34)) { ok = false; break; }
          const uint32_t dst = epi_base + eb * C::kEpiBytes;
          mbar_expect_tx(efull_bar(eb), C::kEpiBytes);
          tma_load_3d(dst, &tmL, efull_bar(eb), n, 0, k0);
          tma_load_3d(dst + kOpB, &tmCa, efull_bar(eb), n, 0, ka);
          if (HAS_G) tma_load_3d(dst + 2 * kOpB, &tmG, efull_bar(eb), n, 0, k0);
          if (++eb == C::kEpiBufs) { eb = 0; ephase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 3..10)
    const int q = warp & 3;              // TMEM lane quarter of this warp
    const int half = (warp - 3) >> 2;    // which 8 of a chunk's 16 columns
    const int r = q * 32 + lane;         // row inside the CTA's 128 rows
    const int kl = r / p.B, bl = r - kl * p.B;
    const int ra = p.a_rev ? (p.kt - 1 - kl) * p.B + bl : r;     // where this row's coefficients sit in their tile
    auto swz = [&](int row, uint32_t piece) { return (uint32_t)row * 64u + ((piece ^ ((uint32_t)(row >> 1) & 3u)) << 4); };
    const uint32_t off0 = swz(r, (uint32_t)half * 2u), off1 = swz(r, (uint32_t)half * 2u + 1u);
    const uint32_t oa0 = swz(ra, (uint32_t)half * 2u), oa1 = swz(ra, (uint32_t)half * 2u + 1u);
    int it = 0, eb = 0; uint32_t ephase = 0;
    bool ok = true;
    for (int t = cta; t < tiles; t += ncta, ++it) {
      const int mt = row_tile(t), nt = t % n_tiles;
      const int as = it & 1;
      const uint32_t aphase = (uint32_t)(it >> 1) & 1u;
      const int row = mt * BM + r;
      const bool valid = row < p.M;
      const int k = mt * p.kt + kl;
      if (ok && !mbar_wait(tfull_bar(as), aphase, abortp, status, 35)) ok = false;
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(as * BNa);
      for (int c = 0; c < BNa / CHa; ++c) {
        if (nt * BNa + c * CHa >= H) break;
        if (ok && !mbar_wait(efull_bar(eb), ephase, abortp, status, 36)) ok = false;
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
          const uint32_t src = epi_base + eb * C::kEpiBytes;
          float l[8], ac[8], g[8], v[8];
          *reinterpret_cast<float4*>(l) = lds4(src + off0);              *reinterpret_cast<float4*>(l + 4) = lds4(src + off1);
          *reinterpret_cast<float4*>(ac) = lds4(src + kOpB + oa0);   *reinterpret_cast<float4*>(ac + 4) = lds4(src + kOpB + oa1);
          if (HAS_G) {
            *reinterpret_cast<float4*>(g) = lds4(src + 2 * kOpB + off0); *reinterpret_cast<float4*>(g + 4) = lds4(src + 2 * kOpB + off1);
          }
          tmem_ld8(taddr + c * CHa + half * 8, v);
          tmem_ld_wait8(v);
          {   // release the buffer only after its values have arrived in registers (see the fused forward kernel)
            uint32_t dep = __float_as_uint(l[0]) ^ __float_as_uint(l[4]) ^ __float_as_uint(ac[0]) ^ __float_as_uint(ac[4]);
            if (HAS_G) dep ^= __float_as_uint(g[0]) ^ __float_as_uint(g[4]);
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_u32(&lds_sink[threadIdx.x])), "r"(dep) : "memory");
          }
          mbar_arrive(eempty_bar(eb));
          if (++eb == C::kEpiBufs) { eb = 0; ephase ^= 1u; }
          if (valid) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float o = ac[e] * l[e] + v[e];
              v[e] = HAS_G ? (p.mode == 1 ? g[e] - o : o + g[e]) : o;
            }
            stg8(p.lout + (i64)k * p.lout_ks + (i64)bl * H + nt * BNa + c * CHa + half * 8, v);
          }
        }
      }
      if (ok) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (PAIR) mbar_arrive_cluster(mapa_shared(tempty_bar(as), 0));
          else mbar_arrive(tempty_bar(as));
        }
      }
    }
  }

  // ------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    if (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

}  // namespace umma
}  // namespace mg
