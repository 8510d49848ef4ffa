// Tensor-core engine: bf16 operands, fp32 accumulation in tensor memory, fp32 states and gates.
// Host launchers, operand-packing kernels and the fused epilogues of the tcgen05 GEMM.
#include <stdio.h>
#include <stdlib.h>

#include "cell.cuh"
#include "umma_engine.cuh"
#include "umma_cell.cuh"
#include "umma_adj.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_pair.cuh"

namespace mg {

namespace {

using namespace umma;
typedef __nv_bfloat16 bf16;

__device__ int g_umma_status = 0;   // first error code of a bounded wait that ran out (0 = none)
int* g_status_ptrs[kMaxDevices] = {nullptr};   // its address on each device

constexpr int kSMs = 148;

// ---------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// Status word of the current device (nullptr on failure); also resolves the tensor-map encoder.
// MGRIT_GRU_TEST_FAIL_ENCODE=1 in the environment makes this fail, so that the error path of a launch that
// cannot be prepared can be exercised from the host without launching anything.
int* status_ptr() {
  static int fail = -1;
  if (fail < 0) { const char* e = getenv("MGRIT_GRU_TEST_FAIL_ENCODE"); fail = (e && e[0] == '1') ? 1 : 0; }
  if (fail) return nullptr;
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return nullptr;
    g_encode = (EncodeTiledFn)fn;
  }
  const int dev = current_device_slot();
  if (dev < 0) return nullptr;
  if (!g_status_ptrs[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_umma_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    g_status_ptrs[dev] = p;
  }
  return g_status_ptrs[dev];
}

// bf16 matrix [rows, inner] with row pitch `pitch` elements; box = 64 x box_rows, 128-byte swizzle
bool make_map(CUtensorMap* m, const bf16* base, uint64_t inner, uint64_t rows, uint64_t pitch, uint32_t box_rows) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch * sizeof(bf16)};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)base, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) fprintf(stderr, "mgrit_gru: cuTensorMapEncodeTiled failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

// fp32 words holding tf32 values: box = 32 x box_rows (again 128-byte rows)
bool make_map(CUtensorMap* m, const float* base, uint64_t inner, uint64_t rows, uint64_t pitch, uint32_t box_rows) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch * sizeof(float)};
  cuuint32_t box[2] = {(cuuint32_t)(BK / 2), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, (void*)base, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) fprintf(stderr, "mgrit_gru: cuTensorMapEncodeTiled (fp32) failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

// ET = bf16, or float for operands that hold tf32 values.  splits > 1 (split-aware epilogues only) cuts the reduction.
template <int BN, int NG, class Epi, class ET>
// a_ext / a_from / a_add: the A operand skips a column block of its array (see GemmShape); a_ext = columns of the array.
bool launch_gemm(int kc, const ET* A, i64 lda, const ET* Bm, i64 ldb, int M, int N, int K, int gate_rows, int b_rows, Epi epi,
                 cudaStream_t s, int splits = 1, bool desc = false, int a_ext = 0, int a_from = 0, int a_add = 0) {
  using C = Cfg<BN, NG>;
  constexpr bool TF32 = sizeof(ET) == 4;
  if (M <= 0 || N <= 0) return true;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_gemm_kernel<BN, NG, Epi, false, TF32>;
  if (!set_smem_once(kern, C::kSmemBytes, attr_set)) return false;
  CUtensorMap ta, tb;
  if (!make_map(&ta, A, (uint64_t)(a_ext > 0 ? a_ext : K), (uint64_t)M, (uint64_t)lda, BM)) return false;
  if (!make_map(&tb, Bm, (uint64_t)K, (uint64_t)b_rows, (uint64_t)ldb, NG > 0 ? BN / NG : BN)) return false;
  const int k_blocks = (K + (TF32 ? BK / 2 : BK) - 1) / (TF32 ? BK / 2 : BK);
  if (splits < 1 || !EpiSplitAware<Epi>::value) splits = 1;
  GemmShape sh{M, N, K, gate_rows, splits, (k_blocks + splits - 1) / splits, desc ? 1 : 0, a_from, a_add};
  int m_tiles = (M + BM - 1) / BM, n_tiles = (N + C::kNPerTile - 1) / C::kNPerTile;
  int tiles = m_tiles * n_tiles * splits;
  int grid = tiles < kSMs ? tiles : kSMs;
  ProfScope prof_(kc, 2.0 * M * (NG > 0 ? (double)NG * N : (double)N) * K, s);
  if (launch_pdl(kern, dim3(grid), dim3(kThreads), C::kSmemBytes, s, ta, tb, sh, epi, status) != cudaSuccess) return false;
  count_launch();
  return true;
}

// The same product on CTA pairs (256 x 256 tiles); K-major operands, N columns in tiles of 256.
// Used when the product has more 128 x 256 tiles than SMs (below that every CTA has at most one tile and the
// single-CTA kernel is as fast).  MGRIT_GRU_GEMM_PAIR=0 in the environment keeps every product on single CTAs.
static bool gemm_pair_enabled(int M, int N) {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_GEMM_PAIR"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1 && (i64)((M + BM - 1) / BM) * ((N + 255) / 256) > kSMs;
}
template <class Epi>
bool launch_gemm_pair(int kc, const bf16* A, i64 lda, const bf16* Bm, i64 ldb, int M, int N, int K, int b_rows, Epi epi, cudaStream_t s,
                      bool desc = false, int a_ext = 0, int a_from = 0, int a_add = 0) {
  if (M <= 0 || N <= 0) return true;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_gemm_pair_kernel<Epi>;
  if (!set_smem_once(kern, pairk::kSmemBytes, attr_set)) return false;
  CUtensorMap ta, tb;
  if (!make_map(&ta, A, (uint64_t)(a_ext > 0 ? a_ext : K), (uint64_t)M, (uint64_t)lda, BM)) return false;
  if (!make_map(&tb, Bm, (uint64_t)K, (uint64_t)b_rows, (uint64_t)ldb, pairk::BN / 2)) return false;
  GemmShape sh{M, N, K, 0, 1, 0, desc ? 1 : 0, a_from, a_add};
  int tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + pairk::BN - 1) / pairk::BN);
  int grid = 2 * (tiles < kSMs / 2 ? tiles : kSMs / 2);
  ProfScope prof_(kc, 2.0 * M * (double)N * K, s);
  if (launch_pdl_cluster(kern, 2, dim3(grid), dim3(kThreads), pairk::kSmemBytes, s, ta, tb, sh, epi, status) != cudaSuccess)
    return false;
  count_launch();
  return true;
}

// D[m, n] = sum_k A[k, m] * B[k, n]: both operands stored with the reduction index as the ROW index
// (A: [K, Mdim], B: [K, Ndim], row-major), consumed as MN-major tensor-core operands -- the shape of the
// weight-gradient reductions dW = dA^T h, which therefore need no transposed copies.
template <class Epi>
bool launch_gemm_mn(int kc, const bf16* A, i64 lda, int Mdim, const bf16* Bm, i64 ldb, int Ndim, int K, int splits, Epi epi,
                    cudaStream_t s, int a_ext = 0, int a_from = 0, int a_add = 0) {
  using C = Cfg<256, 0>;
  if (Mdim <= 0 || Ndim <= 0) return true;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_gemm_kernel<256, 0, Epi, true>;
  if (!set_smem_once(kern, C::kSmemBytes, attr_set)) return false;
  CUtensorMap ta, tb;
  if (!make_map(&ta, A, (uint64_t)(a_ext > 0 ? a_ext : Mdim), (uint64_t)K, (uint64_t)lda, 64)) return false;
  if (!make_map(&tb, Bm, (uint64_t)Ndim, (uint64_t)K, (uint64_t)ldb, 64)) return false;
  const int k_blocks = (K + BK - 1) / BK;
  if (splits < 1) splits = 1;
  GemmShape sh{Mdim, Ndim, K, 0, splits, (k_blocks + splits - 1) / splits, 0, a_from, a_add};
  int tiles = ((Mdim + BM - 1) / BM) * ((Ndim + 255) / 256) * splits;
  int grid = tiles < kSMs ? tiles : kSMs;
  ProfScope prof_(kc, 2.0 * Mdim * (double)Ndim * K, s);
  if (launch_pdl(kern, dim3(grid), dim3(kThreads), C::kSmemBytes, s, ta, tb, sh, epi, status) != cudaSuccess) return false;
  count_launch();
  return true;
}

// 3-D map {column, batch row, k}: rows (k, b) at base + k*ks + b*ld, `inner` columns
bool make_map3(CUtensorMap* m, CUtensorMapDataType dt, size_t esize, const void* base, uint64_t inner, uint64_t B, uint64_t nk,
               uint64_t ld, i64 ks, uint32_t box_inner, uint32_t box_k, CUtensorMapSwizzle sw) {
  if (ks <= 0) ks = (i64)(ld * B);       // a single k: any legal stride
  cuuint64_t dims[3] = {inner, B, nk};
  cuuint64_t strides[2] = {ld * esize, (cuuint64_t)ks * esize};
  cuuint32_t box[3] = {box_inner, (cuuint32_t)B, box_k};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(m, dt, 3, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) fprintf(stderr, "mgrit_gru: cuTensorMapEncodeTiled (3-D) failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

// 2-D map of a row-major [rows, inner] array (row pitch ld elements), box {box_inner, box_rows}
bool make_map2(CUtensorMap* m, CUtensorMapDataType dt, size_t esize, const void* base, uint64_t inner, uint64_t rows, uint64_t ld,
               uint32_t box_inner, uint32_t box_rows, CUtensorMapSwizzle sw) {
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {ld * esize};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(m, dt, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) fprintf(stderr, "mgrit_gru: cuTensorMapEncodeTiled (2-D) failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

// The fused kernel on CTA pairs (256 x 240 tiles) is used when the step has at least one full wave of such tiles;
// smaller steps stay on single CTAs (128 x 192 tiles).  MGRIT_GRU_CELL_PAIR=0 keeps every step on single CTAs.
static bool cell_pair_enabled(int M, int H) {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_CELL_PAIR"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1 && (i64)(M / (2 * BM)) * ((H + 79) / 80) >= kSMs / 2;
}

// 4-D map {column, batch row, slot, interval}: element (c, b, sl, k) at base + k*ks + sl*ss + b*ld + c
bool make_map4(CUtensorMap* m, CUtensorMapDataType dt, size_t esize, const void* base, uint64_t inner, uint64_t B, uint64_t nslots,
               uint64_t nk, uint64_t ld, i64 ss, i64 ks, uint32_t box_inner, uint32_t box_k, CUtensorMapSwizzle sw) {
  if (ks <= 0) ks = (i64)(ld * B);       // a single interval: any legal stride
  if (ss <= 0) ss = (i64)(ld * B);       // a single slot
  cuuint64_t dims[4] = {inner, B, nslots, nk};
  cuuint64_t strides[3] = {ld * esize, (cuuint64_t)ss * esize, (cuuint64_t)ks * esize};
  cuuint32_t box[4] = {box_inner, (cuuint32_t)B, 1, box_k};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = g_encode(m, dt, 4, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) fprintf(stderr, "mgrit_gru: cuTensorMapEncodeTiled (4-D) failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

// Adjoint linearisation on the fused kernel, TMA-staged epilogue operands.
// Rows (k, b), k = 0..nk-1: A rows at A + k*a_ks + b*H (bf16), gi rows at gi + k*gi_ks + b*3H,
// previous state at hp + k*hp_ks + b*H.
template <bool PAIR, bool GIB>
bool launch_lin_geo(int kc, const bf16* A, i64 a_ks, const void* gi, i64 gi_ks, const float* hp, i64 hp_ks, int nk, const bf16* W,
                    CellArgs ca, cudaStream_t s) {
  using C = cellk::CellCfg<false, true, PAIR, GIB>;
  using G = cellk::Geo<PAIR>;
  if (nk <= 0) return true;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_cell_kernel<true, false, PAIR, GIB>;
  if (!set_smem_once(kern, C::kSmemBytes, attr_set)) return false;
  const int B = ca.B, H = ca.H, kt = 128 / B;
  ca.kt = kt; ca.M = nk * B;
  CUtensorMap ta, tb, tgi, thp;
  if (!make_map3(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, A, H, B, nk, H, a_ks, BK, kt, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
  if (!make_map(&tb, W, (uint64_t)H, (uint64_t)3 * H, (uint64_t)H, G::kBox)) return false;
  if (GIB ? !make_map3(&tgi, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, gi, 3 * H, B, nk, 3 * H, gi_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_32B)
          : !make_map3(&tgi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, gi, 3 * H, B, nk, 3 * H, gi_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_64B))
    return false;
  if (!make_map3(&thp, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, hp, H, B, nk, H, hp_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  // the four bf16 coefficient arrays [M, H] are written by TMA stores of [128 x 16] tiles
  CUtensorMap tcr = thp, tcz = thp, tcn = thp, tcp = thp;
  auto cmap = [&](CUtensorMap* m, const bf16* base) {
    return make_map2(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, H, (uint64_t)ca.M, H, cellk::CH, BM, CU_TENSOR_MAP_SWIZZLE_32B);
  };
  if (!cmap(&tcr, ca.cr) || !cmap(&tcz, ca.cz) || !cmap(&tcn, ca.cn) || (ca.cnp && !cmap(&tcp, ca.cnp))) return false;
  CUtensorMap taout = thp;      // with the bf16-staged projection `a` is written by TMA stores too ([128 x 16] fp32 tiles)
  if (GIB && !make_map2(&taout, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ca.a, H, (uint64_t)ca.M, H, cellk::CH, BM, CU_TENSOR_MAP_SWIZZLE_64B))
    return false;
  constexpr int kTileRows = PAIR ? 2 * BM : BM;
  const int tiles = ((ca.M + kTileRows - 1) / kTileRows) * ((H + G::UN - 1) / G::UN);
  SweepArgs sw{};
  sw.n_steps = 1;
  ProfScope prof_(kc, 2.0 * ca.M * 3.0 * H * H, s);
  cudaError_t e;
  if (PAIR) {
    const int grid = 2 * (tiles < kSMs / 2 ? tiles : kSMs / 2);
    e = launch_pdl_cluster(kern, 2, dim3(grid), dim3(cellk::kThreads), C::kSmemBytes, s, ta, tb, tgi, thp, taout, tcr, tcz, tcn, tcp, ca, sw, status);
  } else {
    const int grid = tiles < kSMs ? tiles : kSMs;
    e = launch_pdl(kern, dim3(grid), dim3(cellk::kThreads), C::kSmemBytes, s, ta, tb, tgi, thp, taout, tcr, tcz, tcn, tcp, ca, sw, status);
  }
  if (e != cudaSuccess) return false;
  count_launch();
  return true;
}
// gi: fp32 rows, or (gib) their bf16 copy with the same element indexing
bool launch_lin(int kc, const bf16* A, i64 a_ks, const void* gi, bool gib, i64 gi_ks, const float* hp, i64 hp_ks, int nk, const bf16* W,
                CellArgs ca, cudaStream_t s) {
  const bool pair = cell_pair_enabled(nk * ca.B, ca.H);
  if (gib) return pair ? launch_lin_geo<true, true>(kc, A, a_ks, gi, gi_ks, hp, hp_ks, nk, W, ca, s)
                       : launch_lin_geo<false, true>(kc, A, a_ks, gi, gi_ks, hp, hp_ks, nk, W, ca, s);
  return pair ? launch_lin_geo<true, false>(kc, A, a_ks, gi, gi_ks, hp, hp_ks, nk, W, ca, s)
              : launch_lin_geo<false, false>(kc, A, a_ks, gi, gi_ks, hp, hp_ks, nk, W, ca, s);
}

// Forward steps on the fused kernel: one launch runs sw.n_steps dependent steps over the same rows (k, b), k = 0..nk-1.
// The state (A: bf16 copy, hp: fp32), the input projection and the additive term are addressed as
// base + k*ks + slot*ss + b*ld with the slot coordinate taken from each step (nslots = 1: a single step, coordinate 0).
struct CellFwdOperands {
  const bf16* A; const float* hp; i64 in_ss, in_ks; int in_slots;
  const float* gi; i64 gi_ss, gi_ks; const float* g; i64 g_ss, g_ks; int tgt_slots;
  const bf16* gi_b;      // bf16 copy of gi (same element indexing) or nullptr: staged instead of the fp32 rows
};
template <bool HAS_G, bool PAIR, bool GIB>
bool launch_fwd_geo(int kc, const CellFwdOperands& o, int nk, const bf16* W, CellArgs ca, const SweepArgs& sw, cudaStream_t s) {
  using C = cellk::CellCfg<HAS_G, false, PAIR, GIB>;
  using G = cellk::Geo<PAIR>;
  if (nk <= 0) return true;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_cell_kernel<false, HAS_G, PAIR, GIB>;
  if (!set_smem_once(kern, C::kSmemBytes, attr_set)) return false;
  const int B = ca.B, H = ca.H, kt = 128 / B;
  ca.kt = kt; ca.M = nk * B;
  CUtensorMap ta, tb, tgi, thp, tg;
  const auto f32 = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  if (!make_map4(&ta, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, o.A, H, B, o.in_slots, nk, H, o.in_ss, o.in_ks, BK, kt, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
  if (!make_map(&tb, W, (uint64_t)H, (uint64_t)3 * H, (uint64_t)H, G::kBox)) return false;
  if (GIB ? !make_map4(&tgi, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, o.gi_b, 3 * H, B, o.tgt_slots, nk, 3 * H, o.gi_ss, o.gi_ks, cellk::CH, kt,
                       CU_TENSOR_MAP_SWIZZLE_32B)
          : !make_map4(&tgi, f32, 4, o.gi, 3 * H, B, o.tgt_slots, nk, 3 * H, o.gi_ss, o.gi_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_64B))
    return false;
  if (!make_map4(&thp, f32, 4, o.hp, H, B, o.in_slots, nk, H, o.in_ss, o.in_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  if (HAS_G) {
    if (!make_map4(&tg, f32, 4, o.g, H, B, o.tgt_slots, nk, H, o.g_ss, o.g_ks, cellk::CH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  } else {
    tg = thp;
  }
  constexpr int kTileRows = PAIR ? 2 * BM : BM;
  const int tiles = ((ca.M + kTileRows - 1) / kTileRows) * ((H + G::UN - 1) / G::UN);
  const i64 items = (i64)tiles * sw.n_steps;
  ProfScope prof_(kc, 2.0 * ca.M * 3.0 * H * H * sw.n_steps, s);
  cudaError_t e;
  if (PAIR) {
    const int grid = 2 * (int)(items < kSMs / 2 ? items : kSMs / 2);
    e = launch_pdl_cluster(kern, 2, dim3(grid), dim3(cellk::kThreads), C::kSmemBytes, s, ta, tb, tgi, thp, tg, thp, thp, thp, thp, ca, sw, status);
  } else {
    const int grid = (int)(items < kSMs ? items : kSMs);
    e = launch_pdl(kern, dim3(grid), dim3(cellk::kThreads), C::kSmemBytes, s, ta, tb, tgi, thp, tg, thp, thp, thp, thp, ca, sw, status);
  }
  if (e != cudaSuccess) return false;
  count_launch();
  return true;
}
template <bool HAS_G>
bool launch_fwd(int kc, const CellFwdOperands& o, int nk, const bf16* W, const CellArgs& ca, const SweepArgs& sw, cudaStream_t s) {
  const bool pair = cell_pair_enabled(nk * ca.B, ca.H);
  if (o.gi_b) return pair ? launch_fwd_geo<HAS_G, true, true>(kc, o, nk, W, ca, sw, s) : launch_fwd_geo<HAS_G, false, true>(kc, o, nk, W, ca, sw, s);
  return pair ? launch_fwd_geo<HAS_G, true, false>(kc, o, nk, W, ca, sw, s) : launch_fwd_geo<HAS_G, false, false>(kc, o, nk, W, ca, sw, s);
}

// ---------------------------------------------------------------- epilogues (one output row per thread)
// Each epilogue warp handles 32 rows (its TMEM lane quarter) and one half of the tile's columns.
// Per 16-column chunk the global loads are issued first, then the accumulator is read, so that the
// memory latency of a chunk overlaps its tcgen05.ld and the other warps' work.
__device__ __forceinline__ uint2 pack4(float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<uint32_t*>(&lo);
  o.y = *reinterpret_cast<uint32_t*>(&hi);
  return o;
}
__device__ __forceinline__ float4 unpack4(uint2 v) {
  __nv_bfloat162 lo = *reinterpret_cast<__nv_bfloat162*>(&v.x), hi = *reinterpret_cast<__nv_bfloat162*>(&v.y);
  float2 a = __bfloat1622float2(lo), b = __bfloat1622float2(hi);
  return make_float4(a.x, a.y, b.x, b.y);
}

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
// 32-byte accesses: in these epilogues the lanes of a warp touch 32 different rows, so a 16-byte access uses half
// of each 32-byte sector it moves; one 32-byte access per lane moves whole sectors.
__device__ __forceinline__ void ld8(const float* p, float* v) {
  asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
               : "l"(p));
}
__device__ __forceinline__ void st8(float* p, const float* v) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]),
               "f"(v[5]), "f"(v[6]), "f"(v[7])
               : "memory");
}
__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st4(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ float f4get(const float4& v, int e) { return e == 0 ? v.x : (e == 1 ? v.y : (e == 2 ? v.z : v.w)); }

struct EpiBias {  // out[m, n] = acc + bias[n]      (input projection); outb: optional bf16 copy of the same values; out may be null then
  float* out; i64 ld; const float* bias; int M, N; bf16* outb;
  __device__ void operator()(uint32_t taddr, int row, int n0, int half) const {
    const bool valid = row < M;
    float* o = out + (i64)row * ld + n0;
    const int cbeg = half * 128;
    for (int c0 = cbeg; c0 < cbeg + 128 && n0 + c0 < N; c0 += 16) {
      float v[16];
      tmem_ld16(taddr + c0, v);
      tmem_ld_wait();
      if (valid) {
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
          float4 b = ldg4(bias + n0 + c0 + i);
          v[i] += b.x; v[i + 1] += b.y; v[i + 2] += b.z; v[i + 3] += b.w;
        }
        if (out) {
          st8(o + c0, v);
          st8(o + c0 + 8, v + 8);
        }
        if (outb) {
          const uint2 p0 = pack4(make_float4(v[0], v[1], v[2], v[3])), p1 = pack4(make_float4(v[4], v[5], v[6], v[7]));
          const uint2 p2 = pack4(make_float4(v[8], v[9], v[10], v[11])), p3 = pack4(make_float4(v[12], v[13], v[14], v[15]));
          // sixteen bf16 values = one 32-byte store (a whole sector of this thread's row)
          asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(outb + (i64)row * ld + n0 + c0), "r"(p0.x), "r"(p0.y), "r"(p1.x),
                       "r"(p1.y), "r"(p2.x), "r"(p2.y), "r"(p3.x), "r"(p3.y)
                       : "memory");
        }
      }
    }
  }
};

struct EpiStore {  // out[m, n] = acc            (weight / input gradients)
  static constexpr bool kSplitAware = true;
  float* out; i64 ld; int M, N;
  i64 split_stride;   // split products: range `sp` of the reduction goes to out + sp*split_stride (summed afterwards)
  __device__ void operator()(uint32_t taddr, int row, int n0, int half, int sp) const {
    EpiStore e = *this;
    e.out += (i64)sp * split_stride;
    e(taddr, row, n0, half);
  }
  __device__ void operator()(uint32_t taddr, int row, int n0, int half) const {
    const bool valid = row < M;
    float* o = out + (i64)row * ld + n0;
    const int cbeg = half * 128;
    for (int c0 = cbeg; c0 < cbeg + 128 && n0 + c0 < N; c0 += 16) {
      float v[16];
      tmem_ld16(taddr + c0, v);
      tmem_ld_wait();
      if (valid) {
        st8(o + c0, v);
        st8(o + c0 + 8, v + 8);
      }
    }
  }
};

template <bool FAST = true>
struct EpiFwd {  // GRU cell on the r|z|n accumulator columns of 64 hidden units (FAST: MUFU gate math of the bf16 mode)
  FwdStepArgs a;
  __device__ void operator()(uint32_t taddr, int row, int u0, int half) const {
    const bool valid = row < a.M;
    const int k = valid ? row / a.B : 0, b = valid ? row % a.B : 0;
    const int H = a.H;
    const float* __restrict__ gi = a.gi + (i64)k * a.gi_ks + (i64)b * 3 * H + u0;
    const float* __restrict__ hp = a.hin + (i64)k * a.hin_ks + (i64)b * H + u0;
    float* __restrict__ ho = a.hout + (i64)k * a.hout_ks + (i64)b * H + u0;
    // in mode 1 the previous content of the destination plays the role of the additive term
    const float* __restrict__ ga = a.mode == 1 ? ho : (a.gadd ? a.gadd + (i64)k * a.gadd_ks + (i64)b * H + u0 : nullptr);
    const float* __restrict__ bh = a.b_hh + u0;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      const int c0 = half * 32 + cc * 16;
      float4 gr[4], gz[4], gn[4], h4[4], g4[4];
      if (valid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          gr[i] = ld4(gi + c0 + 4 * i); gz[i] = ld4(gi + H + c0 + 4 * i); gn[i] = ld4(gi + 2 * H + c0 + 4 * i);
          h4[i] = ld4(hp + c0 + 4 * i);
          g4[i] = ga ? ld4(ga + c0 + 4 * i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
      float r[16], z[16], n[16];
      tmem_ld16(taddr + c0, r);
      tmem_ld16(taddr + 64 + c0, z);
      tmem_ld16(taddr + 128 + c0, n);
      tmem_ld_wait();
      if (valid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = c0 + 4 * i;
          float4 br = ldg4(bh + c), bz = ldg4(bh + H + c), bn = ldg4(bh + 2 * H + c);
          float o[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float phi = cell_forward<FAST>(f4get(gr[i], e), f4get(gz[i], e), f4get(gn[i], e), r[4 * i + e] + f4get(br, e),
                                     z[4 * i + e] + f4get(bz, e), n[4 * i + e] + f4get(bn, e), f4get(h4[i], e), a.gamma, a.cell);
            // mode 0: phi + g ;  mode 1: previous - phi
            o[e] = a.mode == 1 ? f4get(g4[i], e) - phi : phi + f4get(g4[i], e);
          }
          st4(ho + c, o[0], o[1], o[2], o[3]);
        }
      }
    }
  }
};

template <bool BF16C = true>
struct EpiLin {  // adjoint coefficients of every step of a level: bf16 mode (MUFU gate math, gate coefficients stored in bf16)
                 // or tf32 modes (precise gate math, fp32 coefficients)
  LinArgs a;
  __device__ void operator()(uint32_t taddr, int row, int u0, int half) const {
    const bool valid = row < a.M;
    const int j1 = valid ? row / a.B : 0, b = valid ? row % a.B : 0;
    const int H = a.H;
    const i64 t = a.t0 + (i64)j1 * a.stride_t;      // fine time the step leaves from
    const float* __restrict__ gi = a.gi + ((t + a.stride_t - 1) * a.B + b) * 3 * H + u0;
    const float* __restrict__ hp = (t == 0 ? a.h0 + (i64)b * H : a.h + ((t - 1) * a.B + b) * H) + u0;
    const i64 o = (i64)row * H + u0;
    const float* __restrict__ bh = a.b_hh + u0;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      const int c0 = half * 32 + cc * 16;
      float4 gr[4], gz[4], gn[4], h4[4];
      if (valid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          gr[i] = ld4(gi + c0 + 4 * i); gz[i] = ld4(gi + H + c0 + 4 * i); gn[i] = ld4(gi + 2 * H + c0 + 4 * i);
          h4[i] = ld4(hp + c0 + 4 * i);
        }
      }
      float r[16], z[16], n[16];
      tmem_ld16(taddr + c0, r);
      tmem_ld16(taddr + 64 + c0, z);
      tmem_ld16(taddr + 128 + c0, n);
      tmem_ld_wait();
      if (valid) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = c0 + 4 * i;
          float4 br = ldg4(bh + c), bz = ldg4(bh + H + c), bn = ldg4(bh + 2 * H + c);
          float oa[4], ocr[4], ocz[4], ocn[4], ocp[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            CellLin L = cell_linearise<BF16C>(f4get(gr[i], e), f4get(gz[i], e), f4get(gn[i], e), r[4 * i + e] + f4get(br, e),
                                       z[4 * i + e] + f4get(bz, e), n[4 * i + e] + f4get(bn, e), f4get(h4[i], e), a.gamma, a.cell);
            oa[e] = L.a; ocr[e] = L.cr; ocz[e] = L.cz; ocn[e] = L.cn; ocp[e] = L.cnp;
          }
          st4(a.a + o + c, oa[0], oa[1], oa[2], oa[3]);
          if constexpr (BF16C) {
            *reinterpret_cast<uint2*>(a.crb + o + c) = pack4(make_float4(ocr[0], ocr[1], ocr[2], ocr[3]));
            *reinterpret_cast<uint2*>(a.czb + o + c) = pack4(make_float4(ocz[0], ocz[1], ocz[2], ocz[3]));
            *reinterpret_cast<uint2*>(a.cnb + o + c) = pack4(make_float4(ocn[0], ocn[1], ocn[2], ocn[3]));
            if (a.cnpb) *reinterpret_cast<uint2*>(a.cnpb + o + c) = pack4(make_float4(ocp[0], ocp[1], ocp[2], ocp[3]));
          } else {
            st4(a.cr + o + c, ocr[0], ocr[1], ocr[2], ocr[3]);
            st4(a.cz + o + c, ocz[0], ocz[1], ocz[2], ocz[3]);
            st4(a.cn + o + c, ocn[0], ocn[1], ocn[2], ocn[3]);
            if (a.cnp) st4(a.cnp + o + c, ocp[0], ocp[1], ocp[2], ocp[3]);
          }
        }
      }
    }
  }
};

template <int BN>
struct EpiAdj {  // lambda_prev = a*lambda + acc (+ source); each epilogue warp half owns BN / 2 columns
  AdjStepArgs a;
  __device__ void operator()(uint32_t taddr, int row, int n0, int half) const {
    const bool valid = row < a.M;
    const int k = valid ? row / a.B : 0, b = valid ? row % a.B : 0;
    const float* __restrict__ li = a.lin + (i64)k * a.lin_ks + (i64)b * a.H + n0;
    const float* __restrict__ ca = a.a + (i64)k * a.coef_ks + (i64)b * a.H + n0;
    float* __restrict__ lo = a.lout + (i64)k * a.lout_ks + (i64)b * a.H + n0;
    const float* __restrict__ ga = a.mode == 1 ? lo : (a.gadd ? a.gadd + (i64)k * a.gadd_ks + (i64)b * a.H + n0 : nullptr);
    const int cbeg = half * (BN / 2), cend = cbeg + BN / 2;
    // The operands of 16 columns come straight from global memory (each lane its own row) and the wait for the
    // accumulator load is a compiler barrier, so the loads of the NEXT 16 columns are issued by hand before the
    // current ones are consumed: two register sets, two column groups per trip.
    auto load = [&](int c0, float* l, float* ac, float* g) {
      if (valid && c0 < cend && n0 + c0 < a.H) {
        ld8(li + c0, l); ld8(li + c0 + 8, l + 8);
        ld8(ca + c0, ac); ld8(ca + c0 + 8, ac + 8);
        if (ga) {
          ld8(ga + c0, g); ld8(ga + c0 + 8, g + 8);
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) g[i] = 0.f;
        }
      }
    };
    auto finish = [&](int c0, const float* l, const float* ac, const float* g) {
      if (n0 + c0 >= a.H) return;          // warp-uniform: the accumulator load is collective
      float v[16];
      tmem_ld16(taddr + c0, v);
      tmem_ld_wait();
      if (valid) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float o = ac[i] * l[i] + v[i];
          v[i] = a.mode == 1 ? g[i] - o : o + g[i];
        }
        st8(lo + c0, v);
        st8(lo + c0 + 8, v + 8);
      }
    };
    float l0[16], a0[16], g0[16], l1[16], a1[16], g1[16];
    load(cbeg, l0, a0, g0);
#pragma unroll 1
    for (int c0 = cbeg; c0 < cend; c0 += 32) {
      load(c0 + 16, l1, a1, g1);
      finish(c0, l0, a0, g0);
      load(c0 + 32, l0, a0, g0);
      finish(c0 + 16, l1, a1, g1);
    }
  }
};

// ---------------------------------------------------------------- operand packing (HBM streams)
constexpr int kPT = 256;
inline int pgrid(i64 items) {
  i64 b = (items + kPT - 1) / kPT, cap = (i64)kSMs * 8;
  return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

__global__ void __launch_bounds__(kPT) convert_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, i64 n4) {
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (i64)gridDim.x * blockDim.x) dst[e] = pack4(src[e]);
}

// dst[m, :] = bf16(src row (k, b)),  m = k*B + b
__global__ void __launch_bounds__(kPT) pack_rows_kernel(const float* __restrict__ src, i64 ks, int B, int H4, i64 M,
                                                        uint2* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  i64 total = M * H4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / H4; int c = (int)(e % H4);
    i64 k = m / B; int b = (int)(m % B);
    dst[e] = pack4(*reinterpret_cast<const float4*>(src + k * ks + ((i64)b * H4 + c) * 4));
  }
}

// dst[m, g*H + i] = bf16(c_g[m, i] * lam[m, i])
__global__ void __launch_bounds__(kPT) pack_adj_kernel(const float* __restrict__ lin, i64 lin_ks, const bf16* __restrict__ cr,
                                                       const bf16* __restrict__ cz, const bf16* __restrict__ cn, i64 coef_ks,
                                                       int B, int H4, i64 M, uint2* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  i64 total = M * H4;
  // L2 hints: the packed operand is read back at once by the product (keep it), the coefficients are dead after this pass
  uint64_t keep, drop;
  asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
  asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(drop));
  auto ldc = [&](const bf16* p) { uint2 v; asm volatile("ld.global.L2::cache_hint.v2.b32 {%0,%1}, [%2], %3;" : "=r"(v.x), "=r"(v.y) : "l"(p), "l"(drop)); return v; };
  auto stk = [&](uint2* p, uint2 v) { asm volatile("st.global.L2::cache_hint.v2.b32 [%0], {%1,%2}, %3;" ::"l"(p), "r"(v.x), "r"(v.y), "l"(keep) : "memory"); };
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / H4; int c = (int)(e % H4);
    i64 k = m / B; int b = (int)(m % B);
    i64 ro = ((i64)b * H4 + c) * 4;
    float4 l = *reinterpret_cast<const float4*>(lin + k * lin_ks + ro);
    float4 r = unpack4(ldc(cr + k * coef_ks + ro));
    float4 z = unpack4(ldc(cz + k * coef_ks + ro));
    float4 n = unpack4(ldc(cn + k * coef_ks + ro));
    i64 o = m * 3 * H4 + c;
    stk(dst + o, pack4(make_float4(r.x * l.x, r.y * l.y, r.z * l.z, r.w * l.w)));
    stk(dst + o + H4, pack4(make_float4(z.x * l.x, z.y * l.y, z.z * l.z, z.w * l.w)));
    stk(dst + o + 2 * H4, pack4(make_float4(n.x * l.x, n.y * l.y, n.z * l.z, n.w * l.w)));
  }
}

// dst[c * dst_ld + col0 + r] = bf16(src[r * C + c]),  src [R, C] fp32
__global__ void __launch_bounds__(1024) transpose_kernel(const float* __restrict__ src, i64 R, int C, bf16* __restrict__ dst,
                                                         i64 dst_ld, i64 col0) {
  __shared__ float tile[32][33];
  i64 r0 = (i64)blockIdx.x * 32; int c0 = blockIdx.y * 32;
  i64 r = r0 + threadIdx.y; int c = c0 + threadIdx.x;
  tile[threadIdx.y][threadIdx.x] = (r < R && c < C) ? src[r * C + c] : 0.f;
  __syncthreads();
  i64 rr = r0 + threadIdx.x; int cc = c0 + threadIdx.y;
  if (rr < R && cc < C) dst[(i64)cc * dst_ld + col0 + rr] = __float2bfloat16(tile[threadIdx.x][threadIdx.y]);
}

// Gradient-pass operands, row-major: dA_h = [cr|cz|cn]*lam and dA_i = [cr|cz|cnp]*lam as bf16 [M, 3H], plus this
// block's fp32 column sums of the four products (bias-gradient partials) to part[blockIdx.x][4][H].
// Row m = (t, b): lam row at lam + t*lam_ts + b*H (lam_ts may be negative: the adjoint keeps its unknowns in
// reversed time order).  Block = 32 float4 columns (128 units) x 8 rows at a time.
__global__ void __launch_bounds__(256) form_dA_rows_kernel(const float* __restrict__ lam, i64 lam_ts, int B, const bf16* __restrict__ cr,
                                                           const bf16* __restrict__ cz, const bf16* __restrict__ cn,
                                                           const bf16* __restrict__ cnp, i64 M, int H, uint2* __restrict__ dA4,
                                                           float* __restrict__ part, int rows_per_block) {
  __shared__ float red[4][8][128];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int H4 = H / 4, c4 = blockIdx.y * 32 + tx;
  const i64 m0 = (i64)blockIdx.x * rows_per_block;
  float4 s[4];
#pragma unroll
  for (int g = 0; g < 4; ++g) s[g] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c4 < H4) {
    for (i64 m = m0 + ty; m < m0 + rows_per_block && m < M; m += 8) {
      i64 e = m * H4 + c4;
      const int t = (int)m / B, bb = (int)m - t * B;       // row counts fit 32 bits (checked by the host)
      float4 l = *reinterpret_cast<const float4*>(lam + (i64)t * lam_ts + ((i64)bb * H4 + c4) * 4);
      float4 r = unpack4(reinterpret_cast<const uint2*>(cr)[e]), z = unpack4(reinterpret_cast<const uint2*>(cz)[e]);
      float4 n = unpack4(reinterpret_cast<const uint2*>(cn)[e]), q = unpack4(reinterpret_cast<const uint2*>(cnp)[e]);
      float4 v[4] = {make_float4(r.x * l.x, r.y * l.y, r.z * l.z, r.w * l.w), make_float4(z.x * l.x, z.y * l.y, z.z * l.z, z.w * l.w),
                     make_float4(n.x * l.x, n.y * l.y, n.z * l.z, n.w * l.w), make_float4(q.x * l.x, q.y * l.y, q.z * l.z, q.w * l.w)};
      i64 o = m * 4 * H4 + c4;
#pragma unroll
      for (int g = 0; g < 4; ++g) dA4[o + g * H4] = pack4(v[g]);
#pragma unroll
      for (int g = 0; g < 4; ++g) { s[g].x += v[g].x; s[g].y += v[g].y; s[g].z += v[g].z; s[g].w += v[g].w; }
    }
  }
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    red[g][ty][tx * 4] = s[g].x; red[g][ty][tx * 4 + 1] = s[g].y; red[g][ty][tx * 4 + 2] = s[g].z; red[g][ty][tx * 4 + 3] = s[g].w;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 4 * 128; e += 256) {
    int g = e / 128, u = e % 128, col = blockIdx.y * 128 + u;
    if (col >= H) continue;
    float acc = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) acc += red[g][r][u];
    part[((i64)blockIdx.x * 4 + g) * H + col] = acc;
  }
}

// Bias gradients from the per-block partials, summed in block order (the same bits on every run):
// db_hh = [sum cr*lam | sum cz*lam | sum cn*lam],  db_ih = [sum cr*lam | sum cz*lam | sum cnp*lam].
__global__ void __launch_bounds__(kPT) sum_db_kernel(const float* __restrict__ part, int nblk, int H, float* __restrict__ db_hh,
                                                     float* __restrict__ db_ih) {
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < 4 * H; e += gridDim.x * blockDim.x) {
    const int g = e / H, col = e % H;
    float acc = 0.f;
    for (int k = 0; k < nblk; ++k) acc += part[((i64)k * 4 + g) * H + col];
    if (g == 0) { db_hh[col] = acc; db_ih[col] = acc; }
    else if (g == 1) { db_hh[H + col] = acc; db_ih[H + col] = acc; }
    else if (g == 2) db_hh[2 * H + col] = acc;
    else db_ih[2 * H + col] = acc;
  }
}

void convert(const float* src, bf16* dst, i64 n, cudaStream_t s) {
  convert_kernel<<<pgrid(n / 4), kPT, 0, s>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(dst), n / 4);
  count_launch();
}
void transpose(const float* src, i64 R, int C, bf16* dst, i64 dst_ld, i64 col0, cudaStream_t s) {
  if (R <= 0) return;
  transpose_kernel<<<dim3((unsigned)((R + 31) / 32), (C + 31) / 32), dim3(32, 32), 0, s>>>(src, R, C, dst, dst_ld, col0);
  count_launch();
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
template <class T> T* take(char* base, size_t* off, size_t n) {
  T* p = base ? reinterpret_cast<T*>(base + *off) : nullptr;
  *off += round_up(n * sizeof(T), 256);
  return p;
}
size_t max_step_rows(const mgrit_gru_cfg* c, const int* N, int L) {
  size_t m = (size_t)c->B;
  for (int l = 0; l + 1 < L; ++l) {
    size_t r = (size_t)((N[l] + c->cf - 1) / c->cf) * c->B;   // relaxation (a ragged level has one more interval) / residual / FAS rows
    if (r > m) m = r;
  }
  return m;
}

}  // namespace

int umma_supported(const mgrit_gru_cfg* c) {
  if (c->H % 64 != 0 || c->I % 16 != 0 || ((i64)c->T * c->B) % 8 != 0) return MGRIT_UNSUPPORTED;
  return MGRIT_OK;
}

void umma_plan_fwd(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, UmmaFwdWs* o) {
  o->maxM = max_step_rows(c, N, L);
  o->W_hh = take<bf16>(base, off, (size_t)3 * c->H * c->H);
  o->W_ih = take<bf16>(base, off, (size_t)3 * c->H * c->I);
  o->xb = take<bf16>(base, off, (size_t)c->T * c->B * c->I);
  o->Apack = take<bf16>(base, off, o->maxM * c->H);
  o->gib = take<bf16>(base, off, (size_t)c->T * c->B * 3 * c->H);
}

void umma_plan_adj(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, UmmaAdjWs* o) {
  size_t TB = (size_t)c->T * c->B, H = c->H, I = c->I;
  o->maxM = max_step_rows(c, N, L);
  o->W_hh = take<bf16>(base, off, 3 * H * H);
  o->W_hhT = take<bf16>(base, off, 3 * H * H);
  o->W_ihT = take<bf16>(base, off, 3 * H * I);
  size_t apack = o->maxM * 3 * H;
  if (TB * H > apack) apack = TB * H;     // the linearisation packs all T*B rows of a level at once
  o->Apack = take<bf16>(base, off, apack);
  o->apack_elems = apack;
  o->dA4 = take<bf16>(base, off, 4 * H * TB);
  o->xb = take<bf16>(base, off, I * TB);
  o->hb0 = take<bf16>(base, off, (size_t)c->B * H + TB * H);   // [h_0; h] contiguous: rows (t, b) of h_{t-1} start at hb0
  o->hb = o->hb0 ? o->hb0 + (size_t)c->B * H : nullptr;
  o->gib = nullptr;
}

int umma_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, UmmaFwdWs* w, cudaStream_t s) {
  const int H = c->H, I = c->I;
  const i64 TB = (i64)c->T * c->B;
  convert(p->W_hh, w->W_hh, (i64)3 * H * H, s);
  convert(p->W_ih, w->W_ih, (i64)3 * H * I, s);
  convert(x, w->xb, TB * I, s);
  // gi = x W_ih^T + b_ih :  M = T*B, N = 3H, K = I
  if (gemm_pair_enabled((int)TB, 3 * H)
          ? !launch_gemm_pair(KC_PROJ, w->xb, I, w->W_ih, I, (int)TB, 3 * H, I, 3 * H, EpiBias{gi, 3 * H, p->b_ih, (int)TB, 3 * H, w->gib}, s)
          : !launch_gemm<256, 0>(KC_PROJ, w->xb, I, w->W_ih, I, (int)TB, 3 * H, I, 0, 3 * H, EpiBias{gi, 3 * H, p->b_ih, (int)TB, 3 * H, w->gib}, s))
    return MGRIT_CUDA_ERROR;
  return MGRIT_OK;
}

int umma_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, const float* h0, const float* h, UmmaAdjWs* w, bool have_hb,
                     cudaStream_t s) {
  const int H = c->H, I = c->I;
  convert(p->W_hh, w->W_hh, (i64)3 * H * H, s);
  if (!have_hb) {      // otherwise w->hb0 already points at the forward call's bf16 copy of [h_0; h]
    convert(h0, w->hb0, (i64)c->B * H, s);
    convert(h, w->hb, (i64)c->T * c->B * H, s);
  }
  transpose(p->W_hh, 3 * H, H, w->W_hhT, 3 * H, 0, s);   // [H, 3H]
  transpose(p->W_ih, 3 * H, I, w->W_ihT, 3 * H, 0, s);   // [I, 3H]
  return status_ptr() ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int umma_fwd_step(const FwdStepArgs& a, UmmaFwdWs* w, cudaStream_t s) {
  bool ok;
  if (a.hin_b && 128 % a.B == 0) {
    // operands through strided tensor maps, bf16 copy of the new state written by the epilogue
    CellArgs ca{};
    ca.B = a.B; ca.H = a.H; ca.b_hh = a.b_hh; ca.gamma = a.gamma; ca.cell = a.cell; ca.mode = a.mode;
    const int nk = a.M / a.B;
    SweepArgs sw{};
    sw.n_steps = 1;
    sw.st[0].hout = a.hout; sw.st[0].hout_ks = a.hout_ks; sw.st[0].hout_b = a.hout_b;
    CellFwdOperands o{};
    o.A = a.hin_b; o.hp = a.hin; o.in_ks = a.hin_ks; o.in_slots = 1;
    o.gi = a.gi; o.gi_b = a.gi_b; o.gi_ks = a.gi_ks; o.tgt_slots = 1;
    // in mode 1 the previous content of the destination plays the role of the additive term
    if (a.mode == 1) { o.g = a.hout; o.g_ks = a.hout_ks; }
    else { o.g = a.gadd; o.g_ks = a.gadd_ks; }
    ok = o.g ? launch_fwd<true>(KC_FWD_STEP, o, nk, w->W_hh, ca, sw, s) : launch_fwd<false>(KC_FWD_STEP, o, nk, w->W_hh, ca, sw, s);
    return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
  }
  if (launch_pdl(pack_rows_kernel, dim3(pgrid((i64)a.M * (a.H / 4))), dim3(kPT), 0, s, a.hin, a.hin_ks, a.B, a.H / 4, (i64)a.M,
                 reinterpret_cast<uint2*>(w->Apack)) != cudaSuccess)
    return MGRIT_CUDA_ERROR;
  count_launch();
  ok = launch_gemm<192, 3>(KC_FWD_STEP, w->Apack, a.H, w->W_hh, a.H, a.M, a.H, a.H, a.H, 3 * a.H, EpiFwd<true>{a}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// MGRIT_GRU_SWEEP=0 in the environment launches every relaxation step on its own.
static bool sweep_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_SWEEP"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

int umma_fwd_sweep(const FwdSweepArgs& a, UmmaFwdWs* w, cudaStream_t s) {
  if (!sweep_enabled() || 128 % a.B != 0 || !a.Ub || a.n < 1 || a.n > kMaxSweepSteps || a.n > kMaxFwdSweepSteps || !a.ctr)
    return MGRIT_UNSUPPORTED;
  const i64 BH = (i64)a.B * a.H;
  CellArgs ca{};
  ca.B = a.B; ca.H = a.H; ca.b_hh = a.b_hh; ca.gamma = a.gamma; ca.cell = a.cell; ca.mode = 0;
  SweepArgs sw{};
  sw.n_steps = a.n; sw.ctr = a.ctr;
  for (int i = 0; i < a.n; ++i) {
    sw.st[i].hout = a.st[i].out; sw.st[i].hout_ks = a.st[i].out_ks; sw.st[i].hout_b = a.st[i].out_b;
    sw.st[i].in_s = a.st[i].in_s; sw.st[i].tgt_s = a.st[i].tgt_s; sw.st[i].dep = i == 0 ? 0 : a.st[i].dep;
  }
  CellFwdOperands o{};
  o.A = a.Ub; o.hp = a.U; o.in_ss = BH; o.in_ks = (i64)a.cf * BH; o.in_slots = a.cf;
  o.gi = a.gi; o.gi_b = a.gi_b; o.gi_ss = a.gi_ss; o.gi_ks = a.gi_ks; o.tgt_slots = a.cf;
  o.g = a.g; o.g_ss = BH; o.g_ks = (i64)a.cf * BH;
  const bool ok = a.g ? launch_fwd<true>(KC_FWD_STEP, o, a.nk, w->W_hh, ca, sw, s) : launch_fwd<false>(KC_FWD_STEP, o, a.nk, w->W_hh, ca, sw, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int umma_linearise(const LinArgs& a, UmmaAdjWs* w, cudaStream_t s) {
  // rows (j-1, b): state entering forward step j of the level = h at fine time t0 + stride*(j-1); w->hb0 holds the
  // bf16 copy of [h_0; h], so fine time t is its slot t, and in fp32 time t >= 1 is slot t - 1 of h
  const i64 BH = (i64)a.B * a.H;
  const int N = a.M / a.B;
  const float* gi0 = a.gi + (a.t0 + a.stride_t - 1) * BH * 3;       // input of the fine step that arrives with step 1
  const bf16* gib0 = a.gi_b ? a.gi_b + (a.t0 + a.stride_t - 1) * BH * 3 : nullptr;   // ... in the bf16 copy
  if (128 % a.B == 0) {
    CellArgs ca{};
    ca.B = a.B; ca.H = a.H; ca.b_hh = a.b_hh; ca.gamma = a.gamma; ca.cell = a.cell;
    ca.a = a.a; ca.cr = a.crb; ca.cz = a.czb; ca.cn = a.cnb; ca.cnp = a.cnpb;
    int done = 0;
    // step 1 starts from h_0: a launch of its own, unless the caller keeps h_0 in the slot in front of h (the layout
    // of MGRIT_FLAG_H_LEADS_WITH_H0) -- then rows (t - 1) of h are valid for t = 0 as well
    if (a.t0 == 0 && a.h0 + BH != a.h) {
      if (!launch_lin(KC_LINEARISE, w->hb0, 0, gib0 ? (const void*)gib0 : (const void*)gi0, gib0 != nullptr, 0, a.h0, 0, 1, w->W_hh, ca, s))
        return MGRIT_CUDA_ERROR;
      done = 1;
    }
    if (N > done) {
      const i64 off = (i64)done * BH;
      ca.a = a.a + off; ca.cr = a.crb + off; ca.cz = a.czb + off; ca.cn = a.cnb + off; ca.cnp = a.cnpb ? a.cnpb + off : nullptr;
      const i64 t1 = a.t0 + (i64)done * a.stride_t;                  // fine time the first of these steps leaves from (>= 1)
      const i64 goff = (i64)done * a.stride_t * BH * 3;
      if (!launch_lin(KC_LINEARISE, w->hb0 + t1 * BH, a.stride_t * BH, gib0 ? (const void*)(gib0 + goff) : (const void*)(gi0 + goff),
                      gib0 != nullptr, a.stride_t * BH * 3, a.h + (t1 - 1) * BH, a.stride_t * BH, N - done, w->W_hh, ca, s))
        return MGRIT_CUDA_ERROR;
    }
    return MGRIT_OK;
  }
  int done = 0;
  if (a.t0 == 0) {
    if (launch_pdl(pack_rows_kernel, dim3(pgrid((i64)a.B * (a.H / 4))), dim3(kPT), 0, s, a.h0, (i64)0, a.B, a.H / 4, (i64)a.B,
                   reinterpret_cast<uint2*>(w->Apack)) != cudaSuccess)
      return MGRIT_CUDA_ERROR;
    count_launch();
    done = 1;
  }
  if (N > done) {
    const i64 t1 = a.t0 + (i64)done * a.stride_t;
    if (launch_pdl(pack_rows_kernel, dim3(pgrid((i64)(N - done) * a.B * (a.H / 4))), dim3(kPT), 0, s, a.h + (t1 - 1) * BH,
                   (i64)(a.stride_t * BH), a.B, a.H / 4, (i64)(N - done) * a.B, reinterpret_cast<uint2*>(w->Apack + (i64)done * BH)) != cudaSuccess)
      return MGRIT_CUDA_ERROR;
    count_launch();
  }
  return launch_gemm<192, 3>(KC_LINEARISE, w->Apack, a.H, w->W_hh, a.H, a.M, a.H, a.H, a.H, 3 * a.H, EpiLin<true>{a}, s) ? MGRIT_OK
                                                                                                                      : MGRIT_CUDA_ERROR;
}

// MGRIT_GRU_ADJ_STAGED=0 in the environment keeps every adjoint product on the plain GEMM with global-load epilogue.
static bool adj_staged_enabled() {
  static int v = -1;
  if (v < 0) { const char* e = getenv("MGRIT_GRU_ADJ_STAGED"); v = (e && e[0] == '0') ? 0 : 1; }
  return v == 1;
}

// The adjoint product with TMA-staged epilogue operands (rows (k, b), 128 % B == 0).
template <bool HAS_G, bool PAIR>
static bool launch_adj_staged(const AdjStepArgs& a, const bf16* Apack, const bf16* W_hhT, const float* g, i64 g_ks, cudaStream_t s) {
  using C = adjk::ACfg<HAS_G, PAIR>;
  int* const status = status_ptr();
  if (!status) return false;
  static bool attr_set[kMaxDevices] = {false};
  auto kern = umma_adj_kernel<HAS_G, PAIR>;
  if (!set_smem_once(kern, C::kSmemBytes, attr_set)) return false;
  const int B = a.B, H = a.H, kt = 128 / B, nk = a.M / B, K = 3 * H;
  AdjKArgs ka{};
  ka.M = a.M; ka.B = B; ka.H = H; ka.kt = kt; ka.nk = nk; ka.lout = a.lout; ka.lout_ks = a.lout_ks; ka.mode = a.mode;
  ka.a_rev = (a.coef_ks < 0 && nk > 1) ? 1 : 0;
  CUtensorMap ta, tb, tl, tca, tg;
  if (!make_map(&ta, Apack, (uint64_t)K, (uint64_t)a.M, (uint64_t)K, BM)) return false;
  if (!make_map(&tb, W_hhT, (uint64_t)K, (uint64_t)H, (uint64_t)K, PAIR ? adjk::ABN / 2 : adjk::ABN)) return false;
  const auto f32 = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  if (!make_map3(&tl, f32, 4, a.lin, H, B, nk, H, a.lin_ks, adjk::ACH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  const float* abase = ka.a_rev ? a.a + (i64)(nk - 1) * a.coef_ks : a.a;      // lowest address when the rows run backwards
  if (!make_map3(&tca, f32, 4, abase, H, B, nk, H, ka.a_rev ? -a.coef_ks : a.coef_ks, adjk::ACH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  if (HAS_G) {
    if (!make_map3(&tg, f32, 4, g, H, B, nk, H, g_ks, adjk::ACH, kt, CU_TENSOR_MAP_SWIZZLE_64B)) return false;
  } else {
    tg = tl;
  }
  constexpr int kTileRows = PAIR ? 2 * BM : BM;
  const int tiles = ((a.M + kTileRows - 1) / kTileRows) * ((H + adjk::ABN - 1) / adjk::ABN);
  cudaError_t e;
  if (PAIR) {
    const int grid = 2 * (tiles < kSMs / 2 ? tiles : kSMs / 2);
    e = launch_pdl_cluster(kern, 2, dim3(grid), dim3(adjk::kAdjThreads), C::kSmemBytes, s, ta, tb, tl, tca, tg, ka, K, status);
  } else {
    const int grid = tiles < kSMs ? tiles : kSMs;
    e = launch_pdl(kern, dim3(grid), dim3(adjk::kAdjThreads), C::kSmemBytes, s, ta, tb, tl, tca, tg, ka, K, status);
  }
  if (e != cudaSuccess) return false;
  count_launch();
  return true;
}

int umma_adj_step(const AdjStepArgs& a, UmmaAdjWs* w, cudaStream_t s) {
  ProfScope prof(KC_ADJ_STEP, 2.0 * a.M * 3.0 * a.H * a.H, s);     // operand packing + product, timed together
  if (launch_pdl(pack_adj_kernel, dim3(pgrid((i64)a.M * (a.H / 4))), dim3(kPT), 0, s, a.lin, a.lin_ks, a.crb, a.czb, a.cnb, a.coef_ks,
                 a.B, a.H / 4, (i64)a.M, reinterpret_cast<uint2*>(w->Apack)) != cudaSuccess)
    return MGRIT_CUDA_ERROR;
  count_launch();
  // Few-row launches (coarse levels, short prefixes) cannot fill the SMs with 256-column tiles and are
  // bound by one CTA streaming all of K; 64-column tiles spread that stream over four times the CTAs.
  const int tiles256 = ((a.M + BM - 1) / BM) * ((a.H + 255) / 256);
  bool ok;
  // strides of the staged operands: positive for the sensitivities, any sign for the coefficient rows
  const bool staged = adj_staged_enabled() && 128 % a.B == 0 && tiles256 * 2 > kSMs && a.lin_ks > 0 && a.lout_ks > 0 &&
                      (a.mode == 1 || !a.gadd || a.gadd_ks > 0);
  if (staged) {
    const float* g = a.mode == 1 ? a.lout : a.gadd;
    const i64 g_ks = a.mode == 1 ? a.lout_ks : a.gadd_ks;
    const bool pair = gemm_pair_enabled(a.M, a.H);
    if (g) ok = pair ? launch_adj_staged<true, true>(a, w->Apack, w->W_hhT, g, g_ks, s) : launch_adj_staged<true, false>(a, w->Apack, w->W_hhT, g, g_ks, s);
    else ok = pair ? launch_adj_staged<false, true>(a, w->Apack, w->W_hhT, nullptr, 0, s) : launch_adj_staged<false, false>(a, w->Apack, w->W_hhT, nullptr, 0, s);
    return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
  }
  if (tiles256 * 2 <= kSMs)
    ok = launch_gemm<64, 0>(KC_ADJ_STEP, w->Apack, 3 * a.H, w->W_hhT, 3 * a.H, a.M, a.H, 3 * a.H, 0, a.H, EpiAdj<64>{a}, s);
  else if (gemm_pair_enabled(a.M, a.H))
    ok = launch_gemm_pair(KC_ADJ_STEP, w->Apack, 3 * a.H, w->W_hhT, 3 * a.H, a.M, a.H, 3 * a.H, a.H, EpiAdj<256>{a}, s);
  else
    ok = launch_gemm<256, 0>(KC_ADJ_STEP, w->Apack, 3 * a.H, w->W_hhT, 3 * a.H, a.M, a.H, 3 * a.H, 0, a.H, EpiAdj<256>{a}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// dst[e] = sum over the `splits` partial products (float4 stream)
__global__ void __launch_bounds__(kPT) sum_splits_kernel(const float4* __restrict__ part, i64 n4, int splits, float4* __restrict__ dst) {
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (i64)gridDim.x * blockDim.x) {
    float4 a = part[e];
    for (int sp = 1; sp < splits; ++sp) {
      float4 b = part[(i64)sp * n4 + e];
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    dst[e] = a;
  }
}

// A weight-gradient product has few output tiles (3H/128 x cols/256) and a very long reduction (T*B): with fewer
// tiles than SMs, or a ragged last wave, the reduction is cut into up to four ranges so that the (tile, range)
// items fill the SMs; the partial products go to `scratch` (scratch_bytes available) and are summed afterwards.
static int pick_splits(int Mdim, int Ndim, int K, size_t scratch_bytes) {
  const int tiles = ((Mdim + BM - 1) / BM) * ((Ndim + 255) / 256), k_blocks = (K + BK - 1) / BK;
  int best = 1; double best_eff = 0.0;
  for (int sp = 1; sp <= 4; ++sp) {
    if (sp > 1 && ((size_t)sp * Mdim * Ndim * sizeof(float) > scratch_bytes || k_blocks / sp < 32)) break;
    const int items = tiles * sp, waves = (items + kSMs - 1) / kSMs;
    const double eff = (double)items / ((double)waves * kSMs);
    if (eff > best_eff + 0.05) { best_eff = eff; best = sp; }
  }
  return best;
}

template <class OutT>
// (a_ld > 0: dA is a column selection of a wider array with a_ld columns -- the first a_from columns and, when a_add != 0,
// the columns behind a gap of a_add)
static bool wgrad_gemm(const bf16* dA, int H3, const bf16* R, int cols, int K, OutT* out, float* scratch, size_t scratch_bytes,
                       cudaStream_t s, int a_ld = 0, int a_from = 0, int a_add = 0) {
  const int splits = (((i64)H3 * cols) % 4 == 0) ? pick_splits(H3, cols, K, scratch_bytes) : 1;
  const i64 lda = a_ld > 0 ? a_ld : H3;
  if (splits == 1)
    return launch_gemm_mn(KC_WGRAD, dA, lda, H3, R, cols, cols, K, 1, EpiStore{out, cols, H3, cols, 0}, s, a_ld, a_from, a_add);
  const i64 n = (i64)H3 * cols;
  if (!launch_gemm_mn(KC_WGRAD, dA, lda, H3, R, cols, cols, K, splits, EpiStore{scratch, cols, H3, cols, n}, s, a_ld, a_from, a_add)) return false;
  sum_splits_kernel<<<pgrid(n / 4), kPT, 0, s>>>(reinterpret_cast<const float4*>(scratch), n / 4, splits, reinterpret_cast<float4*>(out));
  count_launch();
  return true;
}

int umma_gradients(const mgrit_gru_cfg* c, const gru_params* p, const float* x, const float* h0, const float* h, const float* lam,
                   i64 lam_ts, const bf16* cr, const bf16* cz, const bf16* cn, const bf16* cnp, float* dx, const gru_grads* g,
                   UmmaAdjWs* w, bool have_xb, cudaStream_t s) {
  (void)h0; (void)h;
  const int H = c->H, I = c->I, B = c->B;
  const i64 M = (i64)c->T * B;
  // one timing record for the whole pass: operand forming, bias sums, the three products and their split sums
  ProfScope prof(KC_WGRAD, 2.0 * M * 3.0 * H * ((double)H + I + (dx ? I : 0)), s);
  // operands of the three gradient GEMMs, all row-major (the reduction index t,b is the row index)
  // dA4 [M, 4H] = [cr | cz | cn | cn'] * lambda: the operand of the recurrent-weight gradient is its first three column
  // blocks, that of the input-weight gradient and of dx its blocks 0, 1 and 3 (the products skip block 2)
  bf16* dA4 = w->dA4;
  const int rows_per_block = 256;
  // (the step operand buffer is free during the gradient pass: scratch for the bias partials, then for the split
  // partial products of the weight-gradient GEMMs; M >= 8 makes nblk*16H <= 2MH bytes)
  float* scratch = reinterpret_cast<float*>(w->Apack);
  const size_t scratch_bytes = w->apack_elems * sizeof(bf16);
  dim3 grid((unsigned)((M + rows_per_block - 1) / rows_per_block), (H / 4 + 31) / 32);
  if ((size_t)grid.x * 4 * H * sizeof(float) > scratch_bytes) return MGRIT_UNSUPPORTED;
  form_dA_rows_kernel<<<grid, 256, 0, s>>>(lam, lam_ts, B, cr, cz, cn, cnp, M, H, reinterpret_cast<uint2*>(dA4), scratch, rows_per_block);
  sum_db_kernel<<<pgrid(4 * H), kPT, 0, s>>>(scratch, (int)grid.x, H, g->db_hh, g->db_ih);
  count_launch(2);
  if (!have_xb) convert(x, w->xb, M * I, s);     // x as bf16 [M, I]; h_{t-1} as bf16 = [h_0; h] without its last slot (w->hb0)
  bool ok = true;
  // dW_hh[3H, H] = dA_h^T h_prev ;  dW_ih[3H, I] = dA_i^T x    (K = T*B, MN-major operands)
  ok = ok && wgrad_gemm(dA4, 3 * H, w->hb0, H, (int)M, g->dW_hh, scratch, scratch_bytes, s, 4 * H, 3 * H, 0);
  ok = ok && wgrad_gemm(dA4, 3 * H, w->xb, I, (int)M, g->dW_ih, scratch, scratch_bytes, s, 4 * H, 2 * H, H);
  // dx[T*B, I] = dA_i W_ih   (K = 3H, K-major operands)
  if (dx)
    ok = ok && (gemm_pair_enabled((int)M, I)
                    ? launch_gemm_pair(KC_WGRAD, dA4, 4 * H, w->W_ihT, 3 * H, (int)M, I, 3 * H, I, EpiStore{dx, I, (int)M, I, 0}, s, false, 4 * H,
                                       2 * H, H)
                    : launch_gemm<256, 0>(KC_WGRAD, dA4, 4 * H, w->W_ihT, 3 * H, (int)M, I, 3 * H, 0, I, EpiStore{dx, I, (int)M, I, 0}, s, 1,
                                          false, 4 * H, 2 * H, H));
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

void umma_convert(const float* src, __nv_bfloat16* dst, i64 n, cudaStream_t s) { convert(src, dst, n, s); }

// out[M, 3H] = X[M, K] W^T + bias with X fp32 contiguous (converted into xb first) and W already bf16 [3H, K]
int umma_project_rows(const float* X, bf16* xb, const bf16* Wb, const float* bias, float* out, int M, int K, int H3, cudaStream_t s) {
  convert(X, xb, (i64)M * K, s);
  return launch_gemm<256, 0>(KC_PROJ, xb, K, Wb, K, M, H3, K, 0, H3, EpiBias{out, H3, bias, M, H3}, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// out[M, C] = ([cr|cz|cn]*lam of the step `a`) W_ihT^T: the sensitivity a cell sends to its input (a.cnb holding c_n')
int umma_adj_dx(const AdjStepArgs& a, const bf16* W_ihT, int C, float* out, UmmaAdjWs* w, cudaStream_t s) {
  if (launch_pdl(pack_adj_kernel, dim3(pgrid((i64)a.M * (a.H / 4))), dim3(kPT), 0, s, a.lin, a.lin_ks, a.crb, a.czb, a.cnb, a.coef_ks,
                 a.B, a.H / 4, (i64)a.M, reinterpret_cast<uint2*>(w->Apack)) != cudaSuccess)
    return MGRIT_CUDA_ERROR;
  count_launch();
  return launch_gemm<256, 0>(KC_ADJ_STEP, w->Apack, 3 * a.H, W_ihT, 3 * a.H, a.M, C, 3 * a.H, 0, C, EpiStore{out, C, a.M, C, 0}, s)
             ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// ======================================================================================================
// TF32 operand modes: the same persistent tcgen05 GEMM with `.kind::tf32`, fp32 state, fp32 coefficients, the
// row-per-thread epilogues above.  A tf32 value keeps 10 mantissa bits, so one product x*w is good to about 1e-3
// relative.  MGRIT_OPERANDS_TF32 therefore runs every product as the three-term split
//     x w  ~=  x_hi w_hi + x_lo w_hi + x_hi w_lo,     x_hi = tf32(x), x_lo = tf32(x - x_hi)   (the dropped term is 2^-22),
// laid out as ONE product over a three times longer reduction: the operand-forming kernels write A' = [hi | lo | hi] and
// B' = [hi | hi | lo] along K, and the GEMM kernel does not know.  MGRIT_OPERANDS_TF32_1PASS writes only tf32(x).
namespace {

__device__ __forceinline__ float tf32_rna(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
// segment `seg` (0..S-1) of the split of x for an A-side (roleB = false: hi, lo, hi) or B-side (hi, hi, lo) operand
__device__ __forceinline__ float split_part(float x, int seg, bool roleB) {
  const float hi = tf32_rna(x);
  const bool want_lo = roleB ? (seg == 2) : (seg == 1);
  return want_lo ? tf32_rna(x - hi) : hi;
}

// dst[m, seg*K + c] = split(src row (k, b))[c],  m = k*B + b, rows of K floats
__global__ void __launch_bounds__(kPT) split_rows_kernel(const float* __restrict__ src, i64 ks, int B, int K, i64 M, int S, int roleB,
                                                         float* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  const i64 total = M * K;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 m = e / K; const int c = (int)(e % K);
    const i64 k = m / B; const int b = (int)(m % B);
    const float x = src[k * ks + (i64)b * K + c];
    for (int seg = 0; seg < S; ++seg) dst[m * S * K + (i64)seg * K + c] = split_part(x, seg, roleB != 0);
  }
}

// dst[m, seg*3H + g*H + i] = split(c_g[m, i] * lam[m, i])   (A side)
__global__ void __launch_bounds__(kPT) split_adj_kernel(const float* __restrict__ lin, i64 lin_ks, const float* __restrict__ cr,
                                                        const float* __restrict__ cz, const float* __restrict__ cn, i64 coef_ks, int B,
                                                        int H, i64 M, int S, float* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  const i64 total = M * H;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 m = e / H; const int i = (int)(e % H);
    const i64 k = m / B; const int b = (int)(m % B);
    const i64 ro = (i64)b * H + i;
    const float l = lin[k * lin_ks + ro];
    const float v[3] = {cr[k * coef_ks + ro] * l, cz[k * coef_ks + ro] * l, cn[k * coef_ks + ro] * l};
    for (int seg = 0; seg < S; ++seg)
#pragma unroll
      for (int g = 0; g < 3; ++g) dst[m * S * 3 * H + (i64)seg * 3 * H + g * H + i] = split_part(v[g], seg, false);
  }
}

// dst[c, seg*R + r] = split(src row r)[c]; src rows: r < Rfirst ? first + r*C : rest + (r - Rfirst)*C   ([R, C] -> [C, S*R])
__global__ void __launch_bounds__(1024) transpose_split_kernel(const float* __restrict__ first, i64 Rfirst, const float* __restrict__ rest,
                                                               i64 R, int C, int S, int roleB, float* __restrict__ dst) {
  __shared__ float tile[32][33];
  const i64 r0 = (i64)blockIdx.x * 32; const int c0 = blockIdx.y * 32;
  const i64 r = r0 + threadIdx.y; const int c = c0 + threadIdx.x;
  float v = 0.f;
  if (r < R && c < C) v = r < Rfirst ? first[r * C + c] : rest[(r - Rfirst) * C + c];
  tile[threadIdx.y][threadIdx.x] = v;
  __syncthreads();
  const i64 rr = r0 + threadIdx.x; const int cc = c0 + threadIdx.y;
  if (rr < R && cc < C) {
    const float x = tile[threadIdx.x][threadIdx.y];
    for (int seg = 0; seg < S; ++seg) dst[(i64)cc * S * R + (i64)seg * R + rr] = split_part(x, seg, roleB != 0);
  }
}

bool split_rows(const float* src, i64 ks, int B, int K, i64 M, int S, bool roleB, float* dst, cudaStream_t s) {
  if (M <= 0) return true;
  if (launch_pdl(split_rows_kernel, dim3(pgrid(M * K)), dim3(kPT), 0, s, src, ks, B, K, M, S, (int)roleB, dst) != cudaSuccess) return false;
  count_launch();
  return true;
}
void transpose_split(const float* first, i64 Rfirst, const float* rest, i64 R, int C, int S, bool roleB, float* dst, cudaStream_t s) {
  if (R <= 0) return;
  transpose_split_kernel<<<dim3((unsigned)((R + 31) / 32), (C + 31) / 32), dim3(32, 32), 0, s>>>(first, Rfirst, rest, R, C, S, (int)roleB, dst);
  count_launch();
}

}  // namespace

int tf32_supported(const mgrit_gru_cfg* c) {
  // 64 hidden units per gate tile, 16-column epilogue chunks, 16-byte row pitches of the [., S*T*B] gradient operands
  if (c->H % 64 != 0 || c->I % 16 != 0 || ((i64)c->T * c->B) % 4 != 0) return MGRIT_UNSUPPORTED;
  return MGRIT_OK;
}

void tf32_plan_fwd(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, Tf32Ws* o, int ng) {
  const size_t S = c->operands == MGRIT_OPERANDS_TF32 ? 3 : 1, H = c->H, I = c->I, TB = (size_t)c->T * c->B;
  o->S = (int)S; o->ng = ng;
  o->W_hh = take<float>(base, off, ng * H * S * H);
  o->W_ih = take<float>(base, off, ng * H * S * I);
  o->W_hhT = o->W_ihT = o->dAT = o->RT = nullptr;
  size_t ap = max_step_rows(c, N, L) * S * H;
  if (TB * S * I > ap) ap = TB * S * I;
  o->apack_elems = ap;
  o->Apack = take<float>(base, off, ap);
}

void tf32_plan_adj(const mgrit_gru_cfg* c, const int* N, int L, char* base, size_t* off, Tf32Ws* o, int ng) {
  (void)N; (void)L;
  const size_t S = c->operands == MGRIT_OPERANDS_TF32 ? 3 : 1, H = c->H, I = c->I, TB = (size_t)c->T * c->B;
  o->S = (int)S; o->ng = ng;
  o->W_hh = take<float>(base, off, ng * H * S * H);
  o->W_ih = nullptr;
  o->W_hhT = take<float>(base, off, H * S * ng * H);
  o->W_ihT = take<float>(base, off, I * S * ng * H);
  o->apack_elems = TB * S * ng * H;       // the input-gradient product packs all T*B rows of dA; every step needs less
  o->Apack = take<float>(base, off, o->apack_elems);
  o->dAT = take<float>(base, off, ng * H * S * TB);
  o->RT = take<float>(base, off, (H > I ? H : I) * S * TB);
  o->split_scratch = take<float>(base, off, 4 * ng * H * (H > I ? H : I));
}

int tf32_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, Tf32Ws* w, cudaStream_t s) {
  const int H = c->H, I = c->I, S = w->S, GH = w->ng * H;
  const int TB = c->T * c->B;
  if (!status_ptr()) return MGRIT_CUDA_ERROR;
  bool ok = split_rows(p->W_hh, 0, GH, H, GH, S, true, w->W_hh, s) && split_rows(p->W_ih, 0, GH, I, GH, S, true, w->W_ih, s) &&
            split_rows(x, 0, TB, I, TB, S, false, w->Apack, s);
  // gi = x W_ih^T + b_ih :  M = T*B, N = (3 or 4) H, K = S*I
  ok = ok && launch_gemm<256, 0>(KC_PROJ, (const float*)w->Apack, (i64)S * I, (const float*)w->W_ih, (i64)S * I, TB, GH, S * I, 0, GH,
                                     EpiBias{gi, GH, p->b_ih, TB, GH}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int tf32_fwd_step(const FwdStepArgs& a, Tf32Ws* w, cudaStream_t s) {
  const int S = w->S;
  if (!split_rows(a.hin, a.hin_ks, a.B, a.H, a.M, S, false, w->Apack, s)) return MGRIT_CUDA_ERROR;
  return launch_gemm<192, 3>(KC_FWD_STEP, (const float*)w->Apack, (i64)S * a.H, (const float*)w->W_hh, (i64)S * a.H, a.M, a.H, S * a.H, a.H,
                                3 * a.H, EpiFwd<false>{a}, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int tf32_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, Tf32Ws* w, cudaStream_t s) {
  const int H = c->H, I = c->I, S = w->S, GH = w->ng * H;
  if (!status_ptr()) return MGRIT_CUDA_ERROR;
  if (!split_rows(p->W_hh, 0, GH, H, GH, S, true, w->W_hh, s)) return MGRIT_CUDA_ERROR;
  transpose_split(nullptr, 0, p->W_hh, GH, H, S, true, w->W_hhT, s);   // [H, S*GH]
  transpose_split(nullptr, 0, p->W_ih, GH, I, S, true, w->W_ihT, s);   // [I, S*GH]
  return MGRIT_OK;
}

int tf32_linearise(const LinArgs& a, Tf32Ws* w, cudaStream_t s) {
  // rows (j-1, b): state entering forward step j of the level = h at fine time t0 + stride*(j-1) (h_0 for time 0)
  const i64 BH = (i64)a.B * a.H;
  const int N = a.M / a.B, S = w->S;
  int done = 0;
  if (a.t0 == 0) {
    if (!split_rows(a.h0, 0, a.B, a.H, a.B, S, false, w->Apack, s)) return MGRIT_CUDA_ERROR;
    done = 1;
  }
  if (N > done) {
    const i64 t1 = a.t0 + (i64)done * a.stride_t;
    if (!split_rows(a.h + (t1 - 1) * BH, a.stride_t * BH, a.B, a.H, (i64)(N - done) * a.B, S, false, w->Apack + (i64)done * BH * S, s))
      return MGRIT_CUDA_ERROR;
  }
  return launch_gemm<192, 3>(KC_LINEARISE, (const float*)w->Apack, (i64)S * a.H, (const float*)w->W_hh, (i64)S * a.H, a.M, a.H, S * a.H, a.H,
                                3 * a.H, EpiLin<false>{a}, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int tf32_adj_step(const AdjStepArgs& a, Tf32Ws* w, cudaStream_t s) {
  const int S = w->S, K = S * 3 * a.H;
  ProfScope prof(KC_ADJ_STEP, 2.0 * a.M * (double)K * a.H, s);
  if (launch_pdl(split_adj_kernel, dim3(pgrid((i64)a.M * a.H)), dim3(kPT), 0, s, a.lin, a.lin_ks, a.cr, a.cz, a.cn, a.coef_ks, a.B, a.H,
                 (i64)a.M, S, w->Apack) != cudaSuccess)
    return MGRIT_CUDA_ERROR;
  count_launch();
  const int tiles256 = ((a.M + BM - 1) / BM) * ((a.H + 255) / 256);
  bool ok;
  if (tiles256 * 2 <= kSMs)
    ok = launch_gemm<64, 0>(KC_ADJ_STEP, (const float*)w->Apack, (i64)K, (const float*)w->W_hhT, (i64)K, a.M, a.H, K, 0, a.H, EpiAdj<64>{a}, s);
  else
    ok = launch_gemm<256, 0>(KC_ADJ_STEP, (const float*)w->Apack, (i64)K, (const float*)w->W_hhT, (i64)K, a.M, a.H, K, 0, a.H, EpiAdj<256>{a}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// dW[n3, c] = sum_m dA[m, n3] * R[m, c],  R rows: m < Bfirst ? first[m] : rest[m - Bfirst]: both operands transposed (and
// split) so that the reduction index m runs along K-major rows; the long reduction is cut into up to four ranges.
int tf32_wgrad(const float* dA, int M, int H3, const float* first, int Bfirst, const float* rest, int C, float* dW, Tf32Ws* w,
               cudaStream_t s) {
  const int S = w->S, K = S * M;
  ProfScope prof(KC_WGRAD, 2.0 * H3 * (double)C * K, s);
  transpose_split(nullptr, 0, dA, M, H3, S, false, w->dAT, s);          // [3H, S*M]
  transpose_split(first, Bfirst, rest, M, C, S, true, w->RT, s);        // [C,  S*M]
  const size_t scratch_bytes = (size_t)4 * H3 * C * sizeof(float);
  const int splits = (((i64)H3 * C) % 4 == 0) ? pick_splits(H3, C, K, scratch_bytes) : 1;
  if (splits == 1)
    return launch_gemm<256, 0>(KC_WGRAD, (const float*)w->dAT, (i64)K, (const float*)w->RT, (i64)K, H3, C, K, 0, C, EpiStore{dW, C, H3, C, 0}, s)
               ? MGRIT_OK : MGRIT_CUDA_ERROR;
  const i64 n = (i64)H3 * C;
  if (!launch_gemm<256, 0>(KC_WGRAD, (const float*)w->dAT, (i64)K, (const float*)w->RT, (i64)K, H3, C, K, 0, C,
                               EpiStore{w->split_scratch, C, H3, C, n}, s, splits))
    return MGRIT_CUDA_ERROR;
  sum_splits_kernel<<<pgrid(n / 4), kPT, 0, s>>>(reinterpret_cast<const float4*>(w->split_scratch), n / 4, splits, reinterpret_cast<float4*>(dW));
  count_launch();
  return MGRIT_OK;
}

// dx[m, c] = sum_n3 dA[m, n3] * W_ih[n3, c]
int tf32_dgrad(const float* dA, int M, int H3, int C, float* dx, Tf32Ws* w, cudaStream_t s) {
  const int S = w->S, K = S * H3;
  if ((size_t)M * K > w->apack_elems) return MGRIT_UNSUPPORTED;
  if (!split_rows(dA, 0, M, H3, M, S, false, w->Apack, s)) return MGRIT_CUDA_ERROR;
  return launch_gemm<256, 0>(KC_WGRAD, (const float*)w->Apack, (i64)K, (const float*)w->W_ihT, (i64)K, M, C, K, 0, C, EpiStore{dx, C, M, C, 0}, s)
             ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// ---------------------------------------------------------------- Implicit LSTM on the tf32 products
namespace {

// LSTM cell / its transposed-Jacobian coefficients on the i | f | g | o accumulator columns of 64 hidden units, one
// output row per thread, 8 units at a time (precise gate math)
template <bool LIN, bool FAST = false>
struct EpiLstm {
  LstmFwdArgs f;      // !LIN
  LstmLinArgs l;      // LIN
  __device__ void operator()(uint32_t taddr, int row, int u0, int half) const {
    const int M = LIN ? l.M : f.M, B = LIN ? l.B : f.B, H = LIN ? l.H : f.H;
    const bool valid = row < M;
    const int k = valid ? row / B : 0, b = valid ? row % B : 0;
    const float* gi; const float* cpp; const float* bh = (LIN ? l.b_hh : f.b_hh) + u0;
    if (LIN) {
      const i64 t = l.t0 + (i64)k * l.stride_t;
      gi = l.gi + ((t + l.stride_t - 1) * B + b) * 4 * H + u0;
      cpp = (t == 0 ? l.c0 + (i64)b * H : l.c + (t - 1) * l.ts + (i64)b * H) + u0;
    } else {
      gi = f.gi + (i64)k * f.gi_ks + (i64)b * 4 * H + u0;
      cpp = f.cin + (i64)k * f.in_ks + (i64)b * H + u0;
    }
    const i64 o = (i64)row * H + u0;
    const float gamma = LIN ? l.gamma : f.gamma; const int cell = LIN ? l.cell : f.cell;
    // the kernel forms the level-array update itself: destination rows, and what is combined with the raw result
    // (the additive term, or in mode 1 the previous content of the destination)
    float* udst = nullptr; const float* usrc = nullptr;
    if (!LIN && f.up.out) {
      udst = f.up.out + (i64)k * f.up.out_ks + (i64)b * H + u0;
      usrc = f.up.mode == 1 ? udst : (f.up.g ? f.up.g + (i64)k * f.up.g_ks + (i64)b * H + u0 : nullptr);
    }
#pragma unroll 1
    for (int c0 = half * 32; c0 < half * 32 + 32; c0 += 8) {
      float g4[4][8], cp[8], acc[4][8], tc[8], th[8];
      if (valid) {
#pragma unroll
        for (int g = 0; g < 4; ++g) ld8(gi + (i64)g * H + c0, g4[g]);
        ld8(cpp + c0, cp);
        if (!LIN && usrc) { ld8(usrc + c0, tc); ld8(usrc + f.up.part + c0, th); }
      }
#pragma unroll
      for (int g = 0; g < 4; ++g) tmem_ld8(taddr + g * 64 + c0, acc[g]);
      tmem_ld_wait8x4(acc[0], acc[1], acc[2], acc[3]);
      if (valid) {
        float o0[8], o1[8], o2[8], o3[8], o4[8], o5[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int n = c0 + e;
          const float ai = acc[0][e] + __ldg(bh + n), af = acc[1][e] + __ldg(bh + H + n), ag = acc[2][e] + __ldg(bh + 2 * H + n),
                      ao = acc[3][e] + __ldg(bh + 3 * H + n);
          if (LIN) {
            LstmLin L = lstm_linearise<FAST>(g4[0][e], g4[1][e], g4[2][e], g4[3][e], ai, af, ag, ao, cp[e], gamma, cell);
            o0[e] = L.a; o1[e] = L.p; o2[e] = L.ci; o3[e] = L.cf; o4[e] = L.cg; o5[e] = L.co;
          } else {
            LstmOut r = lstm_forward<FAST>(g4[0][e], g4[1][e], g4[2][e], g4[3][e], ai, af, ag, ao, cp[e], gamma, cell);
            o0[e] = r.c; o1[e] = r.h;
          }
        }
        if (LIN) {
          st8(l.a + o + c0, o0); st8(l.p + o + c0, o1);
          if (l.cib) {      // gate coefficients as bf16: eight values = one 16-byte store each
            auto stb = [&](bf16* dst, const float* v) {
              const uint2 q0 = pack4(make_float4(v[0], v[1], v[2], v[3])), q1 = pack4(make_float4(v[4], v[5], v[6], v[7]));
              *reinterpret_cast<uint4*>(dst + o + c0) = make_uint4(q0.x, q0.y, q1.x, q1.y);
            };
            stb(l.cib, o2); stb(l.cfb, o3); stb(l.cgb, o4); stb(l.cob, o5);
          } else {
            st8(l.ci + o + c0, o2); st8(l.cf + o + c0, o3); st8(l.cg + o + c0, o4); st8(l.co + o + c0, o5);
          }
        } else if (udst) {
          if (usrc) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              o0[e] = f.up.mode == 1 ? tc[e] - o0[e] : o0[e] + tc[e];
              o1[e] = f.up.mode == 1 ? th[e] - o1[e] : o1[e] + th[e];
            }
          }
          st8(udst + c0, o0); st8(udst + f.up.part + c0, o1);
        } else {
          st8(f.cout + o + c0, o0); st8(f.hout + o + c0, o1);
        }
      }
    }
  }
};

// cell-part result of an adjoint step: raw to lc_out, or straight into the level array (see LstmUpdate)
__device__ __forceinline__ void lstm_store_lc(const LstmAdjArgs& a, i64 e, i64 kk, int b, int i, float v) {
  if (!a.up.out) { a.lc_out[e] = v; return; }
  float* d = a.up.out + kk * a.up.out_ks + (i64)b * a.H + i;
  if (a.up.mode == 1) *d = *d - v;
  else *d = a.up.g ? v + a.up.g[kk * a.up.g_ks + (i64)b * a.H + i] : v;
}

// hidden-part result of an adjoint step written into the level array: out = acc + g, or (previous content) - acc
template <int BN>
struct EpiUpdate {
  LstmUpdate u; int M, N, B;
  __device__ void operator()(uint32_t taddr, int row, int n0, int half) const {
    const bool valid = row < M;
    const int k = valid ? row / B : 0, b = valid ? row % B : 0;
    float* o = u.out + u.part + (i64)k * u.out_ks + (i64)b * N + n0;
    const float* g = u.mode == 1 ? o : (u.g ? u.g + u.part + (i64)k * u.g_ks + (i64)b * N + n0 : nullptr);
    const int cbeg = half * (BN / 2);
    for (int c0 = cbeg; c0 < cbeg + BN / 2 && n0 + c0 < N; c0 += 16) {
      float v[16], t[16];
      if (valid && g) { ld8(g + c0, t); ld8(g + c0 + 8, t + 8); }
      tmem_ld16(taddr + c0, v);
      tmem_ld_wait();
      if (valid) {
        if (g) {
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = u.mode == 1 ? t[e] - v[e] : v[e] + t[e];
        }
        st8(o + c0, v);
        st8(o + c0 + 8, v + 8);
      }
    }
  }
};

// dst[m, seg*4H + g*H + i] = split(coefficient_g * (g < 3 ? Lc + p*Lh : Lh))   (A side);  lc_out[m, i] = a * (Lc + p*Lh)
__global__ void __launch_bounds__(kPT) split_lstm_adj_kernel(LstmAdjArgs a, int S, float* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  const i64 total = (i64)a.M * a.H;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    const i64 m = e / a.H; const int i = (int)(e % a.H);
    const i64 kk = m / a.B; const int b = (int)(m % a.B);
    const i64 ci = kk * a.coef_ks + (i64)b * a.H + i, li = kk * a.in_ks + (i64)b * a.H + i;
    const float lh = a.lh[li], dc = a.lc[li] + a.p[ci] * lh;
    lstm_store_lc(a, e, kk, b, i, a.a[ci] * dc);
    const float v[4] = {a.ci[ci] * dc, a.cf[ci] * dc, a.cg[ci] * dc, a.co[ci] * lh};
    for (int seg = 0; seg < S; ++seg)
#pragma unroll
      for (int g = 0; g < 4; ++g) dst[m * S * 4 * a.H + (i64)seg * 4 * a.H + g * a.H + i] = split_part(v[g], seg, false);
  }
}

}  // namespace

int tf32_lstm_fwd_step(const LstmFwdArgs& a, Tf32Ws* w, cudaStream_t s) {
  const int S = w->S;
  if (!split_rows(a.hin, a.in_ks, a.B, a.H, a.M, S, false, w->Apack, s)) return MGRIT_CUDA_ERROR;
  EpiLstm<false> epi{};
  epi.f = a;
  return launch_gemm<256, 4>(KC_FWD_STEP, (const float*)w->Apack, (i64)S * a.H, (const float*)w->W_hh, (i64)S * a.H, a.M, a.H, S * a.H, a.H,
                             4 * a.H, epi, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int tf32_lstm_linearise(const LstmLinArgs& a, Tf32Ws* w, cudaStream_t s) {
  // rows (j-1, b): hidden state entering forward step j of the level = h at fine time t0 + stride*(j-1) (h_0 for time 0)
  const int N = a.M / a.B, S = w->S;
  const i64 BHS = (i64)a.B * a.H * S;
  int done = 0;
  if (a.t0 == 0) {
    if (!split_rows(a.h0, 0, a.B, a.H, a.B, S, false, w->Apack, s)) return MGRIT_CUDA_ERROR;
    done = 1;
  }
  if (N > done) {
    const i64 t1 = a.t0 + (i64)done * a.stride_t;
    if (!split_rows(a.h + (t1 - 1) * a.ts, a.stride_t * a.ts, a.B, a.H, (i64)(N - done) * a.B, S, false, w->Apack + (i64)done * BHS, s))
      return MGRIT_CUDA_ERROR;
  }
  EpiLstm<true> epi{};
  epi.l = a;
  return launch_gemm<256, 4>(KC_LINEARISE, (const float*)w->Apack, (i64)S * a.H, (const float*)w->W_hh, (i64)S * a.H, a.M, a.H, S * a.H, a.H,
                             4 * a.H, epi, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int tf32_lstm_adj_step(const LstmAdjArgs& a, Tf32Ws* w, cudaStream_t s) {
  const int S = w->S, K = S * 4 * a.H;
  ProfScope prof(KC_ADJ_STEP, 2.0 * a.M * (double)K * a.H, s);
  if (launch_pdl(split_lstm_adj_kernel, dim3(pgrid((i64)a.M * a.H)), dim3(kPT), 0, s, a, S, w->Apack) != cudaSuccess) return MGRIT_CUDA_ERROR;
  count_launch();
  const bool ok = a.up.out ? launch_gemm<256, 0>(KC_ADJ_STEP, (const float*)w->Apack, (i64)K, (const float*)w->W_hhT, (i64)K, a.M, a.H, K, 0, a.H,
                                                 EpiUpdate<256>{a.up, a.M, a.H, a.B}, s)
                           : launch_gemm<256, 0>(KC_ADJ_STEP, (const float*)w->Apack, (i64)K, (const float*)w->W_hhT, (i64)K, a.M, a.H, K, 0, a.H,
                                                 EpiStore{a.lh_out, a.H, a.M, a.H, 0}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// ---------------------------------------------------------------- Implicit LSTM, bf16 operands
namespace {
// dst[m, g*H + i] = bf16(coefficient_g * (g < 3 ? Lc + p*Lh : Lh));  lc_out[m, i] = a * (Lc + p*Lh)
__global__ void __launch_bounds__(kPT) pack_lstm_adj_kernel(LstmAdjArgs a, bf16* __restrict__ dst) {
  pdl_wait();
  pdl_trigger();
  const int H4 = a.H / 4;
  const i64 total = (i64)a.M * H4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {     // four units per thread
    const i64 m = e / H4; const int i = (int)(e % H4) * 4;
    const i64 kk = m / a.B; const int b = (int)(m % a.B);
    const i64 ci = kk * a.coef_ks + (i64)b * a.H + i, li = kk * a.in_ks + (i64)b * a.H + i;
    const float4 lh = ld4(a.lh + li), lc = ld4(a.lc + li), pp = ld4(a.p + ci), aa = ld4(a.a + ci);
    float4 c0, c1, c2, c3;
    if (a.cib) {
      c0 = unpack4(*reinterpret_cast<const uint2*>(a.cib + ci)); c1 = unpack4(*reinterpret_cast<const uint2*>(a.cfb + ci));
      c2 = unpack4(*reinterpret_cast<const uint2*>(a.cgb + ci)); c3 = unpack4(*reinterpret_cast<const uint2*>(a.cob + ci));
    } else {
      c0 = ld4(a.ci + ci); c1 = ld4(a.cf + ci); c2 = ld4(a.cg + ci); c3 = ld4(a.co + ci);
    }
    const float4 dc = make_float4(lc.x + pp.x * lh.x, lc.y + pp.y * lh.y, lc.z + pp.z * lh.z, lc.w + pp.w * lh.w);
    float4 v = make_float4(aa.x * dc.x, aa.y * dc.y, aa.z * dc.z, aa.w * dc.w);
    if (!a.up.out) {
      *reinterpret_cast<float4*>(a.lc_out + m * a.H + i) = v;
    } else {           // cell-part result straight into the level array (see LstmUpdate)
      float* d = a.up.out + kk * a.up.out_ks + (i64)b * a.H + i;
      if (a.up.mode == 1) {
        const float4 o = ld4(d);
        v = make_float4(o.x - v.x, o.y - v.y, o.z - v.z, o.w - v.w);
      } else if (a.up.g) {
        const float4 g = ld4(a.up.g + kk * a.up.g_ks + (i64)b * a.H + i);
        v = make_float4(v.x + g.x, v.y + g.y, v.z + g.z, v.w + g.w);
      }
      *reinterpret_cast<float4*>(d) = v;
    }
    uint2* q = reinterpret_cast<uint2*>(dst + m * 4 * a.H + i);
    q[0] = pack4(make_float4(c0.x * dc.x, c0.y * dc.y, c0.z * dc.z, c0.w * dc.w));
    q[H4] = pack4(make_float4(c1.x * dc.x, c1.y * dc.y, c1.z * dc.z, c1.w * dc.w));
    q[2 * H4] = pack4(make_float4(c2.x * dc.x, c2.y * dc.y, c2.z * dc.z, c2.w * dc.w));
    q[3 * H4] = pack4(make_float4(c3.x * lh.x, c3.y * lh.y, c3.z * lh.z, c3.w * lh.w));
  }
}
bool pack_rows(const float* src, i64 ks, int B, int H, i64 M, bf16* dst, cudaStream_t s) {
  if (M <= 0) return true;
  if (launch_pdl(pack_rows_kernel, dim3(pgrid(M * (H / 4))), dim3(kPT), 0, s, src, ks, B, H / 4, M, reinterpret_cast<uint2*>(dst)) != cudaSuccess)
    return false;
  count_launch();
  return true;
}
}  // namespace

void lstmbf_plan_fwd(const mgrit_gru_cfg* c, size_t max_rows, char* base, size_t* off, LstmBfWs* o) {
  const size_t H = c->H, I = c->I, TB = (size_t)c->T * c->B;
  *o = LstmBfWs{};
  o->W_hh = take<bf16>(base, off, 4 * H * H);
  o->W_ih = take<bf16>(base, off, 4 * H * I);
  o->apack_elems = max_rows * H > TB * I ? max_rows * H : TB * I;      // a step's rows, or x for the projection
  o->Apack = take<bf16>(base, off, o->apack_elems);
}

void lstmbf_plan_adj(const mgrit_gru_cfg* c, size_t max_rows, char* base, size_t* off, LstmBfWs* o) {
  const size_t H = c->H, I = c->I, TB = (size_t)c->T * c->B;
  *o = LstmBfWs{};
  o->W_hh = take<bf16>(base, off, 4 * H * H);
  o->W_hhT = take<bf16>(base, off, 4 * H * H);
  o->W_ihT = take<bf16>(base, off, 4 * H * I);
  size_t ap = max_rows * 4 * H;
  if (TB * H > ap) ap = TB * H;        // the linearisation packs all T*B rows of a level at once
  o->apack_elems = ap;
  o->Apack = take<bf16>(base, off, ap);
  o->xb = take<bf16>(base, off, TB * I);
  o->hb0 = take<bf16>(base, off, (TB + c->B) * H);
  o->dAb = take<bf16>(base, off, TB * 4 * H);
  o->scratch_bytes = (size_t)4 * 4 * H * (H > I ? H : I) * sizeof(float);
  o->scratch = take<float>(base, off, o->scratch_bytes / sizeof(float));
}

int lstmbf_prepare_fwd(const mgrit_gru_cfg* c, const gru_params* p, const float* x, float* gi, LstmBfWs* w, cudaStream_t s) {
  const int H = c->H, I = c->I, TB = c->T * c->B;
  if (!status_ptr()) return MGRIT_CUDA_ERROR;
  convert(p->W_hh, w->W_hh, (i64)4 * H * H, s);
  convert(p->W_ih, w->W_ih, (i64)4 * H * I, s);
  convert(x, w->Apack, (i64)TB * I, s);
  return launch_gemm<256, 0>(KC_PROJ, w->Apack, I, w->W_ih, I, TB, 4 * H, I, 0, 4 * H, EpiBias{gi, 4 * H, p->b_ih, TB, 4 * H}, s) ? MGRIT_OK
                                                                                                                       : MGRIT_CUDA_ERROR;
}

int lstmbf_prepare_adj(const mgrit_gru_cfg* c, const gru_params* p, LstmBfWs* w, cudaStream_t s) {
  const int H = c->H, I = c->I;
  if (!status_ptr()) return MGRIT_CUDA_ERROR;
  convert(p->W_hh, w->W_hh, (i64)4 * H * H, s);
  transpose(p->W_hh, 4 * H, H, w->W_hhT, 4 * H, 0, s);   // [H, 4H]
  transpose(p->W_ih, 4 * H, I, w->W_ihT, 4 * H, 0, s);   // [I, 4H]
  return MGRIT_OK;
}

int lstmbf_fwd_step(const LstmFwdArgs& a, LstmBfWs* w, cudaStream_t s) {
  if (!pack_rows(a.hin, a.in_ks, a.B, a.H, a.M, w->Apack, s)) return MGRIT_CUDA_ERROR;
  EpiLstm<false, true> epi{};
  epi.f = a;
  return launch_gemm<256, 4>(KC_FWD_STEP, w->Apack, a.H, w->W_hh, a.H, a.M, a.H, a.H, a.H, 4 * a.H, epi, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int lstmbf_linearise(const LstmLinArgs& a, LstmBfWs* w, cudaStream_t s) {
  const int N = a.M / a.B;
  const i64 BH = (i64)a.B * a.H;
  int done = 0;
  if (a.t0 == 0) {
    if (!pack_rows(a.h0, 0, a.B, a.H, a.B, w->Apack, s)) return MGRIT_CUDA_ERROR;
    done = 1;
  }
  if (N > done) {
    const i64 t1 = a.t0 + (i64)done * a.stride_t;
    if (!pack_rows(a.h + (t1 - 1) * a.ts, a.stride_t * a.ts, a.B, a.H, (i64)(N - done) * a.B, w->Apack + (i64)done * BH, s)) return MGRIT_CUDA_ERROR;
  }
  EpiLstm<true, true> epi{};
  epi.l = a;
  return launch_gemm<256, 4>(KC_LINEARISE, w->Apack, a.H, w->W_hh, a.H, a.M, a.H, a.H, a.H, 4 * a.H, epi, s) ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int lstmbf_adj_step(const LstmAdjArgs& a, LstmBfWs* w, cudaStream_t s) {
  const int K = 4 * a.H;
  ProfScope prof(KC_ADJ_STEP, 2.0 * a.M * (double)K * a.H, s);
  if (launch_pdl(pack_lstm_adj_kernel, dim3(pgrid((i64)a.M * (a.H / 4))), dim3(kPT), 0, s, a, w->Apack) != cudaSuccess) return MGRIT_CUDA_ERROR;
  count_launch();
  // few-row steps (coarse levels, the serial sweep): 64-column tiles spread the stream over K over four times the CTAs
  const bool few = ((a.M + BM - 1) / BM) * ((a.H + 255) / 256) * 2 <= kSMs;
  const bool ok = !a.up.out ? launch_gemm<256, 0>(KC_ADJ_STEP, w->Apack, K, w->W_hhT, K, a.M, a.H, K, 0, a.H, EpiStore{a.lh_out, a.H, a.M, a.H, 0}, s)
                  : few     ? launch_gemm<64, 0>(KC_ADJ_STEP, w->Apack, K, w->W_hhT, K, a.M, a.H, K, 0, a.H, EpiUpdate<64>{a.up, a.M, a.H, a.B}, s)
                  // (row tiles in descending order: the operand rows packed last are still in L2)
                  : gemm_pair_enabled(a.M, a.H)
                            ? launch_gemm_pair(KC_ADJ_STEP, w->Apack, K, w->W_hhT, K, a.M, a.H, K, a.H, EpiUpdate<256>{a.up, a.M, a.H, a.B}, s, true)
                            : launch_gemm<256, 0>(KC_ADJ_STEP, w->Apack, K, w->W_hhT, K, a.M, a.H, K, 0, a.H, EpiUpdate<256>{a.up, a.M, a.H, a.B}, s,
                                                  1, true);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

namespace {
// Gradient-pass operand of the LSTM as bf16, row-major: dA[m, :] = [ci*dc | cf*dc | cg*dc | co*Lh] with dc = Lc + p*Lh, plus
// this block's fp32 column sums of the four products (bias-gradient partials) to part[blockIdx.x][4][H].  Row m = (t, b):
// sensitivities at lc / lh + t*lam_ts + b*H (lam_ts may be negative: the adjoint keeps its unknowns in reversed time
// order).  Block = 32 float4 columns (128 units) x 8 rows at a time.
__global__ void __launch_bounds__(256) lstm_form_dA_rows_kernel(const float* __restrict__ lc, const float* __restrict__ lh, i64 lam_ts, int B,
                                                                const float* __restrict__ p, const bf16* __restrict__ ci,
                                                                const bf16* __restrict__ cf, const bf16* __restrict__ cg,
                                                                const bf16* __restrict__ co, i64 M, int H, uint2* __restrict__ dA,
                                                                float* __restrict__ part, int rows_per_block) {
  __shared__ float red[4][8][128];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int H4 = H / 4, c4 = blockIdx.y * 32 + tx;
  const i64 m0 = (i64)blockIdx.x * rows_per_block;
  float4 s[4];
#pragma unroll
  for (int g = 0; g < 4; ++g) s[g] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c4 < H4) {
    for (i64 m = m0 + ty; m < m0 + rows_per_block && m < M; m += 8) {
      const i64 e = (m * H4 + c4) * 4;
      const int t = (int)m / B, bb = (int)m - t * B;       // row counts fit 32 bits (checked by the host)
      const i64 li = (i64)t * lam_ts + ((i64)bb * H4 + c4) * 4;
      const float4 h = ld4(lh + li), c = ld4(lc + li), pp = ld4(p + e);
      const float4 k0 = unpack4(*reinterpret_cast<const uint2*>(ci + e)), k1 = unpack4(*reinterpret_cast<const uint2*>(cf + e));
      const float4 k2 = unpack4(*reinterpret_cast<const uint2*>(cg + e)), k3 = unpack4(*reinterpret_cast<const uint2*>(co + e));
      const float4 dc = make_float4(c.x + pp.x * h.x, c.y + pp.y * h.y, c.z + pp.z * h.z, c.w + pp.w * h.w);
      const float4 v[4] = {make_float4(k0.x * dc.x, k0.y * dc.y, k0.z * dc.z, k0.w * dc.w), make_float4(k1.x * dc.x, k1.y * dc.y, k1.z * dc.z, k1.w * dc.w),
                           make_float4(k2.x * dc.x, k2.y * dc.y, k2.z * dc.z, k2.w * dc.w), make_float4(k3.x * h.x, k3.y * h.y, k3.z * h.z, k3.w * h.w)};
      const i64 o = m * 4 * H4 + c4;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        dA[o + g * H4] = pack4(v[g]);
        s[g].x += v[g].x; s[g].y += v[g].y; s[g].z += v[g].z; s[g].w += v[g].w;
      }
    }
  }
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    red[g][ty][tx * 4] = s[g].x; red[g][ty][tx * 4 + 1] = s[g].y; red[g][ty][tx * 4 + 2] = s[g].z; red[g][ty][tx * 4 + 3] = s[g].w;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < 4 * 128; e += 256) {
    int g = e / 128, u = e % 128, col = blockIdx.y * 128 + u;
    if (col >= H) continue;
    float acc = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) acc += red[g][r][u];
    part[((i64)blockIdx.x * 4 + g) * H + col] = acc;
  }
}
// db_hh = db_ih = the per-block partials summed in block order (the same bits on every run)
__global__ void __launch_bounds__(kPT) lstm_sum_db_kernel(const float* __restrict__ part, int nblk, int H, float* __restrict__ db_hh,
                                                          float* __restrict__ db_ih) {
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < 4 * H; e += gridDim.x * blockDim.x) {
    float acc = 0.f;
    for (int k = 0; k < nblk; ++k) acc += part[(i64)k * 4 * H + e];
    db_hh[e] = acc; db_ih[e] = acc;
  }
}
}  // namespace

// All gradients of the LSTM parameters (and dx) from the step-output sensitivities (lc, lh; rows (t, b) at + t*lam_ts + b*H),
// the level-0 coefficients and the hidden states entering each step (h0, then h_rows + (t-1)*h_ts).
int lstmbf_gradients(const mgrit_gru_cfg* c, const float* lc, const float* lh, i64 lam_ts, const float* p, const bf16* ci, const bf16* cf,
                     const bf16* cg, const bf16* co, const float* x, const float* h0, const float* h_rows, i64 h_ts, const gru_grads* g,
                     float* dx, LstmBfWs* w, cudaStream_t s) {
  const int H = c->H, I = c->I, B = c->B;
  const i64 M = (i64)c->T * B;
  ProfScope prof(KC_WGRAD, 2.0 * M * 4.0 * H * ((double)H + I + (dx ? I : 0)), s);
  const int rows_per_block = 256;
  dim3 grid((unsigned)((M + rows_per_block - 1) / rows_per_block), (H / 4 + 31) / 32);
  if ((size_t)grid.x * 4 * H * sizeof(float) > w->scratch_bytes) return MGRIT_UNSUPPORTED;
  // (the bias partials use the split-product scratch before the weight-gradient products need it)
  lstm_form_dA_rows_kernel<<<grid, 256, 0, s>>>(lc, lh, lam_ts, B, p, ci, cf, cg, co, M, H, reinterpret_cast<uint2*>(w->dAb), w->scratch,
                                                rows_per_block);
  lstm_sum_db_kernel<<<pgrid(4 * H), kPT, 0, s>>>(w->scratch, (int)grid.x, H, g->db_hh, g->db_ih);
  count_launch(2);
  convert(x, w->xb, M * I, s);
  convert(h0, w->hb0, (i64)B * H, s);
  if (c->T > 1 && !pack_rows(h_rows, h_ts, B, H, M - B, w->hb0 + (i64)B * H, s)) return MGRIT_CUDA_ERROR;   // rows (t, b) of h_{t-1} start at hb0
  bool ok = wgrad_gemm(w->dAb, 4 * H, w->hb0, H, (int)M, g->dW_hh, w->scratch, w->scratch_bytes, s);
  ok = ok && wgrad_gemm(w->dAb, 4 * H, w->xb, I, (int)M, g->dW_ih, w->scratch, w->scratch_bytes, s);
  if (dx) ok = ok && launch_gemm<256, 0>(KC_WGRAD, w->dAb, 4 * H, w->W_ihT, 4 * H, (int)M, I, 4 * H, 0, I, EpiStore{dx, I, (int)M, I, 0}, s);
  return ok ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

// Self-test of the bounded waits: one warp waits, with the library's own wait routine and a short limit, on a barrier
// that nothing ever signals.  The wait runs out, records its code in the status word and the kernel returns normally.
namespace {
__global__ void __launch_bounds__(32) wait_probe_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, 90, limit_ns);
  }
}
}  // namespace

int umma_selftest_wait(int limit_ms, cudaStream_t s) {
  if (limit_ms < 1 || limit_ms > 1000) return MGRIT_INVALID_ARG;
  int* const status = status_ptr();
  if (!status) return MGRIT_CUDA_ERROR;
  wait_probe_kernel<<<1, 32, 0, s>>>(status, (unsigned long long)limit_ms * 1000000ull);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? MGRIT_OK : MGRIT_CUDA_ERROR;
}

int umma_device_status() {
  const int dev = current_device_slot();
  if (dev < 0) return -1;
  if (!g_status_ptrs[dev]) return 0;     // no tensor-core kernel has run on this device
  int v = 0;
  if (cudaMemcpy(&v, g_status_ptrs[dev], sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return v;
}

int umma_clear_device_status() {
  const int dev = current_device_slot();
  if (dev < 0) return -1;
  if (!g_status_ptrs[dev]) return 0;
  return cudaMemset(g_status_ptrs[dev], 0, sizeof(int)) == cudaSuccess ? 0 : -1;
}

}  // namespace mg
