// Streaming (HBM-bound) kernels: grid transfers of the multigrid cycle, operand forming for the
// gradient pass, column sums, the classifier head and the SGD update.  float4 accesses,
// coalesced along the hidden dimension; grids sized in multiples of the SM count.
#include <math.h>

#include "common.cuh"

namespace mg {

namespace {

constexpr int kSMs = 148;
constexpr int kThreads = 256;

inline int stream_grid(i64 work_items, int per_block = kThreads) {
  i64 blocks = (work_items + per_block - 1) / per_block;
  i64 cap = (i64)kSMs * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

__device__ __forceinline__ uint2 pack_bf16x4(float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<uint32_t*>(&lo);
  o.y = *reinterpret_cast<uint32_t*>(&hi);
  return o;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Residual at the C-points (r = u_C - v), its squared norm, and restriction by injection
// (Algorithm "MGProp": r_c = R(f(h')), h'_c = R(h');  Eq. "restrict").
__global__ void __launch_bounds__(kThreads) restrict_residual_kernel(const float4* __restrict__ uf, int cf,
                                                                     const float4* __restrict__ v,
                                                                     float4* __restrict__ uc, uint2* __restrict__ ucb,
                                                                     int nc, i64 row4, double* acc) {
  pdl_wait();      // launched with programmatic stream serialisation: nothing is read before the predecessor is done
  pdl_trigger();
  i64 total = (i64)nc * row4;
  float s = 0.f;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 k = e / row4 + 1, c = e % row4;
    float4 u = uf[(k * cf) * row4 + c];
    float4 w = v[k * row4 + c];
    float4 r = make_float4(u.x - w.x, u.y - w.y, u.z - w.z, u.w - w.w);
    s += r.x * r.x + r.y * r.y + r.z * r.z + r.w * r.w;
    uc[k * row4 + c] = u;
    if (ucb) ucb[k * row4 + c] = pack_bf16x4(u);
  }
  __shared__ float part[kThreads / 32];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = threadIdx.x < kThreads / 32 ? part[threadIdx.x] : 0.f;
    t = warp_sum(t);
    if (threadIdx.x == 0 && acc) atomicAdd(acc, (double)t);
  }
}

// Correction h'' = h' + P(h_c* - h'_c): only C-points are read afterwards, so u_{cf k} <- U_k.
__global__ void __launch_bounds__(kThreads) correct_kernel(float4* __restrict__ uf, uint2* __restrict__ ufb, int cf,
                                                           const float4* __restrict__ uc, int nc, i64 row4) {
  pdl_wait();
  pdl_trigger();
  i64 total = (i64)nc * row4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 k = e / row4 + 1, c = e % row4;
    float4 u = uc[k * row4 + c];
    uf[(k * cf) * row4 + c] = u;
    if (ufb) ufb[(k * cf) * row4 + c] = pack_bf16x4(u);
  }
}

__global__ void __launch_bounds__(kThreads) gather_rows_kernel(float4* __restrict__ dst, i64 dst_ks4,
                                                               const float4* __restrict__ src, i64 src_ks4, int nk,
                                                               i64 row4) {
  i64 total = (i64)nk * row4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 k = e / row4, c = e % row4;
    dst[k * dst_ks4 + c] = src[k * src_ks4 + c];
  }
}

// Stacked layers: raw step result tmp[m, :] (rows m = (k, b), contiguous) -> level unknown rows (k, b) at dst + k*dst_ks + b*H:
// mode 0: dst = tmp + g (g optional, same indexing with g_ks);  mode 1: dst = dst - tmp  (FAS right-hand side).
__global__ void __launch_bounds__(kThreads) combine_rows_kernel(const float4* __restrict__ tmp, const float4* __restrict__ g, i64 g_ks4,
                                                                float4* __restrict__ dst, i64 dst_ks4, int B, int H4, i64 M, int mode) {
  i64 total = M * H4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / H4; int c = (int)(e % H4);
    i64 k = m / B; int b = (int)(m % B);
    float4 t = tmp[e];
    float4* d = dst + k * dst_ks4 + (i64)b * H4 + c;
    if (mode == 1) {
      float4 o = *d;
      *d = make_float4(o.x - t.x, o.y - t.y, o.z - t.z, o.w - t.w);
    } else {
      if (g) {
        float4 a = g[k * g_ks4 + (i64)b * H4 + c];
        t = make_float4(t.x + a.x, t.y + a.y, t.z + a.z, t.w + a.w);
      }
      *d = t;
    }
  }
}

__global__ void __launch_bounds__(kThreads) add_rows_kernel(float4* __restrict__ dst, const float4* __restrict__ src, i64 n4) {
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (i64)gridDim.x * blockDim.x) {
    float4 a = dst[e], b = src[e];
    dst[e] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
  }
}

__global__ void __launch_bounds__(kThreads) form_dA_kernel(const float4* __restrict__ lam, const float4* __restrict__ cr,
                                                           const float4* __restrict__ cz, const float4* __restrict__ cn,
                                                           const float4* __restrict__ cnp, float4* __restrict__ dA_h,
                                                           float4* __restrict__ dA_i, i64 M, int H4) {
  i64 total = M * H4;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (i64)gridDim.x * blockDim.x) {
    i64 m = e / H4, c = e % H4;
    float4 l = lam[e], r = cr[e], z = cz[e], n = cn[e], p = cnp[e];
    i64 o = m * 3 * H4 + c;
    float4 vr = make_float4(r.x * l.x, r.y * l.y, r.z * l.z, r.w * l.w);
    float4 vz = make_float4(z.x * l.x, z.y * l.y, z.z * l.z, z.w * l.w);
    dA_h[o] = vr; dA_i[o] = vr;
    dA_h[o + H4] = vz; dA_i[o + H4] = vz;
    dA_h[o + 2 * H4] = make_float4(n.x * l.x, n.y * l.y, n.z * l.z, n.w * l.w);
    dA_i[o + 2 * H4] = make_float4(p.x * l.x, p.y * l.y, p.z * l.z, p.w * l.w);
  }
}

// out[n] = sum_m A[m, n]; one block per 32 columns, deterministic.
__global__ void __launch_bounds__(1024) colsum_kernel(const float* __restrict__ A, i64 M, int N, float* __restrict__ out) {
  __shared__ float part[32][33];
  int n = blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (n < N)
    for (i64 m = threadIdx.y; m < M; m += 32) s += A[m * N + n];
  part[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && n < N) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) t += part[i][threadIdx.x];
    out[n] = t;
  }
}

__global__ void sqrt_to_float_kernel(const double* acc, float* out, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = (float)sqrt(acc[i]);
}

// Classifier head, pass 1: one block per batch row: logits, softmax, the row's loss term, dlogits = (p - onehot)/B.
// A label outside [0, C) marks a row without a target: it adds nothing to the loss and its one-hot term is absent.
__global__ void __launch_bounds__(kThreads) xent_rows_kernel(int B, int H, int C, const float* __restrict__ hT,
                                                             const float* __restrict__ Wc, const float* __restrict__ bc,
                                                             const int32_t* __restrict__ labels, float* __restrict__ rowloss,
                                                             float* __restrict__ dlogits) {
  extern __shared__ float logit[];  // C floats
  int b = blockIdx.x;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int c = warp; c < C; c += nw) {
    float s = 0.f;
    for (int i = lane; i < H; i += 32) s += hT[(i64)b * H + i] * Wc[(i64)c * H + i];
    s = warp_sum(s);
    if (lane == 0) logit[c] = s + bc[c];
  }
  __syncthreads();
  if (warp == 0) {
    float mx = -INFINITY;
    for (int c = lane; c < C; c += 32) mx = fmaxf(mx, logit[c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = 0.f;
    for (int c = lane; c < C; c += 32) se += __expf(logit[c] - mx);
    se = warp_sum(se);
    const int lab = labels[b];
    const bool has_label = lab >= 0 && lab < C;
    float invB = 1.0f / (float)B;
    for (int c = lane; c < C; c += 32) {
      float p = __expf(logit[c] - mx) / se;
      dlogits[(i64)b * C + c] = (p - (c == lab ? 1.f : 0.f)) * invB;
    }
    if (lane == 0) rowloss[b] = has_label ? -((logit[lab] - mx) - logf(se)) * invB : 0.f;
  }
}

// pass 2: dhT = dlogits Wc ; dWc = dlogits^T hT ; dbc = column sums of dlogits ; loss = sum of the row terms in
// row order (fixed order: the same bits on every run).
__global__ void __launch_bounds__(kThreads) xent_grads_kernel(int B, int H, int C, const float* __restrict__ hT,
                                                              const float* __restrict__ Wc,
                                                              const float* __restrict__ dlogits, const float* __restrict__ rowloss,
                                                              float* __restrict__ loss, float* __restrict__ dhT,
                                                              float* __restrict__ dWc, float* __restrict__ dbc) {
  i64 nBH = (i64)B * H, nCH = (i64)C * H;
  for (i64 e = (i64)blockIdx.x * blockDim.x + threadIdx.x; e < nBH + nCH + C + 1; e += (i64)gridDim.x * blockDim.x) {
    if (e == nBH + nCH + C) {
      float s = 0.f;
      for (int b = 0; b < B; ++b) s += rowloss[b];
      *loss = s;
      continue;
    }
    if (e < nBH) {
      int b = e / H, i = e % H;
      float s = 0.f;
      for (int c = 0; c < C; ++c) s += dlogits[(i64)b * C + c] * Wc[(i64)c * H + i];
      dhT[e] = s;
    } else if (e < nBH + nCH) {
      i64 f = e - nBH;
      int c = f / H, i = f % H;
      float s = 0.f;
      for (int b = 0; b < B; ++b) s += dlogits[(i64)b * C + c] * hT[(i64)b * H + i];
      dWc[f] = s;
    } else {
      int c = (int)(e - nBH - nCH);
      float s = 0.f;
      for (int b = 0; b < B; ++b) s += dlogits[(i64)b * C + c];
      dbc[c] = s;
    }
  }
}

__global__ void __launch_bounds__(kThreads) sgd_kernel(float* __restrict__ p, const float* __restrict__ g, size_t n, float lr) {
  size_t n4 = n / 4;
  float4* p4 = reinterpret_cast<float4*>(p);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  size_t stride = (size_t)gridDim.x * blockDim.x, t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (size_t e = t; e < n4; e += stride) {
    float4 a = p4[e], b = g4[e];
    p4[e] = make_float4(a.x - lr * b.x, a.y - lr * b.y, a.z - lr * b.z, a.w - lr * b.w);
  }
  for (size_t e = n4 * 4 + t; e < n; e += stride) p[e] -= lr * g[e];
}

// Adam with bias correction (the optimiser of the paper's experiments; same update as torch.optim.Adam without
// weight decay): m <- b1 m + (1-b1) g, v <- b2 v + (1-b2) g^2, p <- p - lr/(1-b1^t) * m / (sqrt(v)/sqrt(1-b2^t) + eps).
__global__ void __launch_bounds__(kThreads) adam_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m,
                                                        float* __restrict__ v, size_t n, float step_size, float inv_sqrt_bc2,
                                                        float b1, float b2, float eps) {
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride) {
    float gg = g[e];
    float mm = b1 * m[e] + (1.f - b1) * gg;
    float vv = b2 * v[e] + (1.f - b2) * gg * gg;
    m[e] = mm; v[e] = vv;
    p[e] -= step_size * mm / (sqrtf(vv) * inv_sqrt_bc2 + eps);
  }
}

}  // namespace

void stream_adam(float* p, const float* g, float* m, float* v, size_t n, float lr, float b1, float b2, float eps, int step,
                 cudaStream_t s) {
  double bc1 = 1.0 - pow((double)b1, (double)step), bc2 = 1.0 - pow((double)b2, (double)step);
  adam_kernel<<<stream_grid((i64)n), kThreads, 0, s>>>(p, g, m, v, n, (float)(lr / bc1), (float)(1.0 / sqrt(bc2)), b1, b2, eps);
  count_launch();
}

void stream_restrict_residual(const float* uf, int cf, const float* v, float* uc, __nv_bfloat16* ucb, int nc, i64 rowlen, double* acc,
                              cudaStream_t s) {
  i64 row4 = rowlen / 4;
  launch_pdl(restrict_residual_kernel, dim3(stream_grid((i64)nc * row4)), dim3(kThreads), 0, s, reinterpret_cast<const float4*>(uf), cf,
             reinterpret_cast<const float4*>(v), reinterpret_cast<float4*>(uc), reinterpret_cast<uint2*>(ucb), nc, row4, acc);
  count_launch();
}

void stream_correct(float* uf, __nv_bfloat16* ufb, int cf, const float* uc, int nc, i64 rowlen, cudaStream_t s) {
  i64 row4 = rowlen / 4;
  launch_pdl(correct_kernel, dim3(stream_grid((i64)nc * row4)), dim3(kThreads), 0, s, reinterpret_cast<float4*>(uf),
             reinterpret_cast<uint2*>(ufb), cf, reinterpret_cast<const float4*>(uc), nc, row4);
  count_launch();
}

void stream_gather_rows(float* dst, i64 dst_ks, const float* src, i64 src_ks, int nk, i64 rowlen, cudaStream_t s) {
  if (nk <= 0) return;
  i64 row4 = rowlen / 4;
  gather_rows_kernel<<<stream_grid((i64)nk * row4), kThreads, 0, s>>>(reinterpret_cast<float4*>(dst), dst_ks / 4,
                                                                      reinterpret_cast<const float4*>(src), src_ks / 4, nk, row4);
  count_launch();
}

void stream_combine_rows(const float* tmp, const float* g, i64 g_ks, float* dst, i64 dst_ks, int B, int H, i64 M, int mode, cudaStream_t s) {
  combine_rows_kernel<<<stream_grid(M * (H / 4)), kThreads, 0, s>>>(reinterpret_cast<const float4*>(tmp), reinterpret_cast<const float4*>(g),
                                                                   g_ks / 4, reinterpret_cast<float4*>(dst), dst_ks / 4, B, H / 4, M, mode);
  count_launch();
}

void stream_add_rows(float* dst, const float* src, i64 n, cudaStream_t s) {
  add_rows_kernel<<<stream_grid(n / 4), kThreads, 0, s>>>(reinterpret_cast<float4*>(dst), reinterpret_cast<const float4*>(src), n / 4);
  count_launch();
}

void stream_form_dA(const float* lam, const float* cr, const float* cz, const float* cn, const float* cnp, float* dA_h,
                    float* dA_i, i64 M, int H, cudaStream_t s) {
  form_dA_kernel<<<stream_grid(M * (H / 4)), kThreads, 0, s>>>(
      reinterpret_cast<const float4*>(lam), reinterpret_cast<const float4*>(cr), reinterpret_cast<const float4*>(cz),
      reinterpret_cast<const float4*>(cn), reinterpret_cast<const float4*>(cnp), reinterpret_cast<float4*>(dA_h),
      reinterpret_cast<float4*>(dA_i), M, H / 4);
  count_launch();
}

void stream_colsum(const float* A, i64 M, int N, float* out, cudaStream_t s) {
  colsum_kernel<<<(N + 31) / 32, dim3(32, 32), 0, s>>>(A, M, N, out);
  count_launch();
}

void stream_sqrt_to_float(const double* acc, float* out, int n, cudaStream_t s) {
  sqrt_to_float_kernel<<<(n + 63) / 64, 64, 0, s>>>(acc, out, n);
  count_launch();
}

void stream_xent(int B, int H, int C, const float* hT, const float* Wc, const float* bc, const int32_t* labels, float* loss,
                 float* dhT, float* dWc, float* dbc, float* dlogits, cudaStream_t s) {
  float* rowloss = dlogits + (size_t)B * C;      // the scratch holds [B, C] derivatives followed by B row terms
  xent_rows_kernel<<<B, kThreads, (size_t)C * sizeof(float), s>>>(B, H, C, hT, Wc, bc, labels, rowloss, dlogits);
  xent_grads_kernel<<<stream_grid((i64)B * H + (i64)C * H + C + 1), kThreads, 0, s>>>(B, H, C, hT, Wc, dlogits, rowloss, loss, dhT, dWc,
                                                                                     dbc);
  count_launch(2);
}

void stream_sgd(float* p, const float* g, size_t n, float lr, cudaStream_t s) {
  sgd_kernel<<<stream_grid((i64)(n / 4 + 1)), kThreads, 0, s>>>(p, g, n, lr);
  count_launch();
}

}  // namespace mg

// ---------------------------------------------------------------------------------------------------
// Classifier head without any caller-provided or allocated scratch.
//
// Some hosts of this library cannot allocate device memory at the moment they need the loss head: a
// serving or training process that has handed the whole GPU to its own memory arena (cudaMalloc then
// fails or fragments the arena), or a latency-critical loop that must not take the driver's allocator
// lock, which can also synchronise the device.  For them the [B, C] buffer of loss derivatives with
// respect to the logits (and the B per-row loss terms) lives in a fixed array inside the library image.  Every GPU that loads the
// library holds these 256 KiB until the process exits.
namespace mg {
namespace {
constexpr size_t kHeadScratchFloats = 65536;   // B * (C + 1) <= 65536: [B, C] derivatives + B row loss terms
static __device__ __align__(256) float g_head_scratch[kHeadScratchFloats];
float* g_head_scratch_addr[kMaxDevices] = {nullptr};   // device address of the array, per device
}  // namespace
}  // namespace mg

extern "C" int xent_head_fwd_bwd_noalloc(int32_t B, int32_t H, int32_t C, const float* hT, const float* Wc, const float* bc,
                                         const int32_t* labels, float* loss, float* dhT, float* dWc, float* dbc,
                                         mgrit_stream_t stream) {
  using namespace mg;
  if (B <= 0 || H <= 0 || C <= 0 || !hT || !Wc || !bc || !labels || !loss || !dhT || !dWc || !dbc) return MGRIT_INVALID_ARG;
  if (C > 8192) return MGRIT_UNSUPPORTED;
  if ((size_t)B * ((size_t)C + 1) > kHeadScratchFloats) return MGRIT_SCRATCH_LIMIT;
  const int dev = current_device_slot();
  if (dev < 0) return MGRIT_CUDA_ERROR;
  if (!g_head_scratch_addr[dev]) {
    // In host code the array's name is only a handle; the kernels need its address on the current device.
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_head_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return MGRIT_CUDA_ERROR;
    }
    g_head_scratch_addr[dev] = p;
  }
  // Nothing in the scratch has to start at zero: pass 1 overwrites all B*C + B entries before pass 2 reads them.
  stream_xent(B, H, C, hT, Wc, bc, labels, loss, dhT, dWc, dbc, g_head_scratch_addr[dev], (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? MGRIT_OK : MGRIT_CUDA_ERROR;
}
