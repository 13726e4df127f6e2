// ASEntmax's content-dependent scale (Sec. 4.1 of the paper): per query token and head
//   beta = softplus(<x, w_beta_h>),  gamma = s tanh(<x, w_gamma_h>),  c = delta_h + beta (log n)^gamma
// evaluated from the layer input x, and the chain rule from dL/dc back to w_beta, w_gamma, delta and x.
// The attention calls take c as a per-query table (entmax_attn_fwd_rowscale) and return dL/dc
// (entmax_attn_bwd_rowscale); these two kernels close the loop around them.  Small, memory-bound work:
// x is read once per call in the forward kernel; the backward kernel recomputes the projections.
#include <cmath>

#include "common.cuh"

namespace entmax {

namespace {

constexpr int kProjThreads = 256;
constexpr int kProjWarps = kProjThreads / 32;
constexpr int kChunk = 64;          // tokens per CTA in the backward kernel
constexpr int kMaxHeads = 64;

struct ProjArgs {
  int B, H, N, dm;
  int causal, n_mode;
  float s;
};

__device__ __forceinline__ float load_x(const float* p) { return *p; }
__device__ __forceinline__ float load_x(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store_x(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_x(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_add(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// the two projections of one token for one head (all 32 lanes get the sums)
template <typename T>
__device__ __forceinline__ void project(const T* xrow, const float* wb, const float* wg, int dm, int lane, float& pb,
                                        float& pg) {
  float sb = 0.f, sg = 0.f;
  for (int t = lane; t < dm; t += 32) {
    const float xv = load_x(xrow + t);
    sb = fmaf(xv, wb[t], sb);
    sg = fmaf(xv, wg[t], sg);
  }
  pb = warp_add(sb);
  pg = warp_add(sg);
}

// beta, gamma, c and the factors of the chain rule, in double (once per token and head: the cost is nothing, and
// c then agrees with the per-head scale table, which is evaluated the same way)
struct ScalePoint {
  double beta, gamma, c, dc_dpb, dc_dpg;
};
__device__ __forceinline__ ScalePoint scale_point(double pb, double pg, double delta, double s, long n_i) {
  ScalePoint r;
  r.beta = pb > 0.0 ? pb + log1p(exp(-pb)) : log1p(exp(pb));
  const double th = tanh(pg);
  r.gamma = s * th;
  r.c = delta;
  r.dc_dpb = 0.0;
  r.dc_dpg = 0.0;
  if (n_i > 1) {
    const double L = log((double)n_i), Lg = pow(L, r.gamma);
    r.c = delta + r.beta * Lg;
    r.dc_dpb = Lg / (1.0 + exp(-pb));                          // d beta / d pre = sigmoid
    r.dc_dpg = r.beta * Lg * log(L) * s * (1.0 - th * th);     // d gamma / d pre = s (1 - tanh^2)
  }
  return r;
}

template <typename T>
__global__ void __launch_bounds__(kProjThreads) scale_proj_fwd_kernel(ProjArgs a, const T* __restrict__ x,
                                                                      const float* __restrict__ w_beta,
                                                                      const float* __restrict__ w_gamma,
                                                                      const float* __restrict__ delta,
                                                                      float* __restrict__ c_rows) {
  const int lane = threadIdx.x & 31;
  const long tokens = (long)a.B * a.N;
  for (long tok = (long)blockIdx.x * kProjWarps + (threadIdx.x >> 5); tok < tokens; tok += (long)gridDim.x * kProjWarps) {
    const long b = tok / a.N, i = tok - b * a.N;
    const long n_i = (a.n_mode || !a.causal) ? a.N : i + 1;
    const T* xrow = x + tok * a.dm;
    for (int h = 0; h < a.H; ++h) {
      float pb, pg;
      project(xrow, w_beta + (size_t)h * a.dm, w_gamma + (size_t)h * a.dm, a.dm, lane, pb, pg);
      if (lane == 0) c_rows[((size_t)b * a.H + h) * a.N + i] = (float)scale_point(pb, pg, delta[h], a.s, n_i).c;
    }
  }
}

// One CTA per chunk of kChunk tokens: first the chain-rule factors of every (token, head) of the chunk into shared
// memory (a warp per token), then every thread owns columns of d_model and sums over the chunk: dw_beta, dw_gamma by one
// atomic per (head, column) and CTA, dx written directly.
template <typename T>
__global__ void __launch_bounds__(kProjThreads) scale_proj_bwd_kernel(ProjArgs a, const T* __restrict__ x,
                                                                      const float* __restrict__ w_beta,
                                                                      const float* __restrict__ w_gamma,
                                                                      const float* __restrict__ delta,
                                                                      const float* __restrict__ dc_rows,
                                                                      float* __restrict__ dw_beta,
                                                                      float* __restrict__ dw_gamma,
                                                                      float* __restrict__ ddelta, T* __restrict__ dx) {
  extern __shared__ float sm[];
  float* gb = sm;                          // [kChunk][H]
  float* gg = sm + kChunk * a.H;           // [kChunk][H]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long tokens = (long)a.B * a.N;
  const long tok0 = (long)blockIdx.x * kChunk;
  const int n_tok = (int)(tokens - tok0 < kChunk ? tokens - tok0 : kChunk);
  for (int tl = warp; tl < n_tok; tl += kProjWarps) {
    const long tok = tok0 + tl;
    const long b = tok / a.N, i = tok - b * a.N;
    const long n_i = (a.n_mode || !a.causal) ? a.N : i + 1;
    const T* xrow = x + tok * a.dm;
    for (int h = 0; h < a.H; ++h) {
      float pb, pg;
      project(xrow, w_beta + (size_t)h * a.dm, w_gamma + (size_t)h * a.dm, a.dm, lane, pb, pg);
      if (lane == 0) {
        const float g = dc_rows[((size_t)b * a.H + h) * a.N + i];
        const ScalePoint pt = scale_point(pb, pg, delta ? delta[h] : 0.0, a.s, n_i);
        gb[tl * a.H + h] = (float)(g * pt.dc_dpb);
        gg[tl * a.H + h] = (float)(g * pt.dc_dpg);
        if (ddelta) atomicAdd(ddelta + h, g);
      }
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < a.dm; col += kProjThreads) {
    // dx of the chunk's tokens at this column
    if (dx) {
      for (int tl = 0; tl < n_tok; ++tl) {
        float acc = 0.f;
        for (int h = 0; h < a.H; ++h)
          acc = fmaf(gb[tl * a.H + h], w_beta[(size_t)h * a.dm + col], fmaf(gg[tl * a.H + h], w_gamma[(size_t)h * a.dm + col], acc));
        store_x(dx + (tok0 + tl) * a.dm + col, acc);
      }
    }
    // dw of every head at this column, summed over the chunk
    for (int h = 0; h < a.H; ++h) {
      float ab = 0.f, ag = 0.f;
      for (int tl = 0; tl < n_tok; ++tl) {
        const float xv = load_x(x + (tok0 + tl) * a.dm + col);
        ab = fmaf(gb[tl * a.H + h], xv, ab);
        ag = fmaf(gg[tl * a.H + h], xv, ag);
      }
      atomicAdd(dw_beta + (size_t)h * a.dm + col, ab);
      atomicAdd(dw_gamma + (size_t)h * a.dm + col, ag);
    }
  }
}

int check_proj(const entmax_attn_proj_params* p, ProjArgs* a) {
  if (!p) return ENTMAX_ATTN_EINVAL_NULL;
  if (p->batch < 1 || p->heads < 1 || p->heads > kMaxHeads || p->seq < 1 || p->d_model < 1) return ENTMAX_ATTN_EINVAL_SHAPE;
  if ((long long)p->batch * p->heads * p->seq > 0x7fffffffLL / 2) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (p->x_dtype != ENTMAX_ATTN_DTYPE_BF16 && p->x_dtype != ENTMAX_ATTN_DTYPE_FP32) return ENTMAX_ATTN_EINVAL_DTYPE;
  if (!(p->gamma_range > 0.f) || !std::isfinite(p->gamma_range)) return ENTMAX_ATTN_EINVAL_ALPHA;
  a->B = p->batch; a->H = p->heads; a->N = p->seq; a->dm = p->d_model;
  a->causal = p->causal ? 1 : 0;
  a->n_mode = p->n_mode ? 1 : 0;
  a->s = p->gamma_range;
  return ENTMAX_ATTN_OK;
}

}  // namespace

}  // namespace entmax

using namespace entmax;

extern "C" {

int entmax_attn_scale_proj_fwd(const entmax_attn_proj_params* params, const void* x, const float* w_beta,
                               const float* w_gamma, const float* delta, float* c_rows, void* cuda_stream) {
  ProjArgs a;
  int rc = check_proj(params, &a);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!x || !w_beta || !w_gamma || !delta || !c_rows) return ENTMAX_ATTN_EINVAL_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const long tokens = (long)a.B * a.N;
  long ctas = (tokens + kProjWarps - 1) / kProjWarps;
  if (ctas > 148L * 16) ctas = 148L * 16;
  if (params->x_dtype == ENTMAX_ATTN_DTYPE_FP32)
    scale_proj_fwd_kernel<float><<<(int)ctas, kProjThreads, 0, stream>>>(a, static_cast<const float*>(x), w_beta, w_gamma, delta,
                                                                        c_rows);
  else
    scale_proj_fwd_kernel<__nv_bfloat16><<<(int)ctas, kProjThreads, 0, stream>>>(a, static_cast<const __nv_bfloat16*>(x), w_beta,
                                                                                w_gamma, delta, c_rows);
  cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}

int entmax_attn_scale_proj_bwd(const entmax_attn_proj_params* params, const void* x, const float* w_beta,
                               const float* w_gamma, const float* d_scale_rows, float* dw_beta, float* dw_gamma,
                               float* ddelta, void* dx, void* cuda_stream) {
  ProjArgs a;
  int rc = check_proj(params, &a);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!x || !w_beta || !w_gamma || !d_scale_rows || !dw_beta || !dw_gamma) return ENTMAX_ATTN_EINVAL_NULL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = cudaMemsetAsync(dw_beta, 0, sizeof(float) * (size_t)a.H * a.dm, stream);
  if (err == cudaSuccess) err = cudaMemsetAsync(dw_gamma, 0, sizeof(float) * (size_t)a.H * a.dm, stream);
  if (err == cudaSuccess && ddelta) err = cudaMemsetAsync(ddelta, 0, sizeof(float) * (size_t)a.H, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  const long tokens = (long)a.B * a.N;
  const int ctas = (int)((tokens + kChunk - 1) / kChunk);
  const size_t smem = sizeof(float) * 2 * kChunk * a.H;
  if (params->x_dtype == ENTMAX_ATTN_DTYPE_FP32)
    scale_proj_bwd_kernel<float><<<ctas, kProjThreads, smem, stream>>>(a, static_cast<const float*>(x), w_beta, w_gamma, nullptr,
                                                                      d_scale_rows, dw_beta, dw_gamma, ddelta,
                                                                      static_cast<float*>(dx));
  else
    scale_proj_bwd_kernel<__nv_bfloat16><<<ctas, kProjThreads, smem, stream>>>(a, static_cast<const __nv_bfloat16*>(x), w_beta,
                                                                              w_gamma, nullptr, d_scale_rows, dw_beta, dw_gamma,
                                                                              ddelta, static_cast<__nv_bfloat16*>(dx));
  err = cudaGetLastError();
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}

}  // extern "C"
