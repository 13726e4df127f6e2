// Dense-row path on CUDA cores: one CTA per query row, every visible key visited.
//
// Used for (1) float32 problems, where fp32 FMA dot products meet the tighter threshold tolerance that
// bf16 tensor-core inputs cannot, and (2) the rows of a bf16 problem whose support does not fit the
// sparse per-row list of the tensor-core sweep.  Also holds the ASEntmax scale-table kernel and the
// gradient store kernel.
//
// Threshold solve: f(tau) = sum_j [y_j - tau]_+^e - 1 with y = (alpha-1) s and e = 1/(alpha-1) >= 1 is
// convex and decreasing (Eq. 1 of the paper with the sum-to-one condition).  Newton steps started at
// the lower end of the paper's bracket, tau0 = y_max - 1 (App. A), therefore never overshoot the root
// and converge monotonically; no bisection safeguard is needed.
#include "common.cuh"

namespace entmax {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxNewton = 400;

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

// red: kWarps*2 floats of shared memory.  Every thread gets both block sums.
__device__ __forceinline__ float2 block_sum2(float a, float b, float* red) {
  a = warp_sum(a);
  b = warp_sum(b);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) { red[w] = a; red[kWarps + w] = b; }
  __syncthreads();
  float ra = 0.f, rb = 0.f;
#pragma unroll
  for (int i = 0; i < kWarps; ++i) { ra += red[i]; rb += red[kWarps + i]; }
  return make_float2(ra, rb);
}
__device__ __forceinline__ float block_max(float a, float* red) {
  a = warp_max(a);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = a;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int i = 1; i < kWarps; ++i) r = fmaxf(r, red[i]);
  return r;
}

struct RowCtx {
  int grow, bh, b, h, i, nv;
  float c, a, g;
  float slope;  // ALiBi slope in dot-product units (m_h / sm_scale), 0 without ALiBi
  size_t base;  // element offset of (b, h, 0, 0)
};

__device__ __forceinline__ RowCtx make_row(const Problem& p, const float* scale, int grow) {
  RowCtx r;
  r.grow = grow;
  r.bh = grow / p.N;
  r.i = grow - r.bh * p.N;
  r.b = r.bh / p.H;
  r.h = r.bh - r.b * p.H;
  r.nv = p.causal ? r.i + 1 : p.N;
  r.c = scale[(size_t)r.b * p.scale_sb + (size_t)r.h * p.N + r.i];
  r.g = r.c * p.sm_scale;
  r.a = (p.alpha - 1.0f) * r.g;
  r.slope = p.alibi ? p.alibi[r.h] / p.sm_scale : 0.f;
  r.base = (size_t)r.b * p.sb + (size_t)r.h * p.sh;
  return r;
}

// y_j = a_i <q_i,k_j> for every visible key into ybuf; returns the row maximum (block-wide).
template <typename T, int D>
__device__ __forceinline__ float score_pass(const Problem& p, const RowCtx& r, const T* k, const float (&qs)[D / 32],
                                            float* ybuf, float* red) {
  constexpr int PER = D / 32;
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  float wmax = -INFINITY;
  for (int j = w; j < r.nv; j += kWarps) {
    float ks[PER];
    load_slice<PER>(k + r.base + (size_t)j * p.sn + l * PER, ks);
    float dot = 0.f;
#pragma unroll
    for (int t = 0; t < PER; ++t) dot = fmaf(qs[t], ks[t], dot);
    dot = warp_sum(dot);
    // ALiBi: the logit is sm_scale * (dot - slope |i - j|) with slope = m_h / sm_scale
    if (r.slope != 0.f) dot -= r.slope * fabsf((float)(j - r.i));
    float y = r.a * dot;
    if (l == 0) ybuf[j] = y;
    wmax = fmaxf(wmax, y);
  }
  return block_max(wmax, red);
}

__device__ __forceinline__ float newton_tau(const Problem& p, const float* ybuf, int nv, float ymax, float* red) {
  TauIter st = tau_iter_start(ymax);
  for (int it = 0; it < kMaxNewton; ++it) {
    float s0 = 0.f, s1 = 0.f;
    for (int j = threadIdx.x; j < nv; j += kThreads) {
      float y = ybuf[j] - st.tau;
      if (y > 0.f) {
        float ye, ye1;
        pow_pair(y, p.expo_class, p.expo, ye, ye1);
        s0 += ye;
        s1 += ye1;
      }
    }
    float2 s = block_sum2(s0, s1, red);
    if (!tau_iter_update(st, s.x, s.y, p.expo_class, p.expo, 1e-7f)) break;
  }
  return st.tau;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) dense_fwd_kernel(Problem p, const T* __restrict__ q, const T* __restrict__ k,
                                                             const T* __restrict__ v, const float* __restrict__ scale,
                                                             T* __restrict__ o, float* __restrict__ tau_out,
                                                             int32_t* __restrict__ row_cnt, int32_t* __restrict__ dense_cnt,
                                                             Entry* __restrict__ entries,
                                                             const int32_t* __restrict__ row_list,
                                                             const int32_t* __restrict__ row_count,
                                                             float* __restrict__ scratch, size_t scratch_floats) {
  constexpr int PER = D / 32;
  __shared__ float red[2 * kWarps];
  __shared__ float opart[kWarps][D];
  __shared__ int supp_count;
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  const int total = row_list ? *row_count : p.B * p.H * p.N;
  float* ybuf = scratch + (size_t)blockIdx.x * scratch_floats;
  for (int ridx = blockIdx.x; ridx < total; ridx += gridDim.x) {
    const RowCtx r = make_row(p, scale, row_list ? row_list[ridx] : ridx);
    float qs[PER];
    load_slice<PER>(q + r.base + (size_t)r.i * p.sn + l * PER, qs);
    if (threadIdx.x == 0) supp_count = 0;
    const float ymax = score_pass<T, D>(p, r, k, qs, ybuf, red);
    const float tau = newton_tau(p, ybuf, r.nv, ymax, red);
    float acc[PER];
#pragma unroll
    for (int t = 0; t < PER; ++t) acc[t] = 0.f;
    Entry* list = entries ? entries + (size_t)r.grow * kListCap : nullptr;
    for (int j = w; j < r.nv; j += kWarps) {
      const float yj = ybuf[j];
      const float y = yj - tau;
      if (y > 0.f) {
        float pe, pe1;
        pow_pair(y, p.expo_class, p.expo, pe, pe1);
        float vs[PER];
        load_slice<PER>(v + r.base + (size_t)j * p.sn + l * PER, vs);
#pragma unroll
        for (int t = 0; t < PER; ++t) acc[t] = fmaf(pe, vs[t], acc[t]);
        if (l == 0) {
          int slot = atomicAdd(&supp_count, 1);
          if (list && slot < kListCap) { list[slot].y = yj; list[slot].j = j; }
        }
      }
    }
#pragma unroll
    for (int t = 0; t < PER; ++t) opart[w][l * PER + t] = acc[t];
    __syncthreads();
    if (threadIdx.x < D / PER) {
      float out[PER];
#pragma unroll
      for (int t = 0; t < PER; ++t) {
        float s = 0.f;
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) s += opart[ww][threadIdx.x * PER + t];
        out[t] = s;
      }
      store_slice<PER>(o + r.base + (size_t)r.i * p.sn + threadIdx.x * PER, out);
    }
    if (threadIdx.x == 0) {
      tau_out[r.grow] = tau;
      if (row_cnt) row_cnt[r.grow] = supp_count <= kListCap ? supp_count : -2;
      // a support too long for the list: its size alone is kept (same place and form as the dense-tile kernel's)
      if (dense_cnt && supp_count > kListCap) { dense_cnt[2 * (size_t)r.grow] = supp_count; dense_cnt[2 * (size_t)r.grow + 1] = 0; }
    }
    __syncthreads();
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) dense_bwd_kernel(Problem p, const T* __restrict__ q, const T* __restrict__ k,
                                                             const T* __restrict__ v, const T* __restrict__ d_o,
                                                             const float* __restrict__ scale, const float* __restrict__ tau_in,
                                                             T* __restrict__ dq, float* __restrict__ acc_dk,
                                                             float* __restrict__ acc_dv, float* __restrict__ dc_rows,
                                                             const int32_t* __restrict__ row_list,
                                                             const int32_t* __restrict__ row_count,
                                                             float* __restrict__ scratch, size_t scratch_floats) {
  constexpr int PER = D / 32;
  __shared__ float red[2 * kWarps];
  __shared__ float qpart[kWarps][D];
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  const int total = row_list ? *row_count : p.B * p.H * p.N;
  float* ybuf = scratch + (size_t)blockIdx.x * scratch_floats;
  float* dpbuf = ybuf + scratch_floats / 2;
  for (int ridx = blockIdx.x; ridx < total; ridx += gridDim.x) {
    const RowCtx r = make_row(p, scale, row_list ? row_list[ridx] : ridx);
    float qs[PER], gs[PER];
    load_slice<PER>(q + r.base + (size_t)r.i * p.sn + l * PER, qs);
    load_slice<PER>(d_o + r.base + (size_t)r.i * p.sn + l * PER, gs);
    (void)score_pass<T, D>(p, r, k, qs, ybuf, red);
    const float tau = tau_in[r.grow];
    // sum_j u_ij and sum_j u_ij dP_ij over the support
    float su = 0.f, sud = 0.f;
    for (int j = w; j < r.nv; j += kWarps) {
      const float y = ybuf[j] - tau;
      if (y > 0.f) {
        float vs[PER];
        load_slice<PER>(v + r.base + (size_t)j * p.sn + l * PER, vs);
        float dp = 0.f;
#pragma unroll
        for (int t = 0; t < PER; ++t) dp = fmaf(gs[t], vs[t], dp);
        dp = warp_sum(dp);
        float pe, u;
        pow_pair(y, p.expo_class, p.expo, pe, u);
        if (l == 0) { dpbuf[j] = dp; su += u; sud += u * dp; }
      }
    }
    const float2 s = block_sum2(su, sud, red);
    const float rho = s.x > 0.f ? s.y / s.x : 0.f;
    float dcp = 0.f;                                  // sum_j dS_ij y_ij (lane 0 of every warp)
    float acc[PER];
#pragma unroll
    for (int t = 0; t < PER; ++t) acc[t] = 0.f;
    const size_t arow = (size_t)r.bh * p.N;
    for (int j = w; j < r.nv; j += kWarps) {
      const float y = ybuf[j] - tau;
      if (y > 0.f) {
        float pe, u;
        pow_pair(y, p.expo_class, p.expo, pe, u);
        const float gds = r.g * u * (dpbuf[j] - rho);
        if (l == 0) dcp = fmaf(u * (dpbuf[j] - rho), ybuf[j], dcp);
        float ks[PER], dkv[PER], dvv[PER];
        load_slice<PER>(k + r.base + (size_t)j * p.sn + l * PER, ks);
#pragma unroll
        for (int t = 0; t < PER; ++t) {
          acc[t] = fmaf(gds, ks[t], acc[t]);
          dkv[t] = gds * qs[t];
          dvv[t] = pe * gs[t];
        }
        atomic_add_slice<PER>(acc_dk + (arow + j) * D + l * PER, dkv);
        atomic_add_slice<PER>(acc_dv + (arow + j) * D + l * PER, dvv);
      }
    }
#pragma unroll
    for (int t = 0; t < PER; ++t) qpart[w][l * PER + t] = acc[t];
    __syncthreads();
    if (threadIdx.x < D / PER) {
      float out[PER];
#pragma unroll
      for (int t = 0; t < PER; ++t) {
        float sacc = 0.f;
#pragma unroll
        for (int ww = 0; ww < kWarps; ++ww) sacc += qpart[ww][threadIdx.x * PER + t];
        out[t] = sacc;
      }
      store_slice<PER>(dq + r.base + (size_t)r.i * p.sn + threadIdx.x * PER, out);
    }
    if (dc_rows) {
      // dL/dc_i = sum_j dS_ij z_ij, z_ij = y_ij / ((alpha-1) c_i)  (y = (alpha-1) c z)
      const float2 t = block_sum2(dcp, 0.f, red);
      const float denom = (p.alpha - 1.0f) * r.c;
      if (threadIdx.x == 0) dc_rows[r.grow] = denom != 0.f ? t.x / denom : 0.f;
    }
    __syncthreads();
  }
}

// dbeta_h, dgamma_h, ddelta_h from the per-row scale gradients: c_i = delta + beta L^gamma with L = ln n_i
// (rows with n_i = 1 have c_i = delta), so d/ddelta = 1, d/dbeta = L^gamma, d/dgamma = beta L^gamma ln L.
// One CTA per head, fp64 accumulation in a fixed order (reproducible).
__global__ void __launch_bounds__(256) scale_grad_kernel(Problem p, const float* __restrict__ beta,
                                                        const float* __restrict__ gamma,
                                                        const float* __restrict__ dc_rows, float* __restrict__ dbeta,
                                                        float* __restrict__ dgamma, float* __restrict__ ddelta) {
  __shared__ double red[3][256];
  const int h = blockIdx.x;
  const double b = beta[h], g = gamma[h];
  double sb = 0.0, sg = 0.0, sd = 0.0;
  for (long t = threadIdx.x; t < (long)p.B * p.N; t += blockDim.x) {
    const long bb = t / p.N;
    const int i = (int)(t - bb * p.N);
    const double dc = dc_rows[((size_t)bb * p.H + h) * p.N + i];
    const long n = (p.n_mode || !p.causal) ? p.N : i + 1;
    sd += dc;
    if (n > 1) {
      const double L = log((double)n);
      const double Lg = pow(L, g);
      sb += dc * Lg;
      sg += dc * b * Lg * log(L);
    }
  }
  red[0][threadIdx.x] = sb;
  red[1][threadIdx.x] = sg;
  red[2][threadIdx.x] = sd;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      red[0][threadIdx.x] += red[0][threadIdx.x + o];
      red[1][threadIdx.x] += red[1][threadIdx.x + o];
      red[2][threadIdx.x] += red[2][threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    dbeta[h] = (float)red[0][0];
    dgamma[h] = (float)red[1][0];
    ddelta[h] = (float)red[2][0];
  }
}

// c_i = delta_h + beta_h (ln n_i)^gamma_h in fp64, rounded once to fp32 (Eq. "asentmax").
__global__ void scale_table_kernel(Problem p, const float* __restrict__ beta, const float* __restrict__ gamma,
                                   const float* __restrict__ delta, float* __restrict__ scale,
                                   int32_t* __restrict__ status) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= p.H * p.N) return;
  float c = 1.0f;
  if (p.has_scale) {
    const int h = idx / p.N, i = idx - h * p.N;
    const long n = (p.n_mode || !p.causal) ? p.N : i + 1;
    double cd = (double)delta[h];
    if (n > 1) cd += (double)beta[h] * pow(log((double)n), (double)gamma[h]);
    c = (float)cd;
    if (!isfinite(c) && status) atomicOr(status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_BAD_SCALE);
  }
  scale[idx] = c;
}

template <typename T>
__global__ void store_grad_kernel(Problem p, const float* __restrict__ acc, T* __restrict__ out) {
  const size_t total4 = (size_t)p.B * p.H * p.N * p.D / 4;
  for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < total4; t += (size_t)gridDim.x * blockDim.x) {
    const size_t e = t * 4;
    const int dcol = (int)(e % p.D);
    const size_t row = e / p.D;
    const int i = (int)(row % p.N);
    const size_t bh = row / p.N;
    const int h = (int)(bh % p.H);
    const size_t b = bh / p.H;
    float x[4];
    load_slice<4>(acc + e, x);
    store_slice<4>(out + b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + dcol, x);
  }
}

}  // namespace

cudaError_t launch_scale_table(const Problem& p, const float* beta, const float* gamma, const float* delta,
                               float* scale, int32_t* status, cudaStream_t stream) {
  const int total = p.H * p.N;
  scale_table_kernel<<<(total + 255) / 256, 256, 0, stream>>>(p, beta, gamma, delta, scale, status);
  return cudaGetLastError();
}

cudaError_t launch_dense_fwd(const Problem& p, const void* q, const void* k, const void* v, const float* scale,
                             void* o, float* tau, int32_t* row_cnt, int32_t* dense_cnt, Entry* entries,
                             const int32_t* row_list, const int32_t* row_count, float* scratch, size_t scratch_floats,
                             int ctas, cudaStream_t stream) {
#define ENTMAX_LAUNCH(T, D)                                                                                        \
  dense_fwd_kernel<T, D><<<ctas, kThreads, 0, stream>>>(p, (const T*)q, (const T*)k, (const T*)v, scale, (T*)o, \
                                                        tau, row_cnt, dense_cnt, entries, row_list, row_count, scratch, \
                                                        scratch_floats)
  if (p.dtype == ENTMAX_ATTN_DTYPE_FP32) {
    if (p.D == 64) ENTMAX_LAUNCH(float, 64); else ENTMAX_LAUNCH(float, 128);
  } else {
    if (p.D == 64) ENTMAX_LAUNCH(__nv_bfloat16, 64); else ENTMAX_LAUNCH(__nv_bfloat16, 128);
  }
#undef ENTMAX_LAUNCH
  return cudaGetLastError();
}

cudaError_t launch_dense_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                             const float* scale, const float* tau, void* dq, float* acc_dk, float* acc_dv,
                             float* dc_rows, const int32_t* row_list, const int32_t* row_count, float* scratch,
                             size_t scratch_floats, int ctas, cudaStream_t stream) {
#define ENTMAX_LAUNCH(T, D)                                                                                      \
  dense_bwd_kernel<T, D><<<ctas, kThreads, 0, stream>>>(p, (const T*)q, (const T*)k, (const T*)v, (const T*)d_o, \
                                                        scale, tau, (T*)dq, acc_dk, acc_dv, dc_rows, row_list,    \
                                                        row_count,                                                 \
                                                        scratch, scratch_floats)
  if (p.dtype == ENTMAX_ATTN_DTYPE_FP32) {
    if (p.D == 64) ENTMAX_LAUNCH(float, 64); else ENTMAX_LAUNCH(float, 128);
  } else {
    if (p.D == 64) ENTMAX_LAUNCH(__nv_bfloat16, 64); else ENTMAX_LAUNCH(__nv_bfloat16, 128);
  }
#undef ENTMAX_LAUNCH
  return cudaGetLastError();
}

cudaError_t launch_scale_grad(const Problem& p, const float* beta, const float* gamma, const float* dc_rows,
                              float* dbeta, float* dgamma, float* ddelta, cudaStream_t stream) {
  scale_grad_kernel<<<p.H, 256, 0, stream>>>(p, beta, gamma, dc_rows, dbeta, dgamma, ddelta);
  return cudaGetLastError();
}

cudaError_t launch_store_grad(const Problem& p, const float* acc, void* out, cudaStream_t stream) {
  const size_t total4 = (size_t)p.B * p.H * p.N * p.D / 4;
  const int blocks = (int)((total4 + 255) / 256 < 148 * 16 ? (total4 + 255) / 256 : 148 * 16);
  if (p.dtype == ENTMAX_ATTN_DTYPE_FP32) store_grad_kernel<float><<<blocks, 256, 0, stream>>>(p, acc, (float*)out);
  else store_grad_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(p, acc, (__nv_bfloat16*)out);
  return cudaGetLastError();
}

}  // namespace entmax
