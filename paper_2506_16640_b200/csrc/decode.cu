// Decode-shape forward: a few new query rows per sequence against a long key/value cache, sequences of
// different lengths in one batch.  Query t of sequence b sits at position pos = kv_len[b] - q_len + t,
// sees the keys j <= pos, and gets Eq. 1 on its ASEntmax-scaled logits like any row of the full problem
// (n_i = pos + 1).  The path is bound by reading K once from HBM:
//   decode_scores_tc_kernel   (decode_scores_sm100.cu) streams K through TMA and tcgen05, writes
//                             y = a_t (q.k + bias), a_t = (alpha-1) c_t sm_scale, to a score row in the
//                             workspace and the maximum of every chunk of keys;
//   decode_solve_kernel       one CTA per query row: y_max, the candidates above the lower end of the bracket
//                             of App. A (tau >= y_max - 1), Newton from the left on them (e-norm step), then
//                             p = [y - tau]_+^e and O = sum_j p_j v_j as a gather of the support's V rows.
// V is read only on the support.  Rows with more candidates than the CTA's list holds run the same
// Newton iteration and output loop over the whole score row instead.
// All sums are taken in a fixed order: repeated calls give identical bits.
#include "common.cuh"
#include "decode.cuh"

namespace entmax {

namespace {

constexpr int kListSlots = 2048;   // candidate slots of a solve CTA, split evenly among its threads
constexpr int kMaxNewtonD = 64;

// PER consecutive bf16 values (PER = 2 or 4) as floats
template <int PER>
__device__ __forceinline__ void load_bf16_row(const __nv_bfloat16* p, float (&f)[PER]) {
  if constexpr (PER == 4) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(raw.x << 16); f[1] = __uint_as_float(raw.x & 0xffff0000u);
    f[2] = __uint_as_float(raw.y << 16); f[3] = __uint_as_float(raw.y & 0xffff0000u);
  } else {
    const uint32_t raw = *reinterpret_cast<const uint32_t*>(p);
    f[0] = __uint_as_float(raw << 16); f[1] = __uint_as_float(raw & 0xffff0000u);
  }
}

// Sum over the CTA in a fixed order; every thread returns the same value.  `slot` alternates between
// calls so that one barrier per call is enough.
template <int kSolveThreads>
__device__ __forceinline__ float2 block_sum2(float x, float y, float2 (*red)[kSolveThreads / 32], int slot) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    x += __shfl_xor_sync(0xffffffffu, x, o);
    y += __shfl_xor_sync(0xffffffffu, y, o);
  }
  if ((threadIdx.x & 31) == 0) red[slot][threadIdx.x >> 5] = make_float2(x, y);
  __syncthreads();
  float2 s = make_float2(0.f, 0.f);
#pragma unroll
  for (int w = 0; w < kSolveThreads / 32; ++w) {
    s.x += red[slot][w].x;
    s.y += red[slot][w].y;
  }
  return s;
}

template <int D, int kSolveThreads>
__global__ void __launch_bounds__(kSolveThreads) decode_solve_kernel(DecodeArgs a, const __nv_bfloat16* __restrict__ v,
                                                                    const float* __restrict__ scores,
                                                                    const float* __restrict__ chunk_max,
                                                                    __nv_bfloat16* __restrict__ o,
                                                                    float* __restrict__ tau_out,
                                                                    int32_t* __restrict__ support_out,
                                                                    int32_t* __restrict__ status) {
  constexpr int kWarps = kSolveThreads / 32;
  constexpr int kPerThread = kListSlots / kSolveThreads;
  constexpr int kCap = kListSlots;
  constexpr int PER = D / 32;
  __shared__ float cand_y[kCap];      // per-thread slots, then the compact list's p values
  __shared__ int cand_j[kCap];
  __shared__ float list_y[kCap];      // candidates compacted in (thread, slot) order
  __shared__ int list_j[kCap];
  __shared__ float2 red[2][kWarps];
  __shared__ float wmax[kWarps];
  __shared__ int scan[kWarps];
  __shared__ float opart[kWarps][D];
  __shared__ int s_overflow;
  __shared__ float s_tau;
  __shared__ int s_support;
  const int row = blockIdx.x;                       // (b * H + h) * QL + t
  const int t = row % a.QL, bh = row / a.QL, h = bh % a.H, b = bh / a.H;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int len = seq_len(a, b, nullptr);
  const int nv = len - a.QL + t + 1;                // visible keys
  const float* y_row = scores + (size_t)row * a.score_stride;
  if (tid == 0) s_overflow = 0;
  // ---- y_max from the chunk maxima
  float m = -INFINITY;
  const int chunks = (nv + a.chunk_keys - 1) / a.chunk_keys;
  for (int c = tid; c < chunks; c += kSolveThreads) m = fmaxf(m, chunk_max[(size_t)row * a.n_chunks + c]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if (lane == 0) wmax[warp] = m;
  __syncthreads();
  float ymax = wmax[0];
#pragma unroll
  for (int w = 1; w < kWarps; ++w) ymax = fmaxf(ymax, wmax[w]);
  // ---- candidates: y > y_max - 1 (App. A: tau >= y_max - 1), kept per thread in key order
  const float floor_y = ymax - 1.0f;
  int cnt = 0;
  {
    // eight 16-byte loads in flight per thread; a thread meets its keys in increasing order
    const float4* y_row4 = reinterpret_cast<const float4*>(y_row);
    const int groups = (nv + 3) / 4;
    const float4 none = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    for (int g0 = tid; g0 < groups; g0 += 8 * kSolveThreads) {
      float4 yv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int g = g0 + u * kSolveThreads;
        yv[u] = g < groups ? y_row4[g] : none;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float ye[4] = {yv[u].x, yv[u].y, yv[u].z, yv[u].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = 4 * (g0 + u * kSolveThreads) + e;
          if (j < nv && ye[e] > floor_y) {
            if (cnt < kPerThread) {
              cand_y[tid * kPerThread + cnt] = ye[e];
              cand_j[tid * kPerThread + cnt] = j;
            }
            ++cnt;
          }
        }
      }
    }
  }
  if (cnt > kPerThread) s_overflow = 1;
  // ---- compact the candidates in (thread, slot) order
  int incl = cnt < kPerThread ? cnt : kPerThread;
  const int mine = incl;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += up;
  }
  if (lane == 31) scan[warp] = incl;
  __syncthreads();
  const bool dense = s_overflow != 0;
  int base = 0, n_cand = 0;
  for (int w = 0; w < kWarps; ++w) {
    if (w < warp) base += scan[w];
    n_cand += scan[w];
  }
  if (!dense) {
    const int at = base + incl - mine;
    for (int c = 0; c < mine; ++c) {
      list_y[at + c] = cand_y[tid * kPerThread + c];
      list_j[at + c] = cand_j[tid * kPerThread + c];
    }
  }
  __syncthreads();
  if (dense && tid == 0 && status) atomicAdd(status + ENTMAX_ATTN_STATUS_DENSE_ROWS, 1);
  // ---- Newton from the left on f(tau) = sum [y - tau]_+^e - 1, e-norm step
  TauIter st;
  st.tau = st.lo = floor_y;      // y_max - 1, the bracket's lower end (App. A)
  st.hi = ymax;
  float tau = floor_y;
  int support = 0;
  if (!dense) {
    // the first warp alone: shuffles only, no CTA barriers inside the iteration
    if (warp == 0) {
      for (int it = 0; it < kMaxNewtonD; ++it) {
        float s0 = 0.f, s1 = 0.f;
        for (int c = lane; c < n_cand; c += 32) {
          const float d = list_y[c] - st.tau;
          if (d > 0.f) {
            float ye, ye1;
            pow_pair(d, a.expo_class, a.expo, ye, ye1);
            s0 += ye;
            s1 += ye1;
          }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          s0 += __shfl_xor_sync(0xffffffffu, s0, off);
          s1 += __shfl_xor_sync(0xffffffffu, s1, off);
        }
        if (!tau_iter_update(st, s0, s1, a.expo_class, a.expo, 1e-7f)) break;
      }
      tau = st.tau;
      // p of every candidate (0 outside the support), in list order
      int local = 0;
      for (int c = lane; c < n_cand; c += 32) {
        const float d = list_y[c] - tau;
        float ye = 0.f, ye1;
        if (d > 0.f) {
          pow_pair(d, a.expo_class, a.expo, ye, ye1);
          ++local;
        }
        cand_y[c] = ye;
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
      if (lane == 0) {
        s_tau = tau;
        s_support = local;
      }
    }
    __syncthreads();
    tau = s_tau;
    support = s_support;
  } else {
    for (int it = 0; it < kMaxNewtonD; ++it) {
      float s0 = 0.f, s1 = 0.f;
      for (int j = tid; j < nv; j += kSolveThreads) {
        const float d = y_row[j] - st.tau;
        if (d > 0.f) {
          float ye, ye1;
          pow_pair(d, a.expo_class, a.expo, ye, ye1);
          s0 += ye;
          s1 += ye1;
        }
      }
      const float2 s = block_sum2<kSolveThreads>(s0, s1, red, it & 1);
      if (!tau_iter_update(st, s.x, s.y, a.expo_class, a.expo, 1e-7f)) break;
    }
    tau = st.tau;
    __syncthreads();
  }
  // ---- O = sum_j p_j v_j
  const __nv_bfloat16* vbase = v + (size_t)b * a.ksb + (size_t)h * a.ksh + lane * PER;
  float acc[PER];
#pragma unroll
  for (int e = 0; e < PER; ++e) acc[e] = 0.f;
  if (!dense) {
    for (int c = warp; c < n_cand; c += kWarps) {
      const float p = cand_y[c];
      if (p > 0.f) {
        float vf[PER];
        load_bf16_row<PER>(vbase + (size_t)list_j[c] * a.ksn, vf);
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
      }
    }
  } else {
    int local = 0;
    for (int j = warp; j < nv; j += kWarps) {
      const float d = y_row[j] - tau;
      if (d > 0.f) {
        float ye, ye1;
        pow_pair(d, a.expo_class, a.expo, ye, ye1);
        float vf[PER];
        load_bf16_row<PER>(vbase + (size_t)j * a.ksn, vf);
#pragma unroll
        for (int e = 0; e < PER; ++e) acc[e] = fmaf(ye, vf[e], acc[e]);
        ++local;
      }
    }
    if (lane == 0) scan[warp] = local;
    __syncthreads();
    for (int w = 0; w < kWarps; ++w) support += scan[w];
  }
#pragma unroll
  for (int e = 0; e < PER; ++e) opart[warp][lane * PER + e] = acc[e];
  __syncthreads();
  if (tid < D) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) s += opart[w][tid];
    o[(size_t)row * D + tid] = __float2bfloat16(s);
  }
  if (tid == 0) {
    tau_out[row] = tau;
    if (support_out) support_out[row] = support;
  }
}

struct DecodeLayout {
  size_t chunk_max, scores, total;
  size_t score_stride;
  int chunk_keys, n_chunks;
};

// A CTA of the score kernel takes up to 1024 keys, fewer when the problem would otherwise leave SMs idle.
DecodeLayout decode_layout(int B, int H, int QL, int NC) {
  DecodeLayout l;
  const size_t rows = (size_t)B * H * QL;
  l.chunk_keys = 1024;
  while (l.chunk_keys > 128 && (long long)B * H * ((NC + l.chunk_keys - 1) / l.chunk_keys) < 4 * 148) l.chunk_keys /= 2;
  l.n_chunks = (NC + l.chunk_keys - 1) / l.chunk_keys;
  l.score_stride = ((size_t)NC + 31) / 32 * 32;
  size_t off = 0;
  auto take = [&off](size_t bytes) { size_t at = off; off = (off + bytes + 255) / 256 * 256; return at; };
  l.chunk_max = take(rows * l.n_chunks * sizeof(float));
  l.scores = take(rows * l.score_stride * sizeof(float));
  l.total = off;
  return l;
}

int check_decode_params(const entmax_attn_decode_params* p, DecodeArgs* a) {
  if (!p) return ENTMAX_ATTN_EINVAL_NULL;
  if (p->batch < 1 || p->heads < 1 || p->q_len < 1 || p->q_len > ENTMAX_ATTN_DECODE_MAX_Q) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (p->kv_capacity < p->q_len) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (p->head_dim != 64 && p->head_dim != 128) return ENTMAX_ATTN_EINVAL_SHAPE;
  if ((long long)p->batch * p->heads * p->q_len > 0x7fffffffLL / 4) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (!(p->alpha > 1.0f) || !(p->alpha <= kAlphaMax)) return ENTMAX_ATTN_EINVAL_ALPHA;
  if (!(p->sm_scale >= 0.f) || !(p->sm_scale < INFINITY)) return ENTMAX_ATTN_EINVAL_ALPHA;
  a->B = p->batch; a->H = p->heads; a->QL = p->q_len; a->NC = p->kv_capacity; a->D = p->head_dim;
  a->alpha_m1 = p->alpha - 1.0f;
  a->sm_scale = p->sm_scale == 0.f ? 1.0f / sqrtf((float)p->head_dim) : p->sm_scale;
  a->expo = 1.0f / (p->alpha - 1.0f);
  a->expo_class = p->alpha == 2.0f ? kExpo1 : p->alpha == 1.5f ? kExpo2 : p->alpha == 1.25f ? kExpo4 : kExpoGeneral;
  if (p->kv_stride_b == 0 && p->kv_stride_h == 0 && p->kv_stride_n == 0) {
    a->ksn = p->head_dim;
    a->ksh = (int64_t)p->kv_capacity * p->head_dim;
    a->ksb = (int64_t)p->heads * p->kv_capacity * p->head_dim;
  } else {
    a->ksb = p->kv_stride_b; a->ksh = p->kv_stride_h; a->ksn = p->kv_stride_n;
    if (a->ksn < p->head_dim || a->ksh < 1 || a->ksb < 1) return ENTMAX_ATTN_EINVAL_SHAPE;
    if (a->ksn % 8 || a->ksh % 8 || a->ksb % 8) return ENTMAX_ATTN_EINVAL_SHAPE;
  }
  return ENTMAX_ATTN_OK;
}

}  // namespace

}  // namespace entmax

using namespace entmax;

extern "C" size_t entmax_attn_decode_workspace_bytes(const entmax_attn_decode_params* params) {
  DecodeArgs a;
  if (check_decode_params(params, &a) != ENTMAX_ATTN_OK) return 0;
  return decode_layout(a.B, a.H, a.QL, a.NC).total;
}

extern "C" int entmax_attn_decode_fwd(const entmax_attn_decode_params* params, const void* q, const void* k,
                                      const void* v, const int32_t* kv_len, const float* beta, const float* gamma,
                                      const float* delta, const float* alibi_slopes, void* o, float* tau,
                                      int32_t* support_size, void* workspace, size_t workspace_bytes,
                                      int32_t* device_status, void* cuda_stream) {
  DecodeArgs a;
  int rc = check_decode_params(params, &a);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!q || !k || !v || !o || !tau) return ENTMAX_ATTN_EINVAL_NULL;
  const int given = (beta != nullptr) + (gamma != nullptr) + (delta != nullptr);
  if (given != 0 && given != 3) return ENTMAX_ATTN_EINVAL_NULL;
  auto aligned = [](const void* p, uintptr_t m) { return (reinterpret_cast<uintptr_t>(p) & (m - 1)) == 0; };
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) || !aligned(tau, 4)) return ENTMAX_ATTN_EINVAL_ALIGN;
  if ((kv_len && !aligned(kv_len, 4)) || (alibi_slopes && !aligned(alibi_slopes, 4)) ||
      (support_size && !aligned(support_size, 4)))
    return ENTMAX_ATTN_EINVAL_ALIGN;
  const DecodeLayout lay = decode_layout(a.B, a.H, a.QL, a.NC);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < lay.total) return ENTMAX_ATTN_EINVAL_WORKSPACE;
  a.kv_len = kv_len;
  a.alibi = alibi_slopes;
  a.beta = beta; a.gamma = gamma; a.delta = delta;
  a.chunk_keys = lay.chunk_keys;
  a.n_chunks = lay.n_chunks;
  a.score_stride = lay.score_stride;
  int dev = 0, major = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err == cudaSuccess) err = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (err != cudaSuccess) return fail_cuda(err);
  if (major != 10) return ENTMAX_ATTN_EUNSUPPORTED;          // the score kernel needs tcgen05 / TMA
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* chunk_max = reinterpret_cast<float*>(ws + lay.chunk_max);
  float* scores = reinterpret_cast<float*>(ws + lay.scores);
  if (device_status) {
    err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  const int rows = a.B * a.H * a.QL;
  err = launch_decode_scores_tc(a, q, k, scores, chunk_max, device_status, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v);
  __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(o);
  // long rows: more threads per row (more loads in flight); many short rows: smaller CTAs
#define ENTMAX_SOLVE(D, T) \
  decode_solve_kernel<D, T><<<rows, T, 0, stream>>>(a, vb, scores, chunk_max, ob, tau, support_size, device_status)
  if (a.NC >= 16384) {
    if (a.D == 64) ENTMAX_SOLVE(64, 512); else ENTMAX_SOLVE(128, 512);
  } else {
    if (a.D == 64) ENTMAX_SOLVE(64, 256); else ENTMAX_SOLVE(128, 256);
  }
#undef ENTMAX_SOLVE
  err = cudaGetLastError();
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}
