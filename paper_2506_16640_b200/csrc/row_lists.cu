// Per-row kernels of the bf16 path that work on the sparse candidate lists left by the tensor-core
// score sweep (two half-lists per row, see common.cuh): one warp per query row.
//
// Forward: exact threshold on the candidates (Eq. 1 with the sum-to-one condition; Newton from the
// left of the root, see dense_rows.cu), probabilities, and O_i = sum_j p_ij v_j as a gather over the
// support only -- every zero of P is skipped, not just all-zero tiles.
// Backward: the entmax Jacobian dS = u (dP - <u,dP>/sum u), u = p^(2-alpha), on the support, dQ by
// gathering K rows, dK / dV by vector atomics into fp32 accumulators.
#include "common.cuh"

namespace entmax {

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kSlots = kListCap / 32;
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

template <int PER>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&x)[PER]) {
  if constexpr (PER == 2) {
    float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
    x[0] = t.x; x[1] = t.y;
  } else {
    uint2 raw = *reinterpret_cast<const uint2*>(p);
    float2 t0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
    float2 t1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
    x[0] = t0.x; x[1] = t0.y; x[2] = t1.x; x[3] = t1.y;
  }
}
template <int PER>
__device__ __forceinline__ void store_bf16(__nv_bfloat16* p, const float (&x)[PER]) {
  if constexpr (PER == 2) {
    *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(x[0], x[1]);
  } else {
    __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 raw;
    raw.x = *reinterpret_cast<uint32_t*>(&a);
    raw.y = *reinterpret_cast<uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = raw;
  }
}
template <int PER>
__device__ __forceinline__ void atomic_add_slice(float* p, const float (&x)[PER]) {
  if constexpr (PER == 2) atomicAdd(reinterpret_cast<float2*>(p), make_float2(x[0], x[1]));
  else atomicAdd(reinterpret_cast<float4*>(p), make_float4(x[0], x[1], x[2], x[3]));
}

__device__ __forceinline__ void push_dense_row(int grow, int32_t* fb_count, int32_t* fb_list, int32_t* status) {
  const int slot = atomicAdd(fb_count, 1);
  fb_list[slot] = grow;
  if (status) atomicAdd(status + ENTMAX_ATTN_STATUS_DENSE_ROWS, 1);
}

// Bitonic sort of 32*S (key j, value y) pairs held as S registers per lane (element index = 32*s + lane),
// ascending by key.  Keys are distinct key indices (padding uses INT_MAX and sorts to the end).
template <int S>
__device__ __forceinline__ void sort_by_key(int (&jj)[S], float (&y)[S], int lane) {
#pragma unroll
  for (int k = 2; k <= 32 * S; k <<= 1) {
#pragma unroll
    for (int st = k >> 1; st > 0; st >>= 1) {
      if (st >= 32) {
        // partner sits in another register of the same lane
#pragma unroll
        for (int s = 0; s < S; ++s) {
          const int ps = s ^ (st >> 5);
          if (ps > s) {
            const bool up = (((32 * s) & k) == 0);
            const bool swap = up ? (jj[s] > jj[ps]) : (jj[s] < jj[ps]);
            const int tj = swap ? jj[ps] : jj[s];
            const float ty = swap ? y[ps] : y[s];
            jj[ps] = swap ? jj[s] : jj[ps];
            y[ps] = swap ? y[s] : y[ps];
            jj[s] = tj;
            y[s] = ty;
          }
        }
      } else {
#pragma unroll
        for (int s = 0; s < S; ++s) {
          const int idx = 32 * s + lane;
          const int oj = __shfl_xor_sync(0xffffffffu, jj[s], st);
          const float oy = __shfl_xor_sync(0xffffffffu, y[s], st);
          const bool up = ((idx & k) == 0);
          const bool lower = ((lane & st) == 0);
          // the lower index keeps the smaller key when sorting upwards, the larger one otherwise
          const bool take_other = (lower == up) ? (oj < jj[s]) : (oj > jj[s]);
          jj[s] = take_other ? oj : jj[s];
          y[s] = take_other ? oy : y[s];
        }
      }
    }
  }
}

// One query row on S*32 candidate slots: exact threshold (Eq. 1 with the sum-to-one condition), the
// probabilities, O_i as a gather over the support, and the support written back sorted by key index.
// The candidates are sorted by key index first and Newton starts at the bracket's lower end
// (App. A: tau >= y_max - 1), so the result does not depend on the order or on the surplus entries
// the sweep happened to leave in the lists.
template <int D, int S>
__device__ __forceinline__ void solve_row(const Problem& p, const __nv_bfloat16* __restrict__ vbase, Entry* list, int c0,
                                          int c1, float a, __nv_bfloat16* o_row, float* tau_slot, int32_t* cnt_slot,
                                          int lane) {
  constexpr int PER = D / 32;
  float y[S];
  int jj[S];
  float ymax = -INFINITY;
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const int e = lane + 32 * s;                   // dense numbering: first half-list, then second
    y[s] = -INFINITY;
    jj[s] = 0x7fffffff;
    if (e < c0 + c1) {
      const Entry en = list[e < c0 ? e : kHalfCap + e - c0];
      y[s] = a * en.y;
      jj[s] = en.j;
    }
    ymax = fmaxf(ymax, y[s]);
  }
  ymax = warp_max(ymax);
  __syncwarp();   // every slot is in registers before the compaction below overwrites the list
  sort_by_key<S>(jj, y, lane);
  float tau = ymax - 1.0f;
  for (int it = 0; it < kMaxNewton; ++it) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int s = 0; s < S; ++s) {
      const float d = y[s] - tau;
      if (d > 0.f) {
        float ye, ye1;
        pow_pair(d, p.expo_class, p.expo, ye, ye1);
        s0 += ye;
        s1 += ye1;
      }
    }
    s0 = warp_sum(s0);
    s1 = warp_sum(s1);
    if (!(s0 > 1.0f) || !(s1 > 0.f)) break;
    const float step = (s0 - 1.0f) / (p.expo * s1);
    const float next = tau + step;
    if (!(next > tau)) break;
    tau = next;
    if (step <= 1e-7f * fmaxf(1.0f, fabsf(tau))) break;
  }
  float acc[PER];
#pragma unroll
  for (int t = 0; t < PER; ++t) acc[t] = 0.f;
  int kept = 0;
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const float d = y[s] - tau;
    float pe = 0.f, pe1;
    if (d > 0.f) pow_pair(d, p.expo_class, p.expo, pe, pe1);
    const unsigned m = __ballot_sync(0xffffffffu, d > 0.f);
    // compact the list to the exact support, y in Eq. 1's units
    if (d > 0.f) {
      const int pos = kept + __popc(m & ((1u << lane) - 1u));
      list[pos].y = y[s];
      list[pos].j = jj[s];
    }
    kept += __popc(m);
    unsigned rest = m;
    while (rest) {
      const int src = __ffs(rest) - 1;
      rest &= rest - 1;
      const float pj = __shfl_sync(0xffffffffu, pe, src);
      const int kj = __shfl_sync(0xffffffffu, jj[s], src);
      float vs[PER];
      load_bf16<PER>(vbase + (size_t)kj * p.sn, vs);
#pragma unroll
      for (int t = 0; t < PER; ++t) acc[t] = fmaf(pj, vs[t], acc[t]);
    }
  }
  store_bf16<PER>(o_row, acc);
  if (lane == 0) {
    *tau_slot = tau;
    *cnt_slot = kept;
  }
}

template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32) row_fwd_kernel(Problem p, const __nv_bfloat16* __restrict__ v,
                                                                    const float* __restrict__ scale,
                                                                    int32_t* __restrict__ row_cnt,
                                                                    const int32_t* __restrict__ half_cnt,
                                                                    Entry* __restrict__ entries,
                                                                    __nv_bfloat16* __restrict__ o,
                                                                    float* __restrict__ tau_out, int32_t* fb_count,
                                                                    int32_t* fb_list, int32_t* status) {
  constexpr int PER = D / 32;
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  for (int grow = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); grow < total; grow += gridDim.x * kWarpsPerCta) {
    const int c0 = half_cnt[2 * (size_t)grow], c1 = half_cnt[2 * (size_t)grow + 1];
    if (c0 < 0 || c1 < 0 || c0 + c1 == 0) {
      if (lane == 0) {
        row_cnt[grow] = -2;
        push_dense_row(grow, fb_count, fb_list, status);
      }
      continue;
    }
    const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
    const float a = (p.alpha - 1.0f) * (scale[(size_t)h * p.N + i] * p.sm_scale);
    Entry* list = entries + (size_t)grow * kListCap;
    const __nv_bfloat16* vbase = v + (size_t)b * p.sb + (size_t)h * p.sh + lane * PER;
    __nv_bfloat16* o_row = o + (size_t)b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + lane * PER;
    const int n = c0 + c1;
    if (n <= 32) solve_row<D, 1>(p, vbase, list, c0, c1, a, o_row, tau_out + grow, row_cnt + grow, lane);
    else if (n <= 64) solve_row<D, 2>(p, vbase, list, c0, c1, a, o_row, tau_out + grow, row_cnt + grow, lane);
    else if (n <= 128) solve_row<D, 4>(p, vbase, list, c0, c1, a, o_row, tau_out + grow, row_cnt + grow, lane);
    else solve_row<D, kSlots>(p, vbase, list, c0, c1, a, o_row, tau_out + grow, row_cnt + grow, lane);
  }
}

template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32) row_bwd_kernel(
    Problem p, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ scale,
    const float* __restrict__ tau_in, const int32_t* __restrict__ half_cnt, const Entry* __restrict__ entries,
    __nv_bfloat16* __restrict__ dq, float* __restrict__ acc_dk, float* __restrict__ acc_dv, int32_t* fb_count,
    int32_t* fb_list, int32_t* status) {
  constexpr int PER = D / 32;
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  for (int grow = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); grow < total; grow += gridDim.x * kWarpsPerCta) {
    const int c0 = half_cnt[2 * (size_t)grow], c1 = half_cnt[2 * (size_t)grow + 1];
    if (c0 < 0 || c1 < 0) {
      if (lane == 0) push_dense_row(grow, fb_count, fb_list, status);
      continue;
    }
    const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
    const float g = scale[(size_t)h * p.N + i] * p.sm_scale;
    const float a = (p.alpha - 1.0f) * g;
    const float tau = tau_in[grow];
    const size_t hbase = (size_t)b * p.sb + (size_t)h * p.sh + lane * PER;
    float qs[PER], gs[PER];
    load_bf16<PER>(q + hbase + (size_t)i * p.sn, qs);
    load_bf16<PER>(d_o + hbase + (size_t)i * p.sn, gs);
    const Entry* list = entries + (size_t)grow * kListCap;
    float yv[kSlots], dpv[kSlots];
    int jj[kSlots];
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      const int idx = lane + 32 * s;
      yv[s] = -1.0f;
      jj[s] = 0;
      dpv[s] = 0.f;
      if ((idx & (kHalfCap - 1)) < (idx < kHalfCap ? c0 : c1)) {
        const Entry e = list[idx];
        yv[s] = fmaf(a, e.y, -tau);
        jj[s] = e.j;
      }
    }
    // dP_ij = <dO_i, v_j> on the support
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      unsigned rest = __ballot_sync(0xffffffffu, yv[s] > 0.f);
      while (rest) {
        const int src = __ffs(rest) - 1;
        rest &= rest - 1;
        const int kj = __shfl_sync(0xffffffffu, jj[s], src);
        float vs[PER];
        load_bf16<PER>(v + hbase + (size_t)kj * p.sn, vs);
        float dp = 0.f;
#pragma unroll
        for (int t = 0; t < PER; ++t) dp = fmaf(gs[t], vs[t], dp);
        dp = warp_sum(dp);
        if (lane == src) dpv[s] = dp;
      }
    }
    float pe[kSlots], u[kSlots];
    float su = 0.f, sud = 0.f;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      pe[s] = 0.f;
      u[s] = 0.f;
      if (yv[s] > 0.f) pow_pair(yv[s], p.expo_class, p.expo, pe[s], u[s]);
      su += u[s];
      sud += u[s] * dpv[s];
    }
    su = warp_sum(su);
    sud = warp_sum(sud);
    const float rho = su > 0.f ? sud / su : 0.f;
    float acc[PER];
#pragma unroll
    for (int t = 0; t < PER; ++t) acc[t] = 0.f;
    const size_t arow = (size_t)bh * p.N;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      const float gds_own = g * u[s] * (dpv[s] - rho);
      unsigned rest = __ballot_sync(0xffffffffu, yv[s] > 0.f);
      while (rest) {
        const int src = __ffs(rest) - 1;
        rest &= rest - 1;
        const int kj = __shfl_sync(0xffffffffu, jj[s], src);
        const float gds = __shfl_sync(0xffffffffu, gds_own, src);
        const float pj = __shfl_sync(0xffffffffu, pe[s], src);
        float ks[PER], dkv[PER], dvv[PER];
        load_bf16<PER>(k + hbase + (size_t)kj * p.sn, ks);
#pragma unroll
        for (int t = 0; t < PER; ++t) {
          acc[t] = fmaf(gds, ks[t], acc[t]);
          dkv[t] = gds * qs[t];
          dvv[t] = pj * gs[t];
        }
        atomic_add_slice<PER>(acc_dk + (arow + kj) * D + lane * PER, dkv);
        atomic_add_slice<PER>(acc_dv + (arow + kj) * D + lane * PER, dvv);
      }
    }
    store_bf16<PER>(dq + hbase + (size_t)i * p.sn, acc);
  }
}

inline int row_grid(const Problem& p) {
  const long total = (long)p.B * p.H * p.N;
  const long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  const long cap = 148L * 8 * 8;
  return (int)(ctas < cap ? ctas : cap);
}

}  // namespace

cudaError_t launch_row_fwd(const Problem& p, const void* v, const float* scale, int32_t* row_cnt,
                           const int32_t* half_cnt, const float* half_thr, Entry* entries, void* o, float* tau,
                           int32_t* fb_count, int32_t* fb_list, int32_t* status, cudaStream_t stream) {
  const int grid = row_grid(p);
  if (p.D == 64)
    row_fwd_kernel<64><<<grid, kWarpsPerCta * 32, 0, stream>>>(p, (const __nv_bfloat16*)v, scale, row_cnt, half_cnt,
                                                              entries, (__nv_bfloat16*)o, tau, fb_count, fb_list, status);
  else
    row_fwd_kernel<128><<<grid, kWarpsPerCta * 32, 0, stream>>>(p, (const __nv_bfloat16*)v, scale, row_cnt, half_cnt,
                                                               entries, (__nv_bfloat16*)o, tau, fb_count, fb_list, status);
  return cudaGetLastError();
}

cudaError_t launch_row_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                           const float* scale, const float* tau, const int32_t* half_cnt, Entry* entries, void* dq,
                           float* acc_dk, float* acc_dv, int32_t* fb_count, int32_t* fb_list, int32_t* status,
                           cudaStream_t stream) {
  const int grid = row_grid(p);
  if (p.D == 64)
    row_bwd_kernel<64><<<grid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, fb_count, fb_list, status);
  else
    row_bwd_kernel<128><<<grid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, fb_count, fb_list, status);
  return cudaGetLastError();
}

}  // namespace entmax
