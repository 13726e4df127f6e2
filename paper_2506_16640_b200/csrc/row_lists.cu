// Per-row kernels of the bf16 path that work on the sparse candidate lists left by the tensor-core
// score sweep (two half-lists per row, see common.cuh).
//
// Forward: exact threshold on the candidates (Eq. 1 with the sum-to-one condition), probabilities, and
// O_i = sum_j p_ij v_j as a gather over the support only -- every zero of P is skipped, not just
// all-zero tiles.  A warp takes 16 consecutive rows and serves them by list length (8, 16 or 32 lanes per
// row).  alpha = 1.5 and alpha = 2 use the closed form on the sorted candidates (solve_rows_closed); other
// exponents iterate (Newton from the left of the root, see dense_rows.cu) in two stages.
// Backward: the entmax Jacobian dS = u (dP - <u,dP>/sum u), u = p^(2-alpha), on the support, dQ by
// gathering K rows, dK / dV by vector atomics into fp32 accumulators.
#include "common.cuh"

namespace entmax {

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kSlots = kListCap / 32;
constexpr int kMaxNewton = 400;

// Butterfly sum with ascending strides: for values held by lanes 0..W-1 only (zeros elsewhere) the first
// log2(W) steps are exactly sub_sum<W>'s tree and the rest add zeros, so the full-warp and the
// W-lanes-per-row paths give the same bits for the same sorted support.
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

// the row-slice helpers of common.cuh under the names this file uses
template <int PER>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&x)[PER]) { load_slice<PER>(p, x); }
template <int PER>
__device__ __forceinline__ void store_bf16(__nv_bfloat16* p, const float (&x)[PER]) { store_slice<PER>(p, x); }


// reductions over aligned groups of W lanes (W = 8 or 16); the sum takes ascending strides like warp_sum
template <int W>
__device__ __forceinline__ float sub_sum(float x) {
#pragma unroll
  for (int o = 1; o < W; o <<= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
template <int W>
__device__ __forceinline__ float sub_max(float x) {
#pragma unroll
  for (int o = 1; o < W; o <<= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
// N consecutive bf16 (N = 8 or 16, 16-byte aligned) <-> floats
template <int N>
__device__ __forceinline__ void load_bf16_vec(const __nv_bfloat16* p, float (&x)[N]) {
#pragma unroll
  for (int c = 0; c < N / 8; ++c) {
    const uint4 raw = *reinterpret_cast<const uint4*>(p + 8 * c);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[t]));
      x[8 * c + 2 * t] = f.x;
      x[8 * c + 2 * t + 1] = f.y;
    }
  }
}
template <int N>
__device__ __forceinline__ void store_bf16_vec(__nv_bfloat16* p, const float (&x)[N]) {
#pragma unroll
  for (int c = 0; c < N / 8; ++c) {
    uint32_t w[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(x[8 * c + 2 * t], x[8 * c + 2 * t + 1]);
      w[t] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p + 8 * c) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
template <int N>
__device__ __forceinline__ void atomic_add_vec(float* p, const float (&x)[N]) {
#pragma unroll
  for (int c = 0; c < N / 4; ++c)
    red_add_v4(p + 4 * c, x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]);
}

// The rows of a warp that go to the dense path (mask over the warp's lanes, lane l holding row `grow`): one
// slot reservation and one status update for all of them.  A counter bumped once per row is a chain of
// dependent L2 atomics on one address; with every row dense that chain, not the rows' work, set the kernel's time.
__device__ __forceinline__ void push_dense_rows(unsigned mask, int grow, int32_t* fb_count, int32_t* fb_list,
                                                int32_t* status, int lane) {
  if (mask == 0u) return;
  const int leader = __ffs(mask) - 1;
  int base = 0;
  if (lane == leader) {
    base = atomicAdd(fb_count, __popc(mask));
    if (status) atomicAdd(status + ENTMAX_ATTN_STATUS_DENSE_ROWS, __popc(mask));
  }
  base = __shfl_sync(0xffffffffu, base, leader);
  if ((mask >> lane) & 1u) fb_list[base + __popc(mask & ((1u << lane) - 1u))] = grow;
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

// The forward row solve runs in two stages so that its result does not depend on what else the sweep
// happened to leave in the lists (their order and their surplus entries vary from run to run):
//   stage A  Newton on all candidates, in list order -> tau_A, accurate to fp32 rounding;
//   stage B  the entries above tau_A minus a small margin are compacted and sorted by key index, and
//            Newton runs again on this set alone, from the bracket's lower end (App. A: tau >= y_max - 1);
//            its summation order is fixed by the sorted set, so O and tau come out bit-identical
//            unless an entry lies within rounding noise of the margin cut.
constexpr float kKeepMargin = 4e-6f;

// Threshold of Eq. 1 on the entries held by the warp, started at the bracket's lower end y_max - 1 (App. A):
// Newton from the left for e >= 1, bracketed for e < 1 (tau_iter_update)
template <int S>
__device__ __forceinline__ float newton_warp(const Problem& p, const float (&y)[S], float ymax,
                                             float known_below = -INFINITY) {
  // known_below: a value the threshold is known not to lie below (mass >= 1 there); -inf: the bracket's own lower end
  TauIter st = tau_iter_start(ymax);
  st.tau = st.lo = fmaxf(st.lo, known_below);
  for (int it = 0; it < kMaxNewton; ++it) {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int s = 0; s < S; ++s) {
      const float d = y[s] - st.tau;
      if (d > 0.f) {
        float ye, ye1;
        pow_pair(d, p.expo_class, p.expo, ye, ye1);
        s0 += ye;
        s1 += ye1;
      }
    }
    s0 = warp_sum(s0);
    s1 = warp_sum(s1);
    if (!tau_iter_update(st, s0, s1, p.expo_class, p.expo, 1e-7f)) break;
  }
  return st.tau;
}

// Stage A on S*32 candidate slots.  Leaves the kept entries (y in Eq. 1's units) compacted from slot 0
// of the row's list and returns how many there are.
template <int S>
__device__ __forceinline__ int prefilter_row(const Problem& p, Entry* list, int c0, int c1, float a, int lane,
                                             float bound) {
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
  __syncwarp();   // every slot is in registers before the list is overwritten
  // stage A may start from the bound the sweep ended with (a lower bound of the row's threshold, and every key above
  // it is in the list): only its cut is used, so where it starts does not reach the result
  const float tau_a = newton_warp<S>(p, y, ymax, bound);
  const float cut = tau_a - kKeepMargin * fmaxf(1.0f, fabsf(tau_a));
  int kept = 0;
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const bool keep = y[s] > cut;
    const unsigned m = __ballot_sync(0xffffffffu, keep);
    if (keep) {
      const int pos = kept + __popc(m & ((1u << lane) - 1u));
      list[pos].y = y[s];
      list[pos].j = jj[s];
    }
    kept += __popc(m);
  }
  __syncwarp();
  return kept;
}

// Stage B on the `kept` compacted entries (kept <= 32*S): sort by key index, threshold, probabilities,
// O_i as a gather over the support, support written back sorted by key index.
template <int D, int S>
__device__ __forceinline__ void finish_row(const Problem& p, const __nv_bfloat16* __restrict__ vbase, Entry* list,
                                           int kept_in, __nv_bfloat16* o_row, float* tau_slot, int32_t* cnt_slot,
                                           int lane) {
  constexpr int PER = D / 32;
  float y[S];
  int jj[S];
  float ymax = -INFINITY;
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const int e = lane + 32 * s;
    y[s] = -INFINITY;
    jj[s] = 0x7fffffff;
    if (e < kept_in) {
      const Entry en = list[e];
      y[s] = en.y;
      jj[s] = en.j;
    }
    ymax = fmaxf(ymax, y[s]);
  }
  ymax = warp_max(ymax);
  __syncwarp();
  sort_by_key<S>(jj, y, lane);
  const float tau = newton_warp<S>(p, y, ymax);
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

// Out-of-line forms for the rare rows with more than 32 candidates (kept out of the hot loop's code)
__device__ __noinline__ int prefilter_long(const Problem& p, Entry* list, int c0, int c1, float a, int lane,
                                           float bound) {
  const int n = c0 + c1;
  if (n <= 64) return prefilter_row<2>(p, list, c0, c1, a, lane, bound);
  if (n <= 128) return prefilter_row<4>(p, list, c0, c1, a, lane, bound);
  return prefilter_row<kSlots>(p, list, c0, c1, a, lane, bound);
}
template <int D>
__device__ __noinline__ void finish_long(const Problem& p, const __nv_bfloat16* __restrict__ vbase, Entry* list, int kept,
                                         __nv_bfloat16* o_row, float* tau_slot, int32_t* cnt_slot, int lane) {
  if (kept <= 64) finish_row<D, 2>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
  else if (kept <= 128) finish_row<D, 4>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
  else finish_row<D, kSlots>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
}

// One row with the whole warp.
template <int D>
__device__ __forceinline__ void solve_row_full(const Problem& p, const __nv_bfloat16* __restrict__ vbase, Entry* list,
                                               int c0, int c1, float a, float bound, __nv_bfloat16* o_row,
                                               float* tau_slot, int32_t* cnt_slot, int lane) {
  const int n = c0 + c1;
  int kept;
  if (n <= 32) kept = prefilter_row<1>(p, list, c0, c1, a, lane, bound);
  else if (n <= 64) kept = prefilter_row<2>(p, list, c0, c1, a, lane, bound);
  else if (n <= 128) kept = prefilter_row<4>(p, list, c0, c1, a, lane, bound);
  else kept = prefilter_row<kSlots>(p, list, c0, c1, a, lane, bound);
  if (kept <= 32) finish_row<D, 1>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
  else if (kept <= 64) finish_row<D, 2>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
  else if (kept <= 128) finish_row<D, 4>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
  else finish_row<D, kSlots>(p, vbase, list, kept, o_row, tau_slot, cnt_slot, lane);
}

// The same iteration for 32 / W rows at once (W lanes per row); `done` rows keep their tau.
template <int W>
__device__ __forceinline__ float newton_sub(const Problem& p, float y, float ymax, bool done,
                                            float known_below = -INFINITY) {
  TauIter st = tau_iter_start(ymax);
  st.tau = st.lo = fmaxf(st.lo, known_below);
  for (int it = 0; it < kMaxNewton; ++it) {
    const float d = y - st.tau;
    float ye = 0.f, ye1 = 0.f;
    if (d > 0.f) pow_pair(d, p.expo_class, p.expo, ye, ye1);
    const float s0 = sub_sum<W>(ye), s1 = sub_sum<W>(ye1);
    if (!done) done = !tau_iter_update(st, s0, s1, p.expo_class, p.expo, 1e-7f);
    if (__all_sync(0xffffffffu, done)) break;
  }
  return st.tau;
}

// 32 / W rows at once, W lanes per row (W = 8 or 16), for rows with 1..W list entries; same two stages.
template <int D, int W>
__device__ __forceinline__ void solve_rows_sub(const Problem& p, const __nv_bfloat16* __restrict__ v,
                                                const float* __restrict__ scale, Entry* __restrict__ entries,
                                                __nv_bfloat16* __restrict__ o, float* __restrict__ tau_out,
                                                int32_t* __restrict__ row_cnt, const float* __restrict__ half_thr,
                                                int grow, bool active, int c0, int c1, int lane) {
  constexpr int PL = D / W;                        // elements of a V / O row per lane
  const int sl = lane & (W - 1);
  const int base = lane & (32 - W);
  const int n = active ? c0 + c1 : 0;
  const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
  const float a = active ? (p.alpha - 1.0f) * (scale[(size_t)b * p.scale_sb + (size_t)h * p.N + i] * p.sm_scale) : 1.0f;
  Entry* list = entries + (size_t)grow * kListCap;
  float y = -INFINITY;
  int j = 0x7fffffff;
  if (sl < n) {
    const Entry en = list[sl < c0 ? sl : kHalfCap + sl - c0];
    y = a * en.y;
    j = en.j;
  }
  __syncwarp();   // every entry is in registers before the compaction below overwrites the lists
  // stage A
  // stage A starts from the bound the sweep ended with (see prefilter_row)
  float bound = -INFINITY;
  if (active) {
    const float2 ht = *reinterpret_cast<const float2*>(half_thr + 2 * (size_t)grow);
    bound = fmaxf(ht.x, ht.y);
    bound -= kKeepMargin * fmaxf(1.0f, fabsf(bound));
  }
  const float tau_a = newton_sub<W>(p, y, sub_max<W>(y), !active, bound);
  const bool keep = active && y > tau_a - kKeepMargin * fmaxf(1.0f, fabsf(tau_a));
  // keep only those: they move to the end-stable front when sorted with the others' keys pushed to infinity
  j = keep ? j : 0x7fffffff;
  y = keep ? y : -INFINITY;
  // bitonic sort of the W (j, y) pairs of each row, ascending by key index
#pragma unroll
  for (int k = 2; k <= W; k <<= 1) {
#pragma unroll
    for (int st = k >> 1; st > 0; st >>= 1) {
      const int oj = __shfl_xor_sync(0xffffffffu, j, st);
      const float oy = __shfl_xor_sync(0xffffffffu, y, st);
      const bool up = ((sl & k) == 0);
      const bool lower = ((sl & st) == 0);
      const bool take_other = (lower == up) ? (oj < j) : (oj > j);
      j = take_other ? oj : j;
      y = take_other ? oy : y;
    }
  }
  // stage B
  const float tau = newton_sub<W>(p, y, sub_max<W>(y), !active);
  const float d = y - tau;
  const bool in = active && d > 0.f;
  float pe = 0.f, pe1;
  if (in) pow_pair(d, p.expo_class, p.expo, pe, pe1);
  const unsigned m = __ballot_sync(0xffffffffu, in);
  const unsigned msub = (m >> base) & ((1u << W) - 1u);
  if (in) {
    // compact the list to the exact support, y in Eq. 1's units
    const int pos = __popc(msub & ((1u << sl) - 1u));
    list[pos].y = y;
    list[pos].j = j;
  }
  float acc[PL];
#pragma unroll
  for (int t = 0; t < PL; ++t) acc[t] = 0.f;
  const __nv_bfloat16* vbase = v + (size_t)b * p.sb + (size_t)h * p.sh + sl * PL;
#pragma unroll
  for (int t = 0; t < W; ++t) {
    const bool has = (msub >> t) & 1u;
    if (!__any_sync(0xffffffffu, has)) continue;
    const float pj = __shfl_sync(0xffffffffu, pe, base + t);
    const int kj = __shfl_sync(0xffffffffu, j, base + t);
    if (has) {
      float vs[PL];
      if constexpr (PL >= 8) load_bf16_vec<PL>(vbase + (size_t)kj * p.sn, vs);
      else load_bf16<PL>(vbase + (size_t)kj * p.sn, vs);
#pragma unroll
      for (int u = 0; u < PL; ++u) acc[u] = fmaf(pj, vs[u], acc[u]);
    }
  }
  if (active) {
    __nv_bfloat16* o_row = o + (size_t)b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + sl * PL;
    if constexpr (PL >= 8) store_bf16_vec<PL>(o_row, acc);
    else store_bf16<PL>(o_row, acc);
    if (sl == 0) {
      tau_out[grow] = tau;
      row_cnt[grow] = __popc(msub);
    }
  }
}

// Closed-form row solve for e = 2 (alpha = 1.5) and e = 1 (alpha = 2), 32 / W rows at once with W lanes per row
// (W = 8, 16 or 32) and at most W list entries per row.  With the entries sorted by decreasing y and
// u_j = y_max - y_j, the threshold that makes the top k sum to one is, in units below the maximum,
//   e = 2:  t_k = (U1 + sqrt(U1^2 - k (U2 - 1))) / k      (the root of sum_{j<=k} (t - u_j)^2 = 1 with t >= u_k)
//   e = 1:  t_k = (1 + U1) / k                             (sum_{j<=k} (t - u_j) = 1)
// with U1, U2 the prefix sums of u and u^2; the support size k* is the number of k with u_k < t_k (they form a
// prefix) and tau = y_max - t_{k*} -- Eq. 1's threshold without iterating.  Only the top k* entries enter the
// result, so candidates outside the support, which differ from run to run, do not change a bit of it.
// `prescaled`: the list already holds y in Eq. 1's units from slot 0 (c1 = 0).
template <int D, int W, int EC>
__device__ __forceinline__ void solve_rows_closed(const Problem& p, const __nv_bfloat16* __restrict__ v,
                                                  const float* __restrict__ scale, Entry* __restrict__ entries,
                                                  __nv_bfloat16* __restrict__ o, float* __restrict__ tau_out,
                                                  int32_t* __restrict__ row_cnt, int grow, bool active, int c0, int c1,
                                                  bool prescaled, int lane) {
  static_assert(EC == kExpo2 || EC == kExpo1, "closed forms exist for e = 2 and e = 1");
  constexpr int PL = D / W;                        // elements of a V / O row per lane
  constexpr unsigned kWMask = W == 32 ? 0xffffffffu : ((1u << (W & 31)) - 1u);
  const int sl = lane & (W - 1);
  const int base = lane & (32 - W);
  const int n = active ? c0 + c1 : 0;
  const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
  const float a = (active && !prescaled)
                      ? (p.alpha - 1.0f) * (scale[(size_t)b * p.scale_sb + (size_t)h * p.N + i] * p.sm_scale) : 1.0f;
  Entry* list = entries + (size_t)grow * kListCap;
  float y = -INFINITY;
  int j = 0x7fffffff;
  if (sl < n) {
    const Entry en = list[sl < c0 ? sl : kHalfCap + sl - c0];
    y = a * en.y;
    j = en.j;
  }
  __syncwarp();   // every entry is in registers before the compaction below overwrites the lists
  const float ymax = sub_max<W>(y);
  // bitonic sort of the W (y, j) pairs of each row: decreasing y, equal values by increasing key index
#pragma unroll
  for (int k = 2; k <= W; k <<= 1) {
#pragma unroll
    for (int st = k >> 1; st > 0; st >>= 1) {
      const int oj = __shfl_xor_sync(0xffffffffu, j, st);
      const float oy = __shfl_xor_sync(0xffffffffu, y, st);
      const bool up = ((sl & k) == 0);
      const bool lower = ((sl & st) == 0);
      const bool other_first = oy > y || (oy == y && oj < j);
      const bool mine_first = y > oy || (y == oy && j < oj);
      const bool take_other = (lower == up) ? other_first : mine_first;
      j = take_other ? oj : j;
      y = take_other ? oy : y;
    }
  }
  const bool have = sl < n;
  const float u = have ? ymax - y : 0.f;
  float u1 = u, u2 = u * u;
#pragma unroll
  for (int off = 1; off < W; off <<= 1) {
    const float t1 = __shfl_up_sync(0xffffffffu, u1, off, W);
    const float t2 = __shfl_up_sync(0xffffffffu, u2, off, W);
    if (sl >= off) {
      u1 += t1;
      u2 += t2;
    }
  }
  const float kf = (float)(sl + 1);
  float tk;
  if constexpr (EC == kExpo2) {
    const float disc = fmaf(u1, u1, -kf * (u2 - 1.0f));
    tk = disc >= 0.f ? (u1 + sqrtf(disc)) / kf : -INFINITY;
  } else {
    tk = (1.0f + u1) / kf;
  }
  const unsigned okm = (__ballot_sync(0xffffffffu, have && u < tk) >> base) & kWMask;
  const int kstar = okm == kWMask ? W : __ffs(~okm) - 1;          // leading ones; >= 1 for a row with entries
  const float tprime = __shfl_sync(0xffffffffu, tk, base + (kstar > 0 ? kstar - 1 : 0));
  const float tau = ymax - tprime;
  const bool in = active && sl < kstar;
  const float d = tprime - u;
  const float pe = in ? (EC == kExpo2 ? d * d : d) : 0.f;
  if (in) {
    // the list becomes the exact support (by decreasing y), y in Eq. 1's units
    list[sl].y = y;
    list[sl].j = j;
  }
  float acc[PL];
#pragma unroll
  for (int t = 0; t < PL; ++t) acc[t] = 0.f;
  const __nv_bfloat16* vbase = v + (size_t)b * p.sb + (size_t)h * p.sh + sl * PL;
  // (not unrolled: a handful of iterations run, and the three widths of this function share the instruction cache)
#pragma unroll 1
  for (int t = 0; t < W; ++t) {
    const bool has = active && t < kstar;
    if (!__any_sync(0xffffffffu, has)) break;                      // supports are prefixes: nothing further either
    const float pj = __shfl_sync(0xffffffffu, pe, base + t);
    const int kj = __shfl_sync(0xffffffffu, j, base + t);
    if (has) {
      float vs[PL];
      if constexpr (PL >= 8) load_bf16_vec<PL>(vbase + (size_t)kj * p.sn, vs);
      else load_bf16<PL>(vbase + (size_t)kj * p.sn, vs);
#pragma unroll
      for (int u_ = 0; u_ < PL; ++u_) acc[u_] = fmaf(pj, vs[u_], acc[u_]);
    }
  }
  if (active) {
    __nv_bfloat16* o_row = o + (size_t)b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + sl * PL;
    if constexpr (PL >= 8) store_bf16_vec<PL>(o_row, acc);
    else store_bf16<PL>(o_row, acc);
    if (sl == 0) {
      tau_out[grow] = tau;
      row_cnt[grow] = kstar;
    }
  }
}

// Rows with more than kLongRow list entries take the whole warp for a long time each (two-stage solves, gathers over
// dozens of keys) and come in runs -- the start of every causal head, where all visible keys are candidates.  A
// warp that met sixteen of them in its block would work through them one after the other while the rest of the grid
// has finished, so they are only listed here (from the far end of the dense-row list, which has a slot for every
// row) and a second launch gives each of them a warp of its own.  kLongCounter: their count, in the counter block
// that starts at fb_count.
constexpr int kLongCounter = 56;
constexpr int kLongRow = 16;   // list entries from which a row counts as long
__device__ __forceinline__ void push_long_rows(unsigned mask, int grow, int total, int32_t* fb_count, int32_t* fb_list,
                                               int lane) {
  if (mask == 0u) return;
  const int leader = __ffs(mask) - 1;
  int base = 0;
  if (lane == leader) base = atomicAdd(fb_count + kLongCounter, __popc(mask));
  base = __shfl_sync(0xffffffffu, base, leader);
  if ((mask >> lane) & 1u) fb_list[total - 1 - (base + __popc(mask & ((1u << lane) - 1u)))] = grow;
}

// Forward: the rows of a warp for the dense-tile path (see push_dense_rows).  Their 128-row Q tiles are listed once
// (tile_flag arbitrates); of the lanes that name the same tile only the lowest asks.
__device__ __forceinline__ void push_dense_tiles(const Problem& p, unsigned mask, int grow, int32_t* row_cnt,
                                                 int32_t* fb_count, int32_t* fb_list, int32_t* tile_flag,
                                                 int32_t* tile_list, int32_t* tile_count, int32_t* status, int lane) {
  if (mask == 0u) return;
  push_dense_rows(mask, grow, fb_count, fb_list, status, lane);
  if ((mask >> lane) & 1u) {
    row_cnt[grow] = -2;
    const int tiles_per_head = (p.N + 127) / 128;
    const int bh = grow / p.N, i = grow - bh * p.N;
    const int id = bh * tiles_per_head + i / 128;
    const unsigned same = __match_any_sync(mask, id);
    if (lane == __ffs(same) - 1 && atomicExch(tile_flag + id, 1) == 0) tile_list[atomicAdd(tile_count, 1)] = id;
  }
}

// One row with the whole warp: lists of more than 16 entries (closed forms) or any list the sub-warp Newton
// solver did not take.
template <int D, int EC>
__device__ __forceinline__ void row_fwd_whole_warp(const Problem& p, const __nv_bfloat16* __restrict__ v,
                                                   const float* __restrict__ scale, int32_t* __restrict__ row_cnt,
                                                   const float* __restrict__ half_thr, Entry* __restrict__ entries,
                                                   __nv_bfloat16* __restrict__ o, float* __restrict__ tau_out, int grow,
                                                   int c0, int c1, int lane) {
  constexpr int PER = D / 32;
  constexpr bool kClosed = EC == kExpo2 || EC == kExpo1;
  const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
  const float a = (p.alpha - 1.0f) * (scale[(size_t)b * p.scale_sb + (size_t)h * p.N + i] * p.sm_scale);
  Entry* list = entries + (size_t)grow * kListCap;
  const float2 ht = *reinterpret_cast<const float2*>(half_thr + 2 * (size_t)grow);
  float bound = fmaxf(ht.x, ht.y);
  bound -= kKeepMargin * fmaxf(1.0f, fabsf(bound));
  if constexpr (kClosed) {
    // up to 32 entries: closed form with the whole warp; more: Newton prefilter first, and the closed form
    // if what it keeps fits the warp
    const int n = c0 + c1;
    if (n <= 32) {
      solve_rows_closed<D, 32, EC>(p, v, scale, entries, o, tau_out, row_cnt, grow, true, c0, c1, false, lane);
      return;
    }
    const int kept = prefilter_long(p, list, c0, c1, a, lane, bound);
    if (kept <= 32) {
      solve_rows_closed<D, 32, EC>(p, v, scale, entries, o, tau_out, row_cnt, grow, true, kept, 0, true, lane);
      return;
    }
    const __nv_bfloat16* vbase = v + (size_t)b * p.sb + (size_t)h * p.sh + lane * PER;
    __nv_bfloat16* o_row = o + (size_t)b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + lane * PER;
    finish_long<D>(p, vbase, list, kept, o_row, tau_out + grow, row_cnt + grow, lane);
  } else {
    const __nv_bfloat16* vbase = v + (size_t)b * p.sb + (size_t)h * p.sh + lane * PER;
    __nv_bfloat16* o_row = o + (size_t)b * p.sb + (size_t)h * p.sh + (size_t)i * p.sn + lane * PER;
    solve_row_full<D>(p, vbase, list, c0, c1, a, bound, o_row, tau_out + grow, row_cnt + grow, lane);
  }
}

// The rows row_fwd_kernel listed as long (push_long_rows): one warp per row.
template <int D, int EC>
__global__ void __launch_bounds__(kWarpsPerCta * 32) row_fwd_long_kernel(Problem p, const __nv_bfloat16* __restrict__ v,
                                                                         const float* __restrict__ scale,
                                                                         int32_t* __restrict__ row_cnt,
                                                                         const int32_t* __restrict__ half_cnt,
                                                                         const float* __restrict__ half_thr,
                                                                         Entry* __restrict__ entries,
                                                                         __nv_bfloat16* __restrict__ o,
                                                                         float* __restrict__ tau_out,
                                                                         const int32_t* __restrict__ fb_count,
                                                                         const int32_t* __restrict__ fb_list) {
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  const int n_long = fb_count[kLongCounter];
  for (int t = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); t < n_long; t += gridDim.x * kWarpsPerCta) {
    const int grow = fb_list[total - 1 - t];
    const int2 c = *reinterpret_cast<const int2*>(half_cnt + 2 * (size_t)grow);
    row_fwd_whole_warp<D, EC>(p, v, scale, row_cnt, half_thr, entries, o, tau_out, grow, c.x, c.y, lane);
  }
}

// EC: kExpo2 / kExpo1 select the closed-form solvers, kExpoGeneral the Newton ones (any exponent)
template <int D, int EC>
__global__ void __launch_bounds__(kWarpsPerCta * 32) row_fwd_kernel(Problem p, const __nv_bfloat16* __restrict__ v,
                                                                    const float* __restrict__ scale,
                                                                    int32_t* __restrict__ row_cnt,
                                                                    const int32_t* __restrict__ half_cnt,
                                                                    const float* __restrict__ half_thr,
                                                                    Entry* __restrict__ entries,
                                                                    __nv_bfloat16* __restrict__ o,
                                                                    float* __restrict__ tau_out, int32_t* fb_count,
                                                                    int32_t* fb_list, int32_t* tile_flag,
                                                                    int32_t* tile_list, int32_t* tile_count,
                                                                    int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  const int blocks = (total + 15) / 16;
  for (int blk = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); blk < blocks; blk += gridDim.x * kWarpsPerCta) {
    // A warp takes 16 consecutive rows; lane l (and l + 16) looks at row 16*blk + l.  Rows are then served by
    // list length: four at a time with eight lanes each (1..8 entries), two at a time with sixteen lanes
    // each (9..16 entries), the rest one by one with the whole warp.
    constexpr bool kClosed = EC == kExpo2 || EC == kExpo1;
    const int my_row = 16 * blk + (lane & 15);
    int mc0 = 0, mc1 = 0;
    int cls = 3;                                     // 0: <= 8 entries, 1: <= 16, 2: whole warp / dense, 3: no row
    if (my_row < total) {
      const int2 c = *reinterpret_cast<const int2*>(half_cnt + 2 * (size_t)my_row);
      mc0 = c.x;
      mc1 = c.y;
      const int n = mc0 + mc1;
      cls = (mc0 < 0 || mc1 < 0 || n < 1 || n > 16) ? 2 : n <= 8 ? 0 : 1;
    }
    unsigned m8 = __ballot_sync(0xffffffffu, lane < 16 && cls == 0);
    unsigned m16 = __ballot_sync(0xffffffffu, lane < 16 && cls == 1);
    unsigned mfull = __ballot_sync(0xffffffffu, lane < 16 && cls == 2);
    {
      // rows without a usable list go to the dense-tile path, all of the warp's at once
      const unsigned mdense =
          __ballot_sync(0xffffffffu, lane < 16 && my_row < total && (mc0 < 0 || mc1 < 0 || mc0 + mc1 == 0));
      push_dense_tiles(p, mdense, my_row, row_cnt, fb_count, fb_list, tile_flag, tile_list, tile_count, status, lane);
      mfull &= ~mdense;
      // ... and the ones with long lists to a launch of their own
      const unsigned mlong = __ballot_sync(0xffffffffu, lane < 16 && ((mfull >> lane) & 1u) && mc0 + mc1 > (kClosed ? kLongRow : 32));
      push_long_rows(mlong, my_row, total, fb_count, fb_list, lane);
      mfull &= ~mlong;
    }
    if constexpr (kClosed) {
      while (m8) {
        const unsigned src = __fns(m8, 0, (lane >> 3) + 1);        // the row of this group of eight lanes
        const bool active = src < 32u;
        const int c0 = __shfl_sync(0xffffffffu, mc0, active ? src : 0), c1 = __shfl_sync(0xffffffffu, mc1, active ? src : 0);
        solve_rows_closed<D, 8, EC>(p, v, scale, entries, o, tau_out, row_cnt, active ? 16 * blk + (int)src : 0, active, c0,
                                    c1, false, lane);
#pragma unroll
        for (int t = 0; t < 4; ++t) m8 &= m8 - 1;
      }
      while (m16) {
        const unsigned src = __fns(m16, 0, (lane >> 4) + 1);
        const bool active = src < 32u;
        const int c0 = __shfl_sync(0xffffffffu, mc0, active ? src : 0), c1 = __shfl_sync(0xffffffffu, mc1, active ? src : 0);
        solve_rows_closed<D, 16, EC>(p, v, scale, entries, o, tau_out, row_cnt, active ? 16 * blk + (int)src : 0, active,
                                     c0, c1, false, lane);
        m16 &= m16 - 1;
        m16 &= m16 - 1;
      }
    } else {
      // Newton solvers: rows that iterate together wait for the slowest, so only groups of four consecutive
      // rows that all have at most eight entries share a warp; every other row takes the whole warp.
      const unsigned none = __ballot_sync(0xffffffffu, lane < 16 && cls == 3);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const unsigned gm = 0xFu << (4 * g);
        if ((m8 & gm) != 0u && ((m8 | none) & gm) == gm) {
          const int src = 4 * g + (lane >> 3);
          const bool active = (m8 >> src) & 1u;
          const int c0 = __shfl_sync(0xffffffffu, mc0, src), c1 = __shfl_sync(0xffffffffu, mc1, src);
          solve_rows_sub<D, 8>(p, v, scale, entries, o, tau_out, row_cnt, half_thr, active ? 16 * blk + src : 0, active, c0,
                               c1, lane);
        } else {
          mfull |= (m8 | m16) & gm;
        }
      }
    }
    while (mfull) {
      const int src = __ffs(mfull) - 1;
      mfull &= mfull - 1;
      const int grow = 16 * blk + src;
      const int c0 = __shfl_sync(0xffffffffu, mc0, src), c1 = __shfl_sync(0xffffffffu, mc1, src);
      row_fwd_whole_warp<D, EC>(p, v, scale, row_cnt, half_thr, entries, o, tau_out, grow, c0, c1, lane);
    }
  }
}

// Backward of one row with the whole warp: the entmax Jacobian on the support.
template <int D>
__device__ __noinline__ void bwd_row_full(const Problem& p, const __nv_bfloat16* __restrict__ q,
                                             const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                                             const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ scale,
                                             const float* __restrict__ tau_in, const Entry* __restrict__ entries,
                                             __nv_bfloat16* __restrict__ dq, float* __restrict__ acc_dk,
                                             float* __restrict__ acc_dv, float* __restrict__ dc_rows, int grow, int c0,
                                             int c1, bool saved, int pitch, int lane) {
  constexpr int PER = D / 32;
  const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
  const float g = scale[(size_t)b * p.scale_sb + (size_t)h * p.N + i] * p.sm_scale;
  const float a = (p.alpha - 1.0f) * g;
  const float tau = tau_in[grow];
  const size_t hbase = (size_t)b * p.sb + (size_t)h * p.sh + lane * PER;
  float qs[PER], gs[PER];
  load_bf16<PER>(q + hbase + (size_t)i * p.sn, qs);
  load_bf16<PER>(d_o + hbase + (size_t)i * p.sn, gs);
  const Entry* list = entries + (size_t)grow * pitch;
  float yv[kSlots], dpv[kSlots], zz[kSlots];
  int jj[kSlots];
#pragma unroll
  for (int s = 0; s < kSlots; ++s) {
    const int e = lane + 32 * s;                     // dense numbering: first half-list, then second
    yv[s] = -1.0f;
    jj[s] = 0;
    dpv[s] = 0.f;
    zz[s] = 0.f;
    if (e < c0 + c1) {
      const Entry en = list[e < c0 ? e : kHalfCap + e - c0];
      // a list saved by the forward pass holds y = (alpha-1) s in Eq. 1's units, a fresh one raw <q_i, k_j>
      yv[s] = saved ? en.y - tau : fmaf(a, en.y, -tau);
      jj[s] = en.j;
      zz[s] = saved ? en.y / a : en.y;               // raw <q_i, k_j>
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
  if (dc_rows) {
    // dL/dc_i = sum_j dS_ij z_ij with z_ij = <q_i,k_j> sm_scale (chain rule through s = c z)
    float dc = 0.f;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) dc = fmaf(u[s] * (dpv[s] - rho), zz[s], dc);
    dc = warp_sum(dc);
    if (lane == 0) dc_rows[grow] = dc * p.sm_scale;
  }
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

// PL consecutive elements of a row: loads, stores and accumulator adds for any slice width used here
template <int PL>
__device__ __forceinline__ void load_slice_bf16(const __nv_bfloat16* p, float (&x)[PL]) {
  if constexpr (PL >= 8) load_bf16_vec<PL>(p, x);
  else load_bf16<PL>(p, x);
}
template <int PL>
__device__ __forceinline__ void store_slice_bf16(__nv_bfloat16* p, const float (&x)[PL]) {
  if constexpr (PL >= 8) store_bf16_vec<PL>(p, x);
  else store_bf16<PL>(p, x);
}
template <int PL>
__device__ __forceinline__ void add_slice(float* p, const float (&x)[PL]) {
  if constexpr (PL >= 8) atomic_add_vec<PL>(p, x);
  else atomic_add_slice<PL>(p, x);
}

// A lane's share of a row of D elements, W lanes per row: PL = D / W elements.  They are taken as chunks of four
// that interleave across the lanes (chunk c of lane sl = elements [4 W c + 4 sl, +4)), so that what the W lanes
// move in one instruction is contiguous: 16-byte reductions of neighbouring lanes fall into the same 32-byte
// sector instead of half-filling one each, loads and stores stay coalesced.  (PL < 4: one contiguous piece.)
template <int PL, int W>
__device__ __forceinline__ void load_share(const __nv_bfloat16* row, int sl, float (&x)[PL]) {
  if constexpr (PL < 4) {
    load_bf16<PL>(row + sl * PL, x);
  } else {
#pragma unroll
    for (int c = 0; c < PL / 4; ++c) {
      float t[4];
      load_bf16<4>(row + 4 * W * c + 4 * sl, t);
#pragma unroll
      for (int e = 0; e < 4; ++e) x[4 * c + e] = t[e];
    }
  }
}
template <int PL, int W>
__device__ __forceinline__ void store_share(__nv_bfloat16* row, int sl, const float (&x)[PL]) {
  if constexpr (PL < 4) {
    store_bf16<PL>(row + sl * PL, x);
  } else {
#pragma unroll
    for (int c = 0; c < PL / 4; ++c) {
      const float t[4] = {x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]};
      store_bf16<4>(row + 4 * W * c + 4 * sl, t);
    }
  }
}
template <int PL, int W>
__device__ __forceinline__ void add_share(float* row, int sl, const float (&x)[PL]) {
  if constexpr (PL < 4) {
    atomic_add_slice<PL>(row + sl * PL, x);
  } else {
#pragma unroll
    for (int c = 0; c < PL / 4; ++c) red_add_v4(row + 4 * W * c + 4 * sl, x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]);
  }
}

// Backward of 32 / W rows at once, W lanes per row (W = 8, 16 or 32), for rows with at most W list entries.
template <int D, int W>
__device__ __forceinline__ void bwd_rows_sub(const Problem& p, const __nv_bfloat16* __restrict__ q,
                                             const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                                             const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ scale,
                                             const float* __restrict__ tau_in, const Entry* __restrict__ entries,
                                             __nv_bfloat16* __restrict__ dq, float* __restrict__ acc_dk,
                                             float* __restrict__ acc_dv, float* __restrict__ dc_rows, int grow,
                                             bool active, int c0, int c1, bool saved, int pitch, int lane) {
  constexpr int PL = D / W;                        // elements of a row per lane
  constexpr unsigned kWMask = W == 32 ? 0xffffffffu : ((1u << (W & 31)) - 1u);
  const int sl = lane & (W - 1);
  const int base = lane & (32 - W);
  const int n = active ? c0 + c1 : 0;
  const int bh = grow / p.N, i = grow - bh * p.N, b = bh / p.H, h = bh - b * p.H;
  const float g = active ? scale[(size_t)b * p.scale_sb + (size_t)h * p.N + i] * p.sm_scale : 0.f;
  const float a = (p.alpha - 1.0f) * g;
  const float tau = active ? tau_in[grow] : 0.f;
  const size_t hbase = (size_t)b * p.sb + (size_t)h * p.sh;
  float qs[PL], gs[PL];
  load_share<PL, W>(q + hbase + (size_t)i * p.sn, sl, qs);
  load_share<PL, W>(d_o + hbase + (size_t)i * p.sn, sl, gs);
  const Entry* list = entries + (size_t)grow * pitch;
  float yv = -1.0f, zz = 0.f;
  int j = 0;
  if (sl < n) {
    const Entry en = list[sl < c0 ? sl : kHalfCap + sl - c0];
    // a list saved by the forward pass holds y = (alpha-1) s in Eq. 1's units, a fresh one raw <q_i, k_j>
    yv = saved ? en.y - tau : fmaf(a, en.y, -tau);
    j = en.j;
    zz = saved ? en.y / a : en.y;                  // raw <q_i, k_j>
  }
  const bool in = yv > 0.f;
  const unsigned msub = (__ballot_sync(0xffffffffu, in) >> base) & kWMask;
  // dP_ij = <dO_i, v_j> on the support
  float dpv = 0.f;
#pragma unroll 4
  for (int t = 0; t < W; ++t) {
    if (!__any_sync(0xffffffffu, (msub >> t) != 0u)) break;        // no row has entries from slot t on
    const bool has = (msub >> t) & 1u;
    const int kj = __shfl_sync(0xffffffffu, j, base + t);
    float dp = 0.f;
    if (has) {
      float vs[PL];
      load_share<PL, W>(v + hbase + (size_t)kj * p.sn, sl, vs);
#pragma unroll
      for (int u = 0; u < PL; ++u) dp = fmaf(gs[u], vs[u], dp);
    }
    dp = sub_sum<W>(dp);
    if (sl == t) dpv = dp;
  }
  float pe = 0.f, u = 0.f;
  if (in) pow_pair(yv, p.expo_class, p.expo, pe, u);
  const float su = sub_sum<W>(u), sud = sub_sum<W>(u * dpv);
  const float rho = su > 0.f ? sud / su : 0.f;
  const float gds_own = g * u * (dpv - rho);
  if (dc_rows) {
    // dL/dc_i = sum_j dS_ij z_ij with z_ij = <q_i,k_j> sm_scale (chain rule through s = c z)
    const float dc = sub_sum<W>(u * (dpv - rho) * zz);
    if (active && sl == 0) dc_rows[grow] = dc * p.sm_scale;
  }
  float acc[PL];
#pragma unroll
  for (int t = 0; t < PL; ++t) acc[t] = 0.f;
  const size_t arow = (size_t)bh * p.N;
#pragma unroll 4
  for (int t = 0; t < W; ++t) {
    if (!__any_sync(0xffffffffu, (msub >> t) != 0u)) break;
    const bool has = (msub >> t) & 1u;
    const int kj = __shfl_sync(0xffffffffu, j, base + t);
    const float gds = __shfl_sync(0xffffffffu, gds_own, base + t);
    const float pj = __shfl_sync(0xffffffffu, pe, base + t);
    if (has) {
      float ks[PL], dkv[PL], dvv[PL];
      load_share<PL, W>(k + hbase + (size_t)kj * p.sn, sl, ks);
#pragma unroll
      for (int w = 0; w < PL; ++w) {
        acc[w] = fmaf(gds, ks[w], acc[w]);
        dkv[w] = gds * qs[w];
        dvv[w] = pj * gs[w];
      }
      add_share<PL, W>(acc_dk + (arow + kj) * D, sl, dkv);
      add_share<PL, W>(acc_dv + (arow + kj) * D, sl, dvv);
    }
  }
  if (active) store_share<PL, W>(dq + hbase + (size_t)i * p.sn, sl, acc);
}

// (register cap: four CTAs per SM -- this kernel waits on gathers and reductions, occupancy is what hides them)
template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 4) row_bwd_kernel(
    Problem p, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ scale,
    const float* __restrict__ tau_in, const int32_t* __restrict__ half_cnt, const Entry* __restrict__ entries,
    __nv_bfloat16* __restrict__ dq, float* __restrict__ acc_dk, float* __restrict__ acc_dv,
    float* __restrict__ dc_rows, int32_t* fb_count, int32_t* fb_list, int32_t* status, int saved, int pitch) {
  // saved != 0: `half_cnt` is the forward pass's final support size per row (one int per row, -2 = dense
  // row) and `entries` its compacted support lists; `pitch` = list slots per row in `entries`
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  const int blocks = (total + 15) / 16;
  for (int blk = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); blk < blocks; blk += gridDim.x * kWarpsPerCta) {
    // A warp takes 16 consecutive rows; lane l (and l + 16) looks at row 16*blk + l.  Rows are served by list
    // length: four at a time (<= 8 entries), two at a time (<= 16), one at a time (<= 32, or the long form).
    const int my_row = 16 * blk + (lane & 15);
    int mc0 = 0, mc1 = 0;
    int cls = 4;                                     // 0: <= 8 entries, 1: <= 16, 2: <= 32, 3: more / dense, 4: no row
    if (my_row < total) {
      if (saved) {
        mc0 = half_cnt[my_row];
      } else {
        const int2 c = *reinterpret_cast<const int2*>(half_cnt + 2 * (size_t)my_row);
        mc0 = c.x;
        mc1 = c.y;
      }
      const int n = mc0 + mc1;
      cls = (mc0 < 0 || mc1 < 0 || n > 32) ? 3 : n <= 8 ? 0 : n <= 16 ? 1 : 2;
    }
    unsigned m8 = __ballot_sync(0xffffffffu, lane < 16 && cls == 0);
    unsigned m16 = __ballot_sync(0xffffffffu, lane < 16 && cls == 1);
    unsigned m32 = __ballot_sync(0xffffffffu, lane < 16 && cls == 2);
    unsigned mlong = __ballot_sync(0xffffffffu, lane < 16 && cls == 3);
    {
      // rows without a usable list go to the dense path, all of the warp's at once
      const unsigned mdense = __ballot_sync(0xffffffffu, lane < 16 && my_row < total && (mc0 < 0 || mc1 < 0));
      push_dense_rows(mdense, my_row, fb_count, fb_list, status, lane);
      mlong &= ~mdense;
      // ... and the ones with long lists to a launch of their own (see push_long_rows)
      push_long_rows(mlong | m32, my_row, total, fb_count, fb_list, lane);
    }
    while (m8) {
      const unsigned src = __fns(m8, 0, (lane >> 3) + 1);          // the row of this group of eight lanes
      const bool active = src < 32u;
      const int c0 = __shfl_sync(0xffffffffu, mc0, active ? src : 0), c1 = __shfl_sync(0xffffffffu, mc1, active ? src : 0);
      bwd_rows_sub<D, 8>(p, q, k, v, d_o, scale, tau_in, entries, dq, acc_dk, acc_dv, dc_rows,
                         active ? 16 * blk + (int)src : 0, active, c0, c1, saved != 0, pitch, lane);
#pragma unroll
      for (int t = 0; t < 4; ++t) m8 &= m8 - 1;
    }
    while (m16) {
      const unsigned src = __fns(m16, 0, (lane >> 4) + 1);
      const bool active = src < 32u;
      const int c0 = __shfl_sync(0xffffffffu, mc0, active ? src : 0), c1 = __shfl_sync(0xffffffffu, mc1, active ? src : 0);
      bwd_rows_sub<D, 16>(p, q, k, v, d_o, scale, tau_in, entries, dq, acc_dk, acc_dv, dc_rows,
                          active ? 16 * blk + (int)src : 0, active, c0, c1, saved != 0, pitch, lane);
      m16 &= m16 - 1;
      m16 &= m16 - 1;
    }
  }
}

// The rows row_bwd_kernel listed as long (push_long_rows): one warp per row.
template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 4) row_bwd_long_kernel(
    Problem p, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ scale,
    const float* __restrict__ tau_in, const int32_t* __restrict__ half_cnt, const Entry* __restrict__ entries,
    __nv_bfloat16* __restrict__ dq, float* __restrict__ acc_dk, float* __restrict__ acc_dv,
    float* __restrict__ dc_rows, const int32_t* __restrict__ fb_count, const int32_t* __restrict__ fb_list, int saved,
    int pitch) {
  const int lane = threadIdx.x & 31;
  const int total = p.B * p.H * p.N;
  const int n_long = fb_count[kLongCounter];
  for (int t = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5); t < n_long; t += gridDim.x * kWarpsPerCta) {
    const int grow = fb_list[total - 1 - t];
    int c0, c1 = 0;
    if (saved) {
      c0 = half_cnt[grow];
    } else {
      const int2 c = *reinterpret_cast<const int2*>(half_cnt + 2 * (size_t)grow);
      c0 = c.x;
      c1 = c.y;
    }
    if (c0 + c1 <= 32)
      bwd_rows_sub<D, 32>(p, q, k, v, d_o, scale, tau_in, entries, dq, acc_dk, acc_dv, dc_rows, grow, true, c0, c1,
                          saved != 0, pitch, lane);
    else
      bwd_row_full<D>(p, q, k, v, d_o, scale, tau_in, entries, dq, acc_dk, acc_dv, dc_rows, grow, c0, c1, saved != 0,
                      pitch, lane);
  }
}

// Copies every row's final support (at most `slots` entries) from the forward call's lists into a compact
// table; rows without a list, or with a longer one, get the count -2 and are recomputed by the backward pass.
__global__ void save_supports_kernel(int rows, int slots, const int32_t* __restrict__ row_cnt,
                                     const Entry* __restrict__ entries, int32_t* __restrict__ out_cnt,
                                     Entry* __restrict__ out_entries) {
  const long total = (long)rows * slots;
  for (long t = (long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (long)gridDim.x * blockDim.x) {
    const int row = (int)(t / slots), slot = (int)(t - (long)row * slots);
    const int cnt = row_cnt[row];
    const bool fits = cnt >= 0 && cnt <= slots;
    if (slot == 0) out_cnt[row] = fits ? cnt : -2;
    if (fits && slot < cnt) out_entries[(size_t)row * slots + slot] = entries[(size_t)row * kListCap + slot];
  }
}

inline int row_grid(const Problem& p) {
  const long total = ((long)p.B * p.H * p.N + 3) / 4;   // one warp per group of four rows
  const long ctas = (total + kWarpsPerCta - 1) / kWarpsPerCta;
  const long cap = 148L * 8 * 8;
  return (int)(ctas < cap ? ctas : cap);
}

}  // namespace

cudaError_t launch_row_fwd(const Problem& p, const void* v, const float* scale, int32_t* row_cnt,
                           const int32_t* half_cnt, const float* half_thr, Entry* entries, void* o, float* tau,
                           int32_t* fb_count, int32_t* fb_list, int32_t* tile_flag, int32_t* tile_list,
                           int32_t* tile_count, int32_t* status, cudaStream_t stream) {
  const int grid = row_grid(p);
#define ENTMAX_ROW_FWD(D, EC)                                                                                         \
  row_fwd_kernel<D, EC><<<grid, kWarpsPerCta * 32, 0, stream>>>(p, (const __nv_bfloat16*)v, scale, row_cnt, half_cnt, \
                                                                half_thr, entries, (__nv_bfloat16*)o, tau, fb_count,  \
                                                                fb_list,                                              \
                                                                tile_flag, tile_list, tile_count, status)
  if (p.D == 64) {
    if (p.expo_class == kExpo2) ENTMAX_ROW_FWD(64, kExpo2);
    else if (p.expo_class == kExpo1) ENTMAX_ROW_FWD(64, kExpo1);
    else ENTMAX_ROW_FWD(64, kExpoGeneral);
  } else {
    if (p.expo_class == kExpo2) ENTMAX_ROW_FWD(128, kExpo2);
    else if (p.expo_class == kExpo1) ENTMAX_ROW_FWD(128, kExpo1);
    else ENTMAX_ROW_FWD(128, kExpoGeneral);
  }
#undef ENTMAX_ROW_FWD
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  // the rows it listed as long, one warp each (normally none or a few: the launch then ends at once)
  const int lgrid = grid < 148 * 4 ? grid : 148 * 4;
#define ENTMAX_ROW_FWD_LONG(D, EC)                                                                                     \
  row_fwd_long_kernel<D, EC><<<lgrid, kWarpsPerCta * 32, 0, stream>>>(p, (const __nv_bfloat16*)v, scale, row_cnt,       \
                                                                      half_cnt, half_thr, entries, (__nv_bfloat16*)o,  \
                                                                      tau, fb_count, fb_list)
  if (p.D == 64) {
    if (p.expo_class == kExpo2) ENTMAX_ROW_FWD_LONG(64, kExpo2);
    else if (p.expo_class == kExpo1) ENTMAX_ROW_FWD_LONG(64, kExpo1);
    else ENTMAX_ROW_FWD_LONG(64, kExpoGeneral);
  } else {
    if (p.expo_class == kExpo2) ENTMAX_ROW_FWD_LONG(128, kExpo2);
    else if (p.expo_class == kExpo1) ENTMAX_ROW_FWD_LONG(128, kExpo1);
    else ENTMAX_ROW_FWD_LONG(128, kExpoGeneral);
  }
#undef ENTMAX_ROW_FWD_LONG
  return cudaGetLastError();
}

cudaError_t launch_save_supports(const Problem& p, int slots, const int32_t* row_cnt, const Entry* entries,
                                 int32_t* out_cnt, Entry* out_entries, cudaStream_t stream) {
  const int rows = p.B * p.H * p.N;
  const long total = (long)rows * slots;
  const int blocks = (int)((total + 255) / 256 < 148L * 16 ? (total + 255) / 256 : 148L * 16);
  save_supports_kernel<<<blocks, 256, 0, stream>>>(rows, slots, row_cnt, entries, out_cnt, out_entries);
  return cudaGetLastError();
}

cudaError_t launch_row_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                           const float* scale, const float* tau, const int32_t* half_cnt, Entry* entries, void* dq,
                           float* acc_dk, float* acc_dv, float* dc_rows, int32_t* fb_count, int32_t* fb_list,
                           int32_t* status, int saved, int pitch, cudaStream_t stream) {
  const int grid = row_grid(p);
  if (p.D == 64)
    row_bwd_kernel<64><<<grid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, dc_rows, fb_count, fb_list, status, saved, pitch);
  else
    row_bwd_kernel<128><<<grid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, dc_rows, fb_count, fb_list, status, saved, pitch);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  // the rows it listed as long, one warp each (normally none or a few: the launch then ends at once)
  const int lgrid = grid < 148 * 4 ? grid : 148 * 4;
  if (p.D == 64)
    row_bwd_long_kernel<64><<<lgrid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, dc_rows, fb_count, fb_list, saved, pitch);
  else
    row_bwd_long_kernel<128><<<lgrid, kWarpsPerCta * 32, 0, stream>>>(
        p, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, scale,
        tau, half_cnt, entries, (__nv_bfloat16*)dq, acc_dk, acc_dv, dc_rows, fb_count, fb_list, saved, pitch);
  return cudaGetLastError();
}

}  // namespace entmax
