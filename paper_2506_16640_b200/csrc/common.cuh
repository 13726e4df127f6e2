// Internal declarations shared by the translation units of libentmax_attn.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "entmax_attn.h"

namespace entmax {

// Sparse row lists.  The score sweep splits the keys of a row between two threads; each owns one half
// of the row's kListCap list slots: capacity kHalfCap, the fill level at which the sweep tightens the
// threshold and filters the half-list (checked after every 32 keys, so the capacity is never exceeded),
// and the length a filtered half-list may keep -- a row that cannot be brought down to it is handed to
// the dense path.  The row kernels merge the two halves and leave the support compacted from slot 0.
constexpr int kHalfCap = 128;
constexpr int kHalfTrigger = 88;
constexpr int kHalfKeep = 72;
static_assert(kHalfTrigger + 32 <= kHalfCap && kHalfKeep < kHalfTrigger, "half-list bounds");
constexpr int kListCap = 2 * kHalfCap;

// One list slot: y = (alpha-1) * s_ij (or the raw accumulator while a sweep is running), j = key index.
struct __align__(8) Entry {
  float y;
  int32_t j;
};

// Largest alpha the entry points accept (the paper's experiments go up to 64).  Beyond 2 the map is only as well
// conditioned as (spacing of tau)^(1/(alpha-1)) allows: fp32 keeps alpha <= 4 within the output tolerance.
constexpr float kAlphaMax = 64.0f;

// Exponent class of 1/(alpha-1): powers by multiplication for 1, 2, 4; powf otherwise.
enum ExpoClass : int { kExpoGeneral = 0, kExpo1 = 1, kExpo2 = 2, kExpo4 = 4 };

struct Problem {
  int B, H, N, D;
  int causal, n_mode;
  int dtype;
  float alpha, sm_scale;
  float expo;        // e = 1/(alpha-1)
  int expo_class;
  int64_t sb, sh, sn;  // element strides of the [B,H,N,D] tensors
  int has_scale;
  const float* alibi;  // device [H] ALiBi slopes m_h (z_ij += -m_h |i - j|), or nullptr
  int64_t scale_sb;    // batch stride of the scale table in floats: 0 for the per-head table [H,N], H*N for
                       // a caller-provided per-query table [B,H,N]
};

struct WsLayout {
  size_t scale, row_cnt, half_cnt, half_thr, entries, fb_count, sweep_counter, tile_count, fb_list, tile_flag, tile_list, tile_mask, alibi_blob, alibi_kmax, scratch, acc_dk, acc_dv, dc_rows, total;
  int scratch_ctas;     // CTAs of the dense-row kernels (each owns scratch_floats floats)
  size_t scratch_floats;
};

WsLayout make_layout(const Problem& p, bool is_bwd);

// Argument checks shared by every entry point (defined in entmax_attn_api.cu).
// make_problem validates params and fills the internal problem description; check_scale_ptrs wants beta, gamma,
// delta all given or all NULL; fail_cuda records the cudaError_t for entmax_attn_last_cuda_error() on the calling
// thread and returns ENTMAX_ATTN_ECUDA.
int make_problem(const entmax_attn_params* params, Problem* out);
int check_scale_ptrs(const float* beta, const float* gamma, const float* delta, Problem* p);
int fail_cuda(cudaError_t err);
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// y^e and y^(e-1) of a clamped y >= 0 (0 where the entry is outside the support: ok == false), with the
// exponent class fixed at compile time so that the per-element code stays a few instructions
template <int EC>
__device__ __forceinline__ void pow_pair_c(float y, bool ok, float expo, float& ye, float& ye1) {
  if constexpr (EC == kExpo2) { ye1 = y; ye = y * y; }
  else if constexpr (EC == kExpo1) { ye1 = ok ? 1.0f : 0.f; ye = y; }
  else if constexpr (EC == kExpo4) { const float t = y * y; ye1 = t * y; ye = t * t; }
  else {
    ye = 0.f; ye1 = 0.f;
    if (ok) { ye1 = powf(y, expo - 1.0f); ye = ye1 * y; }
  }
}

// y^e and y^(e-1) for y > 0
__device__ __forceinline__ void pow_pair(float y, int expo_class, float expo, float& ye, float& ye1) {
  if (expo_class == kExpo2) { ye1 = y; ye = y * y; }
  else if (expo_class == kExpo1) { ye1 = 1.0f; ye = y; }
  else if (expo_class == kExpo4) { float t = y * y; ye1 = t * y; ye = t * t; }
  else { ye1 = powf(y, expo - 1.0f); ye = ye1 * y; }
}

// One threshold step from the left of the root, given S = sum [y - tau]_+^e (> 1) and S1 = sum [y - tau]_+^(e-1).
// It is Newton on F(tau) = S^(1/e) - 1 rather than on S - 1: the e-norm of an affine function of tau is convex and
// decreasing just like S (so steps from the left never pass the root, Eq. 1's threshold), but nearly linear in tau
// -- exactly linear while the support does not change and the values are equal -- where S is a polynomial of
// degree e.  -F / F' = (S - S^(1-1/e)) / S1.  For e = 1 (sparsemax) it is the plain Newton step (S - 1) / S1.
__device__ __forceinline__ float threshold_step(float s0, float s1, int expo_class, float expo) {
  const float root = expo_class == kExpo1 ? s0
                     : expo_class == kExpo2 ? sqrtf(s0)
                     : expo_class == kExpo4 ? sqrtf(sqrtf(s0)) : powf(s0, 1.0f / expo);
  return (s0 - s0 / root) / s1;
}

// Threshold iteration for any exponent.  For e >= 1 (alpha <= 2) f(tau) = sum [y - tau]_+^e - 1 is convex and
// decreasing, and steps from the left of the root never pass it (threshold_step above).  For e < 1 (alpha > 2) every
// term is concave where positive and drops to zero with infinite slope, so Newton alone can overshoot either way: the
// iteration keeps a bracket (App. A's bisection bracket: lo with mass >= 1, hi with mass < 1), takes the Newton step on
// f when it lands strictly inside and the midpoint otherwise, and ends when the mass is 1 to rounding or on the lower
// end of a bracket that holds no further float.
struct TauIter {
  float tau, lo, hi;
};
__device__ __forceinline__ TauIter tau_iter_start(float ymax) {
  TauIter s;
  s.tau = s.lo = ymax - 1.0f;   // p_max <= 1
  s.hi = ymax;                  // nothing above y_max: mass 0
  return s;
}
// One update from S = sum [y - tau]_+^e and S1 = sum [y - tau]_+^(e-1) taken at s.tau.  Returns false when s.tau is final.
__device__ __forceinline__ bool tau_iter_update(TauIter& s, float s0, float s1, int expo_class, float expo, float rel_tol) {
  if (expo >= 1.0f) {
    if (!(s0 > 1.0f) || !(s1 > 0.f)) return false;
    const float step = threshold_step(s0, s1, expo_class, expo);
    const float next = s.tau + step;
    if (!(next > s.tau)) return false;
    s.tau = next;
    return step > rel_tol * fmaxf(1.0f, fabsf(next));
  }
  if (s0 >= 1.0f) s.lo = s.tau; else s.hi = s.tau;
  float next = s.tau + (s0 - 1.0f) / (expo * s1);      // Newton on f: f' = -e S1
  if (!(next > s.lo && next < s.hi)) next = 0.5f * (s.lo + s.hi);
  // done when the mass is 1 to rounding, or when no float is left strictly inside the bracket (the width of the
  // bracket says nothing here: ties put the root at -n^(1-alpha), far below any tolerance relative to |tau|)
  const bool go = fabsf(s0 - 1.0f) > 16.0f * rel_tol && next > s.lo && next < s.hi;
  if (go) s.tau = next;
  else if (fabsf(s0 - 1.0f) > 16.0f * rel_tol) s.tau = s.lo;
  return go;
}

// Fire-and-forget vector adds to global memory (sm_90+): reductions that return nothing, so no thread waits
// for the old value to come back.
__device__ __forceinline__ void red_add_v4(float* dst, float x, float y, float z, float w) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void red_add_v2(float* dst, float x, float y) {
  asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dst), "f"(x), "f"(y) : "memory");
}

// ---- PER (2 or 4) consecutive elements of a row <-> floats, for float and bfloat16 rows; fp32 vector reductions ----
template <int PER>
__device__ __forceinline__ void load_slice(const float* p, float (&x)[PER]) {
  if constexpr (PER == 2) { float2 t = *reinterpret_cast<const float2*>(p); x[0] = t.x; x[1] = t.y; }
  else { float4 t = *reinterpret_cast<const float4*>(p); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
}
template <int PER>
__device__ __forceinline__ void load_slice(const __nv_bfloat16* p, float (&x)[PER]) {
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
__device__ __forceinline__ void store_slice(float* p, const float (&x)[PER]) {
  if constexpr (PER == 2) *reinterpret_cast<float2*>(p) = make_float2(x[0], x[1]);
  else *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
}
template <int PER>
__device__ __forceinline__ void store_slice(__nv_bfloat16* p, const float (&x)[PER]) {
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
  if constexpr (PER == 2) red_add_v2(p, x[0], x[1]);
  else red_add_v4(p, x[0], x[1], x[2], x[3]);
}

// ---- launchers (each enqueues on `stream` and returns the cudaError_t of the launch) -------------
cudaError_t launch_scale_table(const Problem& p, const float* beta, const float* gamma, const float* delta,
                               float* scale, int32_t* status, cudaStream_t stream);

// dense-row path (CUDA cores): all rows (row_list == nullptr) or the rows in row_list[0 .. *row_count)
cudaError_t launch_dense_fwd(const Problem& p, const void* q, const void* k, const void* v, const float* scale,
                             void* o, float* tau, int32_t* row_cnt, int32_t* dense_cnt, Entry* entries, const int32_t* row_list,
                             const int32_t* row_count, float* scratch, size_t scratch_floats, int ctas,
                             cudaStream_t stream);
cudaError_t launch_dense_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                             const float* scale, const float* tau, void* dq, float* acc_dk, float* acc_dv,
                             float* dc_rows, const int32_t* row_list, const int32_t* row_count, float* scratch,
                             size_t scratch_floats, int ctas, cudaStream_t stream);
// dbeta, dgamma, ddelta [H] from the per-row scale gradients dc_rows [B,H,N]
cudaError_t launch_scale_grad(const Problem& p, const float* beta, const float* gamma, const float* dc_rows,
                              float* dbeta, float* dgamma, float* ddelta, cudaStream_t stream);

// tcgen05 score sweep (bf16): fills the per-row candidate lists.
//   mode 0: threshold search (forward); mode 1: threshold given in tau_in (backward)
cudaError_t launch_sweep(const Problem& p, const void* q, const void* k, const float* scale, const float* tau_in,
                         int mode, int32_t* half_cnt, float* half_thr, Entry* entries, int32_t* work_counter,
                         float* dump, int dump_bh, float* alibi_blob, float* alibi_kmax, int32_t* status,
                         cudaStream_t stream);

// Puts tile_list[0 .. *tile_count) (the Q tiles flagged in tile_flag) into the order the dense-tile kernels hand
// them out in: longest first on causal problems.
cudaError_t order_tiles(const Problem& p, const int32_t* tile_flag, int32_t* tile_list, const int32_t* tile_count,
                        cudaStream_t stream);

// Dense-tile forward on the tensor cores (bf16): recomputes the Q tiles (128 rows) listed in tile_list (= flagged
// in tile_flag; the list is reordered) and writes O and tau of their rows marked row_cnt == -2, and into dense_cnt
// [B*H*N][2] the number of keys with p > 0 each of the row's two threads saw (their sum is the row's support
// size).  *work_counter must be zero on entry.
cudaError_t launch_tile_fwd(const Problem& p, const void* q, const void* k, const void* v, const float* scale,
                            const int32_t* tile_flag, int32_t* tile_list, const int32_t* tile_count,
                            int32_t* work_counter, const int32_t* row_cnt, int32_t* dense_cnt, void* o, float* tau,
                            int32_t* status, cudaStream_t stream);

// Dense-tile backward on the tensor cores (bf16): the rows in row_list[0 .. *row_count) are marked in
// tile_mask, their 128-row Q tiles listed, and dQ (and dc_rows) of those rows written; their dK and dV
// contributions are added to the fp32 accumulators.  tile_mask, tile_flag, *tile_count, *work_counter and
// work_counter[12] must be zero on entry; rho: [B*H*N] floats of scratch.
cudaError_t launch_tile_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                            const float* scale, const float* tau, const int32_t* row_list, const int32_t* row_count,
                            uint32_t* tile_mask, int32_t* tile_flag, int32_t* tile_list, int32_t* tile_count,
                            int32_t* work_counter, float* rho, void* dq,
                            float* acc_dk, float* acc_dv, float* dc_rows, int32_t* status, cudaStream_t stream);

// per-row solve + gather kernels working on the lists (bf16 path); the forward one also lists the
// 128-row Q tiles that hold rows for the dense-tile path (tile_flag must be zero on entry)
cudaError_t launch_row_fwd(const Problem& p, const void* v, const float* scale, int32_t* row_cnt,
                           const int32_t* half_cnt, const float* half_thr, Entry* entries, void* o, float* tau, int32_t* fb_count,
                           int32_t* fb_list, int32_t* tile_flag, int32_t* tile_list, int32_t* tile_count, int32_t* status,
                           cudaStream_t stream);
cudaError_t launch_row_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                           const float* scale, const float* tau, const int32_t* half_cnt, Entry* entries, void* dq,
                           float* acc_dk, float* acc_dv, float* dc_rows, int32_t* fb_count, int32_t* fb_list,
                           int32_t* status, int saved, int pitch, cudaStream_t stream);
// compact copy of the forward call's supports (see entmax_attn_save_supports)
cudaError_t launch_save_supports(const Problem& p, int slots, const int32_t* row_cnt, const Entry* entries,
                                 int32_t* out_cnt, Entry* out_entries, cudaStream_t stream);

// fp32 accumulators [B,H,N,D] contiguous -> strided output tensor of the problem dtype
cudaError_t launch_store_grad(const Problem& p, const float* acc, void* out, cudaStream_t stream);

}  // namespace entmax
