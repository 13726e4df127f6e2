// C ABI of libentmax_attn.so: argument validation, workspace carving and the stream-ordered launch
// sequences of the forward and backward passes.  See include/entmax_attn.h for the contract.
#include <cmath>
#include <cstring>

#include "common.cuh"

namespace entmax {

namespace {

thread_local int g_last_cuda_error = 0;
thread_local cudaEvent_t g_prof_start[2] = {nullptr, nullptr};
thread_local cudaEvent_t g_prof_stop[2] = {nullptr, nullptr};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A second stream per (host thread, device) on which the backward call clears its fp32 accumulators while the
// score sweep, which does not touch them, runs on the caller's stream: forked from and joined back to the
// caller's stream with events, so the caller sees ordinary stream order (and a stream capture stays one graph).
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
thread_local SideStream g_side[64];

cudaError_t side_stream(SideStream** out) {
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  SideStream& s = g_side[dev];
  if (!s.stream) {
    cudaStream_t st = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    err = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking);
    if (err == cudaSuccess) err = cudaEventCreateWithFlags(&e0, cudaEventDisableTiming);
    if (err == cudaSuccess) err = cudaEventCreateWithFlags(&e1, cudaEventDisableTiming);
    if (err != cudaSuccess) {
      if (e0) cudaEventDestroy(e0);
      if (st) cudaStreamDestroy(st);
      return err;
    }
    s.stream = st; s.fork = e0; s.join = e1;
  }
  *out = &s;
  return cudaSuccess;
}

struct SavedLayout {
  size_t counts, entries, total;
};
SavedLayout saved_layout(const Problem& p) {
  const size_t rows = (size_t)p.B * p.H * p.N;
  SavedLayout l;
  l.counts = 0;
  l.entries = align_up(rows * sizeof(int32_t), 256);
  l.total = l.entries + align_up(rows * ENTMAX_ATTN_SAVED_SLOTS * sizeof(Entry), 256);
  return l;
}

int check_workspace(const Problem& p, bool is_bwd, void* ws, size_t ws_bytes, WsLayout* lay) {
  *lay = make_layout(p, is_bwd);
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || ws_bytes < lay->total) return ENTMAX_ATTN_EINVAL_WORKSPACE;
  return ENTMAX_ATTN_OK;
}

int check_device_for_bf16() {
  int dev = 0, major = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return fail_cuda(err);
  err = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (err != cudaSuccess) return fail_cuda(err);
  return major == 10 ? ENTMAX_ATTN_OK : ENTMAX_ATTN_EUNSUPPORTED;
}

}  // namespace

int fail_cuda(cudaError_t err) {
  g_last_cuda_error = (int)err;
  return ENTMAX_ATTN_ECUDA;
}

// Validates params and fills the internal problem description.  Returns a status code.
int make_problem(const entmax_attn_params* params, Problem* out) {
  if (!params) return ENTMAX_ATTN_EINVAL_NULL;
  Problem p;
  p.B = params->batch; p.H = params->heads; p.N = params->seq; p.D = params->head_dim;
  if (p.B < 1 || p.H < 1 || p.N < 1) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (p.D != 64 && p.D != 128) return ENTMAX_ATTN_EINVAL_SHAPE;
  if ((long long)p.B * p.H * p.N > 0x7fffffffLL / 2) return ENTMAX_ATTN_EINVAL_SHAPE;  // row ids are int32
  if (params->dtype != ENTMAX_ATTN_DTYPE_BF16 && params->dtype != ENTMAX_ATTN_DTYPE_FP32) return ENTMAX_ATTN_EINVAL_DTYPE;
  p.dtype = params->dtype;
  p.causal = params->causal ? 1 : 0;
  p.n_mode = params->n_mode ? 1 : 0;
  p.alpha = params->alpha;
  if (!(p.alpha > 1.0f) || !(p.alpha <= kAlphaMax)) return ENTMAX_ATTN_EINVAL_ALPHA;
  p.sm_scale = params->sm_scale;
  if (!std::isfinite(p.sm_scale) || p.sm_scale < 0.f) return ENTMAX_ATTN_EINVAL_ALPHA;
  if (p.sm_scale == 0.f) p.sm_scale = 1.0f / std::sqrt((float)p.D);
  p.expo = 1.0f / (p.alpha - 1.0f);
  p.expo_class = p.alpha == 2.0f ? kExpo1 : p.alpha == 1.5f ? kExpo2 : p.alpha == 1.25f ? kExpo4 : kExpoGeneral;
  if (params->stride_b == 0 && params->stride_h == 0 && params->stride_n == 0) {
    p.sn = p.D;
    p.sh = (int64_t)p.N * p.D;
    p.sb = (int64_t)p.H * p.N * p.D;
  } else {
    p.sb = params->stride_b; p.sh = params->stride_h; p.sn = params->stride_n;
    if (p.sn < p.D || p.sh < 1 || p.sb < 1) return ENTMAX_ATTN_EINVAL_SHAPE;
    if (p.sn % 8 || p.sh % 8 || p.sb % 8) return ENTMAX_ATTN_EINVAL_SHAPE;
  }
  p.has_scale = 0;
  p.scale_sb = 0;
  p.alibi = nullptr;
  *out = p;
  return ENTMAX_ATTN_OK;
}

int check_scale_ptrs(const float* beta, const float* gamma, const float* delta, Problem* p) {
  const int given = (beta != nullptr) + (gamma != nullptr) + (delta != nullptr);
  if (given != 0 && given != 3) return ENTMAX_ATTN_EINVAL_NULL;
  p->has_scale = given == 3;
  return ENTMAX_ATTN_OK;
}

WsLayout make_layout(const Problem& p, bool is_bwd) {
  WsLayout l;
  const size_t rows = (size_t)p.B * p.H * p.N;
  size_t off = 0;
  auto take = [&off](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
  l.scale = take((size_t)p.H * p.N * sizeof(float));
  l.row_cnt = take(rows * sizeof(int32_t));
  l.half_cnt = take(rows * 2 * sizeof(int32_t));
  l.half_thr = take(rows * 2 * sizeof(float));
  l.entries = take(rows * kListCap * sizeof(Entry));
  l.fb_count = take(256);
  l.sweep_counter = l.fb_count + 64;   // same 256-byte block: [0] dense-row count, [16] sweep work counter,
  l.tile_count = l.fb_count + 128;     // [32] number of listed dense tiles, [48] the dense-tile kernels' work counter
  l.fb_list = take(rows * sizeof(int32_t));
  const size_t q_tiles = (size_t)p.B * p.H * ((p.N + 127) / 128);
  l.tile_flag = take(q_tiles * sizeof(int32_t));
  l.tile_list = take(q_tiles * sizeof(int32_t));
  l.tile_mask = take(q_tiles * 4 * sizeof(uint32_t));   // 128 row bits per Q tile (dense-tile backward)
  // ALiBi window of the score sweep: slopes [H] + first K tile of every 256-row work item; key norms per 256-key tile
  const size_t items = (size_t)p.B * p.H * ((p.N + 255) / 256);
  l.alibi_blob = take(((size_t)p.H + items) * sizeof(float));
  l.alibi_kmax = take(items * sizeof(float));
  // dense-row CTAs: enough to fill the machine, few enough that their score rows stay modest
  l.scratch_floats = align_up((size_t)p.N, 32) * (is_bwd ? 2 : 1);   // scores (+ dP in backward)
  size_t ctas = 148 * 4;
  if (ctas > rows) ctas = rows;
  l.scratch_ctas = (int)ctas;
  l.scratch = take(ctas * l.scratch_floats * sizeof(float));
  l.acc_dk = l.acc_dv = l.dc_rows = 0;
  if (is_bwd) {
    l.acc_dk = take(rows * p.D * sizeof(float));
    l.acc_dv = take(rows * p.D * sizeof(float));
    l.dc_rows = take(rows * sizeof(float));
  }
  l.total = off;
  return l;
}

}  // namespace entmax

using namespace entmax;

extern "C" {

size_t entmax_attn_workspace_bytes(const entmax_attn_params* params, int is_bwd) {
  Problem p;
  if (make_problem(params, &p) != ENTMAX_ATTN_OK) return 0;
  return make_layout(p, is_bwd != 0).total;
}

int entmax_attn_workspace_layout(const entmax_attn_params* params, entmax_attn_ws_layout* out) {
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!out) return ENTMAX_ATTN_EINVAL_NULL;
  const WsLayout l = make_layout(p, false);
  out->row_count_offset = l.row_cnt;
  out->entries_offset = l.entries;
  out->scale_offset = l.scale;
  out->dense_count_offset = l.half_cnt;
  out->capacity = kListCap;
  out->keep_limit = kHalfKeep;
  return ENTMAX_ATTN_OK;
}

}  // extern "C"

namespace {

// Forward pass; c_rows, when given, is a per-query scale table [B,H,N] that replaces the one the library
// computes from beta, gamma, delta.
int fwd_impl(const entmax_attn_params* params, const void* q, const void* k, const void* v, const float* beta,
             const float* gamma, const float* delta, const float* c_rows, const float* alibi, void* o, float* tau,
             void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!q || !k || !v || !o || !tau) return ENTMAX_ATTN_EINVAL_NULL;
  rc = check_scale_ptrs(beta, gamma, delta, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (c_rows && (reinterpret_cast<uintptr_t>(c_rows) & 3u)) return ENTMAX_ATTN_EINVAL_ALIGN;
  if (alibi && (reinterpret_cast<uintptr_t>(alibi) & 3u)) return ENTMAX_ATTN_EINVAL_ALIGN;
  // the tensor-core kernels apply the ALiBi term on the causal side only
  if (alibi && p.dtype == ENTMAX_ATTN_DTYPE_BF16 && !p.causal) return ENTMAX_ATTN_EUNSUPPORTED;
  p.alibi = alibi;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(tau)) return ENTMAX_ATTN_EINVAL_ALIGN;
  WsLayout lay;
  rc = check_workspace(p, false, workspace, workspace_bytes, &lay);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (p.dtype == ENTMAX_ATTN_DTYPE_BF16) {
    rc = check_device_for_bf16();
    if (rc != ENTMAX_ATTN_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* scale = reinterpret_cast<float*>(ws + lay.scale);
  int32_t* row_cnt = reinterpret_cast<int32_t*>(ws + lay.row_cnt);
  int32_t* half_cnt = reinterpret_cast<int32_t*>(ws + lay.half_cnt);
  float* half_thr = reinterpret_cast<float*>(ws + lay.half_thr);
  int32_t* sweep_counter = reinterpret_cast<int32_t*>(ws + lay.sweep_counter);
  Entry* entries = reinterpret_cast<Entry*>(ws + lay.entries);
  int32_t* fb_count = reinterpret_cast<int32_t*>(ws + lay.fb_count);
  int32_t* fb_list = reinterpret_cast<int32_t*>(ws + lay.fb_list);
  float* scratch = reinterpret_cast<float*>(ws + lay.scratch);
  cudaError_t err;
  if (device_status) {
    err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  if (c_rows) {
    scale = c_rows;
    p.scale_sb = (int64_t)p.H * p.N;
  } else {
    err = launch_scale_table(p, beta, gamma, delta, reinterpret_cast<float*>(ws + lay.scale), device_status, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  if (p.dtype == ENTMAX_ATTN_DTYPE_FP32) {
    err = launch_dense_fwd(p, q, k, v, scale, o, tau, row_cnt, half_cnt, entries, nullptr, nullptr, scratch, lay.scratch_floats,
                           lay.scratch_ctas, stream);
    return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
  }
  int32_t* tile_flag = reinterpret_cast<int32_t*>(ws + lay.tile_flag);
  int32_t* tile_list = reinterpret_cast<int32_t*>(ws + lay.tile_list);
  int32_t* tile_count = reinterpret_cast<int32_t*>(ws + lay.tile_count);
  err = cudaMemsetAsync(fb_count, 0, 256, stream);   // the whole counter block
  if (err != cudaSuccess) return fail_cuda(err);
  err = cudaMemsetAsync(tile_flag, 0, (size_t)p.B * p.H * ((p.N + 127) / 128) * sizeof(int32_t), stream);
  if (err != cudaSuccess) return fail_cuda(err);
  if (g_prof_start[0]) cudaEventRecord(g_prof_start[0], stream);
  err = launch_sweep(p, q, k, scale, nullptr, 0, half_cnt, half_thr, entries, sweep_counter, nullptr, -1,
                     reinterpret_cast<float*>(ws + lay.alibi_blob), reinterpret_cast<float*>(ws + lay.alibi_kmax),
                     device_status, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  if (g_prof_stop[0]) cudaEventRecord(g_prof_stop[0], stream);
  err = launch_row_fwd(p, v, scale, row_cnt, half_cnt, half_thr, entries, o, tau, fb_count, fb_list, tile_flag, tile_list,
                       tile_count, device_status, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  // rows whose support does not fit the lists: dense tiles on the tensor cores
  err = launch_tile_fwd(p, q, k, v, scale, tile_flag, tile_list, tile_count, tile_count + 16, row_cnt, half_cnt, o, tau,
                        device_status, stream);
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}

}  // namespace

extern "C" {

int entmax_attn_fwd(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                    const float* beta, const float* gamma, const float* delta, void* o, float* tau,
                    void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  return fwd_impl(params, q, k, v, beta, gamma, delta, nullptr, nullptr, o, tau, workspace, workspace_bytes,
                  device_status, cuda_stream);
}

int entmax_attn_fwd_ex(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                       const float* beta, const float* gamma, const float* delta, const entmax_attn_extras* extras,
                       void* o, float* tau, void* workspace, size_t workspace_bytes, int32_t* device_status,
                       void* cuda_stream) {
  const float* c_rows = extras ? extras->c_rows : nullptr;
  const float* alibi = extras ? extras->alibi_slopes : nullptr;
  if (c_rows && (beta || gamma || delta)) return ENTMAX_ATTN_EINVAL_NULL;   // one source of the scale, not two
  return fwd_impl(params, q, k, v, beta, gamma, delta, c_rows, alibi, o, tau, workspace, workspace_bytes, device_status,
                  cuda_stream);
}

int entmax_attn_fwd_rowscale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                             const float* c_rows, void* o, float* tau, void* workspace, size_t workspace_bytes,
                             int32_t* device_status, void* cuda_stream) {
  if (!c_rows) return ENTMAX_ATTN_EINVAL_NULL;
  return fwd_impl(params, q, k, v, nullptr, nullptr, nullptr, c_rows, nullptr, o, tau, workspace, workspace_bytes,
                  device_status, cuda_stream);
}

}  // extern "C"

namespace {

int bwd_impl(const entmax_attn_params* params, const void* q, const void* k, const void* v, const float* beta,
             const float* gamma, const float* delta, const float* c_rows, const float* alibi,
             const void* fwd_workspace, const void* saved_supports, const float* tau, const void* d_o, void* dq,
             void* dk, void* dv, float* d_scale_rows, float* dbeta, float* dgamma, float* ddelta, void* workspace,
             size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!q || !k || !v || !tau || !d_o || !dq || !dk || !dv) return ENTMAX_ATTN_EINVAL_NULL;
  rc = check_scale_ptrs(beta, gamma, delta, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  const int n_param_grads = (dbeta != nullptr) + (dgamma != nullptr) + (ddelta != nullptr);
  if (n_param_grads != 0 && (n_param_grads != 3 || !p.has_scale || c_rows)) return ENTMAX_ATTN_EINVAL_NULL;
  if (c_rows && (reinterpret_cast<uintptr_t>(c_rows) & 3u)) return ENTMAX_ATTN_EINVAL_ALIGN;
  if (alibi && (reinterpret_cast<uintptr_t>(alibi) & 3u)) return ENTMAX_ATTN_EINVAL_ALIGN;
  if (alibi && p.dtype == ENTMAX_ATTN_DTYPE_BF16 && !p.causal) return ENTMAX_ATTN_EUNSUPPORTED;
  p.alibi = alibi;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(tau) || !aligned16(d_o) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv))
    return ENTMAX_ATTN_EINVAL_ALIGN;
  WsLayout lay;
  rc = check_workspace(p, true, workspace, workspace_bytes, &lay);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (p.dtype == ENTMAX_ATTN_DTYPE_BF16) {
    rc = check_device_for_bf16();
    if (rc != ENTMAX_ATTN_OK) return rc;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const float* scale = reinterpret_cast<float*>(ws + lay.scale);
  int32_t* half_cnt = reinterpret_cast<int32_t*>(ws + lay.half_cnt);
  float* half_thr = reinterpret_cast<float*>(ws + lay.half_thr);
  int32_t* sweep_counter = reinterpret_cast<int32_t*>(ws + lay.sweep_counter);
  Entry* entries = reinterpret_cast<Entry*>(ws + lay.entries);
  int32_t* fb_count = reinterpret_cast<int32_t*>(ws + lay.fb_count);
  int32_t* fb_list = reinterpret_cast<int32_t*>(ws + lay.fb_list);
  float* scratch = reinterpret_cast<float*>(ws + lay.scratch);
  float* acc_dk = reinterpret_cast<float*>(ws + lay.acc_dk);
  float* acc_dv = reinterpret_cast<float*>(ws + lay.acc_dv);
  const size_t acc_bytes = (size_t)p.B * p.H * p.N * p.D * sizeof(float);
  // per-row scale gradients: into the caller's array, else (when only the parameter gradients are wanted)
  // into the workspace, else not computed
  float* dc_rows = d_scale_rows ? d_scale_rows : (n_param_grads ? reinterpret_cast<float*>(ws + lay.dc_rows) : nullptr);
  cudaError_t err;
  if (device_status) {
    err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  // with a score sweep ahead (bf16, no saved supports) the accumulators are cleared beside it, otherwise in line
  const bool clear_aside = p.dtype == ENTMAX_ATTN_DTYPE_BF16 && !fwd_workspace && !saved_supports;
  SideStream* side = nullptr;
  if (clear_aside) {
    err = side_stream(&side);
    if (err != cudaSuccess) return fail_cuda(err);
    err = cudaEventRecord(side->fork, stream);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(side->stream, side->fork, 0);
    if (err == cudaSuccess) err = cudaMemsetAsync(acc_dk, 0, acc_bytes, side->stream);
    if (err == cudaSuccess) err = cudaMemsetAsync(acc_dv, 0, acc_bytes, side->stream);
    if (err == cudaSuccess) err = cudaEventRecord(side->join, side->stream);
    if (err != cudaSuccess) return fail_cuda(err);
  } else {
    err = cudaMemsetAsync(acc_dk, 0, acc_bytes, stream);
    if (err != cudaSuccess) return fail_cuda(err);
    err = cudaMemsetAsync(acc_dv, 0, acc_bytes, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  if (c_rows) {
    scale = c_rows;
    p.scale_sb = (int64_t)p.H * p.N;
  } else {
    err = launch_scale_table(p, beta, gamma, delta, reinterpret_cast<float*>(ws + lay.scale), device_status, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  if (p.dtype == ENTMAX_ATTN_DTYPE_FP32) {
    err = launch_dense_bwd(p, q, k, v, d_o, scale, tau, dq, acc_dk, acc_dv, dc_rows, nullptr, nullptr, scratch,
                           lay.scratch_floats, lay.scratch_ctas, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  } else {
    int32_t* tile_flag = reinterpret_cast<int32_t*>(ws + lay.tile_flag);
    int32_t* tile_list = reinterpret_cast<int32_t*>(ws + lay.tile_list);
    int32_t* tile_count = reinterpret_cast<int32_t*>(ws + lay.tile_count);
    uint32_t* tile_mask = reinterpret_cast<uint32_t*>(ws + lay.tile_mask);
    const size_t q_tiles = (size_t)p.B * p.H * ((p.N + 127) / 128);
    err = cudaMemsetAsync(fb_count, 0, 256, stream);   // the whole counter block
    if (err != cudaSuccess) return fail_cuda(err);
    // tile flags, tile list and tile masks are adjacent in the workspace: one memset clears all three
    err = cudaMemsetAsync(tile_flag, 0, lay.tile_mask + q_tiles * 4 * sizeof(uint32_t) - lay.tile_flag, stream);
    if (err != cudaSuccess) return fail_cuda(err);
    if (saved_supports) {
      // the compact copy of the forward call's supports: no score sweep; rows it does not hold count as dense
      const SavedLayout sl = saved_layout(p);
      const uint8_t* sv = static_cast<const uint8_t*>(saved_supports);
      err = launch_row_bwd(p, q, k, v, d_o, scale, tau, reinterpret_cast<const int32_t*>(sv + sl.counts),
                           const_cast<Entry*>(reinterpret_cast<const Entry*>(sv + sl.entries)), dq, acc_dk, acc_dv,
                           dc_rows, fb_count, fb_list, device_status, 1, ENTMAX_ATTN_SAVED_SLOTS, stream);
      if (err != cudaSuccess) return fail_cuda(err);
    } else if (fwd_workspace) {
      // the forward call's workspace still holds every row's support: no score sweep needed
      const WsLayout fl = make_layout(p, false);
      const uint8_t* fws = static_cast<const uint8_t*>(fwd_workspace);
      err = launch_row_bwd(p, q, k, v, d_o, scale, tau, reinterpret_cast<const int32_t*>(fws + fl.row_cnt),
                           const_cast<Entry*>(reinterpret_cast<const Entry*>(fws + fl.entries)), dq, acc_dk, acc_dv,
                           dc_rows, fb_count, fb_list, device_status, 1, kListCap, stream);
      if (err != cudaSuccess) return fail_cuda(err);
    } else {
      if (g_prof_start[1]) cudaEventRecord(g_prof_start[1], stream);
      err = launch_sweep(p, q, k, scale, tau, 1, half_cnt, half_thr, entries, sweep_counter, nullptr, -1,
                         reinterpret_cast<float*>(ws + lay.alibi_blob), reinterpret_cast<float*>(ws + lay.alibi_kmax),
                         device_status, stream);
      if (err != cudaSuccess) return fail_cuda(err);
      if (g_prof_stop[1]) cudaEventRecord(g_prof_stop[1], stream);
      err = cudaStreamWaitEvent(stream, side->join, 0);     // the accumulators are clear from here on
      if (err != cudaSuccess) return fail_cuda(err);
      err = launch_row_bwd(p, q, k, v, d_o, scale, tau, half_cnt, entries, dq, acc_dk, acc_dv, dc_rows, fb_count,
                           fb_list, device_status, 0, kListCap, stream);
      if (err != cudaSuccess) return fail_cuda(err);
    }
    // rows whose support does not fit the lists: dense tiles on the tensor cores
    err = launch_tile_bwd(p, q, k, v, d_o, scale, tau, fb_list, fb_count, tile_mask, tile_flag, tile_list, tile_count, tile_count + 16,
                          reinterpret_cast<float*>(ws + lay.half_thr) /* idle after the sweep: rho of the dense rows */, dq,
                          acc_dk, acc_dv, dc_rows, device_status, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  err = launch_store_grad(p, acc_dk, dk, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  err = launch_store_grad(p, acc_dv, dv, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  if (n_param_grads) {
    err = launch_scale_grad(p, beta, gamma, dc_rows, dbeta, dgamma, ddelta, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  return ENTMAX_ATTN_OK;
}

}  // namespace

extern "C" {

int entmax_attn_bwd_scale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                          const float* beta, const float* gamma, const float* delta, const float* tau,
                          const void* d_o, void* dq, void* dk, void* dv, float* d_scale_rows, float* dbeta,
                          float* dgamma, float* ddelta, void* workspace, size_t workspace_bytes,
                          int32_t* device_status, void* cuda_stream) {
  return bwd_impl(params, q, k, v, beta, gamma, delta, nullptr, nullptr, nullptr, nullptr, tau, d_o, dq, dk, dv, d_scale_rows, dbeta,
                  dgamma, ddelta, workspace, workspace_bytes, device_status, cuda_stream);
}

int entmax_attn_bwd_ex(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                       const float* beta, const float* gamma, const float* delta, const entmax_attn_extras* extras,
                       const float* tau, const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                       size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  entmax_attn_extras ex = {};
  if (extras) ex = *extras;
  if (ex.c_rows && (beta || gamma || delta)) return ENTMAX_ATTN_EINVAL_NULL;
  if (ex.fwd_workspace && (reinterpret_cast<uintptr_t>(ex.fwd_workspace) & 255u)) return ENTMAX_ATTN_EINVAL_WORKSPACE;
  if (ex.saved_supports && (reinterpret_cast<uintptr_t>(ex.saved_supports) & 255u)) return ENTMAX_ATTN_EINVAL_WORKSPACE;
  return bwd_impl(params, q, k, v, beta, gamma, delta, ex.c_rows, ex.alibi_slopes, ex.fwd_workspace, ex.saved_supports, tau,
                  d_o, dq, dk, dv,
                  ex.d_scale_rows, ex.dbeta, ex.dgamma, ex.ddelta, workspace, workspace_bytes, device_status,
                  cuda_stream);
}

int entmax_attn_bwd_rowscale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                             const float* c_rows, const float* tau, const void* d_o, void* dq, void* dk, void* dv,
                             float* d_scale_rows, void* workspace, size_t workspace_bytes, int32_t* device_status,
                             void* cuda_stream) {
  if (!c_rows) return ENTMAX_ATTN_EINVAL_NULL;
  return bwd_impl(params, q, k, v, nullptr, nullptr, nullptr, c_rows, nullptr, nullptr, nullptr, tau, d_o, dq, dk, dv, d_scale_rows,
                  nullptr, nullptr, nullptr, workspace, workspace_bytes, device_status, cuda_stream);
}

int entmax_attn_bwd(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                    const float* beta, const float* gamma, const float* delta, const float* tau,
                    const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                    size_t workspace_bytes, int32_t* device_status, void* cuda_stream) {
  return entmax_attn_bwd_scale(params, q, k, v, beta, gamma, delta, tau, d_o, dq, dk, dv, nullptr, nullptr, nullptr,
                               nullptr, workspace, workspace_bytes, device_status, cuda_stream);
}

int entmax_attn_scores_debug(const entmax_attn_params* params, const void* q, const void* k, int32_t bh,
                             float* s_out, void* workspace, size_t workspace_bytes, int32_t* device_status,
                             void* cuda_stream) {
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (p.dtype != ENTMAX_ATTN_DTYPE_BF16) return ENTMAX_ATTN_EINVAL_DTYPE;
  if (!q || !k || !s_out) return ENTMAX_ATTN_EINVAL_NULL;
  if (bh < 0 || bh >= p.B * p.H) return ENTMAX_ATTN_EINVAL_SHAPE;
  if (!aligned16(q) || !aligned16(k)) return ENTMAX_ATTN_EINVAL_ALIGN;
  WsLayout lay;
  rc = check_workspace(p, false, workspace, workspace_bytes, &lay);
  if (rc != ENTMAX_ATTN_OK) return rc;
  rc = check_device_for_bf16();
  if (rc != ENTMAX_ATTN_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* scale = reinterpret_cast<float*>(ws + lay.scale);
  cudaError_t err;
  if (device_status) {
    err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  err = launch_scale_table(p, nullptr, nullptr, nullptr, scale, device_status, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  err = launch_sweep(p, q, k, scale, nullptr, 0, reinterpret_cast<int32_t*>(ws + lay.half_cnt),
                     reinterpret_cast<float*>(ws + lay.half_thr), reinterpret_cast<Entry*>(ws + lay.entries),
                     reinterpret_cast<int32_t*>(ws + lay.sweep_counter), s_out, bh, nullptr, nullptr, device_status, stream);
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}

size_t entmax_attn_saved_bytes(const entmax_attn_params* params) {
  Problem p;
  if (make_problem(params, &p) != ENTMAX_ATTN_OK || p.dtype != ENTMAX_ATTN_DTYPE_BF16) return 0;
  return saved_layout(p).total;
}

int entmax_attn_save_supports(const entmax_attn_params* params, const void* fwd_workspace, void* saved, size_t saved_bytes,
                              void* cuda_stream) {
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (p.dtype != ENTMAX_ATTN_DTYPE_BF16) return ENTMAX_ATTN_EINVAL_DTYPE;
  if (!fwd_workspace || !saved) return ENTMAX_ATTN_EINVAL_NULL;
  const SavedLayout sl = saved_layout(p);
  if ((reinterpret_cast<uintptr_t>(fwd_workspace) & 255u) || (reinterpret_cast<uintptr_t>(saved) & 255u) ||
      saved_bytes < sl.total)
    return ENTMAX_ATTN_EINVAL_WORKSPACE;
  const WsLayout fl = make_layout(p, false);
  const uint8_t* fws = static_cast<const uint8_t*>(fwd_workspace);
  uint8_t* sv = static_cast<uint8_t*>(saved);
  cudaError_t err = launch_save_supports(p, ENTMAX_ATTN_SAVED_SLOTS, reinterpret_cast<const int32_t*>(fws + fl.row_cnt),
                                         reinterpret_cast<const Entry*>(fws + fl.entries),
                                         reinterpret_cast<int32_t*>(sv + sl.counts), reinterpret_cast<Entry*>(sv + sl.entries),
                                         static_cast<cudaStream_t>(cuda_stream));
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}

int entmax_attn_profile_events(int which, void* start_event, void* stop_event) {
  if (which != 0 && which != 1) return ENTMAX_ATTN_EINVAL_SHAPE;
  if ((start_event == nullptr) != (stop_event == nullptr)) return ENTMAX_ATTN_EINVAL_NULL;
  g_prof_start[which] = static_cast<cudaEvent_t>(start_event);
  g_prof_stop[which] = static_cast<cudaEvent_t>(stop_event);
  return ENTMAX_ATTN_OK;
}

const char* entmax_attn_strerror(int code) {
  switch (code) {
    case ENTMAX_ATTN_OK: return "ok";
    case ENTMAX_ATTN_EINVAL_SHAPE: return "invalid shape or strides (head_dim must be 64 or 128; sizes >= 1; strides multiples of 8)";
    case ENTMAX_ATTN_EINVAL_ALPHA: return "alpha must lie in (1, 64] and sm_scale must be finite and non-negative";
    case ENTMAX_ATTN_EINVAL_DTYPE: return "unknown or unsupported dtype";
    case ENTMAX_ATTN_EINVAL_ALIGN: return "tensor pointers must be 16-byte aligned";
    case ENTMAX_ATTN_EINVAL_WORKSPACE: return "workspace missing, not 256-byte aligned, or too small";
    case ENTMAX_ATTN_EINVAL_NULL: return "a required pointer is NULL (beta, gamma, delta: all or none)";
    case ENTMAX_ATTN_ECUDA: return "a CUDA call failed (see entmax_attn_last_cuda_error)";
    case ENTMAX_ATTN_EUNSUPPORTED: return "the bf16 path needs an sm_100 device";
    case ENTMAX_ATTN_ETOOLARGE: return "the problem does not fit the library's built-in scratch (see entmax_attn_fwd_static)";
    default: return "unknown status";
  }
}

int entmax_attn_last_cuda_error(void) { return g_last_cuda_error; }

int entmax_attn_version(void) { return 200; }   // 0.2.0: decode entry point, dense-tile backward

}  // extern "C"
