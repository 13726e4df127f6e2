// entmax_attn_fwd_static: the dense-row forward pass with its scratch memory inside the library.
//
// The other entry points take a caller-allocated workspace.  Some callers have no way to get one: code
// that runs where device allocation is forbidden or unavailable (inside a region that must not call
// the allocator, in a plugin that is handed tensors but no allocator, in a start-up or recovery path
// that runs before the framework's memory pool exists).  For them this file keeps a fixed scratch
// array in device memory that is part of the loaded library image: every GPU that loads the library
// holds ENTMAX_ATTN_STATIC_SCRATCH_BYTES of it until the process exits, and nothing is ever allocated
// or freed here.
//
// The computation is the one of the dense-row path (dense_rows.cu): the ASEntmax scale table, then one
// CTA per query row: fp32 dot products with every visible key, Newton on the cached scores, p and
// O = P V.  The scratch holds the scale table ([heads, seq] floats) followed by one score row per CTA.
#include <mutex>

#include "common.cuh"

namespace entmax {

namespace {

constexpr size_t kStaticFloats = ENTMAX_ATTN_STATIC_SCRATCH_BYTES / sizeof(float);
constexpr int kMinCtas = 64;     // the size limit guarantees at least this many score rows
constexpr int kMaxCtas = 148 * 4;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol lookup, never
// a device address: the address that kernels may use comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) float g_static_scratch[kStaticFloats];

std::mutex g_setup_mutex;
float* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch on each device, once looked up

// Device address of the scratch array on the current device; looked up once per device.
cudaError_t scratch_address(float** out) {
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    float* ptr = nullptr;
    err = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch);
    if (err != cudaSuccess) return err;
    if (!ptr) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

inline size_t round_up32(size_t x) { return (x + 31) / 32 * 32; }

}  // namespace

}  // namespace entmax

using namespace entmax;

extern "C" int entmax_attn_fwd_static(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                                      const float* beta, const float* gamma, const float* delta, void* o, float* tau,
                                      int32_t* device_status, void* cuda_stream) {
  // ---- validation (the rules and codes of entmax_attn_fwd), before any CUDA call
  Problem p;
  int rc = make_problem(params, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  // ---- the size limit: scale table + at least kMinCtas score rows must fit the fixed array
  const size_t row_floats = round_up32((size_t)p.N);
  const size_t scale_floats = round_up32((size_t)p.H * p.N);
  if (scale_floats + (size_t)kMinCtas * row_floats > kStaticFloats) return ENTMAX_ATTN_ETOOLARGE;
  if (!q || !k || !v || !o || !tau) return ENTMAX_ATTN_EINVAL_NULL;
  rc = check_scale_ptrs(beta, gamma, delta, &p);
  if (rc != ENTMAX_ATTN_OK) return rc;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(tau)) return ENTMAX_ATTN_EINVAL_ALIGN;
  const size_t rows = (size_t)p.B * p.H * p.N;
  size_t ctas = (kStaticFloats - scale_floats) / row_floats;
  if (ctas > (size_t)kMaxCtas) ctas = kMaxCtas;
  if (ctas > rows) ctas = rows;

  float* scratch = nullptr;
  cudaError_t err = scratch_address(&scratch);
  if (err != cudaSuccess) return fail_cuda(err);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (device_status) {
    err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
    if (err != cudaSuccess) return fail_cuda(err);
  }
  // Nothing in the scratch has to start at zero: the scale table is written in full before it is read,
  // and every CTA fills its score row for the keys of a query before it reads them.
  float* scale = scratch;
  float* score_rows = scratch + scale_floats;
  err = launch_scale_table(p, beta, gamma, delta, scale, device_status, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  err = launch_dense_fwd(p, q, k, v, scale, o, tau, nullptr, nullptr, nullptr, nullptr, nullptr, score_rows, row_floats,
                         (int)ctas, stream);
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}
