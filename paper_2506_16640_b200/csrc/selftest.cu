// Self-test of the bounded waits.  Every mbarrier wait of the tensor-core kernels goes through
// sm100::mbar_wait_slow, which gives up after a time limit, raises the CTA's abort word and lets every role leave
// its loop; the kernels then flag ENTMAX_ATTN_FLAG_WAIT_EXPIRED and return.  In a healthy run no wait ever expires,
// so this entry point makes one expire on purpose, the sanctioned way: a barrier that nothing arrives on, waited for
// with a limit of a few milliseconds given by the caller.  Nothing traps, nothing spins past the limit.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace entmax {

namespace {

using namespace sm100;

__global__ void __launch_bounds__(64) wait_expiry_kernel(unsigned long long limit_ns, int32_t* status) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t abort_word;
  const uint32_t bar = smem_u32(&bar_storage), abort_flag = smem_u32(&abort_word);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);            // one arrival expected; nobody will make it
    sts_u32(abort_flag, 0u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const unsigned long long t0 = global_ns();
  bool alive = true;
  if (threadIdx.x >= 32) {
    // the waiting role: the same call the kernels make, with the caller's limit instead of the built-in one
    if (!mbar_try_wait(bar, 0u)) alive = mbar_wait_slow(bar, 0u, abort_flag, limit_ns);
  } else {
    // a second role that notices the abort word, as the other warps of a real kernel do
    while (lds_u32(abort_flag) == 0u && global_ns() - t0 < 4ull * limit_ns + 1000000ull) { }
  }
  const unsigned long long waited = global_ns() - t0;
  __syncthreads();
  if (threadIdx.x == 32 && status) {
    if (!alive && lds_u32(abort_flag)) atomicOr(status + ENTMAX_ATTN_STATUS_FLAGS, ENTMAX_ATTN_FLAG_WAIT_EXPIRED);
    status[ENTMAX_ATTN_STATUS_DENSE_ROWS] = (int32_t)(waited / 1000ull);   // microseconds the wait lasted
  }
}

}  // namespace

}  // namespace entmax

using namespace entmax;

extern "C" int entmax_attn_selftest_wait_expiry(uint64_t limit_ns, int32_t* device_status, void* cuda_stream) {
  if (!device_status) return ENTMAX_ATTN_EINVAL_NULL;
  if (limit_ns == 0 || limit_ns > 100000000ull) return ENTMAX_ATTN_EINVAL_SHAPE;   // at most 100 ms
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t err = cudaMemsetAsync(device_status, 0, sizeof(int32_t) * ENTMAX_ATTN_STATUS_WORDS, stream);
  if (err != cudaSuccess) return fail_cuda(err);
  wait_expiry_kernel<<<1, 64, 0, stream>>>(limit_ns, device_status);
  err = cudaGetLastError();
  return err == cudaSuccess ? ENTMAX_ATTN_OK : fail_cuda(err);
}
