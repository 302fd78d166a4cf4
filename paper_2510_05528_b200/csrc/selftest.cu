// Self-test of the bounded waits: the one path of the tensor-core kernels that ordinary runs never take.
#include "tc_common.cuh"

namespace {

// One warp.  Lane 0 initialises an mbarrier that nothing ever arrives on and waits on it with the given cycle
// limit, through the same routine the tensor-core kernels use.  No bulk copy is in flight and no tensor memory
// is held, so giving up is all there is to clean up: the wait must return false, raise ST_WAIT_TIMEOUTS and
// record ARMOR_ERR_TIMEOUT, and the kernel must end normally.
__global__ void wait_timeout_kernel(long long limit, int32_t* status, int32_t* result) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(tc::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool got = tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, status, limit);
    result[0] = got ? 1 : 0;            // 0: the wait gave up, as it must
    result[1] = abort_flag;             // 1: the CTA-wide abort flag is up, the other roles would leave too
  }
}

}  // namespace

extern "C" armor_status armor_selftest_wait_timeout(armor_ctx* c, int64_t limit_cycles, int32_t* d_result,
                                                    armor_stream_t stream) {
  if (!c || !d_result || limit_cycles < 1 || limit_cycles > 2000000000ll) return ARMOR_ERR_INVALID_ARG;
  wait_timeout_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(limit_cycles, c->status, d_result);
  c->launches++;
  return finish_call(c);
}
