// Self-test of the bounded wait used by the tensor-core kernels: one thread waits on an mbarrier that
// nothing ever arrives at, gives up after `limit` cycles, records kErrTimeout and returns.  The kernel
// always terminates by itself; the context stays usable.
#include "../../include/prism_ops.h"
#include "tc_common.cuh"

namespace prism {
namespace {

__global__ void k_wait_selftest(unsigned long long limit, int* __restrict__ err) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // phase 0 never completes: the wait must return false once the limit has passed
    if (tc::mbar_wait(tc::smem_u32(&bar), 0, err, &abort_flag, limit)) atomicOr(err, kErrInternal);
  }
}

}  // namespace
}  // namespace prism

extern "C" int prism_op_wait_selftest(uint64_t limit_cycles, int32_t* err_word, void* stream) {
  if (!err_word || limit_cycles == 0 || limit_cycles > 2000000000ull) return PRISM_ERR_INVALID_ARG;
  prism::k_wait_selftest<<<1, 32, 0, reinterpret_cast<cudaStream_t>(stream)>>>(limit_cycles, err_word);
  return cudaGetLastError() == cudaSuccess ? PRISM_OK : PRISM_ERR_CUDA;
}
