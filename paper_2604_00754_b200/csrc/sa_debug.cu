// Test hook for the failure path of the bounded waits: a kernel whose only wait can never be
// satisfied, with a short limit, so that the give-up branch of mbar_wait runs on a GPU without
// any kernel being broken for it.
#include "sa_tc_common.cuh"

namespace sa {
namespace {

__global__ void __launch_bounds__(32, 1) wait_timeout_kernel(int* status, long long limit) {
  __shared__ __align__(8) uint64_t barrier;
  __shared__ int gave_up;
  const uint32_t bar = smem_u32(&barrier);
  if (threadIdx.x == 0) {
    gave_up = 0;
    mbar_init(bar, 1);                      // one arrival expected; nobody arrives
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  // every lane waits, as the row threads of the attention kernels do; the first lane whose
  // limit runs out records the status and raises the flag the others leave on
  const bool ok = mbar_wait(bar, 0u, &gave_up, status, limit);
  (void)ok;
}

}  // namespace
}  // namespace sa

extern "C" sa_status sa_debug_wait_timeout(int64_t limit_cycles, sa_stream_t stream) {
  using namespace sa;
  if (limit_cycles < 1 || limit_cycles > (1ll << 31)) return SA_ERR_INVALID_ARG;
  int* status = status_ptr();
  if (!status) return SA_ERR_CUDA;
  wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(status, (long long)limit_cycles);
  bump_launches();
  return cudaGetLastError() == cudaSuccess ? SA_OK : SA_ERR_CUDA;
}
