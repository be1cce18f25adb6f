// isopo_selftest_bounded_wait: makes one of the library's bounded mbarrier waits run out on purpose,
// the safe way, so that the give-up path every tensor-core kernel relies on (abort flag, *info,
// all roles reaching the common teardown) is exercised on real hardware.
//
// One CTA of three warps and one mbarrier that nobody ever arrives on.  No TMA copy, no tensor
// memory, no other barrier is involved, so there is nothing in flight to clean up: warp 0 waits with
// the caller's clock limit through the very mbar_wait the kernels use and gives up; warp 1 waits with
// the kernels' default limit and leaves as soon as it sees the CTA's abort flag; warp 2 plays a role
// that has no waits.  All meet at the teardown barrier and the kernel returns normally.
#include "tc_common.cuh"

namespace isopo {

namespace {

using namespace tc;

__global__ void __launch_bounds__(96) k_wait_probe(long long limit, int32_t* info, int* roles_at_teardown) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  if (warp == 0) {
    mbar_wait(smem_u32(&bar), 0, abort_flag, info, kIdWaitProbe, limit);  // phase 0 never completes: gives up
  } else if (warp == 1) {
    mbar_wait(smem_u32(&bar), 0, abort_flag, info, kIdWaitProbe);         // default limit; released by the abort flag
  }
  // ---- teardown, as in the tensor-core kernels: every role gets here whatever its wait returned
  __syncthreads();
  if ((threadIdx.x & 31) == 0) atomicAdd(roles_at_teardown, 1);
}

}  // namespace

isopo_status wait_probe(long long limit, int32_t* info, int32_t* roles_at_teardown, cudaStream_t st) {
  ISOPO_CUDA_TRY(cudaMemsetAsync(roles_at_teardown, 0, sizeof(int32_t), st));
  {
    LaunchScope scope(kIdWaitProbe, st);
    k_wait_probe<<<1, 96, 0, st>>>(limit, info, roles_at_teardown);
  }
  ISOPO_CUDA_TRY(cudaGetLastError());
  return ISOPO_OK;
}

}  // namespace isopo
