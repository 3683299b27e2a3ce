// A self-check of the bounded device-side waits: one thread block waits on a barrier that nothing ever
// completes, so the wait runs out, the block leaves the way the tensor-core kernels leave after a wait that
// gave up (its tensor memory freed, a flag raised) and the GPU context stays usable.
#include "sm100_ptx.cuh"
#include "ug_common.cuh"

namespace ug {
namespace {

using namespace sm100;

__device__ unsigned int g_selftest_timeout = 0;

__global__ void __launch_bounds__(128) wait_that_runs_out_kernel() {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t tmem_slot;
  const uint32_t bar = smem_u32(&bar_storage);
  const int warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);  // one arrival expected; nobody arrives
    mbar_fence_init();
  }
  if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 32);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  // every warp waits, converged, as the compute warps of the attention kernels do
  const bool ok = mbar_wait_warp(bar, 0);
  if (!ok && (threadIdx.x & 31) == 0) atomicExch(&g_selftest_timeout, 1u);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tmem_dealloc(tmem, 32);
  }
}

}  // namespace

int32_t launch_selftest_wait(cudaStream_t st) {
  {
    KernelScope ks("wait_that_runs_out_kernel", st);
    wait_that_runs_out_kernel<<<1, 128, 0, st>>>();
  }
  return check_launch("bounded-wait self-check kernel");
}

int32_t selftest_take_timeout(bool* timed_out) {
  unsigned int flag = 0, zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(&flag, g_selftest_timeout, sizeof(flag));
  if (e == cudaSuccess && flag) e = cudaMemcpyToSymbol(g_selftest_timeout, &zero, sizeof(zero));
  if (e != cudaSuccess) return fail(UNIGIST_ERR_CUDA, "reading the device status: %s", cudaGetErrorString(e));
  *timed_out = flag != 0;
  return UNIGIST_OK;
}

}  // namespace ug
