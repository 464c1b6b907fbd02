// Self-test of the bounded device-side wait that the tensor-core kernels are built on.
//
// Those kernels never wait without a limit inside their pipelines: a wait that runs out raises the block's abort
// flag, every other wait of the block then returns at once, the block drains, frees its tensor memory and records
// TASKKV_ETIMEOUT.  A healthy run never takes that path, so this file exercises it on purpose in the only safe
// form: a one-block kernel with no copy or MMA in flight waits on a barrier that nothing will ever complete, with a
// small poll limit, and then returns normally.  Nothing faults and nothing is left hanging.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace taskkv {
namespace {

// out[0]: status word (sticky, as in a cache); out[1]: polls of the first wait; out[2]: polls of the second
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(int32_t* out, uint32_t limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(tc::smem_u32(&bar), 1);       // one arrival expected; none will come
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  uint32_t polls1 = 0, polls2 = 0;
  // the whole warp waits, as the role loops of the kernels do
  const bool first = tc::mbar_wait_limit(tc::smem_u32(&bar), 0, &abort_flag, limit, &polls1);
  const bool ok1 = __all_sync(0xffffffffu, first);
  // the block is now aborting: any further wait gives up on its first poll
  const bool second = tc::mbar_wait_limit(tc::smem_u32(&bar), 0, &abort_flag, limit, &polls2);
  const bool ok2 = __all_sync(0xffffffffu, second);
  if (threadIdx.x == 0) {
    if (!ok1 && !ok2 && abort_flag) set_status(out, TASKKV_ETIMEOUT);
    out[1] = (int32_t)polls1;
    out[2] = (int32_t)polls2;
  }
}

}  // namespace
}  // namespace taskkv

extern "C" taskkv_status taskkv_selftest_bounded_wait(int32_t max_polls, int32_t* polls_out, taskkv_stream stream) {
  using namespace taskkv;
  if (max_polls < 1) max_polls = 1;
  if (max_polls > 65536) max_polls = 65536;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t* dev = nullptr;
  if (cudaMalloc(&dev, 3 * sizeof(int32_t)) != cudaSuccess) {
    cudaGetLastError();
    return TASKKV_EALLOC;
  }
  int32_t host[3] = {0, 0, 0};
  cudaError_t e = cudaMemsetAsync(dev, 0, sizeof(host), s);
  if (e == cudaSuccess) {
    LaunchScope ls(K_SELFTEST, s);
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(dev, (uint32_t)max_polls);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(host, dev, sizeof(host), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  cudaFree(dev);
  if (e != cudaSuccess) return TASKKV_ECUDA;
  if (polls_out) *polls_out = host[1];
  // the second wait must have returned on its first poll
  if (host[0] == TASKKV_ETIMEOUT && host[2] != 0) return TASKKV_ECUDA;
  return (taskkv_status)host[0];
}
