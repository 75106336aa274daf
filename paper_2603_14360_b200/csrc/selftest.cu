// Self-test of the bounded device-side wait that every kernel of the library is built on.
//
// A kernel of one warp initialises an mbarrier that nothing ever completes and waits on it with
// the same mbar_wait the scan kernels use, with a limit the host passes.  The wait must give up,
// the kernel must report M2RNN_ERR_TIMEOUT through the status word and return normally: no trap,
// no endless loop, and the context stays usable.  This is how a hung producer (a staging warp that
// died, a copy that never landed) would surface in the scan kernels.
#include "internal.h"
#include "pipeline.cuh"

namespace m2rnn {
namespace {

__global__ void wait_selftest_kernel(long long limit_cycles, int32_t *dev_status, long long *waited_cycles) {
  __shared__ uint64_t never;
  if (threadIdx.x == 0) {
    mbar_init(&never, 1);
    fence_mbar_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  const bool ok = mbar_wait(&never, 0, limit_cycles);
  if (!ok) report_timeout(dev_status);
  if (threadIdx.x == 0 && waited_cycles) *waited_cycles = clock64() - t0;
}

}  // namespace
}  // namespace m2rnn

extern "C" int m2rnn_wait_selftest(int64_t limit_cycles, int32_t *dev_status, int64_t *waited_cycles, void *stream) {
  if (!dev_status) return M2RNN_ERR_NULL;
  // the limit is bounded on the host: a self-test has no business waiting longer than ~50 ms
  if (limit_cycles < 0 || limit_cycles > 100000000) return M2RNN_ERR_SHAPE;
  m2rnn::wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
      (long long)limit_cycles, dev_status, reinterpret_cast<long long *>(waited_cycles));
  if (cudaGetLastError() != cudaSuccess) return M2RNN_ERR_CUDA;
  return M2RNN_OK;
}
