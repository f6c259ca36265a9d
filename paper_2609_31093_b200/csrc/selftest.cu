// Self-test of the bounded device-side waits: the same mbar_wait_bounded every tile kernel uses, on a
// barrier nobody arrives at.  The wait gives up after its limit, the kernel records PISA_ERR_TIMEOUT in
// the status word and returns normally, and the context stays usable.
#include "pisa_common.cuh"
#include "tc_utils.cuh"

namespace pisa {

namespace {
__global__ void __launch_bounds__(32) wait_timeout_kernel(int32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);                 // expects one arrival; none is ever made
    tc::mbar_fence_init();
  }
  __syncwarp();
  if (threadIdx.x == 0) {
    const bool ok = tc::mbar_wait_bounded(&bar, 0u, limit_ns);
    if (!ok) atomicExch(status, (int)PISA_ERR_TIMEOUT);
  }
}
}  // namespace

int launch_wait_timeout(int32_t* status, unsigned long long limit_ns, cudaStream_t s) {
  wait_timeout_kernel<<<1, 32, 0, s>>>(status, limit_ns);
  return check_launch("wait_timeout");
}

}  // namespace pisa
