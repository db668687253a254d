// The give-up path of the bounded mbarrier wait every tcgen05 kernel of this library uses, run on its own:
// one CTA waits on a barrier that nothing will ever arrive on, with a short cycle limit.  No TMA, no TMEM, no
// tensor-core work: the kernel returns after the limit and the status word holds D2C_ETIMEOUT and the wait's
// site number, which is what d2c_sync_status reports after a step whose pipeline wait ran out.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace d2c {
namespace {
constexpr int kProbeSite = 99;

__global__ void __launch_bounds__(64) wait_probe_kernel(int* status, long long limit) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // every thread gives up on its own after `limit` clocks (or earlier, once another thread has)
  mbar_wait(b, 0, &abort_flag, status, kProbeSite, limit);
}
}  // namespace
}  // namespace d2c

extern "C" int d2c_op_wait_probe(int32_t* status, int64_t limit_cycles, void* cuda_stream) {
  using namespace d2c;
  if (!status) { set_global_error("d2c_op_wait_probe: status is null"); return D2C_EINVAL; }
  if (limit_cycles < 1000 || limit_cycles > 2000000000LL) {
    set_global_error("d2c_op_wait_probe: limit_cycles %lld outside [1e3, 2e9]", (long long)limit_cycles);
    return D2C_EINVAL;
  }
  wait_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>(reinterpret_cast<int*>(status), (long long)limit_cycles);
  D2C_LAUNCHED();
  return D2C_OK;
}
