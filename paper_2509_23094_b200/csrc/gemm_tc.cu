// tcgen05 / TMEM GEMM (placeholder until the kernel lands): reports that it is not built.
#include "common.cuh"
namespace d2c {
int launch_gemm_tc(const GemmArgs&, GemmEpilogue, cudaStream_t) {
  set_global_error("tcgen05 GEMM is not built in this library");
  return D2C_ESHAPE;
}
}  // namespace d2c
