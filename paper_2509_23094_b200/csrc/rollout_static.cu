// d2c_op_rollout_static: the rollout chain for callers that must not allocate device memory.
//
// Some users of this library cannot hand it a scratch buffer because they cannot obtain one at the
// point of the call: a serving engine that gave all free HBM to its KV-cache arena at start-up, a
// plug-in that runs inside someone else's stream-ordered region where cudaMalloc's implicit
// synchronisation is not acceptable, or code that simply has no allocator handle.  For them the
// scratch of the rollout kernels lives in a fixed array inside the library image.  Every GPU that
// loads the library carries that array (about 1.2 MB) until the process exits.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int kMaxPositions = 16384;                                   // batch * seq_len accepted by this entry point
constexpr size_t kVec = ((size_t)kMaxPositions * 4 + 255) / 256 * 256;  // one fp32 vector over the positions
constexpr size_t kScratchBytes = 2 * kVec + ((size_t)d2c::kRolloutSplit * kMaxPositions * 4 + kMaxPositions + 255) / 256 * 256;

// In host code this name is only a handle for the runtime, not an address the GPU understands.
static __device__ __align__(256) unsigned char g_rollout_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device, looked up once per device.
int scratch_on_current_device(void** out) {
  int dev = 0;
  D2C_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) { d2c::set_global_error("d2c_op_rollout_static: device ordinal %d not supported", dev); return D2C_ECAPACITY; }
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    D2C_CUDA_OK(cudaGetSymbolAddress(&p, g_rollout_scratch));
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return D2C_OK;
}

}  // namespace

extern "C" int d2c_op_rollout_static(const float* abar, size_t layer_stride, int32_t n_layers, const int32_t* sel_idx,
                                     const int32_t* row_off, int32_t batch, int32_t seq_len, float* c, void* cuda_stream) {
  using namespace d2c;
  if (!abar || !sel_idx || !row_off || !c) { set_global_error("d2c_op_rollout_static: null pointer"); return D2C_EINVAL; }
  if (n_layers < 1 || batch < 1 || seq_len < 1) { set_global_error("d2c_op_rollout_static: bad sizes"); return D2C_EINVAL; }
  if ((long long)batch * seq_len > kMaxPositions) {
    set_global_error("d2c_op_rollout_static: batch*seq_len = %lld exceeds the built-in scratch (%d positions); "
                     "use d2c_op_rollout with caller-provided scratch", (long long)batch * seq_len, kMaxPositions);
    return D2C_ECAPACITY;
  }
  void* base = nullptr;
  int rc = scratch_on_current_device(&base);
  if (rc != D2C_OK) return rc;
  char* sp = static_cast<char*>(base);
  const size_t R = (size_t)batch * seq_len;
  RolloutArgs r{};
  r.abar = abar; r.layer_stride = layer_stride; r.n_layers = n_layers; r.sel_idx = sel_idx; r.row_off = row_off;
  r.batch = batch; r.seq_len = seq_len; r.c = c; r.n_split = kRolloutSplit;
  // same split of the scratch as d2c_op_rollout makes of the caller's buffer
  r.u0 = reinterpret_cast<float*>(sp); r.u1 = reinterpret_cast<float*>(sp + align_up(R * 4, 256));
  r.partial = reinterpret_cast<float*>(sp + 2 * align_up(R * 4, 256));
  return launch_rollout(r, static_cast<cudaStream_t>(cuda_stream));
}
