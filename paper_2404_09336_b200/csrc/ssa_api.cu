// Library-wide entry points of libssa: status strings, version, the timing
// hook and the launch counter.
#include <atomic>

#include "ssa_common.cuh"

namespace ssa {

// Multiprocessors of the current device, asked once per device.  Without a usable device (size queries on a
// machine that has none) the count of a full B200 stands in.
int sm_count() {
  constexpr int kDefault = 148, kMaxDevices = 64;
  static std::atomic<int> cached[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return kDefault;
  }
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return kDefault;
  }
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

static thread_local uint64_t t_launches = 0;
static thread_local cudaEvent_t t_ev_begin = nullptr;
static thread_local cudaEvent_t t_ev_end = nullptr;

void note_launches(int n) { t_launches += (uint64_t)n; }

void take_kernel_events(cudaEvent_t* begin, cudaEvent_t* end) {
  *begin = t_ev_begin;
  *end = t_ev_end;
  t_ev_begin = nullptr;
  t_ev_end = nullptr;
}

}  // namespace ssa

extern "C" {

void ssa_set_kernel_events(void* ev_begin, void* ev_end) {
  ssa::t_ev_begin = (cudaEvent_t)ev_begin;
  ssa::t_ev_end = (cudaEvent_t)ev_end;
}

uint64_t ssa_launch_count(void) { return ssa::t_launches; }

const char* ssa_status_string(int32_t status) {
  switch (status) {
    case SSA_OK: return "ok";
    case SSA_ERR_NULL: return "a required pointer is NULL";
    case SSA_ERR_SHAPE: return "a size is non-positive or out of range";
    case SSA_ERR_DTYPE: return "unsupported dtype";
    case SSA_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case SSA_ERR_CAPACITY: return "index_stride / max_selected inconsistent";
    case SSA_ERR_WORKSPACE: return "workspace missing or too small";
    case SSA_ERR_CUDA: return "CUDA runtime call failed";
    case SSA_ERR_UNSUPPORTED: return "request outside the implemented set";
    default: return "unknown status";
  }
}

int32_t ssa_version(void) { return 101; }

}  // extern "C"
