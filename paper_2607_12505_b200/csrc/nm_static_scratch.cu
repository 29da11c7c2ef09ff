// nm_spmm_static_scratch: the split-K GEMM for callers that cannot allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at the point where they run a layer: an
// inference server whose memory pool was carved up at start-up and is full, a real-time loop
// where an allocation would stall every stream of the device, a plug-in running inside
// another framework's arena.  nm_spmm already leaves allocation to the caller, but a split-K
// plan needs scratch for the partial sums, and these callers have nowhere to take it from.
// Here the scratch is a fixed array that ships with the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "nm_internal.h"

namespace {

// Partial-sum slices of one split-K call.  Lives in every CUDA context that loads this
// library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[NM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};     // device address of g_static_scratch, per device ordinal

// The array's name is only a host-side handle; kernels need its device address, which differs
// per device.  Looked up once per device, with that device current.
nm_status scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return NM_ERR_CUDA;
    }
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return NM_OK;
}

}  // namespace

extern "C" nm_status nm_spmm_static_scratch(const void* X_dev, int64_t ldx, int T, const nm_weight* w,
                                            const nm_plan* plan, void* Y_dev, int64_t ldy, nm_out_dtype od,
                                            uint32_t* status_dev, void* stream) {
  if (!w || w->magic != nm::kWeightMagic) return NM_ERR_INVALID_ARG;
  // An explicit plan is taken at its word: if it needs more than the fixed array it is refused,
  // not shrunk.  Without a plan nm_spmm plans against the size it is handed and degrades by itself
  // (no split-K, on-chip decode instead of the dense scratch copy, the CUDA-core path for operands
  // that TMA cannot address), exactly as it does for a caller-provided workspace.
  if (plan && plan->workspace_bytes > (uint64_t)NM_STATIC_SCRATCH_BYTES) return NM_ERR_WORKSPACE;
  void* scratch = nullptr;
  nm_status st = scratch_address(&scratch);
  if (st != NM_OK) return st;
  // Nothing in the scratch has to start at zero: every slice element that the merge pass
  // reads is written by this call's GEMM kernel first.
  return nm_spmm(X_dev, ldx, T, w, plan, Y_dev, ldy, od, scratch, (size_t)NM_STATIC_SCRATCH_BYTES, status_dev, stream);
}
