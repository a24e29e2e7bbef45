// The layer for callers that cannot allocate device memory.
//
// lqer_linear_stream needs a scratch `workspace` from the caller (the quantised activations
// [X_q | T_q] and a status area).  Some callers have no way to provide one: code that runs
// inside somebody else's memory plan (a plugin of an inference runtime that owns every byte of
// the device and hands out no allocator), code on a path where cudaMalloc's implicit device
// synchronisation is not acceptable, or a process whose device-memory budget was fixed before
// the library was loaded.  For them the scratch lives in a fixed array inside the library
// image.  Every GPU that loads the library holds LQER_STATIC_SCRATCH_BYTES for it until the
// process exits, whether or not this entry point is ever called.
#include <mutex>
#include <unordered_map>

#include "lqer_common.cuh"

namespace lqer {

static __device__ __align__(256) unsigned char g_static_scratch[LQER_STATIC_SCRATCH_BYTES];

// In host code the name g_static_scratch is only a handle for the runtime, not a device
// address: the address is asked for once per device, with that device current.
static std::mutex g_static_mu;
static std::unordered_map<int, void*> g_static_ptr;

static lqer_status_t static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LQER_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mu);
  auto it = g_static_ptr.find(dev);
  if (it == g_static_ptr.end()) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return LQER_ERR_CUDA;
    it = g_static_ptr.emplace(dev, p).first;
  }
  *out = it->second;
  return LQER_OK;
}

}  // namespace lqer

extern "C" lqer_status_t lqer_linear_static(const float* X, int M, const void* packed, float* Y, void* stream) {
  if (X == nullptr || packed == nullptr || Y == nullptr) return LQER_ERR_NULL;
  // what this call needs on the path it takes (decode kernels, or prologue + GEMM with its split-K partial sums):
  // less than lqer_workspace_bytes(M, ...), which covers every batch up to M
  size_t need = 0;
  lqer_status_t st = lqer::call_workspace_bytes(packed, M, &need);
  if (st != LQER_OK) return st;
  if (need > (size_t)LQER_STATIC_SCRATCH_BYTES) return LQER_ERR_STATIC_SCRATCH;   // the fixed array is too small for this shape
  void* scratch = nullptr;
  if ((st = lqer::static_scratch(&scratch)) != LQER_OK) return st;
  // The array keeps whatever the previous call left: the head of the workspace (status area,
  // arrival counters, accumulator) must start at zero.
  if ((st = lqer_workspace_init(scratch, need, stream)) != LQER_OK) return st;
  return lqer_linear_stream(X, M, packed, Y, scratch, need, stream);
}
