#include "lqer_common.cuh"
namespace lqer {
int decode_max_m() { return 0; }
cudaError_t launch_decode(const float*, int, const PackedMeta&, const void*, float*, DeviceStatus*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}
