// placeholder until the tcgen05 kernels land
#include "common.cuh"
namespace etr {
size_t tc_workspace_bytes(const etr_config*) { return 0; }
bool tc_available() { return false; }
etr_status tc_ffn_forward(const etr_config*, const etr_route*, const void*, const void*, const void*,
                          const void*, void*, void*, void*, void*, etr_stats*, void*, cudaStream_t) {
  return ETR_ERR_UNSUPPORTED;
}
etr_status tc_ffn_backward(const etr_config*, const etr_route*, const void*, const void*, const void*,
                           const void*, const void*, const void*, const void*, const void*, void*,
                           void*, void*, void*, void*, void*, etr_stats*, void*, cudaStream_t) {
  return ETR_ERR_UNSUPPORTED;
}
}  // namespace etr
