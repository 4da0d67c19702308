// Tensor-core path (tcgen05 / TMEM / TMA).  Placeholder until the kernels land: reports "not supported".
#include "layer.h"

namespace dare {
bool tc_supported(const dare_layer_config_t&) { return false; }
size_t tc_maps_bytes() { return 0; }
dare_status_t tc_create(dare_layer*) { return DARE_ERR_UNSUPPORTED; }
void tc_destroy(dare_layer*) {}
dare_status_t step_tc(dare_layer*, const void*, const StepGeom&, int, float, void*, cudaStream_t) {
  return DARE_ERR_UNSUPPORTED;
}
}  // namespace dare
