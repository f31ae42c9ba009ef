// Decoded-weight path on the tensor cores (placeholder until the tcgen05 kernel lands).
#include "snn_internal.h"

namespace snn {

bool tc_supported(const Geom&, int) { return false; }
size_t tc_weight_bytes(const Geom&, int, int* Kpad, int* Cpad) {
  *Kpad = 0;
  *Cpad = 0;
  return 0;
}
cudaError_t tc_forward(const LayerDev&, const Geom&, int, const Launch&, int*, int*) {
  return cudaErrorNotSupported;
}

}  // namespace snn
