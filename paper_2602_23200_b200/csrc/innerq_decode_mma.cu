// Warp-MMA decode kernel for the INNER layout (placeholder until the kernel lands).
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {
bool decode_mma_supported(const Layout&) { return false; }
int launch_decode_mma(const Layout&, const unsigned char*, unsigned char*, int, const __half*, __half*, int,
                      cudaStream_t) {
  return -2;
}
}  // namespace iq
