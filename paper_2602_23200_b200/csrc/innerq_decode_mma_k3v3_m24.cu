// Decode kernels of one packed format: 3-bit keys, 3-bit values, 2 / 4 bytes per key / value metadata entry.
#include "innerq_decode_mma.cuh"

namespace iq {
IQ_DEFINE_MMA_FORMAT(3, 3, 2, 4)
}  // namespace iq
