// Decode kernels of one packed format: 2-bit keys, 3-bit values, 4 / 2 bytes per key / value metadata entry.
#include "innerq_decode_mma.cuh"

namespace iq {
IQ_DEFINE_MMA_FORMAT(2, 3, 4, 2)
}  // namespace iq
