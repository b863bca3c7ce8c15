// Decode kernels of one packed format: 4-bit keys, 4-bit values, 2 / 4 bytes per key / value metadata entry.
#include "innerq_decode_mma.cuh"

namespace iq {
IQ_DEFINE_MMA_FORMAT(4, 4, 2, 4)
}  // namespace iq
