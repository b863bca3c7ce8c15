// Decode kernels of one packed format: 2-bit keys, 4-bit values, 4 / 4 bytes per key / value metadata entry.
#include "innerq_decode_mma.cuh"

namespace iq {
IQ_DEFINE_MMA_FORMAT(2, 4, 4, 4)
}  // namespace iq
