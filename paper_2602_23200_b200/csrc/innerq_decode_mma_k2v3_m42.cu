// Decode kernels of one packed format: 2-bit keys, 3-bit values (byte order, integer MMA), 4 / 2 bytes per key /
// value metadata entry.
#include "innerq_decode_i8.cuh"

namespace iq {
IQ_DEFINE_I8_FORMAT(2, 3, 4, 2)
}  // namespace iq
