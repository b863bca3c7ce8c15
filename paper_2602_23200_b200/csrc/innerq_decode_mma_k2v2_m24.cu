// Decode kernels of one packed format: 2-bit keys, 2-bit values (byte order, integer MMA), 2 / 4 bytes per key /
// value metadata entry.
#define IQ_WITH_TIMING_INSTANCES      // also the instances without key-side / value-side work (decode options 6 / 7)
#include "innerq_decode_i8.cuh"

namespace iq {
IQ_DEFINE_I8_FORMAT(2, 2, 2, 4)
}  // namespace iq
