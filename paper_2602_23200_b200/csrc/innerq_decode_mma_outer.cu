// Decode kernels of the outer-grouped comparison cache (keys per channel along tokens, values per token along
// channels, asymmetric): 2-bit and 4-bit codes.
#define IQ_WITH_TIMING_INSTANCES      // also the instances without key-side / value-side work (decode options 6 / 7)
#include "innerq_decode_mma.cuh"

namespace iq {
IQ_DEFINE_MMA_OUTER_FORMAT(2, 2)
IQ_DEFINE_MMA_OUTER_FORMAT(4, 4)
}  // namespace iq
