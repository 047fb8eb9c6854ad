// Instantiations of the tiered flash-decode kernel for one (datatype, head dimension) pair.
#include "decode_attn.cuh"

namespace qevict {
QEVICT_DECODE_DISPATCH(decode_dispatch_h128, __half, 128)
}  // namespace qevict
