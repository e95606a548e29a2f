// Fast solve kernels for series length 16 (draft counts up to 16), supports up to 64 tokens.
#include "gr_fast.cuh"

namespace gr {
namespace GR_FAST_NS {
GR_FAST_INSTANTIATE(16)
}
}  // namespace gr
