// Fast solve kernels for series length 8 (draft counts up to 8), supports up to 64 tokens.
#include "gr_fast.cuh"

namespace gr {
namespace GR_FAST_NS {
GR_FAST_INSTANTIATE(8)
}
}  // namespace gr
