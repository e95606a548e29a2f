// Fast solve kernels for series length 4 (draft counts up to 4), supports up to 64 tokens.
#include "gr_fast.cuh"

namespace gr {
namespace GR_FAST_NS {
GR_FAST_INSTANTIATE(4)
}
}  // namespace gr
