// Fast solve kernels for series length 16 (draft counts up to 16), supports of 65 to 128 tokens.
#define GR_FAST_MP 128
#define GR_FAST_NS fast128
#include "gr_fast.cuh"

namespace gr {
namespace GR_FAST_NS {
GR_FAST_INSTANTIATE(16)
}
}  // namespace gr
