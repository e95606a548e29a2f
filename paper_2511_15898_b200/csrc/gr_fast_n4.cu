// Fast solve kernels for series length 4 (draft counts up to 4).
#include "gr_fast.cuh"

namespace gr {
GR_FAST_INSTANTIATE(4)
}  // namespace gr
