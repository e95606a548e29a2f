// Fast solve kernels for series length 8 (draft counts up to 8).
#include "gr_fast.cuh"

namespace gr {
GR_FAST_INSTANTIATE(8)
}  // namespace gr
