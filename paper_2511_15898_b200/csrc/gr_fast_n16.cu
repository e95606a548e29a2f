// Fast solve kernels for series length 16 (draft counts up to 16).
#include "gr_fast.cuh"

namespace gr {
GR_FAST_INSTANTIATE(16)
}  // namespace gr
