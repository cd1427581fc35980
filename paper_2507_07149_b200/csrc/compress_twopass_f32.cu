// The two-pass compress kernels for f32 inputs (see compress_twopass.cuh).
#include "compress_twopass.cuh"

namespace daf {
DAF_INSTANTIATE_TWOPASS(float)
}
