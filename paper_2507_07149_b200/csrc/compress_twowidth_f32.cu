// The two-width streaming compress kernel for f32 inputs (see compress_twowidth.cuh).
#include "compress_twowidth.cuh"

namespace daf {
DAF_INSTANTIATE_TWO_WIDTH(float)
}
