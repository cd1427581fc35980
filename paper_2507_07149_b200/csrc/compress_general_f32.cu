// The general compress kernel for f32 inputs (see compress_general.cuh).
#include "compress_general.cuh"

namespace daf {
DAF_INSTANTIATE_GENERAL(float)
}
