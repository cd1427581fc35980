// The streaming compress kernel for f32 inputs (see compress_stream.cuh).
#include "compress_stream.cuh"

namespace daf {
DAF_INSTANTIATE_STREAM(float)
}
