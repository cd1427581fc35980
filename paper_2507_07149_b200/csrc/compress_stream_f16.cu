// The streaming compress kernel for f16 inputs (see compress_stream.cuh).
#include "compress_stream.cuh"

namespace daf {
DAF_INSTANTIATE_STREAM(__half)
}
