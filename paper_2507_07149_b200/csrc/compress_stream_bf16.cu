// The streaming compress kernel for bf16 inputs (see compress_stream.cuh).
#include "compress_stream.cuh"

namespace daf {
DAF_INSTANTIATE_STREAM(__nv_bfloat16)
}
