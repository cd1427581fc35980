// The general compress kernel for f16 inputs (see compress_general.cuh).
#include "compress_general.cuh"

namespace daf {
DAF_INSTANTIATE_GENERAL(__half)
}
