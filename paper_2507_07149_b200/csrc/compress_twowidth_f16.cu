// The two-width streaming compress kernel for f16 inputs (see compress_twowidth.cuh).
#include "compress_twowidth.cuh"

namespace daf {
DAF_INSTANTIATE_TWO_WIDTH(__half)
}
