// The two-pass compress kernels for bf16 inputs (see compress_twopass.cuh).
#include "compress_twopass.cuh"

namespace daf {
DAF_INSTANTIATE_TWOPASS(__nv_bfloat16)
}
