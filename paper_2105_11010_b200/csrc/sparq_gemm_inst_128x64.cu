// Instantiates the fused kernel for output tiles of 128 x 128 with 64-byte reduction steps.
#include "sparq_gemm_kernel.cuh"
namespace sparq { SPARQ_DEFINE_GEMM_SHAPE(128, 64) }
