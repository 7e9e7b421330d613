// placeholder until the fused kernel lands
#include "sparq_common.cuh"
namespace sparq { void release_gemm_state() {} }
using namespace sparq;
extern "C" int sparq_gemm_s8(const uint8_t *, int64_t, const int8_t *, int64_t, int64_t, int64_t, int64_t,
                             const sparq_params *, const sparq_epilogue *, void *)
{ return set_error(SPARQ_ERR_UNSUPPORTED, "not built yet"); }
extern "C" int sparq_conv2d_nhwc_s8(const uint8_t *, int, int, int, int, const int8_t *, int, int, int,
                                    int, int, int, int, const sparq_params *, const sparq_epilogue *, void *)
{ return set_error(SPARQ_ERR_UNSUPPORTED, "not built yet"); }
