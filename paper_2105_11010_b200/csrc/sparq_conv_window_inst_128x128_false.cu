// Instantiates the window convolution kernel: 128 x 128 output tiles, 128-channel blocks,
// weights resident in shared memory: false.
#include "sparq_conv_window_kernel.cuh"
namespace sparq { SPARQ_DEFINE_WINDOW_SHAPE(128, 128, false) }
