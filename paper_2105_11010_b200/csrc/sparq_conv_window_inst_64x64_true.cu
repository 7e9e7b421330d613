// Instantiates the window convolution kernel: 128 x 64 output tiles, 64-channel blocks,
// weights resident in shared memory: true.
#include "sparq_conv_window_kernel.cuh"
namespace sparq { SPARQ_DEFINE_WINDOW_SHAPE(64, 64, true) }
