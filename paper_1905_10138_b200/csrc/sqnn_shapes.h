// Network shapes (n_out, n_in) that get kernels specialised at compile time; every other
// shape runs the run-time-shape kernels.  Keep in step with the build script.
#pragma once
#define SQNN_FOR_SHAPES(X) X(40, 12) X(40, 16) X(60, 12) X(80, 8) X(80, 16) X(100, 10) X(200, 10)
