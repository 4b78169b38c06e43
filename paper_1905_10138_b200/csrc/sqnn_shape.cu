// Instantiates the decode and GEMV kernels for one network shape (N_OUT x N_IN given by
// -DSQNN_NO / -DSQNN_NI; 0 x 0 is the run-time-shape fallback).
#include "sqnn_gemv.cuh"

#ifndef SQNN_NO
#error "compile with -DSQNN_NO=<n_out> -DSQNN_NI=<n_in>"
#endif

namespace sqnn {

template <>
int decode_shape<SQNN_NO, SQNN_NI>(const DecodeArgs &A, sqnn_out_mode mode, const uint64_t *d_mask,
                                   const float *d_alpha, uint64_t n, void *d_out, cudaStream_t st)
{
    return launch_decode<SQNN_NO, SQNN_NI>(A, mode, d_mask, d_alpha, n, d_out, st);
}

template <>
int gemv_shape<SQNN_NO, SQNN_NI>(const DecodeArgs &A, const uint64_t *d_mask, const float *d_alpha,
                                 const void *d_x, int x_dtype, int64_t ldx, uint32_t batch, float *d_y,
                                 int64_t ldy, uint64_t m, uint64_t n, cudaStream_t st)
{
    return x_dtype == SQNN_X_BF16
        ? launch_gemv<SQNN_NO, SQNN_NI, __nv_bfloat16>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st)
        : launch_gemv<SQNN_NO, SQNN_NI, float>(A, d_mask, d_alpha, d_x, ldx, batch, d_y, ldy, m, n, st);
}

}  // namespace sqnn
