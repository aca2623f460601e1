// Eq. 4, left-hand side: the calibration Gram matrix C += X^T X.
#include "rosaq_internal.cuh"

namespace rosaq {

int launch_cov(const void *X, int x_dtype, long long n_tokens, int d, long long ldx, int n_blocks, float *C,
               cudaStream_t s) {
  return launch_cov_fma(X, x_dtype, n_tokens, d, ldx, n_blocks, C, s);
}

}  // namespace rosaq
