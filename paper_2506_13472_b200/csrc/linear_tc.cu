// Tensor-core implementation of the GEMM stage (placeholder dispatch while the tcgen05 kernel is brought up).
#include "rosaq_internal.cuh"

namespace rosaq {

int launch_linear_tc(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t,
                     const int32_t *col_map, __half *y, long long ldy, cudaStream_t s) {
  return launch_linear_simt(ctx, x, M, ldx, t, col_map, y, ldy, s);
}

}  // namespace rosaq
