// CUDA-core implementation of the GEMM stage  y = x' . W^  (Eq. 3) over the tiled operand.
// Slow and simple: it fixes the numerical contract (fp16 dequantisation (code - zero) * scale
// rounded once, fp32 accumulation, one fp16 rounding of y) and cross-checks the tensor-core
// kernel.  One thread per output column, 8 tokens per CTA.
#include "rosaq_internal.cuh"

namespace rosaq {

constexpr int kSimtTokens = 8;

template <int kBits>
__global__ void __launch_bounds__(kTileN)
linear_simt_kernel(const __half *__restrict__ x, int M, long long ldx, TiledOperand t,
                   const int32_t *__restrict__ col_map, __half *__restrict__ y, long long ldy) {
  __shared__ float xs[kSimtTokens][kGroup];
  const int nt = blockIdx.x, m0 = blockIdx.y * kSimtTokens, nl = threadIdx.x;
  float acc[kSimtTokens];
#pragma unroll
  for (int m = 0; m < kSimtTokens; ++m) acc[m] = 0.0f;

  const int groups = groups_per_tile(t);
  for (int lg = 0; lg < groups; ++lg) {
    const int k0 = group_k0(t, nt, lg);
    __syncthreads();
    for (int e = nl; e < kSimtTokens * kGroup; e += kTileN) {
      int m = e / kGroup, k = e % kGroup;
      xs[m][k] = (m0 + m < M) ? __half2float(x[(long long)(m0 + m) * ldx + k0 + k]) : 0.0f;
    }
    __syncthreads();
    const uint8_t *tile = t.blob + tile_offset(t, nt, lg);
    if (lg < t.g_fp16) {
      for (int k8 = 0; k8 < kGroup; k8 += 8) {
        uint4 v = *reinterpret_cast<const uint4 *>(tile + fp16_tile_byte(k8, nl));
        const __half *h = reinterpret_cast<const __half *>(&v);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          float w = __half2float(h[e]);
#pragma unroll
          for (int m = 0; m < kSimtTokens; ++m) acc[m] = fmaf(xs[m][k8 + e], w, acc[m]);
        }
      }
    } else {
      constexpr int kWords = kBits == 4 ? 16 : 12;
      uint32_t words[kWords];
      __half sh, zh;
      load_quant_tile_column<kBits>(tile, nl, words, &sh, &zh);
#pragma unroll 4
      for (int k = 0; k < kGroup; ++k) {
        __half c = __ushort2half_rn((unsigned short)get_code<kBits>(words, k));
        float w = __half2float(__hmul(__hsub(c, zh), sh));
#pragma unroll
        for (int m = 0; m < kSimtTokens; ++m) acc[m] = fmaf(xs[m][k], w, acc[m]);
      }
    }
  }
  const int n = nt * kTileN + nl;
  if (n >= t.d_out) return;
  const int col = col_map ? col_map[n] : n;
#pragma unroll
  for (int m = 0; m < kSimtTokens; ++m)
    if (m0 + m < M) y[(long long)(m0 + m) * ldy + col] = __float2half_rn(acc[m]);
}

int launch_linear_simt(const rosaq_ctx *, const __half *x, int M, long long ldx, const TiledOperand &t,
                       const int32_t *col_map, __half *y, long long ldy, cudaStream_t s) {
  dim3 grid(t.n_tiles, (M + kSimtTokens - 1) / kSimtTokens);
  if (t.g_quant > 0 && t.bits == 3)
    linear_simt_kernel<3><<<grid, kTileN, 0, s>>>(x, M, ldx, t, col_map, y, ldy);
  else
    linear_simt_kernel<4><<<grid, kTileN, 0, s>>>(x, M, ldx, t, col_map, y, ldy);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

}  // namespace rosaq
