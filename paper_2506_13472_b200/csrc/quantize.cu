// Offline side of the path: W' = R^T W (Eq. 1), the mixed-precision split of W'
// (Eq. 3, Section 3.3), and the conversions between the tiled layout the GEMM kernels
// read and the plain interchange layout.
//
// Everything that decides an integer code is written with explicit round-to-nearest
// intrinsics (__fmaf_rn, __fdiv_rn, ...) so that the compiler can neither contract nor
// reorder it: the codes must be reproducible bit for bit by a sequential IEEE fp32
// implementation.
#include "rosaq_internal.cuh"

namespace rosaq {

// =====================================================================================
// out[i][n] (+)= sum_k A[k][i] * B[k][n]   -- one fused multiply-add per term, k ascending,
// a single fp32 accumulator per output started at +0 (the canonical chain of W' = R^T W;
// also used, with A = B = X, for the Gram matrix of fp32 calibration activations).
// 128 x 128 output tile per CTA, 256 threads, 8 x 8 outputs per thread, K stepped by 16
// through shared memory.  Zero padding outside [I) x [N) x [K) is harmless: fma(0, 0, acc)
// returns acc.
// =====================================================================================
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }

constexpr int kBM = 128, kBN = 128, kBK = 16;

template <typename TA, typename TB, bool kAccumulate>
__global__ void __launch_bounds__(256)
gemm_tn_fma_kernel(const TA *__restrict__ A, long long lda, long long strideA,
                   const TB *__restrict__ B, long long ldb, long long strideB,
                   float *__restrict__ out, long long ldo, long long strideO,
                   int I, int N, long long K) {
  __shared__ __align__(16) float As[kBK][kBM];
  __shared__ __align__(16) float Bs[kBK][kBN];
  A += blockIdx.z * strideA;
  B += blockIdx.z * strideB;
  out += blockIdx.z * strideO;
  const int i0 = blockIdx.y * kBM, n0 = blockIdx.x * kBN;
  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  // loader mapping: 16 rows x 128 columns, 8 consecutive columns per thread
  const int lr = tid >> 4, lc = (tid & 15) * 8;

  float acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;

  float ra[8], rb[8];
  auto fetch = [&](long long k0) {
    long long k = k0 + lr;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      int i = i0 + lc + e, n = n0 + lc + e;
      ra[e] = (k < K && i < I) ? to_f32<TA>(A[k * lda + i]) : 0.0f;
      rb[e] = (k < K && n < N) ? to_f32<TB>(B[k * ldb + n]) : 0.0f;
    }
  };
  fetch(0);
  for (long long k0 = 0; k0 < K; k0 += kBK) {
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      As[lr][lc + e] = ra[e];
      Bs[lr][lc + e] = rb[e];
    }
    __syncthreads();
    if (k0 + kBK < K) fetch(k0 + kBK);
#pragma unroll
    for (int kk = 0; kk < kBK; ++kk) {
      float a[8], b[8];
      *reinterpret_cast<float4 *>(&a[0]) = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
      *reinterpret_cast<float4 *>(&a[4]) = *reinterpret_cast<const float4 *>(&As[kk][64 + ty * 4]);
      *reinterpret_cast<float4 *>(&b[0]) = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
      *reinterpret_cast<float4 *>(&b[4]) = *reinterpret_cast<const float4 *>(&Bs[kk][64 + tx * 4]);
#pragma unroll
      for (int ia = 0; ia < 8; ++ia)
#pragma unroll
        for (int ib = 0; ib < 8; ++ib) acc[ia][ib] = __fmaf_rn(a[ia], b[ib], acc[ia][ib]);
    }
  }
#pragma unroll
  for (int ia = 0; ia < 8; ++ia) {
    int i = i0 + (ia < 4 ? ty * 4 + ia : 64 + ty * 4 + ia - 4);
    if (i >= I) continue;
#pragma unroll
    for (int ib = 0; ib < 8; ++ib) {
      int n = n0 + (ib < 4 ? tx * 4 + ib : 64 + tx * 4 + ib - 4);
      if (n >= N) continue;
      float *o = out + (long long)i * ldo + n;
      *o = kAccumulate ? __fadd_rn(*o, acc[ia][ib]) : acc[ia][ib];
    }
  }
}

// Block-diagonal (head-wise, Eq. 6) and/or permuted rotation: output row j takes column
// perm[j] of blockdiag(Rb); the chain runs over the dh rows of that column's block only.
// One CTA per output row, threads along the output columns.
template <typename TQ, typename TW>
__global__ void __launch_bounds__(256)
rotate_weights_blockdiag_kernel(const TQ *__restrict__ Rb, int d_in, int dh, const int32_t *__restrict__ perm,
                                const TW *__restrict__ W, int d_out, float *__restrict__ Wp) {
  extern __shared__ float rcol[];  // [dh]
  const int j = blockIdx.x;
  const int p = perm ? perm[j] : j;
  const int h = p / dh, c = p % dh;
  const TQ *R = Rb + (long long)h * dh * dh;
  for (int k = threadIdx.x; k < dh; k += blockDim.x) rcol[k] = to_f32<TQ>(R[(long long)k * dh + c]);
  __syncthreads();
  const TW *Wb = W + (long long)h * dh * d_out;
  for (int n = blockIdx.y * blockDim.x + threadIdx.x; n < d_out; n += gridDim.y * blockDim.x) {
    float acc = 0.0f;
    for (int k = 0; k < dh; ++k) acc = __fmaf_rn(rcol[k], to_f32<TW>(Wb[(long long)k * d_out + n]), acc);
    Wp[(long long)j * d_out + n] = acc;
  }
}

__global__ void cast_weights_kernel(const __half *__restrict__ W, long long n, float *__restrict__ Wp) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  long long stride = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += stride) Wp[i] = __half2float(W[i]);
}

// D W of the scaled (AWQ-style) variant: out[i][n] = d[i] * W[i][n], one fp32 rounding per product
__global__ void scale_rows_kernel(const __half *__restrict__ W, const float *__restrict__ d, int d_out, long long n,
                                  float *__restrict__ out) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  long long stride = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += stride) out[i] = __fmul_rn(d[i / d_out], __half2float(W[i]));
}

template <typename TW>
static int rotate_weights_typed(const void *q, int q_is_f32, int d_in, int n_blocks, const int32_t *perm, const TW *W,
                                int d_out, float *Wp, cudaStream_t s) {
  if (n_blocks == 1 && perm == nullptr && q_is_f32) {
    dim3 grid((d_out + kBN - 1) / kBN, (d_in + kBM - 1) / kBM, 1);
    gemm_tn_fma_kernel<float, TW, false><<<grid, 256, 0, s>>>(
        static_cast<const float *>(q), d_in, 0, W, d_out, 0, Wp, d_out, 0, d_in, d_out, d_in);
  } else {
    int dh = d_in / n_blocks;
    size_t smem = sizeof(float) * dh;
    if (smem > 48 * 1024) {
      cudaError_t e;
      if (q_is_f32)
        e = cudaFuncSetAttribute(rotate_weights_blockdiag_kernel<float, TW>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      else
        e = cudaFuncSetAttribute(rotate_weights_blockdiag_kernel<__half, TW>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
    }
    dim3 grid(d_in, min((d_out + 255) / 256, 8));
    if (q_is_f32)
      rotate_weights_blockdiag_kernel<float, TW><<<grid, 256, smem, s>>>(static_cast<const float *>(q), d_in, dh,
                                                                           perm, W, d_out, Wp);
    else
      rotate_weights_blockdiag_kernel<__half, TW><<<grid, 256, smem, s>>>(static_cast<const __half *>(q), d_in, dh,
                                                                            perm, W, d_out, Wp);
  }
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

int launch_rotate_weights(const void *q, int q_is_f32, int d_in, int n_blocks, const int32_t *perm,
                          const __half *W, int d_out, float *Wp, cudaStream_t s) {
  return rotate_weights_typed<__half>(q, q_is_f32, d_in, n_blocks, perm, W, d_out, Wp, s);
}

// the same chain on a weight that is already fp32 (the scaled weight D W)
int launch_rotate_weights_w32(const void *q, int q_is_f32, int d_in, int n_blocks, const int32_t *perm,
                              const float *W32, int d_out, float *Wp, cudaStream_t s) {
  return rotate_weights_typed<float>(q, q_is_f32, d_in, n_blocks, perm, W32, d_out, Wp, s);
}

int launch_scale_rows(const __half *W, const float *in_scale, int d_in, int d_out, float *out, cudaStream_t s) {
  long long n = (long long)d_in * d_out;
  long long want = (n + 255) / 256;
  int blocks = (int)(want < 148 * 16 ? want : 148 * 16);
  scale_rows_kernel<<<blocks, 256, 0, s>>>(W, in_scale, d_out, n, out);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

int launch_cast_weights(const __half *W, int d_in, int d_out, float *Wp, cudaStream_t s) {
  long long n = (long long)d_in * d_out;
  long long want = (n + 255) / 256;
  int blocks = (int)(want < 148 * 16 ? want : 148 * 16);
  cast_weights_kernel<<<blocks, 256, 0, s>>>(W, n, Wp);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

// Gram matrix on CUDA cores (fp32 products, fp32 accumulate): exact-product path for fp32
// calibration activations and the fallback for shapes the tensor-core kernel does not take.
int launch_cov_fma(const void *X, int x_dtype, long long n_tokens, int d, long long ldx, int n_blocks, float *C,
                   cudaStream_t s) {
  int dh = d / n_blocks;
  dim3 grid((dh + kBN - 1) / kBN, (dh + kBM - 1) / kBM, n_blocks);
  if (x_dtype == ROSAQ_F32) {
    const float *x = static_cast<const float *>(X);
    gemm_tn_fma_kernel<float, float, true><<<grid, 256, 0, s>>>(x, ldx, dh, x, ldx, dh, C, dh, (long long)dh * dh,
                                                                 dh, dh, n_tokens);
  } else {
    const __half *x = static_cast<const __half *>(X);
    gemm_tn_fma_kernel<__half, __half, true><<<grid, 256, 0, s>>>(x, ldx, dh, x, ldx, dh, C, dh,
                                                                   (long long)dh * dh, dh, dh, n_tokens);
  }
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

// =====================================================================================
// Eq. 3 / Section 3.3: salient rows -> fp16; other groups -> asymmetric min/max RTN codes,
// written straight into the tiled layout.  One thread per (group, output column).
// =====================================================================================
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}

template <int kBits>
__global__ void __launch_bounds__(kTileN)
quant_pack_kernel(const float *__restrict__ Wp, TiledOperand t) {
  const int nt = blockIdx.x, g = blockIdx.y, nl = threadIdx.x;
  const int n = nt * kTileN + nl;
  const bool live = n < t.d_out;
  uint8_t *tile = t.blob + tile_offset(t, nt, g);
  const float *col = Wp + (long long)g * kGroup * t.d_out + n;
  if (g < t.g_fp16) {
    for (int k8 = 0; k8 < kGroup; k8 += 8) {
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = live ? col[(long long)(k8 + e) * t.d_out] : 0.0f;
      *reinterpret_cast<uint4 *>(tile + fp16_tile_byte(k8, nl)) =
          make_uint4(pack_half2(v[0], v[1]), pack_half2(v[2], v[3]), pack_half2(v[4], v[5]), pack_half2(v[6], v[7]));
    }
    return;
  }
  constexpr int kWords = kBits == 4 ? 16 : 12;
  uint32_t words[kWords];
#pragma unroll
  for (int w = 0; w < kWords; ++w) words[w] = 0;
  __half sh = __ushort_as_half(0), zh = __ushort_as_half(0);
  if (live) {
    const float qmax = (float)((1 << kBits) - 1);
    float lo = col[0], hi = col[0];
    for (int k = 1; k < kGroup; ++k) {
      float w = col[(long long)k * t.d_out];
      lo = w < lo ? w : lo;
      hi = w > hi ? w : hi;
    }
    float range = __fsub_rn(hi, lo);
    if (range < 1e-5f) range = 1e-5f;
    unsigned short sb = __half_as_ushort(__float2half_rn(__fdiv_rn(range, qmax)));
    if (sb == 0x0000) sb = 0x0001;
    if (sb == 0x7c00) sb = 0x7bff;
    sh = __ushort_as_half(sb);
    const float sf = __half2float(sh);
    float z = -rintf(__fdiv_rn(lo, sf));
    if (z <= 0.0f) z = 0.0f;
    if (z > qmax) z = qmax;
    zh = __float2half_rn(z);
#pragma unroll 8
    for (int k = 0; k < kGroup; ++k) {
      float q = __fadd_rn(rintf(__fdiv_rn(col[(long long)k * t.d_out], sf)), z);
      if (q < 0.0f) q = 0.0f;
      if (q > qmax) q = qmax;
      put_code<kBits>(words, k, (uint32_t)q);
    }
  }
  store_quant_tile_column<kBits>(tile, nl, words, sh, zh);
}

int launch_quant_pack(const float *Wp, const TiledOperand &t, cudaStream_t s) {
  dim3 grid(t.n_tiles, groups_per_tile(t));
  if (t.bits == 3)
    quant_pack_kernel<3><<<grid, kTileN, 0, s>>>(Wp, t);
  else
    quant_pack_kernel<4><<<grid, kTileN, 0, s>>>(Wp, t);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

// =====================================================================================
// tiled <-> interchange layout
// =====================================================================================
template <int kBits>
__global__ void __launch_bounds__(kTileN)
export_kernel(TiledOperand t, uint32_t *__restrict__ qw, __half *__restrict__ scales, __half *__restrict__ zeros,
              __half *__restrict__ salient) {
  const int nt = blockIdx.x, g = blockIdx.y, nl = threadIdx.x;
  const int n = nt * kTileN + nl;
  if (n >= t.d_out) return;
  const uint8_t *tile = t.blob + tile_offset(t, nt, g);
  if (g < t.g_fp16) {
    if (!salient) return;
    for (int k = 0; k < kGroup; ++k)
      salient[(long long)(g * kGroup + k) * t.d_out + n] =
          *reinterpret_cast<const __half *>(tile + fp16_tile_byte(k, nl));
    return;
  }
  constexpr int kWords = kBits == 4 ? 16 : 12;
  uint32_t words[kWords];
  __half sh, zh;
  load_quant_tile_column<kBits>(tile, nl, words, &sh, &zh);
  const int gq = g - t.g_fp16;
  if (scales) scales[(long long)gq * t.d_out + n] = sh;
  if (zeros) zeros[(long long)gq * t.d_out + n] = zh;
  if (!qw) return;
  if (kBits == 4) {
    for (int w = 0; w < 16; ++w) {
      uint32_t v = 0;
      for (int i = 0; i < 8; ++i) v |= get_code<4>(words, w * 8 + i) << (4 * i);
      qw[(long long)(gq * 16 + w) * t.d_out + n] = v;
    }
  } else {
    for (int blk = 0; blk < 4; ++blk) {
      uint32_t v[3] = {0, 0, 0};
      for (int i = 0; i < 32; ++i) {
        uint32_t c = get_code<3>(words, blk * 32 + i);
        for (int b = 0; b < 3; ++b) {
          int bit = 3 * i + b;
          v[bit >> 5] |= ((c >> b) & 1u) << (bit & 31);
        }
      }
      for (int w = 0; w < 3; ++w) qw[(long long)(gq * 12 + blk * 3 + w) * t.d_out + n] = v[w];
    }
  }
}

template <int kBits>
__global__ void __launch_bounds__(kTileN)
import_kernel(TiledOperand t, const uint32_t *__restrict__ qw, const __half *__restrict__ scales,
              const __half *__restrict__ zeros, const __half *__restrict__ salient) {
  const int nt = blockIdx.x, g = blockIdx.y, nl = threadIdx.x;
  const int n = nt * kTileN + nl;
  const bool live = n < t.d_out;
  uint8_t *tile = t.blob + tile_offset(t, nt, g);
  if (g < t.g_fp16) {
    for (int k = 0; k < kGroup; ++k)
      *reinterpret_cast<__half *>(tile + fp16_tile_byte(k, nl)) =
          live ? salient[(long long)(g * kGroup + k) * t.d_out + n] : __ushort_as_half(0);
    return;
  }
  constexpr int kWords = kBits == 4 ? 16 : 12;
  uint32_t words[kWords];
  for (int w = 0; w < kWords; ++w) words[w] = 0;
  __half sh = __ushort_as_half(0), zh = __ushort_as_half(0);
  if (live) {
    const int gq = g - t.g_fp16;
    sh = scales[(long long)gq * t.d_out + n];
    zh = zeros[(long long)gq * t.d_out + n];
    if (kBits == 4) {
      for (int w = 0; w < 16; ++w) {
        uint32_t v = qw[(long long)(gq * 16 + w) * t.d_out + n];
        for (int i = 0; i < 8; ++i) put_code<4>(words, w * 8 + i, (v >> (4 * i)) & 0xf);
      }
    } else {
      for (int blk = 0; blk < 4; ++blk) {
        uint32_t v[3];
        for (int w = 0; w < 3; ++w) v[w] = qw[(long long)(gq * 12 + blk * 3 + w) * t.d_out + n];
        for (int i = 0; i < 32; ++i) {
          uint32_t c = 0;
          for (int b = 0; b < 3; ++b) {
            int bit = 3 * i + b;
            c |= ((v[bit >> 5] >> (bit & 31)) & 1u) << b;
          }
          put_code<3>(words, blk * 32 + i, c);
        }
      }
    }
  }
  store_quant_tile_column<kBits>(tile, nl, words, sh, zh);
}

int launch_export(const TiledOperand &t, uint32_t *qw, __half *scales, __half *zeros, __half *salient,
                  cudaStream_t s) {
  dim3 grid(t.n_tiles, groups_per_tile(t));
  if (grid.y == 0) return ROSAQ_OK;
  if (t.bits == 3)
    export_kernel<3><<<grid, kTileN, 0, s>>>(t, qw, scales, zeros, salient);
  else
    export_kernel<4><<<grid, kTileN, 0, s>>>(t, qw, scales, zeros, salient);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

int launch_import(const TiledOperand &t, const uint32_t *qw, const __half *scales, const __half *zeros,
                  const __half *salient, cudaStream_t s) {
  dim3 grid(t.n_tiles, groups_per_tile(t));
  if (grid.y == 0) return ROSAQ_OK;
  if (t.bits == 3)
    import_kernel<3><<<grid, kTileN, 0, s>>>(t, qw, scales, zeros, salient);
  else
    import_kernel<4><<<grid, kTileN, 0, s>>>(t, qw, scales, zeros, salient);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

// =====================================================================================
// Online rotation operand: R (fp16, block-diagonal) re-tiled as fp16 tiles.  The "weight"
// of the rotation GEMM x . R is R itself: input channel k = row of the block, output
// column = column of the block-diagonal matrix (the permutation is applied when the
// result is stored).
// =====================================================================================
__global__ void __launch_bounds__(kTileN)
rotation_tiles_kernel(const __half *__restrict__ q, int dh, TiledOperand t) {
  // A column tile holds the groups of its (possibly merged) diagonal block: dm channels = block_groups * 128,
  // or all of d_in.  When two 128 x 128 head blocks are merged into one 256 x 256 block the off-diagonal
  // quarters are zero.
  const int nt = blockIdx.x, lg = blockIdx.y, nl = threadIdx.x;
  const int col = nt * kTileN + nl;          // column of blockdiag
  const int h = col / dh, c = col % dh;
  const int dm = t.block_groups > 0 ? t.block_groups * kGroup : t.d_in;
  const int k_base = (col / dm) * dm + lg * kGroup;             // first input channel of this group
  const __half *R = q + (long long)h * dh * dh;
  uint8_t *tile = t.blob + tile_offset(t, nt, lg);
  for (int k = 0; k < kGroup; ++k) {
    const int kg = k_base + k;
    *reinterpret_cast<__half *>(tile + fp16_tile_byte(k, nl)) = kg / dh == h ? R[(long long)(kg % dh) * dh + c] : __float2half(0.f);
  }
}

int launch_rotation_tiles(const __half *q, int d, int n_blocks, const TiledOperand &t, cudaStream_t s) {
  dim3 grid(t.n_tiles, groups_per_tile(t));
  rotation_tiles_kernel<<<grid, kTileN, 0, s>>>(q, d / n_blocks, t);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

__global__ void invert_perm_kernel(const int32_t *__restrict__ perm, int d, int32_t *__restrict__ inv) {
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < d) {
    int p = perm[j];
    if (p >= 0 && p < d) inv[p] = j;
  }
}

// bad[0] = 1 when perm is not a permutation of 0..d-1: an entry out of range, or (inv still -1 somewhere
// after the scatter above) a value that never occurs, i.e. another one occurs twice
__global__ void check_perm_kernel(const int32_t *__restrict__ perm, const int32_t *__restrict__ inv, int d,
                                  int *__restrict__ bad) {
  int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < d && (perm[j] < 0 || perm[j] >= d || inv[j] < 0)) atomicExch(bad, 1);
}

// inv[perm[j]] = j.  Synchronizes the stream; ROSAQ_ERR_INVALID_ARG when perm is not a permutation (nothing
// that indexes with it has been launched then).  `bad` is a device word owned by the caller.
int launch_invert_perm(const int32_t *perm, int d, int32_t *inv, int *bad, cudaStream_t s) {
  if (cudaMemsetAsync(inv, 0xff, sizeof(int32_t) * (size_t)d, s) != cudaSuccess ||
      cudaMemsetAsync(bad, 0, sizeof(int), s) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  invert_perm_kernel<<<(d + 255) / 256, 256, 0, s>>>(perm, d, inv);
  check_perm_kernel<<<(d + 255) / 256, 256, 0, s>>>(perm, inv, d, bad);
  int host = 0;
  if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(&host, bad, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return host ? ROSAQ_ERR_INVALID_ARG : ROSAQ_OK;
}

}  // namespace rosaq
