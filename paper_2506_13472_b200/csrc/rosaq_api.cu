// extern "C" entry points of librosaq: argument checks, handle management, dispatch.
#include <new>

#include "rosaq_internal.cuh"

using namespace rosaq;

namespace {

int cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return ROSAQ_OK;
  (void)cudaGetLastError();
  return e == cudaErrorMemoryAllocation ? ROSAQ_ERR_ALLOC : ROSAQ_ERR_CUDA;
}

// Fills the geometry of a tiled operand; no allocation.
TiledOperand make_geometry(int d_in, int d_out, int bits, int g_fp16, int g_quant, int block_groups) {
  TiledOperand t{};
  t.d_in = d_in;
  t.d_out = d_out;
  t.n_tiles = (d_out + kTileN - 1) / kTileN;
  t.bits = bits;
  t.g_fp16 = g_fp16;
  t.g_quant = g_quant;
  t.block_groups = block_groups;
  t.tile_stride = (long long)g_fp16 * kFp16TileBytes + (long long)g_quant * quant_tile_bytes(bits);
  t.bytes = t.tile_stride * t.n_tiles;
  return t;
}

int alloc_blob(TiledOperand *t) {
  void *p = nullptr;
  size_t bytes = t->bytes > 0 ? (size_t)t->bytes : 16;
  int st = cuda_status(cudaMalloc(&p, bytes));
  if (st != ROSAQ_OK) return st;
  t->blob = static_cast<uint8_t *>(p);
  return ROSAQ_OK;
}

int check_quant_args(int d_in, int d_out, int bits, int group, int k_salient) {
  if (d_in <= 0 || d_out <= 0) return ROSAQ_ERR_INVALID_ARG;
  if (bits != 3 && bits != 4) return ROSAQ_ERR_INVALID_ARG;
  if (group != kGroup) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  if (d_in % kGroup != 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  if (k_salient < 0 || k_salient > d_in || k_salient % kGroup != 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  return ROSAQ_OK;
}

int ensure_workspace(rosaq_ctx *ctx, size_t bytes, cudaStream_t s) {
  if (ctx->ws_bytes >= bytes) return ROSAQ_OK;
  // the old buffer may still be in use by work queued on some stream
  int st = cuda_status(cudaDeviceSynchronize());
  if (st != ROSAQ_OK) return st;
  (void)s;
  if (ctx->ws) (void)cudaFree(ctx->ws);
  ctx->ws = nullptr;
  ctx->ws_bytes = 0;
  size_t want = bytes < (size_t)(4 << 20) ? (size_t)(4 << 20) : bytes;
  st = cuda_status(cudaMalloc(&ctx->ws, want));
  if (st != ROSAQ_OK) return st;
  ctx->ws_bytes = want;
  return ROSAQ_OK;
}

constexpr int kPrefillMinTiles = 40, kPrefillMinUnits = 36;
constexpr int kBlockTokens = 128;

int run_ops(rosaq_ctx *ctx, int M, int n, const PlanOp *ops, cudaStream_t s);

// 65 ... 1536 tokens as blocks of 128: one operation of the persistent launch per block, all in one launch
// (accumulators of 128 tokens; a weight tile is dequantised once per block).
int run_token_blocks(rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t, const int32_t *col_map,
                     __half *y, long long ldy, cudaStream_t s) {
  const int nb = (M + kBlockTokens - 1) / kBlockTokens;
  if (nb > kPlanMaxOps) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  PlanOp ops[kPlanMaxOps];
  for (int b = 0; b < nb; ++b) {
    const int m = std::min(kBlockTokens, M - b * kBlockTokens);
    ops[b] = PlanOp{x + (long long)b * kBlockTokens * ldx, ldx, -1, &t, col_map, y + (long long)b * kBlockTokens * ldy, ldy, m};
  }
  return run_ops(ctx, std::min(M, kBlockTokens), nb, ops, s);
}

int run_gemm(rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t, const int32_t *col_map,
             __half *y, long long ldy, cudaStream_t s) {
  if (ctx->impl == 1) return launch_linear_simt(ctx, x, M, ldx, t, col_map, y, ldy, s);
  if (ctx->impl == 6 && M > 64 && M <= kBlockTokens * kPlanMaxOps) return run_token_blocks(ctx, x, M, ldx, t, col_map, y, ldy, s);
  // Large batches of tokens run a weight on 256-column x 256-token tiles shared by pairs of CTAs -- where
  // the launch is long enough to pay for the exchange of the tiles that two pairs share: at least
  // kPrefillMinTiles tiles and kPrefillMinUnits 128-channel groups per pair of SMs (measured against the
  // per-call kernel on the 7B and 13B shapes at 256 ... 2048 tokens).
  if (prefill_supported(t, col_map) && (ctx->impl == 5 || (ctx->impl == 0 && M > 256))) {
    const long long tiles = (long long)((t.n_tiles + 1) / 2) * ((M + 255) / 256);
    const long long units = tiles * groups_per_tile(t);
    if (ctx->impl == 5 || (tiles >= kPrefillMinTiles && units >= (long long)kPrefillMinUnits * (ctx->sm_count / 2)))
      return launch_linear_prefill(ctx, x, M, ldx, t, y, ldy, s);
  }
  return launch_linear_tc(ctx, x, M, ldx, t, col_map, y, ldy, s);
}

// The persistent launch (rosaq_plan) pays off when a list is long: it saves a launch, a pipeline fill and a
// drain per operation, but a list of one or two operations exposes its own fixed costs (the exchange of
// shared tiles goes through L2 instead of a cluster's shared memory, and the phase after a rotation starts
// only when the rotation's last tile is written).  Measured at 64 tokens, 4096 -> 4096 INT4: a GEMM stage
// alone 15.9 us against 9.7 us on the per-call kernel; rotation + linear 30.5 us against 20.7 us as two
// launches; the ten operations of a 7B decoder layer 66 us against 100 us as seven launches.  So the single
// calls stay on the per-call kernels; implementation 4 routes them through the persistent launch.
bool use_plan(const rosaq_ctx *ctx, int M, bool with_rotation) {
  (void)with_rotation;
  return M <= 64 && ctx->impl == 4;
}

int run_ops(rosaq_ctx *ctx, int M, int n, const PlanOp *ops, cudaStream_t s) {
  PlanLaunch l;
  int st = plan_prepare(ctx, M, n, ops, &l);
  if (st == ROSAQ_OK) st = plan_launch(ctx, l, s);
  plan_release(&l);
  return st;
}

}  // namespace

extern "C" {

const char *rosaq_strerror(int status) {
  switch (status) {
    case ROSAQ_OK: return "ok";
    case ROSAQ_ERR_INVALID_ARG: return "invalid argument";
    case ROSAQ_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case ROSAQ_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
    case ROSAQ_ERR_ALLOC: return "allocation failed";
    case ROSAQ_ERR_CUDA: return "CUDA call failed";
    case ROSAQ_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case ROSAQ_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    default: return "unknown status";
  }
}

int rosaq_create(rosaq_ctx **out, int device) {
  if (!out) return ROSAQ_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  if (device < 0 || device >= count) return ROSAQ_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  int st = cuda_status(cudaGetDeviceProperties(&prop, device));
  if (st != ROSAQ_OK) return st;
  if (prop.major != 10) return ROSAQ_ERR_UNSUPPORTED_ARCH;
  DeviceGuard guard(device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  rosaq_ctx *ctx = new (std::nothrow) rosaq_ctx();
  if (!ctx) return ROSAQ_ERR_ALLOC;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->ws = nullptr;
  ctx->ws_bytes = 0;
  ctx->wait_limit = 1ll << 20;
  ctx->impl = 0;
  ctx->sk_partials = nullptr;
  ctx->sk_arrive = nullptr;
  ctx->sk_ctas = 2 * ctx->sm_count < rosaq::kSkMaxCtas ? 2 * ctx->sm_count : rosaq::kSkMaxCtas;
  ctx->pl_ctas = 0;
  ctx->pl_pairs = 0;
  ctx->pl_mode = 1;   // pairs of CTAs are built and tested but measured slower so far: off unless asked for
  ctx->pl_cost_set = 0;
  ctx->pl_cost[0] = kPlanCostFp16, ctx->pl_cost[1] = kPlanCostQuant, ctx->pl_cost[2] = kPlanCostTile;
  ctx->pl_partials = nullptr;
  ctx->pl_partial_bytes = 0;
  ctx->pl_sync = nullptr;
  ctx->pf_pairs = 0;
  ctx->pf_flags = nullptr;
  st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->d_status), 2 * sizeof(int)));   // [1]: scratch flag of argument checks
  if (st == ROSAQ_OK) st = cuda_status(cudaMemset(ctx->d_status, 0, 2 * sizeof(int)));
  // the stream-K workspace is taken here, once, so that no linear call ever allocates for it
  if (st == ROSAQ_OK)
    st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->sk_partials), (size_t)ctx->sk_ctas * 2 * rosaq::kSkPartialBytes));
  if (st == ROSAQ_OK) st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->sk_arrive), rosaq::kSkCounterInts * sizeof(int)));
  if (st == ROSAQ_OK) st = cuda_status(cudaMemset(ctx->sk_arrive, 0, rosaq::kSkCounterInts * sizeof(int)));
  if (st == ROSAQ_OK) st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->pl_sync), rosaq::kPlSyncWords * sizeof(unsigned)));
  if (st == ROSAQ_OK) st = cuda_status(cudaMemset(ctx->pl_sync, 0, rosaq::kPlSyncWords * sizeof(unsigned)));
  if (st == ROSAQ_OK) st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->pf_flags), (size_t)ctx->sm_count * sizeof(unsigned)));
  if (st == ROSAQ_OK) st = cuda_status(cudaMemset(ctx->pf_flags, 0, (size_t)ctx->sm_count * sizeof(unsigned)));
  // the partial tiles of a launch whose CTAs all share tiles at both ends of two phases (grown if a plan needs more)
  if (st == ROSAQ_OK) {
    const size_t bytes = (size_t)4 * ctx->sk_ctas * rosaq::kSkPartialBytes;
    st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&ctx->pl_partials), bytes));
    if (st == ROSAQ_OK) ctx->pl_partial_bytes = bytes;
  }
  if (st != ROSAQ_OK) {
    if (ctx->pl_sync) (void)cudaFree(ctx->pl_sync);
    if (ctx->pf_flags) (void)cudaFree(ctx->pf_flags);
    if (ctx->pl_partials) (void)cudaFree(ctx->pl_partials);
    if (ctx->d_status) (void)cudaFree(ctx->d_status);
    if (ctx->sk_partials) (void)cudaFree(ctx->sk_partials);
    if (ctx->sk_arrive) (void)cudaFree(ctx->sk_arrive);
    delete ctx;
    return st;
  }
  *out = ctx;
  return ROSAQ_OK;
}

int rosaq_destroy(rosaq_ctx *ctx) {
  if (!ctx) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (guard.ok) {
    (void)cudaDeviceSynchronize();
    if (ctx->ws) (void)cudaFree(ctx->ws);
    if (ctx->d_status) (void)cudaFree(ctx->d_status);
    if (ctx->sk_partials) (void)cudaFree(ctx->sk_partials);
    if (ctx->sk_arrive) (void)cudaFree(ctx->sk_arrive);
    if (ctx->pl_sync) (void)cudaFree(ctx->pl_sync);
    if (ctx->pf_flags) (void)cudaFree(ctx->pf_flags);
    if (ctx->pl_partials) (void)cudaFree(ctx->pl_partials);
    plan_free_schedules(ctx);
    (void)cudaGetLastError();
  }
  delete ctx;
  return ROSAQ_OK;
}

int rosaq_last_status(rosaq_ctx *ctx, void *stream) {
  if (!ctx) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int st = cuda_status(cudaStreamSynchronize(s));
  if (st != ROSAQ_OK) return st;
  int host = 0;
  st = cuda_status(cudaMemcpy(&host, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != ROSAQ_OK) return st;
  if (host != 0) {
    st = cuda_status(cudaMemset(ctx->d_status, 0, sizeof(int)));
    if (st != ROSAQ_OK) return st;
    // a launch that gave up may have left arrival counters of the stream-K exchange behind
    st = cuda_status(cudaMemset(ctx->sk_arrive, 0, rosaq::kSkCounterInts * sizeof(int)));
    if (st != ROSAQ_OK) return st;
    st = cuda_status(cudaMemset(ctx->pl_sync, 0, rosaq::kPlSyncWords * sizeof(unsigned)));
    if (st != ROSAQ_OK) return st;
    st = cuda_status(cudaMemset(ctx->pf_flags, 0, (size_t)ctx->sm_count * sizeof(unsigned)));
    if (st != ROSAQ_OK) return st;
  }
  return host;
}

int64_t rosaq_set_wait_limit(rosaq_ctx *ctx, int64_t iterations) {
  if (!ctx) return 0;
  int64_t prev = ctx->wait_limit;
  if (iterations > 0) ctx->wait_limit = iterations;
  return prev;
}

int rosaq_set_linear_impl(rosaq_ctx *ctx, int impl) {
  if (!ctx) return 0;
  int prev = ctx->impl;
  if (impl >= 0 && impl <= 6) ctx->impl = impl;
  return prev;
}

int rosaq_calib_cov(rosaq_ctx *ctx, const void *X, int x_dtype, int64_t n_tokens, int d, int64_t ldx,
                    int n_blocks, float *C, void *stream) {
  if (!ctx || !X || !C) return ROSAQ_ERR_INVALID_ARG;
  if (x_dtype != ROSAQ_F16 && x_dtype != ROSAQ_F32) return ROSAQ_ERR_INVALID_ARG;
  if (n_tokens < 0 || d <= 0 || n_blocks <= 0 || ldx < d) return ROSAQ_ERR_INVALID_ARG;
  if (d % n_blocks != 0 || d % 8 != 0 || (d / n_blocks) % 8 != 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(X) || !aligned16(C) || (ldx % 8) != 0) return ROSAQ_ERR_ALIGNMENT;
  if (n_tokens == 0) return ROSAQ_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  return launch_cov(ctx, X, x_dtype, n_tokens, d, ldx, n_blocks, C, static_cast<cudaStream_t>(stream));
}

static int quantize_impl(rosaq_ctx *ctx, const void *W, int d_in, int d_out, const rosaq_rot *rot, const float *in_scale,
                         int bits, int group, int k_salient, rosaq_weight **out, void *stream) {
  if (!out) return ROSAQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !W) return ROSAQ_ERR_INVALID_ARG;
  int st = check_quant_args(d_in, d_out, bits, group, k_salient);
  if (st != ROSAQ_OK) return st;
  if (!aligned16(W)) return ROSAQ_ERR_ALIGNMENT;
  if (rot) {
    if (!rot->q || rot->d != d_in || rot->n_blocks <= 0 || d_in % rot->n_blocks != 0) return ROSAQ_ERR_INVALID_ARG;
    if (rot->q_dtype != ROSAQ_F32 && rot->q_dtype != ROSAQ_F16) return ROSAQ_ERR_INVALID_ARG;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  rosaq_weight *w = new (std::nothrow) rosaq_weight();
  if (!w) return ROSAQ_ERR_ALLOC;
  w->group = group;
  w->k_salient = k_salient;
  w->device = ctx->device;
  w->t = make_geometry(d_in, d_out, bits, k_salient / kGroup, (d_in - k_salient) / kGroup, 0);
  float *Wp = nullptr, *Ws = nullptr;
  const size_t fbytes = sizeof(float) * (size_t)d_in * d_out;
  st = alloc_blob(&w->t);
  if (st == ROSAQ_OK && rot && rot->perm) {
    // the rotate kernels index R and W with perm: reject anything that is not a permutation first
    int32_t *inv = nullptr;
    st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&inv), sizeof(int32_t) * (size_t)d_in));
    if (st == ROSAQ_OK) st = launch_invert_perm(rot->perm, d_in, inv, ctx->d_status + 1, s);
    if (inv) (void)cudaFree(inv);
  }
  if (st == ROSAQ_OK) st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&Wp), fbytes));
  if (st == ROSAQ_OK && rot && in_scale) st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&Ws), fbytes));
  if (st == ROSAQ_OK) {
    const __half *Wh = static_cast<const __half *>(W);
    if (rot && in_scale) {
      st = launch_scale_rows(Wh, in_scale, d_in, d_out, Ws, s);
      if (st == ROSAQ_OK)
        st = launch_rotate_weights_w32(rot->q, rot->q_dtype == ROSAQ_F32, d_in, rot->n_blocks, rot->perm, Ws, d_out, Wp, s);
    } else if (rot) {
      st = launch_rotate_weights(rot->q, rot->q_dtype == ROSAQ_F32, d_in, rot->n_blocks, rot->perm, Wh, d_out, Wp, s);
    } else if (in_scale) {
      st = launch_scale_rows(Wh, in_scale, d_in, d_out, Wp, s);
    } else {
      st = launch_cast_weights(Wh, d_in, d_out, Wp, s);
    }
  }
  if (st == ROSAQ_OK) st = launch_quant_pack(Wp, w->t, s);
  if (st == ROSAQ_OK) st = cuda_status(cudaStreamSynchronize(s));
  if (Wp) (void)cudaFree(Wp);
  if (Ws) (void)cudaFree(Ws);
  if (st != ROSAQ_OK) {
    if (w->t.blob) (void)cudaFree(w->t.blob);
    delete w;
    return st;
  }
  *out = w;
  return ROSAQ_OK;
}

int rosaq_quantize(rosaq_ctx *ctx, const void *W, int d_in, int d_out, const rosaq_rot *rot, int bits,
                   int group, int k_salient, rosaq_weight **out, void *stream) {
  return quantize_impl(ctx, W, d_in, d_out, rot, nullptr, bits, group, k_salient, out, stream);
}

int rosaq_quantize_scaled(rosaq_ctx *ctx, const void *W, int d_in, int d_out, const rosaq_rot *rot, const float *in_scale,
                          int bits, int group, int k_salient, rosaq_weight **out, void *stream) {
  if (out) *out = nullptr;
  if (in_scale && !aligned16(in_scale)) return ROSAQ_ERR_ALIGNMENT;
  return quantize_impl(ctx, W, d_in, d_out, rot, in_scale, bits, group, k_salient, out, stream);
}

int rosaq_weight_export(rosaq_ctx *ctx, const rosaq_weight *w, uint32_t *qw, void *scales_f16, void *zeros_f16,
                        void *salient_f16, void *stream) {
  if (!ctx || !w) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  return launch_export(w->t, qw, static_cast<__half *>(scales_f16), static_cast<__half *>(zeros_f16),
                       static_cast<__half *>(salient_f16), static_cast<cudaStream_t>(stream));
}

int rosaq_weight_import(rosaq_ctx *ctx, int d_in, int d_out, int bits, int group, int k_salient,
                        const uint32_t *qw, const void *scales_f16, const void *zeros_f16, const void *salient_f16,
                        rosaq_weight **out, void *stream) {
  if (!out) return ROSAQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx) return ROSAQ_ERR_INVALID_ARG;
  int st = check_quant_args(d_in, d_out, bits, group, k_salient);
  if (st != ROSAQ_OK) return st;
  if (k_salient > 0 && !salient_f16) return ROSAQ_ERR_INVALID_ARG;
  if (k_salient < d_in && (!qw || !scales_f16 || !zeros_f16)) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rosaq_weight *w = new (std::nothrow) rosaq_weight();
  if (!w) return ROSAQ_ERR_ALLOC;
  w->group = group;
  w->k_salient = k_salient;
  w->device = ctx->device;
  w->t = make_geometry(d_in, d_out, bits, k_salient / kGroup, (d_in - k_salient) / kGroup, 0);
  st = alloc_blob(&w->t);
  if (st == ROSAQ_OK)
    st = launch_import(w->t, qw, static_cast<const __half *>(scales_f16), static_cast<const __half *>(zeros_f16),
                       static_cast<const __half *>(salient_f16), s);
  if (st == ROSAQ_OK) st = cuda_status(cudaStreamSynchronize(s));
  if (st != ROSAQ_OK) {
    if (w->t.blob) (void)cudaFree(w->t.blob);
    delete w;
    return st;
  }
  *out = w;
  return ROSAQ_OK;
}

int rosaq_weight_free(rosaq_weight *w) {
  if (!w) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(w->device);
  if (guard.ok && w->t.blob) {
    (void)cudaFree(w->t.blob);
    (void)cudaGetLastError();
  }
  delete w;
  return ROSAQ_OK;
}

int rosaq_weight_info(const rosaq_weight *w, int *d_in, int *d_out, int *bits, int *group, int *k_salient,
                      int64_t *device_bytes) {
  if (!w) return ROSAQ_ERR_INVALID_ARG;
  if (d_in) *d_in = w->t.d_in;
  if (d_out) *d_out = w->t.d_out;
  if (bits) *bits = w->t.bits;
  if (group) *group = w->group;
  if (k_salient) *k_salient = w->k_salient;
  if (device_bytes) *device_bytes = w->t.bytes;
  return ROSAQ_OK;
}

int rosaq_rotation_create(rosaq_ctx *ctx, const rosaq_rot *rot, rosaq_rotation **out, void *stream) {
  if (!out) return ROSAQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !rot || !rot->q) return ROSAQ_ERR_INVALID_ARG;
  if (rot->q_dtype != ROSAQ_F16) return ROSAQ_ERR_INVALID_ARG;
  if (rot->d <= 0 || rot->n_blocks <= 0 || rot->d % rot->n_blocks != 0) return ROSAQ_ERR_INVALID_ARG;
  const int dh = rot->d / rot->n_blocks;
  if (dh % kGroup != 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  if (!aligned16(rot->q)) return ROSAQ_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rosaq_rotation *r = new (std::nothrow) rosaq_rotation();
  if (!r) return ROSAQ_ERR_ALLOC;
  r->d = rot->d;
  r->device = ctx->device;
  r->col_map = nullptr;
  // 128-channel head blocks are stored in pairs, as 256 x 256 blocks with zero off-diagonal quarters (2 MB
  // instead of 1 MB at d = 4096): two adjacent column tiles then multiply the same channels, which lets a
  // pair of SMs share one MMA stream over them
  const int bg = (dh == kGroup && rot->n_blocks % 2 == 0) ? 2 : dh / kGroup;
  r->t = make_geometry(rot->d, rot->d, 4, bg, 0, rot->n_blocks == 1 ? 0 : bg);
  int st = alloc_blob(&r->t);
  if (st == ROSAQ_OK && rot->perm) {
    // checked first: the epilogues store through col_map, so a perm that is not a permutation is an error
    // code here, never a stray write later
    st = cuda_status(cudaMalloc(reinterpret_cast<void **>(&r->col_map), sizeof(int32_t) * rot->d));
    if (st == ROSAQ_OK) st = launch_invert_perm(rot->perm, rot->d, r->col_map, ctx->d_status + 1, s);
  }
  if (st == ROSAQ_OK) st = launch_rotation_tiles(static_cast<const __half *>(rot->q), rot->d, rot->n_blocks, r->t, s);
  if (st == ROSAQ_OK) st = cuda_status(cudaStreamSynchronize(s));
  if (st != ROSAQ_OK) {
    if (r->t.blob) (void)cudaFree(r->t.blob);
    if (r->col_map) (void)cudaFree(r->col_map);
    delete r;
    return st;
  }
  *out = r;
  return ROSAQ_OK;
}

int rosaq_rotation_free(rosaq_rotation *r) {
  if (!r) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(r->device);
  if (guard.ok) {
    if (r->t.blob) (void)cudaFree(r->t.blob);
    if (r->col_map) (void)cudaFree(r->col_map);
    (void)cudaGetLastError();
  }
  delete r;
  return ROSAQ_OK;
}

static int check_act(const void *p, int M, int64_t ld, int d) {
  if (!p || M <= 0 || ld < d) return ROSAQ_ERR_INVALID_ARG;
  if (!aligned16(p) || (ld % 8) != 0) return ROSAQ_ERR_ALIGNMENT;
  return ROSAQ_OK;
}

int rosaq_rotate(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r, void *x_rot,
                 int64_t ldxr, void *stream) {
  if (!ctx || !r) return ROSAQ_ERR_INVALID_ARG;
  int st = check_act(x, M, ldx, r->d);
  if (st == ROSAQ_OK) st = check_act(x_rot, M, ldxr, r->d);
  if (st != ROSAQ_OK) return st;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  if (use_plan(ctx, M, false)) {
    const PlanOp op{static_cast<const __half *>(x), ldx, -1, &r->t, r->col_map, static_cast<__half *>(x_rot), ldxr};
    return run_ops(ctx, M, 1, &op, static_cast<cudaStream_t>(stream));
  }
  return run_gemm(ctx, static_cast<const __half *>(x), M, ldx, r->t, r->col_map, static_cast<__half *>(x_rot), ldxr,
                  static_cast<cudaStream_t>(stream));
}

int rosaq_linear(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r, const rosaq_weight *w,
                 void *y, int64_t ldy, void *stream) {
  if (!ctx || !w) return ROSAQ_ERR_INVALID_ARG;
  int st = check_act(x, M, ldx, w->t.d_in);
  if (st == ROSAQ_OK) st = check_act(y, M, ldy, w->t.d_out);
  if (st != ROSAQ_OK) return st;
  if (r && r->d != w->t.d_in) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half *xin = static_cast<const __half *>(x);
  long long ld = ldx;
  if (r) {
    st = ensure_workspace(ctx, sizeof(__half) * (size_t)M * r->d, s);
    if (st != ROSAQ_OK) return st;
  }
  if (use_plan(ctx, M, r != nullptr)) {
    // one launch: x . R into the workspace (phase 1), the GEMM stage on it (phase 2)
    PlanOp ops[2];
    int n = 0;
    if (r) ops[n++] = PlanOp{xin, ldx, -1, &r->t, r->col_map, static_cast<__half *>(ctx->ws), r->d};
    ops[n] = PlanOp{xin, ldx, r ? 0 : -1, &w->t, nullptr, static_cast<__half *>(y), ldy};
    return run_ops(ctx, M, n + 1, ops, s);
  }
  if (r) {
    st = run_gemm(ctx, xin, M, ldx, r->t, r->col_map, static_cast<__half *>(ctx->ws), r->d, s);
    if (st != ROSAQ_OK) return st;
    xin = static_cast<const __half *>(ctx->ws);
    ld = r->d;
  }
  return run_gemm(ctx, xin, M, ld, w->t, nullptr, static_cast<__half *>(y), ldy, s);
}

int rosaq_linear_multi(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r, int n,
                       const rosaq_weight *const *w, void *const *y, const int64_t *ldy, void *stream) {
  if (!ctx || !w || !y || !ldy || n < 1 || n > 4) return ROSAQ_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (!w[i]) return ROSAQ_ERR_INVALID_ARG;
  int st = check_act(x, M, ldx, w[0]->t.d_in);
  for (int i = 0; i < n && st == ROSAQ_OK; ++i) {
    const TiledOperand &a = w[i]->t, &b = w[0]->t;
    if (a.d_in != b.d_in || a.g_fp16 != b.g_fp16 || a.g_quant != b.g_quant || (b.g_quant > 0 && a.bits != b.bits))
      return ROSAQ_ERR_INVALID_ARG;
    st = check_act(y[i], M, ldy[i], a.d_out);
  }
  if (st != ROSAQ_OK) return st;
  if (r && r->d != w[0]->t.d_in) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half *xin = static_cast<const __half *>(x);
  long long ld = ldx;
  if (r) {
    st = ensure_workspace(ctx, sizeof(__half) * (size_t)M * r->d, s);
    if (st != ROSAQ_OK) return st;
  }
  if (use_plan(ctx, M, r != nullptr)) {
    PlanOp ops[5];
    int k = 0;
    if (r) ops[k++] = PlanOp{xin, ldx, -1, &r->t, r->col_map, static_cast<__half *>(ctx->ws), r->d};
    for (int i = 0; i < n; ++i) ops[k++] = PlanOp{xin, ldx, r ? 0 : -1, &w[i]->t, nullptr, static_cast<__half *>(y[i]), ldy[i]};
    return run_ops(ctx, M, k, ops, s);
  }
  if (r) {
    st = run_gemm(ctx, xin, M, ldx, r->t, r->col_map, static_cast<__half *>(ctx->ws), r->d, s);
    if (st != ROSAQ_OK) return st;
    xin = static_cast<const __half *>(ctx->ws);
    ld = r->d;
  }
  if (ctx->impl == 1) {
    for (int i = 0; i < n && st == ROSAQ_OK; ++i)
      st = launch_linear_simt(ctx, xin, M, ld, w[i]->t, nullptr, static_cast<__half *>(y[i]), ldy[i], s);
    return st;
  }
  const TiledOperand *ts[4];
  __half *ys[4];
  long long ldys[4];
  for (int i = 0; i < n; ++i) ts[i] = &w[i]->t, ys[i] = static_cast<__half *>(y[i]), ldys[i] = ldy[i];
  return launch_linear_tc_multi(ctx, xin, M, ld, n, ts, nullptr, ys, ldys, s);
}

int rosaq_plan_create(rosaq_ctx *ctx, int M, int n_ops, const rosaq_op *ops, rosaq_plan **out) {
  if (!out) return ROSAQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!ctx || !ops || n_ops < 1 || M < 1) return ROSAQ_ERR_INVALID_ARG;
  if (n_ops > kPlanMaxOps || M > 128) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  rosaq_plan *pl = new (std::nothrow) rosaq_plan();
  if (!pl) return ROSAQ_ERR_ALLOC;
  pl->M = M;
  pl->device = ctx->device;
  int st = ROSAQ_OK;
  for (int i = 0; i < n_ops && st == ROSAQ_OK; ++i) {
    const rosaq_op &o = ops[i];
    if ((o.r != nullptr) == (o.w != nullptr) || o.x_from >= i) {
      st = ROSAQ_ERR_INVALID_ARG;
      break;
    }
    const TiledOperand &t = o.r ? o.r->t : o.w->t;
    const void *x = o.x_from >= 0 ? ops[o.x_from].y : o.x;
    const int64_t ldx = o.x_from >= 0 ? ops[o.x_from].ldy : o.ldx;
    if (o.x_from >= 0) {
      const rosaq_op &src = ops[o.x_from];
      const int src_d_out = src.r ? src.r->t.d_out : src.w->t.d_out;
      if (src_d_out != t.d_in) st = ROSAQ_ERR_INVALID_ARG;
    }
    if (st == ROSAQ_OK) st = check_act(x, M, ldx, t.d_in);
    if (st == ROSAQ_OK) st = check_act(o.y, M, o.ldy, t.d_out);
    if (st == ROSAQ_OK && (o.r ? o.r->device : o.w->device) != ctx->device) st = ROSAQ_ERR_INVALID_ARG;
    if (st == ROSAQ_OK)
      pl->ops.push_back(PlanOp{static_cast<const __half *>(x), ldx, o.x_from >= 0 ? o.x_from : -1, &t,
                               o.r ? o.r->col_map : nullptr, static_cast<__half *>(o.y), o.ldy});
  }
  // an output may be read only through x_from (which orders the two operations) and written by one
  // operation: any other overlap of a y with an x or a y would be a race inside the launch
  // (views of M rows: with equal row strides, disjoint column ranges of one wider buffer do not overlap)
  auto overlap = [M](const void *pa, int64_t lda, int da, const void *pb, int64_t ldb, int db) {
    const char *alo = static_cast<const char *>(pa), *blo = static_cast<const char *>(pb);
    const char *ahi = alo + sizeof(__half) * ((size_t)(M - 1) * (size_t)lda + (size_t)da);
    const char *bhi = blo + sizeof(__half) * ((size_t)(M - 1) * (size_t)ldb + (size_t)db);
    if (!(alo < bhi && blo < ahi)) return false;
    if (lda != ldb) return true;
    const long long off = (blo - alo) / (long long)sizeof(__half);
    const long long c = ((off % lda) + lda) % lda;              // b's first column inside a's rows
    return !(c >= da && c + db <= lda);
  };
  for (int i = 0; i < n_ops && st == ROSAQ_OK; ++i) {
    const PlanOp &a = pl->ops[i];
    for (int j = 0; j < n_ops && st == ROSAQ_OK; ++j) {
      const PlanOp &b = pl->ops[j];
      // (an operation's own x too: its tiles read all of x while others already write y)
      if (b.dep != i && overlap(a.y, a.ldy, a.t->d_out, b.x, b.ldx, b.t->d_in)) st = ROSAQ_ERR_INVALID_ARG;
      if (j > i && overlap(a.y, a.ldy, a.t->d_out, b.y, b.ldy, b.t->d_out)) st = ROSAQ_ERR_INVALID_ARG;
    }
  }
  if (st == ROSAQ_OK) {
    DeviceGuard guard(ctx->device);
    st = guard.ok ? plan_prepare(ctx, M, n_ops, pl->ops.data(), &pl->launch) : ROSAQ_ERR_CUDA;
  }
  if (st != ROSAQ_OK) {
    delete pl;
    return st;
  }
  *out = pl;
  return ROSAQ_OK;
}

int rosaq_plan_run(rosaq_ctx *ctx, const rosaq_plan *plan, void *stream) {
  if (!ctx || !plan || plan->device != ctx->device) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  return plan_launch(ctx, plan->launch, static_cast<cudaStream_t>(stream));
}

int rosaq_plan_free(rosaq_plan *plan) {
  if (!plan) return ROSAQ_ERR_INVALID_ARG;
  plan_release(&plan->launch);
  delete plan;
  return ROSAQ_OK;
}

int rosaq_set_plan_costs(rosaq_ctx *ctx, int fp16_group, int quant_group, int tile) {
  if (!ctx || fp16_group < 1 || quant_group < 1 || tile < 0 || fp16_group > 1000 || quant_group > 1000 || tile > 1000)
    return ROSAQ_ERR_INVALID_ARG;
  ctx->pl_cost[0] = fp16_group, ctx->pl_cost[1] = quant_group, ctx->pl_cost[2] = tile;
  ctx->pl_cost_set = 1;
  return ROSAQ_OK;
}

int rosaq_set_plan_pairs(rosaq_ctx *ctx, int enable) {
  if (!ctx) return ROSAQ_ERR_INVALID_ARG;
  const int prev = ctx->pl_mode != 1;
  ctx->pl_mode = enable ? 0 : 1;
  return prev;
}

int rosaq_plan_ctas(rosaq_ctx *ctx) {
  if (!ctx) return ROSAQ_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  const int p = plan_ctas(ctx);
  return p > 0 ? p : ROSAQ_ERR_CUDA;
}

int rosaq_plan_schedule(int n_ops, const int32_t *n_tiles, const int32_t *groups, const int32_t *g_fp16, const int32_t *x_from,
                        const int32_t *copies, int n_ctas, int32_t *piece_begin, int32_t *pieces, int max_pieces) {
  if (n_ops < 1 || n_ops > kPlanMaxOps || !n_tiles || !groups || !g_fp16 || !x_from || n_ctas < 1 || !piece_begin ||
      (!pieces && max_pieces > 0) || max_pieces < 0)
    return ROSAQ_ERR_INVALID_ARG;
  std::vector<PlanGeom> geom(n_ops);
  for (int i = 0; i < n_ops; ++i) geom[i] = PlanGeom{n_tiles[i], groups[i], g_fp16[i], x_from[i] < 0 ? -1 : x_from[i], copies ? copies[i] : 1,
                       copies && copies[i] > 1 ? kPlanCostScatterTile : 0};
  const int cost[3] = {kPlanCostFp16, kPlanCostQuant, kPlanCostTile};
  PlanSchedule s;
  const int st = plan_build_schedule(geom, n_ctas, cost, &s);
  if (st != ROSAQ_OK) return st;
  for (int c = 0; c <= n_ctas; ++c) piece_begin[c] = s.seg_begin[c];
  const int total = (int)s.segs.size();
  for (int k = 0; k < total && k < max_pieces; ++k) {
    const PlanSeg &g = s.segs[k];
    int32_t *o = pieces + (size_t)k * 12;
    o[0] = g.prob, o[1] = g.tile, o[2] = g.g_begin, o[3] = g.g_end, o[4] = g.n_contrib, o[5] = g.contrib_idx;
    o[6] = g.slot0, o[7] = g.counter, o[8] = g.closer_idx, o[9] = g.n_closers, o[10] = g.tok_begin, o[11] = g.tok_end;
  }
  return total;
}

}  // extern "C"
