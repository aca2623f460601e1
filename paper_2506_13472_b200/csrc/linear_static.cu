// rosaq_linear_static: the rotated linear for callers that must not allocate device memory.
//
// rosaq_linear with a rotation keeps the rotated activations x.R in a context workspace that it
// grows with cudaMalloc when a call needs more room.  Some callers cannot live with that: a serving
// process whose memory pool has already claimed every free byte of the device (cudaMalloc simply
// fails there), a latency-critical loop that cannot afford the device-wide synchronisation an
// allocation or free implies, or a host framework that forbids allocations outside its own
// allocator.  This variant runs the same two kernels but keeps x.R in a fixed array that is part
// of the library image, so it never allocates or frees anything.
//
// The array below exists once per device that loads the library and stays until the process
// exits.  In host code its name is only a handle for the runtime, not a device address, so the
// address is looked up once per device with cudaGetSymbolAddress (with that device current) and
// that pointer is what the kernels get.
#include <mutex>

#include "rosaq_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = size_t(4) << 20;  // 4 MiB: M * d_in fp16 values, e.g. 512 tokens x 4096
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void *g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch on each device, once resolved

// Resolves the array's address on `device` (which must be the current device).  No allocation.
int scratch_for_device(int device, void **out) {
  if (device < 0 || device >= kMaxDevices) return ROSAQ_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[device]) {
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_CUDA;
    }
    g_scratch_ptr[device] = p;
  }
  *out = g_scratch_ptr[device];
  return ROSAQ_OK;
}

int run_stage(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, const rosaq::TiledOperand &t,
              const int32_t *col_map, __half *y, long long ldy, cudaStream_t s) {
  if (ctx->impl == 1) return rosaq::launch_linear_simt(ctx, x, M, ldx, t, col_map, y, ldy, s);
  return rosaq::launch_linear_tc(ctx, x, M, ldx, t, col_map, y, ldy, s);
}

}  // namespace

extern "C" int rosaq_linear_static(rosaq_ctx *ctx, const void *x, int M, int64_t ldx, const rosaq_rotation *r,
                                   const rosaq_weight *w, void *y, int64_t ldy, void *stream) {
  if (!ctx || !w || !x || !y || M <= 0) return ROSAQ_ERR_INVALID_ARG;
  if (ldx < w->t.d_in || ldy < w->t.d_out) return ROSAQ_ERR_INVALID_ARG;
  if (!rosaq::aligned16(x) || !rosaq::aligned16(y) || (ldx % 8) != 0 || (ldy % 8) != 0) return ROSAQ_ERR_ALIGNMENT;
  if (r && r->d != w->t.d_in) return ROSAQ_ERR_INVALID_ARG;
  if (r && sizeof(__half) * (size_t)M * (size_t)r->d > kStaticScratchBytes) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  rosaq::DeviceGuard guard(ctx->device);
  if (!guard.ok) return ROSAQ_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half *xin = static_cast<const __half *>(x);
  long long ld = ldx;
  if (r) {
    void *scratch = nullptr;
    int st = scratch_for_device(ctx->device, &scratch);
    if (st != ROSAQ_OK) return st;
    // every element of the [M][d] intermediate is written by the rotation before the GEMM stage reads
    // it (rows past M are zero-filled by the activation copy itself), so nothing has to be cleared
    st = run_stage(ctx, xin, M, ldx, r->t, r->col_map, static_cast<__half *>(scratch), r->d, s);
    if (st != ROSAQ_OK) return st;
    xin = static_cast<const __half *>(scratch);
    ld = r->d;
  }
  return run_stage(ctx, xin, M, ld, w->t, nullptr, static_cast<__half *>(y), ldy, s);
}
