// Internal declarations shared by the translation units of librosaq (CUDA side only).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "rosaq.h"

namespace rosaq {

// ------------------------------------------------------------------------------------
// Tiled operand layout.
//
// A [d_in][d_out] matrix that the GEMM kernels stream is cut into tiles of 128 input
// channels (one quantization group: group size 128, Section 3) by
// 128 output columns.  All tiles of one column tile are contiguous, in input-channel
// order, so that a CTA walking down K reads one linear stretch of memory; every tile is
// a self-contained blob that one bulk copy brings into shared memory:
//
//   fp16 tile   (salient group of Eq. 3, or a tile of a rotation matrix)      32768 B
//     element (k, n) at byte ((k/8)*128 + n)*16 + (k%8)*2
//   INT4 tile                                                         8192 + 512 B
//     16-byte chunk j = k/32 of column n at (j*128 + n)*16; inside it word w = (k%32)/8;
//     inside the word the code of k%8 = i sits in nibble (i even ? i/2 : 4 + i/2), so that
//     (word & 0x000f000f) is the pair (k, k+1) laid out as two fp16 mantissas
//   INT3 tile                                                         6144 + 512 B
//     12 words per column: word index wl = (k/32)*3 + ((k%32)/10) for k%32 < 30, the code of
//     i = k%32 at bit 3*((i%10)/2) + 16*(i%2); codes 30 and 31 of each 32 are spread over bit
//     15 (code 30) and bit 31 (code 31) of the three words, one bit per word;
//     word wl of column n at ((wl/4)*128 + n)*16 + (wl%4)*4
//   quantized tiles end with 128 x {fp16 scale, fp16 zero} (column n at codes_bytes + 4n)
//
// Column k of TMEM then holds the fp16 pair (2k, 2k+1), which is what the chunk order
// above delivers after the in-register dequantisation.
// ------------------------------------------------------------------------------------
constexpr int kTileN = 128;
constexpr int kGroup = 128;
constexpr int kFp16TileBytes = kGroup * kTileN * 2;
constexpr int kInt4CodeBytes = kGroup * kTileN / 2;
constexpr int kInt3CodeBytes = kGroup * kTileN * 3 / 8;
constexpr int kScaleBytes = kTileN * 4;

__host__ __device__ inline int quant_tile_bytes(int bits) {
  return (bits == 4 ? kInt4CodeBytes : kInt3CodeBytes) + kScaleBytes;
}
__host__ __device__ inline int quant_code_bytes(int bits) {
  return bits == 4 ? kInt4CodeBytes : kInt3CodeBytes;
}

struct TiledOperand {
  uint8_t *blob;        // device
  int d_in, d_out;      // logical sizes
  int n_tiles;          // ceil(d_out / 128); the last tile is zero padded
  int bits;             // 3 or 4 (ignored when g_quant == 0)
  int g_fp16;           // leading fp16 groups per column tile
  int g_quant;          // quantized groups that follow
  int block_groups;     // 0: every column tile spans all of d_in.  >0: block-diagonal operand whose
                        // column tile t only holds the `block_groups` groups of its own diagonal
                        // block (then g_fp16 == block_groups, g_quant == 0)
  long long tile_stride;  // bytes between consecutive column tiles
  long long bytes;        // total
};

__host__ __device__ inline int groups_per_tile(const TiledOperand &t) { return t.g_fp16 + t.g_quant; }

// byte offset of local group lg of column tile nt
__host__ __device__ inline long long tile_offset(const TiledOperand &t, int nt, int lg) {
  long long o = (long long)nt * t.tile_stride;
  if (lg < t.g_fp16) return o + (long long)lg * kFp16TileBytes;
  return o + (long long)t.g_fp16 * kFp16TileBytes + (long long)(lg - t.g_fp16) * quant_tile_bytes(t.bits);
}

// first input channel that local group lg of column tile nt multiplies
__host__ __device__ inline int group_k0(const TiledOperand &t, int nt, int lg) {
  if (t.block_groups == 0) return lg * kGroup;
  int tiles_per_block = t.block_groups;  // square blocks: block size = block_groups * 128 columns
  return ((nt / tiles_per_block) * t.block_groups + lg) * kGroup;
}

// ---- positions inside a tile -----------------------------------------------------------
__host__ __device__ inline int fp16_tile_byte(int k, int n) { return ((k >> 3) * kTileN + n) * 16 + (k & 7) * 2; }

__host__ __device__ inline void int4_pos(int k, int n, int *byte, int *shift) {
  int j = k >> 5, w = (k & 31) >> 3, i = k & 7;
  int nib = (i & 1) ? 4 + (i >> 1) : (i >> 1);
  *byte = (j * kTileN + n) * 16 + w * 4;
  *shift = nib * 4;
}

// INT3: codes 0..29 of each 32 occupy one 3-bit field; codes 30/31 are bit-sliced (see above).
__host__ __device__ inline int int3_word_byte(int wl, int n) { return ((wl >> 2) * kTileN + n) * 16 + (wl & 3) * 4; }
__host__ __device__ inline void int3_field(int i /*0..29*/, int *word, int *shift) {
  *word = i / 10;
  *shift = 3 * ((i % 10) >> 1) + 16 * (i & 1);
}

#ifdef __CUDACC__
// ---- per-column access to a quantized tile (code words of one output column in registers) ----
template <int kBits>
__device__ __forceinline__ void put_code(uint32_t *words, int k, uint32_t code) {
  if (kBits == 4) {
    int i = k & 7;
    int nib = (i & 1) ? 4 + (i >> 1) : (i >> 1);
    words[k >> 3] |= code << (nib * 4);
  } else {
    int set = k >> 5, i = k & 31;
    if (i < 30) {
      words[set * 3 + i / 10] |= code << (3 * ((i % 10) >> 1) + 16 * (i & 1));
    } else {
      int bit = 15 + 16 * (i - 30);
#pragma unroll
      for (int b = 0; b < 3; ++b) words[set * 3 + b] |= ((code >> b) & 1u) << bit;
    }
  }
}

template <int kBits>
__device__ __forceinline__ uint32_t get_code(const uint32_t *words, int k) {
  if (kBits == 4) {
    int i = k & 7;
    int nib = (i & 1) ? 4 + (i >> 1) : (i >> 1);
    return (words[k >> 3] >> (nib * 4)) & 0xf;
  } else {
    int set = k >> 5, i = k & 31;
    if (i < 30) return (words[set * 3 + i / 10] >> (3 * ((i % 10) >> 1) + 16 * (i & 1))) & 0x7;
    int bit = 15 + 16 * (i - 30);
    uint32_t c = 0;
#pragma unroll
    for (int b = 0; b < 3; ++b) c |= ((words[set * 3 + b] >> bit) & 1u) << b;
    return c;
  }
}

template <int kBits>
__device__ __forceinline__ void store_quant_tile_column(uint8_t *tile, int n, const uint32_t *words, __half scale,
                                                        __half zero) {
  constexpr int kWords = kBits == 4 ? 16 : 12;
#pragma unroll
  for (int j = 0; j < kWords / 4; ++j)
    *reinterpret_cast<uint4 *>(tile + (j * kTileN + n) * 16) =
        make_uint4(words[4 * j], words[4 * j + 1], words[4 * j + 2], words[4 * j + 3]);
  *reinterpret_cast<uint32_t *>(tile + quant_code_bytes(kBits) + n * 4) =
      (uint32_t)__half_as_ushort(scale) | ((uint32_t)__half_as_ushort(zero) << 16);
}

template <int kBits>
__device__ __forceinline__ void load_quant_tile_column(const uint8_t *tile, int n, uint32_t *words, __half *scale,
                                                       __half *zero) {
  constexpr int kWords = kBits == 4 ? 16 : 12;
#pragma unroll
  for (int j = 0; j < kWords / 4; ++j) {
    uint4 v = *reinterpret_cast<const uint4 *>(tile + (j * kTileN + n) * 16);
    words[4 * j] = v.x, words[4 * j + 1] = v.y, words[4 * j + 2] = v.z, words[4 * j + 3] = v.w;
  }
  uint32_t sz = *reinterpret_cast<const uint32_t *>(tile + quant_code_bytes(kBits) + n * 4);
  *scale = __ushort_as_half((unsigned short)(sz & 0xffff));
  *zero = __ushort_as_half((unsigned short)(sz >> 16));
}

#endif  // __CUDACC__

// ---- handles -----------------------------------------------------------------------------
}  // namespace rosaq

namespace rosaq {
constexpr int kSkMaxCtas = 320;                     // stream-K grid limit (two CTAs per SM)
constexpr int kSkCounterInts = 1024;                // arrival counters (one per column tile of a launch)
constexpr size_t kSkPartialBytes = 128 * 64 * sizeof(float);   // one partial tile: 128 columns x 64 tokens

// ---- the persistent multi-problem launch (linear_plan.cu) --------------------------------
constexpr int kPlanMaxOps = 12;                     // problems in one launch
constexpr int kPlanMaxCtas = 512;
constexpr int kPlMaxCounters = 4096;                // column tiles shared between CTAs in one launch
constexpr int kPlSyncFinished = 0, kPlSyncDone = 4, kPlSyncArrive = 16;   // word offsets in the sync buffer
constexpr int kPlSyncWords = kPlSyncArrive + kPlMaxCounters;
// Relative cost of the work items when a phase is cut into equal shares.  Both kinds of group cost the
// tensor pipe eight MMAs (about 700 cycles in place); an fp16 group also moves 32 KB, which takes an SM's
// share of the HBM bandwidth about 1400 cycles when every SM streams fp16 tiles, less when some run
// quantized groups next to it.  Measured on the 7B decoder layer: 12 : 7 (64.7 us per step; 10 : 7 65.4,
// 14 : 7 64.9, 10 : 5 65.6; 10 : 3 ... 10 : 10 all within 10 %).  Every tile a CTA starts costs a little for switching accumulators; a tile copy whose
// output is scattered keeps the epilogue warps busy for about as long as seven quantized groups keep
// the MMA threads.
constexpr int kPlanCostFp16 = 12, kPlanCostQuant = 7, kPlanCostTile = 1, kPlanCostScatterTile = 48;
// Pairs of CTAs: a quantized group costs each SM half the MMAs, but the measured layer step is again
// shortest near 10 : 7 (76 us; 85 us at 12 : 4, 90 us at 15 : 4) -- a pair is not bound by its bytes either.
constexpr int kPlanPairCostFp16 = 10, kPlanPairCostQuant = 7, kPlanPairCostTile = 1, kPlanPairCostScatterTile = 64;

// One piece of work of a CTA: groups [g_begin, g_end) of column tile `tile` of problem `prob`.
struct PlanSeg {
  int prob, tile, g_begin, g_end;
  int n_contrib;        // CTAs that hold groups of this tile (1: the tile is this CTA's alone)
  int contrib_idx;      // this CTA's position among them, ascending K
  int slot0;            // partial-tile slot of holder 0; holder i uses slot0 + i
  int counter;          // the tile's arrival counter
  int closer_idx;       // >= 0: this CTA adds the partial tiles for token rows closer_idx, + n_closers, ...
  int n_closers;
  int tok_begin, tok_end;   // token rows of y this piece writes when it finishes the tile (a whole tile: all)
};
static_assert(sizeof(PlanSeg) == 48, "three 16-byte loads per piece");

struct PlanGeom {
  int n_tiles, groups, g_fp16;
  int dep;              // index of the problem whose output this one reads, or -1
  int rep;              // >= 1: every tile is computed `rep` times, each copy writing 1/rep of the token rows
  int tile_cost;        // cost of starting a tile (copy) of this problem; 0: the default
};

struct PlanSchedule {
  std::vector<PlanGeom> geom;
  int cost[3];
  int n_ctas = 0, n_counters = 0, n_slots = 0;
  std::vector<PlanSeg> segs;          // per CTA, in processing order
  std::vector<int> seg_begin;         // [n_ctas + 1]
  std::vector<unsigned> done_target;  // per problem: finishing events that complete it
  PlanSeg *d_segs = nullptr;
  int *d_seg_begin = nullptr;
};

struct PlanOp {
  const __half *x;      // input activations (ignored when dep >= 0)
  long long ldx;
  int dep;              // >= 0: the input is the output of that earlier op
  const TiledOperand *t;
  const int32_t *col_map;
  __half *y;
  long long ldy;
  int m = 0;            // token rows of this op; 0: the plan's M
};

struct PlanLaunch {
  void *params = nullptr;   // kernel parameters (tensor maps, problem table), owned
  int n_ctas = 0, bits = 4;
  bool big = false;         // accumulators of 128 tokens (more than 64 tokens per operation)
  bool pair = false;        // clusters of two CTAs sharing an MMA stream
  size_t partial_bytes = 0;
};
}  // namespace rosaq

struct rosaq_ctx {
  int device;
  int sm_count;
  int *d_status;       // device status word (0 or ROSAQ_ERR_TIMEOUT)
  void *ws;            // rotated-activation workspace
  size_t ws_bytes;
  long long wait_limit;
  int impl;            // 0 tensor-core, 1 CUDA-core, 2 tensor-core with CTA pairs, 3 tensor-core without stream-K,
                       // 4 persistent launch for every call, 5 prefill tiles for every weight
  float *sk_partials;  // stream-K: fp32 partial tiles, [sk_ctas][2][64 tokens][128 columns]
  int *sk_arrive;      // stream-K: per-tile arrival counters, zero between launches
  int sk_ctas;         // CTAs the partial-tile workspace was sized for
  // persistent multi-problem launch
  int pl_ctas;                                   // CTAs of its grid, one per SM (0 until first asked for)
  int pl_pairs;                                  // clusters of two CTAs the device keeps resident at once
  int pl_mode;                                   // 0: pairs of CTAs where the operands allow, 1: single CTAs only
  int pl_cost[3];                                // cost of an fp16 group, a quantized group, a tile's epilogue ...
  int pl_cost_set;                               // ... when set through rosaq_set_plan_costs, else the defaults
  float *pl_partials;                            // partial tiles exchanged between CTAs; grown on demand
  size_t pl_partial_bytes;
  unsigned *pl_sync;                             // counters, zero between launches
  std::vector<rosaq::PlanSchedule *> pl_schedules;   // one per geometry seen, owned
  // prefill tiles (pairs of CTAs; the partial tiles of a launch live in pl_partials)
  int pf_pairs;                                  // pairs the device keeps resident at once (0 until first asked for)
  unsigned *pf_flags;                            // [pair][rank]: a partial tile is stored and not yet fetched; zero between launches
};

struct rosaq_weight {
  rosaq::TiledOperand t;
  int group, k_salient, device;
};

struct rosaq_plan {
  std::vector<rosaq::PlanOp> ops;
  int M, device;
  rosaq::PlanLaunch launch;
};

struct rosaq_rotation {
  rosaq::TiledOperand t;
  int32_t *col_map;    // device [d] or nullptr: rotated column p is stored at position col_map[p]
  int d, device;
};

namespace rosaq {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
    if (ok && prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (!ok) (void)cudaGetLastError();
  }
  ~DeviceGuard() {
    if (prev >= 0) (void)cudaSetDevice(prev);
  }
};

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// launchers implemented in the other translation units; all return a rosaq_status
int launch_rotate_weights(const void *q, int q_is_f32, int d_in, int n_blocks, const int32_t *perm,
                          const __half *W, int d_out, float *Wp, cudaStream_t s);
int launch_rotate_weights_w32(const void *q, int q_is_f32, int d_in, int n_blocks, const int32_t *perm,
                              const float *W32, int d_out, float *Wp, cudaStream_t s);
int launch_scale_rows(const __half *W, const float *in_scale, int d_in, int d_out, float *out, cudaStream_t s);
int launch_cast_weights(const __half *W, int d_in, int d_out, float *Wp, cudaStream_t s);
int launch_quant_pack(const float *Wp, const TiledOperand &t, cudaStream_t s);
int launch_export(const TiledOperand &t, uint32_t *qw, __half *scales, __half *zeros, __half *salient,
                  cudaStream_t s);
int launch_import(const TiledOperand &t, const uint32_t *qw, const __half *scales, const __half *zeros,
                  const __half *salient, cudaStream_t s);
int launch_rotation_tiles(const __half *q, int d, int n_blocks, const TiledOperand &t, cudaStream_t s);
int launch_invert_perm(const int32_t *perm, int d, int32_t *inv, int *bad, cudaStream_t s);
int launch_cov_fma(const void *X, int x_dtype, long long n_tokens, int d, long long ldx, int n_blocks, float *C,
                   cudaStream_t s);
int launch_cov(const rosaq_ctx *ctx, const void *X, int x_dtype, long long n_tokens, int d, long long ldx,
               int n_blocks, float *C, cudaStream_t s);
int launch_linear_simt(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t,
                       const int32_t *col_map, __half *y, long long ldy, cudaStream_t s);
int launch_linear_tc(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t,
                     const int32_t *col_map, __half *y, long long ldy, cudaStream_t s);
int launch_linear_tc_multi(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, int n,
                           const TiledOperand *const *ts, const int32_t *col_map, __half *const *ys,
                           const long long *ldys, cudaStream_t s);

bool prefill_supported(const TiledOperand &t, const int32_t *col_map);
int launch_linear_prefill(rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t, __half *y,
                          long long ldy, cudaStream_t s);

int plan_build_schedule(const std::vector<PlanGeom> &ops, int n_ctas, const int *cost, PlanSchedule *out);
int plan_ctas(rosaq_ctx *ctx);
int plan_units(rosaq_ctx *ctx, bool pair);
int plan_prepare(rosaq_ctx *ctx, int M, int n, const PlanOp *ops, PlanLaunch *out);
int plan_launch(rosaq_ctx *ctx, const PlanLaunch &l, cudaStream_t s);
void plan_release(PlanLaunch *l);
void plan_free_schedules(rosaq_ctx *ctx);

}  // namespace rosaq
