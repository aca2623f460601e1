// Eq. 4, left-hand side: the calibration Gram matrix C += X^T X.
//
// fp16 activations go to the tensor cores (tcgen05): the Gram matrix is a symmetric rank-N update,
// C[i][j] = sum_t X[t][i] X[t][j], so both MMA operands are slices of the same row-major X with
// the token index as the contraction dimension -- "MN-major" operands, which TMA delivers directly
// (box = 64 channels x 64 tokens, 128-byte swizzle) without any transposition.  One CTA owns one
// 128 x 256 tile (128 x 128 for blocks of at most 128 channels) of one head block and walks over all
// tokens of the call with fp32 accumulators in tensor memory.  Only tiles that touch the lower
// triangle are computed: with 128-row blocks bi and 256-column blocks bj those are bj <= bi / 2.
// A tile with bj == bi / 2 sits on the diagonal: its rows are a slice of its own columns, so it loads
// one operand and uses it twice, and every element of its 256 x 256 diagonal block is produced
// directly by it or its sibling.  The other tiles add themselves to C and their transpose to the
// mirrored position.  Both triangles are therefore written and C stays exactly symmetric.
//
// fp32 activations (and blocks narrower than 64 channels) keep the CUDA-core path of quantize.cu,
// whose products are exact.
//
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 = epilogue.
// Every wait is bounded (ROSAQ_ERR_TIMEOUT through the context's status word).
#include <cuda.h>

#include <mutex>

#include "rosaq_internal.cuh"

namespace rosaq {

namespace {

constexpr int kCovTile = 128;      // output tile rows (MMA M)
constexpr int kCovTokens = 64;     // tokens per pipeline stage
constexpr int kCovStages = 4;
constexpr int kCovThreads = 192;
constexpr int kBoxBytes = 64 * kCovTokens * 2;          // one TMA box: 64 channels x 64 tokens fp16
constexpr int kOperandBytes = 2 * kBoxBytes;            // 128 channels (operand A)
constexpr int kStageBytes = 6 * kBoxBytes;              // A (2 boxes) and up to 256 channels of B (4 boxes)
constexpr uint32_t kCovTmemCols = 256;
constexpr int kCovDrainPolls = 1 << 16;                 // for work in flight when a CTA gives up (not the context's limit)

struct CovParams {
  float *C;
  int dh, bn;                  // block edge; tile columns (MMA N): 256, or 128 for narrow blocks
  int use3d;                   // the 3-D maps are valid (channel count a multiple of 64)
  long long n_tokens;
  int *status;
  long long wait_limit;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(1000u)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// One instruction for several adjacent 64-channel blocks: the activations are also described as a 3-D
// tensor {64 channels, tokens, 64-channel block}, whose box {64, 64 tokens, n blocks} lands in shared memory
// block after block -- the MN-major operand as it is needed.  (Issuing a TMA costs the producer thread a
// few hundred cycles, so the number of instructions per stage matters.)
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int tok, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(bar), "r"(0), "r"(tok), "r"(blk)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// MN-major operand, 128-byte swizzle: 64-channel blocks kBoxBytes apart (leading offset), groups of
// 8 tokens 1024 bytes apart (stride offset).
__device__ __forceinline__ uint64_t make_mn_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr >> 4) & 0x3fff) | ((uint64_t)(kBoxBytes >> 4) << 16) | (64ull << 32) | (1ull << 46) |
         (2ull << 61);
}

// four MMAs = one stage of 64 tokens; descriptors advance by 16 tokens = 2048 bytes = 128 units of 16 bytes
__device__ __forceinline__ void tc_mma4_ss(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 ta, tb;\n\t"
      "setp.ne.b32 p, %4, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "add.u64 ta, %1, 128;\n\tadd.u64 tb, %2, 128;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], ta, tb, %3, q;\n\t"
      "add.u64 ta, %1, 256;\n\tadd.u64 tb, %2, 256;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], ta, tb, %3, q;\n\t"
      "add.u64 ta, %1, 384;\n\tadd.u64 tb, %2, 384;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], ta, tb, %3, q;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}

struct CovAbort {
  volatile int *flag;
  int *status;
  long long limit;
  __device__ __forceinline__ bool set() const { return *flag != 0; }
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait(bar, parity)) return true;
    for (long long it = 0; it < limit; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((it & 63) == 63 && set()) return false;
    }
    *flag = 1;
    atomicExch(status, (int)ROSAQ_ERR_TIMEOUT);
    return false;
  }
};

__global__ void __launch_bounds__(kCovThreads, 1)
cov_tc_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap map2,
              const __grid_constant__ CUtensorMap map4, const CovParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t bars[2 * kCovStages + 1];
  __shared__ uint32_t misc[2];                       // [0] TMEM base, [1] abort flag
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[kCovStages]);
  const uint32_t bar_d = smem_u32(&bars[2 * kCovStages]);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const CovAbort ab{reinterpret_cast<volatile int *>(&misc[1]), p.status, p.wait_limit};

  // row block bi (128 channels) has the column blocks bj = 0 .. bi / ratio (ratio = bn / 128)
  const int ratio = p.bn / kCovTile;
  int bi = 0, first = 0;
  while (first + bi / ratio + 1 <= (int)blockIdx.x) {
    first += bi / ratio + 1;
    ++bi;
  }
  const int bj = blockIdx.x - first;
  const int h = blockIdx.y;
  const bool diag = bj == bi / ratio;
  const int col_a = h * p.dh + bi * kCovTile, col_b = h * p.dh + bj * p.bn;
  const int b_boxes = p.bn / 64;
  // on a diagonal tile operand A is the slice of B that holds row block bi
  const uint32_t a_in_b = diag ? (uint32_t)((bi % ratio) * kOperandBytes) : 0u;
  const int n_stages_total = (int)((p.n_tokens + kCovTokens - 1) / kCovTokens);

  if (threadIdx.x == 0) {
    for (int i = 0; i < kCovStages; ++i) {
      mbar_init(bar_full + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_d, 1);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc[0])),
                 "n"(kCovTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc[0];

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0, idx = 0;
      uint32_t lap = 0;
      for (int s = 0; s < n_stages_total && !ab.set(); ++s, ++issued) {
        if (!ab.wait(bar_empty + 8 * idx, lap ^ 1u)) break;
        const uint32_t dst = base + idx * kStageBytes;
        const int tok = s * kCovTokens;
        mbar_arrive_expect_tx(bar_full + 8 * idx, (uint32_t)((diag ? 0 : 2) + b_boxes) * kBoxBytes);
        if (p.use3d) {
          if (!diag) tma_load_3d(dst, &map2, bar_full + 8 * idx, tok, col_a >> 6);
          tma_load_3d(dst + kOperandBytes, b_boxes == 4 ? &map4 : &map2, bar_full + 8 * idx, tok, col_b >> 6);
        } else {
          if (!diag) {
            tma_load_2d(dst, &xmap, bar_full + 8 * idx, col_a, tok);
            tma_load_2d(dst + kBoxBytes, &xmap, bar_full + 8 * idx, col_a + 64, tok);
          }
          for (int b = 0; b < b_boxes; ++b)
            tma_load_2d(dst + kOperandBytes + b * kBoxBytes, &xmap, bar_full + 8 * idx, col_b + 64 * b, tok);
        }
        if (++idx == kCovStages) idx = 0, lap ^= 1u;
      }
      if (ab.set()) {  // let loads already in flight land before the CTA goes away
        for (int back = 1; back <= kCovStages && back <= issued; ++back) {
          const int u = issued - back;
          for (int it = 0; it < kCovDrainPolls; ++it)
            if (mbar_try_wait(bar_full + 8 * (u % kCovStages), (u / kCovStages) & 1)) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // fp16 x fp16 -> fp32, both operands MN-major, M = 128, N = bn
      const uint32_t idesc = (1u << 4) | (1u << 15) | (1u << 16) | ((uint32_t)(p.bn >> 3) << 17) |
                             ((uint32_t)(kCovTile >> 4) << 24);
      int idx = 0;
      uint32_t lap = 0, accumulate = 0;
      for (int s = 0; s < n_stages_total; ++s) {
        if (!ab.wait(bar_full + 8 * idx, lap)) break;
        tc_fence_after();
        const uint32_t b_addr = base + idx * kStageBytes + kOperandBytes;
        const uint64_t b = make_mn_desc(b_addr);
        const uint64_t a = make_mn_desc(diag ? b_addr + a_in_b : b_addr - kOperandBytes);
        tc_mma4_ss(tmem, a, b, idesc, accumulate);
        accumulate = 1;
        tc_commit(bar_empty + 8 * idx);
        if (++idx == kCovStages) idx = 0, lap ^= 1u;
      }
      tc_commit(bar_d);
      if (ab.set()) {  // MMAs already issued must retire before the tensor memory is given back
        for (int it = 0; it < kCovDrainPolls; ++it)
          if (mbar_try_wait(bar_d, 0)) break;
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> shared (transposable staging) -> C += tile, C^T += tile^T
    const int quad = warp & 3;                        // warps 2..5 cover the four lane quadrants
    const int row = quad * 32 + lane;                 // tile row i = TMEM lane
    bool have = ab.wait(bar_d, 0);
    have = __all_sync(0xffffffffu, have && !ab.set());
    float *stage = reinterpret_cast<float *>(gen);    // [128][bn + 1] fp32, reuses the operand ring
    const int pitch = p.bn + 1;
    if (have) {
      tc_fence_after();
      const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
      for (int c0 = 0; c0 < p.bn; c0 += 8) {
        uint32_t v[8];
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(lane_addr + c0)
                     : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int e = 0; e < 8; ++e) stage[row * pitch + c0 + e] = __uint_as_float(v[e]);
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");    // the four epilogue warps
    if (!ab.set()) {
      const int tid = threadIdx.x - 64;               // 0..127
      float *Cb = p.C + (long long)h * p.dh * p.dh;
      const int i0 = bi * kCovTile, j0 = bj * p.bn;
      // C[i0 + r][j0 + c] += tile[r][c]: a warp touches 32 consecutive floats of one row of C
      // The update of C is latency-bound (read-modify-write through L2), so each thread keeps eight
      // independent 16-byte loads in flight.  Direct part: C[i0 + r][j0 + 4 q .. + 3] += tile[r][4 q .. + 3].
      const int n_rows = min(kCovTile, p.dh - i0), n_cols = min(p.bn, p.dh - j0);   // both multiples of 8
      {
        const int quads = p.bn >> 2, sets = 128 / quads;   // 64 x 2 or 32 x 4 (column quads x interleaved row sets)
        const int q = tid % quads, r_first = tid / quads;
        if (4 * q < n_cols) {
          float *dst = Cb + (long long)i0 * p.dh + j0 + 4 * q;
          for (int r0 = r_first; r0 < n_rows; r0 += 8 * sets) {
            float4 old[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int r = r0 + sets * e;
              old[e] = r < n_rows ? __ldcg(reinterpret_cast<const float4 *>(dst + (long long)r * p.dh))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int r = r0 + sets * e;
              if (r < n_rows) {
                const float *t = stage + r * pitch + 4 * q;
                *reinterpret_cast<float4 *>(dst + (long long)r * p.dh) =
                    make_float4(__fadd_rn(old[e].x, t[0]), __fadd_rn(old[e].y, t[1]), __fadd_rn(old[e].z, t[2]),
                                __fadd_rn(old[e].w, t[3]));
              }
            }
          }
        }
      }
      // mirror: C[j0 + c][i0 + 4 q .. + 3] += tile[4 q .. + 3][c]
      if (!diag) {
        const int q = tid & 31, c_first = tid >> 5;       // 32 row quads of the tile x 4 interleaved column sets
        if (4 * q < n_rows) {
          float *dst = Cb + (long long)j0 * p.dh + i0 + 4 * q;
          for (int c0 = c_first; c0 < n_cols; c0 += 32) {
            float4 old[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = c0 + 4 * e;
              old[e] = c < n_cols ? __ldcg(reinterpret_cast<const float4 *>(dst + (long long)c * p.dh))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = c0 + 4 * e;
              if (c < n_cols) {
                const float *t = stage + (4 * q) * pitch + c;
                *reinterpret_cast<float4 *>(dst + (long long)c * p.dh) =
                    make_float4(__fadd_rn(old[e].x, t[0]), __fadd_rn(old[e].y, t[pitch]), __fadd_rn(old[e].z, t[2 * pitch]),
                                __fadd_rn(old[e].w, t[3 * pitch]));
              }
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kCovTmemCols) : "memory");
  }
}

// =====================================================================================
// Paired variant for wide blocks: two CTAs of a cluster (two SMs) share one 256 x 256 tile and one
// MMA stream (tcgen05 cta_group::2).  CTA r of the pair owns rows [128 r, 128 r + 128) of the tile
// (operand A and the accumulator in its own tensor memory) and supplies columns [128 r, 128 r + 128)
// of operand B from its own shared memory; the leader (rank 0) issues M = 256, N = 256 MMAs for both.
// Per 64 tokens a CTA loads 32 KB instead of 48 KB and they last 1024 MMA cycles instead of 476, so
// the six stages of the ring cover the TMA latency and the L2 traffic halves.  On a diagonal tile a
// CTA's rows are its own column half: it loads one block and uses it as both operands.
// Handshakes: the loads of both CTAs count their bytes on the leader's barrier (cta_group::2 loads, no
// multicast); the leader's commits are multicast to both CTAs (stage free, accumulator ready).
// =====================================================================================
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * kOperandBytes;      // A rows (or nothing on a diagonal tile) + this CTA's half of B

__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(1000u)
      : "memory");
  return ok != 0;
}
// Loads of a CTA pair: the data lands in the issuing CTA's shared memory, the bytes are counted on the
// leader's barrier (a shared::cluster address), so the leader learns about both halves from one barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t lead_bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(lead_bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *map, uint32_t lead_bar, int tok, int blk) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::
          "r"(dst),
      "l"(map), "r"(lead_bar), "r"(0), "r"(tok), "r"(blk)
      : "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"((unsigned short)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma4_ss_pair(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b64 ta, tb;\n\t"
      "setp.ne.b32 p, %4, 0;\n\tsetp.eq.b32 q, 0, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "add.u64 ta, %1, 128;\n\tadd.u64 tb, %2, 128;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], ta, tb, %3, q;\n\t"
      "add.u64 ta, %1, 256;\n\tadd.u64 tb, %2, 256;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], ta, tb, %3, q;\n\t"
      "add.u64 ta, %1, 384;\n\tadd.u64 tb, %2, 384;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], ta, tb, %3, q;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}

struct PairAbort {
  volatile int *flag;
  int *status;
  long long limit;
  __device__ __forceinline__ bool set() const { return *flag != 0; }
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    for (long long it = 0; it < limit; ++it) {
      if (mbar_try_wait_cluster(bar, parity)) return true;
      if ((it & 63) == 63 && set()) return false;
    }
    *flag = 1;
    atomicExch(status, (int)ROSAQ_ERR_TIMEOUT);
    return false;
  }
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kCovThreads, 1)
cov_tc_pair_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap map2,
                   const CovParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ uint64_t bars[2 * kPairStages + 1];
  __shared__ uint32_t misc[2];                       // [0] TMEM base, [1] abort flag
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_tma = smem_u32(&bars[0]);                       // leader's copy: both CTAs' loads of a stage landed
  const uint32_t bar_empty = smem_u32(&bars[kPairStages]);           // stage free again (multicast commit)
  const uint32_t bar_d = smem_u32(&bars[2 * kPairStages]);           // accumulators final (multicast commit)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const PairAbort ab{reinterpret_cast<volatile int *>(&misc[1]), p.status, p.wait_limit};

  // 256 x 256 tile (bi >= bj) of the lower triangle from the pair index bi (bi + 1) / 2 + bj
  const int pair = blockIdx.x >> 1;
  int bi = 0;
  while ((bi + 1) * (bi + 2) / 2 <= pair) ++bi;
  const int bj = pair - bi * (bi + 1) / 2;
  const int h = blockIdx.y;
  const bool diag = bi == bj;
  const int i0 = bi * 256 + (int)rank * kCovTile, j0 = bj * 256;
  const int col_a = h * p.dh + i0, col_b = h * p.dh + j0 + (int)rank * kCovTile;
  const int n_stages_total = (int)((p.n_tokens + kCovTokens - 1) / kCovTokens);

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPairStages; ++i) {
      mbar_init(bar_tma + 8 * i, 1);
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_d, 1);
    misc[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {   // both CTAs of the pair allocate together, from the same warp index
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&misc[0])),
                 "n"(kCovTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // the peer's barriers and tensor memory exist
  tc_fence_after();
  const uint32_t tmem = misc[0];

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t lead_tma = map_to_rank(bar_tma, 0);     // the leader's barriers, as cluster addresses
      const uint32_t stage_bytes = diag ? kOperandBytes : kPairStageBytes;
      int issued = 0, idx = 0;
      uint32_t lap = 0;
      for (int s = 0; s < n_stages_total && !ab.set(); ++s, ++issued) {
        if (!ab.wait(bar_empty + 8 * idx, lap ^ 1u)) break;
        const uint32_t dst = base + idx * kPairStageBytes;
        const int tok = s * kCovTokens;
        if (rank == 0) mbar_arrive_expect_tx(bar_tma + 8 * idx, 2 * stage_bytes);   // both CTAs' bytes
        const uint32_t lb = lead_tma + 8 * idx;
        if (p.use3d) {
          if (!diag) tma_load_3d_pair(dst, &map2, lb, tok, col_a >> 6);
          tma_load_3d_pair(dst + kOperandBytes, &map2, lb, tok, col_b >> 6);
        } else {
          if (!diag) {
            tma_load_2d_pair(dst, &xmap, lb, col_a, tok);
            tma_load_2d_pair(dst + kBoxBytes, &xmap, lb, col_a + 64, tok);
          }
          tma_load_2d_pair(dst + kOperandBytes, &xmap, lb, col_b, tok);
          tma_load_2d_pair(dst + kOperandBytes + kBoxBytes, &xmap, lb, col_b + 64, tok);
        }
        if (++idx == kPairStages) idx = 0, lap ^= 1u;
      }
      // On a timeout the leader lets the loads of both CTAs land (they are all counted on its barriers)
      // before the final cluster barrier releases the pair; phases whose expectation it never posted
      // cannot complete and are bounded by the drain limit.
      if (ab.set() && rank == 0) {
        for (int back = 1; back <= kPairStages && back <= issued; ++back) {
          const int u = issued - back;
          for (int it = 0; it < kCovDrainPolls; ++it)
            if (mbar_try_wait_cluster(bar_tma + 8 * (u % kPairStages), (u / kPairStages) & 1)) break;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // leader: fp16 x fp16 -> fp32, both operands MN-major, M = 256 (128 rows per CTA), N = 256
      const uint32_t idesc = (1u << 4) | (1u << 15) | (1u << 16) | ((uint32_t)(256 >> 3) << 17) |
                             ((uint32_t)(256 >> 4) << 24);
      int idx = 0;
      uint32_t lap = 0, accumulate = 0;
      for (int s = 0; s < n_stages_total; ++s) {
        if (!ab.wait(bar_tma + 8 * idx, lap)) break;
        tc_fence_after();
        const uint32_t b_addr = base + idx * kPairStageBytes + kOperandBytes;
        const uint64_t b = make_mn_desc(b_addr);
        const uint64_t a = diag ? b : make_mn_desc(b_addr - kOperandBytes);
        tc_mma4_ss_pair(tmem, a, b, idesc, accumulate);
        accumulate = 1;
        tc_commit_pair(bar_empty + 8 * idx);
        if (++idx == kPairStages) idx = 0, lap ^= 1u;
      }
      tc_commit_pair(bar_d);
      if (ab.set()) {  // MMAs already issued must retire before the tensor memory is given back
        for (int it = 0; it < kCovDrainPolls; ++it)
          if (mbar_try_wait_cluster(bar_d, 0)) break;
      }
    }
  } else {
    // ---------------- epilogue: this CTA's 128 rows x 256 columns, as in the single-CTA kernel
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    bool have = ab.wait(bar_d, 0);
    have = __all_sync(0xffffffffu, have && !ab.set());
    float *stage = reinterpret_cast<float *>(gen);    // [128][257] fp32, reuses the operand ring
    constexpr int pitch = 257;
    if (have) {
      tc_fence_after();
      const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
      for (int c0 = 0; c0 < 256; c0 += 8) {
        uint32_t v[8];
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                     : "r"(lane_addr + c0)
                     : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int e = 0; e < 8; ++e) stage[row * pitch + c0 + e] = __uint_as_float(v[e]);
      }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");    // the four epilogue warps
    if (!ab.set() && i0 < p.dh) {
      const int tid = threadIdx.x - 64;               // 0..127
      float *Cb = p.C + (long long)h * p.dh * p.dh;
      const int n_rows = min(kCovTile, p.dh - i0), n_cols = min(256, p.dh - j0);   // both multiples of 8
      // The update of C is latency-bound (read-modify-write through L2), so each thread keeps eight
      // independent 16-byte loads in flight.  Direct part: C[i0 + r][j0 + 4 q .. + 3] += tile[r][4 q .. + 3].
      {
        const int q = tid & 63, r_first = tid >> 6;       // 64 column quads x 2 interleaved row sets
        if (4 * q < n_cols) {
          float *dst = Cb + (long long)i0 * p.dh + j0 + 4 * q;
          for (int r0 = r_first; r0 < n_rows; r0 += 16) {
            float4 old[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int r = r0 + 2 * e;
              old[e] = r < n_rows ? __ldcg(reinterpret_cast<const float4 *>(dst + (long long)r * p.dh))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int r = r0 + 2 * e;
              if (r < n_rows) {
                const float *t = stage + r * pitch + 4 * q;
                *reinterpret_cast<float4 *>(dst + (long long)r * p.dh) =
                    make_float4(__fadd_rn(old[e].x, t[0]), __fadd_rn(old[e].y, t[1]), __fadd_rn(old[e].z, t[2]),
                                __fadd_rn(old[e].w, t[3]));
              }
            }
          }
        }
      }
      // mirror: C[j0 + c][i0 + 4 q .. + 3] += tile[4 q .. + 3][c]
      if (!diag) {
        const int q = tid & 31, c_first = tid >> 5;       // 32 row quads of the tile x 4 interleaved column sets
        if (4 * q < n_rows) {
          float *dst = Cb + (long long)j0 * p.dh + i0 + 4 * q;
          for (int c0 = c_first; c0 < n_cols; c0 += 32) {
            float4 old[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = c0 + 4 * e;
              old[e] = c < n_cols ? __ldcg(reinterpret_cast<const float4 *>(dst + (long long)c * p.dh))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const int c = c0 + 4 * e;
              if (c < n_cols) {
                const float *t = stage + (4 * q) * pitch + c;
                *reinterpret_cast<float4 *>(dst + (long long)c * p.dh) =
                    make_float4(__fadd_rn(old[e].x, t[0]), __fadd_rn(old[e].y, t[pitch]), __fadd_rn(old[e].z, t[2 * pitch]),
                                __fadd_rn(old[e].w, t[3 * pitch]));
              }
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                // neither CTA leaves while the pair's MMAs may touch it
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(kCovTmemCols) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn cov_encode_fn() {
  static const EncodeTiledFn fn = [] {                       // initialised once, thread-safe
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(sym);
    (void)cudaGetLastError();
    return static_cast<EncodeTiledFn>(nullptr);
  }();
  return fn;
}

}  // namespace

int launch_cov(const rosaq_ctx *ctx, const void *X, int x_dtype, long long n_tokens, int d, long long ldx, int n_blocks,
               float *C, cudaStream_t s) {
  const int dh = d / n_blocks;
  EncodeTiledFn encode = cov_encode_fn();
  if (x_dtype != ROSAQ_F16 || dh < 64 || !encode || n_tokens > 0x7fffffffll)
    return launch_cov_fma(X, x_dtype, n_tokens, d, ldx, n_blocks, C, s);

  CUtensorMap xmap;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)n_tokens};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * sizeof(__half)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kCovTokens};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return ROSAQ_ERR_CUDA;
  }
  // 3-D views {64 channels, tokens, 64-channel block} with boxes of 2 and 4 blocks; only when every block
  // is whole (a partial last block would make the last row's box run past the end of the matrix)
  CUtensorMap map2 = xmap, map4 = xmap;
  const bool use3d = d % 64 == 0;
  if (use3d) {
    const cuuint64_t dims3[3] = {64, (cuuint64_t)n_tokens, (cuuint64_t)(d / 64)};
    const cuuint64_t strides3[2] = {(cuuint64_t)ldx * sizeof(__half), 128};
    const cuuint32_t estr3[3] = {1, 1, 1};
    for (int nb = 2; nb <= 4; nb += 2) {
      const cuuint32_t box3[3] = {64, (cuuint32_t)kCovTokens, (cuuint32_t)nb};
      CUresult r = encode(nb == 2 ? &map2 : &map4, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(X), dims3,
                          strides3, box3, estr3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return ROSAQ_ERR_CUDA;
    }
  }
  CovParams p{};
  p.use3d = use3d ? 1 : 0;
  p.C = C;
  p.dh = dh;
  p.bn = dh > kCovTile ? 256 : 128;
  p.n_tokens = n_tokens;
  p.status = ctx->d_status;
  p.wait_limit = ctx->wait_limit;
  const size_t smem = 1024 + (size_t)kCovStages * kStageBytes;   // the 128 x (bn + 1) fp32 staging tile fits inside
  static bool attr_done_all[64] = {};                    // function attributes are per device
  if (ctx->device < 0 || ctx->device >= 64) return ROSAQ_ERR_INVALID_ARG;
  bool &attr_done = attr_done_all[ctx->device];
  static std::mutex attr_mutex;                          // contexts of several host threads share this cache
  std::lock_guard<std::mutex> attr_lock(attr_mutex);
  if (!attr_done) {
    if (cudaFuncSetAttribute(cov_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_CUDA;
    }
    attr_done = true;
  }
  const int n_row_blocks = (dh + kCovTile - 1) / kCovTile, ratio = p.bn / kCovTile;
  int tiles = 0;
  for (int bi = 0; bi < n_row_blocks; ++bi) tiles += bi / ratio + 1;
  if (dh >= 512) {
    // wide blocks: 256 x 256 tiles on CTA pairs
    const size_t smem2 = 1024 + (size_t)kPairStages * kPairStageBytes;
    static bool attr2_done_all[64] = {};
    bool &attr2_done = attr2_done_all[ctx->device];
    if (!attr2_done) {
      if (cudaFuncSetAttribute(cov_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess) {
        (void)cudaGetLastError();
        return ROSAQ_ERR_CUDA;
      }
      attr2_done = true;
    }
    const int nb2 = (dh + 255) / 256;
    dim3 grid2(2 * (nb2 * (nb2 + 1) / 2), n_blocks);
    cov_tc_pair_kernel<<<grid2, kCovThreads, smem2, s>>>(xmap, map2, p);
    return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
  }
  dim3 grid(tiles, n_blocks);
  cov_tc_kernel<<<grid, kCovThreads, smem, s>>>(xmap, map2, map4, p);
  return cudaGetLastError() == cudaSuccess ? ROSAQ_OK : ROSAQ_ERR_CUDA;
}

}  // namespace rosaq
