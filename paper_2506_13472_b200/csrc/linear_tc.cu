// Tensor-core implementation of the GEMM stage  y = x' . W^  (Eq. 3; Eq. 6 for a block-diagonal
// rotation operand) for sm_100a: tcgen05.mma with the weight operand dequantised in registers
// and fed from tensor memory.
//
// Mapping.  The MMA computes D[n][m] = sum_k A[n][k] * B[m][k] with
//   A = one 128-column tile of the weights (MMA-M = 128 output columns), written to TMEM by the
//       dequantisation warps (lane = output column, one 32-bit TMEM column = the fp16 pair (2k,2k+1)),
//   B = the activations x' [tokens][k], K-major in shared memory with the 128-byte swizzle, loaded by
//       TMA straight from the caller's row-major matrix (rows past M are zero-filled by the copy),
//   D = fp32 accumulators in TMEM (128 lanes x tokens columns).
// So the big operand is streamed exactly once, 128-bit coalesced, and never touches shared memory
// in dequantised form.
//
// A CTA owns one column tile (blockIdx.x), one token tile of up to 128 tokens (blockIdx.z) and one
// contiguous range of 128-channel groups (blockIdx.y = its rank in a thread-block cluster that
// splits K).  Warp roles: 0 = weight-tile producer (bulk copies of whole tile blobs), 1 = activation
// producer (TMA), 2 = MMA issuer and TMEM owner, 3..10 = dequantisation, then epilogue.  The split-K
// partial sums are exchanged through distributed shared memory and added in rank order, so the
// result does not depend on timing.
//
// Every wait is bounded: when a limit expires the CTA records ROSAQ_ERR_TIMEOUT in the context's
// status word, stops issuing work, still joins the cluster barriers, frees its TMEM and returns.
#include <cuda.h>

#include <mutex>

#include "linear_common.cuh"

namespace rosaq {

namespace {

constexpr int kThreads = 352;
constexpr int kDequantThreads = 256;
constexpr int kFirstDequantWarp = 3;
constexpr int kTmemCols = 256;
constexpr int kMaxDevices = 64;
constexpr int kMaxProblems = 4;   // weights sharing one activation in a launch (q/k/v, gate/up)
constexpr int kMaxSplits = 8;
// Relative cost of a group when work is divided: an fp16 group is 3.7 times the bytes of an INT4 group,
// but up to 64 tokens a CTA is paced by its eight MMAs and its handshakes per group, not by bytes
// (measured: weights 4 : 1 lose 2-5 % against 1.5 : 1 on the 7B shapes).
constexpr int kCostFp16 = 3, kCostQuant = 2;

struct TcParams {
  // up to kMaxProblems weights of identical geometry (d_in, bits, salient groups) that multiply the same
  // activations: their column tiles are laid side by side along gridDim.x
  int n_prob;
  int tile_start[kMaxProblems + 1];
  const uint8_t *blob[kMaxProblems];
  int d_out[kMaxProblems];
  __half *y[kMaxProblems];
  long long ldy[kMaxProblems];
  long long tile_stride;
  int g_fp16, g_quant, bits, block_groups;
  int M, MT;                 // tokens in the problem, tokens per CTA (multiple of 16, <= 128)
  int S;                     // K splits = cluster size along y
  int g_bounds[kMaxSplits + 1];
  const int32_t *col_map;
  int *status;
  long long wait_limit;
  int NW, NA;                // ring depths: packed-weight slots, stages (TMEM A buffer + activation slot)
};


// kPair: two CTAs with adjacent column tiles (cluster ranks 2j, 2j + 1; blockIdx.x even / odd) run as a
// cta_group::2 pair.  Each dequantises its own 128 columns into its own tensor memory and loads half of
// the token rows; the leader (even rank) issues one M = 256 MMA for both, so the per-SM cost of issuing
// MMAs -- the bound of the single-CTA kernel at small token counts -- halves.
template <int kBits, bool kPair>
__global__ void __launch_bounds__(kThreads, 2)
linear_tc_kernel(const __grid_constant__ CUtensorMap xmap, const TcParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // carve-up (the dynamic window is 1024-byte aligned by the launch code's padding)
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int MT = p.MT;
  const int MTL = kPair ? MT >> 1 : MT;                        // token rows this CTA keeps in shared memory
  const uint32_t x_slot_bytes = (uint32_t)MTL * 256u;
  const uint32_t x_ring = base;                                // NA slots: one per TMEM operand buffer
  const uint32_t w_ring = x_ring + p.NA * x_slot_bytes;
  const uint32_t bars = w_ring + p.NW * kWSlotBytes;          // 8-byte aligned (all sizes multiples of 16)
  const uint32_t bar_w_full = bars, bar_w_empty = bar_w_full + 8 * p.NW;
  const uint32_t bar_x_full = bar_w_empty + 8 * p.NW, bar_a_full = bar_x_full + 8 * p.NA;
  const uint32_t bar_empty = bar_a_full + 8 * p.NA;           // stage (operand buffer + activation slot) free again
  const uint32_t bar_d_full = bar_empty + 8 * p.NA;
  const uint32_t misc = bar_d_full + 8;                        // [0] TMEM base, [1] abort flag
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t *misc_ptr = reinterpret_cast<volatile uint32_t *>(gen + (misc - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int prob = 0;
  while (prob + 1 < p.n_prob && (int)blockIdx.x >= p.tile_start[prob + 1]) ++prob;
  const int nt = blockIdx.x - p.tile_start[prob], split = blockIdx.y, m0 = blockIdx.z * MT;
  const int d_out = p.d_out[prob];
  __half *const y_out = p.y[prob];
  const long long ldy = p.ldy[prob];
  const int g_begin = p.g_bounds[split], g_end = p.g_bounds[split + 1];
  const Abort ab{reinterpret_cast<volatile int *>(misc_ptr + 1), p.status, p.wait_limit, kPair};
  const uint32_t pair_x = kPair ? (blockIdx.x & 1u) : 0u;      // 0 = leader of the pair
  const uint32_t lead_rank = kPair ? 2u * (uint32_t)split : 0u;   // cluster rank of this pair's leader
  const bool is_lead = pair_x == 0;
  const int n_arrive = kPair ? 2 * (kTeamThreads / 32) : kTeamThreads;   // arrivals that complete an a_full phase

  // Let the next kernel of the stream start its own prologue and weight prefetch while this one runs
  // (it only matters when the launches are chained programmatically; otherwise a no-op).
  grid_dep_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.NW; ++i) {
      mbar_init(bar_w_full + 8 * i, 1);
      mbar_init(bar_w_empty + 8 * i, kTeamThreads);
    }
    for (int i = 0; i < p.NA; ++i) {
      mbar_init(bar_x_full + 8 * i, 1);
      mbar_init(bar_a_full + 8 * i, kPair ? n_arrive : n_arrive + 1);   // + the activation copy (single-CTA mode)
      mbar_init(bar_empty + 8 * i, 1);
    }
    mbar_init(bar_d_full, 1);
    misc_ptr[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {
    if (kPair) tmem_alloc_pair<kTmemCols>(misc);             // both CTAs of the pair, same warp index
    else tmem_alloc<kTmemCols>(misc);
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) {                                               // the peer's barriers and tensor memory exist
    cluster_arrive();
    cluster_wait();
  }
  tc_fence_after();
  const uint32_t tmem = misc_ptr[0];
  const uint32_t a_col0 = (MT <= 64) ? 64u : 128u;             // A buffers follow the accumulator columns

  const uint8_t *tile_base = p.blob[prob] + (long long)nt * p.tile_stride;
  const int qbytes = quant_tile_bytes(kBits);

  if (warp == 0) {
    // ---------------- weight-tile producer (weights never depend on the previous kernel: no grid wait)
    if (lane == 0) {
      int uc = 0;
      Ring rw{0, 0};
      for (int g = g_begin; g < g_end && !ab.set(); ++g) {
        const bool f16 = g < p.g_fp16;
        const uint8_t *src = tile_base + (f16 ? (long long)g * kFp16TileBytes
                                              : (long long)p.g_fp16 * kFp16TileBytes + (long long)(g - p.g_fp16) * qbytes);
        const int nsub = f16 ? 4 : 1;
        const uint32_t bytes = f16 ? kFp16SubBytes : qbytes;
        for (int sub = 0; sub < nsub; ++sub, ++uc, rw.advance(p.NW)) {
          const int slot = rw.idx;
          if (!ab.wait_local(bar_w_empty + 8 * slot, rw.lap ^ 1u)) break;
          mbar_arrive_expect_tx(bar_w_full + 8 * slot, bytes);
          bulk_copy_g2s(w_ring + slot * kWSlotBytes, src + (long long)sub * kFp16SubBytes, bytes, bar_w_full + 8 * slot);
        }
      }
      if (ab.set()) {  // let copies already in flight land before the CTA goes away
        for (int back = 1; back <= p.NW && back <= uc; ++back) {
          const int u = uc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (mbar_try_wait(bar_w_full + 8 * (u % p.NW), (u / p.NW) & 1)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- activation producer
    if (lane == 0) {
      grid_dep_wait();                                         // x may be the previous kernel's output
      int gc = 0;
      Ring rs{0, 0};
      // block-diagonal operand: column tile nt only multiplies the channels of its own diagonal block
      const int g_block0 = p.block_groups > 0 ? (nt / p.block_groups) * p.block_groups : 0;
      for (int g = g_begin; g < g_end && !ab.set(); ++g, ++gc, rs.advance(p.NA)) {
        const int slot = rs.idx;
        if (!ab.wait(bar_empty + 8 * slot, rs.lap ^ 1u)) break;
        const int k0 = (g_block0 + g) * kGroup;
        if (kPair) {
          // each CTA loads its half of the token rows; all bytes are counted on the leader's barrier
          if (is_lead) mbar_arrive_expect_tx(bar_x_full + 8 * slot, 2 * x_slot_bytes);
          const uint32_t lb = map_to_rank(bar_x_full + 8 * slot, lead_rank);
          const int mrow = m0 + (int)pair_x * MTL;
          tma_load_2d_pair(x_ring + slot * x_slot_bytes, &xmap, lb, k0, mrow);
          tma_load_2d_pair(x_ring + slot * x_slot_bytes + MTL * 128, &xmap, lb, k0 + 64, mrow);
        } else {
          // the copy completes on the stage's operand barrier: the MMA thread then polls one barrier per group
          mbar_arrive_expect_tx(bar_a_full + 8 * slot, x_slot_bytes);
          tma_load_3d(x_ring + slot * x_slot_bytes, &xmap, bar_a_full + 8 * slot, m0, k0 >> 6);
        }
      }
      // (in a pair the leader's barriers count the loads of both CTAs, and the peer stays until the
      // cluster barrier at the end of the kernel, which the leader reaches after this drain)
      if (ab.set() && is_lead) {
        const uint32_t bar_copy = kPair ? bar_x_full : bar_a_full;
        for (int back = 1; back <= p.NA && back <= gc; ++back) {
          const int u = gc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (ab.poll(bar_copy + 8 * (u % p.NA), (u / p.NA) & 1)) break;
        }
      }
    }
  } else if (warp == 2) {
    // ---------------- MMA issuer: per group one wait pair, eight MMAs, one commit
    if (lane == 0 && is_lead) {
      // M = 128 output columns (256 for a pair), N = MT tokens
      const uint32_t idesc = (1u << 4) | ((uint32_t)(MT >> 3) << 17) | ((kPair ? 16u : 8u) << 24);
      const uint32_t pair_mask = 3u << lead_rank;            // the two CTAs of the pair, for multicast commits
      const uint64_t desc0 = make_b_desc(x_ring);            // descriptor address fields are in 16-byte units
      const uint32_t x_slot16 = x_slot_bytes >> 4, half16 = (uint32_t)(MTL * 128) >> 4;
      Ring rs{0, 0};
      uint32_t accumulate = 0;
      for (int g = g_begin; g < g_end; ++g, rs.advance(p.NA)) {
        const int st = rs.idx;
        if ((kPair && !ab.wait(bar_x_full + 8 * st, rs.lap)) || !ab.wait(bar_a_full + 8 * st, rs.lap)) break;
        tc_fence_after();
        const uint64_t b0 = desc0 + (uint64_t)(st * x_slot16);
        if (kPair) {
          tc_mma8_ts_pair(tmem, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
          tc_commit_mc(bar_empty + 8 * st, pair_mask);
        } else {
          tc_mma8_ts(tmem, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
          tc_commit(bar_empty + 8 * st);
        }
        accumulate = 1;
      }
      if (kPair) tc_commit_mc(bar_d_full, pair_mask);
      else tc_commit(bar_d_full);
      if (ab.set()) {  // MMAs already issued must retire before the tensor memory is given back
        for (int it = 0; it < kDrainPolls; ++it)
          if (ab.poll(bar_d_full, 0)) break;
      }
    }
  } else {
    // ---------------- dequantisation warps: shared memory -> registers -> TMEM
    // Two teams of four warps (one warp per TMEM lane quadrant) take alternate groups, so that the
    // waits, the TMEM store drain and the barrier traffic of one team run under the arithmetic of the
    // other; a thread dequantises all 128 input channels of its output column.
    const int dq = warp - kFirstDequantWarp;       // 0..7
    const int quad = warp & 3;                     // TMEM lane quadrant this warp may touch
    const int team = dq >> 2;
    const int n = quad * 32 + lane;                // output column inside the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    Ring rw{0, 0}, rs{0, 0};
    bool ok = true;
    for (int g = g_begin; g < g_end && ok; ++g, rs.advance(p.NA)) {
      const bool f16 = g < p.g_fp16;
      const int nsub = f16 ? 4 : 1;
      if (((g - g_begin) & 1) != team) {           // the other team's group: only keep the ring positions
        for (int sub = 0; sub < nsub; ++sub) rw.advance(p.NW);
        continue;
      }
      const int st = rs.idx;
      const uint32_t a_addr = lane_addr + a_col0 + st * 64;
      bool got = kPair ? ab.wait_warp(bar_empty + 8 * st, rs.lap ^ 1u) : ab.wait(bar_empty + 8 * st, rs.lap ^ 1u);
      for (int sub = 0; sub < nsub && ok; ++sub, rw.advance(p.NW)) {
        const int slot = rw.idx;
        // A parity wait must not be a whole phase early.  The previous fill of this slot may belong to
        // the other team, which can lag by a group: first see that fill released (the same phase the
        // producer waits for), only then wait for the new one.
        got = got && ab.wait_local(bar_w_empty + 8 * slot, rw.lap ^ 1u) && ab.wait_local(bar_w_full + 8 * slot, rw.lap);
        got = __all_sync(0xffffffffu, got);        // the TMEM instructions below need the whole warp
        if (!got) {
          ok = false;
          break;
        }
        tc_fence_after();
        dequant_unit<kBits>(f16, w_ring + slot * kWSlotBytes, n, a_addr, sub, bar_w_empty + 8 * slot);
      }
      if (!ok) {
        tc_wait_st();                              // stores of earlier slices of this group
        break;
      }
      tc_wait_st();
      tc_fence_before();
      if (kPair) {
        // one arrival per warp, on the leader's barrier
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_rank(bar_a_full + 8 * st, lead_rank));
      } else {
        mbar_arrive(bar_a_full + 8 * st);
      }
    }
  }

  // ---------------- epilogue
  // Lane n of a dequantisation warp holds output column n of the tile; its TMEM columns are the tokens.
  // S == 1: registers -> y.  S > 1: token row m of the tile is owned by cluster rank m % S; every CTA
  // pushes the rows of its partial tile into the owners' shared memory (plain remote stores: no round
  // trip), one cluster barrier later each owner adds the S contributions in rank order (so the sum
  // does not depend on timing) and writes its rows of y.  The receive buffer reuses the operand rings,
  // hence the first cluster barrier: every CTA of the cluster must be done with its main loop.
  // All threads take the barriers whatever happened before; a CTA whose waits expired only skips the
  // memory traffic.
  const bool is_epi = warp >= kFirstDequantWarp;
  const int quad = warp & 3, hf = is_epi ? (warp - kFirstDequantWarp) >> 2 : 0;
  const int n = quad * 32 + lane;
  const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
  const int half_cols = MT >> 1, col0 = hf * half_cols;
  bool have_d = false;
  if (is_epi) {
    have_d = ab.wait(bar_d_full, 0);
    have_d = __all_sync(0xffffffffu, have_d && !ab.set());
    if (have_d) tc_fence_after();
  }
  if (p.S == 1) {
    if (have_d) {
      grid_dep_wait();                                       // y may still be read by the previous kernel
      const int n_glob = nt * kTileN + n;
      const bool n_ok = n_glob < d_out;
      const long long out_col = n_ok ? (p.col_map ? p.col_map[n_glob] : n_glob) : 0;
      for (int c0 = 0; c0 < half_cols; c0 += 8) {
        uint32_t v[8];
        tmem_ld8(lane_addr + col0 + c0, v);
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int mg = m0 + col0 + c0 + e;
          if (n_ok && mg < p.M) y_out[(long long)mg * ldy + out_col] = __float2half_rn(__uint_as_float(v[e]));
        }
      }
    }
  } else {
    const uint32_t rank = (uint32_t)split;                   // the K split of this CTA owns token rows rank, rank + S, ...
    const int rows_max = (MT + p.S - 1) / p.S;               // rows any rank can own
    const uint32_t recv = base;                              // [source rank][row slot][128] fp32
    cluster_arrive();                                        // #1: this CTA no longer touches its rings
    cluster_wait();
    if (have_d) {
      // token m = col0 + c goes to rank m % S, row slot m / S; walked without division
      int r = col0 % p.S, jrow = col0 / p.S;
      for (int c0 = 0; c0 < half_cols; c0 += 8) {
        uint32_t v[8];
        tmem_ld8(lane_addr + col0 + c0, v);
        tc_wait_ld();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t dst = recv + (uint32_t)(((int)rank * rows_max + jrow) * kTileN + n) * 4u;
          st_cluster_u32(map_to_rank(dst, kPair ? 2u * (uint32_t)r + pair_x : (uint32_t)r), v[e]);
          if (++r == p.S) {
            r = 0;
            ++jrow;
          }
        }
      }
    }
    cluster_arrive();                                        // #2: release my pushes, acquire everybody else's
    cluster_wait();
    if (is_epi && !ab.set()) {
      grid_dep_wait();                                       // y may still be read by the previous kernel
      const int tid = threadIdx.x - kFirstDequantWarp * 32;
      const int rows = (MT - (int)rank + p.S - 1) / p.S;     // token rows rank, rank + S, ...
      const int n0 = nt * kTileN;
      for (int it = tid; it < rows * 32; it += kDequantThreads) {
        const int jrow = it >> 5, i4 = it & 31;
        const uint8_t *src = gen + (uint32_t)(jrow * kTileN + i4 * 4) * 4u;
        float4 acc = *reinterpret_cast<const float4 *>(src);
        for (int sp = 1; sp < p.S; ++sp) {
          const float4 v = *reinterpret_cast<const float4 *>(src + (size_t)sp * rows_max * kTileN * 4);
          acc.x += v.x, acc.y += v.y, acc.z += v.z, acc.w += v.w;
        }
        const int mg = m0 + (int)rank + jrow * p.S, nn = n0 + i4 * 4;
        if (mg >= p.M || nn >= d_out) continue;
        __align__(8) __half h[4] = {__float2half_rn(acc.x), __float2half_rn(acc.y), __float2half_rn(acc.z),
                                    __float2half_rn(acc.w)};
        __half *row = y_out + (long long)mg * ldy;
        if (!p.col_map && nn + 3 < d_out) {
          *reinterpret_cast<uint2 *>(row + nn) = *reinterpret_cast<const uint2 *>(h);
        } else {
          for (int e = 0; e < 4 && nn + e < d_out; ++e) row[p.col_map ? p.col_map[nn + e] : nn + e] = h[e];
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (kPair && p.S == 1) {                                   // the pair gives its tensor memory back together
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 2) {
    __syncwarp();
    if (kPair) tmem_dealloc_pair<kTmemCols>(tmem);
    else tmem_dealloc<kTmemCols>(tmem);
  }
}

// ---------------------------------------------------------------------------------- stream-K variant
// For token tiles of at most 64 tokens and operands with enough column tiles, the (tile, group) list of
// the whole launch is cut into one contiguous range per CTA (two CTAs per SM, equal cost), so every SM
// streams the same number of bytes whatever the tile count.  A range covers the tail of one tile and the
// head of the next at most: two accumulators in tensor memory, one main loop over both, one epilogue.
// A tile shared by several CTAs is finished by the one that holds its last groups: the others store
// their fp32 partial tile to a workspace and count themselves in; the finisher waits for them (they all
// have lower block indices, hence were dispatched before it), adds the partials in ascending K order
// and its own accumulator last, and writes y.  The sum order is fixed, so results are reproducible.
constexpr int kMaxSkCtas = kSkMaxCtas;
constexpr int kSkStages = 2;                       // one TMEM operand buffer + activation slot per team
constexpr int kSkTokens = 64;                      // token capacity of an accumulator and of a partial tile

struct SkParams {
  int n_prob;
  int tile_start[kMaxProblems + 1];
  const uint8_t *blob[kMaxProblems];
  int d_out[kMaxProblems];
  __half *y[kMaxProblems];
  long long ldy[kMaxProblems];
  long long tile_stride;
  int g_fp16, g_quant, block_groups;
  int G;                     // groups per tile
  int M, MT;
  int NW;
  const int32_t *col_map;
  int *status;
  long long wait_limit;
  float *partials;           // [CTA][2][64 tokens][128 columns]
  int *arrive;               // [tile]: partial tiles stored so far; zero between launches
  int bounds[kMaxSkCtas + 1];   // CTA i owns entries [bounds[i], bounds[i + 1]) of the tile-major (tile, group) list
};

struct SkTile {
  int prob, nt;
  const uint8_t *base;
};

__device__ __forceinline__ SkTile sk_tile(const SkParams &p, int tile) {
  int prob = 0;
  while (prob + 1 < p.n_prob && tile >= p.tile_start[prob + 1]) ++prob;
  const int nt = tile - p.tile_start[prob];
  return SkTile{prob, nt, p.blob[prob] + (long long)nt * p.tile_stride};
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ int ld_acquire(const int *ptr) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

template <int kBits>
__global__ void __launch_bounds__(kThreads, 2)
linear_sk_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ SkParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int MT = p.MT;
  const uint32_t x_slot_bytes = (uint32_t)MT * 256u;
  const uint32_t x_ring = base;
  const uint32_t w_ring = x_ring + kSkStages * x_slot_bytes;
  const uint32_t bars = w_ring + p.NW * kWSlotBytes;
  const uint32_t bar_w_full = bars, bar_w_empty = bar_w_full + 8 * p.NW;
  const uint32_t bar_x_full = bar_w_empty + 8 * p.NW, bar_a_full = bar_x_full + 8 * kSkStages;
  const uint32_t bar_empty = bar_a_full + 8 * kSkStages;
  const uint32_t bar_d_full = bar_empty + 8 * kSkStages;       // two: one per accumulator
  const uint32_t misc = bar_d_full + 16;                       // [0] TMEM base, [1] abort flag
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t *misc_ptr = reinterpret_cast<volatile uint32_t *>(gen + (misc - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x;
  const int u_begin = p.bounds[cta], n_units = p.bounds[cta + 1] - u_begin;
  const int tile0 = u_begin / p.G, g0 = u_begin - tile0 * p.G;
  const int len0 = n_units < p.G - g0 ? n_units : p.G - g0;    // entries of the first tile; the rest start the next tile
  const Abort ab{reinterpret_cast<volatile int *>(misc_ptr + 1), p.status, p.wait_limit, false};

  grid_dep_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.NW; ++i) {
      mbar_init(bar_w_full + 8 * i, 1);
      mbar_init(bar_w_empty + 8 * i, kTeamThreads);
    }
    for (int i = 0; i < kSkStages; ++i) {
      mbar_init(bar_x_full + 8 * i, 1);
      mbar_init(bar_a_full + 8 * i, kTeamThreads + 1);         // + the activation copy
      mbar_init(bar_empty + 8 * i, 1);
      mbar_init(bar_d_full + 8 * i, 1);
    }
    misc_ptr[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) tmem_alloc<kTmemCols>(misc);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc_ptr[0];
  // columns: accumulator of the first tile at 0, of the second at 64, operand buffers at 128 and 192
  const uint32_t a_col0 = 2 * kSkTokens;
  const int qbytes = quant_tile_bytes(kBits);

  if (warp == 0) {
    // ---------------- weight-tile producer
    if (lane == 0) {
      int uc = 0;
      Ring rw{0, 0};
      int tile = tile0, g = g0;
      const uint8_t *tile_base = sk_tile(p, tile).base;
      for (int j = 0; j < n_units && !ab.set(); ++j) {
        const bool f16 = g < p.g_fp16;
        const uint8_t *src = tile_base + (f16 ? (long long)g * kFp16TileBytes
                                              : (long long)p.g_fp16 * kFp16TileBytes + (long long)(g - p.g_fp16) * qbytes);
        const int nsub = f16 ? 4 : 1;
        const uint32_t bytes = f16 ? kFp16SubBytes : qbytes;
        bool live = true;
        for (int sub = 0; sub < nsub; ++sub, ++uc, rw.advance(p.NW)) {
          const int slot = rw.idx;
          if (!ab.wait_local(bar_w_empty + 8 * slot, rw.lap ^ 1u)) {
            live = false;
            break;
          }
          mbar_arrive_expect_tx(bar_w_full + 8 * slot, bytes);
          bulk_copy_g2s(w_ring + slot * kWSlotBytes, src + (long long)sub * kFp16SubBytes, bytes, bar_w_full + 8 * slot);
        }
        if (!live) break;
        if (++g == p.G && j + 1 < n_units) {
          g = 0;
          tile_base = sk_tile(p, ++tile).base;
        }
      }
      if (ab.set()) {  // let copies already in flight land before the CTA goes away
        for (int back = 1; back <= p.NW && back <= uc; ++back) {
          const int u = uc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (mbar_try_wait(bar_w_full + 8 * (u % p.NW), (u / p.NW) & 1)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- activation producer
    if (lane == 0) {
      grid_dep_wait();                                         // x may be the previous kernel's output
      int gc = 0;
      Ring rs{0, 0};
      int tile = tile0, g = g0;
      auto block0 = [&](int t) {
        const int nt = sk_tile(p, t).nt;
        return p.block_groups > 0 ? (nt / p.block_groups) * p.block_groups : 0;
      };
      int g_block0 = block0(tile);
      for (int j = 0; j < n_units && !ab.set(); ++j, ++gc, rs.advance(kSkStages)) {
        const int slot = rs.idx;
        if (!ab.wait(bar_empty + 8 * slot, rs.lap ^ 1u)) break;
        const int k0 = (g_block0 + g) * kGroup;
        mbar_arrive_expect_tx(bar_a_full + 8 * slot, x_slot_bytes);
        tma_load_3d(x_ring + slot * x_slot_bytes, &xmap, bar_a_full + 8 * slot, 0, k0 >> 6);
        if (++g == p.G && j + 1 < n_units) {
          g = 0;
          g_block0 = block0(++tile);
        }
      }
      if (ab.set()) {
        for (int back = 1; back <= kSkStages && back <= gc; ++back) {
          const int u = gc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (mbar_try_wait(bar_a_full + 8 * (u % kSkStages), (u / kSkStages) & 1)) break;
        }
      }
    }
  } else if (warp == 2) {
    // ---------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | ((uint32_t)(MT >> 3) << 17) | (8u << 24);
      const uint64_t desc0 = make_b_desc(x_ring);
      const uint32_t x_slot16 = x_slot_bytes >> 4, half16 = (uint32_t)(MT * 128) >> 4;
      Ring rs{0, 0};
      uint32_t accumulate = 0;
      int g = g0, seg = 0, committed = 0;
      for (int j = 0; j < n_units; ++j, rs.advance(kSkStages)) {
        const int st = rs.idx;
        if (!ab.wait(bar_a_full + 8 * st, rs.lap)) break;
        tc_fence_after();
        const uint64_t b0 = desc0 + (uint64_t)(st * x_slot16);
        tc_mma8_ts(tmem + seg * kSkTokens, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
        tc_commit(bar_empty + 8 * st);
        accumulate = 1;
        if (++g == p.G || j + 1 == n_units) {                  // this tile's share is complete
          tc_commit(bar_d_full + 8 * seg);
          ++seg, ++committed;
          g = 0;
          accumulate = 0;
        }
      }
      if (ab.set()) {  // MMAs already issued must retire before the tensor memory is given back
        const uint32_t bar = bar_d_full + 8 * (committed < 2 ? committed : 1);
        if (committed < 2) tc_commit(bar);
        for (int it = 0; it < kDrainPolls; ++it)
          if (mbar_try_wait(bar, 0)) break;
      }
    }
  } else {
    // ---------------- dequantisation: two teams on alternate entries, team = stage
    const int dq = warp - kFirstDequantWarp;
    const int quad = warp & 3;
    const int team = dq >> 2;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    Ring rw{0, 0}, rs{0, 0};
    bool ok = true;
    int g = g0;
    for (int j = 0; j < n_units && ok; ++j, rs.advance(kSkStages)) {
      const bool f16 = g < p.g_fp16;
      const int nsub = f16 ? 4 : 1;
      if (++g == p.G) g = 0;
      if ((j & 1) != team) {
        for (int sub = 0; sub < nsub; ++sub) rw.advance(p.NW);
        continue;
      }
      const int st = rs.idx;
      const uint32_t a_addr = lane_addr + a_col0 + st * 64;
      bool got = ab.wait(bar_empty + 8 * st, rs.lap ^ 1u);
      for (int sub = 0; sub < nsub && ok; ++sub, rw.advance(p.NW)) {
        const int slot = rw.idx;
        // first see the slot's previous fill released (it may belong to the other team, which can lag by
        // an entry), then wait for the new one: a parity wait must not be a whole phase early
        got = got && ab.wait_local(bar_w_empty + 8 * slot, rw.lap ^ 1u) && ab.wait_local(bar_w_full + 8 * slot, rw.lap);
        got = __all_sync(0xffffffffu, got);
        if (!got) {
          ok = false;
          break;
        }
        tc_fence_after();
        dequant_unit<kBits>(f16, w_ring + slot * kWSlotBytes, n, a_addr, sub, bar_w_empty + 8 * slot);
      }
      tc_wait_st();
      if (!ok) break;
      tc_fence_before();
      mbar_arrive(bar_a_full + 8 * st);
    }
  }

  // ---------------- epilogue: one pass per tile this CTA touched
  // Thread (column n = TMEM lane, half hf of the tokens) owns tokens col0 .. col0 + MT/2 - 1 of column n.
  const bool is_epi = warp >= kFirstDequantWarp;
  if (is_epi) {
    const int quad = warp & 3, hf = (warp - kFirstDequantWarp) >> 2;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    const int half_cols = MT >> 1, col0 = hf * half_cols;
    const bool lead = threadIdx.x == kFirstDequantWarp * 32;
    grid_dep_wait();                       // y, the partial tiles and the counters may still be in use by the previous kernel
    const int n_seg = len0 < n_units ? 2 : 1;
    // the second tile first: its partial tile waits for nobody, while finishing the first tile may wait
    for (int seg = n_seg - 1; seg >= 0; --seg) {
      const int tile = tile0 + seg;
      const int gs = seg == 0 ? g0 : 0, len = seg == 0 ? len0 : n_units - len0;
      bool have_d = ab.wait(bar_d_full + 8 * seg, 0);
      have_d = __all_sync(0xffffffffu, have_d && !ab.set());
      if (have_d) tc_fence_after();
      const SkTile tr = sk_tile(p, tile);
      const int d_out = p.d_out[tr.prob];
      __half *const y_out = p.y[tr.prob];
      const long long ldy = p.ldy[tr.prob];
      const uint32_t d_addr = lane_addr + seg * kSkTokens + col0;
      const bool finisher = gs + len == p.G;                   // holds the tile's last groups
      if (!finisher) {
        // store the partial tile [token][column] (a warp writes 128 contiguous bytes per token) and
        // count this CTA in
        if (have_d) {
          uint32_t *dst = reinterpret_cast<uint32_t *>(p.partials) + (((long long)cta * 2 + seg) * kSkTokens + col0) * kTileN + n;
          for (int c0 = 0; c0 < half_cols; c0 += 8) {
            uint32_t v[8];
            tmem_ld8(d_addr + c0, v);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) dst[(c0 + e) * kTileN] = v[e];
          }
        }
        epi_bar();                                             // all stores of the CTA are issued ...
        if (lead && !ab.set()) {
          __threadfence();                                     // ... and ordered before the count (cumulative fence)
          atomicAdd(p.arrive + tile, 1);
        }
        continue;
      }
      // the finisher: contributors cf .. cta - 1 hold the earlier groups of this tile
      int cf = cta;
      while (cf > 0 && p.bounds[cf] > tile * p.G) --cf;
      const int k_lower = cta - cf;
      if (k_lower > 0) {
        if (lead) {
          bool seen = false;
          for (long long it = 0; it < p.wait_limit && !seen; ++it) {
            seen = ld_acquire(p.arrive + tile) >= k_lower;
            if (!seen && (it & 63) == 63 && ab.set()) break;
          }
          if (!seen && !ab.set()) ab.raise();
        }
        epi_bar();
        have_d = have_d && !ab.set();
      }
      if (have_d) {
        const int n_glob = tr.nt * kTileN + n;
        const bool n_ok = n_glob < d_out;
        const long long out_col = n_ok ? (p.col_map ? p.col_map[n_glob] : n_glob) : 0;
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
        for (int c = cf; c < cta; ++c) {                       // ascending K; up to 32 coalesced loads in flight
          const int slot = (c == cf && p.bounds[cf] < tile * p.G) ? 1 : 0;   // the tile is that CTA's second one
          const float *src = p.partials + (((long long)c * 2 + slot) * kSkTokens + col0) * kTileN + n;
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = e < half_cols ? __ldcg(src + e * kTileN) : 0.f;
#pragma unroll
          for (int e = 0; e < 32; ++e) acc[e] += v[e];
        }
#pragma unroll
        for (int c0 = 0; c0 < 32; c0 += 8) {
          if (c0 < half_cols) {
            uint32_t v[8];
            tmem_ld8(d_addr + c0, v);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float r = acc[c0 + e] + __uint_as_float(v[e]);
              const int mg = col0 + c0 + e;
              if (n_ok && mg < p.M) y_out[(long long)mg * ldy + out_col] = __float2half_rn(r);
            }
          }
        }
      }
      if (k_lower > 0) {
        epi_bar();                                             // every thread has read the partial tiles
        if (lead && !ab.set()) p.arrive[tile] = 0;             // ready for the next launch
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    __syncwarp();
    tmem_dealloc<kTmemCols>(tmem);
  }
}

// ---------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
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

size_t smem_bytes(int MT, int NW, int NA) {
  size_t b = 1024 + (size_t)NA * MT * 256 + (size_t)NW * kWSlotBytes + 8 * (2 * NW + 3 * NA + 1) + 16;
  // never less than a third of an SM's shared memory: at most two CTAs share an SM, which is also what
  // their 2 x 256 tensor-memory columns allow
  return b < 80 * 1024 ? 80 * 1024 : b;
}


// {64 channels, tokens, 64-channel block} view of the row-major activations, box = one group (two blocks)
// of MT tokens; rows past M are zero-filled by the copy
bool encode_x_map3(EncodeTiledFn encode, CUtensorMap *map, const __half *x, int M, long long ldx, int d_in, int MT) {
  const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(d_in / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)ldx * sizeof(__half), 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)MT, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half *>(x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t sk_smem_bytes(int MT, int NW) {
  size_t b = 1024 + (size_t)kSkStages * MT * 256 + (size_t)NW * kWSlotBytes + 8 * (2 * NW + 4 * kSkStages) + 16;
  return b < 80 * 1024 ? 80 * 1024 : b;
}

// Cuts the tile-major (tile, group) list into P ranges of equal cost, every cut on a group boundary.
// False when a range would be empty or touch more than two tiles.
bool sk_bounds(int T, int G, int g_fp16, int P, int *bounds) {
  const long long FW = kCostFp16, QW = kCostQuant;
  const long long C = FW * g_fp16 + QW * (G - g_fp16), N = C * T;
  for (int i = 0; i <= P; ++i) {
    const long long c = N * i / P;
    const long long tile = c / C, within = c % C;
    const long long g = within < FW * g_fp16 ? within / FW : g_fp16 + (within - FW * g_fp16) / QW;
    bounds[i] = (int)(tile * G + g);
  }
  bounds[P] = T * G;
  for (int i = 0; i < P; ++i) {
    if (bounds[i + 1] <= bounds[i]) return false;
    if ((bounds[i + 1] - 1) / G - bounds[i] / G > 1) return false;
  }
  return true;
}

}  // namespace

// Launch policy of the per-call kernels (fixed; measured on the 7B / 13B shapes):
//   kUsePdl      launches are chained with programmatic stream serialization
//   kSkTileRatio the equal-share variant is used when CTAs <= kSkTileRatio x column tiles
constexpr bool kUsePdl = true;
constexpr int kSkTileRatio = 2;

static int launch_linear_sk(const rosaq_ctx *ctx, const __half *x, long long ldx, const TiledOperand &t, const SkParams &q,
                            int P, cudaStream_t s) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return ROSAQ_ERR_CUDA;
  CUtensorMap xmap;
  if (!encode_x_map3(encode, &xmap, x, q.M, ldx, t.d_in, q.MT)) return ROSAQ_ERR_CUDA;
  const size_t smem = sk_smem_bytes(q.MT, q.NW);
  const bool int3 = t.g_quant > 0 && t.bits == 3;
  auto kern = int3 ? linear_sk_kernel<3> : linear_sk_kernel<4>;
  static size_t attr_smem_all[kMaxDevices][2] = {};       // function attributes are per device
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return ROSAQ_ERR_INVALID_ARG;
  size_t *attr_smem = attr_smem_all[ctx->device];
  static std::mutex attr_mutex;                           // contexts of several host threads share these caches
  std::lock_guard<std::mutex> attr_lock(attr_mutex);
  if (attr_smem[int3 ? 1 : 0] < smem) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess ||
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_CUDA;
    }
    attr_smem[int3 ? 1 : 0] = smem;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(P, 1, 1);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (kUsePdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, xmap, q);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

int launch_linear_tc(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t,
                     const int32_t *col_map, __half *y, long long ldy, cudaStream_t s) {
  const TiledOperand *ts[1] = {&t};
  __half *ys[1] = {y};
  long long ldys[1] = {ldy};
  return launch_linear_tc_multi(ctx, x, M, ldx, 1, ts, col_map, ys, ldys, s);
}

// n weights of identical geometry applied to the same activations in one launch
int launch_linear_tc_multi(const rosaq_ctx *ctx, const __half *x, int M, long long ldx, int n,
                           const TiledOperand *const *ts, const int32_t *col_map, __half *const *ys,
                           const long long *ldys, cudaStream_t s) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return ROSAQ_ERR_CUDA;
  if (n < 1 || n > kMaxProblems) return ROSAQ_ERR_INVALID_ARG;
  const TiledOperand &t = *ts[0];
  const int G = groups_per_tile(t);
  if (G <= 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;

  TcParams p{};
  p.n_prob = n;
  int n_tiles_all = 0;
  for (int i = 0; i < n; ++i) {
    const TiledOperand &ti = *ts[i];
    if (ti.d_in != t.d_in || ti.g_fp16 != t.g_fp16 || ti.g_quant != t.g_quant || ti.block_groups != t.block_groups ||
        (t.g_quant > 0 && ti.bits != t.bits))
      return ROSAQ_ERR_INVALID_ARG;
    p.tile_start[i] = n_tiles_all;
    p.blob[i] = ti.blob;
    p.d_out[i] = ti.d_out;
    p.y[i] = ys[i];
    p.ldy[i] = ldys[i];
    n_tiles_all += ti.n_tiles;
  }
  p.tile_start[n] = n_tiles_all;
  p.tile_stride = t.tile_stride;
  p.g_fp16 = t.g_fp16;
  p.g_quant = t.g_quant;
  p.bits = t.bits;
  p.block_groups = t.block_groups;
  p.M = M;
  const int m_tiles = (M + 127) / 128;
  const int per_tile = (M + m_tiles - 1) / m_tiles;
  p.MT = ((per_tile + 15) / 16) * 16;
  p.col_map = col_map;
  p.status = ctx->d_status;
  p.wait_limit = ctx->wait_limit;
  // stages (TMEM operand buffer + activation slot of MT x 128 channels): 3 next to 64 accumulator
  // columns, 2 next to 128; the rest of a half SM's shared memory goes to the packed-weight ring
  p.NA = p.MT <= 64 ? 3 : 2;
  // CTA pairs: adjacent column tiles of one weight, token count a multiple of 32 (MMA N of a pair)
  // (a block-diagonal operand pairs up only if both tiles of a pair multiply the same channels)
  // Off unless asked for (linear implementation 2): on the decode shapes measured so far the pair's
  // cross-CTA handshakes cost more than the halved MMA issue saves.
  bool pair = ctx->impl == 2 && p.MT % 32 == 0 && t.block_groups % 2 == 0;
  for (int i = 0; i < n && pair; ++i) pair = ts[i]->n_tiles % 2 == 0;
  // stream-K variant: token tile of at most 64 tokens, one token tile, and so many column tiles that a tile
  // is shared by two or three CTAs at most (its finisher reads the others' partial tiles one after the
  // other; measured at 64 tokens: 4096 -> 22016, 172 tiles, 23.4 us against 28.4 with cluster splits;
  // with 96 tiles 0.7 us slower, with 86 tiles 2.2 us slower)
  if (ctx->impl == 0 && !pair && m_tiles == 1 && p.MT <= kSkTokens && ctx->sk_partials) {
    const int P = ctx->sk_ctas < 2 * ctx->sm_count ? ctx->sk_ctas : 2 * ctx->sm_count;
    if (n_tiles_all <= P && n_tiles_all <= kSkCounterInts && (long long)n_tiles_all * kSkTileRatio >= P) {
      SkParams q{};
      if (sk_bounds(n_tiles_all, G, t.g_fp16, P, q.bounds)) {
        q.n_prob = n;
        for (int i = 0; i <= n; ++i) q.tile_start[i] = p.tile_start[i];
        for (int i = 0; i < n; ++i) q.blob[i] = p.blob[i], q.d_out[i] = p.d_out[i], q.y[i] = p.y[i], q.ldy[i] = p.ldy[i];
        q.tile_stride = p.tile_stride;
        q.g_fp16 = p.g_fp16, q.g_quant = p.g_quant, q.block_groups = p.block_groups;
        q.G = G, q.M = M, q.MT = p.MT;
        q.col_map = col_map, q.status = p.status, q.wait_limit = p.wait_limit;
        q.partials = ctx->sk_partials, q.arrive = ctx->sk_arrive;
        {
          const int budget = 110 * 1024 - 1024 - kSkStages * p.MT * 256 - 256;
          const int nw = budget / kWSlotBytes;
          q.NW = nw > 10 ? 10 : nw;
        }
        return launch_linear_sk(ctx, x, ldx, t, q, P, s);
      }
    }
  }
  const int MTL = pair ? p.MT / 2 : p.MT;                  // token rows a CTA keeps in shared memory
  {
    const int budget = 110 * 1024 - 1024 - p.NA * MTL * 256 - 256;
    int nw = budget / kWSlotBytes;
    p.NW = nw > 10 ? 10 : nw;
  }

  // K splits: fill about two CTAs per SM; each split gets a contiguous range of groups of roughly
  // equal cost
  const int tiles = n_tiles_all * m_tiles;
  // (measured: cluster launches place a little less than two CTAs per SM; asking for more than about
  // 2 x SMs - 32 CTAs spills into a second wave)
  int S = (2 * ctx->sm_count - 32) / (tiles > 0 ? tiles : 1);
  const int max_splits = pair ? kMaxSplits / 2 : kMaxSplits;    // a cluster holds the S splits of both CTAs of a pair
  // (six splits measured faster than eight on the 32-tile shapes: the exchange grows with the cluster)
  const int auto_cap = pair ? max_splits : 6;
  S = S < 1 ? 1 : (S > auto_cap ? auto_cap : S);
  if (S > G) S = G;
  p.S = S;
  {
    // bound sp is the first group whose
    // preceding cost reaches sp/S of the total, clamped so that every range keeps a group
    auto cost_before = [&](int g) {
      return g <= t.g_fp16 ? (long long)kCostFp16 * g : (long long)kCostFp16 * t.g_fp16 + (long long)kCostQuant * (g - t.g_fp16);
    };
    const long long total = cost_before(G);
    p.g_bounds[0] = 0;
    for (int sp = 1; sp < S; ++sp) {
      int g = p.g_bounds[sp - 1] + 1;
      while (g < G - (S - sp) && cost_before(g) * S < total * sp) ++g;
      p.g_bounds[sp] = g;
    }
    p.g_bounds[S] = G;
  }

  CUtensorMap xmap;
  if (!pair) {
    if (!encode_x_map3(encode, &xmap, x, M, ldx, t.d_in, p.MT)) return ROSAQ_ERR_CUDA;
  } else {
    const cuuint64_t dims[2] = {(cuuint64_t)t.d_in, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)ldx * sizeof(__half)};
    const cuuint32_t box[2] = {64, (cuuint32_t)MTL};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half *>(x), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return ROSAQ_ERR_CUDA;
  }

  const size_t smem = smem_bytes(MTL, p.NW, p.NA);
  const bool int3 = t.g_quant > 0 && t.bits == 3;
  auto kern = pair ? (int3 ? linear_tc_kernel<3, true> : linear_tc_kernel<4, true>)
                   : (int3 ? linear_tc_kernel<3, false> : linear_tc_kernel<4, false>);
  // The opt-in limit is kept equal to what the launches really need (never a rounder, larger figure):
  // the driver sizes the shared-memory carve-out and the CTAs per SM from this attribute, and with
  // 2 x (limit + 1 KB) above the SM's 228 KB only one CTA would be resident.
  static size_t attr_smem_all[kMaxDevices][4] = {};      // function attributes are per device
  if (ctx->device < 0 || ctx->device >= kMaxDevices) return ROSAQ_ERR_INVALID_ARG;
  size_t *attr_smem = attr_smem_all[ctx->device];
  const int ki = (int3 ? 1 : 0) + (pair ? 2 : 0);
  static std::mutex attr_mutex;                          // contexts of several host threads share these caches
  std::lock_guard<std::mutex> attr_lock(attr_mutex);
  if (attr_smem[ki] < smem) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess ||
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_CUDA;
    }
    attr_smem[ki] = smem;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(n_tiles_all, S, m_tiles);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (S > 1 || pair) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = pair ? 2 : 1;
    attr[na].val.clusterDim.y = S;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  if (kUsePdl) {
    // programmatic dependent launch: this kernel may start while the previous kernel of the stream is
    // still running; it touches x and y only after griddepcontrol.wait
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, xmap, p);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

}  // namespace rosaq

extern "C" int rosaq_plan_equal_shares(int n_tiles, int groups, int g_fp16, int n_ctas, int32_t *bounds) {
  if (n_tiles <= 0 || groups <= 0 || g_fp16 < 0 || g_fp16 > groups || n_ctas <= 0 || !bounds) return ROSAQ_ERR_INVALID_ARG;
  if ((long long)n_tiles * groups > 0x7fffffffll) return ROSAQ_ERR_INVALID_ARG;
  static_assert(sizeof(int) == sizeof(int32_t), "bounds are written as int");
  return rosaq::sk_bounds(n_tiles, groups, g_fp16, n_ctas, reinterpret_cast<int *>(bounds)) ? ROSAQ_OK
                                                                                           : ROSAQ_ERR_UNSUPPORTED_SHAPE;
}
