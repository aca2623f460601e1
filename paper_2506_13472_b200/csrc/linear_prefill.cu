// The GEMM stage  y = x . W^  (Eq. 3) for prefill-sized batches: more than 128 tokens.
//
// Why another kernel.  With a few hundred tokens the stage is bound by the tensor pipe, not by the weight
// stream, and what counts is how many tokens share one dequantisation of a weight tile and how often an
// operand byte is fetched from L2: a tcgen05.mma of 128 x N x 16 runs at full rate from N = 128 on (64
// cycles, 128 for N = 256; 55 for N = 64 is 58 %), a weight tile dequantised for 128 tokens costs as many
// instructions as one dequantised for 256, and a CTA that multiplies 128 columns with 256 tokens on its own
// pulls 64 KB of activations per 128-channel group.  Here two CTAs of a cluster (adjacent SMs) share a
// 256-column x 256-token tile as a cta_group::2 pair: rank r dequantises column tile 2 c + r into its own
// tensor memory (the A operand, 128 lanes each) and loads 128 of the 256 token rows (its half of the B
// operand, 32 KB per group), the leader issues M = 256, N = 256 MMAs for both, and each CTA ends up with the
// accumulator of its own 128 columns for all 256 tokens.  A weight tile is dequantised once per 256 tokens.
//
// Work is cut the stream-K way: the list of (tile, 128-channel group) units, token blocks of one column pair
// next to each other so that the second one finds the packed weights in L2, is cut into one contiguous range
// of equal length per pair of CTAs (a 13B projection at 512 tokens is 108 tiles for 74 pairs: whole tiles
// would take two rounds, equal ranges take 1.46).  A pair therefore holds at most one tile without its first
// groups -- the first piece of its range: it stores that partial tile (fp32) in its own slot of a workspace
// and raises its flag -- then whole tiles, and at the end of its range possibly a tile without its last groups:
// it owns that tile, waits for the flags of the pairs that hold the rest (they went through it at the
// start of their ranges, long before), adds their partial tiles in ascending K order and writes y.  A flag
// has one writer and one reader, which puts it back to zero once the partial tile is in its shared memory:
// every launch, replays of a captured launch included, starts from zero flags.  The launch is cooperative:
// every pair is resident, and a pair only ever waits for work that other pairs do first in their ranges.
//
// Per CTA: warp 0 = weight-tile producer (bulk copies; one sub-ring of slots per dequantisation team),
// 1 = activation producer (TMA, bytes of both CTAs counted on the leader's barrier), 2 = MMA issuer (leader
// only; also owns the tensor memory), 4..19 = four dequantisation teams (group j of the CTA's stream goes
// to team and operand buffer j mod 4), 20..27 = epilogue (two warps per TMEM lane quadrant, 128 tokens
// each).  Tensor memory: accumulator in columns 0..255, four operand buffers of 64 columns behind it, so the
// accumulator is single: the epilogue of a tile (about a microsecond) is not overlapped with the next
// tile's MMAs, only with its copies and its dequantisation.  Loads carry no cluster multicast.
// Every wait is bounded; a CTA that gives up records ROSAQ_ERR_TIMEOUT, lets its copies and MMAs in flight
// finish, frees its tensor memory and returns.
#include <cuda.h>

#include <mutex>

#include "linear_common.cuh"

namespace rosaq {

namespace {

constexpr int kPfTmemCols = 512;
constexpr int kPfTokens = 256;                      // tokens per tile = N of the MMA
constexpr int kPfRows = kPfTokens / 2;              // token rows a CTA keeps in shared memory
constexpr int kPfStages = 4;                        // operand buffers, each with its activation slot
constexpr int kPfTeams = 4;
constexpr int kPfFirstDequantWarp = 4, kPfFirstEpiWarp = kPfFirstDequantWarp + 4 * kPfTeams;
constexpr int kPfEpiThreads = 256;
constexpr int kPfThreads = kPfFirstEpiWarp * 32 + kPfEpiThreads;   // 896
constexpr int kPfXSlotBytes = kPfRows * 256;        // 128 tokens x 128 channels of fp16
constexpr int kPfNW = 8;                            // weight slots: two per team
constexpr int kPfSmemBytes = 1024 + kPfStages * kPfXSlotBytes + kPfNW * kWSlotBytes + 8 * (2 * kPfNW + 2 * kPfStages + 5) + 16;

struct alignas(64) PfParams {
  CUtensorMap xmap;
  const uint8_t *blob;
  __half *y;
  long long tile_stride, ldy;
  int d_out, n_tiles, g_fp16, groups;
  int n_col_pairs, n_tok_blocks, M;
  int units;                  // (column pairs x token blocks) x groups
  float *partials;            // [pair][rank][256 tokens][128 columns]
  unsigned *flags;            // [pair][rank]: 1 while the slot holds a partial tile that nobody has fetched yet
  int *status;
  long long wait_limit;
};

__device__ __forceinline__ int pf_range_begin(int pair, int n_pairs, int units) {
  return (int)(((long long)pair * units) / n_pairs);
}
// next piece of the range [u, end): groups [g0, g1) of work item wk; false when the range is used up
__device__ __forceinline__ bool pf_next_piece(int &u, int end, int G, int &wk, int &g0, int &g1) {
  if (u >= end) return false;
  wk = u / G;
  g0 = u - wk * G;
  const int len = min(G - g0, end - u);
  g1 = g0 + len;
  u += len;
  return true;
}
// the 256 epilogue threads agree on whether to go on (all of them always come here)
__device__ __forceinline__ bool pf_epi_vote(bool v) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, 1, 256, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)v)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ unsigned pf_ld_acquire(const unsigned *ptr) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}

// sixteen tokens t0 .. of one output column, rounded once, rows past M left alone
__device__ __forceinline__ void pf_store_rows(const uint32_t *v, __half *y_col, int t0, int M, long long ldy, bool n_ok) {
  __half *yp = y_col + (long long)t0 * ldy;
  if (n_ok && t0 + 16 <= M) {
#pragma unroll
    for (int e = 0; e < 16; ++e, yp += ldy) *yp = __float2half_rn(__uint_as_float(v[e]));
  } else if (n_ok) {
#pragma unroll
    for (int e = 0; e < 16; ++e, yp += ldy)
      if (t0 + e < M) *yp = __float2half_rn(__uint_as_float(v[e]));
  }
}

template <int kBits>
__global__ void __launch_bounds__(kPfThreads, 1)
linear_prefill_kernel(const __grid_constant__ PfParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t x_ring = base;
  const uint32_t w_ring = x_ring + kPfStages * kPfXSlotBytes;
  const uint32_t bars = w_ring + kPfNW * kWSlotBytes;
  const uint32_t bar_w_full = bars, bar_w_empty = bar_w_full + 8 * kPfNW;
  const uint32_t bar_a_full = bar_w_empty + 8 * kPfNW;         // operand buffers written + activation slots landed (leader's)
  const uint32_t bar_s_empty = bar_a_full + 8 * kPfStages;     // stage consumed by its MMAs (both CTAs)
  const uint32_t bar_d_full = bar_s_empty + 8 * kPfStages;     // accumulator complete (both CTAs)
  const uint32_t bar_d_empty = bar_d_full + 8;                 // accumulator drained by both CTAs (leader's)
  const uint32_t bar_drain = bar_d_empty + 8;
  const uint32_t bar_merge = bar_drain + 8;                    // a partial tile has landed in the activation ring
  const uint32_t misc = bar_drain + 16;                        // [0] TMEM base, [1] abort flag
  uint32_t *misc_ptr = reinterpret_cast<uint32_t *>(smem_raw + (misc - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = blockIdx.x & 1u;                       // position in the pair; 0 = leader
  const bool is_lead = rank == 0;
  const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);
  const int u_begin = pf_range_begin(pair, n_pairs, p.units), u_end = pf_range_begin(pair + 1, n_pairs, p.units);
  const Abort ab{reinterpret_cast<volatile int *>(misc_ptr + 1), p.status, p.wait_limit, true};

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPfNW; ++i) {
      mbar_init(bar_w_full + 8 * i, 1);
      mbar_init(bar_w_empty + 8 * i, kTeamThreads);
    }
    for (int i = 0; i < kPfStages; ++i) {
      mbar_init(bar_a_full + 8 * i, 2 * (kTeamThreads / 32) + 1);   // a team's warps in both CTAs + the activation copies
      mbar_init(bar_s_empty + 8 * i, 1);
    }
    mbar_init(bar_d_full, 1);
    mbar_init(bar_d_empty, 2 * (kPfEpiThreads / 32));          // one arrival per epilogue warp of both CTAs
    mbar_init(bar_drain, 1);
    mbar_init(bar_merge, 1);
    misc_ptr[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) tmem_alloc_pair<kPfTmemCols>(misc);           // both CTAs of the pair, same warp index
  tc_fence_before();
  __syncthreads();
  cluster_arrive();                                            // the peer's barriers and tensor memory exist
  cluster_wait();
  tc_fence_after();
  const uint32_t tmem = misc_ptr[0];
  const uint32_t a_col0 = kPfTokens;                           // operand buffers follow the accumulator
  const int qbytes = quant_tile_bytes(kBits);
  const int G = p.groups;

  if (warp == 0) {
    // ---------------- weight-tile producer
    if (lane == 0) {
      constexpr int NWT = kPfNW / kPfTeams;
      uint32_t idx4 = 0, lap4 = 0;
      unsigned long long fills4 = 0;
      int j = 0;
      bool live = true;
      int u = u_begin, wk, g0, g1;
      while (live && !ab.set() && pf_next_piece(u, u_end, G, wk, g0, g1)) {
        // (the second CTA of a pair on an odd last tile streams that tile again; its results are dropped)
        int my_tile = 2 * (wk / p.n_tok_blocks) + (int)rank;
        if (my_tile >= p.n_tiles) my_tile = p.n_tiles - 1;
        const uint8_t *tile_base = p.blob + (long long)my_tile * p.tile_stride;
        for (int g = g0; g < g1 && live; ++g, ++j) {
          const bool f16 = g < p.g_fp16;
          const uint8_t *src = tile_base + (f16 ? (long long)g * kFp16TileBytes
                                                : (long long)p.g_fp16 * kFp16TileBytes + (long long)(g - p.g_fp16) * qbytes);
          const int nsub = f16 ? 4 : 1;
          const uint32_t bytes = f16 ? kFp16SubBytes : qbytes;
          const int team = j & (kPfTeams - 1);
          uint32_t idx = (idx4 >> (8 * team)) & 0xffu;
          for (int sub = 0; sub < nsub; ++sub) {
            const int slot = team * NWT + (int)idx;
            if (!ab.wait_local(bar_w_empty + 8 * slot, ((lap4 >> team) & 1u) ^ 1u)) {
              live = false;
              break;
            }
            mbar_arrive_expect_tx(bar_w_full + 8 * slot, bytes);
            bulk_copy_g2s(w_ring + slot * kWSlotBytes, src + (long long)sub * kFp16SubBytes, bytes, bar_w_full + 8 * slot);
            fills4 += 1ull << (16 * team);
            if (++idx == (uint32_t)NWT) {
              idx = 0;
              lap4 ^= 1u << team;
            }
          }
          idx4 = (idx4 & ~(0xffu << (8 * team))) | (idx << (8 * team));
        }
      }
      if (ab.set()) {  // let copies already in flight land before the CTA goes away
        for (int team = 0; team < kPfTeams; ++team) {
          const int f = (int)((fills4 >> (16 * team)) & 0xffffu);
          for (int back = 1; back <= NWT && back <= f; ++back) {
            const int u = f - back;
            for (int it = 0; it < kDrainPolls; ++it)
              if (mbar_try_wait(bar_w_full + 8 * (team * NWT + u % NWT), (u / NWT) & 1)) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- activation producer: this CTA's 128 token rows of every group
    if (lane == 0) {
      int gc = 0;
      Ring rs{0, 0};
      bool live = true;
      int u = u_begin, wk, g0, g1;
      while (live && !ab.set() && pf_next_piece(u, u_end, G, wk, g0, g1)) {
        const int tok0 = (wk % p.n_tok_blocks) * kPfTokens + (int)rank * kPfRows;
        for (int g = g0; g < g1; ++g, ++gc, rs.advance(kPfStages)) {
          const int slot = rs.idx;
          if (!ab.wait(bar_s_empty + 8 * slot, rs.lap ^ 1u)) {
            live = false;
            break;
          }
          // all bytes are counted on the leader's barrier
          if (is_lead) mbar_arrive_expect_tx(bar_a_full + 8 * slot, 2 * kPfXSlotBytes);
          tma_load_3d_pair(x_ring + slot * kPfXSlotBytes, &p.xmap, map_to_rank(bar_a_full + 8 * slot, 0), tok0, 2 * g);
        }
      }
      // (the leader's barriers count the copies of both CTAs, and the peer stays until the cluster barrier
      // at the end of the kernel, which the leader reaches after this drain)
      if (ab.set() && is_lead) {
        for (int back = 1; back <= kPfStages && back <= gc; ++back) {
          const int u = gc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (ab.poll(bar_a_full + 8 * (u % kPfStages), (u / kPfStages) & 1)) break;
        }
      }
    }
  } else if (warp == 2) {
    // ---------------- MMA issuer (leader): per group one wait, eight MMAs of 256 x 256 x 16, one commit
    if (lane == 0 && is_lead) {
      const uint32_t idesc = (1u << 4) | ((uint32_t)(kPfTokens >> 3) << 17) | (16u << 24);
      const uint64_t desc0 = make_b_desc(x_ring);
      constexpr uint32_t x_slot16 = kPfXSlotBytes >> 4, half16 = (uint32_t)(kPfRows * 128) >> 4;
      Ring rs{0, 0};
      int n_done = 0;
      bool live = true, issued = false;
      int u = u_begin, wk, g0, g1;
      for (; live && pf_next_piece(u, u_end, G, wk, g0, g1); ++n_done) {
        if (!ab.wait(bar_d_empty, (uint32_t)(n_done & 1) ^ 1u)) break;   // the previous piece has been drained
        tc_fence_after();
        uint32_t accumulate = 0;
        for (int g = g0; g < g1; ++g, rs.advance(kPfStages)) {
          const int st = rs.idx;
          if (!ab.wait(bar_a_full + 8 * st, rs.lap)) {
            live = false;
            break;
          }
          tc_fence_after();
          const uint64_t b0 = desc0 + (uint64_t)(st * x_slot16);
          tc_mma8_ts_pair(tmem, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
          tc_commit_mc(bar_s_empty + 8 * st, 3);               // frees the stage in both CTAs
          accumulate = 1;
          issued = true;
        }
        if (!live) break;
        tc_commit_mc(bar_d_full, 3);
      }
      if (ab.set() && issued) {  // MMAs already issued must retire before the tensor memory is given back
        tc_commit_mc(bar_drain, 1);
        for (int it = 0; it < kDrainPolls; ++it)
          if (ab.poll(bar_drain, 0)) break;
      }
    }
  } else if (warp >= kPfFirstDequantWarp && warp < kPfFirstEpiWarp) {
    // ---------------- dequantisation: group j of the CTA's stream goes to team and operand buffer j mod 4
    const int quad = warp & 3;
    const int team = (warp - kPfFirstDequantWarp) >> 2;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    constexpr int NWT = kPfNW / kPfTeams;
    const uint32_t my_ring = w_ring + team * NWT * kWSlotBytes, my_full = bar_w_full + 8 * team * NWT,
                   my_empty = bar_w_empty + 8 * team * NWT;
    const uint32_t a_addr = lane_addr + a_col0 + team * 64;
    const uint32_t my_s_empty = bar_s_empty + 8 * team, my_a_full = bar_a_full + 8 * team;
    Ring rw{0, 0};
    bool ok = true;
    int j0 = 0;                                      // position of the tile's first group in the CTA's stream
    uint32_t use = 0;                                // how often this team's buffer was used before
    int u = u_begin, wk, g0, g1;
    while (ok && pf_next_piece(u, u_end, G, wk, g0, g1)) {
      for (int g = g0 + ((team - j0) & (kPfTeams - 1)); g < g1 && ok; g += kPfTeams, ++use) {
        const bool f16 = g < p.g_fp16;
        const int nsub = f16 ? 4 : 1;
        bool got = ab.wait(my_s_empty, (use & 1u) ^ 1u);
        for (int sub = 0; sub < nsub && ok; ++sub, rw.advance(NWT)) {
          got = got && ab.wait_local(my_full + 8 * rw.idx, rw.lap);
          got = __all_sync(0xffffffffu, got);        // the TMEM instructions below need the whole warp
          if (!got) {
            ok = false;
            break;
          }
          tc_fence_after();
          dequant_unit<kBits>(f16, my_ring + rw.idx * kWSlotBytes, n, a_addr, sub, my_empty + 8 * rw.idx);
        }
        tc_wait_st();
        if (!ok) break;
        tc_fence_before();
        __syncwarp();                                // one arrival per warp, on the leader's barrier
        if (lane == 0) mbar_arrive_cluster(map_to_rank(my_a_full, 0));
      }
      j0 += g1 - g0;
    }
  } else if (warp >= kPfFirstEpiWarp) {
    // ---------------- epilogue: thread = (output column n of this CTA's tile = TMEM lane, 128 of the 256
    // tokens = TMEM columns); a warp's store covers 32 consecutive columns of one token row
    const int quad = warp & 3;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    const int c_begin = ((warp - kPfFirstEpiWarp) >> 2) * kPfRows;
    const bool lead = threadIdx.x == kPfFirstEpiWarp * 32;
    constexpr long long kSlotFloats = (long long)kPfTokens * kTileN;             // one CTA's partial tile
    float *const my_slot = p.partials + (long long)(2 * pair + (int)rank) * kSlotFloats + n;
    int n_done = 0;
    uint32_t merge_phase = 0;
    int u = u_begin, wk, g0, g1;
    for (; pf_next_piece(u, u_end, G, wk, g0, g1); ++n_done) {
      const bool have_d = ab.wait(bar_d_full, (uint32_t)(n_done & 1));
      if (!pf_epi_vote(have_d && !ab.set())) break;
      tc_fence_after();
      const int tile = 2 * (wk / p.n_tok_blocks) + (int)rank;
      const int n_glob = tile * kTileN + n;
      const bool n_ok = tile < p.n_tiles && n_glob < p.d_out;
      const int tok0 = (wk % p.n_tok_blocks) * kPfTokens;
      if (g0 > 0) {
        // a tile without its first groups: store the partial tile, then raise this CTA's flag
        for (int c0 = c_begin; c0 < c_begin + kPfRows && tok0 + c0 < p.M; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(lane_addr + c0, v);
          tc_wait_ld();
          float *dp = my_slot + (long long)c0 * kTileN;
#pragma unroll
          for (int e = 0; e < 16; ++e) dp[e * kTileN] = __uint_as_float(v[e]);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(map_to_rank(bar_d_empty, 0));
        __threadfence();
        pf_epi_vote(true);
        if (lead) {
          __threadfence();
          atomicExch(p.flags + 2 * pair + (int)rank, 1u);
        }
        continue;
      }
      // the tile's first groups are here: this CTA writes y.  The pairs pair + 1 .. last hold the tile's other groups.
      int last = pair;
      if (g1 < G) {
        const int uu = wk * G + G - 1;                         // the tile's last unit
        last = (int)(((long long)uu * n_pairs) / p.units);
        while (last + 1 < n_pairs && pf_range_begin(last + 1, n_pairs, p.units) <= uu) ++last;
        while (last > pair && pf_range_begin(last, n_pairs, p.units) > uu) --last;
        bool got = true;
        if (lead) {
          for (int h = pair + 1; h <= last && got; ++h) {
            const unsigned *f = p.flags + 2 * h + (int)rank;
            got = false;
            for (long long it = 0; it < ab.limit && !got; ++it) {
              got = pf_ld_acquire(f) != 0u;
              if (!got && (it & 15) == 15) {
                if (ab.set()) break;
                __nanosleep(64);
              }
            }
          }
          if (!got && !ab.set()) ab.raise();
        }
        if (!pf_epi_vote(got && !ab.set())) break;
      }
      // The other holders' partial tiles, in ascending K order.  This is the last piece of the range, so the
      // activation ring (4 x 32 KB = one partial tile of this CTA) is free: a partial tile comes in as four bulk
      // copies and is added to the accumulator in tensor memory from shared memory -- read straight from L2,
      // sixteen loads at a time per thread, a tile took 6 us.
      bool alive = true;
      for (int h = pair + 1; h <= last && alive; ++h) {
        if (lead) {
          const float *src = p.partials + (long long)(2 * h + (int)rank) * kSlotFloats;
          mbar_arrive_expect_tx(bar_merge, (uint32_t)(kSlotFloats * sizeof(float)));
          for (int q = 0; q < kPfStages; ++q)
            bulk_copy_g2s(x_ring + q * kPfXSlotBytes, src + (long long)q * (kPfXSlotBytes / 4), kPfXSlotBytes, bar_merge);
        }
        const bool landed = ab.wait_local(bar_merge, merge_phase);
        merge_phase ^= 1u;
        if (lead && landed) p.flags[2 * h + (int)rank] = 0u;    // fetched: the slot is free for the next launch
        if (!pf_epi_vote(landed && !ab.set())) {
          alive = false;
          break;
        }
        for (int c0 = c_begin; c0 < c_begin + kPfRows && tok0 + c0 < p.M; c0 += 16) {
          uint32_t v[16];
          tmem_ld16(lane_addr + c0, v);
          const uint32_t sp = x_ring + (uint32_t)((c0 * kTileN + n) * 4);
          float w[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) w[e] = __uint_as_float(lds32(sp + e * kTileN * 4));
          tc_wait_ld();
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__fadd_rn(__uint_as_float(v[e]), w[e]));
          tmem_st16(lane_addr + c0, v);
        }
        tc_wait_st();
        pf_epi_vote(true);                                     // everybody has read the tile: the next one may land
      }
      if (!alive) break;
      // (the load of the next sixteen tokens is in flight while these are rounded and stored)
      __half *y_col = p.y + (n_ok ? n_glob : 0);
      const int c_end = min(c_begin + kPfRows, ((p.M - tok0 + 15) / 16) * 16);
      uint32_t va[16], vb[16];
      if (c_begin < c_end) tmem_ld16(lane_addr + c_begin, va);
      for (int c0 = c_begin; c0 < c_end; c0 += 32) {
        tc_wait_ld();
        if (c0 + 16 < c_end) tmem_ld16(lane_addr + c0 + 16, vb);
        pf_store_rows(va, y_col, tok0 + c0, p.M, p.ldy, n_ok);
        if (c0 + 16 < c_end) {
          tc_wait_ld();
          if (c0 + 32 < c_end) tmem_ld16(lane_addr + c0 + 32, va);
          pf_store_rows(vb, y_col, tok0 + c0 + 16, p.M, p.ldy, n_ok);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(bar_d_empty, 0));
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_arrive();     // the leader's MMAs write the peer's tensor memory, the peer arrives on the leader's barriers
  cluster_wait();
  if (warp == 2) {
    __syncwarp();
    tmem_dealloc_pair<kPfTmemCols>(tmem);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn prefill_encode_fn() {
  static const EncodeTiledFn fn = [] {                       // thread-safe: initialised once
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

int prefill_set_attrs(void (*kern)(PfParams)) {
  if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess ||
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

std::mutex g_pf_mu;
bool g_pf_attr_done[64] = {};                                // per device, both code widths at once

int prefill_prepare_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ROSAQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_pf_mu);
  if (!g_pf_attr_done[dev]) {
    if (prefill_set_attrs(linear_prefill_kernel<4>) != ROSAQ_OK || prefill_set_attrs(linear_prefill_kernel<3>) != ROSAQ_OK)
      return ROSAQ_ERR_CUDA;
    g_pf_attr_done[dev] = true;
  }
  return ROSAQ_OK;
}

void prefill_config(cudaLaunchConfig_t *cfg, cudaLaunchAttribute *attr, int n_pairs, cudaStream_t s) {
  cfg->gridDim = dim3(2 * n_pairs);
  cfg->blockDim = dim3(kPfThreads);
  cfg->dynamicSmemBytes = kPfSmemBytes;
  cfg->stream = s;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeCooperative;               // all pairs resident: the waits between pairs cannot starve
  attr[1].val.cooperative = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 2;
}

// pairs of CTAs that the device keeps resident at once (an SM without a free neighbour in its GPC cannot
// host half a pair); 0 when the query fails
int prefill_pairs(rosaq_ctx *ctx) {
  if (ctx->pf_pairs > 0) return ctx->pf_pairs;
  if (prefill_prepare_device() != ROSAQ_OK) return 0;
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[2];
  prefill_config(&cfg, attr, ctx->sm_count / 2, nullptr);
  cfg.numAttrs = 1;                                          // (the cluster shape only)
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, linear_prefill_kernel<4>, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    return 0;
  }
  if (clusters > ctx->sm_count / 2) clusters = ctx->sm_count / 2;
  ctx->pf_pairs = clusters;
  return clusters;
}

int prefill_launch(void (*kern)(PfParams), const PfParams &p, int n_pairs, cudaStream_t s) {
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[2];
  prefill_config(&cfg, attr, n_pairs, s);
  if (cudaLaunchKernelEx(&cfg, kern, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

}  // namespace

// Shapes this kernel takes: a dense operand with quantized groups (a weight), no column map.
bool prefill_supported(const TiledOperand &t, const int32_t *col_map) {
  return t.block_groups == 0 && t.g_quant > 0 && col_map == nullptr && (t.bits == 3 || t.bits == 4);
}

int launch_linear_prefill(rosaq_ctx *ctx, const __half *x, int M, long long ldx, const TiledOperand &t, __half *y,
                          long long ldy, cudaStream_t s) {
  EncodeTiledFn encode = prefill_encode_fn();
  if (!encode) return ROSAQ_ERR_CUDA;
  if (!prefill_supported(t, nullptr) || M < 1) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  const int max_pairs = prefill_pairs(ctx);
  if (max_pairs < 1) return ROSAQ_ERR_CUDA;
  PfParams p{};
  // {64 channels, tokens, 64-channel block} view of the row-major activations, box = one group (two blocks) of
  // 128 tokens; rows past M are zero-filled by the copy
  const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(t.d_in / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)ldx * sizeof(__half), 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)kPfRows, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  if (encode(&p.xmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half *>(x), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return ROSAQ_ERR_CUDA;
  p.blob = t.blob;
  p.y = y;
  p.tile_stride = t.tile_stride;
  p.ldy = ldy;
  p.d_out = t.d_out;
  p.n_tiles = t.n_tiles;
  p.g_fp16 = t.g_fp16;
  p.groups = groups_per_tile(t);
  p.n_col_pairs = (t.n_tiles + 1) / 2;
  p.n_tok_blocks = (M + kPfTokens - 1) / kPfTokens;
  p.M = M;
  const long long units = (long long)p.n_col_pairs * p.n_tok_blocks * p.groups;
  if (units < 1 || units > (1ll << 30)) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  p.units = (int)units;
  const int n_pairs = units < max_pairs ? (int)units : max_pairs;
  // one slot of 2 x 256 x 128 floats per pair, in the workspace of the persistent launch (launches of one
  // context do not overlap on the GPU)
  if (ctx->pl_partial_bytes < (size_t)n_pairs * 2 * kPfTokens * kTileN * sizeof(float)) return ROSAQ_ERR_ALLOC;
  p.partials = ctx->pl_partials;
  p.flags = ctx->pf_flags;
  p.status = ctx->d_status;
  p.wait_limit = ctx->wait_limit;
  return t.bits == 4 ? prefill_launch(linear_prefill_kernel<4>, p, n_pairs, s)
                     : prefill_launch(linear_prefill_kernel<3>, p, n_pairs, s);
}

}  // namespace rosaq
