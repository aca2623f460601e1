// One persistent launch for a list of GEMM-stage problems  y = x . W^  (Eq. 3; x . R of Eq. 2 / Eq. 6 is the
// same contraction with R's fp16 tiles as the operand), for up to 64 tokens.
//
// Why.  At decode sizes a single linear streams its weights in a microsecond or two, less than what a
// launch spends filling its pipeline, draining its accumulators and exchanging split-K partial sums.
// Here all linears of a list -- a rotation and the linears that consume it, or every linear of a decoder
// layer -- run in ONE grid of one CTA per SM.  The list is cut into phases (a problem whose input is the
// output of another one runs in the phase after it); inside a phase the tile-major (problem, column tile,
// 128-channel group) list is cut into one contiguous range of equal cost per CTA.  A CTA walks through
// its ranges phase by phase:
//   * the packed-weight ring never drains: the producer warp streams on across tile, problem and phase
//     boundaries (weights depend on nothing);
//   * two accumulators in tensor memory alternate between consecutive pieces (a piece = the groups of one
//     column tile that a CTA holds), so the MMA warp starts the next piece while four epilogue warps
//     drain the previous one;
//   * a column tile whose groups are spread over several CTAs is summed through a workspace in L2: every
//     holder stores its fp32 partial tile and counts itself in; the holders for which this tile is the
//     last piece of their range ("closers") wait for the count, then each adds the partial tiles of a
//     share of the token rows, in ascending K order whatever the timing, and writes those rows of y.
//     Closers come to the tile at the end of their range, the other holders at the beginning of theirs,
//     so nobody waits long;
//   * a problem that reads another problem's output waits (activation producer only) until every tile of
//     that output has been written, counted in a per-problem counter.
// The launch is cooperative (one CTA per SM), so the whole grid is resident and every wait is on work
// that some resident CTA performs without waiting for anything later in the list.
// Every wait is bounded: when a limit expires the CTA records ROSAQ_ERR_TIMEOUT in the context's status
// word, stops issuing work, lets its copies and MMAs in flight finish, frees its tensor memory and
// returns.  The last CTA to leave clears the counters, so the next launch starts from zero whatever
// happened.
//
// One CTA owns an SM.  A tcgen05.mma of 128 x N x 16 costs 55 cycles of the tensor pipe for every N <= 64
// (measured back to back), eight of them per 128-channel group: 440 cycles, 542 with the group's commit,
// against 375 cycles for the group's bytes from HBM.  Two CTAs per SM only take turns on that pipe and
// lengthen each other's dequantise -> MMA -> release chain; one CTA with one issuing thread spent 900
// cycles per group in place, with TWO issuing threads 700: groups with an even position in the CTA's stream
// accumulate into one tile, odd ones into another, and the epilogue adds the two.  Instruction issue
// comes next (1700 warp instructions per group = 430 cycles of the four schedulers), which is why every
// role walks only over its own groups and the epilogue loops carry no per-element address arithmetic.
// Warp 0 = weight-tile producer (bulk copies, L2 evict-first; one sub-ring of slots per team), 1 =
// activation producer (TMA), 2 and 3 = MMA issuers (2 also owns the tensor memory), 4..19 = four
// dequantisation teams (group j goes to team and operand buffer j mod 4), 20..27 = epilogue (two warps per
// TMEM lane quadrant, half of the tokens each).  Tensor memory (512 columns): accumulators of piece parity b
// and issuer i at (2b + i) * 64, operand buffers from 256.
#include <cuda.h>

#include <algorithm>
#include <new>
#include <vector>

#include "linear_common.cuh"

namespace rosaq {

namespace {

constexpr int kPlTmemCols = 512;
constexpr int kPlTeams = 4;                         // dequantisation teams of four warps
constexpr int kPlStages = kPlTeams;                 // TMEM operand buffers, each with its activation slot: one per team ...
constexpr int kPlPairStages = 6;                    // ... six in a pair of CTAs (one issuing thread, two accumulators)
constexpr int kPlMaxStages = 6;
constexpr int kPlTokens = 64;                       // token capacity of an accumulator and of a partial tile
constexpr int kPlFirstDequantWarp = 4, kPlFirstEpiWarp = kPlFirstDequantWarp + 4 * kPlTeams;
constexpr int kPlEpiThreads = 256;                  // two warps per TMEM lane quadrant
constexpr int kPlThreads = kPlFirstEpiWarp * 32 + kPlEpiThreads;   // 896
constexpr int kPlSmemBytes = 227 * 1024;            // the whole SM

struct PlProblem {
  const uint8_t *blob;
  __half *y;
  const int32_t *col_map;
  long long tile_stride, ldy;
  int d_out, n_tiles, g_fp16, block_groups;
  int dep;                    // problem whose output this one reads, or -1
  unsigned dep_target;        // finishing events that complete problem `dep`
  int signal;                 // some problem reads this one's output: count finishing events
  int m;                      // token rows of this problem (<= the launch's token capacity)
};

struct alignas(64) PlParams {
  CUtensorMap xmap[kPlanMaxOps];
  PlProblem prob[kPlanMaxOps];
  const PlanSeg *segs;
  const int *seg_begin;       // [CTAs + 1]
  float *partials;            // [slot][token][128 columns]
  unsigned *sync;             // kPlSyncFinished, kPlSyncDone + problem, kPlSyncArrive + counter
  int *status;
  long long wait_limit;
  int n_counters, M, MT, NW, slot_floats;
};

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *ptr) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_copy_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ PlanSeg load_seg(const PlanSeg *s) {
  PlanSeg r;
  const int4 *q = reinterpret_cast<const int4 *>(s);
  int4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
  r.prob = a.x, r.tile = a.y, r.g_begin = a.z, r.g_end = a.w;
  r.n_contrib = b.x, r.contrib_idx = b.y, r.slot0 = b.z, r.counter = b.w;
  r.closer_idx = c.x, r.n_closers = c.y, r.tok_begin = c.z, r.tok_end = c.w;
  return r;
}
// waits until *ctr >= target; false when the wait gave up
__device__ __forceinline__ bool wait_counter(const Abort &ab, const unsigned *ctr, unsigned target) {
  for (long long it = 0; it < ab.limit; ++it) {
    if (ld_acquire_u32(ctr) >= target) return true;
    if ((it & 15) == 15) {
      if (ab.set()) return false;
      __nanosleep(64);
    }
  }
  if (ld_acquire_u32(ctr) >= target) return true;
  ab.raise();
  return false;
}

template <int CH>
__device__ __forceinline__ void tmem_ld_chunk(uint32_t taddr, uint32_t *v) {
  if (CH == 16) tmem_ld16(taddr, v);
  else tmem_ld8(taddr, v);
}

// Finishes tokens [c_begin, c_end) of one output column from the accumulator in tensor memory: adds, when
// `keep`, the partial tiles 1 .. S-1 of the workspace in that order (this CTA's groups come first), rounds
// once and writes the rows inside [t0, t1).  CH loads from the workspace are in flight per thread.
// Tokens [c0, c0 + CH) of one column: the sum of the two issuers' accumulators (`both`), or the one that
// holds the only group of a one-group piece (d_addr then points at it).
template <int CH>
__device__ __forceinline__ void epi_load_acc(uint32_t d_addr, bool both, int c0, float *acc) {
  uint32_t v[CH];
  tmem_ld_chunk<CH>(d_addr + c0, v);
  tc_wait_ld();
#pragma unroll
  for (int e = 0; e < CH; ++e) acc[e] = __uint_as_float(v[e]);
  if (both) {
    tmem_ld_chunk<CH>(d_addr + kPlTokens + c0, v);
    tc_wait_ld();
#pragma unroll
    for (int e = 0; e < CH; ++e) acc[e] = __fadd_rn(acc[e], __uint_as_float(v[e]));
  }
}

template <int CH>
__device__ __forceinline__ void epi_finish(uint32_t d_addr, bool both, int c_begin, int c_end, bool keep, int S, const float *src0,
                                           long long slot_floats, int M, bool n_ok, int t0, int t1, __half *y_col,
                                           long long ldy) {
  for (int c0 = c_begin; c0 < c_end; c0 += CH) {
    if (c0 >= t1 || c0 + CH <= t0) continue;
    float acc[CH];
    epi_load_acc<CH>(d_addr, both, c0, acc);
    if (keep) {
      // two holders' tiles per round trip to L2 (a round trip costs 1.4 us and more while the weight stream
      // runs, and the readers of this tile wait for it), added in holder order
      for (int i = 1; i < S; i += 2) {
        const float *src = src0 + (long long)i * slot_floats + c0 * kTileN;
        const bool two = i + 1 < S;
        const float *src2 = two ? src + slot_floats : src;
        float w[CH], w2[CH];
        if (c0 + CH <= M) {
#pragma unroll
          for (int e = 0; e < CH; ++e) w[e] = __ldcg(src + e * kTileN);
#pragma unroll
          for (int e = 0; e < CH; ++e) w2[e] = __ldcg(src2 + e * kTileN);
        } else {
#pragma unroll
          for (int e = 0; e < CH; ++e) w[e] = c0 + e < M ? __ldcg(src + e * kTileN) : 0.f;
#pragma unroll
          for (int e = 0; e < CH; ++e) w2[e] = c0 + e < M ? __ldcg(src2 + e * kTileN) : 0.f;
        }
#pragma unroll
        for (int e = 0; e < CH; ++e) acc[e] = __fadd_rn(acc[e], w[e]);
        if (two) {
#pragma unroll
          for (int e = 0; e < CH; ++e) acc[e] = __fadd_rn(acc[e], w2[e]);
        }
      }
    }
    __half *yp = y_col + (long long)c0 * ldy;
    if (n_ok && c0 >= t0 && c0 + CH <= t1) {                  // the usual case: the whole batch is written
#pragma unroll
      for (int e = 0; e < CH; ++e, yp += ldy) *yp = __float2half_rn(acc[e]);
    } else {
#pragma unroll
      for (int e = 0; e < CH; ++e, yp += ldy) {
        const int mg = c0 + e;
        if (n_ok && mg >= t0 && mg < t1) *yp = __float2half_rn(acc[e]);
      }
    }
  }
}

// Stores tokens [c_begin, c_end) of one column of the accumulator to a partial tile [token][128 columns].
template <int CH>
__device__ __forceinline__ void epi_store_partial(uint32_t d_addr, bool both, int c_begin, int c_end, int M, float *dst) {
  for (int c0 = c_begin; c0 < c_end && c0 < M; c0 += CH) {
    float acc[CH];
    epi_load_acc<CH>(d_addr, both, c0, acc);
    float *dp = dst + c0 * kTileN;
    if (c0 + CH <= M) {
#pragma unroll
      for (int e = 0; e < CH; ++e) dp[e * kTileN] = acc[e];
    } else {
#pragma unroll
      for (int e = 0; e < CH; ++e)
        if (c0 + e < M) dp[e * kTileN] = acc[e];
    }
  }
}

// kPair: the CTAs of a cluster of two (ranks 0 and 1, adjacent SMs) run as a cta_group::2 pair on one
// schedule entry: a piece is then the groups of TWO adjacent column tiles, rank r dequantises tile 2 t + r into
// its own tensor memory and loads half of the token rows, and the leader (rank 0) issues one M = 256 MMA for
// both.  An MMA instruction costs the same 55 cycles whether it covers 128 or 256 rows, so the pair needs
// 222 cycles of each SM's tensor pipe per 128-channel group where a single CTA needs 440 -- less than the
// 375 cycles the group's bytes take.  Barriers that both CTAs feed live in the leader; its commits are
// multicast to both.
// kMode 2: a single CTA with accumulators of 128 tokens: two of them (one per piece parity) and the four
// operand buffers fill the tensor memory, so there is one issuing thread, as in a pair; a group then costs
// eight MMAs of N = 128 (64 cycles each: the full rate of the pipe) and its dequantisation serves twice the tokens.
template <int kBits, int kMode>
__global__ void __launch_bounds__(kPlThreads, 1)
linear_plan_kernel(const __grid_constant__ PlParams p) {
  constexpr bool kPair = kMode == 1, kBig = kMode == 2, kOne = kMode != 0;
  constexpr int kTok = kBig ? 2 * kPlTokens : kPlTokens;       // token capacity of an accumulator
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int MT = p.MT;
  const int MTL = kPair ? MT >> 1 : MT;                        // token rows this CTA keeps in shared memory
  const uint32_t x_slot_bytes = (uint32_t)MTL * 256u;
  const uint32_t x_ring = base;
  // operand buffers: a single CTA has two issuing threads with an accumulator each per piece parity (256
  // columns) and one buffer per team; a pair has one issuing thread (an MMA over both SMs costs no more than
  // one over one) and spends the columns on two more buffers, which hides the longer chain of a pair
  // (dequantise -> remote arrive -> MMA -> multicast commit)
  constexpr int NS = kPair ? kPlPairStages : kPlStages;
  const uint32_t w_ring = x_ring + NS * x_slot_bytes;
  const uint32_t bars = w_ring + p.NW * kWSlotBytes;
  const uint32_t bar_w_full = bars, bar_w_empty = bar_w_full + 8 * p.NW;
  const uint32_t bar_a_full = bar_w_empty + 8 * p.NW;          // operand buffer written + activation slot landed
  const uint32_t bar_s_empty = bar_a_full + 8 * kPlMaxStages;  // stage consumed by its MMAs
  const uint32_t bar_d_full = bar_s_empty + 8 * kPlMaxStages;  // accumulator complete (two accumulators)
  const uint32_t bar_d_empty = bar_d_full + 16;                // accumulator drained
  const uint32_t bar_drain = bar_d_empty + 16;                 // two: one per issuer
  const uint32_t misc = bar_drain + 16;                         // [0] TMEM base, [1] abort flag, [2] last CTA out
  uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t *misc_ptr = reinterpret_cast<volatile uint32_t *>(gen + (misc - base));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? (blockIdx.x & 1u) : 0u;        // position in the pair; 0 = leader
  const bool is_lead = rank == 0;
  const int cta = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;   // entry of the schedule
  const int s_begin = p.seg_begin[cta], s_end = p.seg_begin[cta + 1];
  const Abort ab{reinterpret_cast<volatile int *>(misc_ptr + 1), p.status, p.wait_limit, kPair};
  const int tile_mul = kPair ? 2 : 1;                          // this CTA's column tile of a piece: tile_mul * tile + rank

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.NW; ++i) {
      mbar_init(bar_w_full + 8 * i, 1);
      mbar_init(bar_w_empty + 8 * i, kTeamThreads);
    }
    for (int i = 0; i < NS; ++i) {
      // a team's arrivals (per thread; in a pair per warp, from both CTAs) + the activation copy
      mbar_init(bar_a_full + 8 * i, (kPair ? 2 * (kTeamThreads / 32) : kTeamThreads) + 1);
      mbar_init(bar_s_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_d_full + 8 * i, kOne ? 1 : 2);             // the issuing threads
      mbar_init(bar_d_empty + 8 * i, (kPair ? 2 : 1) * (kPlEpiThreads / 32));   // one arrival per epilogue warp
      mbar_init(bar_drain + 8 * i, 1);
    }
    misc_ptr[1] = 0;
    misc_ptr[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {
    if (kPair) tmem_alloc_pair<kPlTmemCols>(misc);             // both CTAs of the pair, same warp index
    else tmem_alloc<kPlTmemCols>(misc);
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) {                                                 // the peer's barriers and tensor memory exist
    cluster_arrive();
    cluster_wait();
  }
  tc_fence_after();
  const uint32_t tmem = misc_ptr[0];
  const uint32_t a_col0 = (kPair ? 2 : 4) * kPlTokens;         // operand buffers follow the accumulators (two of 128 columns when kBig)
  const int qbytes = quant_tile_bytes(kBits);

  if (warp == 0) {
    // ---------------- weight-tile producer: streams every piece of every phase, waits for ring slots only
    if (lane == 0) {
      // The ring is split into one sub-ring of NWT slots per dequantisation team (group j of the CTA's stream
      // belongs to team j mod 4): a sub-ring has one consumer, which takes its slots in order, so a full /
      // empty pair of barriers per slot is enough.  Positions of the four sub-rings: a byte each in idx4,
      // a bit each in lap4; fills per team in fills4 (16 bits each, only looked at when giving up).
      const uint64_t pol = policy_evict_first();
      const int NWT = p.NW >> 2;
      uint32_t idx4 = 0, lap4 = 0;
      unsigned long long fills4 = 0;
      int j = 0;
      bool live = true;
      for (int si = s_begin; si < s_end && live && !ab.set(); ++si) {
        const PlanSeg s = load_seg(p.segs + si);
        const PlProblem &P = p.prob[s.prob];
        // (the second CTA of a pair on an odd last tile streams that tile again; its results are dropped)
        int my_tile = tile_mul * s.tile + (int)rank;
        if (my_tile >= P.n_tiles) my_tile = P.n_tiles - 1;
        const uint8_t *tile_base = P.blob + (long long)my_tile * P.tile_stride;
        const int g_fp16 = P.g_fp16;
        for (int g = s.g_begin; g < s.g_end && live; ++g, ++j) {
          const bool f16 = g < g_fp16;
          const uint8_t *src = tile_base + (f16 ? (long long)g * kFp16TileBytes
                                                : (long long)g_fp16 * kFp16TileBytes + (long long)(g - g_fp16) * qbytes);
          const int nsub = f16 ? 4 : 1;
          const uint32_t bytes = f16 ? kFp16SubBytes : qbytes;
          const int team = j & (kPlTeams - 1);
          uint32_t idx = (idx4 >> (8 * team)) & 0xffu;
          for (int sub = 0; sub < nsub; ++sub) {
            const int slot = team * NWT + (int)idx;
            if (!ab.wait_local(bar_w_empty + 8 * slot, ((lap4 >> team) & 1u) ^ 1u)) {
              live = false;
              break;
            }
            mbar_arrive_expect_tx(bar_w_full + 8 * slot, bytes);
            bulk_copy_g2s_hint(w_ring + slot * kWSlotBytes, src + (long long)sub * kFp16SubBytes, bytes,
                               bar_w_full + 8 * slot, pol);
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
        for (int team = 0; team < kPlTeams; ++team) {
          const int f = (int)((fills4 >> (16 * team)) & 0xffffu);     // (mod 65536: only the last NWT fills matter)
          for (int back = 1; back <= NWT && back <= f; ++back) {
            const int u = f - back;
            for (int it = 0; it < kDrainPolls; ++it)
              if (mbar_try_wait(bar_w_full + 8 * (team * NWT + u % NWT), (u / NWT) & 1)) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- activation producer
    if (lane == 0) {
      int gc = 0;
      Ring rs{0, 0};
      int last_prob = -1;
      bool live = true;
      for (int si = s_begin; si < s_end && live && !ab.set(); ++si) {
        const PlanSeg s = load_seg(p.segs + si);
        const PlProblem &P = p.prob[s.prob];
        if (s.prob != last_prob) {
          last_prob = s.prob;
          if (P.dep >= 0) {
            // the input is another problem's output: every tile of it must have been written (by generic
            // stores of other CTAs, read here by the copy engine: hence the proxy fence after the acquire)
            if (!wait_counter(ab, p.sync + kPlSyncDone + P.dep, P.dep_target)) break;
            asm volatile("fence.proxy.async;" ::: "memory");
          }
        }
        // block-diagonal operand: a column tile only multiplies the channels of its own diagonal block
        const int g_block0 = P.block_groups > 0 ? ((tile_mul * s.tile + (int)rank) / P.block_groups) * P.block_groups : 0;
        const CUtensorMap *map = &p.xmap[s.prob];
        for (int g = s.g_begin; g < s.g_end; ++g, ++gc, rs.advance(NS)) {
          const int slot = rs.idx;
          if (!ab.wait(bar_s_empty + 8 * slot, rs.lap ^ 1u)) {
            live = false;
            break;
          }
          const int k0 = (g_block0 + g) * kGroup;
          if (kPair) {
            // each CTA loads its half of the token rows; all bytes are counted on the leader's barrier
            if (is_lead) mbar_arrive_expect_tx(bar_a_full + 8 * slot, 2 * x_slot_bytes);
            tma_load_3d_pair(x_ring + slot * x_slot_bytes, map, map_to_rank(bar_a_full + 8 * slot, 0), (int)rank * MTL, k0 >> 6);
          } else {
            mbar_arrive_expect_tx(bar_a_full + 8 * slot, x_slot_bytes);
            tma_load_3d(x_ring + slot * x_slot_bytes, map, bar_a_full + 8 * slot, 0, k0 >> 6);
          }
        }
      }
      // (in a pair the leader's barriers count the copies of both CTAs, and the peer stays until the cluster
      // barrier at the end of the kernel, which the leader reaches after this drain)
      if (ab.set() && is_lead) {
        for (int back = 1; back <= NS && back <= gc; ++back) {
          const int u = gc - back;
          for (int it = 0; it < kDrainPolls; ++it)
            if (ab.poll(bar_a_full + 8 * (u % NS), (u / NS) & 1)) break;
        }
      }
    }
  } else if (warp == 2 || warp == 3) {
    // ---------------- MMA issuers: issuer i takes the groups whose position j in the CTA's stream has
    // j mod 2 == i (operand buffers i and i + 2) and accumulates them into its own tile; per group one
    // wait, eight MMAs, one commit.  Every piece is committed by both (an issuer without a group in a
    // one-group piece arrives by hand), so the epilogue waits for one barrier.
    if (lane == 0 && is_lead && !(kOne && warp == 3)) {        // (a pair, or a CTA with wide accumulators, has one issuing thread)
      const int me = warp - 2;
      constexpr int kStep = kOne ? 1 : 2;                      // issuers that share the stream
      // M = 128 output columns (256 for a pair), N = MT tokens
      const uint32_t idesc = (1u << 4) | ((uint32_t)(MT >> 3) << 17) | ((kPair ? 16u : 8u) << 24);
      const uint64_t desc0 = make_b_desc(x_ring);
      const uint32_t x_slot16 = x_slot_bytes >> 4, half16 = (uint32_t)(MTL * 128) >> 4;
      int nseg = 0, j = 0;
      bool live = true, issued = false;
      for (int si = s_begin; si < s_end && live; ++si, ++nseg) {
        const PlanSeg s = load_seg(p.segs + si);
        const int buf = nseg & 1;
        if (!ab.wait(bar_d_empty + 8 * buf, ((nseg >> 1) & 1) ^ 1u)) break;   // the piece before last has been drained
        tc_fence_after();
        const uint32_t d_tmem = tmem + (uint32_t)(kOne ? buf : 2 * buf + me) * kTok;
        uint32_t accumulate = 0;
        const int g_first = kOne ? s.g_begin : s.g_begin + ((me - j) & 1), j_base = j - s.g_begin;
        j += s.g_end - s.g_begin;
        for (int g = g_first; g < s.g_end; g += kStep) {
          const int j = j_base + g;
          const int st = j % NS;                               // (a constant: a mask or a multiply)
          if (!ab.wait(bar_a_full + 8 * st, (uint32_t)(j / NS) & 1u)) {
            live = false;
            break;
          }
          tc_fence_after();
          const uint64_t b0 = desc0 + (uint64_t)(st * x_slot16);
          if (kPair) {
            tc_mma8_ts_pair(d_tmem, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
            tc_commit_mc(bar_s_empty + 8 * st, 3);             // frees the stage in both CTAs
          } else {
            tc_mma8_ts(d_tmem, tmem + a_col0 + st * 64, b0, b0 + (uint64_t)half16, idesc, accumulate);
            tc_commit(bar_s_empty + 8 * st);
          }
          accumulate = 1;
          issued = true;
        }
        if (!live) break;
        if (kPair) {
          if (accumulate) tc_commit_mc(bar_d_full + 8 * buf, 3);
          else {
            mbar_arrive_cluster(map_to_rank(bar_d_full + 8 * buf, 0));
            mbar_arrive_cluster(map_to_rank(bar_d_full + 8 * buf, 1));
          }
        } else {
          if (accumulate) tc_commit(bar_d_full + 8 * buf);
          else mbar_arrive(bar_d_full + 8 * buf);
        }
      }
      if (ab.set() && issued) {  // MMAs already issued must retire before the tensor memory is given back
        if (kPair) tc_commit_mc(bar_drain + 8 * me, 1);
        else tc_commit(bar_drain + 8 * me);
        for (int it = 0; it < kDrainPolls; ++it)
          if (ab.poll(bar_drain + 8 * me, 0)) break;
      }
    }
  } else if (warp >= kPlFirstDequantWarp && warp < kPlFirstEpiWarp) {
    // ---------------- dequantisation: group j of the CTA's stream goes to team and operand buffer j mod 4;
    // a team walks over its own groups only and takes the slots of its own sub-ring in order
    const int quad = warp & 3;
    const int team = (warp - kPlFirstDequantWarp) >> 2;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    const int NWT = p.NW >> 2;
    const uint32_t my_ring = w_ring + team * NWT * kWSlotBytes, my_full = bar_w_full + 8 * team * NWT,
                   my_empty = bar_w_empty + 8 * team * NWT;

    Ring rw{0, 0};
    bool ok = true;
    int j0 = 0;                                      // position of the piece's first group in the CTA's stream
    for (int si = s_begin; si < s_end && ok; ++si) {
      const PlanSeg s = load_seg(p.segs + si);
      const int g_fp16 = p.prob[s.prob].g_fp16;
      for (int g = s.g_begin + ((team - j0) & (kPlTeams - 1)); g < s.g_end && ok; g += kPlTeams) {
        const bool f16 = g < g_fp16;
        const int nsub = f16 ? 4 : 1;
        const uint32_t j = (uint32_t)(j0 + g - s.g_begin);
        const uint32_t st = j % NS, use = j / NS;                          // the group's buffer; how often it was used before
        const uint32_t a_addr = lane_addr + a_col0 + st * 64;
        const uint32_t my_s_empty = bar_s_empty + 8 * st, my_a_full = bar_a_full + 8 * st;
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
        if (kPair) {                                           // one arrival per warp, on the leader's barrier
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(map_to_rank(my_a_full, 0));
        } else {
          mbar_arrive(my_a_full);
        }
      }
      j0 += s.g_end - s.g_begin;
    }
  } else if (warp >= kPlFirstEpiWarp) {
    // ---------------- epilogue: one pass per piece.  Thread = (output column n of the tile = TMEM lane,
    // half of the tokens = TMEM columns).  Loads from the workspace are issued in batches before they are
    // used: the exchange is bound by L2 latency, not by bandwidth.
    const int quad = warp & 3;
    const int n = quad * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
    const bool lead = threadIdx.x == kPlFirstEpiWarp * 32;
    const int half_tok = MT >> 1;
    const int c_begin = ((warp - kPlFirstEpiWarp) >> 2) * half_tok, c_end = c_begin + half_tok;
    const bool wide = (half_tok & 15) == 0;                    // sixteen tokens per batch, else eight
    int nseg = 0, j0 = 0;
    for (int si = s_begin; si < s_end; ++si, ++nseg) {
      const PlanSeg s = load_seg(p.segs + si);
      const PlProblem &P = p.prob[s.prob];
      const int buf = nseg & 1;
      // the piece's groups have positions j0 .. in the CTA's stream: even ones went to issuer 0's tile
      const bool both = !kOne && s.g_end - s.g_begin > 1;
      const int first_acc = (both || kOne) ? 0 : (j0 & 1);
      j0 += s.g_end - s.g_begin;
      bool have_d = ab.wait(bar_d_full + 8 * buf, (nseg >> 1) & 1);
      have_d = __all_sync(0xffffffffu, have_d && !ab.set());
      if (!have_d) break;
      tc_fence_after();
      const uint32_t d_addr = lane_addr + (uint32_t)(kOne ? buf : 2 * buf + first_acc) * kTok;
      const int n_glob = (tile_mul * s.tile + (int)rank) * kTileN + n;
      const bool n_ok = n_glob < P.d_out;
      const long long out_col = n_ok ? (P.col_map ? P.col_map[n_glob] : n_glob) : 0;
      __half *const y_out = P.y;
      const long long ldy = P.ldy;
      const int S = s.n_contrib;
      const bool sole = S == 1;
      // the only closer of a shared tile (it holds the tile's first groups) keeps its accumulator and adds
      // the other holders' partial tiles to it
      const bool keep = !sole && s.n_closers == 1 && s.closer_idx == 0;
      // (the two CTAs of a pair exchange their own tiles: slots and counters are interleaved by rank)
      unsigned *ctr = p.sync + kPlSyncArrive + tile_mul * s.counter + rank;
      const long long slot_step = (long long)tile_mul * p.slot_floats;            // from one holder's slot to the next
      const float *src0 = p.partials + ((long long)tile_mul * s.slot0 + rank) * p.slot_floats + n;
      if (keep) {
        if (lead) wait_counter(ab, ctr, (unsigned)(S - 1));
        epi_bar();
        if (ab.set()) break;
      }
      if (sole || keep) {
        // token rows this piece writes (the schedule counts them in 64ths of the capacity)
        const int t0 = s.tok_begin * (kTok / kPlTokens), t1 = min(s.tok_end * (kTok / kPlTokens), P.m);
        if (wide) epi_finish<16>(d_addr, both, c_begin, c_end, keep, S, src0, slot_step, P.m, n_ok, t0, t1, y_out + out_col, ldy);
        else epi_finish<8>(d_addr, both, c_begin, c_end, keep, S, src0, slot_step, P.m, n_ok, t0, t1, y_out + out_col, ldy);
        tc_fence_before();
        __syncwarp();                                          // one arrival per warp, where the issuers wait
        if (lane == 0) {
          if (kPair) mbar_arrive_cluster(map_to_rank(bar_d_empty + 8 * buf, 0));
          else mbar_arrive(bar_d_empty + 8 * buf);
        }
        if (P.signal) {
          epi_bar();                                           // all stores of the CTA are issued ...
          if (lead) {
            __threadfence();                                   // ... and ordered before the count (cumulative fence)
            atomicAdd(p.sync + kPlSyncDone + s.prob, 1u);
          }
        }
        continue;
      }
      // store the partial tile [token][column] (a warp writes 128 contiguous bytes per token), give the
      // accumulator back, count this CTA in
      {
        float *dst = p.partials + ((long long)tile_mul * (s.slot0 + s.contrib_idx) + rank) * p.slot_floats + n;
        if (wide) epi_store_partial<16>(d_addr, both, c_begin, c_end, P.m, dst);
        else epi_store_partial<8>(d_addr, both, c_begin, c_end, P.m, dst);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(map_to_rank(bar_d_empty + 8 * buf, 0));
        else mbar_arrive(bar_d_empty + 8 * buf);
      }
      epi_bar();
      if (lead) {
        __threadfence();
        atomicAdd(ctr, 1u);
      }
      if (s.closer_idx < 0) continue;
      // one of several closers: when every holder has stored its partial tile, add them for token rows
      // closer_idx, closer_idx + n_closers, ... in ascending K order and write those rows of y
      if (lead) wait_counter(ab, ctr, (unsigned)S);
      epi_bar();
      if (ab.set()) break;
      {
        // (the two warps of a quadrant take alternate batches of eight rows; 32 loads are in flight per
        // thread and round; a holder index past S adds +0, which changes nothing)
        const int nc = s.n_closers;
        const int t0 = s.tok_begin * (kTok / kPlTokens), t1 = min(s.tok_end * (kTok / kPlTokens), P.m);
        for (int r0 = s.closer_idx + ((warp - kPlFirstEpiWarp) >> 2) * 8 * nc; r0 < t1; r0 += 16 * nc) {
          float acc[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) acc[u] = 0.f;
          for (int i = 0; i < S; i += 4) {
            float w[8][4];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int r = r0 + u * nc;
#pragma unroll
              for (int k = 0; k < 4; ++k)
                w[u][k] = (r < t1 && i + k < S) ? __ldcg(src0 + (long long)(i + k) * slot_step + r * kTileN) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
              for (int k = 0; k < 4; ++k) acc[u] = __fadd_rn(acc[u], w[u][k]);
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int r = r0 + u * nc;
            if (n_ok && r >= t0 && r < t1) y_out[(long long)r * ldy + out_col] = __float2half_rn(acc[u]);
          }
        }
      }
      if (P.signal) {
        epi_bar();
        if (lead) {
          __threadfence();
          atomicAdd(p.sync + kPlSyncDone + s.prob, 1u);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (kPair) {          // the leader's MMAs write the peer's tensor memory, the peer arrives on the leader's barriers
    cluster_arrive();
    cluster_wait();
  }
  if (warp == 2) {
    __syncwarp();
    if (kPair) tmem_dealloc_pair<kPlTmemCols>(tmem);
    else tmem_dealloc<kPlTmemCols>(tmem);
  }
  // the last CTA to leave puts every counter back to zero for the next launch
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned old = atomicAdd(p.sync + kPlSyncFinished, 1u);
    __threadfence();
    misc_ptr[2] = old == gridDim.x - 1 ? 1u : 0u;
  }
  __syncthreads();
  if (misc_ptr[2]) {
    for (int i = threadIdx.x; i < p.n_counters; i += kPlThreads) p.sync[kPlSyncArrive + i] = 0;
    if (threadIdx.x < kPlanMaxOps) p.sync[kPlSyncDone + threadIdx.x] = 0;
    if (threadIdx.x == 0) p.sync[kPlSyncFinished] = 0;
  }
}

// ---------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn plan_encode_fn() {
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

// {64 channels, tokens, 64-channel block} view of the row-major activations, box = one group (two blocks)
// of MT tokens; rows past M are zero-filled by the copy
bool plan_encode_x(CUtensorMap *map, const __half *x, int M, long long ldx, int d_in, int MT) {
  EncodeTiledFn encode = plan_encode_fn();
  if (!encode) return false;
  const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(d_in / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)ldx * sizeof(__half), 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)MT, 2};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half *>(x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ring depth and shared memory for MTL token rows per CTA
int plan_nw(int MTL, int ns) {
  const int budget = kPlSmemBytes - 1024 - ns * MTL * 256 - 512;
  const int nw = (budget / kWSlotBytes) & ~3;          // four sub-rings of equal depth, one per team
  return nw > 20 ? 20 : nw;
}

size_t plan_smem_bytes(int MTL, int NW, int ns) {
  return 1024 + (size_t)ns * MTL * 256 + (size_t)NW * kWSlotBytes + 8 * (2 * NW + 2 * kPlMaxStages + 6) + 16;
}

template <typename K>
int plan_set_attrs(K kern, size_t smem) {
  if (cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess ||
      cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------- the cut
// Phases: a problem without a dependency is in phase 0, otherwise one phase after the problem it reads.
// Inside a phase the (problem, tile, group) list, problems in the order given, is cut into n_ctas
// contiguous ranges of equal cost (cost[0] per fp16 group, cost[1] per quantized group, cost[2] per tile
// started, for its epilogue); a range may be empty when a phase has little work.
int plan_build_schedule(const std::vector<PlanGeom> &ops, int n_ctas, const int *cost, PlanSchedule *out) {
  const int n = (int)ops.size();
  if (n < 1 || n > kPlanMaxOps || n_ctas < 1) return ROSAQ_ERR_INVALID_ARG;
  std::vector<int> phase(n, 0);
  int n_phases = 1;
  for (int i = 0; i < n; ++i) {
    if (ops[i].n_tiles < 1 || ops[i].groups < 1 || ops[i].g_fp16 < 0 || ops[i].g_fp16 > ops[i].groups) return ROSAQ_ERR_INVALID_ARG;
    if (ops[i].rep < 1 || ops[i].rep > 16) return ROSAQ_ERR_INVALID_ARG;
    if (ops[i].dep >= i) return ROSAQ_ERR_INVALID_ARG;
  }
  // Phases: an operation runs after the one whose output it reads.  Operations that neither read nor feed
  // another one go BETWEEN the producers and their consumers: while the CTAs work through them, the
  // epilogue warps close the producers' shared tiles in the background (partial tiles through L2, counters:
  // 6 to 9 us on a 7B layer), so that the consumers' activation copies find those outputs complete.
  std::vector<char> feeds(n, 0);
  bool any_dep = false, any_free = false;
  for (int i = 0; i < n; ++i)
    if (ops[i].dep >= 0) feeds[ops[i].dep] = 1, any_dep = true;
  for (int i = 0; i < n; ++i) any_free = any_free || (ops[i].dep < 0 && !feeds[i]);
  const int step = any_dep && any_free ? 2 : 1;
  for (int i = 0; i < n; ++i) {
    if (ops[i].dep >= 0) phase[i] = phase[ops[i].dep] + step;
    else phase[i] = (step == 2 && !feeds[i]) ? 1 : 0;
    n_phases = std::max(n_phases, phase[i] + 1);
  }
  std::vector<std::vector<PlanSeg>> per_cta(n_ctas);
  out->done_target.assign(n, 0u);
  out->n_counters = 0;
  out->n_slots = 0;
  struct Holder {
    int cta, seg;      // position in per_cta[cta]
    bool last;         // the last piece of that CTA's range in this phase
  };
  for (int ph = 0; ph < n_phases; ++ph) {
    // unit u of the phase: (op, tile, group); prefix[u] = cost of the units before u
    struct Tile {
      int op, tile, copy;      // copy: which of the op's `rep` replicas of this tile (each writes a share of the token rows)
      long long first_unit;
    };
    std::vector<Tile> tiles;
    long long n_units = 0;
    for (int i = 0; i < n; ++i) {
      if (phase[i] != ph) continue;
      for (int t = 0; t < ops[i].n_tiles; ++t)
        for (int r = 0; r < ops[i].rep; ++r) {
          tiles.push_back(Tile{i, t, r, n_units});
          n_units += ops[i].groups;
        }
    }
    if (n_units == 0) continue;
    if (n_units > 0x3fffffffll) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
    std::vector<long long> prefix((size_t)n_units + 1);
    {
      long long c = 0;
      size_t u = 0;
      for (const Tile &t : tiles) {
        const PlanGeom &g = ops[t.op];
        for (int k = 0; k < g.groups; ++k, ++u) {
          prefix[u] = c;
          c += (k < g.g_fp16 ? cost[0] : cost[1]) + (k == 0 ? (g.tile_cost > 0 ? g.tile_cost : cost[2]) : 0);
        }
      }
      prefix[u] = c;
    }
    const long long total = prefix[(size_t)n_units];
    std::vector<long long> bounds(n_ctas + 1);
    for (int i = 0; i <= n_ctas; ++i) {
      // first unit whose preceding cost reaches i / n_ctas of the total
      const long long want = (total * i + n_ctas - 1) / n_ctas;
      bounds[i] = std::lower_bound(prefix.begin(), prefix.end(), want) - prefix.begin();
      if (bounds[i] > n_units) bounds[i] = n_units;
    }
    bounds[0] = 0;
    bounds[n_ctas] = n_units;
    std::vector<std::vector<Holder>> holders(tiles.size());
    size_t ti = 0;
    for (int c = 0; c < n_ctas; ++c) {
      long long u = bounds[c];
      const long long end = bounds[c + 1];
      while (u < end) {
        while (ti + 1 < tiles.size() && tiles[ti + 1].first_unit <= u) ++ti;
        const Tile &t = tiles[ti];
        const long long tile_end = t.first_unit + ops[t.op].groups;
        const long long stop = std::min(end, tile_end);
        PlanSeg s{};
        s.prob = t.op;
        s.tile = t.tile;
        s.g_begin = (int)(u - t.first_unit);
        s.g_end = (int)(stop - t.first_unit);
        s.n_contrib = 1;
        s.closer_idx = -1;
        s.tok_begin = kPlTokens * t.copy / ops[t.op].rep;
        s.tok_end = kPlTokens * (t.copy + 1) / ops[t.op].rep;
        holders[ti].push_back(Holder{c, (int)per_cta[c].size(), stop == end});
        per_cta[c].push_back(s);
        u = stop;
      }
    }
    for (size_t k = 0; k < tiles.size(); ++k) {
      const std::vector<Holder> &h = holders[k];
      if (h.empty()) return ROSAQ_ERR_CUDA;                    // cannot happen: the ranges cover the list
      const int S = (int)h.size();
      if (S == 1) {
        out->done_target[tiles[k].op] += 1u;
        continue;
      }
      int n_closers = 0;
      for (const Holder &x : h) n_closers += x.last ? 1 : 0;
      int ci = 0;
      for (int j = 0; j < S; ++j) {
        PlanSeg &s = per_cta[h[j].cta][h[j].seg];
        s.n_contrib = S;
        s.contrib_idx = j;
        s.slot0 = out->n_slots;
        s.counter = out->n_counters;
        s.n_closers = n_closers;
        s.closer_idx = h[j].last ? ci++ : -1;
      }
      out->n_slots += S;
      out->n_counters += 1;
      out->done_target[tiles[k].op] += (unsigned)n_closers;
    }
  }
  out->segs.clear();
  out->seg_begin.assign(n_ctas + 1, 0);
  for (int c = 0; c < n_ctas; ++c) {
    out->seg_begin[c] = (int)out->segs.size();
    out->segs.insert(out->segs.end(), per_cta[c].begin(), per_cta[c].end());
  }
  out->seg_begin[n_ctas] = (int)out->segs.size();
  out->n_ctas = n_ctas;
  return ROSAQ_OK;
}

template <typename K>
static int plan_launch_kernel(K kern, const PlanLaunch &l, const PlParams &q, size_t smem, cudaStream_t s) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(l.n_ctas, 1, 1);
  cfg.blockDim = dim3(kPlThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeCooperative;        // all CTAs resident: the waits between CTAs cannot starve
  attr[na].val.cooperative = 1;
  ++na;
  if (l.pair) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 2;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  if (cudaLaunchKernelEx(&cfg, kern, q) != cudaSuccess) {
    (void)cudaGetLastError();
    return ROSAQ_ERR_CUDA;
  }
  return ROSAQ_OK;
}

// Entries of the schedule = CTAs (one per SM), or, for pairs, clusters of two CTAs that the device keeps
// resident at once (an SM without a free neighbour in its GPC cannot host half a pair).  0 when pairs are
// not available.
int plan_units(rosaq_ctx *ctx, bool pair) {
  if (ctx->pl_ctas <= 0) {
    if (plan_set_attrs(linear_plan_kernel<4, 0>, kPlSmemBytes) != ROSAQ_OK ||
        plan_set_attrs(linear_plan_kernel<3, 0>, kPlSmemBytes) != ROSAQ_OK ||
        plan_set_attrs(linear_plan_kernel<4, 1>, kPlSmemBytes) != ROSAQ_OK ||
        plan_set_attrs(linear_plan_kernel<3, 1>, kPlSmemBytes) != ROSAQ_OK ||
        plan_set_attrs(linear_plan_kernel<4, 2>, kPlSmemBytes) != ROSAQ_OK ||
        plan_set_attrs(linear_plan_kernel<3, 2>, kPlSmemBytes) != ROSAQ_OK)
      return 0;
    int p = ctx->sm_count;
    if (p > kPlanMaxCtas) p = kPlanMaxCtas;
    ctx->pl_ctas = p;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * (p / 2), 1, 1);
    cfg.blockDim = dim3(kPlThreads);
    cfg.dynamicSmemBytes = kPlSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, linear_plan_kernel<4, 1>, &cfg) != cudaSuccess) {
      (void)cudaGetLastError();
      clusters = 0;
    }
    if (clusters > p / 2) clusters = p / 2;
    ctx->pl_pairs = clusters;
  }
  return pair ? ctx->pl_pairs : ctx->pl_ctas;
}

int plan_ctas(rosaq_ctx *ctx) {
  const int pairs = plan_units(ctx, true);
  return ctx->pl_mode != 1 && pairs > 0 ? 2 * pairs : plan_units(ctx, false);
}

// Looks the schedule of this geometry up in the context's cache, or builds and uploads it.
static int plan_get_schedule(rosaq_ctx *ctx, const std::vector<PlanGeom> &geom, int P, const int *cost,
                             const PlanSchedule **out) {
  if (P <= 0) return ROSAQ_ERR_CUDA;
  for (PlanSchedule *s : ctx->pl_schedules) {
    if (s->n_ctas != P || s->geom.size() != geom.size() || s->cost[0] != cost[0] || s->cost[1] != cost[1] || s->cost[2] != cost[2])
      continue;
    bool same = true;
    for (size_t i = 0; i < geom.size() && same; ++i)
      same = s->geom[i].n_tiles == geom[i].n_tiles && s->geom[i].groups == geom[i].groups && s->geom[i].g_fp16 == geom[i].g_fp16 &&
             s->geom[i].dep == geom[i].dep && s->geom[i].rep == geom[i].rep && s->geom[i].tile_cost == geom[i].tile_cost;
    if (same) {
      *out = s;
      return ROSAQ_OK;
    }
  }
  PlanSchedule *s = new (std::nothrow) PlanSchedule();
  if (!s) return ROSAQ_ERR_ALLOC;
  s->geom = geom;
  for (int i = 0; i < 3; ++i) s->cost[i] = cost[i];
  int st = plan_build_schedule(geom, P, cost, s);
  if (st == ROSAQ_OK && s->n_counters > kPlMaxCounters) st = ROSAQ_ERR_UNSUPPORTED_SHAPE;
  if (st == ROSAQ_OK) {
    const size_t seg_bytes = std::max<size_t>(s->segs.size(), 1) * sizeof(PlanSeg), beg_bytes = (size_t)(P + 1) * sizeof(int);
    if (cudaMalloc(reinterpret_cast<void **>(&s->d_segs), seg_bytes) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void **>(&s->d_seg_begin), beg_bytes) != cudaSuccess) {
      (void)cudaGetLastError();
      st = ROSAQ_ERR_ALLOC;
    } else if ((!s->segs.empty() && cudaMemcpy(s->d_segs, s->segs.data(), s->segs.size() * sizeof(PlanSeg), cudaMemcpyHostToDevice) != cudaSuccess) ||
               cudaMemcpy(s->d_seg_begin, s->seg_begin.data(), beg_bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
      (void)cudaGetLastError();
      st = ROSAQ_ERR_CUDA;
    }
  }
  if (st != ROSAQ_OK) {
    if (s->d_segs) (void)cudaFree(s->d_segs);
    if (s->d_seg_begin) (void)cudaFree(s->d_seg_begin);
    delete s;
    return st;
  }
  ctx->pl_schedules.push_back(s);
  *out = s;
  return ROSAQ_OK;
}

void plan_free_schedules(rosaq_ctx *ctx) {
  for (PlanSchedule *s : ctx->pl_schedules) {
    if (s->d_segs) (void)cudaFree(s->d_segs);
    if (s->d_seg_begin) (void)cudaFree(s->d_seg_begin);
    delete s;
  }
  ctx->pl_schedules.clear();
}

// Checks the ops, finds their schedule, makes sure the exchange workspace is large enough and fills the
// kernel parameters.  May allocate (a new geometry, a larger workspace); launches nothing.
int plan_prepare(rosaq_ctx *ctx, int M, int n, const PlanOp *ops, PlanLaunch *out) {
  if (n < 1 || n > kPlanMaxOps || M < 1 || M > 2 * kPlTokens) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  std::vector<PlanGeom> geom(n);
  int bits = 0;
  const bool big = M > kPlTokens;                      // accumulators of 128 tokens, single CTAs, one issuing thread
  // pairs of CTAs (two adjacent column tiles per MMA) unless an operand's adjacent tiles multiply different
  // channels (a block-diagonal operand with an odd number of groups per block) or pairs are switched off
  bool pair = !big && ctx->pl_mode != 1 && plan_units(ctx, true) > 0;
  for (int i = 0; i < n && pair; ++i) pair = ops[i].t->block_groups % 2 == 0;
  const int tile_div = pair ? 2 : 1;
  for (int i = 0; i < n; ++i) {
    const TiledOperand &t = *ops[i].t;
    const int G = groups_per_tile(t);
    if (G <= 0) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
    if (t.g_quant > 0) {
      if (bits != 0 && bits != t.bits) return ROSAQ_ERR_UNSUPPORTED_SHAPE;   // one code width per launch
      bits = t.bits;
    }
    if (ops[i].dep >= i) return ROSAQ_ERR_INVALID_ARG;
    // a permuted output is a scatter of 2-byte elements, bound by the store rate of an SM: the tiles of a
    // block-diagonal rotation (little arithmetic) are computed four times over, each copy writing a
    // quarter of the token rows from another SM
    const int rep = ops[i].col_map && G <= 2 ? 4 : 1;
    // (and such a copy keeps the epilogue warps of its CTA busy for about as long as sixteen quantized
    // groups keep the MMA threads: counted as that, so that these tiles spread over many CTAs)
    geom[i] = PlanGeom{(t.n_tiles + tile_div - 1) / tile_div, G, t.g_fp16, ops[i].dep, rep,
                       rep > 1 ? (pair ? kPlanPairCostScatterTile : kPlanCostScatterTile) : 0};
  }
  const int dflt_single[3] = {kPlanCostFp16, kPlanCostQuant, kPlanCostTile};
  const int dflt_pair[3] = {kPlanPairCostFp16, kPlanPairCostQuant, kPlanPairCostTile};
  const int *cost = ctx->pl_cost_set ? ctx->pl_cost : (pair ? dflt_pair : dflt_single);
  const PlanSchedule *s = nullptr;
  int st = plan_get_schedule(ctx, geom, plan_units(ctx, pair), cost, &s);
  if (st != ROSAQ_OK) return st;
  if (tile_div * s->n_counters > kPlMaxCounters) return ROSAQ_ERR_UNSUPPORTED_SHAPE;
  const int MT = pair ? ((M + 31) / 32) * 32 : ((M + 15) / 16) * 16;
  const int MTL = MT / tile_div;                       // token rows a CTA keeps in shared memory
  const int slot_floats = MT * kTileN;
  const size_t need = (size_t)tile_div * std::max(s->n_slots, 1) * slot_floats * sizeof(float);
  if (ctx->pl_partial_bytes < need) {
    // the old buffer may still be in use by work queued on some stream
    if (cudaDeviceSynchronize() != cudaSuccess) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_CUDA;
    }
    if (ctx->pl_partials) (void)cudaFree(ctx->pl_partials);
    ctx->pl_partials = nullptr;
    ctx->pl_partial_bytes = 0;
    if (cudaMalloc(reinterpret_cast<void **>(&ctx->pl_partials), need) != cudaSuccess) {
      (void)cudaGetLastError();
      return ROSAQ_ERR_ALLOC;
    }
    ctx->pl_partial_bytes = need;
  }
  PlParams *q = new (std::nothrow) PlParams();
  if (!q) return ROSAQ_ERR_ALLOC;
  for (int i = 0; i < n; ++i) {
    const TiledOperand &t = *ops[i].t;
    const __half *x = ops[i].dep >= 0 ? ops[ops[i].dep].y : ops[i].x;
    const long long ldx = ops[i].dep >= 0 ? ops[ops[i].dep].ldy : ops[i].ldx;
    const int m = ops[i].m > 0 ? ops[i].m : M;
    if (m > M || !plan_encode_x(&q->xmap[i], x, m, ldx, t.d_in, MTL)) {
      delete q;
      return ROSAQ_ERR_CUDA;
    }
    PlProblem &P = q->prob[i];
    P.blob = t.blob;
    P.y = ops[i].y;
    P.col_map = ops[i].col_map;
    P.tile_stride = t.tile_stride;
    P.ldy = ops[i].ldy;
    P.d_out = t.d_out;
    P.n_tiles = t.n_tiles;
    P.g_fp16 = t.g_fp16;
    P.block_groups = t.block_groups;
    P.dep = ops[i].dep;
    P.dep_target = ops[i].dep >= 0 ? (unsigned)tile_div * s->done_target[ops[i].dep] : 0u;   // both CTAs of a pair count
    P.signal = 0;
    P.m = m;
  }
  for (int i = 0; i < n; ++i)
    if (ops[i].dep >= 0) q->prob[ops[i].dep].signal = 1;
  q->segs = s->d_segs;
  q->seg_begin = s->d_seg_begin;
  q->partials = ctx->pl_partials;
  q->sync = ctx->pl_sync;
  q->status = ctx->d_status;
  q->wait_limit = ctx->wait_limit;
  q->n_counters = tile_div * s->n_counters;
  q->M = M;
  q->MT = MT;
  q->NW = plan_nw(MTL, pair ? kPlPairStages : kPlStages);
  q->slot_floats = slot_floats;
  out->params = q;
  out->n_ctas = tile_div * s->n_ctas;
  out->pair = pair;
  out->big = big;
  out->bits = bits == 3 ? 3 : 4;
  out->partial_bytes = need;
  return ROSAQ_OK;
}

void plan_release(PlanLaunch *l) {
  delete static_cast<PlParams *>(l->params);
  l->params = nullptr;
}

int plan_launch(rosaq_ctx *ctx, const PlanLaunch &l, cudaStream_t s) {
  PlParams *q = static_cast<PlParams *>(l.params);
  if (!q) return ROSAQ_ERR_INVALID_ARG;
  if (ctx->pl_partial_bytes < l.partial_bytes) return ROSAQ_ERR_INVALID_ARG;
  q->partials = ctx->pl_partials;                      // the workspace may have grown since the plan was made
  q->wait_limit = ctx->wait_limit;
  const size_t smem = plan_smem_bytes(l.pair ? q->MT / 2 : q->MT, q->NW, l.pair ? kPlPairStages : kPlStages);
  if (l.pair) return l.bits == 3 ? plan_launch_kernel(linear_plan_kernel<3, 1>, l, *q, smem, s)
                                 : plan_launch_kernel(linear_plan_kernel<4, 1>, l, *q, smem, s);
  if (l.big) return l.bits == 3 ? plan_launch_kernel(linear_plan_kernel<3, 2>, l, *q, smem, s)
                                : plan_launch_kernel(linear_plan_kernel<4, 2>, l, *q, smem, s);
  return l.bits == 3 ? plan_launch_kernel(linear_plan_kernel<3, 0>, l, *q, smem, s)
                     : plan_launch_kernel(linear_plan_kernel<4, 0>, l, *q, smem, s);
}

}  // namespace rosaq
