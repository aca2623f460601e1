// Pieces shared by the GEMM-stage kernels (linear_tc.cu, linear_plan.cu): sizes of the operand rings,
// the in-register dequantisation of one packed tile into a TMEM operand buffer, bounded waits.
#pragma once

#include "ptx.cuh"
#include "rosaq_internal.cuh"

namespace rosaq {

constexpr int kTeamThreads = 128;                          // one dequantisation team: a warp per TMEM lane quadrant
constexpr int kWSlotBytes = kInt4CodeBytes + kScaleBytes;  // 8704: one quantized tile or a quarter fp16 tile
constexpr int kFp16SubBytes = kFp16TileBytes / 4;          // 32 input channels of an fp16 tile
// polls (about a microsecond each) granted to work already in flight when a CTA gives up: unlike the
// waits of the pipeline this bound does not follow the context's wait limit, so that a shortened limit
// can never let a CTA retire under its own copies or MMAs
constexpr int kDrainPolls = 1 << 16;

// ---------------------------------------------------------------------------------- dequantisation
// (code - zero) * scale in fp16, exact subtraction then one rounding: codes are spliced into the
// mantissa of a power-of-two constant (1024, 128, 64 or 16 depending on the bit position), which
// turns them into fp16 integers without a conversion instruction.
struct ScaleZero {
  uint32_t s2, z1024, z128, z64, z16;
  __device__ __forceinline__ explicit ScaleZero(uint32_t sz) {
    const uint32_t s = sz & 0xffffu, z = sz >> 16;
    s2 = s | (s << 16);
    const uint32_t zz = z | (z << 16);
    auto add = [&](uint32_t c) {
      __half2 r = __hadd2(*reinterpret_cast<const __half2 *>(&zz), *reinterpret_cast<const __half2 *>(&c));
      return *reinterpret_cast<uint32_t *>(&r);
    };
    z1024 = add(0x64006400u);
    z128 = add(0x58005800u);
    z64 = add(0x54005400u);
    z16 = add(0x4C004C00u);
  }
};

// one word = 8 INT4 codes -> 4 fp16 pairs (k, k+1), (k+2, k+3), (k+4, k+5), (k+6, k+7)
__device__ __forceinline__ void dequant_int4_word(uint32_t q, const ScaleZero &c, uint32_t *out) {
  const uint32_t q8 = q >> 8;
  out[0] = h2_sub_mul(lop_and_or(q, 0x000f000fu, 0x64006400u), c.z1024, c.s2);
  out[1] = h2_sub_mul(lop_and_or(q, 0x00f000f0u, 0x54005400u), c.z64, c.s2);
  out[2] = h2_sub_mul(lop_and_or(q8, 0x000f000fu, 0x64006400u), c.z1024, c.s2);
  out[3] = h2_sub_mul(lop_and_or(q8, 0x00f000f0u, 0x54005400u), c.z64, c.s2);
}

// three words = 32 INT3 codes -> 16 fp16 pairs
__device__ __forceinline__ void dequant_int3_set(uint32_t a, uint32_t b, uint32_t cc, const ScaleZero &c,
                                                 uint32_t *out) {
  const uint32_t w[3] = {a, b, cc};
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const uint32_t q = w[i], q9 = q >> 9;
    out[5 * i + 0] = h2_sub_mul(lop_and_or(q, 0x00070007u, 0x64006400u), c.z1024, c.s2);
    out[5 * i + 1] = h2_sub_mul(lop_and_or(q, 0x00380038u, 0x58005800u), c.z128, c.s2);
    out[5 * i + 2] = h2_sub_mul(lop_and_or(q, 0x01c001c0u, 0x4C004C00u), c.z16, c.s2);
    out[5 * i + 3] = h2_sub_mul(lop_and_or(q9, 0x00070007u, 0x64006400u), c.z1024, c.s2);
    out[5 * i + 4] = h2_sub_mul(lop_and_or(q9, 0x00380038u, 0x58005800u), c.z128, c.s2);
  }
  const uint32_t tail = ((a >> 15) & 0x00010001u) | ((b >> 14) & 0x00020002u) | ((cc >> 13) & 0x00040004u);
  out[15] = h2_sub_mul(tail | 0x64006400u, c.z1024, c.s2);
}

// One unit of the weight ring (a quantized group, or 32 input channels of an fp16 group) of output
// column n: shared memory -> registers -> the TMEM operand buffer at a_addr.  The slot is released
// only after instructions that depend on every loaded word have been issued: an arrive placed right
// behind the loads can be performed while they are still queued (seen when the other CTA of the SM kept
// the load/store unit busy with global stores), and the producer then refills the slot under them.
template <int kBits>
__device__ __forceinline__ void dequant_unit(bool f16, uint32_t slot_base, int n, uint32_t a_addr, int sub,
                                             uint32_t bar_release) {
  const uint32_t ws = slot_base + n * 16;
  if (f16) {
    // a quarter of an fp16 group: 32 input channels = 16 TMEM columns
    uint32_t r[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4 *>(&r[4 * j]) = lds128(ws + j * (kTileN * 16));
    tmem_st16(a_addr + 16 * sub, r);
    mbar_arrive(bar_release);
  } else if (kBits == 4) {
    const ScaleZero c(lds32(slot_base + kInt4CodeBytes + n * 4));
    uint4 q[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) q[j] = lds128(ws + j * (kTileN * 16));
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t r[16];
      dequant_int4_word(q[j].x, c, &r[0]);
      dequant_int4_word(q[j].y, c, &r[4]);
      dequant_int4_word(q[j].z, c, &r[8]);
      dequant_int4_word(q[j].w, c, &r[12]);
      tmem_st16(a_addr + 16 * j, r);
    }
    mbar_arrive(bar_release);
  } else {
    const ScaleZero c(lds32(slot_base + kInt3CodeBytes + n * 4));
    // the column's 12 words: 4 sets of 3 words = 32 codes = 16 TMEM columns each
    uint32_t w12[12];
#pragma unroll
    for (int j = 0; j < 3; ++j) *reinterpret_cast<uint4 *>(&w12[4 * j]) = lds128(ws + j * (kTileN * 16));
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t r[16];
      dequant_int3_set(w12[3 * j], w12[3 * j + 1], w12[3 * j + 2], c, r);
      tmem_st16(a_addr + 16 * j, r);
    }
    mbar_arrive(bar_release);
  }
}

// ---------------------------------------------------------------------------------- the kernel
struct Abort {
  volatile int *flag;     // shared
  int *status;            // global
  long long limit;
  bool cluster_scope;     // barriers also receive arrivals from the peer CTA of a pair
  __device__ __forceinline__ bool set() const { return *flag != 0; }
  __device__ __forceinline__ void raise() const {
    *flag = 1;
    atomicExch(status, (int)ROSAQ_ERR_TIMEOUT);
  }
  // false when the wait gave up (or somebody else already did)
  __device__ __forceinline__ bool poll(uint32_t bar, uint32_t parity) const {
    return cluster_scope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity);
  }
  // barriers that only this CTA's threads and copies feed: CTA scope whatever the mode
  __device__ __forceinline__ bool wait_local(uint32_t bar, uint32_t parity) const {
    if (mbar_try_wait(bar, parity)) return true;
    for (long long it = 0; it < limit; ++it) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((it & 63) == 63 && set()) return false;
    }
    raise();
    return false;
  }
  // one cluster-scope poll per warp instead of thirty-two, verdict broadcast (also the warp-level sync)
  __device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity) const {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = wait(bar, parity) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
  }
  __device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity) const {
    if (poll(bar, parity)) return true;
    for (long long it = 0; it < limit; ++it) {
      if (poll(bar, parity)) return true;
      if ((it & 63) == 63 && set()) return false;
    }
    raise();
    return false;
  }
};

// Position in a ring of n slots plus the parity of the current lap, advanced without division
// (the role warps run on a single lane: an integer division there costs hundreds of cycles).
struct Ring {
  int idx;
  uint32_t lap;
  __device__ __forceinline__ void advance(int n) {
    if (++idx == n) {
      idx = 0;
      lap ^= 1u;
    }
  }
};

}  // namespace rosaq
