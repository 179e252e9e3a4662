// Device-side pieces shared by the kernels of the TILES layout (tq_tiles.cu, tq_wide.cu): the
// shared-memory plan, the table copy, the per-warp ring of raw words, the 16-token lookup, and the
// block-fixed-point form of the activations.  Everything sits in an unnamed namespace: each
// translation unit that includes this file gets its own copy.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "tq_internal.h"
#include "tq_sm100.cuh"

namespace {

using namespace tq_sm100;

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kRingWords = TQ_TILES_RING_WORDS;     // 4 KB per warp
constexpr int kChunkWords = 512;                    // one bulk copy: 2 KB of raw words
constexpr int kSlots = kRingWords / kChunkWords;    // chunks per ring
constexpr int kL2Ahead = 8;                         // token tiles prefetched into L2 ahead of their use (<= 8: padding)
constexpr uint32_t kNoBlock = 0xFFFFFFFFu;
constexpr int kDigits = 4;    // signed base-256 digits of a fixed-point activation
constexpr int kFixBits = 30;  // |X| <= 2^kFixBits
constexpr uint32_t kMissBase = 0x10000u - TQ_TILES_RING_WORDS;  // first miss token
static_assert(kSlots == 2 && (kRingWords & (kRingWords - 1)) == 0 && kRingWords - kChunkWords >= 512, "ring geometry: a tile has up to 512 raw words");

__host__ __device__ inline uint32_t align_up_u32(uint32_t v, uint32_t a) { return (v + a - 1) / a * a; }

// Shared-memory plan, identical on host and device.
struct TilesSmem {
  uint32_t ring, x, bar, misc, total;
};
__host__ __device__ inline TilesSmem tiles_smem(uint32_t table_words, uint32_t x_words, int warps) {
  TilesSmem L;
  L.ring = align_up_u32(table_words * 4u, 16u);
  L.x = L.ring + (uint32_t)warps * kRingWords * 4u;
  L.bar = align_up_u32(L.x + x_words * 4u, 16u);
  L.misc = L.bar + (uint32_t)warps * kSlots * 8u;
  L.total = L.misc + 1024u;
  return L;
}

struct TilesSeg {
  uint32_t mat, rb_begin, rb_end;
};

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// The table into shared memory with bulk copies (one thread issues them; nothing waits until the
// first lookup, so the activation set-up and the first loads of the streams overlap the copy).
constexpr uint32_t kTableBarOffset = 400u;  // inside the misc area of the shared-memory plan
// withhold_last (test hook): the barrier is told to expect the whole table but the last copy is not made, so
// the barrier never completes and every wait for the table runs into its limit.
__device__ __forceinline__ void table_load_async(uint32_t tbl_addr, uint32_t bar, const uint32_t* table, uint32_t words,
                                                 bool withhold_last = false) {
  const uint32_t bytes = words * 4u;
  mbar_expect_tx(bar, bytes);
  for (uint32_t off = 0; off < bytes; off += 8192u) {
    if (withhold_last && off + 8192u >= bytes) break;
    bulk_g2s(tbl_addr + off, reinterpret_cast<const uint8_t*>(table) + off, min(8192u, bytes - off), bar);
  }
}

// ---- activations as block fixed point ------------------------------------------------------
// A vector whose largest magnitude has the bf16 bit pattern `amax_bits` (sign cleared) satisfies
// max |x| < 2^e with e = exponent field - 126, and is put on the grid X = round(x * 2^(kFixBits - e)).
// The power of two spans [2^-98, 2^156], so it is applied as two float factors; both products are
// exact wherever the result matters (a power of two times a bf16 value).
struct FixScale {
  float s1, s2;  // X = round(x * s1 * s2)
  int e;
  bool finite;   // false: the vector holds an Inf or a NaN
};
__device__ __forceinline__ FixScale fix_scale(uint32_t amax_bits) {
  FixScale f;
  f.finite = amax_bits < 0x7F80u;
  f.e = (int)(min(amax_bits, 0x7F7Fu) >> 7) - 126;  // in [-126, 128]
  const int k = kFixBits - f.e, k1 = k / 2, k2 = k - k1;
  f.s1 = __uint_as_float((uint32_t)(127 + k1) << 23);
  f.s2 = __uint_as_float((uint32_t)(127 + k2) << 23);
  return f;
}
// 2^(e - kFixBits) as a double, built from its exponent field; NaN for a non-finite vector.
__device__ __forceinline__ double fix_out_scale(const FixScale& f) {
  return f.finite ? __longlong_as_double((long long)(1023 + f.e - kFixBits) << 52)
                  : __longlong_as_double(0x7FF8000000000000ll);
}
// Largest magnitude of four bf16 values (bit patterns, monotonic; Inf and NaN sort last).
__device__ __forceinline__ uint32_t amax4(uint2 v, uint32_t m) {
  const uint32_t a0 = v.x & 0x7FFF7FFFu, a1 = v.y & 0x7FFF7FFFu;
  return max(max(m, a0 & 0xFFFFu), max(a0 >> 16, max(a1 & 0xFFFFu, a1 >> 16)));
}
// Digits of one activation group (4 columns) -> four words, word k holding digit k of the four
// values.  X = d0 + 2^8 d1 + 2^16 d2 + 2^24 d3 with balanced digits (signed bytes): d0 is the low
// byte of X, d1 byte 1 of X + 2^7, d2 byte 2 of X + 2^7 + 2^15, d3 byte 3 of X + 2^7 + 2^15 + 2^23.
__device__ __forceinline__ void fix_digits(uint2 v, float s1, float s2, uint32_t (&w)[kDigits], long long* sum) {
  const uint32_t h[4] = {v.x << 16, v.x & 0xFFFF0000u, v.y << 16, v.y & 0xFFFF0000u};
  uint32_t X[4], Y[4], Z[4], U[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int xi = __float2int_rn(__uint_as_float(h[i]) * s1 * s2);
    if (sum) *sum += xi;
    X[i] = (uint32_t)xi;
    Y[i] = X[i] + 128u;
    Z[i] = X[i] + 32896u;
    U[i] = X[i] + 8421504u;
  }
  w[0] = __byte_perm(__byte_perm(X[0], X[1], 0x0040), __byte_perm(X[2], X[3], 0x0040), 0x5410);
  w[1] = __byte_perm(__byte_perm(Y[0], Y[1], 0x0051), __byte_perm(Y[2], Y[3], 0x0051), 0x5410);
  w[2] = __byte_perm(__byte_perm(Z[0], Z[1], 0x0062), __byte_perm(Z[2], Z[3], 0x0062), 0x5410);
  w[3] = __byte_perm(__byte_perm(U[0], U[1], 0x0073), __byte_perm(U[2], U[3], 0x0073), 0x5410);
}

// Bounded in attempts and in time (about 2 s).  Kept out of line and free of references so that the
// caller's state stays in registers.
#ifndef TQ_WAIT_SLOW_INLINING
#define TQ_WAIT_SLOW_INLINING __noinline__
#endif
__device__ TQ_WAIT_SLOW_INLINING bool tiles_wait_slow(uint32_t bar, uint32_t par, volatile uint32_t* dead_flag) {
  const uint64_t t_start = global_ns();
  bool ok = false;
  for (uint32_t i = 0; i < kSpinLimit && !ok; ++i) {
    ok = mbar_try(bar, par);
    if ((i & 63u) == 63u && (*dead_flag || global_ns() - t_start > 2000000000ull)) break;
  }
  return __all_sync(kFull, ok);
}

// What every CTA of these kernels carries: the shared-memory plan, the table and this warp's raw ring.
//
// Raw ring: chunk c of a matrix's raw stream (words 512c .. 512c+511) always lands in half c mod 2
// of the ring, the place its tokens point to.  A tile has at most 512 raw words, so the two chunks in
// flight always cover the tile being looked up.  The barriers are used round robin in issue order,
// which is also the order of the waits: use number n takes barrier n mod 2 and completes its phase
// (n / 2) mod 2.
struct CtaBase {
  uint8_t* smem;
  TilesSmem L;
  uint32_t tbl_addr;             // shared address of the table (start of dynamic shared memory)
  uint32_t warp, lane;
  uint32_t ring_addr, bar_base;  // shared addresses of this warp's ring and of its first barrier
  uint32_t n_issued = 0, n_waited = 0;
  bool table_ready = false;

  __device__ __forceinline__ volatile uint32_t* dead_flag() { return reinterpret_cast<uint32_t*>(smem + L.misc); }

  // Barriers, table copy (asynchronous: wait_table() before the first lookup), one CTA barrier.
  __device__ __forceinline__ void setup(uint8_t* smem_raw, const TilesSmem& plan, int warps, const uint32_t* table,
                                        uint32_t table_words, bool withhold_last_table_chunk = false) {
    smem = smem_raw;
    L = plan;
    tbl_addr = smem_u32(smem_raw);
    warp = threadIdx.x >> 5;
    lane = threadIdx.x & 31u;
    ring_addr = tbl_addr + L.ring + warp * (kRingWords * 4u);
    bar_base = tbl_addr + L.bar + warp * (kSlots * 8u);
    if (threadIdx.x < (uint32_t)warps * kSlots) mbar_init(tbl_addr + L.bar + threadIdx.x * 8u, 1u);
    if (threadIdx.x == 0) {
      *dead_flag() = 0u;
      mbar_init(tbl_addr + L.misc + kTableBarOffset, 1u);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (threadIdx.x == 0)
      table_load_async(tbl_addr, tbl_addr + L.misc + kTableBarOffset, table, table_words, withhold_last_table_chunk);
    __syncthreads();
  }
  // After a wait has run out: copies that were issued may still be landing in this CTA's shared memory, so
  // the CTA stays a little (2 ms) before it ends.
  __device__ __forceinline__ void linger_after_failure() {
    if (*dead_flag())
      for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  // False if the bounded wait ran out.
  __device__ __forceinline__ bool wait_table() {
    if (table_ready) return true;
    const uint32_t bar = tbl_addr + L.misc + kTableBarOffset;
    if (!__all_sync(kFull, mbar_try(bar, 0u)) && !tiles_wait_slow(bar, 0u, dead_flag())) return false;
    table_ready = true;
    return true;
  }
  __device__ __forceinline__ void issue_chunk(const uint32_t* raw, uint32_t pos) {  // pos: first word, multiple of 256
    if (lane == 0) {
      const uint32_t bar = bar_base + (n_issued & (kSlots - 1u)) * 8u;
      mbar_expect_tx(bar, kChunkWords * 4u);
      bulk_g2s(ring_addr + ((pos * 4u) & (kRingWords * 4u - 1u)), raw + pos, kChunkWords * 4u, bar);
    }
    ++n_issued;
  }
  __device__ __forceinline__ bool wait_chunk() {
    const uint32_t bar = bar_base + (n_waited & (kSlots - 1u)) * 8u;
    const uint32_t par = (n_waited / kSlots) & 1u;
    ++n_waited;
    if (__all_sync(kFull, mbar_try(bar, par))) return true;  // one answer per warp: the slow path votes too
    return tiles_wait_slow(bar, par, dead_flag());
  }
  // The 16 words of this lane's tokens: a token below kMissBase indexes the table, any other names
  // the ring slot of its raw word.
  __device__ __forceinline__ void lookup16(const uint4 (&q)[2], uint32_t (&w)[16]) const {
    const uint32_t miss_adj4 = ring_addr - 4u * kMissBase;
    const uint32_t R[8] = {q[0].x, q[0].y, q[0].z, q[0].w, q[1].x, q[1].y, q[1].z, q[1].w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      asm volatile(
          "{\n\t.reg .pred p0, p1;\n\t.reg .u32 t0, t1, b0, b1, a0, a1;\n\t"
          "and.b32 t0, %2, 0xFFFF;\n\t"
          "shr.u32 t1, %2, 16;\n\t"
          "setp.ge.u32 p0, t0, 64512;\n\t"
          "setp.ge.u32 p1, t1, 64512;\n\t"
          "selp.u32 b0, %4, %3, p0;\n\t"
          "selp.u32 b1, %4, %3, p1;\n\t"
          "mad.lo.u32 a0, t0, 4, b0;\n\t"
          "mad.lo.u32 a1, t1, 4, b1;\n\t"
          "ld.shared.u32 %0, [a0];\n\t"
          "ld.shared.u32 %1, [a1];\n\t}"
          : "=r"(w[2 * i]), "=r"(w[2 * i + 1])
          : "r"(R[i]), "r"(tbl_addr), "r"(miss_adj4));
    }
  }
};

}  // namespace
