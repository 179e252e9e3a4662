// Device half of libtq (sm_100a): upload, tq_decompress, tq_fused_gemv and the row quantizer.
//
// Token parse shared by the kernels (Listing 4 made data-parallel).  One warp owns one row
// segment and walks it in tiles of 256 uint16 slots; a lane holds 8 consecutive slots (one
// 128-bit load).  A slot equal to 0xFFFF is always a marker (raw slots hold bytes, codes stop at
// 65534), so a slot is raw exactly when one of the 4 slots before it is a marker.  A group is
// "completed" at a code slot or at the 4th raw slot after a marker; the lane that holds the
// completing slot also sees the 4 slots before its own 8 (two registers shuffled from the lane
// below, or carried over from the previous tile), which is all it needs to produce the group's 4
// bytes.  The group's index inside the row is a warp prefix sum of the per-lane completion counts
// plus a running base.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>
#include <new>

#include "tq_internal.h"

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kThreads = kWarpsPerCta * 32;
constexpr unsigned kFull = 0xFFFFFFFFu;

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// bit 15 / bit 31 set when the low / high half of a equals 0xFFFF (exact for validated streams:
// the only false positive is 0xFFFE directly after a marker, which validation rules out).
__device__ __forceinline__ uint32_t esc_bits(uint32_t a) {
  return ~(a + 0x00010001u) & a & 0x80008000u;
}

constexpr uint32_t kRing = 512;  // per-warp ring of decoded groups (uint32 each); > 256 + 31

// Exact variant for token planes, where any token may follow a marker: bit 15 / 31 set iff the
// low / high half equals 0xFFFF.
__device__ __forceinline__ uint32_t esc_bits_exact(uint32_t a) {
  const uint32_t t = (~a & 0x7FFF7FFFu) + 0x7FFF7FFFu;
  return ~t & a & 0x80008000u;
}

// Walks one row segment.  Each tile is handled in two phases.  Phase 1: every lane turns the
// groups completed inside its 8 slots into packed 4-byte words (table loads are issued together,
// before any use) and stores them, in row order, into the warp's ring in shared memory.  Phase 2:
// the ring is drained 32 groups at a time, lane i taking group done+i, so the consumer sees
// consecutive groups on consecutive lanes (conflict-free x reads, coalesced stores).  Fewer than
// 32 left-over groups wait for the next tile; the row end flushes them.
// consume(group_index, packed4bytes) is called once per group.  Returns the groups seen.
template <class Consume>
__device__ __forceinline__ uint32_t decode_row(const uint4* __restrict__ tok, uint32_t n_slots,
                                               const uint32_t* __restrict__ table, uint32_t K,
                                               uint32_t groups_per_row, uint32_t* __restrict__ ring,
                                               uint32_t& status_bits, Consume&& consume) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t n_chunks = (n_slots + 7u) >> 3;
  const uint32_t n_tiles = (n_chunks + 31u) >> 5;
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

  uint4 cur = lane < n_chunks ? ldg_stream(tok + lane) : zero4;
  uint4 nxt = lane + 32u < n_chunks ? ldg_stream(tok + lane + 32u) : zero4;
  uint32_t base = 0, done = 0, carryE = 0, carryZ = 0, carryW = 0, bad = 0;

  for (uint32_t t = 0; t < n_tiles; ++t) {
    const uint32_t pf = (t + 2u) * 32u + lane;
    const uint4 nn = pf < n_chunks ? ldg_stream(tok + pf) : zero4;

    const int left = (int)n_slots - (int)(t * 256u + lane * 8u);
    const uint32_t V = left >= 8 ? 0xFFu : (left <= 0 ? 0u : ((1u << left) - 1u));

    const uint32_t e = (esc_bits(cur.x) >> 15) | (esc_bits(cur.y) >> 13) | (esc_bits(cur.z) >> 11) |
                       (esc_bits(cur.w) >> 9);
    const uint32_t E = (e | (e >> 15)) & V;

    uint32_t prevE = __shfl_up_sync(kFull, E, 1);
    uint32_t pz = __shfl_up_sync(kFull, cur.z, 1);
    uint32_t pw = __shfl_up_sync(kFull, cur.w, 1);
    if (lane == 0) { prevE = carryE; pz = carryZ; pw = carryW; }

    const uint32_t X = (prevE >> 4) | (E << 4);                       // markers over the 12-slot window
    const uint32_t R = (X | (X >> 1) | (X >> 2) | (X >> 3)) & 0xFFu;  // own slots that are raw
    const uint32_t CODE = ~R & ~E & V;                                // own slots holding a code
    const uint32_t C = (CODE | X) & V;                                // own slots completing a group

    const uint32_t n = __popc(C);
    uint32_t incl = n;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      uint32_t v = __shfl_up_sync(kFull, incl, d);
      if (lane >= (uint32_t)d) incl += v;
    }
    uint32_t g = base + incl - n;
    base += __shfl_sync(kFull, incl, 31);
    carryE = __shfl_sync(kFull, E, 31);
    carryZ = __shfl_sync(kFull, cur.z, 31);
    carryW = __shfl_sync(kFull, cur.w, 31);

    // ---- phase 1: words of the completed groups ----
    const uint32_t W[6] = {pz, pw, cur.x, cur.y, cur.z, cur.w};
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t reg = W[2 + (j >> 1)];
      const uint32_t idx = (j & 1) ? (reg >> 16) : (reg & 0xFFFFu);
      const uint32_t cl = min(idx, K);
      uint32_t v = 0u;
      if (CODE & (1u << j)) {
        v = __ldg(table + cl);  // word 0 of the table is zero
        bad |= (idx ^ cl) | (idx == 0u);
      }
      w[j] = v;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (X & (1u << j)) {  // 4th raw slot after a marker at window slot j: low bytes of slots j+1..j+4
        if (j & 1) {
          w[j] = __byte_perm(W[(j + 1) >> 1], W[((j + 1) >> 1) + 1], 0x6420);
        } else {
          const uint32_t t3 = __byte_perm(W[j >> 1], W[(j >> 1) + 1], 0x0642);
          w[j] = __byte_perm(t3, W[(j >> 1) + 2], 0x4210);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (C & (1u << j)) {
        ring[g & (kRing - 1u)] = w[j];
        ++g;
      }
    }
    __syncwarp();

    // ---- phase 2: drain full batches of 32 groups ----
    const uint32_t lim = min(base, groups_per_row);
    while (done + 32u <= lim) {
      const uint32_t grp = done + lane;
      consume(grp, ring[grp & (kRing - 1u)]);
      done += 32u;
    }
    cur = nxt;
    nxt = nn;
  }
  {
    const uint32_t lim = min(base, groups_per_row);
    const uint32_t grp = done + lane;
    if (grp < lim) consume(grp, ring[grp & (kRing - 1u)]);
  }
  __syncwarp();  // the ring is reused by this warp's next row
  if (bad) status_bits |= TQ_STATUS_BAD_CODE;
  return base;
}

// ---------------------------------------------------------------------------------------------
// tq_decompress: expand to bytes in HBM.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 4)
decompress_kernel(const uint4* __restrict__ tokens, const tq_rowseg* __restrict__ rowseg,
                  const uint32_t* __restrict__ table, uint32_t K, uint32_t rows, uint32_t cols,
                  uint32_t* __restrict__ out, uint32_t* __restrict__ status) {
  __shared__ uint32_t rings[kWarpsPerCta][kRing];
  const uint32_t warp = threadIdx.x >> 5;
  const uint32_t gpr = cols >> 2;
  uint32_t bits = 0;
  for (uint32_t row = blockIdx.x * kWarpsPerCta + warp; row < rows; row += gridDim.x * kWarpsPerCta) {
    const tq_rowseg seg = rowseg[row];
    uint32_t* orow = out + (size_t)row * gpr;
    const uint32_t seen = decode_row(tokens + seg.chunk_off, seg.n_slots, table, K, gpr, rings[warp], bits,
                                     [&](uint32_t g, uint32_t w) { orow[g] = w; });
    if (seen != gpr) bits |= TQ_STATUS_BAD_ROW;
  }
  if (bits) atomicOr(status, bits);
}

// ---------------------------------------------------------------------------------------------
// tq_fused_gemv: decode -> dequantise -> dot product, batch NB (1..4) per pass.
// x is staged once per CTA in shared memory as fp32, one float4 per group of 4 columns.
// A byte b becomes a float through the bit pattern 0x4B000000 | b' (= 2^23 + b') minus a
// constant; with b' = b ^ 0x80 and the constant 2^23 + 128 this is the int8 value of b, with
// b' = b and 2^23 the unsigned one.
// ---------------------------------------------------------------------------------------------
template <int NB>
__global__ void __launch_bounds__(kThreads, 4)
gemv_kernel(const uint4* __restrict__ tokens, const tq_rowseg* __restrict__ rowseg,
            const float* __restrict__ scale, const float* __restrict__ zero, int has_zero,
            const uint32_t* __restrict__ table, uint32_t K, uint32_t rows, uint32_t cols,
            const __nv_bfloat16* __restrict__ x, float* __restrict__ y, uint32_t xor_mask,
            float magic, uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) float xs[];  // [NB][cols]
  __shared__ uint32_t rings[kWarpsPerCta][kRing];
  __shared__ float sumx[NB];
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t gpr = cols >> 2;

  for (uint32_t i = threadIdx.x; i < NB * (cols >> 1); i += kThreads) {
    const __nv_bfloat162 v = reinterpret_cast<const __nv_bfloat162*>(x)[i];
    reinterpret_cast<float2*>(xs)[i] = __bfloat1622float2(v);
  }
  if (threadIdx.x < NB) sumx[threadIdx.x] = 0.f;
  __syncthreads();
  if (has_zero) {
    for (int b = 0; b < NB; ++b) {
      float s = 0.f;
      for (uint32_t i = threadIdx.x; i < cols; i += kThreads) s += xs[b * cols + i];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(kFull, s, d);
      if (lane == 0) atomicAdd(&sumx[b], s);
    }
    __syncthreads();
  }

  uint32_t bits = 0;
  for (uint32_t row = blockIdx.x * kWarpsPerCta + warp; row < rows; row += gridDim.x * kWarpsPerCta) {
    const tq_rowseg seg = rowseg[row];
    float acc[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b] = 0.f;
    const uint32_t seen = decode_row(
        tokens + seg.chunk_off, seg.n_slots, table, K, gpr, rings[warp], bits, [&](uint32_t g, uint32_t w) {
          w ^= xor_mask;
          const float f0 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7540)) - magic;
          const float f1 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7541)) - magic;
          const float f2 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7542)) - magic;
          const float f3 = __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7543)) - magic;
#pragma unroll
          for (int b = 0; b < NB; ++b) {
            const float4 xv = reinterpret_cast<const float4*>(xs + b * cols)[g];
            acc[b] = fmaf(f0, xv.x, acc[b]);
            acc[b] = fmaf(f1, xv.y, acc[b]);
            acc[b] = fmaf(f2, xv.z, acc[b]);
            acc[b] = fmaf(f3, xv.w, acc[b]);
          }
        });
    if (seen != gpr) bits |= TQ_STATUS_BAD_ROW;
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      float a = acc[b];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(kFull, a, d);
      acc[b] = a;
    }
    if (lane == 0) {
      const float s = scale[row];
      const float z = has_zero ? zero[row] : 0.f;
#pragma unroll
      for (int b = 0; b < NB; ++b) y[(size_t)b * rows + row] = s * (acc[b] - z * sumx[b]);
    }
  }
  if (bits) atomicOr(status, bits);
}

// ---------------------------------------------------------------------------------------------
// PLANES layout.  One warp owns one row and walks it in passes of 256 groups; lane L holds the 8
// consecutive tokens of groups 8L..8L+7 of the pass (one 128-bit load).  A token is a code, the
// marker 0xFFFF (its 4 bytes are the next word of the row's raw plane; the word's rank is the
// number of markers before it, a warp prefix sum plus a popcount) or 0 (padding, decodes to zero
// bytes through word 0 of the table).  All loads of a pass are issued before any use.
// done(j, w) receives the packed bytes of the lane's j-th group, j = 0..7 (static).
// ---------------------------------------------------------------------------------------------
template <class Pass>
__device__ __forceinline__ void planes_row(const uint4* __restrict__ codes, uint32_t gpr_pad,
                                           const uint32_t* __restrict__ raw, const uint32_t* __restrict__ table,
                                           uint32_t K, uint32_t& bad, Pass&& pass_done) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t n_vec = gpr_pad >> 3;           // 128-bit loads in the row
  const uint32_t n_pass = (n_vec + 31u) >> 5;
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  uint4 cur = lane < n_vec ? ldg_stream(codes + lane) : zero4;
  uint4 nxt = lane + 32u < n_vec ? ldg_stream(codes + lane + 32u) : zero4;
  uint32_t rawcur = 0;
  for (uint32_t p = 0; p < n_pass; ++p) {
    const uint32_t pf = (p + 2u) * 32u + lane;
    const uint4 nn = pf < n_vec ? ldg_stream(codes + pf) : zero4;
    const uint32_t e = (esc_bits_exact(cur.x) >> 15) | (esc_bits_exact(cur.y) >> 13) | (esc_bits_exact(cur.z) >> 11) |
                       (esc_bits_exact(cur.w) >> 9);
    const uint32_t E = (e | (e >> 15)) & 0xFFu;
    const uint32_t n = __popc(E);
    uint32_t incl = n;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      uint32_t v = __shfl_up_sync(kFull, incl, d);
      if (lane >= (uint32_t)d) incl += v;
    }
    const uint32_t* rp = raw + rawcur + (incl - n);
    rawcur += __shfl_sync(kFull, incl, 31);
    const uint32_t T[4] = {cur.x, cur.y, cur.z, cur.w};
    uint32_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t tok = (j & 1) ? (T[j >> 1] >> 16) : (T[j >> 1] & 0xFFFFu);
      if (E & (1u << j)) {
        w[j] = __ldg(rp + __popc(E & ((1u << j) - 1u)));
      } else {
        const uint32_t cl = min(tok, K);
        bad |= tok ^ cl;
        w[j] = __ldg(table + cl);
      }
    }
    pass_done(p, w);
    cur = nxt;
    nxt = nn;
  }
}

__global__ void __launch_bounds__(kThreads, 4)
decompress_planes_kernel(const uint16_t* __restrict__ codes, uint32_t gpr_pad, const uint32_t* __restrict__ rawbase,
                         const uint32_t* __restrict__ raw, const uint32_t* __restrict__ table, uint32_t K,
                         uint32_t rows, uint32_t cols, uint32_t* __restrict__ out, uint32_t* __restrict__ status) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t gpr = cols >> 2;
  const bool vec_ok = (cols & 15u) == 0u;
  uint32_t bad = 0;
  for (uint32_t row = blockIdx.x * kWarpsPerCta + warp; row < rows; row += gridDim.x * kWarpsPerCta) {
    uint32_t* orow = out + (size_t)row * gpr;
    planes_row(reinterpret_cast<const uint4*>(codes + (size_t)row * gpr_pad), gpr_pad, raw + rawbase[row], table, K,
               bad, [&](uint32_t p, const uint32_t (&w)[8]) {
                 const uint32_t g0 = p * 256u + lane * 8u;
                 if (vec_ok && g0 + 8u <= gpr) {
                   uint4* o = reinterpret_cast<uint4*>(orow + g0);
                   o[0] = make_uint4(w[0], w[1], w[2], w[3]);
                   o[1] = make_uint4(w[4], w[5], w[6], w[7]);
                 } else {
#pragma unroll
                   for (int j = 0; j < 8; ++j)
                     if (g0 + j < gpr) orow[g0 + j] = w[j];
                 }
               });
  }
  if (bad) atomicOr(status, TQ_STATUS_BAD_CODE);
}

// x is staged per CTA as fp32 float4 per group, permuted so that the group 8L+j of pass p sits at
// slot p*256 + j*32 + L: the 32 lanes of a warp read 32 consecutive float4 at every step j.
template <int NB>
__global__ void __launch_bounds__(kThreads, 4)
gemv_planes_kernel(const uint16_t* __restrict__ codes, uint32_t gpr_pad, const uint32_t* __restrict__ rawbase,
                   const uint32_t* __restrict__ raw, const float* __restrict__ scale, const float* __restrict__ zero,
                   int has_zero, const uint32_t* __restrict__ table, uint32_t K, uint32_t rows, uint32_t cols,
                   const __nv_bfloat16* __restrict__ x, float* __restrict__ y, uint32_t xor_mask, float magic,
                   uint32_t* __restrict__ status) {
  extern __shared__ __align__(16) float xs[];  // [NB][n_pass*256] float4
  __shared__ float sumx[NB];
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t gpr = cols >> 2;
  const uint32_t slots = ((gpr_pad + 255u) >> 8) << 8;  // float4 slots per batch column
  float4* xs4 = reinterpret_cast<float4*>(xs);

  float part[NB];
#pragma unroll
  for (int b = 0; b < NB; ++b) part[b] = 0.f;
  for (uint32_t i = threadIdx.x; i < slots; i += kThreads) {
    const uint32_t r = i & 255u;
    const uint32_t g = (i & ~255u) + ((r & 31u) << 3) + (r >> 5);
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (g < gpr) {
        const uint2 raw2 = reinterpret_cast<const uint2*>(x + (size_t)b * cols)[g];
        v.x = __uint_as_float(raw2.x << 16);
        v.y = __uint_as_float(raw2.x & 0xFFFF0000u);
        v.z = __uint_as_float(raw2.y << 16);
        v.w = __uint_as_float(raw2.y & 0xFFFF0000u);
      }
      xs4[(size_t)b * slots + i] = v;
      part[b] += (v.x + v.y) + (v.z + v.w);
    }
  }
  if (threadIdx.x < NB) sumx[threadIdx.x] = 0.f;
  __syncthreads();
  if (has_zero) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      float s = part[b];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(kFull, s, d);
      if (lane == 0) atomicAdd(&sumx[b], s);
    }
  }
  __syncthreads();

  uint32_t bad = 0;
  for (uint32_t row = blockIdx.x * kWarpsPerCta + warp; row < rows; row += gridDim.x * kWarpsPerCta) {
    float acc[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b] = 0.f;
    planes_row(reinterpret_cast<const uint4*>(codes + (size_t)row * gpr_pad), gpr_pad, raw + rawbase[row], table, K,
               bad, [&](uint32_t p, const uint32_t (&w)[8]) {
                 const float4* xp = xs4 + p * 256u + lane;
#pragma unroll
                 for (int j = 0; j < 8; ++j) {
                   const uint32_t v = w[j] ^ xor_mask;
                   const float f0 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7540)) - magic;
                   const float f1 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7541)) - magic;
                   const float f2 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7542)) - magic;
                   const float f3 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7543)) - magic;
#pragma unroll
                   for (int b = 0; b < NB; ++b) {
                     const float4 xv = xp[(size_t)b * slots + j * 32];
                     acc[b] = fmaf(f0, xv.x, acc[b]);
                     acc[b] = fmaf(f1, xv.y, acc[b]);
                     acc[b] = fmaf(f2, xv.z, acc[b]);
                     acc[b] = fmaf(f3, xv.w, acc[b]);
                   }
                 }
               });
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      float a = acc[b];
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) a += __shfl_xor_sync(kFull, a, d);
      acc[b] = a;
    }
    if (lane == 0) {
      const float s = scale[row];
      const float z = has_zero ? zero[row] : 0.f;
#pragma unroll
      for (int b = 0; b < NB; ++b) y[(size_t)b * rows + row] = s * (acc[b] - z * sumx[b]);
    }
  }
  if (bad) atomicOr(status, TQ_STATUS_BAD_CODE);
}

// ---------------------------------------------------------------------------------------------
// Per-row symmetric int8 quantizer (one CTA per row).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
quantize_rows_kernel(const float* __restrict__ w, uint32_t rows, uint32_t cols, int8_t* __restrict__ q,
                     float* __restrict__ scale) {
  __shared__ float red[8];
  __shared__ float s_sh;
  for (uint32_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const float* wr = w + (size_t)row * cols;
    float amax = 0.f;
    for (uint32_t c = threadIdx.x; c < cols; c += 256) amax = fmaxf(amax, fabsf(wr[c]));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, d));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
      float m = red[0];
      for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i]);
      const float s = m > 0.f ? __fdiv_rn(m, 127.0f) : 1.0f;
      s_sh = s;
      scale[row] = s;
    }
    __syncthreads();
    const float s = s_sh;
    for (uint32_t c = threadIdx.x; c < cols; c += 256) {
      float v = rintf(__fdiv_rn(wr[c], s));
      v = fminf(fmaxf(v, -127.f), 127.f);
      q[(size_t)row * cols + c] = (int8_t)v;
    }
    __syncthreads();
  }
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  }
  return n;
}

thread_local char g_cuda_msg[256] = "";

// Records the text of a CUDA failure for tq_last_cuda_error and maps it to TQ_ERR_CUDA.
inline int cuda_ok(cudaError_t e, const char* what = "") {
  if (e == cudaSuccess) return TQ_OK;
  snprintf(g_cuda_msg, sizeof(g_cuda_msg), "%s: %s (%s)", what, cudaGetErrorString(e), cudaGetErrorName(e));
  return TQ_ERR_CUDA;
}

template <int NB>
int launch_gemv(const tq_dmat* m, const __nv_bfloat16* x, float* y, cudaStream_t st) {
  const uint32_t rows = m->info.rows, cols = m->info.cols;
  const size_t smem = (size_t)NB * cols * sizeof(float);
  if (smem + 20 * 1024 > 48 * 1024) {  // static shared memory counts too
    if (int rc = tq_ensure_dynamic_smem((const void*)gemv_kernel<NB>, smem, "gemv: raising the dynamic shared memory limit"))
      return rc;
  }
  int per_sm = 0;
  if (int rc = cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gemv_kernel<NB>, kThreads, smem),
                       "gemv: occupancy query"))
    return rc;
  if (per_sm < 1) {
    snprintf(g_cuda_msg, sizeof(g_cuda_msg), "gemv: %zu bytes of shared memory do not fit one CTA", smem);
    return TQ_ERR_CUDA;
  }
  const uint32_t need = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  const uint32_t grid = std::min<uint32_t>(need, (uint32_t)(sm_count() * per_sm));
  gemv_kernel<NB><<<grid, kThreads, smem, st>>>(
      reinterpret_cast<const uint4*>(m->d_tokens), m->d_rowseg, m->d_scale, m->d_zero, m->has_zero,
      m->dict->d_table, m->dict->K, rows, cols, x, y, m->info.levels_signed ? 0x80808080u : 0u,
      m->info.levels_signed ? 8388736.0f : 8388608.0f, m->d_status);
  return cuda_ok(cudaGetLastError(), "gemv launch");
}

template <int NB>
int launch_gemv_planes(const tq_dmat* m, const __nv_bfloat16* x, float* y, cudaStream_t st) {
  const uint32_t rows = m->info.rows, cols = m->info.cols;
  const size_t slots = ((size_t)(m->gpr_pad + 255u) >> 8) << 8;
  const size_t smem = (size_t)NB * slots * sizeof(float4);
  if (smem + 4 * 1024 > 48 * 1024) {
    if (int rc = tq_ensure_dynamic_smem((const void*)gemv_planes_kernel<NB>, smem, "gemv(planes): raising the dynamic shared memory limit"))
      return rc;
  }
  int per_sm = 0;
  if (int rc = cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gemv_planes_kernel<NB>, kThreads, smem),
                       "gemv(planes): occupancy query"))
    return rc;
  if (per_sm < 1) {
    snprintf(g_cuda_msg, sizeof(g_cuda_msg), "gemv(planes): %zu bytes of shared memory do not fit one CTA", smem);
    return TQ_ERR_CUDA;
  }
  const uint32_t need = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  const uint32_t grid = std::min<uint32_t>(need, (uint32_t)(sm_count() * per_sm));
  gemv_planes_kernel<NB><<<grid, kThreads, smem, st>>>(
      m->d_codes, m->gpr_pad, m->d_rawbase, m->d_raw, m->d_scale, m->d_zero, m->has_zero, m->dict->d_table,
      m->dict->K, rows, cols, x, y, m->info.levels_signed ? 0x80808080u : 0u,
      m->info.levels_signed ? 8388736.0f : 8388608.0f, m->d_status);
  return cuda_ok(cudaGetLastError(), "gemv(planes) launch");
}

}  // namespace

int tq_cuda_status(int cuda_error, const char* what) { return cuda_ok((cudaError_t)cuda_error, what); }

int tq_ensure_dynamic_smem(const void* func, size_t bytes, const char* what) {
  static std::mutex mu;
  static std::map<std::pair<int, const void*>, size_t> raised;  // (device, kernel) -> limit set so far
  int dev = 0;
  if (int rc = cuda_ok(cudaGetDevice(&dev), what)) return rc;
  std::lock_guard<std::mutex> lock(mu);
  size_t& have = raised[std::make_pair(dev, func)];
  if (bytes > have) {
    if (int rc = cuda_ok(cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes), what)) return rc;
    have = bytes;
  }
  return TQ_OK;
}

extern "C" {

const char* tq_last_cuda_error(void) { return g_cuda_msg; }

int tq_quantize_rows_device(const float* d_w, uint32_t rows, uint32_t cols, int8_t* d_q, float* d_scale,
                            void* cuda_stream) {
  if (!d_w || !d_q || !d_scale || rows == 0 || cols == 0) return TQ_ERR_INVALID_ARG;
  const uint32_t grid = std::min<uint32_t>(rows, (uint32_t)sm_count() * 8u);
  quantize_rows_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(d_w, rows, cols, d_q, d_scale);
  return cuda_ok(cudaGetLastError());
}

int tq_dict_upload_size(const tq_dict* d, uint64_t* device_bytes) {
  if (!d || !device_bytes) return TQ_ERR_INVALID_ARG;
  // always the full 16-bit index range, zero past the last entry: any token is a safe index
  (void)d;
  *device_bytes = 65536ull * 4 + 256 + (uint64_t)kMapSlots * sizeof(tq_map_slot);  // table, then the window -> code map
  return TQ_OK;
}

int tq_dict_upload(const tq_dict* d, void* d_buf, uint64_t d_buf_bytes, void* cuda_stream, tq_ddict** out) {
  if (!d || !d_buf || !out || ((uintptr_t)d_buf & 255)) return TQ_ERR_INVALID_ARG;
  uint64_t need = 0;
  tq_dict_upload_size(d, &need);
  if (d_buf_bytes < need) return TQ_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (int rc = cuda_ok(cudaMemsetAsync(d_buf, 0, need, st), "table upload")) return rc;
  if (d->K) {
    if (int rc = cuda_ok(cudaMemcpyAsync(static_cast<uint8_t*>(d_buf) + 4, d->entries.data(), (size_t)d->K * 4,
                                         cudaMemcpyHostToDevice, st), "table upload"))
      return rc;
  }
  std::vector<tq_map_slot> map(kMapSlots);
  for (uint32_t i = 0; i < kMapSlots; ++i) map[i] = tq_map_slot{d->map_key[i], d->map_code[i]};
  uint8_t* d_map = static_cast<uint8_t*>(d_buf) + 65536ull * 4 + 256;
  if (int rc = cuda_ok(cudaMemcpyAsync(d_map, map.data(), map.size() * sizeof(tq_map_slot), cudaMemcpyHostToDevice, st), "table upload"))
    return rc;
  if (int rc = cuda_ok(cudaStreamSynchronize(st), "table upload")) return rc;
  tq_ddict* dd = new (std::nothrow) tq_ddict();
  if (!dd) return TQ_ERR_NOMEM;
  dd->K = d->K;
  dd->d_table = static_cast<const uint32_t*>(d_buf);
  dd->d_map = reinterpret_cast<const tq_map_slot*>(d_map);
  try {
    dd->h_table.assign((size_t)d->K + 1, 0u);
  } catch (const std::bad_alloc&) {
    delete dd;
    return TQ_ERR_NOMEM;
  }
  if (d->K) std::memcpy(dd->h_table.data() + 1, d->entries.data(), (size_t)d->K * 4);
  *out = dd;
  return TQ_OK;
}

void tq_ddict_free(tq_ddict* d) { delete d; }

int tq_upload_size(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols, int layout,
                   uint64_t* device_bytes) {
  if (!device_bytes) return TQ_ERR_INVALID_ARG;
  if (layout == TQ_LAYOUT_STREAM)
    return tq_build_stream_image(stream, stream_len, rows, cols, 0xFFFFFFFFu, nullptr, nullptr, device_bytes, nullptr);
  if (layout == TQ_LAYOUT_PLANES)
    return tq_build_planes_image(stream, stream_len, rows, cols, 0xFFFFFFFFu, nullptr, nullptr, device_bytes, nullptr);
  if (layout == TQ_LAYOUT_TILES)
    return tq_build_tiles_image(stream, stream_len, rows, cols, 0xFFFFFFFFu, nullptr, nullptr, nullptr, device_bytes, nullptr);
  return TQ_ERR_INVALID_ARG;
}

int tq_upload(const tq_ddict* dict, const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
              const float* row_scale, const float* row_zero, int levels_signed, int layout, void* d_buf,
              uint64_t d_buf_bytes, void* cuda_stream, tq_dmat** out) {
  if (!dict || !stream || !row_scale || !d_buf || !out || ((uintptr_t)d_buf & 255) ||
      (layout != TQ_LAYOUT_STREAM && layout != TQ_LAYOUT_PLANES && layout != TQ_LAYOUT_TILES))
    return TQ_ERR_INVALID_ARG;
  if (cols / 4 > 65504u) return TQ_ERR_UNSUPPORTED_SHAPE;  // per-row marker counts are 16-bit
  cudaStream_t st = (cudaStream_t)cuda_stream;
  tq_dmat* m = new (std::nothrow) tq_dmat();
  if (!m) return TQ_ERR_NOMEM;
  uint8_t* base = static_cast<uint8_t*>(d_buf);
  uint64_t need = 0, n_hits = 0, n_miss = 0;
  int rc;
  if (layout == TQ_LAYOUT_STREAM) {
    tq_host_image img;
    rc = tq_build_stream_image(stream, stream_len, rows, cols, dict->K, row_scale, row_zero, &need, &img);
    if (rc == TQ_OK && d_buf_bytes < need) rc = TQ_ERR_BUFFER_TOO_SMALL;
    if (rc == TQ_OK) rc = cuda_ok(cudaMemcpyAsync(d_buf, img.blob.data(), img.blob.size(), cudaMemcpyHostToDevice, st), "upload");
    if (rc == TQ_OK) rc = cuda_ok(cudaStreamSynchronize(st), "upload");
    if (rc != TQ_OK) { delete m; return rc; }
    m->d_status = reinterpret_cast<uint32_t*>(base + img.off_status);
    m->d_rowseg = reinterpret_cast<const tq_rowseg*>(base + img.off_rowseg);
    m->d_scale = reinterpret_cast<const float*>(base + img.off_scale);
    m->d_zero = reinterpret_cast<const float*>(base + img.off_zero);
    m->d_tokens = reinterpret_cast<const uint16_t*>(base + img.off_tokens);
    m->token_chunks = img.token_chunks;
    n_hits = img.n_hits;
    n_miss = img.n_miss;
    m->info.payload_bytes = img.token_chunks * 16 + (uint64_t)rows * (sizeof(tq_rowseg) + 4 + (row_zero ? 4 : 0));
  } else if (layout == TQ_LAYOUT_TILES) {
    tq_tiles_image img;
    rc = tq_build_tiles_image(stream, stream_len, rows, cols, dict->K, dict->h_table.data(), row_scale, row_zero, &need, &img);
    if (rc == TQ_OK && d_buf_bytes < need) rc = TQ_ERR_BUFFER_TOO_SMALL;
    if (rc == TQ_OK) rc = cuda_ok(cudaMemcpyAsync(d_buf, img.blob.data(), img.blob.size(), cudaMemcpyHostToDevice, st), "upload");
    if (rc == TQ_OK) rc = cuda_ok(cudaStreamSynchronize(st), "upload");
    if (rc != TQ_OK) { delete m; return rc; }
    m->d_status = reinterpret_cast<uint32_t*>(base + img.off_status);
    m->d_scale = reinterpret_cast<const float*>(base + img.off_scale);
    m->d_zero = reinterpret_cast<const float*>(base + img.off_zero);
    tq_tiles_desc& t = m->tiles;
    t.tokens = reinterpret_cast<const uint4*>(base + img.off_tokens);
    t.raw = reinterpret_cast<const uint32_t*>(base + img.off_raw);
    t.tile_raw = reinterpret_cast<const uint32_t*>(base + img.off_tile_raw);
    t.scale = m->d_scale;
    t.zero = m->d_zero;
    t.status = m->d_status;
    t.rows = rows;
    t.cols = cols;
    t.steps = img.steps;
    t.row_blocks = img.row_blocks;
    t.has_zero = row_zero != nullptr;
    t.table_words = TQ_TILES_TABLE_WORDS;
    t.xdig = base + tq_tiles_layout(rows, cols).off_xdig(img.n_raw);
    m->rb_raw = std::move(img.rb_raw);
    n_hits = img.n_hits;
    n_miss = img.n_miss;
    const uint64_t n_tiles = (uint64_t)img.steps * img.row_blocks;
    m->info.payload_bytes = n_tiles * 1024 + img.n_raw * 4 + (n_tiles + 1) * 4 + (uint64_t)rows * (4 + (row_zero ? 4 : 0));
    m->info.n_raw_words = img.n_raw;
  } else {
    tq_planes_image img;
    rc = tq_build_planes_image(stream, stream_len, rows, cols, dict->K, row_scale, row_zero, &need, &img);
    if (rc == TQ_OK && d_buf_bytes < need) rc = TQ_ERR_BUFFER_TOO_SMALL;
    if (rc == TQ_OK) rc = cuda_ok(cudaMemcpyAsync(d_buf, img.blob.data(), img.blob.size(), cudaMemcpyHostToDevice, st), "upload");
    if (rc == TQ_OK) rc = cuda_ok(cudaStreamSynchronize(st), "upload");
    if (rc != TQ_OK) { delete m; return rc; }
    m->d_status = reinterpret_cast<uint32_t*>(base + img.off_status);
    m->d_rawbase = reinterpret_cast<const uint32_t*>(base + img.off_rawbase);
    m->d_rawidx = reinterpret_cast<const uint16_t*>(base + img.off_rawidx);
    m->d_scale = reinterpret_cast<const float*>(base + img.off_scale);
    m->d_zero = reinterpret_cast<const float*>(base + img.off_zero);
    m->d_codes = reinterpret_cast<const uint16_t*>(base + img.off_codes);
    m->d_raw = reinterpret_cast<const uint32_t*>(base + img.off_raw);
    m->gpr_pad = img.gpr_pad;
    m->nidx_pad = img.nidx_pad;
    n_hits = img.n_hits;
    n_miss = img.n_miss;
    m->info.payload_bytes = (uint64_t)rows * img.gpr_pad * 2 + n_miss * 4 + (uint64_t)rows * (4 + 4 + (row_zero ? 4 : 0));
  }
  m->dict = dict;
  m->has_zero = row_zero != nullptr;
  m->zero_bf16_exact = tq_zero_bf16_exact(row_zero, rows, levels_signed != 0);
  m->info.rows = rows;
  m->info.cols = cols;
  m->info.K = dict->K;
  m->info.layout = layout;
  m->info.levels_signed = levels_signed != 0;
  m->info.n_hits = n_hits;
  m->info.n_miss = n_miss;
  m->info.stream_bytes = 2 * (n_hits + 5 * n_miss);
  if (layout != TQ_LAYOUT_TILES) m->info.n_raw_words = n_miss;
  m->info.device_bytes = need;
  *out = m;
  return TQ_OK;
}

int tq_upload_device_size(uint32_t rows, uint32_t cols, uint64_t* device_bytes) {
  if (!device_bytes || rows == 0 || cols == 0) return TQ_ERR_INVALID_ARG;
  if (cols % 4 != 0 || cols > TQ_TILES_MAX_COLS) return TQ_ERR_UNSUPPORTED_SHAPE;
  const tq_tiles_geometry geo = tq_tiles_layout(rows, cols);
  if (geo.n_tiles >= (1ull << 31) || (uint64_t)rows * (cols / 4) >= (1ull << 32) - 65536) return TQ_ERR_UNSUPPORTED_SHAPE;
  *device_bytes = geo.total((uint64_t)rows * (cols / 4));  // every group raw
  return TQ_OK;
}

int tq_upload_device(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols,
                     const float* d_row_scale, const float* d_row_zero, int levels_signed, void* d_buf,
                     uint64_t d_buf_bytes, void* cuda_stream, tq_dmat** out) {
  if (!dict || !d_levels || !d_row_scale || !d_buf || !out || ((uintptr_t)d_buf & 255) || ((uintptr_t)d_levels & 15))
    return TQ_ERR_INVALID_ARG;
  uint64_t need = 0;
  if (int rc = tq_upload_device_size(rows, cols, &need)) return rc;
  if (d_buf_bytes < need) return TQ_ERR_BUFFER_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  uint8_t* base = static_cast<uint8_t*>(d_buf);
  if (int rc = tq_tiles_build_device(dict, d_levels, rows, cols, d_row_scale, d_row_zero, base, cuda_stream)) return rc;
  const tq_tiles_geometry geo = tq_tiles_layout(rows, cols);
  tq_dmat* m = new (std::nothrow) tq_dmat();
  if (!m) return TQ_ERR_NOMEM;
  std::vector<uint32_t> tile_raw;
  std::vector<float> zeros;
  unsigned long long counters[2] = {0, 0};
  int rc = TQ_OK;
  try {
    tile_raw.resize(geo.n_tiles + 1);
    if (d_row_zero) zeros.resize(rows);
  } catch (const std::bad_alloc&) {
    rc = TQ_ERR_NOMEM;
  }
  if (rc == TQ_OK && d_row_zero)
    rc = cuda_ok(cudaMemcpyAsync(zeros.data(), d_row_zero, (size_t)rows * 4, cudaMemcpyDeviceToHost, st), "device upload");
  if (rc == TQ_OK)
    rc = cuda_ok(cudaMemcpyAsync(tile_raw.data(), base + geo.off_tile_raw, tile_raw.size() * 4, cudaMemcpyDeviceToHost, st), "device upload");
  if (rc == TQ_OK) rc = cuda_ok(cudaMemcpyAsync(counters, base + 64, sizeof(counters), cudaMemcpyDeviceToHost, st), "device upload");
  if (rc == TQ_OK) rc = cuda_ok(cudaStreamSynchronize(st), "device upload");
  if (rc != TQ_OK) {
    delete m;
    return rc;
  }
  const uint64_t n_raw = tile_raw[geo.n_tiles];
  m->rb_raw.resize((size_t)geo.row_blocks + 1);
  for (uint32_t rb = 0; rb <= geo.row_blocks; ++rb) m->rb_raw[rb] = tile_raw[(uint64_t)rb * geo.steps];
  m->dict = dict;
  m->has_zero = d_row_zero != nullptr;
  m->zero_bf16_exact = tq_zero_bf16_exact(d_row_zero ? zeros.data() : nullptr, rows, levels_signed != 0);
  m->d_status = reinterpret_cast<uint32_t*>(base + geo.off_status);
  m->d_scale = reinterpret_cast<const float*>(base + geo.off_scale);
  m->d_zero = reinterpret_cast<const float*>(base + geo.off_zero);
  tq_tiles_desc& t = m->tiles;
  t.tokens = reinterpret_cast<const uint4*>(base + geo.off_tokens);
  t.raw = reinterpret_cast<const uint32_t*>(base + geo.off_raw);
  t.tile_raw = reinterpret_cast<const uint32_t*>(base + geo.off_tile_raw);
  t.scale = m->d_scale;
  t.zero = m->d_zero;
  t.status = m->d_status;
  t.rows = rows;
  t.cols = cols;
  t.steps = geo.steps;
  t.row_blocks = geo.row_blocks;
  t.has_zero = d_row_zero != nullptr;
  t.table_words = TQ_TILES_TABLE_WORDS;
  t.xdig = base + geo.off_xdig(n_raw);
  m->info.rows = rows;
  m->info.cols = cols;
  m->info.K = dict->K;
  m->info.layout = TQ_LAYOUT_TILES;
  m->info.levels_signed = levels_signed != 0;
  m->info.n_hits = counters[0];
  m->info.n_miss = counters[1];
  m->info.stream_bytes = 2 * (counters[0] + 5 * counters[1]);
  m->info.n_raw_words = n_raw;
  m->info.payload_bytes = geo.n_tiles * 1024 + n_raw * 4 + (geo.n_tiles + 1) * 4 + (uint64_t)rows * (4 + (d_row_zero ? 4 : 0));
  m->info.device_bytes = geo.total(n_raw);
  *out = m;
  return TQ_OK;
}

int tq_upload_device_rows(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols, uint32_t row_begin,
                          uint32_t row_end, const float* d_row_scale, const float* d_row_zero, int levels_signed,
                          void* d_buf, uint64_t d_buf_bytes, void* cuda_stream, tq_dmat** out) {
  if (!d_levels || !d_row_scale || row_begin >= row_end || row_end > rows || cols == 0) return TQ_ERR_INVALID_ARG;
  // a row range of a row-major matrix is a matrix of its own: same table, its own image
  const uint8_t* first = d_levels + (uint64_t)row_begin * cols;
  if ((uintptr_t)first & 15) return TQ_ERR_INVALID_ARG;
  return tq_upload_device(dict, first, row_end - row_begin, cols, d_row_scale + row_begin,
                          d_row_zero ? d_row_zero + row_begin : nullptr, levels_signed, d_buf, d_buf_bytes, cuda_stream, out);
}

int tq_dmat_get_info(const tq_dmat* m, tq_dmat_info* info) {
  if (!m || !info) return TQ_ERR_INVALID_ARG;
  *info = m->info;
  return TQ_OK;
}

void tq_dmat_free(tq_dmat* m) { delete m; }

int tq_decompress(const tq_dmat* m, uint8_t* d_codes, void* cuda_stream) {
  if (!m || !d_codes || ((uintptr_t)d_codes & 15)) return TQ_ERR_INVALID_ARG;
  const uint32_t need = (m->info.rows + kWarpsPerCta - 1) / kWarpsPerCta;
  const uint32_t grid = std::min<uint32_t>(need, (uint32_t)sm_count() * 8u);
  if (m->info.layout == TQ_LAYOUT_TILES) return tq_tiles_decompress(m, d_codes, cuda_stream);
  if (m->info.layout == TQ_LAYOUT_PLANES) {
    decompress_planes_kernel<<<grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(
        m->d_codes, m->gpr_pad, m->d_rawbase, m->d_raw, m->dict->d_table, m->dict->K, m->info.rows, m->info.cols,
        reinterpret_cast<uint32_t*>(d_codes), m->d_status);
    return cuda_ok(cudaGetLastError(), "decompress(planes) launch");
  }
  decompress_kernel<<<grid, kThreads, 0, (cudaStream_t)cuda_stream>>>(
      reinterpret_cast<const uint4*>(m->d_tokens), m->d_rowseg, m->dict->d_table, m->dict->K, m->info.rows,
      m->info.cols, reinterpret_cast<uint32_t*>(d_codes), m->d_status);
  return cuda_ok(cudaGetLastError());
}

int tq_fused_gemv(const tq_dmat* m, const void* d_x_bf16, int B, float* d_y, void* cuda_stream) {
  if (!m || !d_x_bf16 || !d_y || B < 1 || B > 32 || ((uintptr_t)d_x_bf16 & 15)) return TQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(d_x_bf16);
  const uint32_t rows = m->info.rows, cols = m->info.cols;
  if (m->info.layout == TQ_LAYOUT_TILES) return tq_tiles_gemv(m, x, B, d_y, cuda_stream);
  // fp32 x for up to 4 batch columns must fit the 227 KB of shared memory
  const bool planes = m->info.layout == TQ_LAYOUT_PLANES;
  const size_t xcols = planes ? ((((size_t)m->gpr_pad + 255) >> 8) << 10) : cols;  // staged columns per batch column
  const int max_nb = 4 * xcols * 4 <= 200 * 1024 ? 4 : (2 * xcols * 4 <= 200 * 1024 ? 2 : 1);
  if (xcols * 4 > 200 * 1024) return TQ_ERR_UNSUPPORTED_SHAPE;
  for (int b0 = 0; b0 < B;) {
    const int nb = std::min(B - b0, max_nb);
    int rc;
    const __nv_bfloat16* xb = x + (size_t)b0 * cols;
    float* yb = d_y + (size_t)b0 * rows;
    switch (nb) {
      case 1: rc = planes ? launch_gemv_planes<1>(m, xb, yb, st) : launch_gemv<1>(m, xb, yb, st); break;
      case 2: rc = planes ? launch_gemv_planes<2>(m, xb, yb, st) : launch_gemv<2>(m, xb, yb, st); break;
      case 3: rc = planes ? launch_gemv_planes<3>(m, xb, yb, st) : launch_gemv<3>(m, xb, yb, st); break;
      default: rc = planes ? launch_gemv_planes<4>(m, xb, yb, st) : launch_gemv<4>(m, xb, yb, st); break;
    }
    if (rc != TQ_OK) return rc;
    b0 += nb;
  }
  return TQ_OK;
}

int tq_fused_gemv_host(const tq_dmat* m, const void* h_x_bf16, int B, float* h_y, void* d_x_stage,
                       float* d_y_stage, void* cuda_stream) {
  if (!m || !h_x_bf16 || !h_y || !d_x_stage || !d_y_stage || B < 1 || B > 32) return TQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(d_x_stage, h_x_bf16, (size_t)B * m->info.cols * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return TQ_ERR_CUDA;
  int rc = tq_fused_gemv(m, d_x_stage, B, d_y_stage, cuda_stream);
  if (rc != TQ_OK) return rc;
  if (cudaMemcpyAsync(h_y, d_y_stage, (size_t)B * m->info.rows * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TQ_ERR_CUDA;
  return TQ_OK;
}

// Staging memory of tq_fused_gemv_host_static: lives in the library image, so every GPU that
// loads the library holds these 1.5 MiB until the process exits.  Host code cannot use the
// symbol as a pointer; static_stage() asks the runtime for its address on the current device.
constexpr uint64_t kStaticXElems = 262144;  // bf16 elements of x the staging area can hold
constexpr uint64_t kStaticYElems = 262144;  // fp32 elements of y the staging area can hold
static __device__ __align__(256) unsigned char g_static_stage[kStaticXElems * 2 + kStaticYElems * 4];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mu;
static unsigned char* g_static_ptr[kMaxDevices] = {};

// Device address of g_static_stage on the current device (looked up once per device).
static int static_stage(unsigned char** out) {
  int dev = -1;
  if (int rc = cuda_ok(cudaGetDevice(&dev), "static staging: current device")) return rc;
  if (dev < 0 || dev >= kMaxDevices) return TQ_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    if (int rc = cuda_ok(cudaGetSymbolAddress(&p, g_static_stage), "static staging: symbol address")) return rc;
    g_static_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[dev];
  return TQ_OK;
}

int tq_fused_gemv_host_static(const tq_dmat* m, const void* h_x_bf16, int B, float* h_y, void* cuda_stream) {
  if (!m || !h_x_bf16 || !h_y || B < 1 || B > 32) return TQ_ERR_INVALID_ARG;
  if ((uint64_t)B * m->info.cols > kStaticXElems || (uint64_t)B * m->info.rows > kStaticYElems) {
    snprintf(g_cuda_msg, sizeof(g_cuda_msg),
             "tq_fused_gemv_host_static: B*cols = %llu (limit %llu) or B*rows = %llu (limit %llu) exceeds the "
             "built-in staging area; use tq_fused_gemv_host with caller-provided staging",
             (unsigned long long)B * m->info.cols, (unsigned long long)kStaticXElems,
             (unsigned long long)B * m->info.rows, (unsigned long long)kStaticYElems);
    return TQ_ERR_UNSUPPORTED_SHAPE;
  }
  // The staging array that is looked up belongs to the current device; the kernel runs where the
  // matrix lives.  A caller who has another device current would hand the kernel that device's address.
  int dev = -1;
  cudaPointerAttributes attr{};
  if (int rc = cuda_ok(cudaGetDevice(&dev), "static staging: current device")) return rc;
  if (int rc = cuda_ok(cudaPointerGetAttributes(&attr, m->d_status), "static staging: device of the matrix")) return rc;
  if (attr.type != cudaMemoryTypeDevice || attr.device != dev) {
    snprintf(g_cuda_msg, sizeof(g_cuda_msg),
             "tq_fused_gemv_host_static: the matrix lives on device %d but device %d is current", attr.device, dev);
    return TQ_ERR_INVALID_ARG;
  }
  unsigned char* stage = nullptr;
  if (int rc = static_stage(&stage)) return rc;
  return tq_fused_gemv_host(m, h_x_bf16, B, h_y, stage, reinterpret_cast<float*>(stage + kStaticXElems * 2),
                            cuda_stream);
}

int tq_device_status(const tq_dmat* m, void* cuda_stream, uint32_t* status) {
  if (!m || !status) return TQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (cudaMemcpyAsync(status, m->d_status, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return TQ_ERR_CUDA;
  if (cudaMemsetAsync(m->d_status, 0, 4, st) != cudaSuccess) return TQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TQ_ERR_CUDA;
  return TQ_OK;
}

}  // extern "C"
