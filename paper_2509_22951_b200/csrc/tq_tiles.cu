// Kernels of the TILES layout (sm_100a): fused decode + GEMV on the 8-bit integer tensor-core
// path, and decompress.
//
// Why integer MMAs for a matrix-vector product.  A decoded group is a 32-bit word holding four
// 8-bit levels of one row -- exactly one A-operand register of mma.m16n8k32 (16 rows x 32 columns
// of 8-bit values, 32-bit accumulators).  A warp that owns 16 rows therefore feeds every word it
// looks up to the tensor core as is: no unpacking, no int->float conversion, no FMA chain.  The
// activations take the B operand.  A bf16 activation vector is turned, once per CTA, into a
// block-fixed-point integer X[c] = round(x[c] * 2^(30-e)) (2^e > max |x|, so |X| <= 2^30) and
// split into four balanced base-256 digits X = d0 + 2^8 d1 + 2^16 d2 + 2^24 d3, each a signed
// byte; the four digit vectors are four of the eight B columns.  All sums are exact integers, so
//   y[r] = scale_r * ( 2^(e-30) * (D0 + 2^8 D1 + 2^16 D2 + 2^24 D3) - zero_r * 2^(e-30) * sum_c X[c] )
// differs from the exact product only by the rounding of x to a grid 30 bits below the power of
// two above its largest element: |error of the sum for row r| <= 2^(e-31) * sum_c |q[r][c] - zero_r|.
// An element keeps all 8 significant bits of its bf16 value while it is no more than 2^22 times
// smaller than the largest one.  The result does not depend on how the columns are split among
// warps.  Two batch columns fill one MMA (8 of 8 B columns).
//
// Data movement.  One persistent CTA per SM keeps the table (TQ_TILES_TABLE_WORDS words) in shared
// memory: lookups there are bank-conflict limited, not tag limited like divergent global loads.
// Each warp walks a contiguous run of tiles.  Token tiles come through registers, two tiles
// ahead.  Raw words come through a per-warp ring of TQ_TILES_RING_WORDS words in shared memory
// that one lane keeps filled with 2 KB bulk copies (cp.async.bulk + mbarrier); raw word p of
// the matrix always sits in ring slot p mod ring size, and that slot number is what a miss token
// carries, so a lookup is: token -> (token >= 0xFC00 ? ring : table)[token] -> MMA operand.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <new>
#include <vector>

#include "tq_tiles_common.cuh"

namespace {

// One segment with everything a CTA needs to run it, in one 128-byte line: [begin, end) are the segments
// of the CTA the record belongs to, seg and desc this segment and its matrix.
struct SegRecord {
  uint32_t begin, end;
  TilesSeg seg;
  uint32_t pad0;
  tq_tiles_desc desc;
  uint32_t pad1[2];
};
static_assert(sizeof(SegRecord) == 128, "one record = one 128-byte line, fetched by one warp");

struct TilesParams {
  const SegRecord* firsts;    // stack mode: DEVICE, per CTA the record of its first segment; nullptr in single-matrix mode
  const SegRecord* recs;      // stack mode: DEVICE, one record per segment, grouped by CTA
  tq_tiles_desc one;          // single-matrix mode
  const uint32_t* table;      // 65536 words, zero past the last entry
  uint32_t table_words;       // words of it kept in shared memory
  uint32_t xstride;           // words per digit column in shared memory
  uint32_t test_withhold;     // test hook (tq_test_withhold_table_chunk): expect a table chunk that is never copied
  };

template <bool SIGNED>
__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  if (SIGNED) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}

// Per-CTA values of the activation vectors of the current segment.
struct XInfo {
  double out_scale[2];  // 2^(e-30), NaN for a vector with a non-finite element
};
// Places inside the misc area of the shared-memory plan (TilesCta): XInfo at +192, the warps' sums of the
// fixed-point values at +512.
// The record of the CTA's first segment, fetched by one warp during the set-up (gemv_tiles_kernel): at +768.
// Barrier "the digits of this segment's activations are in shared memory" (one arrival per warp): at +416.
constexpr uint32_t kXReadyBarOffset = 416u;
constexpr uint32_t kFirstSegmentOffset = 768u;
static_assert(kFirstSegmentOffset + sizeof(SegRecord) <= 1024u, "misc area of the shared-memory plan");
constexpr int kTilesWarpsC = 16;
constexpr uint32_t kXInfoOffset = 192u, kWarpSumsOffset = 512u, kWarpSumsFromXInfo = kWarpSumsOffset - kXInfoOffset;

// Turns the 16 x 8 accumulator tile (MMA fragment layout: lane 4g+t holds rows g, g+8 and columns
// 2t, 2t+1) of row block rb into y.  Lane L gathers the four digit sums of row L & 15, batch
// column L >> 4 with shuffles.
template <int NB>
__device__ __noinline__ void tiles_finalize(const float* __restrict__ scale, const float* __restrict__ zero,
                                            float* __restrict__ y, uint32_t rows, uint32_t has_zero, const XInfo* xi,
                                            uint32_t rb, int c0, int c1, int c2, int c3) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t row = lane & 15u, b = lane >> 4;
  long long Y = 0;
#pragma unroll
  for (int k = 0; k < kDigits; ++k) {
    const uint32_t col = min((uint32_t)kDigits * b + k, 7u);
    const uint32_t src = (row & 7u) * 4u + (col >> 1);
    const int v0 = __shfl_sync(kFull, c0, src), v1 = __shfl_sync(kFull, c1, src);
    const int v2 = __shfl_sync(kFull, c2, src), v3 = __shfl_sync(kFull, c3, src);
    const int lo = (col & 1u) ? v1 : v0, hi = (col & 1u) ? v3 : v2;
    Y += (long long)((row & 8u) ? hi : lo) << (8 * k);
  }
  const uint32_t r = rb * 16u + row;
  if (b < (uint32_t)NB && r < rows) {
    double v = (double)Y * xi->out_scale[b];
    if (has_zero) {  // zero_r * sum_c x[c] on the same grid: the warps' sums of the fixed-point values
      const long long* warp_sums = reinterpret_cast<const long long*>(reinterpret_cast<const uint8_t*>(xi) + kWarpSumsFromXInfo);
      long long sx = 0;
      for (int w = 0; w < kTilesWarpsC; ++w) sx += warp_sums[b * kTilesWarpsC + w];
      v -= (double)zero[r] * (xi->out_scale[b] * (double)sx);
    }
    y[(size_t)b * rows + r] = (float)((double)scale[r] * v);
  }
}

template <int W, int NB, bool SIGNED>
struct TilesCta : CtaBase {
  static constexpr int kThreads = W * 32;
  static constexpr int NCOL = kDigits * NB;
  static_assert(W == kTilesWarpsC, "tiles_finalize sums the per-warp values of kTilesWarpsC warps");

  uint32_t xstride;
  uint32_t x_phase = 0;  // segments run so far: the phase the x-ready barrier completes next
  bool dead = false, waited = false;

  __device__ __forceinline__ uint32_t* misc_u32() { return reinterpret_cast<uint32_t*>(smem + L.misc); }
  // misc (1 KB): [0] dead flag; +16 partial ids [2W]; +192 XInfo; +224 per-warp maxima [NB][W]; +400 table
  // barrier; +416 x-ready barrier; +512 per-warp sums of the fixed-point values [NB][W] (64-bit); +768 the
  // record of the CTA's first segment
  __device__ __forceinline__ uint32_t* part_ids() { return misc_u32() + 4; }
  __device__ __forceinline__ XInfo* xinfo() { return reinterpret_cast<XInfo*>(smem + L.misc + kXInfoOffset); }
  __device__ __forceinline__ uint32_t* warp_max() { return reinterpret_cast<uint32_t*>(smem + L.misc + 224); }
  __device__ __forceinline__ long long* warp_sum() { return reinterpret_cast<long long*>(smem + L.misc + kWarpSumsOffset); }

  // ---- activation vectors -> digit columns in shared memory --------------------------------
  // Every thread keeps its groups of x in registers between the search for the largest magnitude and
  // the conversion, so x is read once; one CTA barrier in the middle (per-warp maxima); the caller tells
  // the x-ready barrier when this warp's share is written.  Rows of up to kMaxItems * kThreads groups (10240 columns) fit; longer rows
  // do not come here (their digits would not fit beside the table either).
  static constexpr int kMaxItems = 5;
  template <class Mid>
  __device__ __forceinline__ void prepare_x(const tq_tiles_desc& d, Mid&& between) {
    const uint32_t tid = threadIdx.x;
    const uint32_t G = d.cols >> 2;
    uint32_t* xs = reinterpret_cast<uint32_t*>(smem + L.x);
    const uint2* xg = reinterpret_cast<const uint2*>(d.x);
    uint2 v[NB][kMaxItems];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      uint32_t m = 0;
#pragma unroll
      for (int it = 0; it < kMaxItems; ++it) {
        const uint32_t g = tid + (uint32_t)it * kThreads;
        v[b][it] = g < G ? __ldg(xg + (size_t)b * G + g) : make_uint2(0u, 0u);
        m = amax4(v[b][it], m);
      }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) m = max(m, __shfl_xor_sync(kFull, m, s));
      if (lane == 0) warp_max()[b * W + warp] = m;
    }
    __syncthreads();
    between();  // work that needs the rings free and does not need x: placed behind the loads of x
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      uint32_t mb = 0;
#pragma unroll
      for (int w = 0; w < W; ++w) mb = max(mb, warp_max()[b * W + w]);
      const FixScale f = fix_scale(mb);
      const float s1 = f.finite ? f.s1 : 0.f;  // a non-finite vector: all digits zero, NaN output scale
      long long sum = 0;
#pragma unroll
      for (int it = 0; it < kMaxItems; ++it) {
        const uint32_t g = tid + (uint32_t)it * kThreads;
        if (g < G) {
          uint32_t w[kDigits];
          fix_digits(v[b][it], s1, f.s2, w, &sum);
#pragma unroll
          for (int k = 0; k < kDigits; ++k) xs[(kDigits * b + k) * xstride + g] = w[k];
        }
      }
      if (d.has_zero) {
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) sum += __shfl_xor_sync(kFull, sum, s);
        if (lane == 0) warp_sum()[b * W + warp] = sum;
      }
      if (tid == 0) xinfo()->out_scale[b] = fix_out_scale(f);
    }
    // digit words of the groups between G and the end of the last tile are never initialised: they
    // only ever multiply the zero bytes that token 0 decodes to, and integers have no NaN.
  }

  // ---- results ----------------------------------------------------------------------------
  __device__ __forceinline__ void finalize(const tq_tiles_desc& d, uint32_t rb, int c0, int c1, int c2, int c3) {
    tiles_finalize<NB>(d.scale, d.zero, d.y, d.rows, d.has_zero, xinfo(), rb, c0, c1, c2, c3);
  }

  // Partial sums of a row block shared with a neighbouring warp; parked in the warp's own ring,
  // which is idle by then.
  __device__ __forceinline__ void store_partial(uint32_t slot, uint32_t rb, const int (&c)[4]) {
    int4* p = reinterpret_cast<int4*>(smem + L.ring + warp * (kRingWords * 4u) + slot * 512u);
    p[lane] = make_int4(c[0], c[1], c[2], c[3]);
    if (lane == 0) part_ids()[2 * warp + slot] = rb;
  }

  // ---- the start of a warp's run, fetched before the activations are prepared ----------------
  // The tile index and the tokens are constant data, so their loads are issued at the very start of a
  // segment (for a CTA's first segment: before the wait for the preceding kernel) and their latency
  // passes under the set-up of the activations; the first raw chunks follow as soon as the rings are free.
  // The values travel as plain variables: gathered in a struct the same code was measured 3 % slower in
  // the tile loop (the compiler then recomputes loop constants in every iteration).
  __device__ __forceinline__ void load_head(const tq_tiles_desc& d, uint32_t t0, uint32_t t1, uint32_t& h_rd,
                                            uint32_t& h_stop_pos, uint4 (&h_q)[2][2], uint32_t (&h_tr)[2]) {
    h_rd = __ldg(d.tile_raw + t0);
    h_stop_pos = __ldg(d.tile_raw + t1);  // raw words of the run end here
    const uint4* tok = d.tokens + (size_t)t0 * 64u + lane;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      h_q[k][0] = ldg_stream(tok + k * 64);
      h_q[k][1] = ldg_stream(tok + k * 64 + 32);
      h_tr[k] = __ldg(d.tile_raw + t0 + 1 + k);
    }
    // the row scales of the row blocks this run shares with its neighbours are wanted by whoever merges
    // the partial sums at the end of the segment: brought near now
    const uint32_t S = d.steps;
    if (lane < 4u) {
      const uint32_t t = (lane & 1u) ? t1 : t0;
      const float* a = ((lane & 2u) ? d.zero : d.scale) + (size_t)(t / S) * 16u;
      if (t % S != 0u && ((lane & 2u) == 0u || d.has_zero)) asm volatile("prefetch.global.L1 [%0];" ::"l"(a));
    }
  }
  __device__ __forceinline__ void first_chunks(const tq_tiles_desc& d, uint32_t h_rd, uint32_t h_stop_pos,
                                               uint32_t& h_w_pos, uint32_t& h_i_pos) {
    h_w_pos = h_rd & ~(uint32_t)(kChunkWords - 1);  // first word of the next chunk to wait for
    h_i_pos = h_w_pos;                              // first word of the next chunk to issue
    for (int k = 0; k < kSlots && h_i_pos < h_stop_pos; ++k, h_i_pos += kChunkWords) issue_chunk(d.raw, h_i_pos);
  }

  // ---- one warp, tiles [t0, t1) of matrix d -------------------------------------------------
  // Tile i of the run uses token registers q[i & 1] and word buffer i & 1; its words are consumed
  // by the MMAs while tile i + 1 is being looked up, and its token registers are reloaded (two
  // tiles ahead) only after the last use, so no register is copied while a load into it is in
  // flight.
  // rd, stop_pos, q, tr: what load_head fetched; w_pos, i_pos: where first_chunks left the raw stream
  // (q[k], tr[k]: tokens of tile t0 + k and the index of the first raw word behind it).
  __device__ __forceinline__ void run_tiles(const tq_tiles_desc& d, uint32_t t0, uint32_t t1, uint32_t rd,
                                            const uint32_t stop_pos, uint32_t w_pos, uint32_t i_pos, uint4 (&q)[2][2],
                                            uint32_t (&tr)[2]) {
    if (!wait_table()) {  // the table copy started with the kernel; its first use is here
      dead = true;
      *dead_flag() = 1u;
      if (lane == 0) atomicOr(d.status, TQ_STATUS_WAIT_EXPIRED);
      return;
    }
    const uint32_t S = d.steps;
    const uint32_t g = lane >> 2, t = lane & 3u;
    // lanes whose B column is not in use read the last used column: what they feed the MMA only
    // reaches accumulator columns nobody reads
    const uint32_t x_lane = tbl_addr + L.x + (min(g, (uint32_t)NCOL - 1u) * xstride + 8u * t) * 4u;


    const uint4* tok = d.tokens + (size_t)t0 * 64u + lane + 2 * 64;
    const uint4* tok_end = d.tokens + (size_t)t1 * 64u;  // lane 0's view of the end of the run
    const uint32_t* trp = d.tile_raw + t0 + 1 + 2;

    uint32_t s_p = t0 % S, rb = t0 / S;  // step and row block of the tile whose words await the MMAs
    bool from_start = s_p == 0;
    uint32_t first_rb = kNoBlock;
    int first_acc[4] = {0, 0, 0, 0};
    int acc[4] = {0, 0, 0, 0}, acc2[4] = {0, 0, 0, 0};  // two chains of MMAs, summed at the end of a row block
    uint32_t wbuf[2][16];

    auto lookups = [&](int k) -> bool {  // tile words -> wbuf[k], then reload q[k] two tiles ahead
      const uint32_t rd_next = tr[k];
      while (rd_next > w_pos) {  // the chunks holding this tile's raw words [rd, rd_next)
        if (!wait_chunk()) return false;
        w_pos += kChunkWords;
      }
      lookup16(q[k], wbuf[k]);
      q[k][0] = ldg_stream(tok);
      q[k][1] = ldg_stream(tok + 32);
      tr[k] = __ldg(trp);
      tok += 64;
      ++trp;
      rd = rd_next;
      return true;
    };
    auto refill = [&](bool prefetch) {
      // every lane has issued its reads of the chunks below rd; the warp barrier orders them before
      // the copies that overwrite those chunks
      __syncwarp();
      const uint32_t lim = min(stop_pos, (rd & ~(uint32_t)(kChunkWords - 1)) + kRingWords);
      for (; i_pos < lim; i_pos += kChunkWords) issue_chunk(d.raw, i_pos);
      // the two token tiles kL2Ahead tiles further on (every other tile): brought into L2 now, so that
      // the register loads two tiles ahead of their use find them there (tok already points two tiles
      // ahead; a prefetch that runs past the run's end stays inside the padding of the token array)
      if (prefetch && lane == 0 && tok + (kL2Ahead - 2) * 64 < tok_end) bulk_prefetch_l2(tok + (kL2Ahead - 2) * 64, 2048u);
    };
    auto consume = [&](const uint32_t (&wc)[16]) {
      uint4 xa, xb;
      const uint32_t xp = x_lane + 128u * s_p;
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(xa.x), "=r"(xa.y), "=r"(xa.z), "=r"(xa.w) : "r"(xp));
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+16];" : "=r"(xb.x), "=r"(xb.y), "=r"(xb.z), "=r"(xb.w) : "r"(xp));
      mma_s8<SIGNED>(acc, wc[0], wc[8], wc[1], wc[9], xa.x, xa.y);
      mma_s8<SIGNED>(acc2, wc[2], wc[10], wc[3], wc[11], xa.z, xa.w);
      mma_s8<SIGNED>(acc, wc[4], wc[12], wc[5], wc[13], xb.x, xb.y);
      mma_s8<SIGNED>(acc2, wc[6], wc[14], wc[7], wc[15], xb.z, xb.w);
      if (++s_p == S) {  // the row block is complete
        s_p = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += acc2[i];
        if (from_start) {
          finalize(d, rb, acc[0], acc[1], acc[2], acc[3]);
        } else {  // the run began inside this row block: keep its sums for the merge
          first_rb = rb;
#pragma unroll
          for (int i = 0; i < 4; ++i) first_acc[i] = acc[i];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = acc2[i] = 0;
        from_start = true;
        ++rb;
        // the row scales of the block that starts now are wanted when it ends: asked for a whole row block ahead
        // (behind the last row block this is the start of the zero points, inside the same image)
        if (lane == 0) asm volatile("prefetch.global.L1 [%0];" ::"l"(d.scale + (size_t)rb * 16u));
      }
    };

    const uint32_t n = t1 - t0;
    bool ok = lookups(0);
    if (ok) refill(true);
    // the first tile has been looked up while other warps were still converting activations; the MMAs need them
    if (ok) {
      const uint32_t xbar = tbl_addr + L.misc + kXReadyBarOffset, par = (x_phase - 1u) & 1u;
      ok = __all_sync(kFull, mbar_try(xbar, par)) || tiles_wait_slow(xbar, par, dead_flag());
    }
    uint32_t i = 1;
    for (; ok && i + 1 < n; i += 2) {
      ok = lookups(1);
      if (!ok) break;
      consume(wbuf[0]);
      refill(false);
      ok = lookups(0);
      if (!ok) break;
      consume(wbuf[1]);
      refill(true);
    }
    if (ok && i < n) {
      ok = lookups(1);
      if (ok) {
        consume(wbuf[0]);
        consume(wbuf[1]);
      }
    } else if (ok) {
      consume(wbuf[0]);
    }
    while (ok && n_waited < n_issued) ok = wait_chunk();  // nothing may still be landing when the ring is reused
    if (!ok) {
      dead = true;
      *dead_flag() = 1u;
      if (lane == 0) atomicOr(d.status, TQ_STATUS_WAIT_EXPIRED);
      return;
    }
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[k] += acc2[k];
    if (!from_start) {
      store_partial(0, rb, acc);  // the whole run lies inside one row block
    } else {
      if (first_rb != kNoBlock) store_partial(0, first_rb, first_acc);
      if (s_p != 0) store_partial(1, rb, acc);  // the run ended inside a row block
    }
  }

  // ---- one segment: row blocks [rb0, rb1) of matrix d, all warps ----------------------------
  __device__ void run_segment(const tq_tiles_desc& d, uint32_t rb0, uint32_t rb1) {
    static_assert(2 * W == 32, "the merge below looks at the 2 W partial-sum slots with one lane each");
    const uint64_t T = (uint64_t)(rb1 - rb0) * d.steps;
    const uint32_t t0 = rb0 * d.steps + (uint32_t)(T * warp / W);
    const uint32_t t1 = rb0 * d.steps + (uint32_t)(T * (warp + 1) / W);
    const bool has_tiles = t0 < t1 && !dead;
    uint32_t h_rd = 0, h_stop = 0, h_w = 0, h_i = 0, h_tr[2];
    uint4 h_q[2][2];
    if (has_tiles) load_head(d, t0, t1, h_rd, h_stop, h_q, h_tr);
    if (!waited) {  // x is the first thing read that a preceding kernel may have written
      asm volatile("griddepcontrol.wait;" ::: "memory");
      waited = true;
    }
    __syncthreads();  // the previous segment is done with x and with the partials in the rings
    prepare_x(d, [&] {
      if (has_tiles) first_chunks(d, h_rd, h_stop, h_w, h_i);
    });
    if (lane < 2) part_ids()[2 * warp + lane] = kNoBlock;
    // no CTA barrier here: a warp tells the x-ready barrier that its share of the digits is written and goes on
    // to its first lookups; it waits for the other warps' shares before its first MMA (run_tiles)
    __syncwarp();
    if (lane == 0) mbar_arrive(tbl_addr + L.misc + kXReadyBarOffset);
    ++x_phase;
    if (has_tiles && !*dead_flag()) run_tiles(d, t0, t1, h_rd, h_stop, h_w, h_i, h_q, h_tr);
    __syncthreads();
    // Partial row blocks: the slots of one block are adjacent (warp order = tile order).  The k-th
    // block that has partial sums is summed and finished by warp k mod W.
    if (!*dead_flag()) {
      const uint32_t id = part_ids()[lane];
      const uint32_t used = __ballot_sync(kFull, id != kNoBlock);
      const uint32_t below = used & ((1u << lane) - 1u);
      const uint32_t prev = __shfl_sync(kFull, id, below ? 31 - __clz(below) : 0);
      uint32_t firsts = __ballot_sync(kFull, id != kNoBlock && (below == 0u || prev != id));
      for (uint32_t k = 0; firsts != 0u; ++k) {
        const uint32_t e0 = __ffs(firsts) - 1u;
        firsts &= firsts - 1u;
        const uint32_t e1 = firsts ? __ffs(firsts) - 1u : 32u;
        if (k % W != warp) continue;
        int sum[4] = {0, 0, 0, 0};
        for (uint32_t c = e0 & ~7u; c < e1; c += 8u) {  // eight loads in flight at a time
          int4 v[8];
#pragma unroll
          for (uint32_t i = 0; i < 8u; ++i) {
            const uint32_t e = c + i;
            const bool on = e >= e0 && e < e1 && ((used >> e) & 1u);
            v[i] = on ? reinterpret_cast<const int4*>(smem + L.ring + (e >> 1) * (kRingWords * 4u) + (e & 1u) * 512u)[lane]
                      : make_int4(0, 0, 0, 0);
          }
#pragma unroll
          for (uint32_t i = 0; i < 8u; ++i) {
            sum[0] += v[i].x;
            sum[1] += v[i].y;
            sum[2] += v[i].z;
            sum[3] += v[i].w;
          }
        }
        finalize(d, __shfl_sync(kFull, id, e0), sum[0], sum[1], sum[2], sum[3]);
      }
    }
  }
};

template <int W, int NB, bool SIGNED>
__global__ void __launch_bounds__(W * 32, 1) gemv_tiles_kernel(const TilesParams p) {
  extern __shared__ __align__(1024) uint8_t tiles_smem_raw[];
  TilesCta<W, NB, SIGNED> cta;
  // launched with programmatic stream serialisation: the next kernel of the stream may start its own
  // set-up while this one runs, and this one has come this far (barriers, table copy under way)
  // while its predecessor was still running.  Nothing above reads or writes what a predecessor
  // produces (the table and the weights are constant); the activations are first read below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // The record of the CTA's first segment (work split and matrix descriptor: constant data) is fetched by
  // warp 1 with one load before the set-up and parked in shared memory, so that its latency overlaps the
  // barrier set-up and the start of the table copy, and no register holds it meanwhile (registers are
  // short in the tile loop).
  const TilesSmem plan = tiles_smem(p.table_words, (uint32_t)kDigits * NB * p.xstride, W);
  SegRecord* first = reinterpret_cast<SegRecord*>(tiles_smem_raw + plan.misc + kFirstSegmentOffset);
  if (p.firsts != nullptr && (threadIdx.x >> 5) == 1u)
    reinterpret_cast<uint32_t*>(first)[threadIdx.x & 31u] =
        __ldg(reinterpret_cast<const uint32_t*>(p.firsts + blockIdx.x) + (threadIdx.x & 31u));
  if (threadIdx.x == 0) mbar_init(smem_u32(tiles_smem_raw) + plan.misc + kXReadyBarOffset, (uint32_t)W);
  cta.setup(tiles_smem_raw, plan, W, p.table, p.table_words, p.test_withhold != 0u);  // fence, ends with a CTA barrier
  cta.xstride = p.xstride;
  // griddepcontrol.wait: in run_segment, behind the loads of constant data that open a segment

  if (p.firsts == nullptr) {
    const uint32_t nrb = p.one.row_blocks;
    const uint32_t rb0 = (uint32_t)((uint64_t)nrb * blockIdx.x / gridDim.x);
    const uint32_t rb1 = (uint32_t)((uint64_t)nrb * (blockIdx.x + 1) / gridDim.x);
    if (rb0 < rb1) cta.run_segment(p.one, rb0, rb1);
    else if (cta.warp == 0) cta.wait_table();  // nothing may still be landing in shared memory when the CTA ends
  } else {
    uint32_t si = first->begin;
    TilesSeg sg = first->seg;
    tq_tiles_desc d = first->desc;
    if (si >= first->end && cta.warp == 0) cta.wait_table();  // a CTA without work: as above
    while (si < first->end) {  // the bound is read again rather than kept across a segment
      // the next record comes near while this segment runs
      if (threadIdx.x == 0 && si + 1 < first->end) asm volatile("prefetch.global.L1 [%0];" ::"l"(p.recs + si + 1));
      cta.run_segment(d, sg.rb_begin, sg.rb_end);
      if (++si < first->end) {
        sg = p.recs[si].seg;
        d = p.recs[si].desc;
      }
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");  // a CTA without work completes after its predecessors too
  cta.linger_after_failure();
}


// ---------------------------------------------------------------------------------------------
// Decompress: one warp per tile, table and raw words read from global memory.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
decompress_tiles_kernel(const tq_tiles_desc d, const uint32_t* __restrict__ table, uint32_t* __restrict__ out) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
  const uint32_t n_tiles = d.steps * d.row_blocks;
  const uint32_t g = lane >> 2, t = lane & 3u;
  const uint32_t gpr = d.cols >> 2;
  uint32_t bad = 0;
  for (uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; tile < n_tiles; tile += warps) {
    const uint32_t rb = tile / d.steps, s = tile % d.steps;
    const uint4 a = ldg_stream(d.tokens + (size_t)tile * 64u + lane);
    const uint4 b = ldg_stream(d.tokens + (size_t)tile * 64u + 32u + lane);
    const uint32_t rd = __ldg(d.tile_raw + tile);
    const uint32_t R[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint32_t tk = (j & 1) ? (R[j >> 1] >> 16) : (R[j >> 1] & 0xFFFFu);
      if (tk >= kMissBase) {
        // the token names the ring slot of its raw word: its position modulo the ring size
        w[j] = __ldg(d.raw + rd + ((tk - rd) & (kRingWords - 1u)));
      } else {
        bad |= tk >= d.table_words;
        w[j] = __ldg(table + tk);
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint32_t r = rb * 16u + g + 8u * h;
      const uint32_t g0 = 32u * s + 8u * t;
      if (r >= d.rows || g0 >= gpr) continue;
      uint32_t* o = out + (size_t)r * gpr + g0;
      if (g0 + 8u <= gpr && ((gpr & 3u) == 0u)) {
        reinterpret_cast<uint4*>(o)[0] = make_uint4(w[8 * h], w[8 * h + 1], w[8 * h + 2], w[8 * h + 3]);
        reinterpret_cast<uint4*>(o)[1] = make_uint4(w[8 * h + 4], w[8 * h + 5], w[8 * h + 6], w[8 * h + 7]);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (g0 + i < gpr) o[i] = w[8 * h + i];
      }
    }
  }
  if (bad) atomicOr(d.status, TQ_STATUS_BAD_CODE);
}


constexpr int kTilesWarps = 16;
constexpr int kDecompWarps = 16;
constexpr uint32_t kSmemLimit = 232448u;  // 227 KB per CTA

// ---------------------------------------------------------------------------------------------
// Decompress for large inputs: the data path of the GEMV kernel (table in shared memory, raw words
// through the ring, two-tile register pipeline, no L2 prefetch) with the MMAs replaced by 32-byte stores.  A lane
// holds, per tile and half, the 8 words of one row = 32 consecutive bytes of the output row; the 4
// lanes of a quad cover 128 consecutive bytes.
// ---------------------------------------------------------------------------------------------
struct DecompParams {
  const tq_tiles_desc* mats;   // stack mode: DEVICE array; nullptr in single-matrix mode
  const TilesSeg* segs;
  const uint32_t* cta_seg;
  uint8_t* const* outs;        // stack mode: DEVICE array of output pointers, one per matrix
  tq_tiles_desc one;           // single-matrix mode
  uint8_t* out_one;
  const uint32_t* table;
  uint32_t table_words;
  uint32_t levels_signed;      // bf16 output: how to read a level byte
};

template <int W, bool BF16>
struct DecompCta : CtaBase {
  uint32_t levels_signed;

  // tiles [t0, t1) of matrix d -> out (rows x cols bytes, row-major; or whole tiles of bf16)
  __device__ void run_tiles(const tq_tiles_desc& d, uint32_t* __restrict__ out, uint32_t t0, uint32_t t1) {
    if (!wait_table()) {  // the table copy started with the kernel; its first use is here
      if (lane == 0) atomicOr(d.status, TQ_STATUS_WAIT_EXPIRED);
      return;
    }
    const uint32_t S = d.steps, gpr = d.cols >> 2;
    const uint32_t g = lane >> 2, t = lane & 3u;
    const bool vec_ok = (gpr & 3u) == 0u;  // every row starts on a 16-byte boundary
    // ... on a 32-byte one (bf16 rows have a pitch of whole tiles)
    const bool wide_ok = (BF16 || (gpr & 7u) == 0u) && (reinterpret_cast<uintptr_t>(out) & 31u) == 0u;
    const uint32_t xor_mask = levels_signed ? 0x80808080u : 0u;          // int8 bit pattern -> biased byte
    const float magic = levels_signed ? 8388736.0f : 8388608.0f;         // 2^23 (+ 128): as_float(0x4B000000 | byte) - magic = level

    uint32_t rd = __ldg(d.tile_raw + t0);
    const uint32_t stop_pos = __ldg(d.tile_raw + t1);
    uint32_t w_pos = rd & ~(uint32_t)(kChunkWords - 1), i_pos = w_pos;
    for (int k = 0; k < kSlots && i_pos < stop_pos; ++k, i_pos += kChunkWords) issue_chunk(d.raw, i_pos);
    const uint4* tok = d.tokens + (size_t)t0 * 64u + lane;
    const uint32_t* trp = d.tile_raw + t0 + 1;
    uint4 q[2][2];
    uint32_t tr[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      q[k][0] = ldg_stream(tok + k * 64);
      q[k][1] = ldg_stream(tok + k * 64 + 32);
      tr[k] = __ldg(trp + k);
    }
    tok += 2 * 64;
    trp += 2;
    uint32_t s = t0 % S, rb = t0 / S;
    bool ok = true;

    auto step = [&](int k) {
      const uint32_t rd_next = tr[k];
      while (ok && rd_next > w_pos) {
        ok = wait_chunk();
        w_pos += kChunkWords;
      }
      if (!ok) return;
      uint32_t w[16];
      lookup16(q[k], w);
      q[k][0] = ldg_stream(tok);
      q[k][1] = ldg_stream(tok + 32);
      tr[k] = __ldg(trp);
      tok += 64;
      ++trp;
      rd = rd_next;
      const uint32_t g0 = 32u * s + 8u * t;
      if (BF16) {
        // level - zero point as bf16 into whole tiles (row pitch S * 128 columns): no bounds to check
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t r = rb * 16u + g + 8u * h;
          const float off = magic + (d.has_zero ? __ldg(d.zero + r) : 0.f);
          uint32_t* o = out + ((size_t)r * (S * 32u) + g0) * 2u;  // 2 words of bf16 per group
#pragma unroll
          for (int i = 0; i < 8; i += 4) {
            uint32_t pk[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t v = w[8 * h + i + e] ^ xor_mask;
              const float f0 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7540)) - off;
              const float f1 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7541)) - off;
              const float f2 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7542)) - off;
              const float f3 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7543)) - off;
              const __nv_bfloat162 lo = __floats2bfloat162_rn(f0, f1), hi = __floats2bfloat162_rn(f2, f3);
              pk[2 * e] = *reinterpret_cast<const uint32_t*>(&lo);
              pk[2 * e + 1] = *reinterpret_cast<const uint32_t*>(&hi);
            }
            if (wide_ok) {  // one whole 32-byte sector per store
              asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(o + 2 * i), "r"(pk[0]), "r"(pk[1]),
                           "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7])
                           : "memory");
            } else {
              asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(o + 2 * i), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3])
                           : "memory");
              asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(o + 2 * i + 4), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]),
                           "r"(pk[7])
                           : "memory");
            }
          }
        }
      }
#pragma unroll
      for (int h = 0; h < 2 && !BF16; ++h) {
        const uint32_t r = rb * 16u + g + 8u * h;
        if (r < d.rows && g0 < gpr) {
          uint32_t* o = out + (size_t)r * gpr + g0;
          if (wide_ok && g0 + 8u <= gpr) {  // one whole 32-byte sector per lane
            asm volatile("st.global.cs.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(o), "r"(w[8 * h]), "r"(w[8 * h + 1]),
                         "r"(w[8 * h + 2]), "r"(w[8 * h + 3]), "r"(w[8 * h + 4]), "r"(w[8 * h + 5]), "r"(w[8 * h + 6]),
                         "r"(w[8 * h + 7])
                         : "memory");
          } else if (vec_ok && g0 + 8u <= gpr) {
            asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(o), "r"(w[8 * h]), "r"(w[8 * h + 1]),
                         "r"(w[8 * h + 2]), "r"(w[8 * h + 3])
                         : "memory");
            asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(o + 4), "r"(w[8 * h + 4]), "r"(w[8 * h + 5]),
                         "r"(w[8 * h + 6]), "r"(w[8 * h + 7])
                         : "memory");
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (g0 + i < gpr) o[i] = w[8 * h + i];
          }
        }
      }
      if (++s == S) {
        s = 0;
        ++rb;
      }
      __syncwarp();
      const uint32_t lim = min(stop_pos, (rd & ~(uint32_t)(kChunkWords - 1)) + kRingWords);
      for (; i_pos < lim; i_pos += kChunkWords) issue_chunk(d.raw, i_pos);
      // no L2 prefetch of the tokens here: with as many bytes written as read it was measured to cost
      // 5 % (prefetched lines are pushed out by the stores before their use)
    };

    for (uint32_t i = t0; i < t1 && ok; i += 2) {
      step(0);
      if (i + 1 < t1 && ok) step(1);
    }
    while (ok && n_waited < n_issued) ok = wait_chunk();
    if (!ok) {
      *dead_flag() = 1u;
      if (lane == 0) atomicOr(d.status, TQ_STATUS_WAIT_EXPIRED);
    }
  }

  __device__ void run_segment(const tq_tiles_desc& d, uint8_t* out, uint32_t rb0, uint32_t rb1) {
    const uint64_t T = (uint64_t)(rb1 - rb0) * d.steps;
    const uint32_t t0 = rb0 * d.steps + (uint32_t)(T * warp / W);
    const uint32_t t1 = rb0 * d.steps + (uint32_t)(T * (warp + 1) / W);
    if (t0 < t1 && !*dead_flag()) run_tiles(d, reinterpret_cast<uint32_t*>(out), t0, t1);
  }
};

template <int W, bool BF16>
__global__ void __launch_bounds__(W * 32, 1) decompress_tiles_smem_kernel(const DecompParams p) {
  extern __shared__ __align__(1024) uint8_t tiles_smem_raw[];
  DecompCta<W, BF16> cta;
  cta.setup(tiles_smem_raw, tiles_smem(p.table_words, 0u, W), W, p.table, p.table_words);
  cta.levels_signed = p.levels_signed;
  if (p.mats == nullptr) {
    const uint32_t nrb = p.one.row_blocks;
    const uint32_t rb0 = (uint32_t)((uint64_t)nrb * blockIdx.x / gridDim.x);
    const uint32_t rb1 = (uint32_t)((uint64_t)nrb * (blockIdx.x + 1) / gridDim.x);
    if (rb0 < rb1) cta.run_segment(p.one, p.out_one, rb0, rb1);
  } else {
    for (uint32_t si = p.cta_seg[blockIdx.x]; si < p.cta_seg[blockIdx.x + 1]; ++si) {
      const TilesSeg sg = p.segs[si];
      const tq_tiles_desc d = p.mats[sg.mat];
      cta.run_segment(d, p.outs[sg.mat], sg.rb_begin, sg.rb_end);
    }
  }
  cta.linger_after_failure();
}

template <bool BF16>
int launch_decomp(const DecompParams& p, uint32_t grid, cudaStream_t st) {
  auto kern = decompress_tiles_smem_kernel<kDecompWarps, BF16>;
  const size_t smem = tiles_smem(p.table_words, 0u, kDecompWarps).total;
  if (int rc = tq_ensure_dynamic_smem((const void*)kern, smem, "decompress(tiles): raising the dynamic shared memory limit")) return rc;
  kern<<<grid, kDecompWarps * 32, smem, st>>>(p);
  return tq_cuda_status((int)cudaGetLastError(), "decompress(tiles) launch");
}

// Launch with programmatic stream serialisation (see gemv_tiles_kernel).
template <class Kern>
int launch_pdl(Kern kern, uint32_t grid, uint32_t threads, size_t smem, cudaStream_t st, const TilesParams& p) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return tq_cuda_status((int)cudaLaunchKernelEx(&cfg, kern, p), "gemv(tiles) launch");
}

std::atomic<int> g_test_withhold{0};

template <int NB, bool SIGNED>
int launch_tiles(TilesParams p, uint32_t grid, size_t smem, cudaStream_t st) {
  p.test_withhold = (uint32_t)g_test_withhold.load();
  auto kern = gemv_tiles_kernel<kTilesWarps, NB, SIGNED>;
  if (int rc = tq_ensure_dynamic_smem((const void*)kern, smem, "gemv(tiles): raising the dynamic shared memory limit")) return rc;
  return launch_pdl(kern, grid, kTilesWarps * 32, smem, st, p);
}

}  // namespace

// Batch columns one launch can take for this matrix (2, 1, or 0 if even one does not fit).
int tq_tiles_max_nb(const tq_dmat* m) {
  const uint32_t xstride = m->tiles.steps * 32u + 4u;
  for (int nb = 2; nb >= 1; --nb)
    if (tiles_smem(m->tiles.table_words, (uint32_t)kDigits * nb * xstride, kTilesWarps).total <= kSmemLimit) return nb;
  return 0;
}

// x: bf16 [B][cols], y: fp32 [B][rows], B in 1..32.  One or two vectors whose digits fit beside the
// table for a whole row take the narrow kernel (tensor-core MACs inside the decoding warps); anything
// else is one pass of the tcgen05 kernel, whose digit planes go through the scratch area of the
// matrix's own image.
int tq_tiles_gemv(const tq_dmat* m, const void* x, int B, float* y, void* cuda_stream) {
  const int narrow = tq_tiles_max_nb(m);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const bool sg = m->info.levels_signed != 0;
  if (B <= narrow) {
    TilesParams p{};
    p.one = m->tiles;
    p.one.x = x;
    p.one.y = y;
    p.table = m->dict->d_table;
    p.table_words = m->tiles.table_words;
    p.xstride = m->tiles.steps * 32u + 4u;
    const uint32_t grid = std::min<uint32_t>(m->tiles.row_blocks, (uint32_t)sm_count());
    const size_t smem = tiles_smem(p.table_words, (uint32_t)kDigits * B * p.xstride, kTilesWarps).total;
    if (B == 1) return sg ? launch_tiles<1, true>(p, grid, smem, st) : launch_tiles<1, false>(p, grid, smem, st);
    return sg ? launch_tiles<2, true>(p, grid, smem, st) : launch_tiles<2, false>(p, grid, smem, st);
  }
  tq_tiles_desc one = m->tiles;
  one.x = x;
  one.y = y;
  // whole row blocks per warp, 16 decoding warps per CTA: as many CTAs as there are groups of 16 row blocks
  const uint32_t grid = std::min<uint32_t>((m->tiles.row_blocks + kWideGroupRowBlocks - 1u) / kWideGroupRowBlocks, (uint32_t)sm_count());
  return tq_wide_launch(nullptr, 1, nullptr, nullptr, &one, m->dict->d_table, m->tiles.table_words, B, sg, grid, cuda_stream);
}

int tq_tiles_decompress(const tq_dmat* m, uint8_t* d_codes, void* cuda_stream) {
  const uint32_t n_tiles = m->tiles.steps * m->tiles.row_blocks;
  // loading the table into every SM's shared memory pays off from a few thousand tiles per SM on
  if ((uint64_t)n_tiles >= 64ull * (uint64_t)sm_count()) {
    DecompParams p{};
    p.one = m->tiles;
    p.out_one = d_codes;
    p.table = m->dict->d_table;
    p.table_words = m->tiles.table_words;
    return launch_decomp<false>(p, std::min<uint32_t>(m->tiles.row_blocks, (uint32_t)sm_count()), (cudaStream_t)cuda_stream);
  }
  const uint32_t grid = std::min<uint32_t>((n_tiles + 7u) / 8u, (uint32_t)sm_count() * 8u);
  decompress_tiles_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(m->tiles, m->dict->d_table,
                                                                       reinterpret_cast<uint32_t*>(d_codes));
  return tq_cuda_status((int)cudaGetLastError(), "decompress(tiles) launch");
}

// The matrix as bf16 (level - zero point) in whole tiles: row_blocks * 16 rows of steps * 128 columns.
int tq_tiles_decode_bf16(const tq_dmat* m, void* d_out, void* cuda_stream) {
  if (!m->zero_bf16_exact) return TQ_ERR_UNSUPPORTED_SHAPE;  // level - zero point would be rounded
  DecompParams p{};
  p.one = m->tiles;
  p.out_one = static_cast<uint8_t*>(d_out);
  p.table = m->dict->d_table;
  p.table_words = m->tiles.table_words;
  p.levels_signed = m->info.levels_signed != 0;
  return launch_decomp<true>(p, std::min<uint32_t>(m->tiles.row_blocks, (uint32_t)sm_count()), (cudaStream_t)cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Stack: many matrices, one persistent launch.
// ---------------------------------------------------------------------------------------------
namespace {
// Charge for a segment start (activations converted again, pipelines refilled, a CTA barrier or two), in
// bytes of stream.  Measured on the 3B and 1B stacks from 16 KB to 1.5 MB: the step time falls up to 384 KB
// (3B 0.536 -> 0.526 ms, 1B 0.237 -> 0.229 ms against 96 KB) and rises again beyond 768 KB.
constexpr uint64_t kSegmentOverheadBytes = 384 * 1024;

struct StackPlan {
  std::vector<TilesSeg> segs;
  std::vector<uint32_t> cta_seg;
};

// Row blocks in matrix order, cut into `grid` consecutive shares of equal cost (bytes streamed plus
// a fixed charge per segment start).
struct PlanMat {
  uint32_t steps, row_blocks;
  const uint32_t* rb_raw;  // row_blocks + 1: index of each row block's first raw word
};

// mats[0..n): the matrices to split; ids[i] is the index recorded in the segments for mats[i].
StackPlan plan_stack(const PlanMat* mats, const uint32_t* ids, int n, uint32_t grid) {
  auto rb_cost = [&](const PlanMat& m, uint32_t rb) -> uint64_t {
    return (uint64_t)m.steps * 1024 + (uint64_t)(m.rb_raw[rb + 1] - m.rb_raw[rb]) * 4;
  };
  uint64_t total = 0;
  for (int i = 0; i < n; ++i)
    total += (uint64_t)mats[i].steps * 1024 * mats[i].row_blocks + (uint64_t)mats[i].rb_raw[mats[i].row_blocks] * 4;
  total += kSegmentOverheadBytes * ((uint64_t)n + grid);
  const uint64_t share = total / grid + 1;
  StackPlan pl;
  pl.cta_seg.push_back(0);
  uint64_t acc = 0;  // cost given to the current CTA
  for (int i = 0; i < n; ++i) {
    const PlanMat& m = mats[i];
    uint32_t rb = 0;
    while (rb < m.row_blocks) {
      if (acc + kSegmentOverheadBytes >= share && pl.cta_seg.size() < grid) {  // no room for a useful segment
        pl.cta_seg.push_back((uint32_t)pl.segs.size());
        acc = 0;
      }
      acc += kSegmentOverheadBytes;
      const uint32_t begin = rb;
      const bool last_cta = pl.cta_seg.size() >= grid;
      while (rb < m.row_blocks && (last_cta || acc < share)) acc += rb_cost(m, rb++);
      pl.segs.push_back(TilesSeg{ids[i], begin, rb});
      if (acc >= share && !last_cta) {
        pl.cta_seg.push_back((uint32_t)pl.segs.size());
        acc = 0;
      }
    }
  }
  while (pl.cta_seg.size() < (size_t)grid + 1) pl.cta_seg.push_back((uint32_t)pl.segs.size());
  return pl;
}

// Work split for the tcgen05 kernel.  Its 16 decoding warps walk whole row blocks in step, so the unit
// of work is a group of consecutive row blocks of one matrix: 16 of them (256 rows), or fewer when
// there is not enough work to give every CTA such a group (then fewer warps of more CTAs are busy).
// Groups go to the CTAs longest first, each to the CTA with the least work so far; a CTA's groups
// are then put in matrix order and neighbours merged into one segment.
StackPlan plan_wide(const PlanMat* mats, const uint32_t* ids, int n, uint32_t grid) {
  uint64_t total_rb = 0;
  for (int i = 0; i < n; ++i) total_rb += mats[i].row_blocks;
  const uint32_t G = kWideGroupRowBlocks;
  uint32_t gsz = G;
  if (total_rb < (uint64_t)G * grid) gsz = (uint32_t)std::max<uint64_t>(1, (total_rb + grid - 1) / grid);
  struct Unit {
    uint64_t cost;
    uint32_t mat, rb0, rb1;  // mat: index into mats
  };
  std::vector<Unit> units;
  for (int i = 0; i < n; ++i) {
    const PlanMat& m = mats[i];
    for (uint32_t rb = 0; rb < m.row_blocks; rb += gsz) {
      const uint32_t end = std::min(m.row_blocks, rb + gsz);
      // every warp is busy for as long as the longest row block of the group takes
      uint64_t longest = 0;
      for (uint32_t r = rb; r < end; ++r) longest = std::max<uint64_t>(longest, (uint64_t)m.steps * 1024 + (uint64_t)(m.rb_raw[r + 1] - m.rb_raw[r]) * 4);
      units.push_back(Unit{longest * G + 8192, (uint32_t)i, rb, end});
    }
  }
  std::vector<uint32_t> order(units.size());
  for (uint32_t u = 0; u < order.size(); ++u) order[u] = u;
  std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return units[a].cost > units[b].cost; });
  std::vector<uint64_t> load(grid, 0);
  std::vector<std::vector<uint32_t>> mine(grid);
  // least-loaded CTA by a heap of (load, cta)
  std::vector<std::pair<uint64_t, uint32_t>> heap;
  for (uint32_t c = 0; c < grid; ++c) heap.emplace_back(0ull, c);
  auto cmp = [](const std::pair<uint64_t, uint32_t>& a, const std::pair<uint64_t, uint32_t>& b) { return a > b; };
  std::make_heap(heap.begin(), heap.end(), cmp);
  for (uint32_t u : order) {
    std::pop_heap(heap.begin(), heap.end(), cmp);
    auto& top = heap.back();
    top.first += units[u].cost;
    mine[top.second].push_back(u);
    std::push_heap(heap.begin(), heap.end(), cmp);
  }
  StackPlan pl;
  pl.cta_seg.push_back(0);
  for (uint32_t c = 0; c < grid; ++c) {
    std::sort(mine[c].begin(), mine[c].end());  // units were made in (matrix, row block) order
    for (size_t k = 0; k < mine[c].size(); ++k) {
      const Unit& u = units[mine[c][k]];
      const bool full = u.rb1 - u.rb0 == G;
      if (!pl.segs.empty() && pl.cta_seg.back() < pl.segs.size() && full && pl.segs.back().mat == ids[u.mat] &&
          pl.segs.back().rb_end == u.rb0 && (pl.segs.back().rb_end - pl.segs.back().rb_begin) % G == 0)
        pl.segs.back().rb_end = u.rb1;  // whole groups merge: the warps keep 1, 2, ... row blocks each
      else
        pl.segs.push_back(TilesSeg{ids[u.mat], u.rb0, u.rb1});
    }
    pl.cta_seg.push_back((uint32_t)pl.segs.size());
  }
  return pl;
}

inline uint64_t align256(uint64_t v) { return (v + 255) / 256 * 256; }
}  // namespace

extern "C" {

void tq_test_withhold_table_chunk(int on) { g_test_withhold.store(on ? 1 : 0); }

int tq_stack_plan_host(int n_mats, const uint32_t* steps, const uint32_t* row_blocks, const uint32_t* const* rb_raw,
                       uint32_t n_ctas, uint32_t* segs, uint32_t segs_cap, uint32_t* n_segs, uint32_t* cta_seg) {
  if (n_mats < 1 || !steps || !row_blocks || !rb_raw || n_ctas < 1 || !segs || !n_segs || !cta_seg) return TQ_ERR_INVALID_ARG;
  std::vector<PlanMat> pm((size_t)n_mats);
  for (int i = 0; i < n_mats; ++i) {
    if (!rb_raw[i] || steps[i] == 0 || row_blocks[i] == 0) return TQ_ERR_INVALID_ARG;
    pm[i] = PlanMat{steps[i], row_blocks[i], rb_raw[i]};
  }
  std::vector<uint32_t> ids((size_t)n_mats);
  for (int i = 0; i < n_mats; ++i) ids[i] = (uint32_t)i;
  const StackPlan pl = plan_stack(pm.data(), ids.data(), n_mats, n_ctas);
  *n_segs = (uint32_t)pl.segs.size();
  if (pl.segs.size() > segs_cap) return TQ_ERR_BUFFER_TOO_SMALL;
  for (size_t i = 0; i < pl.segs.size(); ++i) {
    segs[3 * i] = pl.segs[i].mat;
    segs[3 * i + 1] = pl.segs[i].rb_begin;
    segs[3 * i + 2] = pl.segs[i].rb_end;
  }
  for (uint32_t c = 0; c <= n_ctas; ++c) cta_seg[c] = pl.cta_seg[c];
  return TQ_OK;
}

namespace {
constexpr int kStackPlans = 4;
// Does a row of this matrix fit the narrow kernel (digits of one whole row beside the table)?
bool short_rows(const tq_dmat* m, int nb) {
  return tiles_smem(m->tiles.table_words, (uint32_t)kDigits * nb * (m->tiles.steps * 32u + 4u), kTilesWarps).total <= kSmemLimit;
}
// Which kernels a stack of B vectors runs: B = 1 (and B = 2 where two vectors' digits fit for every
// short-row matrix) takes the narrow kernel for the matrices with short rows and the tcgen05 kernel
// for the others; any other B is one pass of the tcgen05 kernel over all matrices.
struct StackRoute {
  bool narrow;       // plan[1] through the narrow kernel with B vectors
  bool wide_long;    // plan[2] through the tcgen05 kernel
  bool wide_all;     // plan[3] through the tcgen05 kernel
};
StackRoute stack_route(const tq_dmat* const* mats, int n_mats, int B) {
  bool any_short = false, any_long = false, fits_b = B <= 2;
  for (int i = 0; i < n_mats; ++i) {
    const bool sh = short_rows(mats[i], 1);
    any_short |= sh;
    any_long |= !sh;
    if (sh && B == 2 && !short_rows(mats[i], 2)) fits_b = false;
  }
  StackRoute r{};
  if (B >= 1 && fits_b && any_short) {
    r.narrow = true;
    r.wide_long = any_long;
  } else if (B >= 1) {
    r.wide_all = true;
  }
  return r;
}
// Records of the narrow kernel's split: at most n_mats + grid segments (every matrix starts one, every CTA
// boundary splits at most one), and one record per CTA.
uint64_t stack_record_bytes(int n_mats, uint64_t grid) { return align256(((uint64_t)n_mats + 2 * grid) * sizeof(SegRecord)); }
uint64_t stack_plan_bytes(int n_mats, uint64_t grid, uint64_t total_rb) {
  // the tcgen05 plan can hold one segment per group of row blocks (or per CTA for small stacks)
  const uint64_t max_segs = std::max<uint64_t>((uint64_t)n_mats + grid, total_rb / kWideGroupRowBlocks + (uint64_t)n_mats + grid);
  return align256(max_segs * sizeof(TilesSeg)) + align256((grid + 1) * 4);
}
}  // namespace

int tq_stack_size(const tq_dmat* const* mats, int n_mats, int B, uint64_t* device_bytes) {
  if (!mats || n_mats < 1 || B < 0 || B > 32 || !device_bytes) return TQ_ERR_INVALID_ARG;
  const uint64_t grid = (uint64_t)sm_count();
  uint64_t total_rb = 0, scratch = 0;
  for (int i = 0; i < n_mats; ++i) {
    if (!mats[i]) return TQ_ERR_INVALID_ARG;
    if (mats[i]->info.layout != TQ_LAYOUT_TILES) return TQ_ERR_UNSUPPORTED_SHAPE;
    total_rb += mats[i]->tiles.row_blocks;
  }
  const StackRoute r = stack_route(mats, n_mats, B);
  for (int i = 0; i < n_mats; ++i)
    if (r.wide_all || (r.wide_long && !short_rows(mats[i], 1))) scratch += tq_wide_scratch_bytes(mats[i]->tiles.steps, B);
  *device_bytes = align256((uint64_t)n_mats * sizeof(tq_tiles_desc)) + kStackPlans * stack_plan_bytes(n_mats, grid, total_rb) +
                  stack_record_bytes(n_mats, grid) + 1024 + scratch;
  return TQ_OK;
}

int tq_stack_create(const tq_dmat* const* mats, const void* const* d_x, float* const* d_y, int n_mats, int B,
                    void* d_buf, uint64_t d_buf_bytes, void* cuda_stream, tq_stack** out) {
  const bool bound = d_x && d_y;  // without operands the stack serves tq_decompress_stack only
  if (!mats || (!bound && (d_x || d_y)) || n_mats < 1 || (bound && (B < 1 || B > 32)) || !d_buf || !out ||
      ((uintptr_t)d_buf & 255))
    return TQ_ERR_INVALID_ARG;
  if (!bound) B = 0;
  uint64_t need = 0;
  if (int rc = tq_stack_size(mats, n_mats, B, &need)) return rc;
  if (d_buf_bytes < need) return TQ_ERR_BUFFER_TOO_SMALL;
  for (int i = 0; i < n_mats; ++i) {
    const tq_dmat* m = mats[i];
    if (!m || (bound && (!d_x[i] || !d_y[i] || ((uintptr_t)d_x[i] & 15)))) return TQ_ERR_INVALID_ARG;
    if (m->info.layout != TQ_LAYOUT_TILES || m->dict != mats[0]->dict ||
        m->info.levels_signed != mats[0]->info.levels_signed)
      return TQ_ERR_UNSUPPORTED_SHAPE;  // one table, one kind of level, TILES layout
  }
  tq_stack* s = new (std::nothrow) tq_stack();
  if (!s) return TQ_ERR_NOMEM;
  s->n = n_mats;
  s->B = B;
  s->levels_signed = mats[0]->info.levels_signed;
  for (int i = 0; i < n_mats; ++i) s->zero_bf16_exact = s->zero_bf16_exact && mats[i]->zero_bf16_exact;
  s->grid = (uint32_t)sm_count();
  s->table_words = mats[0]->tiles.table_words;
  s->d_table = mats[0]->dict->d_table;
  const StackRoute route = stack_route(mats, n_mats, B);
  s->run_narrow = route.narrow;
  s->run_wide_long = route.wide_long;
  s->run_wide_all = route.wide_all;

  uint64_t total_rb = 0;
  for (int i = 0; i < n_mats; ++i) total_rb += mats[i]->tiles.row_blocks;
  uint8_t* base = static_cast<uint8_t*>(d_buf);
  const uint64_t plan_bytes = stack_plan_bytes(n_mats, s->grid, total_rb);
  const uint64_t segs_bytes = plan_bytes - align256((s->grid + 1) * 4);
  const uint64_t off_plans = align256((uint64_t)n_mats * sizeof(tq_tiles_desc));
  const uint64_t off_records = off_plans + kStackPlans * plan_bytes;
  uint64_t off_scratch = (off_records + stack_record_bytes(n_mats, s->grid) + 1023) / 1024 * 1024;

  std::vector<tq_tiles_desc> descs((size_t)n_mats);
  for (int i = 0; i < n_mats; ++i) {
    descs[i] = mats[i]->tiles;
    descs[i].x = bound ? d_x[i] : nullptr;
    descs[i].y = bound ? d_y[i] : nullptr;
    descs[i].xdig = nullptr;
    if (route.wide_all || (route.wide_long && !short_rows(mats[i], 1))) {  // digit planes of this matrix's vectors
      descs[i].xdig = base + off_scratch;
      off_scratch += tq_wide_scratch_bytes(mats[i]->tiles.steps, B);
    }
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int rc = tq_cuda_status((int)cudaMemcpyAsync(base, descs.data(), descs.size() * sizeof(tq_tiles_desc), cudaMemcpyHostToDevice, st), "stack upload");
  // [0] all matrices, split by tiles (decompress, bf16 decode); [1] the matrices whose rows are short enough
  // for the narrow kernel; [2] the others and [3] all matrices, split for the tcgen05 kernel
  StackPlan pls[kStackPlans];  // kept alive until the copies have been made
  std::vector<SegRecord> records;
  for (int k = 0; k < kStackPlans && rc == TQ_OK; ++k) {
    std::vector<PlanMat> pm;
    std::vector<uint32_t> ids;
    uint32_t max_steps = 0;
    for (int i = 0; i < n_mats; ++i) {
      const bool sh = short_rows(mats[i], 1);
      if (k == 0 || k == 3 || (k == 1) == sh) {
        pm.push_back(PlanMat{mats[i]->tiles.steps, mats[i]->tiles.row_blocks, mats[i]->rb_raw.data()});
        ids.push_back((uint32_t)i);
        max_steps = std::max(max_steps, mats[i]->tiles.steps);
      }
    }
    tq_stack_plan& sp = s->plan[k];
    sp.n_mats = (uint32_t)pm.size();
    sp.xstride = max_steps * 32u + 4u;
    if (pm.empty()) continue;
    if (k == 1 && !route.narrow) continue;
    if (k == 2 && !route.wide_long) continue;
    if (k == 3 && !route.wide_all) continue;
    pls[k] = k >= 2 ? plan_wide(pm.data(), ids.data(), (int)pm.size(), s->grid) : plan_stack(pm.data(), ids.data(), (int)pm.size(), s->grid);
    if (pls[k].segs.size() * sizeof(TilesSeg) > segs_bytes) rc = TQ_ERR_BUFFER_TOO_SMALL;
    uint8_t* pb = base + off_plans + (uint64_t)k * plan_bytes;
    if (rc == TQ_OK)
      rc = tq_cuda_status((int)cudaMemcpyAsync(pb, pls[k].segs.data(), pls[k].segs.size() * sizeof(TilesSeg), cudaMemcpyHostToDevice, st), "stack upload");
    if (rc == TQ_OK)
      rc = tq_cuda_status((int)cudaMemcpyAsync(pb + segs_bytes, pls[k].cta_seg.data(), pls[k].cta_seg.size() * 4, cudaMemcpyHostToDevice, st), "stack upload");
    sp.d_segs = pb;
    sp.d_cta_seg = reinterpret_cast<const uint32_t*>(pb + segs_bytes);
    sp.n_segs = (uint32_t)pls[k].segs.size();
    if (k == 1 && rc == TQ_OK) {  // the narrow kernel's records: per segment, then per CTA
      const StackPlan& pl = pls[k];
      const size_t n_segs = pl.segs.size();
      if ((n_segs + s->grid) * sizeof(SegRecord) > stack_record_bytes(n_mats, s->grid)) rc = TQ_ERR_BUFFER_TOO_SMALL;
      records.assign(n_segs + s->grid, SegRecord{});
      for (uint32_t c = 0; c < s->grid && rc == TQ_OK; ++c) {
        const uint32_t b = pl.cta_seg[c], e = pl.cta_seg[c + 1];
        for (uint32_t i = b; i < e; ++i) {
          records[i].begin = b;
          records[i].end = e;
          records[i].seg = pl.segs[i];
          records[i].desc = descs[pl.segs[i].mat];
        }
        if (b < e) {
          records[n_segs + c] = records[b];
          sp.grid_used = c + 1;
        }
      }
      if (rc == TQ_OK)
        rc = tq_cuda_status((int)cudaMemcpyAsync(base + off_records, records.data(), records.size() * sizeof(SegRecord), cudaMemcpyHostToDevice, st), "stack upload");
      sp.d_recs = base + off_records;
      sp.d_firsts = base + off_records + n_segs * sizeof(SegRecord);
    }
  }
  if (rc == TQ_OK) rc = tq_cuda_status((int)cudaStreamSynchronize(st), "stack upload");
  if (rc != TQ_OK) {
    delete s;
    return rc;
  }
  s->d_descs = reinterpret_cast<const tq_tiles_desc*>(base);
  *out = s;
  return TQ_OK;
}

namespace {
// The launches of one tq_fused_gemv_stack call.  launch == false only counts them.
int stack_run(const tq_stack* s, bool launch, cudaStream_t st, int* n_launches) {
  const bool sg = s->levels_signed != 0;
  if (s->run_narrow) {
    const tq_stack_plan& sp = s->plan[1];
    ++*n_launches;
    if (launch) {
      TilesParams p{};
      p.firsts = static_cast<const SegRecord*>(sp.d_firsts);
      p.recs = static_cast<const SegRecord*>(sp.d_recs);
      p.table = s->d_table;
      p.table_words = s->table_words;
      p.xstride = sp.xstride;
      const size_t smem = tiles_smem(p.table_words, (uint32_t)kDigits * s->B * p.xstride, kTilesWarps).total;
      const uint32_t grid = sp.grid_used;  // the split fills the CTAs in order: the rest would only copy the table
      int rc;
      if (s->B == 1) rc = sg ? launch_tiles<1, true>(p, grid, smem, st) : launch_tiles<1, false>(p, grid, smem, st);
      else rc = sg ? launch_tiles<2, true>(p, grid, smem, st) : launch_tiles<2, false>(p, grid, smem, st);
      if (rc != TQ_OK) return rc;
    }
  }
  if (s->run_wide_long || s->run_wide_all) {
    const tq_stack_plan& sp = s->plan[s->run_wide_all ? 3 : 2];
    *n_launches += 2;  // digit planes, then the fused kernel
    if (launch)
      return tq_wide_launch(s->d_descs, s->n, sp.d_segs, sp.d_cta_seg, nullptr, s->d_table, s->table_words, s->B, sg, s->grid, st);
  }
  return TQ_OK;
}
}  // namespace

int tq_fused_gemv_stack(const tq_stack* s, void* cuda_stream) {
  if (!s || s->B < 1) return TQ_ERR_INVALID_ARG;
  int n = 0;
  return stack_run(s, true, (cudaStream_t)cuda_stream, &n);
}

int tq_fused_gemv_stack_host(const tq_stack* s, const void* h_x, void* d_x_arena, uint64_t x_bytes, float* h_y,
                             const float* d_y_arena, uint64_t y_bytes, void* cuda_stream) {
  if (!s || !h_x || !d_x_arena || !h_y || !d_y_arena) return TQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (int rc = tq_cuda_status((int)cudaMemcpyAsync(d_x_arena, h_x, x_bytes, cudaMemcpyHostToDevice, st), "stack: copy of x"))
    return rc;
  if (int rc = tq_fused_gemv_stack(s, cuda_stream)) return rc;
  return tq_cuda_status((int)cudaMemcpyAsync(h_y, d_y_arena, y_bytes, cudaMemcpyDeviceToHost, st), "stack: copy of y");
}

int tq_decompress_stack(const tq_stack* s, uint8_t* const* d_out_ptrs, void* cuda_stream) {
  if (!s || !d_out_ptrs) return TQ_ERR_INVALID_ARG;
  DecompParams p{};
  p.mats = s->d_descs;
  p.segs = static_cast<const TilesSeg*>(s->plan[0].d_segs);
  p.cta_seg = s->plan[0].d_cta_seg;
  p.outs = d_out_ptrs;
  p.table = s->d_table;
  p.table_words = s->table_words;
  return launch_decomp<false>(p, s->grid, (cudaStream_t)cuda_stream);
}

int tq_decode_bf16_stack(const tq_stack* s, void* const* d_workspace_ptrs, void* cuda_stream) {
  if (!s || !d_workspace_ptrs) return TQ_ERR_INVALID_ARG;
  if (!s->zero_bf16_exact) return TQ_ERR_UNSUPPORTED_SHAPE;  // level - zero point would be rounded
  DecompParams p{};
  p.mats = s->d_descs;
  p.segs = static_cast<const TilesSeg*>(s->plan[0].d_segs);
  p.cta_seg = s->plan[0].d_cta_seg;
  p.outs = reinterpret_cast<uint8_t* const*>(d_workspace_ptrs);
  p.table = s->d_table;
  p.table_words = s->table_words;
  p.levels_signed = s->levels_signed != 0;
  return launch_decomp<true>(p, s->grid, (cudaStream_t)cuda_stream);
}

int tq_stack_launches(const tq_stack* s) {
  if (!s) return TQ_ERR_INVALID_ARG;
  int n = 0;
  stack_run(s, false, nullptr, &n);
  return n;
}

void tq_stack_free(tq_stack* s) { delete s; }

}  // extern "C"
