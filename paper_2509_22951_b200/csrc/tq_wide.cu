// Fused decode + product for 3..32 activation vectors (TILES layout, sm_100a): the decoding warps
// of the narrow kernel, with the multiply-accumulates handed to the 5th-generation tensor core.
//
// One persistent CTA per SM.  16 decoding warps each walk whole row blocks (16 rows) of the CTA's
// share, all in step: in step k every warp decodes the tile of its row block that covers columns
// 128k .. 128k+127 (tokens through registers two tiles ahead, raw words through the warp's ring,
// 16 shared-memory lookups per lane -- the data path of gemv_tiles_kernel).  A decoded 32-bit word
// holds four 8-bit levels of one row, and the 16 words a lane ends up with are, as they stand, its
// share of a 16-row x 128-byte slice of an 8-bit A operand in tensor memory: one tcgen05.st
// (16x256b.x4) per tile puts them there, the warp's position in tensor memory fixed by its index
// (lanes 32 (w & 3) + 16 ((w >> 2) & 1) .. +15 of operand half w >> 3).  Two operand halves of 128
// rows make the CTA's step 256 rows x 128 columns.
//
// The activations are the B operand.  A first, small kernel turns every vector into the four
// signed base-256 digit planes of its 30-bit block-fixed-point form (tq_tiles_common.cuh) and
// writes them to scratch memory in the exact byte order of the shared-memory operand (K-major,
// 128-byte swizzle, one slice of N x 128 bytes per step, N = 4 x vectors rounded up to 16), so the
// main kernel's loader warp brings a step's slice in with plain bulk copies.  One thread issues,
// per step and operand half, four tcgen05.mma.kind::i8 (M 128, N, K 32) that accumulate exact
// 32-bit integer sums in tensor memory; tcgen05.commit hands stages back through mbarriers.  After
// the last step of a row block every decoding warp reads its own 16 rows of the accumulators back
// (tcgen05.ld 16x256b), combines the four digit sums of each vector and writes y.  The arithmetic
// is that of the narrow kernel, so the results are bit-identical to it.
//
// Every wait is bounded; a wait that runs out raises TQ_STATUS_WAIT_EXPIRED, all roles leave their
// loops, and tensor memory is released on every path.
#include <algorithm>
#include <cstdio>
#include <vector>

// the slow path of a wait inlined: a call there makes the compiler spill around every wait of the roles below
#define TQ_WAIT_SLOW_INLINING __forceinline__
#include "tq_tiles_common.cuh"

namespace {

constexpr int kDecodeWarps = 16;
constexpr int kLoaderWarp = 16, kMmaWarp = 17;
constexpr int kWideThreads = (kDecodeWarps + 2) * 32;  // + loader warp + MMA warp
constexpr uint32_t kTmemCols = 512;    // all of it: 2 x N accumulator columns, then 2 x a_stages x 32 operand columns
constexpr uint32_t kStepCols = 32;     // 128 bytes of a row = 32 columns of tensor memory
constexpr uint32_t kMaxAStages = 8;    // A-operand stages in tensor memory: as many as fit, at most this
constexpr uint32_t kSmemLimit = 232448u;
constexpr uint32_t kHdrBytes = 512u;   // scratch header: out_scale[32], sum_x[32] (doubles)
static_assert((TQ_TILES_TABLE_WORDS * 4u) % 1024u == 0, "the B-operand stages behind the table and the rings must be 1024-byte aligned");

// misc area of the shared-memory plan: [0] dead flag, [8] tensor-memory base, barriers from 16 on
constexpr uint32_t kOffTmem = 8, kOffAFull = 16, kOffAEmpty = 80, kOffBFull = 144, kOffBEmpty = 176, kOffAccFull = 208,
                   kOffAccFree = 216;

struct WideParams {
  const tq_tiles_desc* mats;  // stack mode: DEVICE array; nullptr in single-matrix mode
  const TilesSeg* segs;       // stack mode: segments, grouped by CTA
  const uint32_t* cta_seg;    // stack mode: gridDim.x + 1 offsets into segs
  tq_tiles_desc one;          // single-matrix mode
  const uint32_t* table;
  uint32_t table_words;
  uint32_t nb;                // vectors, 1..32
  uint32_t n_cols;            // N: digit rows of the B operand, 4 * nb rounded up to a multiple of 16
  uint32_t b_stages;          // B-operand stages in shared memory (2..4)
  uint32_t a_stages;          // A-operand stages in tensor memory (4..8): (512 - 2 N) / 64, at most kMaxAStages
};

// Row of the B operand (= accumulator column) that holds digit k of vector b: the two digits a
// thread reads back from one 8-column group of the accumulator are digits 2i, 2i+1 of one vector.
__host__ __device__ inline uint32_t digit_row(uint32_t b, uint32_t k) {
  return 8u * (2u * (b >> 2) + (k >> 1)) + 2u * (b & 3u) + (k & 1u);
}

// ---------------------------------------------------------------------------------------------
// Activations -> digit planes in operand order.  grid = (vectors, matrices), 256 threads.
// Group gi of a row (4 columns) belongs to step gi / 32; inside the step, group 8t + 2i + c
// (t = 0..3, i = 0..3, c = 0..1) is the word a decoding lane (g, t) stores to column 8i + 2t + c
// of its tensor-memory rows, so its digits go to byte 4 (8i + 2t + c) of the 128-byte operand row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) wide_prepare_kernel(const tq_tiles_desc* __restrict__ mats, const tq_tiles_desc one,
                                                           uint32_t n_cols) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ uint32_t s_amax;
  __shared__ unsigned long long s_sum;
  const tq_tiles_desc d = mats ? mats[blockIdx.y] : one;
  if (d.xdig == nullptr) return;  // a matrix of the stack that another kernel serves
  const uint32_t b = blockIdx.x, tid = threadIdx.x, lane = tid & 31u;
  const uint32_t G = d.cols >> 2;
  const uint2* xg = reinterpret_cast<const uint2*>(d.x) + (size_t)b * G;
  if (tid == 0) {
    s_amax = 0u;
    s_sum = 0ull;
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");  // x may come from the kernel before this one
  __syncthreads();
  uint32_t m = 0;
  for (uint32_t g = tid; g < G; g += 256u) m = amax4(__ldg(xg + g), m);
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) m = max(m, __shfl_xor_sync(kFull, m, s));
  if (lane == 0) atomicMax(&s_amax, m);
  __syncthreads();
  const FixScale f = fix_scale(s_amax);
  const float s1 = f.finite ? f.s1 : 0.f;  // a non-finite vector: all digits zero, NaN output scale
  uint8_t* stage0 = d.xdig + kHdrBytes;
  uint32_t row[kDigits];
#pragma unroll
  for (int k = 0; k < kDigits; ++k) row[k] = digit_row(b, (uint32_t)k);
  long long sum = 0;
  for (uint32_t gi = tid; gi < G; gi += 256u) {
    uint32_t w[kDigits];
    fix_digits(__ldg(xg + gi), s1, f.s2, w, &sum);
    const uint32_t step = gi >> 5, gg = gi & 31u;
    const uint32_t t = gg >> 3, j = gg & 7u;
    const uint32_t col = 8u * (j >> 1) + 2u * t + (j & 1u);  // word of the 128-byte operand row
    uint8_t* st = stage0 + (size_t)step * n_cols * 128u;
#pragma unroll
    for (int k = 0; k < kDigits; ++k) {
      const uint32_t n = row[k];
      *reinterpret_cast<uint32_t*>(st + n * 128u + ((((col >> 2) ^ (n & 7u)) << 4) | ((col & 3u) << 2))) = w[k];
    }
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) sum += __shfl_xor_sync(kFull, sum, s);
  if (lane == 0) atomicAdd(&s_sum, (unsigned long long)sum);
  __syncthreads();
  if (tid == 0) {
    double* hdr = reinterpret_cast<double*>(d.xdig);
    const double os = fix_out_scale(f);
    hdr[b] = os;
    hdr[32 + b] = os * (double)(long long)s_sum;
  }
}

// ---------------------------------------------------------------------------------------------
// The main kernel.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_arrive_one(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <bool SIGNED>
__device__ __forceinline__ constexpr uint32_t i8_idesc(uint32_t n) {
  // s32 accumulators (2 << 4); A: 8-bit levels, signed or unsigned (bit 7); B: signed digits (1 << 10);
  // both K-major; N >> 3 at bit 17; M >> 4 at bit 24
  return (2u << 4) | ((SIGNED ? 1u : 0u) << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ void umma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The CTA's segments in order: (matrix, first row block, one past the last).  Fields of a matrix are
// read where they are needed (FIELD below), not copied as a whole: the loader and MMA warps run on a
// small register budget.
struct SegWalk {
  uint32_t si, se;
  bool single_pending;
  __device__ explicit SegWalk(const WideParams& p) : si(0), se(0), single_pending(p.mats == nullptr) {
    if (p.mats != nullptr) {
      si = p.cta_seg[blockIdx.x];
      se = p.cta_seg[blockIdx.x + 1];
    }
  }
  __device__ __forceinline__ bool next(const WideParams& p, uint32_t& mat, uint32_t& rb0, uint32_t& rb1) {
    if (p.mats == nullptr) {
      if (!single_pending) return false;
      single_pending = false;
      mat = 0;
      const uint32_t nrb = p.one.row_blocks;
      rb0 = (uint32_t)((uint64_t)nrb * blockIdx.x / gridDim.x);
      rb1 = (uint32_t)((uint64_t)nrb * (blockIdx.x + 1) / gridDim.x);
      return rb0 < rb1;
    }
    if (si >= se) return false;
    const TilesSeg sg = p.segs[si++];
    mat = sg.mat;
    rb0 = sg.rb_begin;
    rb1 = sg.rb_end;
    return true;
  }
};
#define FIELD(name) (p.mats ? p.mats[mat].name : p.one.name)

struct WideCta : CtaBase {
  uint32_t misc_addr;
  uint32_t tmem_base;

  __device__ __forceinline__ uint32_t bar(uint32_t off, uint32_t idx = 0) const { return misc_addr + off + idx * 8u; }
  // One answer per warp; all 32 lanes call.
  __device__ __forceinline__ bool wait(uint32_t b, uint32_t parity) {
    if (__all_sync(kFull, mbar_try(b, parity))) return true;
    return tiles_wait_slow(b, parity, dead_flag());
  }
};

template <bool SIGNED>
__global__ void __launch_bounds__(kWideThreads, 1) gemv_wide_kernel(const WideParams p) {
  extern __shared__ __align__(1024) uint8_t tiles_smem_raw[];
  WideCta cta;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const TilesSmem plan = tiles_smem(p.table_words, p.b_stages * p.n_cols * 32u, kDecodeWarps);
  const uint32_t smem0 = smem_u32(tiles_smem_raw);
  cta.misc_addr = smem0 + plan.misc;
  if (threadIdx.x == 64) {
    for (uint32_t i = 0; i < kMaxAStages; ++i) {
      mbar_init(cta.bar(kOffAFull, i), kDecodeWarps);
      mbar_init(cta.bar(kOffAEmpty, i), 1u);
    }
    for (uint32_t i = 0; i < 4; ++i) {
      mbar_init(cta.bar(kOffBFull, i), 1u);
      mbar_init(cta.bar(kOffBEmpty, i), 1u);
    }
    mbar_init(cta.bar(kOffAccFull), 1u);
    mbar_init(cta.bar(kOffAccFree), kDecodeWarps);
  }
  cta.setup(tiles_smem_raw, plan, kDecodeWarps, p.table, p.table_words);  // fences, table copy, CTA barrier
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tiles_smem_raw + plan.misc + kOffTmem);
  if (cta.warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  cta.tmem_base = *tmem_slot;
  // the digit planes and the scratch header are written by the kernel before this one
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const uint32_t warp = cta.warp, lane = cta.lane;
  const uint32_t N = p.n_cols;
  const uint32_t stage_bytes = N * 128u;
  const uint32_t nst = p.a_stages;
  const uint32_t a_col0 = 2u * N;  // tensor-memory columns: accumulator halves at 0 and N, then the A stages
  bool ok = true;
  SegWalk walk(p);
  uint32_t mat, rb0, rb1;

  // (18 warps leave 96 registers per thread, which the decoding warps fit without spilling.)
  if (warp == kLoaderWarp) {
    // ---- B operand: one slice of digit planes per step, scratch -> shared memory ------------------
    uint32_t gb = 0;
    while (ok && walk.next(p, mat, rb0, rb1)) {
      const uint32_t S = FIELD(steps), n_iter = ((rb1 - rb0 + kDecodeWarps - 1) / kDecodeWarps) * S;
      const uint8_t* src0 = FIELD(xdig) + kHdrBytes;
      for (uint32_t i = 0, s = 0; i < n_iter && ok; ++i) {
        const uint32_t bst = gb % p.b_stages;
        if (gb >= p.b_stages) ok = cta.wait(cta.bar(kOffBEmpty, bst), ((gb / p.b_stages) - 1u) & 1u);
        if (ok && lane == 0) {
          const uint32_t full = cta.bar(kOffBFull, bst);
          const uint32_t dst = smem0 + plan.x + bst * stage_bytes;
          const uint8_t* src = src0 + (size_t)s * stage_bytes;
          mbar_expect_tx(full, stage_bytes);
          for (uint32_t off = 0; off < stage_bytes; off += 8192u) bulk_g2s(dst + off, src + off, min(8192u, stage_bytes - off), full);
        }
        __syncwarp();
        ++gb;
        if (++s == S) s = 0;
      }
    }
  } else if (warp == kMmaWarp) {
    // ---- tensor core: 2 halves x 4 MMAs (K = 32 each) per step -------------------------------------
    const uint32_t idesc = i8_idesc<SIGNED>(N);
    uint32_t gs = 0, rr = 0;
    uint32_t st = 0, st_wraps = 0;  // A stage of step gs and how often the stages have wrapped: gs = st_wraps * nst + st
    while (ok && walk.next(p, mat, rb0, rb1)) {
      const uint32_t S = FIELD(steps), nrb = rb1 - rb0, R = (nrb + kDecodeWarps - 1) / kDecodeWarps, n_iter = R * S;
      const bool upper = nrb > 8u * R;  // some warp of the second operand half has rows
      for (uint32_t i = 0, s = 0; i < n_iter && ok; ++i) {
        if (s == 0 && rr > 0) ok = cta.wait(cta.bar(kOffAccFree), (rr - 1u) & 1u);  // the accumulators have been read
        const uint32_t bst = gs % p.b_stages;
        if (ok) ok = cta.wait(cta.bar(kOffBFull, bst), (gs / p.b_stages) & 1u);
        if (ok) ok = cta.wait(cta.bar(kOffAFull, st), st_wraps & 1u);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (lane == 0) {
          const uint32_t b_tile = smem0 + plan.x + bst * stage_bytes;
#pragma unroll
          for (uint32_t h = 0; h < 2; ++h) {
            if (h == 1 && !upper) break;
            const uint32_t a = cta.tmem_base + a_col0 + (h * nst + st) * kStepCols;
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k)
              umma_i8_ts(cta.tmem_base + h * N, a + 8u * k, umma_desc(b_tile + k * 32u), idesc, (s | k) != 0u);
          }
          umma_commit(cta.bar(kOffAEmpty, st));
          umma_commit(cta.bar(kOffBEmpty, bst));
          if (s == S - 1u) umma_commit(cta.bar(kOffAccFull));
        }
        __syncwarp();
        ++gs;
        if (++st == nst) {
          st = 0;
          ++st_wraps;
        }
        if (++s == S) {
          s = 0;
          ++rr;
        }
      }
    }
  } else if (warp < kDecodeWarps) {
    // ---- decoding warps ---------------------------------------------------------------------------
    const uint32_t g = lane >> 2, t = lane & 3u;
    const uint32_t half = warp >> 3;
    const uint32_t lane_field = (32u * (warp & 3u) + 16u * ((warp >> 2) & 1u)) << 16;
    const uint32_t a_base = cta.tmem_base + lane_field + a_col0 + half * nst * kStepCols;
    const uint32_t acc_base = cta.tmem_base + lane_field + half * N;
    uint32_t rr = 0;
    uint32_t st = 0, st_wraps = 0;  // A stage of the next step and how often the stages have wrapped
    bool table_ok = false;
    while (ok && walk.next(p, mat, rb0, rb1)) {
      if (!table_ok) {  // the table copy started with the kernel; its first use is below
        ok = table_ok = cta.wait_table();
        if (!ok) break;
      }
      const uint32_t S = FIELD(steps), R = (rb1 - rb0 + kDecodeWarps - 1) / kDecodeWarps;
      const uint32_t* const raw = FIELD(raw);
      const uint32_t my0 = min(rb1, rb0 + warp * R), my1 = min(rb1, my0 + R);
      const uint32_t t0 = my0 * S, t1 = my1 * S;
      const uint32_t n_real = t1 - t0, n_iter = R * S;

      uint32_t rd = 0, stop_pos = 0, w_pos = 0, i_pos = 0;
      const uint4* tok = FIELD(tokens) + (size_t)t0 * 64u + lane;
      const uint32_t* trp = FIELD(tile_raw) + t0 + 1;
      uint4 q[2][2] = {};
      uint32_t tr[2] = {0, 0};
      if (n_real) {
        rd = __ldg(trp - 1);
        stop_pos = __ldg(trp - 1 + n_real);
#pragma unroll
        for (int k = 0; k < 2; ++k) {  // the tokens do not wait for the tile index: asked for before its first use
          q[k][0] = ldg_stream(tok + k * 64);
          q[k][1] = ldg_stream(tok + k * 64 + 32);
          tr[k] = __ldg(trp + k);
        }
        tok += 2 * 64;
        trp += 2;
        w_pos = i_pos = rd & ~(uint32_t)(kChunkWords - 1);
        for (int k = 0; k < kSlots && i_pos < stop_pos; ++k, i_pos += kChunkWords) cta.issue_chunk(raw, i_pos);
      }
      uint32_t w[16];
      uint32_t s_p = 0, rb = my0;
      bool pending = false;  // a tile has been stored whose arrival on the stage's barrier is still due
      uint32_t pending_stage = 0;
      // (Reading a finished row block's accumulators back a few tiles into the next row block, and prefetching the
      // token tiles into L2 as the one-vector kernel does, were both measured slower: +6 % each at 8 vectors.)
      bool drain_due = false, drain_real = false;
      uint32_t drain_rb = 0;

      auto lookups = [&](int k) {  // tile words -> w; token registers reloaded two tiles ahead; ring refilled
        const uint32_t rd_next = tr[k];
        while (ok && rd_next > w_pos) {
          ok = cta.wait_chunk();
          w_pos += kChunkWords;
        }
        if (!ok) return;
        cta.lookup16(q[k], w);
        q[k][0] = ldg_stream(tok);
        q[k][1] = ldg_stream(tok + 32);
        tr[k] = __ldg(trp);
        tok += 64;
        ++trp;
        rd = rd_next;
        __syncwarp();  // every lane has issued its reads of the chunks below rd
        const uint32_t lim = min(stop_pos, (rd & ~(uint32_t)(kChunkWords - 1)) + kRingWords);
        for (; i_pos < lim; i_pos += kChunkWords) cta.issue_chunk(raw, i_pos);
      };
      auto publish = [&]() {  // the stored tile is in tensor memory: tell the MMA warp
        if (!pending) return;
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        if (lane == 0) mbar_arrive_one(cta.bar(kOffAFull, pending_stage));
        pending = false;
      };
      // the accumulators of row block drain_rb (rows of this warp, round rr) -> y
      auto drain = [&]() {
        if (!drain_due) return;
        drain_due = false;
        const bool real = drain_real;
        const uint32_t rb = drain_rb;
        // the row scales are asked for before the wait for the last MMAs of the row block, not after it
        const uint32_t rows = FIELD(rows), has_zero = FIELD(has_zero);
        const float* const scale = FIELD(scale);
        const float* const zero = FIELD(zero);
        const uint32_t r_lo = rb * 16u + g, r_hi = r_lo + 8u;
        const float sc_lo = (real && r_lo < rows) ? __ldg(scale + r_lo) : 0.f, sc_hi = (real && r_hi < rows) ? __ldg(scale + r_hi) : 0.f;
        const float z_lo = (real && has_zero && r_lo < rows) ? __ldg(zero + r_lo) : 0.f;
        const float z_hi = (real && has_zero && r_hi < rows) ? __ldg(zero + r_hi) : 0.f;
        ok = ok && cta.wait(cta.bar(kOffAccFull), rr & 1u);
        if (ok && real) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          float* const y = FIELD(y);
          const double* const hdr = reinterpret_cast<const double*>(FIELD(xdig));
          for (uint32_t bq = 0; bq * 16u < N; ++bq) {
            int v[8];
            asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                         : "r"(acc_base + 16u * bq));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const uint32_t b = 4u * bq + t;
            if (b < p.nb) {
              const double os = hdr[b], sx = hdr[32 + b];
              const long long y_lo = (long long)v[0] + ((long long)v[1] << 8) + ((long long)v[4] << 16) + ((long long)v[5] << 24);
              const long long y_hi = (long long)v[2] + ((long long)v[3] << 8) + ((long long)v[6] << 16) + ((long long)v[7] << 24);
              if (r_lo < rows) y[(size_t)b * rows + r_lo] = (float)((double)sc_lo * ((double)y_lo * os - (double)z_lo * sx));
              if (r_hi < rows) y[(size_t)b * rows + r_hi] = (float)((double)sc_hi * ((double)y_hi * os - (double)z_hi * sx));
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_one(cta.bar(kOffAccFree));
        ++rr;
      };
      auto step = [&](int k, uint32_t i) {
        const bool real = i < n_real;
        if (real) lookups(k);  // this tile's words, in flight while the previous store completes
        publish();
        if (ok && st_wraps != 0u) ok = cta.wait(cta.bar(kOffAEmpty, st), (st_wraps - 1u) & 1u);
        if (!ok) return;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (real) {
          asm volatile(
              "tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(
                  a_base + st * kStepCols),
              "r"(w[0]), "r"(w[1]), "r"(w[8]), "r"(w[9]), "r"(w[2]), "r"(w[3]), "r"(w[10]), "r"(w[11]), "r"(w[4]), "r"(w[5]),
              "r"(w[12]), "r"(w[13]), "r"(w[6]), "r"(w[7]), "r"(w[14]), "r"(w[15])
              : "memory");
        }
        pending = true;
        pending_stage = st;
        if (++st == nst) {
          st = 0;
          ++st_wraps;
        }
        if (++s_p == S) {  // the row block is complete: all warps read their rows of the accumulators back
          s_p = 0;
          publish();
          drain_due = true;
          drain_real = real;
          drain_rb = rb;
          drain();
          ++rb;
        }
      };

      for (uint32_t i = 0; i < n_iter && ok; i += 2) {
        step(0, i);
        if (i + 1u < n_iter && ok) step(1, i + 1u);
      }
      if (ok) publish();
      while (ok && cta.n_waited < cta.n_issued) ok = cta.wait_chunk();  // nothing may still be landing when the ring is reused
    }
  }

  // a CTA without work has not waited for its copy of the table yet: nothing may still be landing in
  // shared memory when the CTA ends
  if (warp == 0 && ok) ok = cta.wait_table();
  if (!ok) {
    *cta.dead_flag() = 1u;
    if (lane == 0) atomicOr(p.mats ? p.mats[0].status : p.one.status, TQ_STATUS_WAIT_EXPIRED);
    // copies that are still in flight target this CTA's shared memory: give them time to land
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(cta.tmem_base), "r"(kTmemCols) : "memory");
  }
}

uint32_t wide_n_cols(int nb) { return (uint32_t)((nb + 3) / 4) * 16u; }

template <class Kern, class Params>
int launch_pdl(Kern kern, dim3 grid, uint32_t threads, size_t smem, cudaStream_t st, const Params& p) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return tq_cuda_status((int)cudaLaunchKernelEx(&cfg, kern, p), "gemv(tiles, tensor core) launch");
}

}  // namespace

uint64_t tq_wide_scratch_bytes(uint32_t steps, int nb) {
  const uint64_t v = kHdrBytes + (uint64_t)steps * wide_n_cols(nb) * 128u;
  return (v + 1023u) / 1024u * 1024u;
}

// The two launches of one product (or of all products of a stack): digit planes, then the fused
// decode + tensor-core kernel.  d_mats == nullptr: single matrix `one`.
int tq_wide_launch(const tq_tiles_desc* d_mats, int n_mats, const void* d_segs, const uint32_t* d_cta_seg,
                   const tq_tiles_desc* one, const uint32_t* d_table, uint32_t table_words, int nb, bool levels_signed,
                   uint32_t grid, void* cuda_stream) {
  if (nb < 1 || nb > 32) return TQ_ERR_INVALID_ARG;
  WideParams p{};
  p.mats = d_mats;
  p.segs = static_cast<const TilesSeg*>(d_segs);
  p.cta_seg = d_cta_seg;
  if (one) p.one = *one;
  p.table = d_table;
  p.table_words = table_words;
  p.nb = (uint32_t)nb;
  p.n_cols = wide_n_cols(nb);
  // as many B-operand stages as fit beside the table and the rings, 2 to 4
  uint32_t stages = 4;
  while (stages > 2 && tiles_smem(table_words, stages * p.n_cols * 32u, kDecodeWarps).total > kSmemLimit) --stages;
  p.b_stages = stages;
  p.a_stages = std::min<uint32_t>(kMaxAStages, (kTmemCols - 2u * p.n_cols) / (2u * kStepCols));
  const size_t smem = tiles_smem(table_words, stages * p.n_cols * 32u, kDecodeWarps).total;
  if (smem > kSmemLimit) return TQ_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  tq_tiles_desc none{};
  wide_prepare_kernel<<<dim3((unsigned)nb, (unsigned)(d_mats ? n_mats : 1)), 256, 0, st>>>(d_mats, one ? *one : none, p.n_cols);
  if (int rc = tq_cuda_status((int)cudaGetLastError(), "gemv(tiles, tensor core): digit planes launch")) return rc;
  if (levels_signed) {
    auto kern = gemv_wide_kernel<true>;
    if (int rc = tq_ensure_dynamic_smem((const void*)kern, smem, "gemv(tiles, tensor core): raising the dynamic shared memory limit")) return rc;
    return launch_pdl(kern, dim3(grid), kWideThreads, smem, st, p);
  }
  auto kern = gemv_wide_kernel<false>;
  if (int rc = tq_ensure_dynamic_smem((const void*)kern, smem, "gemv(tiles, tensor core): raising the dynamic shared memory limit")) return rc;
  return launch_pdl(kern, dim3(grid), kWideThreads, smem, st, p);
}
