// tq_fused_gemm: prefill-sized product Y[M][rows] = X[M][cols] * W^T with W decoded on the fly
// from the PLANES layout into bf16 tiles that feed tcgen05 tensor-core MMAs (sm_100a).
//
// One CTA computes a 128-row x 256-token tile of Y^T.  Per K stage of 128 columns:
//   * 8 producer warps decode the 128 x 128 weight tile (one row x 32 groups per warp pass: a
//     coalesced token load, a ballot for the rank of each marker inside the row's raw plane, one
//     table or raw lookup per lane) and store it as bf16 (value - zero point, exact for integer
//     zero points) in the 128-byte-swizzled K-major layout the MMA reads;
//   * one thread streams the matching 256 x 128 tile of X with two TMA loads (hardware swizzle);
//   * one thread issues 8 tcgen05.mma (M=128, N=256, K=16) into a 128 x 256 fp32 accumulator in
//     tensor memory and commits to the stage's "empty" barrier.
// After the last stage the 8 producer warps read the accumulator back (tcgen05.ld), apply the row
// scale in fp32 and store Y.  Every wait is bounded; on expiry the CTA raises a status bit, drains
// its copies, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdio>

#include "tq_internal.h"
#include "tq_sm100.cuh"

namespace {

using namespace tq_sm100;

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int BM = 128;            // weight rows per CTA (MMA M)
constexpr int BN = 256;            // tokens per CTA (MMA N)
constexpr int BK = 128;            // columns per stage: two 64-column swizzle atoms
constexpr int kStages = 2;
constexpr int kProducerWarps = 8;
constexpr int kGemmThreads = (kProducerWarps + 2) * 32;  // + TMA warp + MMA warp
constexpr uint32_t A_ATOM = BM * 128;                    // 16 KB: 128 rows x 64 bf16
constexpr uint32_t B_ATOM = BN * 128;                    // 32 KB: 256 tokens x 64 bf16
constexpr uint32_t STAGE_BYTES = 2 * A_ATOM + 2 * B_ATOM;  // 96 KB
constexpr uint32_t SMEM_BYTES = kStages * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
struct GemmParams {
  const uint16_t* codes;
  const uint32_t* rawbase;
  const uint16_t* rawidx;
  const uint32_t* raw;
  const uint32_t* table;
  const float* scale;
  const float* zero;
  float* Y;
  uint32_t* status;
  uint32_t K, rows, cols, gpr_pad, nidx_pad, M;
  uint32_t xor_mask;
  float magic;
  int has_zero;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_x, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + kStages * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  const uint32_t accum_bar = bar_base + 8u * (2 * kStages);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + kStages * STAGE_BYTES + 8 * (2 * kStages + 1));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t n0 = blockIdx.x * BN;   // first token of this CTA
  const uint32_t r0 = blockIdx.y * BM;   // first weight row of this CTA
  const uint32_t n_stage = (p.gpr_pad * 4u + BK - 1) / BK;  // gpr_pad is a multiple of 32 groups = 128 columns

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), kProducerWarps + 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(accum_bar, 1);
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = *tmem_slot;

  if (warp < kProducerWarps) {
    // ------------------------------------------------------------------ producers: decode A tiles
    bool alive = true;
    uint32_t bad = 0;
    for (uint32_t it = 0; it < n_stage && alive; ++it) {
      const int s = it % kStages;
      if (it >= kStages) alive = mbar_wait(empty_bar(s), ((it / kStages) - 1) & 1, abort_flag);
      if (!alive) break;
      uint8_t* a_tile = gen_base + s * STAGE_BYTES;
      // this warp's 16 rows: warp, warp + 8, ...
      uint32_t tok[16], rbase[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint32_t row = r0 + warp + 8u * i;
        tok[i] = 0u;
        rbase[i] = 0u;
        if (row < p.rows) {
          tok[i] = __ldg(p.codes + (size_t)row * p.gpr_pad + it * 32u + lane);
          rbase[i] = __ldg(p.rawbase + row) + __ldg(p.rawidx + (size_t)row * p.nidx_pad + it);
        }
      }
      uint32_t w[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const bool esc = tok[i] == 0xFFFFu;
        const uint32_t m = __ballot_sync(kFull, esc);
        const uint32_t rank = __popc(m & ((1u << lane) - 1u));
        if (esc) {
          w[i] = __ldg(p.raw + rbase[i] + rank);
        } else {
          const uint32_t cl = min(tok[i], p.K);
          bad |= tok[i] ^ cl;
          w[i] = __ldg(p.table + cl);
        }
      }
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const uint32_t rl = warp + 8u * i;  // row inside the tile
        const uint32_t row = r0 + rl;
        const float z = (p.has_zero && row < p.rows) ? __ldg(p.zero + row) : 0.f;
        const uint32_t v = w[i] ^ p.xor_mask;
        const float f0 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7540)) - p.magic - z;
        const float f1 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7541)) - p.magic - z;
        const float f2 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7542)) - p.magic - z;
        const float f3 = __uint_as_float(__byte_perm(v, 0x4B000000u, 0x7543)) - p.magic - z;
        __nv_bfloat162 lo = __floats2bfloat162_rn(f0, f1);
        __nv_bfloat162 hi = __floats2bfloat162_rn(f2, f3);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo);
        packed.y = *reinterpret_cast<uint32_t*>(&hi);
        const uint32_t atom = lane >> 4, g = lane & 15u;  // 16 groups = 64 columns per atom
        const uint32_t off = atom * A_ATOM + rl * 128u + (((g >> 1) ^ (rl & 7u)) << 4) + ((g & 1u) << 3);
        *reinterpret_cast<uint2*>(a_tile + off) = packed;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> visible to the MMA
      __syncwarp();
      if (lane == 0) mbar_arrive(full_bar(s));
    }
    if (bad) atomicOr(p.status, TQ_STATUS_BAD_CODE);

    // ------------------------------------------------------------------ epilogue
    if (alive) alive = mbar_wait(accum_bar, 0, abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (alive) {
      const uint32_t lane_base = (warp & 3u) * 32u;       // the TMEM lanes this warp may read
      const uint32_t col_half = (warp >> 2) * (BN / 2);   // warps 0-3: tokens 0..127, warps 4-7: 128..255
      const uint32_t row = r0 + lane_base + lane;
      const float sc = row < p.rows ? __ldg(p.scale + row) : 0.f;
#pragma unroll 1
      for (uint32_t c = 0; c < BN / 2; c += 32) {
        uint32_t v[32];
        const uint32_t taddr = tmem_acc + (lane_base << 16) + col_half + c;
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
            "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
              "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
              "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (row < p.rows) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t token = n0 + col_half + c + j;
            if (token < p.M) p.Y[(size_t)token * p.rows + row] = sc * __uint_as_float(v[j]);
          }
        }
      }
    }
  } else if (warp == kProducerWarps) {
    // ------------------------------------------------------------------ TMA: stream X tiles
    if (lane == 0) {
      bool alive = true;
      uint32_t issued = 0;
      for (uint32_t it = 0; it < n_stage && alive; ++it) {
        const int s = it % kStages;
        if (it >= kStages) alive = mbar_wait(empty_bar(s), ((it / kStages) - 1) & 1, abort_flag);
        if (!alive) break;
        const uint32_t b_tile = base + s * STAGE_BYTES + 2 * A_ATOM;
        mbar_expect_tx(full_bar(s), 2 * B_ATOM);
        tma_load_2d(b_tile, &tmap_x, (int)(it * BK), (int)n0, full_bar(s));
        tma_load_2d(b_tile + B_ATOM, &tmap_x, (int)(it * BK + 64), (int)n0, full_bar(s));
        issued = it + 1;
      }
      if (!alive) {
        // let the copies already in flight land before the CTA's shared memory is released
        for (uint32_t it = (issued > kStages ? issued - kStages : 0); it < issued; ++it) {
          for (uint32_t i = 0; i < (1u << 16); ++i) __nanosleep(64);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(BM, BN);
      bool alive = true;
      for (uint32_t it = 0; it < n_stage && alive; ++it) {
        const int s = it % kStages;
        alive = mbar_wait(full_bar(s), (it / kStages) & 1, abort_flag);
        if (!alive) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_tile = base + s * STAGE_BYTES, b_tile = a_tile + 2 * A_ATOM;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          const uint32_t atom = k >> 2, koff = (k & 3) * 32;
          umma_bf16(tmem_acc, umma_desc(a_tile + atom * A_ATOM + koff), umma_desc(b_tile + atom * B_ATOM + koff), idesc,
                    (it | (uint32_t)k) != 0u);
        }
        umma_commit(empty_bar(s));
      }
      if (alive) umma_commit(accum_bar);
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(BN) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, TQ_STATUS_WAIT_EXPIRED);
}

}  // namespace

extern "C" int tq_fused_gemm(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, void* cuda_stream) {
  if (!m || !d_X_bf16 || !d_Y || M < 1 || ((uintptr_t)d_X_bf16 & 15)) return TQ_ERR_INVALID_ARG;
  if (m->info.layout != TQ_LAYOUT_PLANES) return TQ_ERR_UNSUPPORTED_SHAPE;  // needs the fixed-stride token plane
  if (!m->zero_bf16_exact) return TQ_ERR_UNSUPPORTED_SHAPE;                 // level - zero point would be rounded to bf16
  if ((m->info.cols * 2u) % 16u != 0) return TQ_ERR_UNSUPPORTED_SHAPE;     // TMA row pitch must be a multiple of 16 bytes
  EncodeTiledFn enc = encode_fn();
  if (!enc) return tq_cuda_status((int)cudaErrorUnknown, "gemm: cuTensorMapEncodeTiled not available");

  CUtensorMap tmap;
  const cuuint64_t gdim[2] = {m->info.cols, (cuuint64_t)M};
  const cuuint64_t gstride[1] = {(cuuint64_t)m->info.cols * 2};
  const cuuint32_t box[2] = {64, BN};
  const cuuint32_t estr[2] = {1, 1};
  CUresult cr = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_X_bf16), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return tq_cuda_status((int)cudaErrorInvalidValue, "gemm: tensor map encode failed");

  if (int rc = tq_ensure_dynamic_smem((const void*)gemm_kernel, SMEM_BYTES, "gemm: raising the dynamic shared memory limit")) return rc;
  GemmParams p;
  p.codes = m->d_codes;
  p.rawbase = m->d_rawbase;
  p.rawidx = m->d_rawidx;
  p.raw = m->d_raw;
  p.table = m->dict->d_table;
  p.scale = m->d_scale;
  p.zero = m->d_zero;
  p.Y = d_Y;
  p.status = m->d_status;
  p.K = m->dict->K;
  p.rows = m->info.rows;
  p.cols = m->info.cols;
  p.gpr_pad = m->gpr_pad;
  p.nidx_pad = m->nidx_pad;
  p.M = (uint32_t)M;
  p.xor_mask = m->info.levels_signed ? 0x80808080u : 0u;
  p.magic = m->info.levels_signed ? 8388736.0f : 8388608.0f;
  p.has_zero = m->has_zero;
  dim3 grid((M + BN - 1) / BN, (m->info.rows + BM - 1) / BM);
  gemm_kernel<<<grid, kGemmThreads, SMEM_BYTES, (cudaStream_t)cuda_stream>>>(tmap, p);
  return tq_cuda_status((int)cudaGetLastError(), "gemm launch");
}
