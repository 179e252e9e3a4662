// tq_fused_gemm_ws: the prefill-sized product for the TILES layout in two pipelined phases that
// share a caller-provided workspace (sm_100a).
//
// Why two phases.  A weight tile decoded inside the GEMM is decoded again for every tile of tokens
// that meets it (8 times at M = 2048 with 256-token tiles), and the table the decode wants in
// shared memory (136 KB) competes with the operand stages the tensor core wants there.  Decoding
// a whole layer once costs a few tens of microseconds at HBM speed, and a layer's bf16 weights
// (<= 50 MB for every LLaMA-3.2 matrix but the output head) stay in the 126 MB L2 for the product
// that follows.  So: phase 1 streams the compressed layer once and writes bf16 (level - zero point,
// exact) into the workspace; phase 2 is a persistent tcgen05 GEMM whose operands both arrive by TMA
// -- 128 weight rows x 256 tokens per tile, 64 columns per stage, 4 stages, two 256-column
// accumulators in tensor memory so that the epilogue of one tile overlaps the MMAs of the next.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>

#include "tq_internal.h"
#include "tq_sm100.cuh"

namespace {

using namespace tq_sm100;

constexpr int BM = 128;   // weight rows per tile (MMA M)
// tokens per tile (MMA N) is a template parameter: 256, or 128 where that fills the SMs better
constexpr int BK = 64;    // columns per stage: one 128-byte swizzle atom of bf16
constexpr int kStages = 4;
constexpr uint32_t A_BYTES = BM * BK * 2;  // 16 KB
constexpr int kThreads = 6 * 32;  // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
template <int BN>
struct Geo {
  static constexpr uint32_t B_BYTES = BN * BK * 2;  // 32 or 16 KB
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr uint32_t SMEM_BYTES = kStages * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};
struct GemmWsParams {
  const float* scale;
  float* Y;
  uint32_t* status;
  uint32_t rows, cols, M;
  uint32_t row_tiles, token_tiles;
};

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ws_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const GemmWsParams p) {
  constexpr uint32_t STAGE_BYTES = Geo<BN>::STAGE_BYTES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // operand tiles need 1024-byte alignment
  uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + kStages * STAGE_BYTES;
  auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
  auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (kStages + s); };
  auto acc_full = [&](uint32_t b) { return bar_base + 8u * (2 * kStages + b); };
  auto acc_empty = [&](uint32_t b) { return bar_base + 8u * (2 * kStages + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + kStages * STAGE_BYTES + 8 * (2 * kStages + 4));
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t n_tiles = p.row_tiles * p.token_tiles;
  const uint32_t n_k = (p.cols + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (uint32_t b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), 4);
    }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA: both operands
    if (lane == 0) {
      bool alive = true;
      uint32_t it = 0;
      for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
        const int r0 = (int)((tile / p.token_tiles) * BM), n0 = (int)((tile % p.token_tiles) * BN);
        for (uint32_t ks = 0; ks < n_k && alive; ++ks, ++it) {
          const uint32_t s = it % kStages;
          alive = mbar_wait(empty_bar(s), ((it / kStages) & 1u) ^ 1u, abort_flag);
          if (!alive) break;
          const uint32_t a_tile = base + s * STAGE_BYTES;
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          tma_load_2d(a_tile, &tmap_w, (int)(ks * BK), r0, full_bar(s));
          tma_load_2d(a_tile + A_BYTES, &tmap_x, (int)(ks * BK), n0, full_bar(s));
        }
      }
      if (!alive) {  // let the copies already in flight land before the CTA's shared memory is released
        for (uint32_t i = 0; i < (1u << 14); ++i) __nanosleep(256);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(BM, BN);
      bool alive = true;
      uint32_t it = 0, local = 0;
      for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++local) {
        const uint32_t buf = local & 1u, use = local >> 1;
        alive = mbar_wait(acc_empty(buf), (use & 1u) ^ 1u, abort_flag);  // the epilogue has drained this accumulator
        if (!alive) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_acc + buf * BN;
        for (uint32_t ks = 0; ks < n_k && alive; ++ks, ++it) {
          const uint32_t s = it % kStages;
          alive = mbar_wait(full_bar(s), (it / kStages) & 1u, abort_flag);
          if (!alive) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_tile = base + s * STAGE_BYTES, b_tile = a_tile + A_BYTES;
#pragma unroll
          for (uint32_t k = 0; k < BK / 16; ++k)
            umma_bf16(d_tmem, umma_desc(a_tile + k * 32u), umma_desc(b_tile + k * 32u), idesc, (ks | k) != 0u);
          umma_commit(empty_bar(s));
        }
        if (alive) umma_commit(acc_full(buf));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: TMEM -> scale -> Y
    const uint32_t quarter = warp & 3u;  // the TMEM lanes this warp may read: 32 * (warp % 4) ..
    bool alive = true;
    uint32_t local = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++local) {
      const uint32_t buf = local & 1u, use = local >> 1;
      const uint32_t r0 = (tile / p.token_tiles) * BM, n0 = (tile % p.token_tiles) * BN;
      alive = mbar_wait(acc_full(buf), use & 1u, abort_flag);
      if (!alive) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t row = r0 + quarter * 32u + lane;
      const float sc = row < p.rows ? __ldg(p.scale + row) : 0.f;
#pragma unroll 1
      for (uint32_t c = 0; c < BN; c += 32) {
        uint32_t v[32];
        const uint32_t taddr = tmem_acc + ((quarter * 32u) << 16) + buf * BN + c;
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
            const uint32_t token = n0 + c + j;
            if (token < p.M) p.Y[(size_t)token * p.rows + row] = sc * __uint_as_float(v[j]);
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty(buf));
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(2 * BN) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status, TQ_STATUS_WAIT_EXPIRED);
}

}  // namespace

extern "C" {

int tq_gemm_workspace_size(const tq_dmat* m, uint64_t* bytes) {
  if (!m || !bytes) return TQ_ERR_INVALID_ARG;
  if (m->info.layout != TQ_LAYOUT_TILES) return TQ_ERR_UNSUPPORTED_SHAPE;
  *bytes = (uint64_t)m->tiles.row_blocks * 16 * m->tiles.steps * 128 * 2;  // whole tiles of bf16
  return TQ_OK;
}

int tq_decode_bf16(const tq_dmat* m, void* d_workspace, uint64_t workspace_bytes, void* cuda_stream) {
  if (!m || !d_workspace || ((uintptr_t)d_workspace & 255)) return TQ_ERR_INVALID_ARG;
  if (m->info.layout != TQ_LAYOUT_TILES) return TQ_ERR_UNSUPPORTED_SHAPE;
  uint64_t need = 0;
  tq_gemm_workspace_size(m, &need);
  if (workspace_bytes < need) return TQ_ERR_BUFFER_TOO_SMALL;
  return tq_tiles_decode_bf16(m, d_workspace, cuda_stream);
}

int tq_fused_gemm_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, void* d_workspace,
                     uint64_t workspace_bytes, void* cuda_stream) {
  if (!d_X_bf16 || !d_Y || M < 1) return TQ_ERR_INVALID_ARG;
  if (int rc = tq_decode_bf16(m, d_workspace, workspace_bytes, cuda_stream)) return rc;
  return tq_gemm_bf16_ws(m, d_X_bf16, M, d_Y, d_workspace, cuda_stream);
}

int tq_gemm_bf16_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, const void* d_workspace,
                    void* cuda_stream) {
  if (!m || !d_X_bf16 || !d_Y || !d_workspace || M < 1 || ((uintptr_t)d_X_bf16 & 15) || ((uintptr_t)d_workspace & 255))
    return TQ_ERR_INVALID_ARG;
  if (m->info.layout != TQ_LAYOUT_TILES) return TQ_ERR_UNSUPPORTED_SHAPE;
  if ((m->info.cols * 2u) % 16u != 0) return TQ_ERR_UNSUPPORTED_SHAPE;  // TMA row pitch must be a multiple of 16 bytes
  EncodeTiledFn enc = encode_fn();
  if (!enc) return tq_cuda_status((int)cudaErrorUnknown, "gemm: cuTensorMapEncodeTiled not available");

  const uint32_t rows_pad = m->tiles.row_blocks * 16u, pitch = m->tiles.steps * 128u;
  CUtensorMap tmap_w;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t gdim[2] = {m->info.cols, rows_pad};
    const cuuint64_t gstride[1] = {(cuuint64_t)pitch * 2};
    const cuuint32_t box[2] = {BK, BM};
    if (enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_workspace), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return tq_cuda_status((int)cudaErrorInvalidValue, "gemm: tensor map of the weights");
  }
  GemmWsParams p;
  p.scale = m->d_scale;
  p.Y = d_Y;
  p.status = m->d_status;
  p.rows = m->info.rows;
  p.cols = m->info.cols;
  p.M = (uint32_t)M;
  p.row_tiles = (m->info.rows + BM - 1) / BM;
  // 256-token tiles halve the operand traffic per flop; 128-token tiles where they leave fewer SMs idle
  const uint32_t sms = (uint32_t)sm_count();
  auto fill = [&](uint32_t bn) {
    const uint32_t tiles = p.row_tiles * (((uint32_t)M + bn - 1) / bn);
    return (double)tiles / (double)(((tiles + sms - 1) / sms) * sms);
  };
  // (measured: at M = 2048 the narrow tile loses more to operand traffic than it gains in SM fill, so it
  // is kept for token counts that leave half of a 256-token tile empty)
  const bool narrow = (uint32_t)M <= 128u && fill(128) >= fill(256);
  const uint32_t bn = narrow ? 128u : 256u;
  p.token_tiles = ((uint32_t)M + bn - 1) / bn;
  CUtensorMap tmap_x;
  {
    const cuuint64_t gdim[2] = {m->info.cols, (cuuint64_t)M};
    const cuuint64_t gstride[1] = {(cuuint64_t)m->info.cols * 2};
    const cuuint32_t box[2] = {BK, bn};
    if (enc(&tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_X_bf16), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return tq_cuda_status((int)cudaErrorInvalidValue, "gemm: tensor map of the activations");
  }
  const uint32_t grid = std::min<uint32_t>(p.row_tiles * p.token_tiles, sms);
  static bool configured = false;
  if (!configured) {
    int rc = tq_cuda_status((int)cudaFuncSetAttribute(gemm_ws_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                      (int)Geo<256>::SMEM_BYTES), "gemm: raising the dynamic shared memory limit");
    if (rc == TQ_OK)
      rc = tq_cuda_status((int)cudaFuncSetAttribute(gemm_ws_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                    (int)Geo<128>::SMEM_BYTES), "gemm: raising the dynamic shared memory limit");
    if (rc != TQ_OK) return rc;
    configured = true;
  }
  if (narrow)
    gemm_ws_kernel<128><<<grid, kThreads, Geo<128>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(tmap_w, tmap_x, p);
  else
    gemm_ws_kernel<256><<<grid, kThreads, Geo<256>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(tmap_w, tmap_x, p);
  return tq_cuda_status((int)cudaGetLastError(), "gemm launch");
}

}  // extern "C"
