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
#include <new>
#include <vector>

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

// What one output tile needs: the two tensor maps, where it sits, how many 64-column stages it
// takes, and where its results go.
struct TileInfo {
  const CUtensorMap* map_w;
  const CUtensorMap* map_x;
  const float* scale;
  float* Y;
  uint32_t rows, n_k, r0, n0;
};

// One matrix: tensor maps in the kernel's parameter space.
struct SingleSrc {
  const CUtensorMap* map_w;
  const CUtensorMap* map_x;
  GemmWsParams p;
  __device__ __forceinline__ uint32_t total() const { return p.row_tiles * p.token_tiles; }
  __device__ __forceinline__ uint32_t M() const { return p.M; }
  __device__ __forceinline__ uint32_t* status() const { return p.status; }
  // `cursor` (unused here) and `fresh` (the maps were not used by this thread before) serve GroupSrc
  template <int BN>
  __device__ __forceinline__ TileInfo locate(uint32_t tile, uint32_t& cursor, bool& fresh) const {
    (void)cursor;
    fresh = false;
    TileInfo t;
    t.map_w = map_w;
    t.map_x = map_x;
    t.scale = p.scale;
    t.Y = p.Y;
    t.rows = p.rows;
    t.n_k = (p.cols + BK - 1) / BK;
    t.r0 = (tile / p.token_tiles) * BM;
    t.n0 = (tile % p.token_tiles) * BN;
    return t;
  }
};

// Several matrices, one token count: the tiles of all of them in one sequence.  Everything lives in
// DEVICE memory, the tensor maps included (2 per matrix: weights, activations; 128 bytes each).
struct GroupEntry {
  const float* scale;
  float* Y;
  uint32_t rows, cols;
};
struct GroupSrc {
  const CUtensorMap* maps;
  const GroupEntry* groups;
  const uint32_t* tile_begin;  // n_groups + 1
  uint32_t* status_word;
  uint32_t n_groups, token_tiles, n_tokens, n_tiles;
  __device__ __forceinline__ uint32_t total() const { return n_tiles; }
  __device__ __forceinline__ uint32_t M() const { return n_tokens; }
  __device__ __forceinline__ uint32_t* status() const { return status_word; }
  // Tiles come in ascending order, so the group index only moves forward from `cursor`.
  template <int BN>
  __device__ __forceinline__ TileInfo locate(uint32_t tile, uint32_t& cursor, bool& fresh) const {
    uint32_t g = cursor == 0xFFFFFFFFu ? 0u : cursor;
    while (g + 1 < n_groups && tile >= __ldg(tile_begin + g + 1)) ++g;
    fresh = g != cursor;
    cursor = g;
    const uint32_t local = tile - __ldg(tile_begin + g);
    const GroupEntry e = groups[g];
    TileInfo t;
    t.map_w = maps + 2 * g;
    t.map_x = maps + 2 * g + 1;
    t.scale = e.scale;
    t.Y = e.Y;
    t.rows = e.rows;
    t.n_k = (e.cols + BK - 1) / BK;
    t.r0 = (local / token_tiles) * BM;
    t.n0 = (local % token_tiles) * BN;
    return t;
  }
};

// A tensor map read from global memory: the copy unit reads it through its own path, so the thread
// that is about to use it orders that read after the writes that made the map.
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* map) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(map) : "memory");
}

template <int BN, class Src>
__device__ __forceinline__ void gemm_ws_body(const Src& src) {
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
  const uint32_t n_tiles = src.total();

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
      uint32_t cursor = 0xFFFFFFFFu;
      for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x) {
        bool fresh;
        const TileInfo t = src.template locate<BN>(tile, cursor, fresh);
        if (fresh) {
          tensormap_acquire(t.map_w);
          tensormap_acquire(t.map_x);
        }
        for (uint32_t ks = 0; ks < t.n_k && alive; ++ks, ++it) {
          const uint32_t s = it % kStages;
          alive = mbar_wait(empty_bar(s), ((it / kStages) & 1u) ^ 1u, abort_flag);
          if (!alive) break;
          const uint32_t a_tile = base + s * STAGE_BYTES;
          mbar_expect_tx(full_bar(s), STAGE_BYTES);
          tma_load_2d(a_tile, t.map_w, (int)(ks * BK), (int)t.r0, full_bar(s));
          tma_load_2d(a_tile + A_BYTES, t.map_x, (int)(ks * BK), (int)t.n0, full_bar(s));
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
      uint32_t it = 0, local = 0, cursor = 0xFFFFFFFFu;
      for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++local) {
        bool fresh;
        const uint32_t n_k = src.template locate<BN>(tile, cursor, fresh).n_k;
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
    uint32_t local = 0, cursor = 0xFFFFFFFFu;
    const uint32_t n_tokens = src.M();
    for (uint32_t tile = blockIdx.x; tile < n_tiles && alive; tile += gridDim.x, ++local) {
      const uint32_t buf = local & 1u, use = local >> 1;
      bool fresh;
      const TileInfo t = src.template locate<BN>(tile, cursor, fresh);
      const uint32_t n0 = t.n0;
      alive = mbar_wait(acc_full(buf), use & 1u, abort_flag);
      if (!alive) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t row = t.r0 + quarter * 32u + lane;
      const float sc = row < t.rows ? __ldg(t.scale + row) : 0.f;
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
        if (row < t.rows) {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t token = n0 + c + j;
            if (token < n_tokens) t.Y[(size_t)token * t.rows + row] = sc * __uint_as_float(v[j]);
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
  if (threadIdx.x == 0 && *abort_flag) atomicOr(src.status(), TQ_STATUS_WAIT_EXPIRED);
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ws_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_x, const GemmWsParams p) {
  gemm_ws_body<BN>(SingleSrc{&tmap_w, &tmap_x, p});
}

template <int BN>
__global__ void __launch_bounds__(kThreads, 1) gemm_ws_group_kernel(const GroupSrc src) {
  gemm_ws_body<BN>(src);
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

}  // extern "C"

namespace {

// Tensor maps of one product: the weights as bf16 in a workspace (rows padded to whole tiles, pitch of
// whole tiles), the activations [M][cols]; boxes of 64 columns x 128 rows / bn tokens, 128-byte swizzle.
int encode_maps(const tq_dmat* m, const void* d_workspace, const void* d_X_bf16, uint32_t M, uint32_t bn, CUtensorMap* map_w,
                CUtensorMap* map_x) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return tq_cuda_status((int)cudaErrorUnknown, "gemm: cuTensorMapEncodeTiled not available");
  const uint32_t rows_pad = m->tiles.row_blocks * 16u, pitch = m->tiles.steps * 128u;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t gdim[2] = {m->info.cols, rows_pad};
    const cuuint64_t gstride[1] = {(cuuint64_t)pitch * 2};
    const cuuint32_t box[2] = {BK, BM};
    if (enc(map_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_workspace), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return tq_cuda_status((int)cudaErrorInvalidValue, "gemm: tensor map of the weights");
  }
  {
    const cuuint64_t gdim[2] = {m->info.cols, (cuuint64_t)M};
    const cuuint64_t gstride[1] = {(cuuint64_t)m->info.cols * 2};
    const cuuint32_t box[2] = {BK, bn};
    if (enc(map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(d_X_bf16), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return tq_cuda_status((int)cudaErrorInvalidValue, "gemm: tensor map of the activations");
  }
  return TQ_OK;
}

int configure_gemm_kernels() {
  const void* kerns[4] = {(const void*)gemm_ws_kernel<256>, (const void*)gemm_ws_kernel<128>, (const void*)gemm_ws_group_kernel<256>,
                          (const void*)gemm_ws_group_kernel<128>};
  const int smem[4] = {(int)Geo<256>::SMEM_BYTES, (int)Geo<128>::SMEM_BYTES, (int)Geo<256>::SMEM_BYTES, (int)Geo<128>::SMEM_BYTES};
  for (int i = 0; i < 4; ++i)
    if (int rc = tq_ensure_dynamic_smem(kerns[i], (size_t)smem[i], "gemm: raising the dynamic shared memory limit")) return rc;
  return TQ_OK;
}

inline uint64_t align256(uint64_t v) { return (v + 255) / 256 * 256; }

}  // namespace

struct tq_gemm_plan {
  GroupSrc src{};
  uint32_t bn = 256, grid = 0;
};

extern "C" {

int tq_gemm_bf16_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, const void* d_workspace,
                    void* cuda_stream) {
  if (!m || !d_X_bf16 || !d_Y || !d_workspace || M < 1 || ((uintptr_t)d_X_bf16 & 15) || ((uintptr_t)d_workspace & 255))
    return TQ_ERR_INVALID_ARG;
  if (m->info.layout != TQ_LAYOUT_TILES) return TQ_ERR_UNSUPPORTED_SHAPE;
  if ((m->info.cols * 2u) % 16u != 0) return TQ_ERR_UNSUPPORTED_SHAPE;  // TMA row pitch must be a multiple of 16 bytes
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
  CUtensorMap tmap_w, tmap_x;
  if (int rc = encode_maps(m, d_workspace, d_X_bf16, (uint32_t)M, bn, &tmap_w, &tmap_x)) return rc;
  const uint32_t grid = std::min<uint32_t>(p.row_tiles * p.token_tiles, sms);
  if (int rc = configure_gemm_kernels()) return rc;
  if (narrow)
    gemm_ws_kernel<128><<<grid, kThreads, Geo<128>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(tmap_w, tmap_x, p);
  else
    gemm_ws_kernel<256><<<grid, kThreads, Geo<256>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(tmap_w, tmap_x, p);
  return tq_cuda_status((int)cudaGetLastError(), "gemm launch");
}

int tq_gemm_plan_size(int n_mats, uint64_t* device_bytes) {
  if (n_mats < 1 || !device_bytes) return TQ_ERR_INVALID_ARG;
  *device_bytes = align256((uint64_t)n_mats * 2 * sizeof(CUtensorMap)) + align256((uint64_t)n_mats * sizeof(GroupEntry)) +
                  align256(((uint64_t)n_mats + 1) * 4) + 256 /* status word */;
  return TQ_OK;
}

int tq_gemm_plan_create(const tq_dmat* const* mats, const void* const* d_X_bf16, float* const* d_Y,
                        const void* const* d_workspaces, int n_mats, int M, void* d_buf, uint64_t d_buf_bytes,
                        void* cuda_stream, tq_gemm_plan** out) {
  if (!mats || !d_X_bf16 || !d_Y || !d_workspaces || n_mats < 1 || M < 1 || !d_buf || ((uintptr_t)d_buf & 255) || !out)
    return TQ_ERR_INVALID_ARG;
  uint64_t need = 0;
  tq_gemm_plan_size(n_mats, &need);
  if (d_buf_bytes < need) return TQ_ERR_BUFFER_TOO_SMALL;
  for (int i = 0; i < n_mats; ++i) {
    if (!mats[i] || !d_X_bf16[i] || !d_Y[i] || !d_workspaces[i] || ((uintptr_t)d_X_bf16[i] & 15) || ((uintptr_t)d_workspaces[i] & 255))
      return TQ_ERR_INVALID_ARG;
    if (mats[i]->info.layout != TQ_LAYOUT_TILES || (mats[i]->info.cols * 2u) % 16u != 0) return TQ_ERR_UNSUPPORTED_SHAPE;
  }
  const uint32_t bn = (uint32_t)M <= 128u ? 128u : 256u;
  const uint32_t token_tiles = ((uint32_t)M + bn - 1) / bn;
  // longest rows first: the tiles that take longest start first, so the last, partly filled round of
  // tiles is made of short ones
  std::vector<int> order((size_t)n_mats);
  for (int i = 0; i < n_mats; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return mats[a]->info.cols > mats[b]->info.cols; });
  std::vector<CUtensorMap> maps((size_t)n_mats * 2);
  std::vector<GroupEntry> groups((size_t)n_mats);
  std::vector<uint32_t> tile_begin((size_t)n_mats + 1);
  uint64_t tiles = 0;
  for (int k = 0; k < n_mats; ++k) {
    const tq_dmat* m = mats[order[k]];
    if (int rc = encode_maps(m, d_workspaces[order[k]], d_X_bf16[order[k]], (uint32_t)M, bn, &maps[2 * k], &maps[2 * k + 1])) return rc;
    groups[k] = GroupEntry{m->d_scale, d_Y[order[k]], m->info.rows, m->info.cols};
    tile_begin[k] = (uint32_t)tiles;
    tiles += (uint64_t)((m->info.rows + BM - 1) / BM) * token_tiles;
    if (tiles > 0x7FFFFFFFull) return TQ_ERR_UNSUPPORTED_SHAPE;
  }
  tile_begin[n_mats] = (uint32_t)tiles;
  if (int rc = configure_gemm_kernels()) return rc;
  tq_gemm_plan* pl = new (std::nothrow) tq_gemm_plan();
  if (!pl) return TQ_ERR_NOMEM;
  uint8_t* base = static_cast<uint8_t*>(d_buf);
  const uint64_t off_groups = align256(maps.size() * sizeof(CUtensorMap));
  const uint64_t off_begin = off_groups + align256(groups.size() * sizeof(GroupEntry));
  const uint64_t off_status = off_begin + align256(tile_begin.size() * 4);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int rc = tq_cuda_status((int)cudaMemcpyAsync(base, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, st), "gemm plan upload");
  if (rc == TQ_OK)
    rc = tq_cuda_status((int)cudaMemcpyAsync(base + off_groups, groups.data(), groups.size() * sizeof(GroupEntry), cudaMemcpyHostToDevice, st), "gemm plan upload");
  if (rc == TQ_OK)
    rc = tq_cuda_status((int)cudaMemcpyAsync(base + off_begin, tile_begin.data(), tile_begin.size() * 4, cudaMemcpyHostToDevice, st), "gemm plan upload");
  if (rc == TQ_OK) rc = tq_cuda_status((int)cudaMemsetAsync(base + off_status, 0, 256, st), "gemm plan upload");
  if (rc == TQ_OK) rc = tq_cuda_status((int)cudaStreamSynchronize(st), "gemm plan upload");  // the host vectors go away
  if (rc != TQ_OK) {
    delete pl;
    return rc;
  }
  pl->src.maps = reinterpret_cast<const CUtensorMap*>(base);
  pl->src.groups = reinterpret_cast<const GroupEntry*>(base + off_groups);
  pl->src.tile_begin = reinterpret_cast<const uint32_t*>(base + off_begin);
  pl->src.status_word = reinterpret_cast<uint32_t*>(base + off_status);
  pl->src.n_groups = (uint32_t)n_mats;
  pl->src.token_tiles = token_tiles;
  pl->src.n_tokens = (uint32_t)M;
  pl->src.n_tiles = (uint32_t)tiles;
  pl->bn = bn;
  pl->grid = std::min<uint32_t>((uint32_t)tiles, (uint32_t)sm_count());
  *out = pl;
  return TQ_OK;
}

int tq_gemm_plan_run(const tq_gemm_plan* pl, void* cuda_stream) {
  if (!pl) return TQ_ERR_INVALID_ARG;
  if (pl->bn == 128u)
    gemm_ws_group_kernel<128><<<pl->grid, kThreads, Geo<128>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(pl->src);
  else
    gemm_ws_group_kernel<256><<<pl->grid, kThreads, Geo<256>::SMEM_BYTES, (cudaStream_t)cuda_stream>>>(pl->src);
  return tq_cuda_status((int)cudaGetLastError(), "gemm plan launch");
}

int tq_gemm_plan_status(const tq_gemm_plan* pl, void* cuda_stream, uint32_t* status) {
  if (!pl || !status) return TQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (int rc = tq_cuda_status((int)cudaMemcpyAsync(status, pl->src.status_word, 4, cudaMemcpyDeviceToHost, st), "gemm plan status")) return rc;
  return tq_cuda_status((int)cudaStreamSynchronize(st), "gemm plan status");
}

void tq_gemm_plan_free(tq_gemm_plan* pl) { delete pl; }

}  // extern "C"
