// Device-side encoder: from 8-bit levels resident on the GPU straight to the TQ_LAYOUT_TILES image
// (Listing 3's decision per aligned group -- in the table or not -- plus the tiling of tq_upload),
// without a trip through the host.  The image is byte for byte the one the host builder makes.
//
// Three kernels on the caller's stream: (1) one warp per tile looks every group of the tile up in
// the window -> code map and counts the groups that go to the raw stream (not in the table, or
// coded beyond what the kernels keep in shared memory); (2) one CTA turns the per-tile counts into
// the tile_raw index; (3) one warp per tile looks the groups up again and writes tokens and raw
// words, numbering a tile's raw words slot by slot with warp ballots.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "tq_internal.h"

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr uint32_t kMissBase = 0x10000u - TQ_TILES_RING_WORDS;

struct EncodeParams {
  const uint8_t* levels;   // rows x cols, row-major
  const tq_map_slot* map;
  uint32_t rows, cols, gpr, steps, n_tiles;
  uint32_t* tile_raw;      // n_tiles + 1 + 8 entries
  uint16_t* tokens;        // n_tiles x 512
  uint32_t* raw;
  unsigned long long* counters;  // [0] groups found in the table, [1] groups not found
};

// Code of a 4-byte window, 0 if it is not in the table.
__device__ __forceinline__ uint32_t find_code(const tq_map_slot* __restrict__ map, uint32_t key) {
  uint32_t h = (key * 0x9E3779B1u) >> 14;
  for (uint32_t probes = 0; probes < kMapSlots; ++probes) {
    const uint2 s = __ldg(reinterpret_cast<const uint2*>(map) + h);  // {key, code}
    if (s.y == 0u) return 0u;
    if (s.x == key) return s.y;
    h = (h + 1u) & (kMapSlots - 1u);
  }
  return 0u;
}

// The 16 groups of this lane in tile (rb, s): words w[8h + i] = the 4 levels of row 16 rb + g + 8h,
// group 32 s + 8 t + i; valid bit set where that group exists.
__device__ __forceinline__ uint32_t load_lane_groups(const EncodeParams& p, uint32_t rb, uint32_t s, uint32_t lane,
                                                     uint32_t (&w)[16]) {
  const uint32_t g = lane >> 2, t = lane & 3u;
  const uint32_t g0 = 32u * s + 8u * t;
  uint32_t valid = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t r = rb * 16u + g + 8u * h;
    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.levels + (size_t)r * p.cols) + g0;
    if (r < p.rows && g0 + 8u <= p.gpr && (p.gpr & 3u) == 0u) {  // 32 aligned bytes
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(src)), b = __ldg(reinterpret_cast<const uint4*>(src) + 1);
      w[8 * h] = a.x; w[8 * h + 1] = a.y; w[8 * h + 2] = a.z; w[8 * h + 3] = a.w;
      w[8 * h + 4] = b.x; w[8 * h + 5] = b.y; w[8 * h + 6] = b.z; w[8 * h + 7] = b.w;
      valid |= 0xFFu << (8 * h);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        w[8 * h + i] = 0u;
        if (r < p.rows && g0 + i < p.gpr) {
          w[8 * h + i] = __ldg(src + i);
          valid |= 1u << (8 * h + i);
        }
      }
    }
  }
  return valid;
}

__global__ void __launch_bounds__(256) tiles_count_kernel(const EncodeParams p) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
  unsigned long long hits = 0, misses = 0;
  for (uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; tile < p.n_tiles; tile += warps) {
    uint32_t w[16];
    const uint32_t valid = load_lane_groups(p, tile / p.steps, tile % p.steps, lane, w);
    uint32_t n_raw = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (valid & (1u << j)) {
        const uint32_t c = find_code(p.map, w[j]);
        hits += c != 0u;
        misses += c == 0u;
        n_raw += (c == 0u || c >= TQ_TILES_TABLE_WORDS);
      }
    }
#pragma unroll
    for (int sft = 16; sft > 0; sft >>= 1) n_raw += __shfl_xor_sync(kFull, n_raw, sft);
    if (lane == 0) p.tile_raw[tile + 1] = n_raw;  // shifted by one: the scan turns counts into start indices
  }
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) {
    hits += __shfl_xor_sync(kFull, hits, sft);
    misses += __shfl_xor_sync(kFull, misses, sft);
  }
  if (lane == 0) {
    atomicAdd(p.counters, hits);
    atomicAdd(p.counters + 1, misses);
  }
}

// tile_raw[i + 1] holds the count of tile i; make tile_raw the inclusive running sum (tile_raw[0] = 0)
// and fill the 8 read-ahead entries with the total.  One CTA of 1024 threads.
__global__ void __launch_bounds__(1024) tiles_scan_kernel(uint32_t* tile_raw, uint32_t n_tiles) {
  __shared__ uint32_t part[1024];
  const uint32_t tid = threadIdx.x;
  const uint32_t per = (n_tiles + 1023u) / 1024u;
  const uint32_t b = min(n_tiles, tid * per), e = min(n_tiles, b + per);
  uint32_t sum = 0;
  for (uint32_t i = b; i < e; ++i) sum += tile_raw[i + 1];
  part[tid] = sum;
  __syncthreads();
  for (uint32_t d = 1; d < 1024; d <<= 1) {  // inclusive scan of the per-thread sums
    const uint32_t v = tid >= d ? part[tid - d] : 0u;
    __syncthreads();
    part[tid] += v;
    __syncthreads();
  }
  uint32_t run = part[tid] - sum;
  if (tid == 0) tile_raw[0] = 0u;
  for (uint32_t i = b; i < e; ++i) {
    run += tile_raw[i + 1];
    tile_raw[i + 1] = run;
  }
  __syncthreads();
  if (tid < 8) tile_raw[n_tiles + 1 + tid] = part[1023];
}

__global__ void __launch_bounds__(256) tiles_fill_kernel(const EncodeParams p) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
  for (uint32_t tile = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; tile < p.n_tiles; tile += warps) {
    uint32_t w[16];
    const uint32_t valid = load_lane_groups(p, tile / p.steps, tile % p.steps, lane, w);
    uint32_t pos = p.tile_raw[tile];
    uint32_t tk[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      uint32_t c = 0u;
      bool is_raw = false;
      if (valid & (1u << j)) {
        c = find_code(p.map, w[j]);
        is_raw = c == 0u || c >= TQ_TILES_TABLE_WORDS;
      }
      // slot j of all lanes, lanes ascending: the numbering of the host builder
      const uint32_t m = __ballot_sync(kFull, is_raw);
      if (is_raw) {
        const uint32_t q = pos + __popc(m & ((1u << lane) - 1u));
        p.raw[q] = w[j];
        c = kMissBase | (q & (TQ_TILES_RING_WORDS - 1u));
      }
      pos += __popc(m);
      tk[j] = c;  // a group that does not exist keeps token 0
    }
    uint4* out = reinterpret_cast<uint4*>(p.tokens + (size_t)tile * 512u);
    out[lane] = make_uint4(tk[0] | (tk[1] << 16), tk[2] | (tk[3] << 16), tk[4] | (tk[5] << 16), tk[6] | (tk[7] << 16));
    out[32 + lane] = make_uint4(tk[8] | (tk[9] << 16), tk[10] | (tk[11] << 16), tk[12] | (tk[13] << 16), tk[14] | (tk[15] << 16));
  }
}

int sm_count_enc() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  return n;
}

}  // namespace

// Fills d_image (zeroed here; sized for the worst case of every group raw) on cuda_stream; the
// caller reads tile_raw and the counters at byte 64 of the image back after synchronising.
int tq_tiles_build_device(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols,
                          const float* d_row_scale, const float* d_row_zero, uint8_t* d_image, void* cuda_stream) {
  const tq_tiles_geometry geo = tq_tiles_layout(rows, cols);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // everything up to the raw words starts as zero: padding rows, read-ahead padding, counters, status
  if (int rc = tq_cuda_status((int)cudaMemsetAsync(d_image, 0, geo.off_raw, st), "device upload: clearing the image")) return rc;
  if (int rc = tq_cuda_status((int)cudaMemcpyAsync(d_image + geo.off_scale, d_row_scale, (size_t)rows * 4, cudaMemcpyDeviceToDevice, st),
                              "device upload: scales"))
    return rc;
  if (d_row_zero) {
    if (int rc = tq_cuda_status((int)cudaMemcpyAsync(d_image + geo.off_zero, d_row_zero, (size_t)rows * 4, cudaMemcpyDeviceToDevice, st),
                                "device upload: zero points"))
      return rc;
  }
  EncodeParams p{};
  p.levels = d_levels;
  p.map = dict->d_map;
  p.rows = rows;
  p.cols = cols;
  p.gpr = cols / 4;
  p.steps = geo.steps;
  p.n_tiles = (uint32_t)geo.n_tiles;
  p.tile_raw = reinterpret_cast<uint32_t*>(d_image + geo.off_tile_raw);
  p.tokens = reinterpret_cast<uint16_t*>(d_image + geo.off_tokens);
  p.raw = reinterpret_cast<uint32_t*>(d_image + geo.off_raw);
  p.counters = reinterpret_cast<unsigned long long*>(d_image + 64);
  const uint32_t grid = std::min<uint32_t>((p.n_tiles + 7u) / 8u, (uint32_t)sm_count_enc() * 8u);
  tiles_count_kernel<<<grid, 256, 0, st>>>(p);
  tiles_scan_kernel<<<1, 1024, 0, st>>>(p.tile_raw, p.n_tiles);
  tiles_fill_kernel<<<grid, 256, 0, st>>>(p);
  return tq_cuda_status((int)cudaGetLastError(), "device upload: encode kernels");
}
