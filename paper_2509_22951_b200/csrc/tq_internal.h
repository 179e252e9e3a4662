// Internal declarations shared by the host (tq_host.cpp) and device (tq_device.cu) halves of
// libtq.  Nothing here crosses the C ABI.
#pragma once

#include <cstdint>
#include <vector>

#include <vector_types.h>

#include "tq.h"

struct tq_dict {
  uint32_t K = 0;
  std::vector<uint8_t> entries;  // K x 4, rank order
  std::vector<uint64_t> counts;  // K
  // open-addressing lookup: 4-byte window -> code (0 = empty slot)
  uint32_t map_mask = 0;
  std::vector<uint32_t> map_key;
  std::vector<uint16_t> map_code;
  uint64_t n_windows = 0, n_distinct = 0;
};

// Slot of the device-side lookup from a 4-byte window to its code (open addressing, 2^18 slots,
// slot = (key * 0x9E3779B1) >> 14, linear probing, code 0 = empty): the host table's own map.
struct tq_map_slot {
  uint32_t key;
  uint32_t code;
};
constexpr uint32_t kMapSlots = 1u << 18;

struct tq_ddict {
  uint32_t K = 0;
  const tq_map_slot* d_map = nullptr;  // DEVICE: kMapSlots slots
  // DEVICE: K + 1 words indexed by code; word 0 is zero (token 0 = padding), word c holds entry
  // c - 1 with byte i of the window in bits 8i..8i+7
  const uint32_t* d_table = nullptr;
  std::vector<uint32_t> h_table;  // HOST copy of the same K + 1 words
};

// Row descriptor of the STREAM layout: where the row's token segment starts (in 16-byte units
// from the start of the token area) and how many uint16 slots it holds.
struct tq_rowseg {
  uint32_t chunk_off;
  uint32_t n_slots;
};

// What a kernel needs to know about one matrix in the TILES layout (all pointers DEVICE).
struct tq_tiles_desc {
  const uint4* tokens;       // n_tiles x 1 KB token tiles
  const uint32_t* raw;       // raw words in tile order (512-byte aligned, readable 16 KB past the end)
  const uint32_t* tile_raw;  // n_tiles + 1: index of each tile's first raw word
  const float* scale;        // rows
  const float* zero;         // rows (valid when has_zero)
  uint32_t* status;
  const void* x;             // bf16 [B][cols]
  float* y;                  // fp32 [B][rows]
  uint32_t rows, cols;
  uint32_t steps;            // tiles per row block = ceil(cols / 128)
  uint32_t row_blocks;       // ceil(rows / 16)
  uint32_t has_zero;
  uint32_t table_words;      // tokens are < table_words or the marker
  // scratch of the tcgen05 kernel: 512-byte header (per vector: output scale, scaled sum of the fixed-point
  // values) + one slice of digit planes per step (tq_wide_scratch_bytes); nullptr where it is not used
  uint8_t* xdig;
};

struct tq_dmat {
  tq_dmat_info info{};
  const tq_ddict* dict = nullptr;
  uint32_t* d_status = nullptr;        // DEVICE: status word
  const tq_rowseg* d_rowseg = nullptr; // DEVICE: rows entries
  const float* d_scale = nullptr;      // DEVICE: rows
  const float* d_zero = nullptr;       // DEVICE: rows
  const uint16_t* d_tokens = nullptr;  // DEVICE: token area, 256-byte aligned (STREAM layout)
  uint64_t token_chunks = 0;           // token area length in 16-byte units
  int has_zero = 0;
  // every level - zero point is an integer of magnitude <= 256, i.e. exact as bf16 (what the workspace
  // GEMM stores); false for zero points that are fractional or far outside the level range
  bool zero_bf16_exact = true;
  // PLANES layout
  const uint32_t* d_rawbase = nullptr; // DEVICE: rows + 1, index of each row's first raw word
  const uint16_t* d_rawidx = nullptr;  // DEVICE: rows x nidx_pad, markers before group 32*c of the row
  const uint16_t* d_codes = nullptr;   // DEVICE: rows x gpr_pad tokens
  const uint32_t* d_raw = nullptr;     // DEVICE: raw words
  uint32_t gpr_pad = 0, nidx_pad = 0;
  // TILES layout
  tq_tiles_desc tiles{};
  std::vector<uint32_t> rb_raw;  // HOST: row_blocks + 1, index of each row block's first raw word
};

// Host-side image of a matrix in the STREAM layout, ready for one cudaMemcpy.
struct tq_host_image {
  std::vector<uint8_t> blob;
  uint64_t off_status = 0, off_rowseg = 0, off_scale = 0, off_zero = 0, off_tokens = 0;
  uint64_t token_chunks = 0;
  uint64_t n_hits = 0, n_miss = 0;
};

struct tq_planes_image {
  std::vector<uint8_t> blob;
  uint64_t off_status = 0, off_rawbase = 0, off_rawidx = 0, off_scale = 0, off_zero = 0, off_codes = 0, off_raw = 0;
  uint32_t gpr_pad = 0, nidx_pad = 0;
  uint64_t n_hits = 0, n_miss = 0;
};

// Where the parts of a TQ_LAYOUT_TILES image lie (byte offsets from its 256-byte aligned start).
// One definition for the host builder and the device builder, whose images must be identical.
struct tq_tiles_geometry {
  uint32_t steps, row_blocks;
  uint64_t n_tiles, rows_pad;
  uint64_t off_status, off_scale, off_zero, off_tile_raw, off_tokens, off_raw;
  // behind the raw words (and their 16 KB of read-ahead padding): the scratch of the tcgen05 kernel for
  // calls on this matrix alone, sized for 32 vectors (512 + steps * 128 * 128 bytes)
  uint64_t off_xdig(uint64_t n_raw) const { return (off_raw + n_raw * 4 + 16384 + 1023) / 1024 * 1024; }
  uint64_t total(uint64_t n_raw) const { return off_xdig(n_raw) + (512 + (uint64_t)steps * 16384 + 1023) / 1024 * 1024; }
};
inline tq_tiles_geometry tq_tiles_layout(uint32_t rows, uint32_t cols) {
  auto up = [](uint64_t v, uint64_t a) { return (v + a - 1) / a * a; };
  tq_tiles_geometry g{};
  g.steps = (cols / 4 + 31u) / 32u;
  g.row_blocks = (rows + 15u) / 16u;
  g.n_tiles = (uint64_t)g.steps * g.row_blocks;
  g.rows_pad = (uint64_t)g.row_blocks * 16;
  g.off_status = 0;  // status word; bytes 64.. of this 256-byte header are scratch counters of the device builder
  g.off_scale = 256;
  g.off_zero = up(g.off_scale + g.rows_pad * 4, 256);
  g.off_tile_raw = up(g.off_zero + g.rows_pad * 4, 256);
  g.off_tokens = up(g.off_tile_raw + (g.n_tiles + 1 + 8) * 4, 1024);  // 8 entries read ahead by the kernels
  // 8 KB of token padding and 16 KB of raw padding: prefetches past the last tile stay inside the buffer
  g.off_raw = up(g.off_tokens + g.n_tiles * 1024 + 8192, 1024);
  return g;
}

struct tq_tiles_image {
  std::vector<uint8_t> blob;
  uint64_t off_status = 0, off_scale = 0, off_zero = 0, off_tile_raw = 0, off_tokens = 0, off_raw = 0;
  uint32_t steps = 0, row_blocks = 0;
  uint64_t n_hits = 0, n_miss = 0;  // of the paper's stream
  uint64_t n_raw = 0;               // raw words of the image: n_miss + the groups whose code is >= table_words
  std::vector<uint32_t> rb_raw;     // row_blocks + 1, index of each row block's first raw word
};

int tq_num_threads();

// True if level - zero is an integer of magnitude <= 256 for every level of the given kind and every
// zero point of the list (zero == nullptr: no zero points).
inline bool tq_zero_bf16_exact(const float* zero, uint32_t rows, bool levels_signed) {
  if (!zero) return true;
  const float lo = levels_signed ? -128.f : 0.f, hi = levels_signed ? 127.f : 255.f;
  for (uint32_t r = 0; r < rows; ++r) {
    const float z = zero[r];
    if (!(z == (float)(int)z) || hi - z > 256.f || z - lo > 256.f) return false;
  }
  return true;
}

// Maps a cudaError_t (passed as int) to TQ_OK / TQ_ERR_CUDA and records its text for tq_last_cuda_error.
int tq_cuda_status(int cuda_error, const char* what);

// Raises a kernel's limit of dynamic shared memory to `bytes` on the current device, once per device
// and kernel (the attribute belongs to the device the call is made on); safe to call from several
// host threads.  func: the kernel's host-side address.
int tq_ensure_dynamic_smem(const void* func, size_t bytes, const char* what);

// Validates the stream and computes the layout size; if img != nullptr also builds the image.
// K == 0xFFFFFFFF skips the code-range check (size query without a table).
int tq_build_stream_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                          uint32_t K, const float* row_scale, const float* row_zero,
                          uint64_t* device_bytes, tq_host_image* img);
// table: HOST, K + 1 words indexed by code (needed only when img != nullptr).
int tq_build_tiles_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                         uint32_t K, const uint32_t* table, const float* row_scale, const float* row_zero,
                         uint64_t* device_bytes, tq_tiles_image* img);
int tq_build_planes_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                          uint32_t K, const float* row_scale, const float* row_zero,
                          uint64_t* device_bytes, tq_planes_image* img);

// TILES layout entry points (tq_tiles.cu).  x: bf16 [B][cols], y: fp32 [B][rows], any B >= 1.
int tq_tiles_max_nb(const tq_dmat* m);
int tq_tiles_gemv(const tq_dmat* m, const void* x, int nb, float* y, void* cuda_stream);
int tq_tiles_decompress(const tq_dmat* m, uint8_t* d_codes, void* cuda_stream);
// bf16 (level - zero point) in whole tiles: row_blocks * 16 rows, row pitch steps * 128 columns
int tq_tiles_decode_bf16(const tq_dmat* m, void* d_out, void* cuda_stream);

// A set of TILES matrices bound to their operands, with the work split among the CTAs of one
// persistent launch (tq_tiles.cu).
// One split of (a subset of) a stack's matrices among the CTAs.
struct tq_stack_plan {
  const void* d_segs = nullptr;         // DEVICE: segments, grouped by CTA
  const uint32_t* d_cta_seg = nullptr;  // DEVICE: grid + 1 offsets into the segments
  uint32_t n_segs = 0, n_mats = 0;
  uint32_t xstride = 0;                 // words per digit column a whole row of its longest matrix needs
  // the split of the narrow kernel only: one 128-byte record per segment (segment + matrix descriptor) and
  // per CTA the record of its first segment; CTAs grid_used.. have no segment and are not launched
  const void* d_recs = nullptr;
  const void* d_firsts = nullptr;
  uint32_t grid_used = 0;
};

struct tq_stack {
  int n = 0, B = 0;
  int levels_signed = 0;
  bool zero_bf16_exact = true;  // of every matrix
  uint32_t grid = 0, table_words = 0;
  const uint32_t* d_table = nullptr;
  const tq_tiles_desc* d_descs = nullptr;  // DEVICE
  // [0] all matrices, split by tiles (decompress, bf16 decode); [1] those whose rows are short enough for
  // the kernel that keeps a whole row of activation digits in shared memory; [2] the others and [3] all
  // matrices, split into groups of whole row blocks for the tcgen05 kernel
  tq_stack_plan plan[4];
  bool run_narrow = false, run_wide_long = false, run_wide_all = false;  // kernels one tq_fused_gemv_stack call launches
};

// The tcgen05 fused decode + product for 1..32 vectors (tq_wide.cu): two launches on cuda_stream (digit
// planes of the activations into each matrix's scratch, then the fused kernel).  d_mats != nullptr: a
// stack (DEVICE descriptors, segments grouped by CTA); else the single matrix *one*.
uint64_t tq_wide_scratch_bytes(uint32_t steps, int nb);
constexpr uint32_t kWideGroupRowBlocks = 16;  // row blocks the tcgen05 kernel's CTA works on at a time: one per decoding warp
int tq_wide_launch(const tq_tiles_desc* d_mats, int n_mats, const void* d_segs, const uint32_t* d_cta_seg,
                   const tq_tiles_desc* one, const uint32_t* d_table, uint32_t table_words, int nb, bool levels_signed,
                   uint32_t grid, void* cuda_stream);

// Phase 2 of the workspace GEMM (tq_gemm_ws.cu), declared here for tq_fused_gemm_ws.
extern "C" int tq_gemm_bf16_ws(const tq_dmat* m, const void* d_X_bf16, int M, float* d_Y, const void* d_workspace,
                               void* cuda_stream);

// Device-side builder of the TILES image (tq_encode.cu).
int tq_tiles_build_device(const tq_ddict* dict, const uint8_t* d_levels, uint32_t rows, uint32_t cols,
                          const float* d_row_scale, const float* d_row_zero, uint8_t* d_image, void* cuda_stream);

// A host table from windows that are already ranked (tq_host.cpp; used by the device-side builder).
int tq_dict_from_ranked(const uint32_t* keys, const uint64_t* counts, uint32_t K, uint64_t n_windows,
                        uint64_t n_distinct, tq_dict** out);
