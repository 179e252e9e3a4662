// tq_build_dictionary_device: Listing 2's table from 8-bit levels that are on the GPU.
//
// The counting is the expensive part (one window per byte: 3.2 G windows for LLaMA-3.2-3B) and is
// done on the device; the ranking of the few survivors is done on the host with the same rule as
// tq_build_dictionary (count descending, then first occurrence), so both give the same table.
//   per matrix:  window keys (4 consecutive bytes, stride 1)  ->  radix sort  ->  run lengths
//                ->  (key, count) of every distinct window added into one hash table
//   then:        all counts sorted descending -> the count c* of rank top_k; the windows with
//                count >= c* are the candidates (every tie at c* included)
//                ->  one more pass over the windows finds each candidate's first position
//                ->  host: sort candidates by (count desc, first asc), keep top_k.
// The sort and the run-length encoding are CUB's (library routines for an offline step); the
// key, hash and selection kernels are this file's.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <cub/device/device_radix_sort.cuh>
#include <cub/device/device_run_length_encode.cuh>

#include "tq_internal.h"

namespace {

constexpr uint32_t kEmpty = 0xFFFFFFFFu;          // empty slot; the window 0xFFFFFFFF itself lives in the extra last slot
constexpr uint64_t kMaxCandidates = 1ull << 24;  // beyond this many ties at the cut the host builder is the tool

inline uint64_t up256(uint64_t v) { return (v + 255) / 256 * 256; }

// keys[i] = bytes i .. i+3 of the matrix, little endian, for i in [0, n - 3).
__global__ void window_keys_kernel(const uint8_t* __restrict__ levels, uint64_t n, uint32_t* __restrict__ keys) {
  const uint32_t* words = reinterpret_cast<const uint32_t*>(levels);
  const uint64_t n_words = n / 4;  // whole words
  for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; 4 * j + 3 < n; j += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t w0 = words[j];
    uint32_t w1 = 0;
    if (j + 1 < n_words) {
      w1 = words[j + 1];
    } else {
      for (uint64_t b = 4 * (j + 1); b < n; ++b) w1 |= (uint32_t)levels[b] << (8 * (b - 4 * (j + 1)));
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (4 * j + k + 3 < n) keys[4 * j + k] = __funnelshift_r(w0, w1, 8 * k);
  }
}

struct HashTable {
  uint32_t* key;    // slots + 1 entries (the last one belongs to the window 0xFFFFFFFF)
  uint32_t* count;  // slots + 1
  uint32_t mask;    // slots - 1
  uint32_t* overflow;
};

__device__ __forceinline__ uint32_t slot_of(uint32_t key, uint32_t mask) { return (key * 0x9E3779B1u) & mask; }

// (key, count) of one matrix's distinct windows into the table of all matrices.
__global__ void accumulate_kernel(const uint32_t* __restrict__ uniq, const uint32_t* __restrict__ cnt,
                                  const uint32_t* __restrict__ n_runs, HashTable t) {
  const uint32_t n = *n_runs;
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint32_t key = uniq[i];
    if (key == kEmpty) {
      atomicAdd(&t.count[t.mask + 1u], cnt[i]);
      t.key[t.mask + 1u] = key;
      continue;
    }
    uint32_t h = slot_of(key, t.mask);
    bool done = false;
    for (uint32_t probes = 0; probes <= t.mask; ++probes) {
      const uint32_t prev = atomicCAS(&t.key[h], kEmpty, key);
      if (prev == kEmpty || prev == key) {
        atomicAdd(&t.count[h], cnt[i]);
        done = true;
        break;
      }
      h = (h + 1u) & t.mask;
    }
    if (!done) atomicExch(t.overflow, 1u);
  }
}

// counts of all occupied slots, densely, for the sort that finds the cut.
__global__ void gather_counts_kernel(HashTable t, uint32_t* __restrict__ out, uint32_t* __restrict__ n_out) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= t.mask + 1u; i += gridDim.x * blockDim.x) {
    const uint32_t c = t.count[i];
    if (c) out[atomicAdd(n_out, 1u)] = c;
  }
}

// (key, count) of the slots with count >= cut.
__global__ void gather_candidates_kernel(HashTable t, uint32_t cut, uint32_t cap, uint32_t* __restrict__ ckey,
                                         uint32_t* __restrict__ ccount, uint32_t* __restrict__ n_out) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i <= t.mask + 1u; i += gridDim.x * blockDim.x) {
    const uint32_t c = t.count[i];
    if (c && c >= cut) {
      const uint32_t o = atomicAdd(n_out, 1u);
      if (o < cap) {
        ckey[o] = t.key[i];
        ccount[o] = c;
      }
    }
  }
}

// Small table from candidate key to candidate index.
__global__ void build_cand_map_kernel(const uint32_t* __restrict__ ckey, uint32_t n, uint32_t* mkey, uint32_t* midx,
                                      uint32_t mmask) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint32_t key = ckey[i];
    uint32_t h = slot_of(key, mmask);
    for (;;) {  // the map has at least twice as many slots as candidates
      const uint32_t prev = atomicCAS(&midx[h], kEmpty, i);
      if (prev == kEmpty) {
        mkey[h] = key;
        break;
      }
      h = (h + 1u) & mmask;
    }
  }
}

// first[c] = smallest global window position at which candidate c occurs.
__global__ void first_seen_kernel(const uint32_t* __restrict__ keys, uint64_t n_windows, uint32_t base,
                                  const uint32_t* __restrict__ mkey, const uint32_t* __restrict__ midx, uint32_t mmask,
                                  uint32_t* __restrict__ first) {
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_windows; i += (uint64_t)gridDim.x * blockDim.x) {
    const uint32_t key = keys[i];
    uint32_t h = slot_of(key, mmask);
    for (;;) {
      const uint32_t idx = midx[h];
      if (idx == kEmpty) break;
      if (mkey[h] == key) {
        const uint32_t g = base + (uint32_t)i;
        if (g < first[idx]) atomicMin(&first[idx], g);  // the plain read filters almost every atomic out
        break;
      }
      h = (h + 1u) & mmask;
    }
  }
}

struct Plan {
  uint64_t max_n = 0, total_windows = 0;
  uint32_t slots = 0;
  size_t cub_bytes = 0;
  uint64_t off_keys_a, off_keys_b, off_uniq, off_cnt, off_hkey, off_hcount, off_misc, off_cub, off_ckey, off_ccount, off_mkey,
      off_midx, off_first, total;
};

int make_plan(const uint64_t* n_elems, int n_mats, Plan* p) {
  for (int m = 0; m < n_mats; ++m) {
    p->max_n = std::max<uint64_t>(p->max_n, n_elems[m]);
    p->total_windows += n_elems[m] >= 4 ? n_elems[m] - 3 : 0;
  }
  if (p->total_windows >= (1ull << 32) || p->max_n >= (1ull << 31)) return TQ_ERR_UNSUPPORTED_SHAPE;
  uint64_t want = std::min<uint64_t>(std::max<uint64_t>(2 * p->total_windows, 1u << 16), 1ull << 28);
  uint32_t slots = 1u << 16;
  while (slots < want) slots <<= 1;
  p->slots = slots;
  size_t a = 0, b = 0;
  const int n_max = (int)std::max<uint64_t>(p->max_n, 1);
  cub::DeviceRadixSort::SortKeys(nullptr, a, (const uint32_t*)nullptr, (uint32_t*)nullptr, n_max);
  cub::DeviceRunLengthEncode::Encode(nullptr, b, (const uint32_t*)nullptr, (uint32_t*)nullptr, (uint32_t*)nullptr,
                                     (uint32_t*)nullptr, n_max);
  size_t c = 0;
  cub::DeviceRadixSort::SortKeysDescending(nullptr, c, (const uint32_t*)nullptr, (uint32_t*)nullptr, (int)std::min<uint64_t>((uint64_t)slots + 1, 1u << 30));
  p->cub_bytes = std::max(std::max(a, b), c);
  uint64_t o = 0;
  auto take = [&](uint64_t bytes) { uint64_t r = o; o += up256(bytes); return r; };
  const uint64_t per_mat = std::max<uint64_t>(p->max_n, (uint64_t)slots + 1) * 4;  // these buffers also serve the count sort
  p->off_keys_a = take(per_mat);
  p->off_keys_b = take(per_mat);
  p->off_uniq = take(p->max_n * 4);
  p->off_cnt = take(p->max_n * 4);
  p->off_hkey = take(((uint64_t)slots + 1) * 4);
  p->off_hcount = take(((uint64_t)slots + 1) * 4);
  p->off_misc = take(256);
  p->off_cub = take(p->cub_bytes);
  p->off_ckey = take(kMaxCandidates * 4);
  p->off_ccount = take(kMaxCandidates * 4);
  p->off_mkey = take(kMaxCandidates * 2 * 4);
  p->off_midx = take(kMaxCandidates * 2 * 4);
  p->off_first = take(kMaxCandidates * 4);
  p->total = o;
  return TQ_OK;
}

}  // namespace

extern "C" {

int tq_build_dictionary_device_size(const uint64_t* n_elems, int n_mats, uint64_t* workspace_bytes) {
  if (!n_elems || n_mats < 1 || !workspace_bytes) return TQ_ERR_INVALID_ARG;
  Plan p;
  if (int rc = make_plan(n_elems, n_mats, &p)) return rc;
  *workspace_bytes = p.total;
  return TQ_OK;
}

int tq_build_dictionary_device(const uint8_t* const* d_mats, const uint64_t* n_elems, int n_mats, uint32_t top_k,
                               void* d_workspace, uint64_t workspace_bytes, void* cuda_stream, tq_dict** out) {
  if (!d_mats || !n_elems || n_mats < 1 || !d_workspace || !out || ((uintptr_t)d_workspace & 255)) return TQ_ERR_INVALID_ARG;
  for (int m = 0; m < n_mats; ++m)
    if (n_elems[m] && (!d_mats[m] || ((uintptr_t)d_mats[m] & 3))) return TQ_ERR_INVALID_ARG;
  Plan p;
  if (int rc = make_plan(n_elems, n_mats, &p)) return rc;
  if (workspace_bytes < p.total) return TQ_ERR_BUFFER_TOO_SMALL;
  const uint32_t Kt = std::min<uint32_t>(top_k, TQ_MAX_ENTRIES);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  uint8_t* ws = static_cast<uint8_t*>(d_workspace);
  uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + p.off_keys_a);
  uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + p.off_keys_b);
  uint32_t* uniq = reinterpret_cast<uint32_t*>(ws + p.off_uniq);
  uint32_t* cnt = reinterpret_cast<uint32_t*>(ws + p.off_cnt);
  uint32_t* misc = reinterpret_cast<uint32_t*>(ws + p.off_misc);  // [0] runs, [1] overflow, [2] distinct, [3] candidates
  HashTable t{reinterpret_cast<uint32_t*>(ws + p.off_hkey), reinterpret_cast<uint32_t*>(ws + p.off_hcount), p.slots - 1u, misc + 1};
  auto ck = [](cudaError_t e, const char* what) { return tq_cuda_status((int)e, what); };

  if (int rc = ck(cudaMemsetAsync(t.key, 0xFF, ((size_t)p.slots + 1) * 4, st), "table build: clearing")) return rc;
  if (int rc = ck(cudaMemsetAsync(t.count, 0, ((size_t)p.slots + 1) * 4, st), "table build: clearing")) return rc;
  if (int rc = ck(cudaMemsetAsync(misc, 0, 256, st), "table build: clearing")) return rc;

  // ---- counts of every distinct window, matrix by matrix (windows never span two matrices) ----
  for (int m = 0; m < n_mats; ++m) {
    if (n_elems[m] < 4) continue;
    const uint64_t nw = n_elems[m] - 3;
    const uint32_t grid = (uint32_t)std::min<uint64_t>((n_elems[m] / 4 + 255) / 256, 148 * 16);
    window_keys_kernel<<<grid, 256, 0, st>>>(d_mats[m], n_elems[m], keys_a);
    size_t cb = p.cub_bytes;
    if (int rc = ck(cub::DeviceRadixSort::SortKeys(ws + p.off_cub, cb, keys_a, keys_b, (int)nw, 0, 32, st), "table build: sort")) return rc;
    cb = p.cub_bytes;
    if (int rc = ck(cub::DeviceRunLengthEncode::Encode(ws + p.off_cub, cb, keys_b, uniq, cnt, misc, (int)nw, st), "table build: run lengths"))
      return rc;
    accumulate_kernel<<<148 * 8, 256, 0, st>>>(uniq, cnt, misc, t);
  }
  // ---- the count of rank top_k ----
  gather_counts_kernel<<<148 * 8, 256, 0, st>>>(t, keys_a, misc + 2);
  uint32_t h_misc[4] = {0, 0, 0, 0};
  if (int rc = ck(cudaMemcpyAsync(h_misc, misc, 16, cudaMemcpyDeviceToHost, st), "table build")) return rc;
  if (int rc = ck(cudaStreamSynchronize(st), "table build")) return rc;
  if (h_misc[1]) return TQ_ERR_BUFFER_TOO_SMALL;  // more distinct windows than the hash table holds
  const uint32_t n_distinct = h_misc[2];
  uint32_t cut = 1;
  if (n_distinct > Kt && Kt > 0) {
    size_t cb = p.cub_bytes;
    if (int rc = ck(cub::DeviceRadixSort::SortKeysDescending(ws + p.off_cub, cb, keys_a, keys_b, (int)n_distinct, 0, 32, st), "table build: sort of counts"))
      return rc;
    if (int rc = ck(cudaMemcpyAsync(&cut, keys_b + (Kt - 1), 4, cudaMemcpyDeviceToHost, st), "table build")) return rc;
    if (int rc = ck(cudaStreamSynchronize(st), "table build")) return rc;
  }
  // ---- candidates and their first positions ----
  uint32_t* ckey = reinterpret_cast<uint32_t*>(ws + p.off_ckey);
  uint32_t* ccount = reinterpret_cast<uint32_t*>(ws + p.off_ccount);
  uint32_t* mkey = reinterpret_cast<uint32_t*>(ws + p.off_mkey);
  uint32_t* midx = reinterpret_cast<uint32_t*>(ws + p.off_midx);
  uint32_t* first = reinterpret_cast<uint32_t*>(ws + p.off_first);
  uint32_t n_cand = 0;
  if (Kt > 0 && n_distinct > 0) {
    gather_candidates_kernel<<<148 * 8, 256, 0, st>>>(t, cut, (uint32_t)kMaxCandidates, ckey, ccount, misc + 3);
    if (int rc = ck(cudaMemcpyAsync(&n_cand, misc + 3, 4, cudaMemcpyDeviceToHost, st), "table build")) return rc;
    if (int rc = ck(cudaStreamSynchronize(st), "table build")) return rc;
    if (n_cand > kMaxCandidates) return TQ_ERR_UNSUPPORTED_SHAPE;  // an enormous tie at the cut: use tq_build_dictionary
  }
  std::vector<uint32_t> hk(n_cand), hc(n_cand), hf(n_cand);
  if (n_cand) {
    uint32_t mslots = 1u << 4;
    while (mslots < 2 * n_cand + 2) mslots <<= 1;
    if (int rc = ck(cudaMemsetAsync(midx, 0xFF, (size_t)mslots * 4, st), "table build")) return rc;
    if (int rc = ck(cudaMemsetAsync(first, 0xFF, (size_t)n_cand * 4, st), "table build")) return rc;
    build_cand_map_kernel<<<(n_cand + 255) / 256, 256, 0, st>>>(ckey, n_cand, mkey, midx, mslots - 1u);
    uint64_t base = 0;
    for (int m = 0; m < n_mats; ++m) {
      if (n_elems[m] < 4) continue;
      const uint64_t nw = n_elems[m] - 3;
      const uint32_t grid = (uint32_t)std::min<uint64_t>((n_elems[m] / 4 + 255) / 256, 148 * 16);
      window_keys_kernel<<<grid, 256, 0, st>>>(d_mats[m], n_elems[m], keys_a);
      first_seen_kernel<<<148 * 16, 256, 0, st>>>(keys_a, nw, (uint32_t)base, mkey, midx, mslots - 1u, first);
      base += nw;
    }
    int rc = ck(cudaMemcpyAsync(hk.data(), ckey, (size_t)n_cand * 4, cudaMemcpyDeviceToHost, st), "table build");
    if (rc == TQ_OK) rc = ck(cudaMemcpyAsync(hc.data(), ccount, (size_t)n_cand * 4, cudaMemcpyDeviceToHost, st), "table build");
    if (rc == TQ_OK) rc = ck(cudaMemcpyAsync(hf.data(), first, (size_t)n_cand * 4, cudaMemcpyDeviceToHost, st), "table build");
    if (rc == TQ_OK) rc = ck(cudaStreamSynchronize(st), "table build");
    if (rc != TQ_OK) return rc;
  }
  // ---- host: rank the candidates exactly as tq_build_dictionary does ----
  std::vector<uint32_t> order(n_cand);
  for (uint32_t i = 0; i < n_cand; ++i) order[i] = i;
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return hc[a] != hc[b] ? hc[a] > hc[b] : hf[a] < hf[b]; });
  const uint32_t K = std::min<uint32_t>(n_cand, Kt);
  std::vector<uint32_t> rk(K);
  std::vector<uint64_t> rc64(K);
  for (uint32_t r = 0; r < K; ++r) {
    rk[r] = hk[order[r]];
    rc64[r] = hc[order[r]];
  }
  return tq_dict_from_ranked(rk.data(), rc64.data(), K, p.total_windows, n_distinct, out);
}

}  // extern "C"
