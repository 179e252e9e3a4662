// Host half of libtq: quantizers (Listing 1 and the per-row variant), the frequent-sequence
// table (Listing 2), the token-stream encoder (Listing 3) and the validation + row segmentation
// that tq_upload performs before the copy to the device.  Multithreaded with std::thread.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <new>
#include <thread>
#include <unordered_set>

#include "tq_internal.h"

namespace {

std::atomic<int> g_threads{0};

template <class F>
void parallel_run(int nt, F&& f) {
  if (nt <= 1) {
    f(0);
    return;
  }
  std::vector<std::thread> th;
  th.reserve(nt);
  for (int t = 0; t < nt; ++t) th.emplace_back([&f, t] { f(t); });
  for (auto& x : th) x.join();
}

inline uint32_t mix_bucket(uint32_t key) { return key * 0x9E3779B1u; }

inline uint32_t load_key(const uint8_t* p) {
  return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}

// Enumerates the windows with global index g in [g0, g1) in visiting order (matrix order, then
// position) and calls fn(key, g).  starts[m] is the global index of matrix m's first window.
template <class F>
void for_each_window(const uint8_t* const* mats, const std::vector<uint64_t>& starts, uint64_t g0,
                     uint64_t g1, F&& fn) {
  if (g0 >= g1) return;
  size_t m = std::upper_bound(starts.begin(), starts.end(), g0) - starts.begin() - 1;
  uint64_t g = g0;
  while (g < g1) {
    while (starts[m + 1] <= g) ++m;  // skip matrices without windows
    const uint8_t* p = mats[m];
    uint64_t i = g - starts[m];
    uint64_t iend = std::min(g1, starts[m + 1]) - starts[m];
    uint32_t key = load_key(p + i);
    fn(key, g);
    ++g;
    for (++i; i < iend; ++i, ++g) {
      key = (key >> 8) | ((uint32_t)p[i + 3] << 24);
      fn(key, g);
    }
  }
}

void radix_sort_u32(uint32_t* a, uint32_t* tmp, size_t n) {
  if (n < 512) {
    std::sort(a, a + n);
    return;
  }
  constexpr int BITS = 11, R = 1 << BITS;
  size_t h0[R] = {0}, h1[R] = {0}, h2[R] = {0};
  for (size_t i = 0; i < n; ++i) {
    uint32_t v = a[i];
    h0[v & (R - 1)]++;
    h1[(v >> BITS) & (R - 1)]++;
    h2[v >> (2 * BITS)]++;
  }
  size_t s0 = 0, s1 = 0, s2 = 0;
  for (int i = 0; i < R; ++i) {
    size_t c0 = h0[i], c1 = h1[i], c2 = h2[i];
    h0[i] = s0; h1[i] = s1; h2[i] = s2;
    s0 += c0; s1 += c1; s2 += c2;
  }
  for (size_t i = 0; i < n; ++i) { uint32_t v = a[i]; tmp[h0[v & (R - 1)]++] = v; }
  for (size_t i = 0; i < n; ++i) { uint32_t v = tmp[i]; a[h1[(v >> BITS) & (R - 1)]++] = v; }
  for (size_t i = 0; i < n; ++i) { uint32_t v = a[i]; tmp[h2[v >> (2 * BITS)]++] = v; }
  std::memcpy(a, tmp, n * sizeof(uint32_t));
}

struct Cand {
  uint32_t key;
  uint64_t count;
  uint64_t first;
};

void finish_dict(tq_dict* d) {
  d->map_mask = (1u << 18) - 1;
  d->map_key.assign(d->map_mask + 1, 0);
  d->map_code.assign(d->map_mask + 1, 0);
  for (uint32_t r = 0; r < d->K; ++r) {
    uint32_t key = load_key(&d->entries[4 * (size_t)r]);
    uint32_t h = (key * 0x9E3779B1u) >> 14;
    bool dup = false;
    while (d->map_code[h] != 0) {
      if (d->map_key[h] == key) { dup = true; break; }
      h = (h + 1) & d->map_mask;
    }
    if (dup) continue;  // first (lowest) code wins, as a dict lookup would
    d->map_key[h] = key;
    d->map_code[h] = (uint16_t)(r + 1);
  }
}

inline uint16_t dict_find(const tq_dict* d, uint32_t key) {
  uint32_t h = (key * 0x9E3779B1u) >> 14;
  while (true) {
    uint16_t c = d->map_code[h];
    if (c == 0) return 0;
    if (d->map_key[h] == key) return c;
    h = (h + 1) & d->map_mask;
  }
}

}  // namespace

int tq_num_threads() {
  int n = g_threads.load();
  if (n <= 0) {
    n = (int)std::thread::hardware_concurrency();
    if (n <= 0) n = 1;
    if (n > 64) n = 64;
  }
  return n;
}

// A table from windows already ranked (keys little endian: byte i of the window in bits 8i..8i+7).
int tq_dict_from_ranked(const uint32_t* keys, const uint64_t* counts, uint32_t K, uint64_t n_windows,
                        uint64_t n_distinct, tq_dict** out) {
  if (!out || (K && (!keys || !counts)) || K > TQ_MAX_ENTRIES) return TQ_ERR_INVALID_ARG;
  tq_dict* d = new (std::nothrow) tq_dict();
  if (!d) return TQ_ERR_NOMEM;
  try {
    d->K = K;
    d->n_windows = n_windows;
    d->n_distinct = n_distinct;
    d->entries.resize(4 * (size_t)K);
    d->counts.assign(counts, counts + K);
    for (uint32_t r = 0; r < K; ++r) {
      d->entries[4 * (size_t)r + 0] = (uint8_t)keys[r];
      d->entries[4 * (size_t)r + 1] = (uint8_t)(keys[r] >> 8);
      d->entries[4 * (size_t)r + 2] = (uint8_t)(keys[r] >> 16);
      d->entries[4 * (size_t)r + 3] = (uint8_t)(keys[r] >> 24);
    }
    finish_dict(d);
  } catch (const std::bad_alloc&) {
    delete d;
    return TQ_ERR_NOMEM;
  }
  *out = d;
  return TQ_OK;
}

extern "C" {

const char* tq_strerror(int s) {
  switch (s) {
    case TQ_OK: return "ok";
    case TQ_ERR_INVALID_ARG: return "invalid argument";
    case TQ_ERR_CORRUPT_STREAM: return "corrupt token stream";
    case TQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case TQ_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case TQ_ERR_CUDA: return "CUDA error";
    case TQ_ERR_TIMEOUT: return "bounded wait expired";
    case TQ_ERR_NOMEM: return "out of host memory";
    default: return "unknown status";
  }
}

int tq_set_num_threads(int n) {
  g_threads.store(n > 0 ? std::min(n, 256) : 0);
  return tq_num_threads();
}

int tq_quantize_tensor_bits(const float* x, uint64_t n, int bits, uint8_t* q, float* scale, float* zero) {
  if (!x || !q || !scale || !zero || n == 0 || bits < 1 || bits > 8) return TQ_ERR_INVALID_ARG;
  const float maxq = (float)((1 << bits) - 1);
  float lo = x[0], hi = x[0];
  for (uint64_t i = 1; i < n; ++i) {
    lo = std::min(lo, x[i]);
    hi = std::max(hi, x[i]);
  }
  const float s = (hi - lo) / maxq;
  if (!(s > 0.0f)) return TQ_ERR_INVALID_ARG;
  const float z = std::nearbyintf(-lo / s);
  const int nt = (int)std::min<uint64_t>(tq_num_threads(), n / 65536 + 1);
  parallel_run(nt, [&](int t) {
    uint64_t a = n * t / nt, b = n * (t + 1) / nt;
    for (uint64_t i = a; i < b; ++i) {
      float v = std::nearbyintf(x[i] / s) + z;
      v = v < 0.0f ? 0.0f : (v > maxq ? maxq : v);
      q[i] = (uint8_t)v;
    }
  });
  *scale = s;
  *zero = z;
  return TQ_OK;
}

int tq_quantize_tensor(const float* x, uint64_t n, uint8_t* q, float* scale, float* zero) {
  return tq_quantize_tensor_bits(x, n, 8, q, scale, zero);
}

int tq_quantize_rows(const float* w, uint32_t rows, uint32_t cols, int8_t* q, float* scale) {
  if (!w || !q || !scale || rows == 0 || cols == 0) return TQ_ERR_INVALID_ARG;
  const int nt = (int)std::min<uint64_t>(tq_num_threads(), (uint64_t)rows * cols / 65536 + 1);
  parallel_run(nt, [&](int t) {
    uint32_t r0 = (uint32_t)((uint64_t)rows * t / nt), r1 = (uint32_t)((uint64_t)rows * (t + 1) / nt);
    for (uint32_t r = r0; r < r1; ++r) {
      const float* wr = w + (uint64_t)r * cols;
      int8_t* qr = q + (uint64_t)r * cols;
      float amax = 0.0f;
      for (uint32_t c = 0; c < cols; ++c) amax = std::max(amax, std::fabs(wr[c]));
      const float s = amax > 0.0f ? amax / 127.0f : 1.0f;
      scale[r] = s;
      for (uint32_t c = 0; c < cols; ++c) {
        float v = std::nearbyintf(wr[c] / s);
        v = v < -127.0f ? -127.0f : (v > 127.0f ? 127.0f : v);
        qr[c] = (int8_t)v;
      }
    }
  });
  return TQ_OK;
}

int tq_dict_from_entries(const uint8_t* entries, uint32_t K, tq_dict** out) {
  if (!out || (K && !entries) || K > TQ_MAX_ENTRIES) return TQ_ERR_INVALID_ARG;
  tq_dict* d = new (std::nothrow) tq_dict();
  if (!d) return TQ_ERR_NOMEM;
  d->K = K;
  d->entries.assign(entries, entries + 4 * (size_t)K);
  d->counts.assign(K, 0);
  finish_dict(d);
  *out = d;
  return TQ_OK;
}

int tq_build_dictionary(const uint8_t* const* mats, const uint64_t* n_elems, int n_mats,
                        uint32_t top_k, tq_dict** out) {
  if (!out || n_mats < 0 || (n_mats > 0 && (!mats || !n_elems))) return TQ_ERR_INVALID_ARG;
  for (int m = 0; m < n_mats; ++m)
    if (n_elems[m] && !mats[m]) return TQ_ERR_INVALID_ARG;
  const uint32_t Kt = std::min<uint32_t>(top_k, TQ_MAX_ENTRIES);

  std::vector<uint64_t> starts(n_mats + 1, 0);
  for (int m = 0; m < n_mats; ++m) starts[m + 1] = starts[m] + (n_elems[m] >= 4 ? n_elems[m] - 3 : 0);
  const uint64_t N = starts[n_mats];
  if (N >= (1ull << 32)) return TQ_ERR_UNSUPPORTED_SHAPE;

  tq_dict* d = new (std::nothrow) tq_dict();
  if (!d) return TQ_ERR_NOMEM;
  d->n_windows = N;
  std::vector<Cand> chosen;

  try {
    if (N > 0 && Kt > 0) {
      const int T = (int)std::min<uint64_t>(tq_num_threads(), N / (1u << 18) + 1);
      int log2P = 0;
      while (log2P < 12 && (N >> (log2P + 19)) > 0) ++log2P;  // ~512 Ki keys per bucket
      const uint32_t P = 1u << log2P;
      auto bucket_of = [log2P](uint32_t key) -> uint32_t {
        return log2P ? (mix_bucket(key) >> (32 - log2P)) : 0u;
      };
      auto slice = [&](int t) { return N * (uint64_t)t / (uint64_t)T; };

      // --- scatter the window keys into hash buckets (stable within a bucket) ---
      std::vector<uint32_t> keys(N);
      std::vector<uint64_t> cnt((size_t)T * P, 0);
      parallel_run(T, [&](int t) {
        uint64_t* c = &cnt[(size_t)t * P];
        for_each_window(mats, starts, slice(t), slice(t + 1), [&](uint32_t key, uint64_t) { c[bucket_of(key)]++; });
      });
      std::vector<uint64_t> bstart(P + 1, 0);
      {
        uint64_t run = 0;
        for (uint32_t b = 0; b < P; ++b) {
          bstart[b] = run;
          for (int t = 0; t < T; ++t) {
            uint64_t c = cnt[(size_t)t * P + b];
            cnt[(size_t)t * P + b] = run;
            run += c;
          }
        }
        bstart[P] = run;
      }
      parallel_run(T, [&](int t) {
        uint64_t* o = &cnt[(size_t)t * P];
        for_each_window(mats, starts, slice(t), slice(t + 1), [&](uint32_t key, uint64_t) { keys[o[bucket_of(key)]++] = key; });
      });

      // --- sort every bucket, histogram the run lengths ---
      uint64_t max_bucket = 0;
      for (uint32_t b = 0; b < P; ++b) max_bucket = std::max(max_bucket, bstart[b + 1] - bstart[b]);
      constexpr uint32_t HB = 1u << 16;
      std::vector<std::vector<uint64_t>> hist(T, std::vector<uint64_t>(HB, 0));
      std::vector<std::vector<uint64_t>> big(T);
      std::atomic<uint32_t> next{0};
      parallel_run(T, [&](int t) {
        std::vector<uint32_t> tmp(max_bucket);
        for (;;) {
          uint32_t b = next.fetch_add(1);
          if (b >= P) break;
          uint32_t* a = keys.data() + bstart[b];
          size_t n = bstart[b + 1] - bstart[b];
          radix_sort_u32(a, tmp.data(), n);
          for (size_t i = 0; i < n;) {
            size_t j = i + 1;
            while (j < n && a[j] == a[i]) ++j;
            uint64_t c = j - i;
            if (c < HB) hist[t][c]++; else big[t].push_back(c);
            i = j;
          }
        }
      });
      std::vector<uint64_t> H(HB, 0), B;
      for (int t = 0; t < T; ++t) {
        for (uint32_t i = 0; i < HB; ++i) H[i] += hist[t][i];
        B.insert(B.end(), big[t].begin(), big[t].end());
      }
      std::sort(B.begin(), B.end(), std::greater<uint64_t>());
      uint64_t distinct = B.size();
      for (uint32_t i = 1; i < HB; ++i) distinct += H[i];
      d->n_distinct = distinct;

      // --- the count of the last rank that makes the cut, and how many lie above it ---
      uint64_t cstar = 1, n_above = 0, n_tied = 0;
      if (distinct <= Kt) {
        cstar = 0;  // everything is kept
        n_above = distinct;
      } else {
        uint64_t cum = 0;
        bool found = false;
        for (size_t i = 0; i < B.size() && !found;) {
          size_t j = i;
          while (j < B.size() && B[j] == B[i]) ++j;
          if (cum + (j - i) >= Kt) { cstar = B[i]; n_above = cum; n_tied = j - i; found = true; }
          cum += j - i;
          i = j;
        }
        for (uint32_t c = HB - 1; c >= 1 && !found; --c) {
          if (H[c] == 0) continue;
          if (cum + H[c] >= Kt) { cstar = c; n_above = cum; n_tied = H[c]; found = true; }
          cum += H[c];
        }
      }
      // Above this many windows sharing the cut-off count, the first-seen ones are found by an
      // in-order walk instead of a hash map over all of them (TQ_TIE_LIMIT overrides, for tests).
      uint64_t TIE_LIMIT = 1ull << 25;
      if (const char* e = std::getenv("TQ_TIE_LIMIT")) TIE_LIMIT = std::strtoull(e, nullptr, 10);
      const bool ties_in_map = n_tied <= TIE_LIMIT;
      const uint64_t min_count = ties_in_map ? std::max<uint64_t>(cstar, 1) : cstar + 1;

      // --- collect the candidates (count >= min_count) ---
      std::vector<std::vector<Cand>> part(T);
      next.store(0);
      parallel_run(T, [&](int t) {
        for (;;) {
          uint32_t b = next.fetch_add(1);
          if (b >= P) break;
          const uint32_t* a = keys.data() + bstart[b];
          size_t n = bstart[b + 1] - bstart[b];
          for (size_t i = 0; i < n;) {
            size_t j = i + 1;
            while (j < n && a[j] == a[i]) ++j;
            if (j - i >= min_count) part[t].push_back({a[i], (uint64_t)(j - i), ~0ull});
            i = j;
          }
        }
      });
      std::vector<Cand> cand;
      for (auto& p : part) cand.insert(cand.end(), p.begin(), p.end());

      // --- first occurrence of every candidate: one parallel pass over the windows ---
      uint32_t mbits = 4;
      while ((1ull << mbits) < 2 * cand.size() + 2) ++mbits;
      const uint64_t msize = 1ull << mbits;
      std::vector<uint32_t> mkey(msize, 0);
      std::vector<uint32_t> midx(msize, 0xFFFFFFFFu);
      auto mhash = [mbits](uint32_t key) -> uint64_t {
        return (uint64_t)(key * 0x9E3779B1u) >> (32 - mbits);
      };
      for (size_t i = 0; i < cand.size(); ++i) {
        uint64_t h = mhash(cand[i].key) & (msize - 1);
        while (midx[h] != 0xFFFFFFFFu) h = (h + 1) & (msize - 1);
        mkey[h] = cand[i].key;
        midx[h] = (uint32_t)i;
      }
      std::vector<uint64_t> first(cand.size() + 1, ~0ull);
      parallel_run(T, [&](int t) {
        for_each_window(mats, starts, slice(t), slice(t + 1), [&](uint32_t key, uint64_t g) {
          uint64_t h = mhash(key) & (msize - 1);
          while (midx[h] != 0xFFFFFFFFu) {
            if (mkey[h] == key) {
              uint64_t* f = &first[midx[h]];
              uint64_t cur = __atomic_load_n(f, __ATOMIC_RELAXED);
              while (g < cur && !__atomic_compare_exchange_n(f, &cur, g, false, __ATOMIC_RELAXED, __ATOMIC_RELAXED)) {}
              return;
            }
            h = (h + 1) & (msize - 1);
          }
        });
      });
      for (size_t i = 0; i < cand.size(); ++i) cand[i].first = first[i];

      if (!ties_in_map) {
        // Very many windows share the cut-off count: take the earliest-seen ones by walking the
        // windows in order; membership is decided by counting the key's run in its sorted bucket.
        uint64_t quota = Kt - n_above;
        std::unordered_set<uint32_t> seen;
        for_each_window(mats, starts, 0, N, [&](uint32_t key, uint64_t g) {
          if (quota == 0) return;
          uint32_t b = bucket_of(key);
          const uint32_t* a = keys.data() + bstart[b];
          const uint32_t* e = keys.data() + bstart[b + 1];
          auto lo = std::lower_bound(a, e, key);
          auto hi = std::upper_bound(lo, e, key);
          if ((uint64_t)(hi - lo) != cstar) return;
          if (!seen.insert(key).second) return;
          cand.push_back({key, cstar, g});
          --quota;
        });
      }
      std::sort(cand.begin(), cand.end(), [](const Cand& a, const Cand& b) {
        return a.count != b.count ? a.count > b.count : a.first < b.first;
      });
      if (cand.size() > Kt) cand.resize(Kt);
      chosen.swap(cand);
    }
  } catch (const std::bad_alloc&) {
    delete d;
    return TQ_ERR_NOMEM;
  }

  d->K = (uint32_t)chosen.size();
  d->entries.resize(4 * (size_t)d->K);
  d->counts.resize(d->K);
  for (uint32_t r = 0; r < d->K; ++r) {
    uint32_t key = chosen[r].key;
    d->entries[4 * (size_t)r + 0] = (uint8_t)key;
    d->entries[4 * (size_t)r + 1] = (uint8_t)(key >> 8);
    d->entries[4 * (size_t)r + 2] = (uint8_t)(key >> 16);
    d->entries[4 * (size_t)r + 3] = (uint8_t)(key >> 24);
    d->counts[r] = chosen[r].count;
  }
  finish_dict(d);
  *out = d;
  return TQ_OK;
}

int tq_dict_entries(const tq_dict* d, uint32_t* K, const uint8_t** entries, const uint64_t** counts) {
  if (!d || !K || !entries) return TQ_ERR_INVALID_ARG;
  *K = d->K;
  *entries = d->entries.data();
  if (counts) *counts = d->counts.data();
  return TQ_OK;
}

void tq_dict_free(tq_dict* d) { delete d; }

int tq_encode(const tq_dict* d, const uint8_t* codes, uint64_t n, uint16_t* out, uint64_t out_cap,
              uint64_t* out_len, uint64_t* n_hits, uint64_t* n_miss) {
  if (!d || (n && !codes) || !out_len) return TQ_ERR_INVALID_ARG;
  const uint64_t nb = n / 4, r = n % 4;
  const int T = (int)std::min<uint64_t>(tq_num_threads(), nb / (1u << 16) + 1);
  std::vector<uint64_t> miss(T + 1, 0);
  auto blk = [&](int t) { return nb * (uint64_t)t / (uint64_t)T; };
  parallel_run(T, [&](int t) {
    uint64_t m = 0;
    for (uint64_t b = blk(t); b < blk(t + 1); ++b) m += dict_find(d, load_key(codes + 4 * b)) == 0;
    miss[t + 1] = m;
  });
  for (int t = 0; t < T; ++t) miss[t + 1] += miss[t];
  const uint64_t M = miss[T], H = nb - M;
  const uint64_t len = H + 5 * M + (r ? 1 + r : 0);
  *out_len = len;
  if (n_hits) *n_hits = H;
  if (n_miss) *n_miss = M;
  if (!out) return TQ_OK;
  if (out_cap < len) return TQ_ERR_BUFFER_TOO_SMALL;
  parallel_run(T, [&](int t) {
    uint64_t b0 = blk(t);
    uint16_t* o = out + b0 + 4 * miss[t];
    for (uint64_t b = b0; b < blk(t + 1); ++b) {
      const uint8_t* p = codes + 4 * b;
      uint16_t c = dict_find(d, load_key(p));
      if (c) {
        *o++ = c;
      } else {
        o[0] = TQ_ESCAPE; o[1] = p[0]; o[2] = p[1]; o[3] = p[2]; o[4] = p[3];
        o += 5;
      }
    }
  });
  if (r) {
    uint16_t* o = out + H + 5 * M;
    *o++ = TQ_ESCAPE;
    for (uint64_t j = 0; j < r; ++j) *o++ = codes[4 * nb + j];
  }
  return TQ_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Validation and row segmentation of a token stream (the host part of tq_upload).
//
// A slot is RAW exactly when one of the 4 slots before it holds the marker: raw slots carry bytes
// (<= 255) and codes stop at 65534, so in a well-formed stream the marker value never appears
// anywhere but at a marker.  That makes the classification local, so the stream can be checked in
// parallel pieces; the checks below (raw slots <= 255, codes in 1..K, 4 slots after each marker,
// rows*cols/4 groups in total) are together equivalent to Listing 4's sequential walk succeeding.
// ---------------------------------------------------------------------------------------------
namespace {
inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }
}  // namespace

// Validates the stream and finds where every row's tokens start.
static int scan_stream(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols, uint32_t K,
                       std::vector<uint64_t>& row_start, uint64_t& H, uint64_t& M) {
  if (!stream || rows == 0 || cols == 0) return TQ_ERR_INVALID_ARG;
  if (cols % 4 != 0) return TQ_ERR_UNSUPPORTED_SHAPE;
  const uint64_t bpr = cols / 4, nb = (uint64_t)rows * bpr;
  if (stream_len < nb || stream_len > 5 * nb) return TQ_ERR_CORRUPT_STREAM;

  const int T = (int)std::min<uint64_t>(tq_num_threads(), stream_len / (1u << 18) + 1);
  auto cut = [&](int t) { return stream_len * (uint64_t)t / (uint64_t)T; };
  auto raw_left_at = [&](uint64_t p) -> uint32_t {
    for (uint32_t k = 1; k <= 4 && k <= p; ++k)
      if (stream[p - k] == TQ_ESCAPE) return 5 - k;
    return 0;
  };
  std::vector<uint64_t> hits(T, 0), miss(T, 0);
  std::atomic<int> bad{0};
  parallel_run(T, [&](int t) {
    uint64_t p = cut(t), e = cut(t + 1), h = 0, m = 0;
    uint32_t raw = raw_left_at(p);
    for (; p < e; ++p) {
      const uint16_t v = stream[p];
      if (raw) {
        if (v > 255) { bad.store(1); return; }
        --raw;
      } else if (v == TQ_ESCAPE) {
        if (p + 4 >= stream_len) { bad.store(1); return; }  // 4 raw slots must follow
        ++m;
        raw = 4;
      } else {
        if (v == 0 || (K != 0xFFFFFFFFu && v > K)) { bad.store(1); return; }
        ++h;
      }
    }
    hits[t] = h;
    miss[t] = m;
  });
  if (bad.load()) return TQ_ERR_CORRUPT_STREAM;
  H = 0;
  M = 0;
  std::vector<uint64_t> first_block(T + 1, 0);
  for (int t = 0; t < T; ++t) {
    H += hits[t];
    M += miss[t];
    first_block[t + 1] = first_block[t] + hits[t] + miss[t];
  }
  if (H + M != nb || H + 5 * M != stream_len) return TQ_ERR_CORRUPT_STREAM;

  row_start.assign((size_t)rows + 1, 0);
  row_start[rows] = stream_len;
  parallel_run(T, [&](int t) {
    uint64_t p = cut(t), e = cut(t + 1), blk = first_block[t];
    uint32_t raw = raw_left_at(p);
    uint64_t next_row_blk = (blk + bpr - 1) / bpr * bpr;
    for (; p < e; ++p) {
      if (raw) { --raw; continue; }
      if (blk == next_row_blk) {
        row_start[blk / bpr] = p;
        next_row_blk += bpr;
      }
      ++blk;
      if (stream[p] == TQ_ESCAPE) raw = 4;
    }
  });
  return TQ_OK;
}

int tq_build_stream_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                          uint32_t K, const float* row_scale, const float* row_zero,
                          uint64_t* device_bytes, tq_host_image* img) {
  std::vector<uint64_t> row_start;
  uint64_t H = 0, M = 0;
  int rc = scan_stream(stream, stream_len, rows, cols, K, row_start, H, M);
  if (rc != TQ_OK) return rc;

  std::vector<uint64_t> chunk_off((size_t)rows + 1, 0);
  for (uint32_t r = 0; r < rows; ++r) chunk_off[r + 1] = chunk_off[r] + (row_start[r + 1] - row_start[r] + 7) / 8;
  const uint64_t token_chunks = chunk_off[rows];
  if (token_chunks >= (1ull << 32)) return TQ_ERR_UNSUPPORTED_SHAPE;

  const uint64_t off_status = 0;
  const uint64_t off_rowseg = 256;
  const uint64_t off_scale = align_up(off_rowseg + (uint64_t)rows * sizeof(tq_rowseg), 256);
  const uint64_t off_zero = align_up(off_scale + (uint64_t)rows * 4, 256);
  const uint64_t off_tokens = align_up(off_zero + (uint64_t)rows * 4, 256);
  const uint64_t total = align_up(off_tokens + token_chunks * 16 + 256, 256);
  if (device_bytes) *device_bytes = total;
  if (!img) return TQ_OK;
  if (!row_scale) return TQ_ERR_INVALID_ARG;

  try {
    img->blob.assign(total, 0);
  } catch (const std::bad_alloc&) {
    return TQ_ERR_NOMEM;
  }
  img->off_status = off_status;
  img->off_rowseg = off_rowseg;
  img->off_scale = off_scale;
  img->off_zero = off_zero;
  img->off_tokens = off_tokens;
  img->token_chunks = token_chunks;
  img->n_hits = H;
  img->n_miss = M;
  uint8_t* base = img->blob.data();
  std::memcpy(base + off_scale, row_scale, (size_t)rows * 4);
  if (row_zero) std::memcpy(base + off_zero, row_zero, (size_t)rows * 4);
  tq_rowseg* seg = reinterpret_cast<tq_rowseg*>(base + off_rowseg);
  uint16_t* tok = reinterpret_cast<uint16_t*>(base + off_tokens);
  const int T2 = (int)std::min<uint64_t>(tq_num_threads(), stream_len / (1u << 18) + 1);
  parallel_run(T2, [&](int t) {
    uint32_t r0 = (uint32_t)((uint64_t)rows * t / T2), r1 = (uint32_t)((uint64_t)rows * (t + 1) / T2);
    for (uint32_t r = r0; r < r1; ++r) {
      const uint64_t n = row_start[r + 1] - row_start[r];
      seg[r].chunk_off = (uint32_t)chunk_off[r];
      seg[r].n_slots = (uint32_t)n;
      std::memcpy(tok + chunk_off[r] * 8, stream + row_start[r], n * 2);
    }
  });
  return TQ_OK;
}

// ---------------------------------------------------------------------------------------------
// PLANES layout: a lossless re-tiling of the same tokens.  Every group keeps its 16-bit token in a
// fixed-stride code plane (row-major, row stride padded to a multiple of 32 groups with token 0,
// which decodes to four zero bytes); the 4 raw bytes that follow a marker move, packed into one
// 32-bit word, to a compact raw plane in row-major group order.  raw_base[r] is the index of row
// r's first raw word; raw_idx[r][c] counts the row's markers before group 32*c.
// ---------------------------------------------------------------------------------------------
int tq_build_planes_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                          uint32_t K, const float* row_scale, const float* row_zero,
                          uint64_t* device_bytes, tq_planes_image* img) {
  std::vector<uint64_t> row_start;
  uint64_t H = 0, M = 0;
  int rc = scan_stream(stream, stream_len, rows, cols, K, row_start, H, M);
  if (rc != TQ_OK) return rc;
  if (M >= (1ull << 32)) return TQ_ERR_UNSUPPORTED_SHAPE;

  const uint32_t gpr = cols / 4;
  const uint32_t gpr_pad = (gpr + 31u) / 32u * 32u;
  const uint32_t nidx = gpr_pad / 32u + 1u;
  const uint32_t nidx_pad = (nidx + 1u) & ~1u;

  const uint64_t off_status = 0;
  const uint64_t off_rawbase = 256;
  const uint64_t off_rawidx = align_up(off_rawbase + ((uint64_t)rows + 1) * 4, 256);
  const uint64_t off_scale = align_up(off_rawidx + (uint64_t)rows * nidx_pad * 2, 256);
  const uint64_t off_zero = align_up(off_scale + (uint64_t)rows * 4, 256);
  const uint64_t off_codes = align_up(off_zero + (uint64_t)rows * 4, 256);
  const uint64_t off_raw = align_up(off_codes + (uint64_t)rows * gpr_pad * 2 + 256, 256);
  const uint64_t total = align_up(off_raw + M * 4 + 256, 256);
  if (device_bytes) *device_bytes = total;
  if (!img) return TQ_OK;
  if (!row_scale) return TQ_ERR_INVALID_ARG;
  try {
    img->blob.assign(total, 0);
  } catch (const std::bad_alloc&) {
    return TQ_ERR_NOMEM;
  }
  img->off_status = off_status;
  img->off_rawbase = off_rawbase;
  img->off_rawidx = off_rawidx;
  img->off_scale = off_scale;
  img->off_zero = off_zero;
  img->off_codes = off_codes;
  img->off_raw = off_raw;
  img->gpr_pad = gpr_pad;
  img->nidx_pad = nidx_pad;
  img->n_hits = H;
  img->n_miss = M;
  uint8_t* base = img->blob.data();
  std::memcpy(base + off_scale, row_scale, (size_t)rows * 4);
  if (row_zero) std::memcpy(base + off_zero, row_zero, (size_t)rows * 4);
  uint32_t* rawbase = reinterpret_cast<uint32_t*>(base + off_rawbase);
  uint16_t* rawidx = reinterpret_cast<uint16_t*>(base + off_rawidx);
  uint16_t* codes = reinterpret_cast<uint16_t*>(base + off_codes);
  uint32_t* raw = reinterpret_cast<uint32_t*>(base + off_raw);

  // markers per row: a row with h coded groups and m escaped ones occupies h + 5m slots
  for (uint32_t r = 0; r < rows; ++r) {
    const uint64_t n = row_start[r + 1] - row_start[r];
    rawbase[r + 1] = rawbase[r] + (uint32_t)((n - gpr) / 4);
  }
  const int T = (int)std::min<uint64_t>(tq_num_threads(), stream_len / (1u << 18) + 1);
  parallel_run(T, [&](int t) {
    uint32_t r0 = (uint32_t)((uint64_t)rows * t / T), r1 = (uint32_t)((uint64_t)rows * (t + 1) / T);
    for (uint32_t r = r0; r < r1; ++r) {
      const uint16_t* s = stream + row_start[r];
      uint16_t* c = codes + (uint64_t)r * gpr_pad;
      uint16_t* ix = rawidx + (uint64_t)r * nidx_pad;
      uint32_t* rw = raw + rawbase[r];
      uint32_t nraw = 0;
      for (uint32_t g = 0; g < gpr; ++g) {
        if ((g & 31u) == 0) ix[g >> 5] = (uint16_t)nraw;
        const uint16_t v = *s++;
        c[g] = v;
        if (v == TQ_ESCAPE) {
          rw[nraw++] = (uint32_t)(s[0] & 0xFF) | ((uint32_t)(s[1] & 0xFF) << 8) | ((uint32_t)(s[2] & 0xFF) << 16) |
                       ((uint32_t)(s[3] & 0xFF) << 24);
          s += 4;
        }
      }
      for (uint32_t k = (gpr + 31u) >> 5; k < nidx; ++k) ix[k] = (uint16_t)nraw;
    }
  });
  return TQ_OK;
}

// ---------------------------------------------------------------------------------------------
// TILES layout: the content of PLANES, ordered for a warp that decodes 16 rows at a time straight
// into the operand registers of an 8-bit tensor-core MMA.  A tile covers a row block of 16 rows and
// a step of 32 groups (128 columns) and is 1 KB of tokens: lane l = 4*g + t of the warp owns, for
// h = 0, 1, the 8 tokens of row 16*rb + g + 8*h, groups 32*s + 8*t .. + 7, stored at byte
// h*512 + l*16 of the tile (one 128-bit load per lane and half).  Tiles are stored row block by
// row block, step by step.  Rows past the matrix and groups past the row hold token 0, which
// decodes to four zero bytes.  The 4 raw bytes behind each marker are packed into one word of a
// single raw stream, tile by tile; tile_raw[i] is the index of tile i's first raw word.  In place
// of the marker 0xFFFF the token of such a group is 0xFC00 + (p mod 1024), p being the index of
// its raw word in that stream: the kernels stage the stream through a ring of
// TQ_TILES_RING_WORDS = 1024 words in which word p sits in slot p mod 1024, so the token is the
// address of its word and no marker counting is needed.  (A tile holds at most 512 raw words, so
// p is recovered from tile_raw[i] and the token.)
//
// The kernels keep the whole table they index in shared memory, which holds TQ_TILES_TABLE_WORDS
// words.  A group whose code is beyond that is therefore stored the way Listing 3 stores a group
// that is not in the table -- marker in the token tile, its 4 bytes (taken from the table) in the
// raw stream -- which is the stream Listing 3 would have produced with top_k =
// TQ_TILES_TABLE_WORDS - 1, since the table is ranked and a shorter one is a prefix of it.
// Decoding gives the same bytes; the image is 4 bytes larger per such group.
// ---------------------------------------------------------------------------------------------
int tq_build_tiles_image(const uint16_t* stream, uint64_t stream_len, uint32_t rows, uint32_t cols,
                         uint32_t K, const uint32_t* table, const float* row_scale, const float* row_zero,
                         uint64_t* device_bytes, tq_tiles_image* img) {
  std::vector<uint64_t> row_start;
  uint64_t H = 0, M = 0;
  int rc = scan_stream(stream, stream_len, rows, cols, K, row_start, H, M);
  if (rc != TQ_OK) return rc;
  if (M >= (1ull << 32) - 65536) return TQ_ERR_UNSUPPORTED_SHAPE;
  if (cols > TQ_TILES_MAX_COLS) return TQ_ERR_UNSUPPORTED_SHAPE;  // 32-bit accumulators of the integer MMA

  const uint32_t gpr = cols / 4;
  const uint32_t steps = (gpr + 31u) / 32u;
  const uint32_t row_blocks = (rows + 15u) / 16u;
  const uint64_t n_tiles = (uint64_t)steps * row_blocks;
  if (n_tiles >= (1ull << 31)) return TQ_ERR_UNSUPPORTED_SHAPE;
  const uint64_t rows_pad = (uint64_t)row_blocks * 16;
  const uint32_t limit = TQ_TILES_TABLE_WORDS;
  const uint32_t miss_base = 0x10000u - TQ_TILES_RING_WORDS;
  static_assert(TQ_TILES_TABLE_WORDS <= 0x10000u - TQ_TILES_RING_WORDS, "codes and miss tokens must not overlap");

  // pass 1: raw words per tile (markers and codes beyond the shared-memory table)
  std::vector<uint32_t> tile_raw_v;
  try {
    tile_raw_v.assign(n_tiles + 1, 0);
  } catch (const std::bad_alloc&) {
    return TQ_ERR_NOMEM;
  }
  const int T = (int)std::min<uint64_t>(tq_num_threads(), row_blocks);
  parallel_run(T, [&](int t) {
    const uint32_t b0 = (uint32_t)((uint64_t)row_blocks * t / T), b1 = (uint32_t)((uint64_t)row_blocks * (t + 1) / T);
    for (uint32_t rb = b0; rb < b1; ++rb) {
      uint32_t* cnt = tile_raw_v.data() + (uint64_t)rb * steps + 1;  // shifted by one: becomes the prefix sum below
      for (uint32_t i = 0; i < 16; ++i) {
        const uint32_t r = rb * 16 + i;
        if (r >= rows) break;
        const uint16_t* s = stream + row_start[r];
        for (uint32_t g = 0; g < gpr; ++g) {
          const uint16_t v = *s;
          if (v == TQ_ESCAPE) {
            ++cnt[g >> 5];
            s += 5;
          } else {
            if (v >= limit) ++cnt[g >> 5];
            ++s;
          }
        }
      }
    }
  });
  uint64_t n_raw = 0;
  for (uint64_t i = 0; i < n_tiles; ++i) {
    n_raw += tile_raw_v[i + 1];
    if (n_raw >= (1ull << 32) - 65536) return TQ_ERR_UNSUPPORTED_SHAPE;
    tile_raw_v[i + 1] = (uint32_t)n_raw;
  }

  const tq_tiles_geometry geo = tq_tiles_layout(rows, cols);
  const uint64_t off_status = geo.off_status, off_scale = geo.off_scale, off_zero = geo.off_zero;
  const uint64_t off_tile_raw = geo.off_tile_raw, off_tokens = geo.off_tokens, off_raw = geo.off_raw;
  const uint64_t total = geo.total(n_raw);
  if (device_bytes) *device_bytes = total;
  if (!img) return TQ_OK;
  if (!row_scale || !table) return TQ_ERR_INVALID_ARG;
  try {
    img->blob.assign(total, 0);
  } catch (const std::bad_alloc&) {
    return TQ_ERR_NOMEM;
  }
  img->off_status = off_status;
  img->off_scale = off_scale;
  img->off_zero = off_zero;
  img->off_tile_raw = off_tile_raw;
  img->off_tokens = off_tokens;
  img->off_raw = off_raw;
  img->steps = steps;
  img->row_blocks = row_blocks;
  img->n_hits = H;
  img->n_miss = M;
  img->n_raw = n_raw;
  img->rb_raw.resize((size_t)row_blocks + 1);
  for (uint32_t rb = 0; rb <= row_blocks; ++rb) img->rb_raw[rb] = tile_raw_v[(uint64_t)rb * steps];
  uint8_t* base = img->blob.data();
  std::memcpy(base + off_scale, row_scale, (size_t)rows * 4);
  if (row_zero) std::memcpy(base + off_zero, row_zero, (size_t)rows * 4);
  uint32_t* tile_raw = reinterpret_cast<uint32_t*>(base + off_tile_raw);
  std::memcpy(tile_raw, tile_raw_v.data(), (n_tiles + 1) * 4);
  for (int i = 1; i <= 8; ++i) tile_raw[n_tiles + i] = (uint32_t)n_raw;  // read ahead by the kernels, never used
  uint16_t* tokens = reinterpret_cast<uint16_t*>(base + off_tokens);
  uint32_t* raw = reinterpret_cast<uint32_t*>(base + off_raw);

  // pass 2: tokens and raw words in tile order.  A row's groups are met in ascending order, so one
  // cursor per row is enough.  Inside a tile the raw words are numbered slot by slot (slot j = 8h + i
  // of every lane, lanes ascending), so the words one lookup instruction of the warp reads are
  // neighbours in shared memory.
  parallel_run(T, [&](int t) {
    const uint32_t b0 = (uint32_t)((uint64_t)row_blocks * t / T), b1 = (uint32_t)((uint64_t)row_blocks * (t + 1) / T);
    uint32_t word[32][16];
    bool is_raw[32][16];
    for (uint32_t rb = b0; rb < b1; ++rb) {
      const uint16_t* cur[16];
      for (uint32_t i = 0; i < 16; ++i) cur[i] = rb * 16 + i < rows ? stream + row_start[rb * 16 + i] : nullptr;
      for (uint32_t s = 0; s < steps; ++s) {
        const uint64_t tile = (uint64_t)rb * steps + s;
        uint16_t* tk = tokens + tile * 512;
        for (uint32_t lane = 0; lane < 32; ++lane) {
          const uint32_t g = lane >> 2, q = lane & 3u;
          for (uint32_t h = 0; h < 2; ++h) {
            const uint16_t*& c = cur[g + 8 * h];
            for (uint32_t i = 0; i < 8; ++i) {
              const uint32_t grp = 32 * s + 8 * q + i, j = 8 * h + i;
              is_raw[lane][j] = false;
              word[lane][j] = 0;  // token 0: four zero bytes
              if (!c || grp >= gpr) continue;
              const uint16_t v = *c++;
              if (v == TQ_ESCAPE) {
                is_raw[lane][j] = true;
                word[lane][j] = (uint32_t)(c[0] & 0xFF) | ((uint32_t)(c[1] & 0xFF) << 8) |
                                ((uint32_t)(c[2] & 0xFF) << 16) | ((uint32_t)(c[3] & 0xFF) << 24);
                c += 4;
              } else if (v >= limit) {
                is_raw[lane][j] = true;
                word[lane][j] = table[v];
              } else {
                word[lane][j] = v;
              }
            }
          }
        }
        uint32_t pos = tile_raw[tile];
        for (uint32_t j = 0; j < 16; ++j) {
          for (uint32_t lane = 0; lane < 32; ++lane) {
            uint16_t* out = tk + (j >> 3) * 256 + lane * 8 + (j & 7u);
            if (is_raw[lane][j]) {
              raw[pos] = word[lane][j];
              *out = (uint16_t)(miss_base | (pos & (TQ_TILES_RING_WORDS - 1u)));
              ++pos;
            } else {
              *out = (uint16_t)word[lane][j];
            }
          }
        }
      }
    }
  });
  return TQ_OK;
}

extern "C" int tq_tiles_image_host(const tq_dict* d, const uint16_t* stream, uint64_t stream_len, uint32_t rows,
                                   uint32_t cols, const float* row_scale, const float* row_zero, uint8_t* out,
                                   uint64_t out_cap, uint64_t* out_bytes, uint64_t* offsets, uint32_t* dims) {
  if (!d || !out_bytes) return TQ_ERR_INVALID_ARG;
  if (!out) return tq_build_tiles_image(stream, stream_len, rows, cols, d->K, nullptr, nullptr, nullptr, out_bytes, nullptr);
  if (!offsets || !dims) return TQ_ERR_INVALID_ARG;
  std::vector<uint32_t> table((size_t)d->K + 1, 0);
  if (d->K) std::memcpy(table.data() + 1, d->entries.data(), (size_t)d->K * 4);
  tq_tiles_image img;
  int rc = tq_build_tiles_image(stream, stream_len, rows, cols, d->K, table.data(), row_scale, row_zero, out_bytes, &img);
  if (rc != TQ_OK) return rc;
  if (out_cap < img.blob.size()) return TQ_ERR_BUFFER_TOO_SMALL;
  std::memcpy(out, img.blob.data(), img.blob.size());
  offsets[0] = img.off_scale;
  offsets[1] = img.off_zero;
  offsets[2] = img.off_tile_raw;
  offsets[3] = img.off_tokens;
  offsets[4] = img.off_raw;
  dims[0] = img.steps;
  dims[1] = img.row_blocks;
  return TQ_OK;
}
