/*
 * Tiny-QMoE CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded, obviously-correct restatement of what the
 * paper's pipeline computes: the naive min-max quantizer (Listing 1), the
 * 4-gram dictionary (Listing 2), the uint16 token stream encoder (Listing 3),
 * the decoder (Listing 4) and the dense layer product that consumes the
 * decoded weights (Section 2.3, Section 5 "Model Loading").  It shares no code,
 * header, table or helper with the CUDA library; only tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it.
 *
 * No blocking, fusion, SIMD or threading.  The quantizers and the table builder
 * take the steps of the listings they cite, in the paper's order; the coder and
 * the decoder are written from the definition of the stream format (Section 4),
 * so that each can be checked against the paper by eye.
 *
 * Pins (see tests/test_oracle_pins.py): round trip exactness, the stream-size
 * identity, closed forms (constant input, empty table, all-hit), brute-force
 * window counting on tiny inputs, hand-worked fixtures, quantizer end points
 * and error bound, and a library fp64 GEMV.  The one thing with no pin is the
 * paper's Table 1 (model sizes): it cannot be derived from the listings and is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define TQO_ESCAPE 0xFFFFu      /* Listing 3: marker that precedes raw values   */
#define TQO_SEQ 4               /* Listing 2: sequence_length default            */
#define TQO_MAX_ENTRIES 65534u  /* codes 1..65534; 65535 would collide with the
                                   escape marker that the decoder tests first   */

/* ------------------------------------------------------------------------ */
/* Listing 1: naive min-max quantizer, per tensor, maxq = 2^bits - 1 levels   */
/* above zero (bits = 8 in the paper's pipeline; Section 3 also tried 2, 4,  */
/* 6).  All arithmetic in fp32 with round-half-to-even, as the listing's     */
/* tensor ops do.  Writes the integer level q (0..maxq); returns scale and   */
/* zero.  Returns -1 when the range is empty (scale would be 0) or bits is   */
/* not an integer in 1..8 (the listing's ternary branch, bits = 1.5, makes   */
/* no integer level and is not part of this path).                           */
/* ------------------------------------------------------------------------ */
int tqo_quantize_paper_bits(const float *x, uint64_t n, int bits, uint8_t *q,
                            float *scale_out, float *zero_out) {
  if (n == 0 || bits < 1 || bits > 8) return -1;
  const float maxq = (float)((1 << bits) - 1);
  float xmin = x[0], xmax = x[0];
  for (uint64_t i = 1; i < n; ++i) {
    if (x[i] < xmin) xmin = x[i];
    if (x[i] > xmax) xmax = x[i];
  }
  float scale = (xmax - xmin) / maxq;
  if (!(scale > 0.0f)) return -1;
  float zero = nearbyintf(-xmin / scale);
  for (uint64_t i = 0; i < n; ++i) {
    float v = nearbyintf(x[i] / scale) + zero;
    if (v < 0.0f) v = 0.0f;
    if (v > maxq) v = maxq;
    q[i] = (uint8_t)v;
  }
  *scale_out = scale;
  *zero_out = zero;
  return 0;
}

int tqo_quantize_paper(const float *x, uint64_t n, uint8_t *q, float *scale_out,
                       float *zero_out) {
  return tqo_quantize_paper_bits(x, n, 8, q, scale_out, zero_out);
}

/* ------------------------------------------------------------------------ */
/* The benchmark configurations' quantizer (not in the paper): per output    */
/* row, symmetric, s_r = max|w| / 127, q = clamp(round(w / s_r), -127, 127). */
/* An all-zero row gets s_r = 1.  The byte that is dictionary coded is the   */
/* two's-complement pattern of q (Listing 2's astype(uint8)).                */
/* ------------------------------------------------------------------------ */
void tqo_quantize_rows(const float *w, uint32_t rows, uint32_t cols, int8_t *q,
                       float *scale) {
  for (uint32_t r = 0; r < rows; ++r) {
    const float *wr = w + (uint64_t)r * cols;
    float amax = 0.0f;
    for (uint32_t c = 0; c < cols; ++c) {
      float a = fabsf(wr[c]);
      if (a > amax) amax = a;
    }
    float s = amax > 0.0f ? amax / 127.0f : 1.0f;
    scale[r] = s;
    for (uint32_t c = 0; c < cols; ++c) {
      float v = nearbyintf(wr[c] / s);
      if (v < -127.0f) v = -127.0f;
      if (v > 127.0f) v = 127.0f;
      q[(uint64_t)r * cols + c] = (int8_t)v;
    }
  }
}

/* ------------------------------------------------------------------------ */
/* Listing 2: count every stride-1 window of L consecutive bytes over each   */
/* flattened matrix (windows never span two matrices), keep the top_k most   */
/* frequent, code = rank + 1.  L is the listing's sequence_length parameter  */
/* (default 4, the value the paper's pipeline runs with; 1..8 here).  Ties   */
/* keep first-insertion order, which is what a stable descending sort of an  */
/* insertion-ordered counter gives.                                          */
/* ------------------------------------------------------------------------ */
typedef struct {
  uint64_t key;    /* the L bytes, byte i of the window in bits 8i..8i+7 */
  uint64_t count;
  uint64_t first;  /* insertion order */
  uint32_t used;
} tqo_slot;

typedef struct {
  uint32_t seq;                   /* L: bytes per window / per table entry  */
  uint32_t n_entries;             /* K                                      */
  uint8_t *entries;               /* K x L, rank order                      */
  uint64_t *counts;               /* K, occurrence count of each entry      */
  uint64_t n_distinct;            /* distinct windows seen                  */
  uint64_t n_windows;             /* total windows counted                  */
  /* lookup map for the encoder: key -> code */
  uint32_t map_cap;
  uint64_t *map_key;
  uint16_t *map_code;             /* 0 = empty */
} tqo_dict;

static uint64_t tqo_hash(uint64_t k) {
  k ^= k >> 33;
  k *= 0xff51afd7ed558ccdull;
  k ^= k >> 33;
  k *= 0xc4ceb9fe1a85ec53ull;
  k ^= k >> 33;
  return k;
}

/* the L bytes at w as one integer */
static uint64_t tqo_window(const uint8_t *w, uint32_t L) {
  uint64_t key = 0;
  for (uint32_t j = 0; j < L; ++j) key |= (uint64_t)w[j] << (8 * j);
  return key;
}

static int tqo_cmp_rank(const void *a, const void *b) {
  const tqo_slot *x = (const tqo_slot *)a, *y = (const tqo_slot *)b;
  if (x->count != y->count) return x->count > y->count ? -1 : 1;
  if (x->first != y->first) return x->first < y->first ? -1 : 1;
  return 0;
}

static void tqo_map_insert(tqo_dict *d, uint64_t key, uint16_t code) {
  uint64_t m = d->map_cap - 1, h = tqo_hash(key) & m;
  while (d->map_code[h] != 0) h = (h + 1) & m;
  d->map_key[h] = key;
  d->map_code[h] = code;
}

/* code of a window, 0 if it is not in the table */
static uint16_t tqo_map_find(const tqo_dict *d, uint64_t key) {
  uint64_t m = d->map_cap - 1, h = tqo_hash(key) & m;
  while (d->map_code[h] != 0) {
    if (d->map_key[h] == key) return d->map_code[h];
    h = (h + 1) & m;
  }
  return 0;
}

void tqo_dict_free(tqo_dict *d) {
  if (!d) return;
  free(d->entries);
  free(d->counts);
  free(d->map_key);
  free(d->map_code);
  free(d);
}

static tqo_dict *tqo_dict_alloc(uint32_t K, uint32_t L) {
  tqo_dict *d = (tqo_dict *)calloc(1, sizeof(tqo_dict));
  if (!d) return NULL;
  d->seq = L;
  d->n_entries = K;
  d->entries = (uint8_t *)malloc(K ? (size_t)K * L : L);
  d->counts = (uint64_t *)calloc(K ? K : 1, 8);
  d->map_cap = 1u << 18; /* > 2 x 65534 */
  d->map_key = (uint64_t *)calloc(d->map_cap, sizeof(uint64_t));
  d->map_code = (uint16_t *)calloc(d->map_cap, sizeof(uint16_t));
  return d;
}

tqo_dict *tqo_build_dictionary_seq(const uint8_t *const *mats, const uint64_t *n_elems,
                                   int n_mats, uint32_t top_k, uint32_t L) {
  if (L < 1 || L > 8) return NULL;
  uint64_t cap = 1024;
  uint64_t used = 0, windows = 0;
  tqo_slot *tab = (tqo_slot *)calloc(cap, sizeof(tqo_slot));
  if (!tab) return NULL;
  for (int m = 0; m < n_mats; ++m) {
    const uint8_t *w = mats[m];
    uint64_t n = n_elems[m];
    for (uint64_t i = 0; i + L <= n; ++i) {
      uint64_t key = tqo_window(w + i, L);
      if ((used + 1) * 10 > cap * 6) { /* grow at 60 % load */
        uint64_t ncap = cap * 2;
        tqo_slot *nt = (tqo_slot *)calloc(ncap, sizeof(tqo_slot));
        if (!nt) { free(tab); return NULL; }
        for (uint64_t s = 0; s < cap; ++s)
          if (tab[s].used) {
            uint64_t h = tqo_hash(tab[s].key) & (ncap - 1);
            while (nt[h].used) h = (h + 1) & (ncap - 1);
            nt[h] = tab[s];
          }
        free(tab);
        tab = nt;
        cap = ncap;
      }
      uint64_t h = tqo_hash(key) & (cap - 1);
      while (tab[h].used && tab[h].key != key) h = (h + 1) & (cap - 1);
      if (!tab[h].used) {
        tab[h].used = 1;
        tab[h].key = key;
        tab[h].count = 0;
        tab[h].first = used++;
      }
      tab[h].count++;
      windows++;
    }
  }
  /* compact, rank */
  tqo_slot *all = (tqo_slot *)malloc((used ? used : 1) * sizeof(tqo_slot));
  uint64_t k = 0;
  for (uint64_t s = 0; s < cap; ++s)
    if (tab[s].used) all[k++] = tab[s];
  free(tab);
  qsort(all, used, sizeof(tqo_slot), tqo_cmp_rank);

  uint64_t K = used;
  if (K > top_k) K = top_k;
  if (K > TQO_MAX_ENTRIES) K = TQO_MAX_ENTRIES;

  tqo_dict *d = tqo_dict_alloc((uint32_t)K, L);
  d->n_distinct = used;
  d->n_windows = windows;
  for (uint64_t r = 0; r < K; ++r) {
    for (uint32_t j = 0; j < L; ++j) d->entries[L * r + j] = (uint8_t)(all[r].key >> (8 * j));
    d->counts[r] = all[r].count;
    tqo_map_insert(d, all[r].key, (uint16_t)(r + 1)); /* code = rank + 1 */
  }
  free(all);
  return d;
}

tqo_dict *tqo_build_dictionary(const uint8_t *const *mats, const uint64_t *n_elems,
                               int n_mats, uint32_t top_k) {
  return tqo_build_dictionary_seq(mats, n_elems, n_mats, top_k, TQO_SEQ);
}

/* Build a dictionary object from an explicit entry list (rank order), so the
 * encoder/decoder can be exercised with hand-made tables. */
tqo_dict *tqo_dict_from_entries_seq(const uint8_t *entries, uint32_t K, uint32_t L) {
  if (K > TQO_MAX_ENTRIES || L < 1 || L > 8) return NULL;
  tqo_dict *d = tqo_dict_alloc(K, L);
  memcpy(d->entries, entries, (size_t)K * L);
  for (uint32_t r = 0; r < K; ++r) {
    uint64_t key = tqo_window(entries + (size_t)L * r, L);
    if (tqo_map_find(d, key) == 0) tqo_map_insert(d, key, (uint16_t)(r + 1));
  }
  return d;
}

tqo_dict *tqo_dict_from_entries(const uint8_t *entries, uint32_t K) {
  return tqo_dict_from_entries_seq(entries, K, TQO_SEQ);
}

uint32_t tqo_dict_size(const tqo_dict *d) { return d->n_entries; }
uint32_t tqo_dict_seq(const tqo_dict *d) { return d->seq; }
const uint8_t *tqo_dict_entries(const tqo_dict *d) { return d->entries; }
const uint64_t *tqo_dict_counts(const tqo_dict *d) { return d->counts; }
uint64_t tqo_dict_distinct(const tqo_dict *d) { return d->n_distinct; }
uint64_t tqo_dict_windows(const tqo_dict *d) { return d->n_windows; }

/* ------------------------------------------------------------------------ */
/* The stream format (Section 4; Listing 3 writes it, Listing 4 reads it).   */
/* The n bytes of a matrix are cut into consecutive blocks of L bytes (the   */
/* last block may be shorter).  A full block that is a table entry is one    */
/* uint16 item, its code; any other block is the marker 0xFFFF followed by   */
/* its bytes, each widened to uint16.  So block j starts at slot             */
/* sum over the blocks before it of (1 if coded, else 1 + its length).       */
/*                                                                           */
/* tqo_encode states exactly that: classify every block, place every block   */
/* by the running sum, fill the slots.  out == NULL: size query.  Returns    */
/* the stream length in uint16 units, or (uint64_t)-1 if cap is too small.   */
/* n_hits / n_miss (may be NULL) count the coded / marked full blocks.       */
/* ------------------------------------------------------------------------ */
uint64_t tqo_encode(const tqo_dict *d, const uint8_t *w, uint64_t n, uint16_t *out,
                    uint64_t cap, uint64_t *n_hits, uint64_t *n_miss) {
  const uint32_t L = d->seq;
  const uint64_t n_full = n / L, tail = n % L;
  const uint64_t n_blocks = n_full + (tail ? 1 : 0);
  uint16_t *code = (uint16_t *)malloc((n_blocks ? n_blocks : 1) * sizeof(uint16_t));
  if (!code) return (uint64_t)-1;
  uint64_t hits = 0;
  for (uint64_t j = 0; j < n_full; ++j) {
    code[j] = tqo_map_find(d, tqo_window(w + j * L, L));
    hits += code[j] != 0;
  }
  if (tail) code[n_full] = 0; /* a short block is never a table entry */
  const uint64_t len = hits + (n_full - hits) * (1 + (uint64_t)L) + (tail ? 1 + tail : 0);
  if (n_hits) *n_hits = hits;
  if (n_miss) *n_miss = n_full - hits;
  if (out) {
    if (len > cap) { free(code); return (uint64_t)-1; }
    uint64_t slot = 0;
    for (uint64_t j = 0; j < n_blocks; ++j) {
      const uint64_t blen = j < n_full ? L : tail;
      if (code[j]) {
        out[slot++] = code[j];
      } else {
        out[slot++] = TQO_ESCAPE;
        for (uint64_t e = 0; e < blen; ++e) out[slot++] = w[j * L + e];
      }
    }
  }
  free(code);
  return len;
}

/* ------------------------------------------------------------------------ */
/* tqo_decode reads the same format back.  First the items are located: an   */
/* item is either one slot (a code) or a marker with the up to L slots that  */
/* follow it (fewer only when the stream ends: the short last block, which   */
/* is how Listing 4's slice behaves).  Then every item is expanded: a code   */
/* to its table entry, a marked item to the low bytes of its slots.  Returns */
/* the number of bytes produced, -1 for a code that is not in the table      */
/* (Listing 4 raises there), -2 if out is too small, -3 out of memory.       */
/* ------------------------------------------------------------------------ */
int64_t tqo_decode(const tqo_dict *d, const uint16_t *s, uint64_t len, uint8_t *out,
                   uint64_t cap) {
  const uint32_t L = d->seq;
  uint64_t *start = (uint64_t *)malloc((len ? len : 1) * sizeof(uint64_t));
  if (!start) return -3;
  uint64_t n_items = 0;
  for (uint64_t pos = 0; pos < len;) {
    start[n_items++] = pos;
    pos += s[pos] == TQO_ESCAPE ? 1 + (uint64_t)L : 1;
  }
  uint64_t o = 0;
  int64_t rc = 0;
  for (uint64_t it = 0; it < n_items && rc == 0; ++it) {
    const uint64_t pos = start[it];
    if (s[pos] == TQO_ESCAPE) {
      const uint64_t avail = len - (pos + 1);
      const uint64_t take = avail < L ? avail : L;
      if (o + take > cap) { rc = -2; break; }
      for (uint64_t e = 0; e < take; ++e) out[o++] = (uint8_t)s[pos + 1 + e];
    } else {
      const uint16_t c = s[pos];
      if (c == 0 || c > d->n_entries) { rc = -1; break; }
      if (o + L > cap) { rc = -2; break; }
      for (uint32_t e = 0; e < L; ++e) out[o++] = d->entries[(uint64_t)L * (c - 1) + e];
    }
  }
  free(start);
  return rc ? rc : (int64_t)o;
}

/* ------------------------------------------------------------------------ */
/* The layer that consumes the decoded weights (Section 2.3; Listing 1's     */
/* dequantisation scale * (q - zero)): y[b][r] = s_r * sum_c (q[r][c]-z_r) * */
/* x[b][c], everything in fp64.  is_signed: the byte is an int8 pattern.     */
/* zero may be NULL (all zero).  No bias (LLaMA linears have none).          */
/* ------------------------------------------------------------------------ */
void tqo_layer_forward(const uint8_t *q, int is_signed, uint32_t rows, uint32_t cols,
                       const float *scale, const float *zero, const double *x,
                       uint32_t batch, double *y) {
  for (uint32_t b = 0; b < batch; ++b)
    for (uint32_t r = 0; r < rows; ++r) {
      double z = zero ? (double)zero[r] : 0.0;
      double acc = 0.0;
      for (uint32_t c = 0; c < cols; ++c) {
        uint8_t byte = q[(uint64_t)r * cols + c];
        double v = is_signed ? (double)(int8_t)byte : (double)byte;
        acc += (v - z) * x[(uint64_t)b * cols + c];
      }
      y[(uint64_t)b * rows + r] = (double)scale[r] * acc;
    }
}
