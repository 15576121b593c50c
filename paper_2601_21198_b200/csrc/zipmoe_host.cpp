// Host side of the library: offline encoder, container validation and the
// planner that turns a blob into per-chunk descriptors for a decode launch.
// Paper Section 3.1 ("Offline Initialization"): bit-field decomposition,
// exponent stream cut into independently compressed shards (E-chunks),
// sign+mantissa bytes packed raw (SM-chunks), everything serialised with its
// metadata.  No CUDA in this file.
#include <algorithm>
#include <queue>
#include <thread>
#include <vector>

#include "zipmoe_format.h"

namespace zipmoe {

zipmoe_status make_geometry(uint64_t rows, uint64_t cols, uint32_t layout, uint32_t chunk_elems, Geometry *g) {
  *g = Geometry();
  if (rows > 0xFFFFFFFFull || cols > 0xFFFFFFFFull) return ZIPMOE_ERR_INVALID_ARG;
  if (chunk_elems == 0 || chunk_elems % kIterElems) return ZIPMOE_ERR_INVALID_ARG;
  if (chunk_elems > ZIPMOE_TILE_ELEMS_MAX && chunk_elems % ZIPMOE_TILE_ELEMS_MAX) return ZIPMOE_ERR_INVALID_ARG;
  g->n_elems = rows * cols;
  g->rows = (uint32_t)rows;
  g->cols = (uint32_t)cols;
  g->layout = layout;
  g->chunk_elems = chunk_elems;
  g->tile_elems = std::min<uint32_t>(chunk_elems, ZIPMOE_TILE_ELEMS_MAX);
  g->iters = g->tile_elems / kIterElems;
  g->tiles_per_chunk = chunk_elems / g->tile_elems;
  uint64_t n_tiles;
  if (layout == ZIPMOE_LAYOUT_LINEAR) {
    n_tiles = (g->n_elems + g->tile_elems - 1) / g->tile_elems;
    g->sm_bytes = align_up(g->n_elems, 16);
  } else if (layout == ZIPMOE_LAYOUT_BLOCKED) {
    if (g->tile_elems != ZIPMOE_TILE_ELEMS_MAX || rows % 16 || cols % 256) return ZIPMOE_ERR_INVALID_ARG;
    g->tiles_per_rowblk = (uint32_t)(cols / 256);
    n_tiles = (rows / 16) * (cols / 256);
    g->sm_bytes = g->n_elems;
  } else {
    return ZIPMOE_ERR_INVALID_ARG;
  }
  if (n_tiles > 0xFFFFFFFFull) return ZIPMOE_ERR_UNSUPPORTED;
  g->n_tiles = (uint32_t)n_tiles;
  g->n_chunks = (g->n_tiles + g->tiles_per_chunk - 1) / g->tiles_per_chunk;
  g->payload_off = align_up(kChunkOffOff + 8ull * (g->n_chunks + 1), 16);
  return ZIPMOE_OK;
}

namespace {

struct Opts {
  uint32_t chunk_elems, max_code_len, layout, n_threads;
};

zipmoe_status resolve_opts(const zipmoe_encode_opts *o, Opts *r) {
  r->chunk_elems = (o && o->chunk_elems) ? o->chunk_elems : 65536u;
  r->max_code_len = (o && o->max_code_len) ? o->max_code_len : 8u;
  r->layout = o ? o->layout : ZIPMOE_LAYOUT_LINEAR;
  r->n_threads = (o && o->n_threads) ? o->n_threads : 1u;
  if (r->max_code_len < 8 || r->max_code_len > ZIPMOE_MAX_CODE_LEN) return ZIPMOE_ERR_INVALID_ARG;
  if (r->n_threads > 256) r->n_threads = 256;
  return ZIPMOE_OK;
}

uint64_t tile_record_max(uint32_t) { return kRecordHeadBytes + (uint64_t)kMaxRows * kRowBytes; }

// Huffman code lengths by the usual greedy merge on a min-heap.  When the tree
// is deeper than `limit` the rare symbols' counts are flattened (halved,
// rounding up, never below one) and the tree rebuilt: each pass brings the
// counts closer together, and equal counts give depth ceil(log2 m) <= 8, so the
// loop ends.  The result is a true Huffman code of the flattened counts: Kraft
// sum exactly one, slightly above optimal cost when the limit binds.
void huffman_lengths(const uint64_t *hist, uint32_t limit, uint8_t *len) {
  std::memset(len, 0, 256);
  std::vector<int> live;
  for (int s = 0; s < 256; ++s)
    if (hist[s]) live.push_back(s);
  if (live.empty()) return;
  if (live.size() == 1) {  // keep the code complete: a dummy sibling of length one
    len[live[0]] = 1;
    len[(live[0] + 1) & 255] = 1;
    return;
  }
  std::vector<uint64_t> w(live.size());
  for (size_t a = 0; a < live.size(); ++a) w[a] = hist[live[a]];
  const int m = (int)live.size();
  for (;;) {
    std::vector<int> parent(2 * m - 1, -1);
    using Node = std::pair<uint64_t, int>;
    std::priority_queue<Node, std::vector<Node>, std::greater<Node>> heap;
    for (int a = 0; a < m; ++a) heap.push({w[a], a});
    int next = m;
    while (heap.size() > 1) {
      Node x = heap.top(); heap.pop();
      Node y = heap.top(); heap.pop();
      parent[x.second] = parent[y.second] = next;
      heap.push({x.first + y.first, next});
      ++next;
    }
    uint32_t deepest = 0;
    for (int a = 0; a < m; ++a) {
      uint32_t d = 0;
      for (int v = a; parent[v] >= 0; v = parent[v]) ++d;
      len[live[a]] = (uint8_t)std::min<uint32_t>(d, 255);
      deepest = std::max(deepest, d);
    }
    if (deepest <= limit) return;
    for (auto &x : w) x = (x + 1) >> 1;
  }
}

void canonical_codes(const uint8_t *len, uint32_t *code) {
  uint32_t count[ZIPMOE_MAX_CODE_LEN + 2] = {0}, next[ZIPMOE_MAX_CODE_LEN + 2] = {0};
  for (int s = 0; s < 256; ++s) count[len[s]]++;
  count[0] = 0;
  uint32_t c = 0;
  for (uint32_t L = 1; L <= ZIPMOE_MAX_CODE_LEN; ++L) {
    next[L] = c;
    c = (c + count[L]) << 1;
  }
  for (int s = 0; s < 256; ++s) code[s] = len[s] ? next[len[s]]++ : 0;
}

// Appends codes to a word stream, most significant bit of each word first.
struct BitWriter {
  uint32_t *dst;
  uint64_t acc = 0;   // pending bits, right-aligned
  uint32_t fill = 0;  // number of pending bits (< 32 between calls)
  explicit BitWriter(uint32_t *p) : dst(p) {}
  void put(uint32_t code, uint32_t nbits) {
    acc = (acc << nbits) | code;
    fill += nbits;
    if (fill >= 32) {
      fill -= 32;
      *dst++ = (uint32_t)(acc >> fill);
    }
  }
  void flush() {
    if (fill) *dst++ = (uint32_t)(acc << (32 - fill));
    fill = 0;
  }
};

inline uint32_t reverse32(uint32_t v) {
  v = ((v >> 1) & 0x55555555u) | ((v & 0x55555555u) << 1);
  v = ((v >> 2) & 0x33333333u) | ((v & 0x33333333u) << 2);
  v = ((v >> 4) & 0x0F0F0F0Fu) | ((v & 0x0F0F0F0Fu) << 4);
  v = ((v >> 8) & 0x00FF00FFu) | ((v & 0x00FF00FFu) << 8);
  return (v >> 16) | (v << 16);
}

template <typename F>
void parallel_for(uint32_t n, uint32_t n_threads, F body) {
  n_threads = std::max<uint32_t>(1, std::min(n_threads, n));
  if (n_threads == 1) {
    for (uint32_t k = 0; k < n; ++k) body(k);
    return;
  }
  std::vector<std::thread> pool;
  for (uint32_t t = 0; t < n_threads; ++t)
    pool.emplace_back([=]() {
      for (uint32_t k = t; k < n; k += n_threads) body(k);
    });
  for (auto &th : pool) th.join();
}

// Code bits of every lane's forward stream (even iterations) and backward stream (odd iterations) of tile q.
void tile_stream_bits(const Geometry &g, const uint16_t *x, const uint8_t *len, uint32_t q, uint32_t *fbits,
                      uint32_t *bbits) {
  const uint32_t valid = g.tile_valid(q);
  const uint64_t origin = g.tile_origin(q), pitch = g.row_pitch();
  for (uint32_t lane = 0; lane < kLanes; ++lane) {
    uint32_t bits[2] = {0, 0};
    for (uint32_t i = 0; i < g.iters; ++i) {
      uint32_t pos = (i * kLanes + lane) * kGroup;
      if (pos >= valid) break;
      uint32_t cnt = std::min(kGroup, valid - pos);
      const uint16_t *p = x + origin + i * pitch + lane * kGroup;
      for (uint32_t j = 0; j < cnt; ++j) bits[i & 1] += len[(p[j] >> 7) & 0xFF];
    }
    fbits[lane] = bits[0];
    bbits[lane] = bits[1];
  }
}

// Which column takes which backward stream, and how many rows the record needs.  All columns of a record are
// equally high, so the record is as high as its fullest column: the lane with the k-th longest forward stream
// shares its column with the k-th shortest backward stream, which keeps the fullest column close to the mean.
uint32_t pair_streams(const uint32_t *fbits, const uint32_t *bbits, uint8_t *bcol) {
  uint8_t by_f[kLanes], by_b[kLanes];
  for (uint32_t a = 0; a < kLanes; ++a) by_f[a] = by_b[a] = (uint8_t)a;
  std::stable_sort(by_f, by_f + kLanes, [&](uint8_t a, uint8_t b) { return fbits[a] > fbits[b]; });
  std::stable_sort(by_b, by_b + kLanes, [&](uint8_t a, uint8_t b) { return bbits[a] < bbits[b]; });
  uint32_t rows = 1;
  for (uint32_t a = 0; a < kLanes; ++a) {
    bcol[by_b[a]] = by_f[a];
    rows = std::max(rows, (fbits[by_f[a]] + bbits[by_b[a]] + 31) / 32);
  }
  return rows;
}

}  // namespace
}  // namespace zipmoe

using namespace zipmoe;

extern "C" {

uint32_t zipmoe_version(void) { return 100; }

const char *zipmoe_status_string(zipmoe_status s) {
  switch (s) {
    case ZIPMOE_OK: return "ok";
    case ZIPMOE_ERR_INVALID_ARG: return "invalid argument";
    case ZIPMOE_ERR_BAD_FORMAT: return "bad container format";
    case ZIPMOE_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case ZIPMOE_ERR_CUDA: return "CUDA error";
    case ZIPMOE_ERR_DECODE_CORRUPT: return "corrupt compressed data";
    case ZIPMOE_ERR_UNSUPPORTED: return "unsupported shape or option";
    default: return "unknown status";
  }
}

zipmoe_status zipmoe_encode_bound(uint64_t rows, uint64_t cols, const zipmoe_encode_opts *opts,
                                  uint64_t *blob_bytes_max) {
  if (!blob_bytes_max) return ZIPMOE_ERR_INVALID_ARG;
  Opts o;
  Geometry g;
  zipmoe_status rc = resolve_opts(opts, &o);
  if (rc == ZIPMOE_OK) rc = make_geometry(rows, cols, o.layout, o.chunk_elems, &g);
  if (rc != ZIPMOE_OK) return rc;
  uint64_t table = align_up(4ull * (g.tiles_per_chunk + 1), 16);
  *blob_bytes_max = g.payload_off + (uint64_t)g.n_tiles * tile_record_max(g.tile_elems) + (uint64_t)g.n_chunks * table +
                    g.sm_bytes;
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_encode(const uint16_t *bf16, uint64_t rows, uint64_t cols, const zipmoe_encode_opts *opts,
                            void *blob_v, uint64_t blob_cap, uint64_t *blob_bytes) {
  if (!blob_bytes || (!bf16 && rows != 0 && cols != 0) || !blob_v) return ZIPMOE_ERR_INVALID_ARG;
  Opts o;
  Geometry g;
  zipmoe_status rc = resolve_opts(opts, &o);
  if (rc == ZIPMOE_OK) rc = make_geometry(rows, cols, o.layout, o.chunk_elems, &g);
  if (rc != ZIPMOE_OK) return rc;
  uint8_t *blob = static_cast<uint8_t *>(blob_v);

  // histogram of exponent bytes over the whole tensor (one code per tensor)
  std::vector<uint64_t> part((size_t)o.n_threads * 256, 0);
  const uint64_t n = g.n_elems;
  parallel_for(o.n_threads, o.n_threads, [&](uint32_t t) {
    uint64_t lo = n * t / o.n_threads, hi = n * (t + 1) / o.n_threads;
    uint64_t *h = &part[(size_t)t * 256];
    for (uint64_t k = lo; k < hi; ++k) h[(bf16[k] >> 7) & 0xFF]++;
  });
  uint64_t hist[256] = {0};
  for (uint32_t t = 0; t < o.n_threads; ++t)
    for (int s = 0; s < 256; ++s) hist[s] += part[(size_t)t * 256 + s];

  uint8_t len[256];
  uint32_t code[256];
  huffman_lengths(hist, o.max_code_len, len);
  canonical_codes(len, code);

  // pass 1: size of every tile record, then of every chunk
  std::vector<uint32_t> rec_units(g.n_tiles);  // record size in 16-byte units
  parallel_for(g.n_chunks, o.n_threads, [&](uint32_t k) {
    uint32_t q0 = k * g.tiles_per_chunk, m = g.chunk_tiles(k), fbits[kLanes], bbits[kLanes];
    uint8_t bcol[kLanes];
    for (uint32_t t = 0; t < m; ++t) {
      tile_stream_bits(g, bf16, len, q0 + t, fbits, bbits);
      rec_units[q0 + t] = (kRecordHeadBytes + pair_streams(fbits, bbits, bcol) * kRowBytes) / 16;
    }
  });
  std::vector<uint64_t> chunk_byte(g.n_chunks + 1, 0);
  for (uint32_t k = 0; k < g.n_chunks; ++k) {
    uint32_t q0 = k * g.tiles_per_chunk, m = g.chunk_tiles(k);
    uint64_t units = align_up(4ull * (m + 1), 16) / 16;
    for (uint32_t t = 0; t < m; ++t) units += rec_units[q0 + t];
    chunk_byte[k + 1] = chunk_byte[k] + units * 16;
  }
  const uint64_t payload_bytes = chunk_byte[g.n_chunks];
  const uint64_t sm_off = g.payload_off + payload_bytes;
  const uint64_t total = sm_off + g.sm_bytes;
  *blob_bytes = total;
  if (blob_cap < total) return ZIPMOE_ERR_BUFFER_TOO_SMALL;

  // header, table, chunk offsets
  std::memset(blob, 0, g.payload_off);
  store_le<uint32_t>(blob + 0, kMagic);
  store_le<uint32_t>(blob + 4, kVersion);
  store_le<uint64_t>(blob + 8, g.n_elems);
  store_le<uint32_t>(blob + 16, g.rows);
  store_le<uint32_t>(blob + 20, g.cols);
  store_le<uint32_t>(blob + 24, g.layout);
  store_le<uint32_t>(blob + 28, g.chunk_elems);
  store_le<uint32_t>(blob + 32, g.tile_elems);
  store_le<uint32_t>(blob + 36, o.max_code_len);
  store_le<uint32_t>(blob + 40, g.n_chunks);
  store_le<uint32_t>(blob + 44, g.n_tiles);
  store_le<uint64_t>(blob + 48, payload_bytes);
  store_le<uint64_t>(blob + 56, g.sm_bytes);
  std::memcpy(blob + kTableOff, len, 256);
  for (uint32_t k = 0; k <= g.n_chunks; ++k) store_le<uint64_t>(blob + kChunkOffOff + 8ull * k, chunk_byte[k] * 8);

  // pass 2: tile tables, tile records and the sign+mantissa bytes, chunk by chunk
  uint8_t *pay = blob + g.payload_off;
  uint8_t *smsec = blob + sm_off;
  if (g.sm_bytes > g.n_elems) std::memset(smsec + g.n_elems, 0, g.sm_bytes - g.n_elems);
  parallel_for(g.n_chunks, o.n_threads, [&](uint32_t k) {
    uint32_t q0 = k * g.tiles_per_chunk, m = g.chunk_tiles(k);
    uint8_t *chunk = pay + chunk_byte[k];
    uint64_t table_bytes = align_up(4ull * (m + 1), 16);
    std::memset(chunk, 0, table_bytes);
    uint32_t unit = (uint32_t)(table_bytes / 16);
    for (uint32_t t = 0; t < m; ++t) {
      const uint32_t q = q0 + t;
      store_le<uint32_t>(chunk + 4ull * t, unit);
      uint8_t *rec = chunk + (uint64_t)unit * 16;
      const uint64_t rec_bytes = (uint64_t)rec_units[q] * 16;
      std::memset(rec, 0, rec_bytes);
      const uint32_t rows = (uint32_t)((rec_bytes - kRecordHeadBytes) / kRowBytes);
      const uint32_t valid = g.tile_valid(q);
      const uint64_t origin = g.tile_origin(q), pitch = g.row_pitch();
      uint32_t fbits[kLanes], bbits[kLanes];
      tile_stream_bits(g, bf16, len, q, fbits, bbits);
      pair_streams(fbits, bbits, rec);   // rec[lane] = the column of the lane's backward stream
      uint32_t words[kMaxRows * kLanes];   // [rows][32], copied into the record once complete
      std::memset(words, 0, (size_t)rows * kRowBytes);
      for (uint32_t lane = 0; lane < kLanes; ++lane) {
        // both streams are first written as plain word streams (first bit = bit 31 of word 0) ...
        uint32_t fw[kMaxRows + 1] = {0}, bw[kMaxRows + 1] = {0};
        BitWriter f(fw), b(bw);
        for (uint32_t i = 0; i < g.iters; ++i) {
          uint32_t pos = (i * kLanes + lane) * kGroup;
          if (pos >= valid) break;
          uint32_t cnt = std::min(kGroup, valid - pos);
          const uint16_t *p = bf16 + origin + i * pitch + lane * kGroup;
          for (uint32_t j = 0; j < cnt; ++j) {
            uint32_t s = (p[j] >> 7) & 0xFF;
            if (i & 1) b.put(code[s], len[s]);
            else f.put(code[s], len[s]);
          }
        }
        f.flush();
        b.flush();
        // ... then the forward stream goes down its own column from row 0, and the backward stream up the
        // column it was paired with from the last row, bit-reversed as a whole (its k-th bit is the column's
        // bit 32 * rows - 1 - k).  The two never share a bit, so or-ing them into the rows is safe.
        const uint32_t fwords = (fbits[lane] + 31) / 32, bwords = (bbits[lane] + 31) / 32, bc = rec[lane];
        for (uint32_t r = 0; r < fwords; ++r) words[r * kLanes + lane] |= fw[r];
        for (uint32_t r = 0; r < bwords; ++r) words[(rows - 1 - r) * kLanes + bc] |= reverse32(bw[r]);
      }
      std::memcpy(rec + kRecordHeadBytes, words, (size_t)rows * kRowBytes);   // (little-endian host)
      // sign+mantissa bytes of the tile, in tile order
      uint8_t *smt = smsec + (uint64_t)q * g.tile_elems;
      for (uint32_t i = 0; i < g.iters; ++i) {
        uint32_t pos = i * kIterElems;
        if (pos >= valid) break;
        uint32_t cnt = std::min(kIterElems, valid - pos);
        const uint16_t *p = bf16 + origin + i * pitch;
        for (uint32_t e = 0; e < cnt; ++e) smt[pos + e] = (uint8_t)(((p[e] >> 8) & 0x80) | (p[e] & 0x7F));
      }
      unit += rec_units[q];
    }
    store_le<uint32_t>(chunk + 4ull * m, unit);
  });
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_blob_info_get(const void *blob_v, uint64_t bytes, zipmoe_blob_info *info) {
  if (!blob_v || !info) return ZIPMOE_ERR_INVALID_ARG;
  const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
  if (bytes < kChunkOffOff + 8) return ZIPMOE_ERR_BAD_FORMAT;
  if (load_le<uint32_t>(blob) != kMagic || load_le<uint32_t>(blob + 4) != kVersion) return ZIPMOE_ERR_BAD_FORMAT;
  uint64_t n = load_le<uint64_t>(blob + 8);
  uint32_t rows = load_le<uint32_t>(blob + 16), cols = load_le<uint32_t>(blob + 20);
  if ((uint64_t)rows * cols != n) return ZIPMOE_ERR_BAD_FORMAT;
  Geometry g;
  if (make_geometry(rows, cols, load_le<uint32_t>(blob + 24), load_le<uint32_t>(blob + 28), &g) != ZIPMOE_OK)
    return ZIPMOE_ERR_BAD_FORMAT;
  uint32_t mcl = load_le<uint32_t>(blob + 36);
  if (g.tile_elems != load_le<uint32_t>(blob + 32) || g.n_chunks != load_le<uint32_t>(blob + 40) ||
      g.n_tiles != load_le<uint32_t>(blob + 44) || mcl < 1 || mcl > ZIPMOE_MAX_CODE_LEN)
    return ZIPMOE_ERR_BAD_FORMAT;
  uint64_t payload_bytes = load_le<uint64_t>(blob + 48);
  if (payload_bytes % 16 || load_le<uint64_t>(blob + 56) != g.sm_bytes) return ZIPMOE_ERR_BAD_FORMAT;
  uint64_t total = g.payload_off + payload_bytes + g.sm_bytes;
  if (total < payload_bytes || total > bytes) return ZIPMOE_ERR_BAD_FORMAT;
  info->n_elems = n;
  info->rows = rows;
  info->cols = cols;
  info->layout = g.layout;
  info->chunk_elems = g.chunk_elems;
  info->tile_elems = g.tile_elems;
  info->max_code_len = mcl;
  info->n_chunks = g.n_chunks;
  info->n_tiles = g.n_tiles;
  info->table_off = kTableOff;
  info->chunk_off_off = kChunkOffOff;
  info->payload_off = g.payload_off;
  info->payload_bytes = payload_bytes;
  info->sm_off = g.payload_off + payload_bytes;
  info->sm_bytes = g.sm_bytes;
  info->total_bytes = total;
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_blob_validate(const void *blob_v, uint64_t bytes) {
  zipmoe_blob_info info;
  zipmoe_status rc = zipmoe_blob_info_get(blob_v, bytes, &info);
  if (rc != ZIPMOE_OK) return rc;
  const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
  Geometry g;
  make_geometry(info.rows, info.cols, info.layout, info.chunk_elems, &g);

  // complete prefix code
  const uint8_t *len = blob + kTableOff;
  uint64_t kraft = 0;
  for (int s = 0; s < 256; ++s) {
    if (len[s] > info.max_code_len) return ZIPMOE_ERR_BAD_FORMAT;
    if (len[s]) kraft += 1ull << (ZIPMOE_MAX_CODE_LEN - len[s]);
  }
  if (info.n_elems == 0) return kraft == 0 || kraft == (1ull << ZIPMOE_MAX_CODE_LEN) ? ZIPMOE_OK : ZIPMOE_ERR_BAD_FORMAT;
  if (kraft != (1ull << ZIPMOE_MAX_CODE_LEN)) return ZIPMOE_ERR_BAD_FORMAT;

  const uint8_t *pay = blob + info.payload_off;
  uint64_t prev = load_le<uint64_t>(blob + kChunkOffOff);
  if (prev != 0) return ZIPMOE_ERR_BAD_FORMAT;
  for (uint32_t k = 0; k < g.n_chunks; ++k) {
    uint64_t next = load_le<uint64_t>(blob + kChunkOffOff + 8ull * (k + 1));
    if (next % 128 || next < prev || next / 8 > info.payload_bytes) return ZIPMOE_ERR_BAD_FORMAT;
    const uint8_t *chunk = pay + prev / 8;
    uint64_t chunk_bytes = (next - prev) / 8;
    uint32_t m = g.chunk_tiles(k), q0 = k * g.tiles_per_chunk;
    uint64_t table_bytes = align_up(4ull * (m + 1), 16);
    if (table_bytes > chunk_bytes) return ZIPMOE_ERR_BAD_FORMAT;
    if ((uint64_t)load_le<uint32_t>(chunk) * 16 != table_bytes) return ZIPMOE_ERR_BAD_FORMAT;
    if ((uint64_t)load_le<uint32_t>(chunk + 4ull * m) * 16 != chunk_bytes) return ZIPMOE_ERR_BAD_FORMAT;
    for (uint32_t t = 0; t < m; ++t) {
      uint64_t r0 = (uint64_t)load_le<uint32_t>(chunk + 4ull * t) * 16;
      uint64_t r1 = (uint64_t)load_le<uint32_t>(chunk + 4ull * (t + 1)) * 16;
      // a record is the column table and at least one whole row of 32 words
      if (r1 < r0 + kRecordHeadBytes + kRowBytes || r1 > chunk_bytes || (r1 - r0 - kRecordHeadBytes) % kRowBytes)
        return ZIPMOE_ERR_BAD_FORMAT;
      if (r1 - r0 > tile_record_max(g.tile_elems)) return ZIPMOE_ERR_BAD_FORMAT;
      // every column holds exactly one backward stream
      uint32_t seen = 0;
      for (uint32_t lane = 0; lane < kLanes; ++lane) {
        const uint32_t c = chunk[r0 + lane];
        if (c >= kLanes || (seen >> c) & 1u) return ZIPMOE_ERR_BAD_FORMAT;
        seen |= 1u << c;
      }
      // a column has room for at least one bit per element of its two streams
      const uint32_t valid = g.tile_valid(q0 + t);
      const uint64_t col_bits = (r1 - r0 - kRecordHeadBytes) / kRowBytes * 32;
      uint32_t felems[kLanes], belems[kLanes];
      for (uint32_t lane = 0; lane < kLanes; ++lane) {
        felems[lane] = belems[lane] = 0;
        for (uint32_t i = 0; i < g.iters; ++i) {
          uint32_t pos = (i * kLanes + lane) * kGroup;
          if (pos < valid) ((i & 1) ? belems : felems)[lane] += std::min(kGroup, valid - pos);
        }
      }
      for (uint32_t lane = 0; lane < kLanes; ++lane)
        if (felems[chunk[r0 + lane]] + belems[lane] > col_bits) return ZIPMOE_ERR_BAD_FORMAT;
    }
    prev = next;
  }
  if (prev / 8 != info.payload_bytes) return ZIPMOE_ERR_BAD_FORMAT;
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_blob_plan(const void *blob_v, uint64_t bytes, uint64_t payload_base, uint64_t sm_base,
                               uint64_t out_base, uint32_t table_id, uint32_t chunk_base, uint32_t tile_base,
                               zipmoe_chunk_desc *descs, zipmoe_table *table) {
  zipmoe_blob_info info;
  zipmoe_status rc = zipmoe_blob_info_get(blob_v, bytes, &info);
  if (rc != ZIPMOE_OK) return rc;
  if ((!descs && info.n_chunks) || !table) return ZIPMOE_ERR_INVALID_ARG;
  if (payload_base % 16 || sm_base % 16 || out_base % 8) return ZIPMOE_ERR_INVALID_ARG;
  const uint8_t *blob = static_cast<const uint8_t *>(blob_v);
  Geometry g;
  make_geometry(info.rows, info.cols, info.layout, info.chunk_elems, &g);
  std::memcpy(table->code_len, blob + kTableOff, 256);
  // largest tile record of the tensor, from the chunks' tile tables
  uint32_t max_record = 0;
  for (uint32_t k = 0; k < g.n_chunks; ++k) {
    const uint64_t at = info.payload_off + load_le<uint64_t>(blob + kChunkOffOff + 8ull * k) / 8;
    const uint32_t m = g.chunk_tiles(k);
    if (at + 4ull * (m + 1) > info.payload_off + info.payload_bytes) return ZIPMOE_ERR_BAD_FORMAT;
    for (uint32_t t = 0; t < m; ++t) {
      const uint64_t o0 = load_le<uint32_t>(blob + at + 4ull * t), o1 = load_le<uint32_t>(blob + at + 4ull * (t + 1));
      // (a damaged tile table must not wrap this into a small hint that selects the narrow kernel)
      if (o1 < o0 || (o1 - o0) * 16 > tile_record_max(g.tile_elems)) return ZIPMOE_ERR_BAD_FORMAT;
      max_record = std::max(max_record, (uint32_t)((o1 - o0) * 16));
    }
  }
  for (uint32_t k = 0; k < g.n_chunks; ++k) {
    zipmoe_chunk_desc &d = descs[k];
    uint32_t q0 = k * g.tiles_per_chunk, m = g.chunk_tiles(k);
    d.payload_off = payload_base + load_le<uint64_t>(blob + kChunkOffOff + 8ull * k) / 8;
    d.sm_off = sm_base + (uint64_t)q0 * g.tile_elems;
    d.out_off = out_base;
    d.row_pitch = (uint32_t)g.row_pitch();
    d.tiles_per_rowblk = g.tiles_per_rowblk;
    d.tile0 = q0;
    d.n_tiles = m;
    d.tile_elems = g.tile_elems;
    d.last_tile_elems = g.tile_valid(q0 + m - 1);
    d.table_id = table_id;
    d.tile_prefix = tile_base + q0;
    d.run_first_chunk = chunk_base;
    d.run_first_tile = tile_base;
    d.run_end_tile = tile_base + g.n_tiles;
    d.tiles_per_chunk = g.tiles_per_chunk;
    d.max_record_bytes = max_record;
    d.reserved = 0;
  }
  return ZIPMOE_OK;
}

}  // extern "C"

// ---- planning one launch over several blobs ---------------------------------------------------
extern "C" {

zipmoe_status zipmoe_launch_plan_size(const void *const *blobs, const uint64_t *blob_bytes, uint32_t n_blobs,
                                      zipmoe_launch_info *info) {
  if (!info || (n_blobs && (!blobs || !blob_bytes))) return ZIPMOE_ERR_INVALID_ARG;
  zipmoe_launch_info li = {};
  for (uint32_t i = 0; i < n_blobs; ++i) {
    zipmoe_blob_info bi;
    zipmoe_status rc = zipmoe_blob_info_get(blobs[i], blob_bytes[i], &bi);
    if (rc != ZIPMOE_OK) return rc;
    li.payload_bytes += bi.payload_bytes;              // multiples of 16 by construction
    li.sm_bytes += align_up(bi.sm_bytes, 16);
    li.out_elems += align_up(bi.n_elems, 8);
    if ((uint64_t)li.n_chunks + bi.n_chunks > 0xFFFFFFFFull || (uint64_t)li.n_tiles + bi.n_tiles > 0xFFFFFFFFull)
      return ZIPMOE_ERR_UNSUPPORTED;
    li.n_chunks += bi.n_chunks;
    li.n_tiles += bi.n_tiles;
  }
  li.n_tables = n_blobs;
  *info = li;
  return ZIPMOE_OK;
}

zipmoe_status zipmoe_launch_plan(const void *const *blobs, const uint64_t *blob_bytes, uint32_t n_blobs, uint8_t *payload,
                                 uint8_t *sm, zipmoe_chunk_desc *descs, zipmoe_table *tables, uint32_t *tensor_first_chunk,
                                 uint64_t *out_base, zipmoe_launch_info *info) {
  zipmoe_launch_info li;
  zipmoe_status rc = zipmoe_launch_plan_size(blobs, blob_bytes, n_blobs, &li);
  if (rc != ZIPMOE_OK) return rc;
  if (!info || (n_blobs && (!payload || !sm || !tables)) || (li.n_chunks && !descs)) return ZIPMOE_ERR_INVALID_ARG;
  uint64_t pay = 0, smo = 0, out = 0;
  uint32_t chunk_base = 0, tile_base = 0;
  li.max_record_bytes = 0;
  li.max_code_len = 0;
  for (uint32_t i = 0; i < n_blobs; ++i) {
    const uint8_t *blob = static_cast<const uint8_t *>(blobs[i]);
    zipmoe_blob_info bi;
    zipmoe_blob_info_get(blob, blob_bytes[i], &bi);
    std::memcpy(payload + pay, blob + bi.payload_off, bi.payload_bytes);
    std::memcpy(sm + smo, blob + bi.sm_off, bi.sm_bytes);
    std::memset(sm + smo + bi.sm_bytes, 0, align_up(bi.sm_bytes, 16) - bi.sm_bytes);
    rc = zipmoe_blob_plan(blob, blob_bytes[i], pay, smo, out, i, chunk_base, tile_base, descs + chunk_base, tables + i);
    if (rc != ZIPMOE_OK) return rc;
    if (tensor_first_chunk) tensor_first_chunk[i] = chunk_base;
    if (out_base) out_base[i] = out;
    if (bi.n_chunks) li.max_record_bytes = std::max(li.max_record_bytes, descs[chunk_base].max_record_bytes);
    for (int s = 0; s < 256; ++s) li.max_code_len = std::max<uint32_t>(li.max_code_len, tables[i].code_len[s]);
    pay += bi.payload_bytes;
    smo += align_up(bi.sm_bytes, 16);
    out += align_up(bi.n_elems, 8);
    chunk_base += bi.n_chunks;
    tile_base += bi.n_tiles;
  }
  std::memset(payload + pay, 0, ZIPMOE_DEVICE_PAD_BYTES);
  std::memset(sm + smo, 0, ZIPMOE_DEVICE_PAD_BYTES);
  // the promise the fastest kernel variant wants holds exactly when the plan says so
  li.flags = (li.max_record_bytes > 0 && li.max_record_bytes <= ZIPMOE_NARROW_RECORD_BYTES && li.max_code_len <= 8)
                 ? ZIPMOE_DECODE_SHORT_CODES
                 : 0u;
  *info = li;
  return ZIPMOE_OK;
}

}  // extern "C"
