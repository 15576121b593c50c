/*
 * zipmoe_oracle.c -- CPU oracle for the ZipMoE lossless bf16 expert codec.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow,
 * single-threaded restatement of what the decode path computes, written so
 * that it can be checked against the paper by eye.  It shares no code, table
 * or helper with the CUDA library; only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.
 *
 * What it follows:
 *   - bf16 fields (1 sign, 8 exponent, 7 mantissa bits): paper Section 2.2,
 *     "BF16 Parameters".
 *   - bit-field decomposition into an exponent stream and a sign+mantissa
 *     byte stream; exponent stream cut into K shards that are compressed
 *     independently (E-chunks); sign+mantissa kept as raw bytes (SM-chunks):
 *     paper Section 3.1, "Offline Initialization".
 *   - re-assembly of the two streams into bf16: paper Section 3.3,
 *     "Memory-Coalesced Tensor Recovery Kernel".
 *   - the compressor slot (the paper plugs LZ4/ZSTD in and leaves the API
 *     open, Section 6 "Other Compressors") is filled with an order-0
 *     canonical Huffman code over exponent bytes, the quantity the paper's
 *     own entropy analysis measures (Fig. 2, Fig. 3).
 *
 * The container layout ("ZMOE v3") is this project's own; it is written out
 * in full below because the decoder is defined by it.  Every function that
 * has an independent pin (closed form, brute force, textbook special case)
 * is pinned in tests/test_oracle_*.py.  The one part that cannot be pinned
 * against anything but itself is the byte-exact blob layout produced by
 * zo_encode (tie-breaks between equally good codes and the pairing of
 * streams into columns are free): "parity unpinned" for blob bytes; only
 * decodability and size bounds bind.
 *
 * ---------------------------------------------------------------------------
 * ZMOE v3 container (all integers little-endian)
 *
 *   offset  0  u32 magic 0x454F4D5A      4  u32 version (3)
 *           8  u64 n_elems              16  u32 rows     20 u32 cols
 *          24  u32 layout (0 linear, 1 blocked)          28 u32 chunk_elems
 *          32  u32 tile_elems           36  u32 max_code_len
 *          40  u32 n_chunks             44  u32 n_tiles
 *          48  u64 payload_bytes        56  u64 sm_bytes
 *          64  u8  code_len[256]        (0 = symbol unused)
 *         320  u64 chunk_bit_off[n_chunks + 1]   (bit offsets into the payload
 *                                                 section, multiples of 128)
 *         then zero padding to a 16-byte boundary, the payload section
 *         (payload_bytes) and the sign+mantissa section (sm_bytes).
 *
 *   A tile is 256*I elements (I = tile_elems/256, 1 <= I <= 16), seen as I
 *   "iterations" x 32 "lanes" x 8 elements.  Position pos = (i*32 + lane)*8 + j.
 *     linear  layout: tile q covers flat elements q*tile_elems + pos
 *                     (those >= n_elems do not exist).
 *     blocked layout: the tensor is rows x cols, rows % 16 == 0, cols % 256 == 0,
 *                     tile_elems = 4096; tile q is the 16 x 256 block with
 *                     rb = q / (cols/256), cb = q % (cols/256), and
 *                     flat = (rb*16 + i)*cols + cb*256 + lane*8 + j.
 *   Chunk k holds tiles [k*tpc, min((k+1)*tpc, n_tiles)), tpc = chunk_elems/tile_elems.
 *
 *   Chunk payload (at byte chunk_bit_off[k]/8 of the payload section):
 *     u32 tile_off[m + 1]   in 16-byte units from the chunk start (m = tiles
 *                           in the chunk); tile_off[0] is the padded size of
 *                           this table, tile_off[m] the size of the chunk;
 *     zero padding to 16 bytes, then m tile records.
 *   Tile record of W rows (32 + 128*W bytes; W >= 1 follows from the record's size):
 *     u8  bcol[32]          the column that holds lane L's backward stream:
 *                           a permutation of 0..31;
 *     u32 word[W][32]       row r, column c at byte 32 + (r*32 + c)*4.
 *   Column c is a string of 32*W bits: its bit y is bit 31 - (y mod 32) of
 *   word[y / 32][c].  Every lane has two code streams:
 *     the forward stream codes the lane's existing elements of the even
 *       iterations i = 0, 2, 4, ... < I (j = 0..7 inside each); its k-th bit is
 *       bit k of column `lane`;
 *     the backward stream codes those of the odd iterations i = 1, 3, 5, ... < I;
 *       its k-th bit is bit 32*W - 1 - k of column bcol[lane].
 *   The two streams that share a column must not overlap; the bits between
 *   their ends are zero.  (Word r of all 32 columns is one contiguous 128-byte
 *   row, so 32 readers that each follow one column touch 32 different
 *   addresses modulo 128 bytes whatever their positions; pairing a long
 *   forward stream with a short backward stream keeps W near the mean.  The
 *   paper leaves the order of elements inside a shard open.)  An encoder may
 *   choose any permutation and any W that fits; this oracle pairs the lanes in
 *   descending order of forward bits with the lanes in ascending order of
 *   backward bits and takes the smallest W.
 *
 *   Sign+mantissa section: byte q*tile_elems + pos holds
 *     (sign << 7) | mantissa  of the element at (q, pos); zero padded to 16.
 *
 *   Codes are canonical: symbols ordered by (length, symbol value) receive
 *   consecutive code values; the first code of length L+1 is
 *   (first code of length L + number of codes of length L) * 2.
 * ---------------------------------------------------------------------------
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ZO_OK 0
#define ZO_ERR_ARG (-1)
#define ZO_ERR_FORMAT (-2)
#define ZO_ERR_SPACE (-3)
#define ZO_ERR_CORRUPT (-4)

#define ZO_MAGIC 0x454F4D5Au
#define ZO_HEADER_BYTES 64u
#define ZO_TABLE_OFF 64u
#define ZO_CHUNKOFF_OFF 320u
#define ZO_MAX_CODE_LEN 12
#define ZO_VERSION 3u
#define ZO_REC_HEAD 32u /* u8 bcol[32] */
#define ZO_MAX_ROWS 48u /* 128 codes of at most 12 bits in a column */

/* ---- little-endian field access ---------------------------------------- */
static uint32_t rd32(const uint8_t *p) {
  return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24);
}
static uint64_t rd64(const uint8_t *p) { return (uint64_t)rd32(p) | ((uint64_t)rd32(p + 4) << 32); }
static void wr32(uint8_t *p, uint32_t v) {
  p[0] = (uint8_t)v; p[1] = (uint8_t)(v >> 8); p[2] = (uint8_t)(v >> 16); p[3] = (uint8_t)(v >> 24);
}
static void wr64(uint8_t *p, uint64_t v) { wr32(p, (uint32_t)v); wr32(p + 4, (uint32_t)(v >> 32)); }
static uint64_t round_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

/* ---- bit-field decomposition and re-assembly (Sections 2.2, 3.1, 3.3) -- */

/* A bf16 pattern b is sign(1) | exponent(8) | mantissa(7).  The exponent byte
 * is bits 14..7; the sign+mantissa byte keeps the sign in bit 7 and the
 * mantissa in bits 6..0.  Patterns are never interpreted as numbers. */
void zo_split(const uint16_t *x, uint64_t n, uint8_t *exp, uint8_t *sm) {
  for (uint64_t k = 0; k < n; ++k) {
    uint16_t b = x[k];
    exp[k] = (uint8_t)((b >> 7) & 0xFF);
    sm[k] = (uint8_t)(((b >> 8) & 0x80) | (b & 0x7F));
  }
}

void zo_merge(const uint8_t *exp, const uint8_t *sm, uint64_t n, uint16_t *x) {
  for (uint64_t k = 0; k < n; ++k)
    x[k] = (uint16_t)((((uint16_t)sm[k] & 0x80) << 8) | ((uint16_t)exp[k] << 7) | (sm[k] & 0x7F));
}

void zo_histogram(const uint8_t *exp, uint64_t n, uint64_t *hist) {
  memset(hist, 0, 256 * sizeof(uint64_t));
  for (uint64_t k = 0; k < n; ++k) hist[exp[k]]++;
}

/* ---- optimal length-limited prefix code (package-merge) ---------------- */

typedef struct {
  uint64_t w;        /* total weight of the leaves inside the item */
  uint8_t cnt[256];  /* how many times each symbol's leaf is inside */
} zo_item;

static int item_less(const zo_item *a, const zo_item *b, int a_is_leaf, int b_is_leaf) {
  /* order by weight; at equal weight a leaf goes before a package (this keeps
   * the total cost minimal and the maximum length small; any rule is valid) */
  if (a->w != b->w) return a->w < b->w;
  return a_is_leaf && !b_is_leaf;
}

/* Code lengths minimising sum(hist[s] * len[s]) subject to len <= max_len and
 * Kraft equality.  Degenerate histograms: no symbol -> all lengths 0; one
 * symbol s -> s and (s+1) mod 256 get length 1 each, so that the code is
 * still complete and every element costs one bit. */
int zo_code_lengths(const uint64_t *hist, int max_len, uint8_t *len) {
  int sym[256], m = 0;
  memset(len, 0, 256);
  if (max_len < 1 || max_len > ZO_MAX_CODE_LEN) return ZO_ERR_ARG;
  for (int s = 0; s < 256; ++s)
    if (hist[s]) sym[m++] = s;
  if (m == 0) return ZO_OK;
  if (m == 1) {
    len[sym[0]] = 1;
    len[(sym[0] + 1) & 0xFF] = 1;
    return ZO_OK;
  }
  if (((uint64_t)1 << max_len) < (uint64_t)m) return ZO_ERR_ARG;

  /* leaves sorted by (weight, symbol) ascending: insertion sort, m <= 256 */
  for (int a = 1; a < m; ++a) {
    int s = sym[a], b = a - 1;
    while (b >= 0 && hist[sym[b]] > hist[s]) { sym[b + 1] = sym[b]; --b; }
    sym[b + 1] = s;
  }

  zo_item *prev = (zo_item *)calloc(512, sizeof(zo_item));
  zo_item *cur = (zo_item *)calloc(512, sizeof(zo_item));
  zo_item *pack = (zo_item *)calloc(256, sizeof(zo_item));
  if (!prev || !cur || !pack) { free(prev); free(cur); free(pack); return ZO_ERR_SPACE; }

  /* the list for the smallest coin (2^-max_len) is the leaves alone */
  int n_prev = m;
  for (int a = 0; a < m; ++a) {
    memset(&prev[a], 0, sizeof(zo_item));
    prev[a].w = hist[sym[a]];
    prev[a].cnt[sym[a]] = 1;
  }
  for (int level = 2; level <= max_len; ++level) {
    /* package: pair up neighbours of the previous list, dropping an odd last */
    int n_pack = n_prev / 2;
    for (int a = 0; a < n_pack; ++a) {
      pack[a].w = prev[2 * a].w + prev[2 * a + 1].w;
      for (int s = 0; s < 256; ++s) pack[a].cnt[s] = (uint8_t)(prev[2 * a].cnt[s] + prev[2 * a + 1].cnt[s]);
    }
    /* merge: the leaves again, together with the packages, by weight */
    int ia = 0, ib = 0, n_cur = 0;
    zo_item leaf;
    while (ia < m || ib < n_pack) {
      int take_leaf;
      if (ia < m) {
        memset(&leaf, 0, sizeof leaf);
        leaf.w = hist[sym[ia]];
        leaf.cnt[sym[ia]] = 1;
      }
      if (ia >= m) take_leaf = 0;
      else if (ib >= n_pack) take_leaf = 1;
      else take_leaf = !item_less(&pack[ib], &leaf, 0, 1);
      if (take_leaf) { cur[n_cur++] = leaf; ++ia; }
      else { cur[n_cur++] = pack[ib]; ++ib; }
    }
    zo_item *t = prev; prev = cur; cur = t;
    n_prev = n_cur;
  }
  /* the 2m-2 cheapest items of the largest coin's list buy total width m-1;
   * a symbol's length is the number of chosen items its leaf sits in */
  int take = 2 * m - 2;
  if (take > n_prev) { free(prev); free(cur); free(pack); return ZO_ERR_ARG; }
  for (int a = 0; a < take; ++a)
    for (int s = 0; s < 256; ++s) len[s] = (uint8_t)(len[s] + prev[a].cnt[s]);
  free(prev); free(cur); free(pack);
  return ZO_OK;
}

/* Canonical code values from lengths.  Returns ZO_ERR_FORMAT unless the
 * lengths form a complete prefix code (Kraft sum exactly 1) or are all 0. */
int zo_canonical_codes(const uint8_t *len, uint32_t *code) {
  uint32_t count[ZO_MAX_CODE_LEN + 2] = {0}, next[ZO_MAX_CODE_LEN + 2] = {0};
  uint64_t kraft = 0;
  int used = 0;
  for (int s = 0; s < 256; ++s) {
    code[s] = 0;
    if (len[s] > ZO_MAX_CODE_LEN) return ZO_ERR_FORMAT;
    if (len[s]) {
      count[len[s]]++;
      kraft += (uint64_t)1 << (ZO_MAX_CODE_LEN - len[s]);
      used++;
    }
  }
  if (used == 0) return ZO_OK;
  if (kraft != ((uint64_t)1 << ZO_MAX_CODE_LEN)) return ZO_ERR_FORMAT;
  uint32_t c = 0;
  for (int L = 1; L <= ZO_MAX_CODE_LEN; ++L) {
    next[L] = c;
    c = (c + count[L]) << 1;
  }
  for (int s = 0; s < 256; ++s)
    if (len[s]) code[s] = next[len[s]]++;
  return ZO_OK;
}

/* ---- container geometry ------------------------------------------------- */

typedef struct {
  uint64_t n_elems;
  uint32_t rows, cols, layout, chunk_elems, tile_elems, max_code_len, n_chunks, n_tiles;
  uint64_t payload_bytes, sm_bytes;
  uint64_t payload_off, sm_off, total_bytes; /* derived */
} zo_header;

static int geometry(uint64_t rows, uint64_t cols, uint32_t layout, uint32_t chunk_elems, zo_header *h) {
  memset(h, 0, sizeof *h);
  if (rows > 0xFFFFFFFFu || cols > 0xFFFFFFFFu) return ZO_ERR_ARG;
  if (chunk_elems == 0 || chunk_elems % 256) return ZO_ERR_ARG;
  if (chunk_elems > 4096 && chunk_elems % 4096) return ZO_ERR_ARG;
  h->n_elems = rows * cols;
  h->rows = (uint32_t)rows;
  h->cols = (uint32_t)cols;
  h->layout = layout;
  h->chunk_elems = chunk_elems;
  h->tile_elems = chunk_elems < 4096 ? chunk_elems : 4096;
  if (layout == 0) {
    uint64_t t = (h->n_elems + h->tile_elems - 1) / h->tile_elems;
    if (t > 0xFFFFFFFFu) return ZO_ERR_ARG;
    h->n_tiles = (uint32_t)t;
    h->sm_bytes = round_up(h->n_elems, 16);
  } else if (layout == 1) {
    if (h->tile_elems != 4096 || rows % 16 || cols % 256) return ZO_ERR_ARG;
    h->n_tiles = (uint32_t)((rows / 16) * (cols / 256));
    h->sm_bytes = h->n_elems;
  } else {
    return ZO_ERR_ARG;
  }
  uint32_t tpc = h->chunk_elems / h->tile_elems;
  h->n_chunks = (h->n_tiles + tpc - 1) / tpc;
  h->payload_off = round_up(ZO_CHUNKOFF_OFF + 8ull * (h->n_chunks + 1), 16);
  return ZO_OK;
}

/* flat element index of (tile q, position pos), or UINT64_MAX if the element
 * does not exist (linear layout, past the end of the tensor) */
static uint64_t elem_of(const zo_header *h, uint64_t q, uint32_t pos) {
  if (h->layout == 0) {
    uint64_t f = q * h->tile_elems + pos;
    return f < h->n_elems ? f : UINT64_MAX;
  }
  uint32_t tpr = h->cols / 256;
  uint64_t rb = q / tpr, cb = q % tpr;
  uint32_t i = pos / 256, within = pos % 256;
  return (rb * 16 + i) * (uint64_t)h->cols + cb * 256 + within;
}

uint64_t zo_encode_bound(uint64_t rows, uint64_t cols, uint32_t layout, uint32_t chunk_elems) {
  zo_header h;
  if (geometry(rows, cols, layout, chunk_elems, &h) != ZO_OK) return 0;
  uint64_t per_tile = ZO_REC_HEAD + 128ull * ZO_MAX_ROWS;
  uint64_t tpc = h.chunk_elems / h.tile_elems;
  uint64_t per_chunk = round_up(4 * (tpc + 1), 16);
  return h.payload_off + h.n_tiles * per_tile + h.n_chunks * per_chunk + h.sm_bytes + 64;
}

/* ---- bit access: bit y of column c of a tile record (see the layout above) -- */
static uint8_t *column_word(const uint8_t *rec, uint32_t c, uint64_t y) {
  return (uint8_t *)rec + ZO_REC_HEAD + ((y >> 5) * 32 + c) * 4;
}
static void put_bit(uint8_t *rec, uint32_t c, uint64_t y, uint32_t bit) {
  uint8_t *w = column_word(rec, c, y);
  uint32_t at = 31 - (uint32_t)(y & 31);
  wr32(w, (rd32(w) & ~((uint32_t)1 << at)) | ((bit & 1u) << at));
}
static uint32_t get_bit(const uint8_t *rec, uint32_t c, uint64_t y) {
  return (rd32(column_word(rec, c, y)) >> (31 - (uint32_t)(y & 31))) & 1u;
}

/* ---- encoder ------------------------------------------------------------ */

int zo_encode(const uint16_t *x, uint64_t rows, uint64_t cols, uint32_t layout, uint32_t chunk_elems,
              int max_code_len, uint8_t *blob, uint64_t cap, uint64_t *blob_bytes) {
  zo_header h;
  int rc = geometry(rows, cols, layout, chunk_elems, &h);
  if (rc != ZO_OK) return rc;
  if (max_code_len < 8 || max_code_len > ZO_MAX_CODE_LEN) return ZO_ERR_ARG;
  h.max_code_len = (uint32_t)max_code_len;
  uint64_t n = h.n_elems;
  if (cap < zo_encode_bound(rows, cols, layout, chunk_elems)) return ZO_ERR_SPACE;

  uint8_t *exp = (uint8_t *)malloc(n ? n : 1), *sm = (uint8_t *)malloc(n ? n : 1);
  if (!exp || !sm) { free(exp); free(sm); return ZO_ERR_SPACE; }
  zo_split(x, n, exp, sm);

  uint64_t hist[256];
  uint8_t len[256];
  uint32_t code[256];
  zo_histogram(exp, n, hist);
  rc = zo_code_lengths(hist, max_code_len, len);
  if (rc == ZO_OK) rc = zo_canonical_codes(len, code);
  if (rc != ZO_OK) { free(exp); free(sm); return rc; }

  memset(blob, 0, cap < h.payload_off ? cap : h.payload_off);
  memcpy(blob + ZO_TABLE_OFF, len, 256);

  uint8_t *pay = blob + h.payload_off;
  uint64_t at = 0; /* byte position in the payload section */
  uint32_t I = h.tile_elems / 256, tpc = h.chunk_elems / h.tile_elems;
  for (uint32_t k = 0; k < h.n_chunks; ++k) {
    uint32_t q0 = k * tpc, q1 = q0 + tpc < h.n_tiles ? q0 + tpc : h.n_tiles, m = q1 - q0;
    wr64(blob + ZO_CHUNKOFF_OFF + 8ull * k, at * 8);
    uint8_t *chunk = pay + at;
    uint64_t table_bytes = round_up(4ull * (m + 1), 16);
    memset(chunk, 0, table_bytes);
    uint64_t rel = table_bytes; /* byte position inside the chunk */
    for (uint32_t t = 0; t < m; ++t) {
      uint64_t q = (uint64_t)q0 + t;
      wr32(chunk + 4ull * t, (uint32_t)(rel / 16));
      uint8_t *rec = chunk + rel;
      /* code bits of every lane's forward stream (even iterations) and backward stream (odd iterations) */
      uint64_t fbits[32], bbits[32];
      for (uint32_t lane = 0; lane < 32; ++lane) {
        fbits[lane] = bbits[lane] = 0;
        for (uint32_t i = 0; i < I; ++i)
          for (uint32_t j = 0; j < 8; ++j) {
            uint64_t f = elem_of(&h, q, (i * 32 + lane) * 8 + j);
            if (f == UINT64_MAX) continue;
            if (i % 2 == 0) fbits[lane] += len[exp[f]];
            else bbits[lane] += len[exp[f]];
          }
      }
      /* pairing: the column with the k-th longest forward stream takes the k-th shortest backward stream
       * (ties by lane number); any permutation would be valid, this one keeps the columns level */
      uint32_t by_f[32], by_b[32], bcol[32];
      for (uint32_t a = 0; a < 32; ++a) by_f[a] = by_b[a] = a;
      for (uint32_t a = 1; a < 32; ++a)
        for (uint32_t b = a; b > 0; --b) {
          if (fbits[by_f[b]] > fbits[by_f[b - 1]]) { uint32_t t2 = by_f[b]; by_f[b] = by_f[b - 1]; by_f[b - 1] = t2; }
          if (bbits[by_b[b]] < bbits[by_b[b - 1]]) { uint32_t t2 = by_b[b]; by_b[b] = by_b[b - 1]; by_b[b - 1] = t2; }
        }
      uint64_t W = 1;
      for (uint32_t a = 0; a < 32; ++a) {
        bcol[by_b[a]] = by_f[a];
        uint64_t need = (fbits[by_f[a]] + bbits[by_b[a]] + 31) / 32;
        if (need > W) W = need;
      }
      if (W > ZO_MAX_ROWS) { free(exp); free(sm); return ZO_ERR_ARG; }
      uint64_t rec_bytes = ZO_REC_HEAD + 128 * W;
      memset(rec, 0, rec_bytes);
      for (uint32_t lane = 0; lane < 32; ++lane) rec[lane] = (uint8_t)bcol[lane];
      for (uint32_t lane = 0; lane < 32; ++lane) {
        uint64_t fwd = 0, bwd = 32 * W; /* next bit of the forward stream; one past the next bit of the backward stream */
        for (uint32_t i = 0; i < I; ++i)
          for (uint32_t j = 0; j < 8; ++j) {
            uint64_t f = elem_of(&h, q, (i * 32 + lane) * 8 + j);
            if (f == UINT64_MAX) continue;
            uint32_t sy = exp[f];
            for (int b = len[sy] - 1; b >= 0; --b) {
              if (i % 2 == 0) put_bit(rec, lane, fwd++, (code[sy] >> b) & 1u);
              else put_bit(rec, bcol[lane], --bwd, (code[sy] >> b) & 1u);
            }
          }
      }
      rel += rec_bytes;
    }
    wr32(chunk + 4ull * m, (uint32_t)(rel / 16));
    at += rel;
  }
  wr64(blob + ZO_CHUNKOFF_OFF + 8ull * h.n_chunks, at * 8);
  h.payload_bytes = at;
  h.sm_off = h.payload_off + h.payload_bytes;
  h.total_bytes = h.sm_off + h.sm_bytes;

  uint8_t *smsec = blob + h.sm_off;
  memset(smsec, 0, h.sm_bytes);
  for (uint64_t q = 0; q < h.n_tiles; ++q)
    for (uint32_t pos = 0; pos < h.tile_elems; ++pos) {
      uint64_t f = elem_of(&h, q, pos);
      if (f != UINT64_MAX) smsec[q * h.tile_elems + pos] = sm[f];
    }

  wr32(blob + 0, ZO_MAGIC);
  wr32(blob + 4, ZO_VERSION);
  wr64(blob + 8, h.n_elems);
  wr32(blob + 16, h.rows);
  wr32(blob + 20, h.cols);
  wr32(blob + 24, h.layout);
  wr32(blob + 28, h.chunk_elems);
  wr32(blob + 32, h.tile_elems);
  wr32(blob + 36, h.max_code_len);
  wr32(blob + 40, h.n_chunks);
  wr32(blob + 44, h.n_tiles);
  wr64(blob + 48, h.payload_bytes);
  wr64(blob + 56, h.sm_bytes);
  *blob_bytes = h.total_bytes;
  free(exp); free(sm);
  return ZO_OK;
}

/* ---- decoder ------------------------------------------------------------ */

static int parse_header(const uint8_t *blob, uint64_t bytes, zo_header *h) {
  if (bytes < ZO_CHUNKOFF_OFF + 8) return ZO_ERR_FORMAT;
  if (rd32(blob) != ZO_MAGIC || rd32(blob + 4) != ZO_VERSION) return ZO_ERR_FORMAT;
  zo_header g;
  uint64_t n = rd64(blob + 8);
  uint32_t rows = rd32(blob + 16), cols = rd32(blob + 20);
  if ((uint64_t)rows * cols != n) return ZO_ERR_FORMAT;
  if (geometry(rows, cols, rd32(blob + 24), rd32(blob + 28), &g) != ZO_OK) return ZO_ERR_FORMAT;
  if (g.tile_elems != rd32(blob + 32) || g.n_chunks != rd32(blob + 40) || g.n_tiles != rd32(blob + 44))
    return ZO_ERR_FORMAT;
  g.max_code_len = rd32(blob + 36);
  if (g.max_code_len < 1 || g.max_code_len > ZO_MAX_CODE_LEN) return ZO_ERR_FORMAT;
  g.payload_bytes = rd64(blob + 48);
  if (g.sm_bytes != rd64(blob + 56)) return ZO_ERR_FORMAT;
  if (g.payload_bytes % 16) return ZO_ERR_FORMAT;
  g.sm_off = g.payload_off + g.payload_bytes;
  g.total_bytes = g.sm_off + g.sm_bytes;
  if (g.total_bytes > bytes || g.sm_off < g.payload_off) return ZO_ERR_FORMAT;
  *h = g;
  return ZO_OK;
}

/* Decode chunk k into its place in the full tensor `out` (n_elems entries).
 * One code bit at a time: extend the code value until it falls inside the
 * range of codes of the current length (first code, count), then look the
 * symbol up in the (length, symbol)-ordered list. */
int zo_decode_chunk(const uint8_t *blob, uint64_t bytes, uint32_t k, uint16_t *out) {
  zo_header h;
  int rc = parse_header(blob, bytes, &h);
  if (rc != ZO_OK) return rc;
  if (k >= h.n_chunks) return ZO_ERR_ARG;

  const uint8_t *len = blob + ZO_TABLE_OFF;
  uint32_t count[ZO_MAX_CODE_LEN + 2] = {0}, first[ZO_MAX_CODE_LEN + 2] = {0}, base[ZO_MAX_CODE_LEN + 2] = {0};
  uint8_t order[256];
  uint32_t code_unused[256];
  if (zo_canonical_codes(len, code_unused) != ZO_OK) return ZO_ERR_FORMAT;
  for (int s = 0; s < 256; ++s) {
    if (len[s] > h.max_code_len) return ZO_ERR_FORMAT;
    if (len[s]) count[len[s]]++;
  }
  {
    uint32_t c = 0, b = 0;
    for (int L = 1; L <= ZO_MAX_CODE_LEN; ++L) {
      first[L] = c; base[L] = b;
      c = (c + count[L]) << 1;
      b += count[L];
    }
    uint32_t fill[ZO_MAX_CODE_LEN + 2];
    memcpy(fill, base, sizeof fill);
    for (int s = 0; s < 256; ++s)
      if (len[s]) order[fill[len[s]]++] = (uint8_t)s;
  }

  uint64_t off0 = rd64(blob + ZO_CHUNKOFF_OFF + 8ull * k), off1 = rd64(blob + ZO_CHUNKOFF_OFF + 8ull * (k + 1));
  if (off0 % 128 || off1 % 128 || off1 < off0 || off1 / 8 > h.payload_bytes) return ZO_ERR_CORRUPT;
  const uint8_t *chunk = blob + h.payload_off + off0 / 8;
  uint64_t chunk_bytes = (off1 - off0) / 8;

  uint32_t I = h.tile_elems / 256, tpc = h.chunk_elems / h.tile_elems;
  uint32_t q0 = k * tpc, q1 = q0 + tpc < h.n_tiles ? q0 + tpc : h.n_tiles, m = q1 - q0;
  if (round_up(4ull * (m + 1), 16) > chunk_bytes) return ZO_ERR_CORRUPT;
  if ((uint64_t)rd32(chunk + 4ull * m) * 16 != chunk_bytes) return ZO_ERR_CORRUPT;
  const uint8_t *smsec = blob + h.sm_off;

  for (uint32_t t = 0; t < m; ++t) {
    uint64_t q = (uint64_t)q0 + t;
    uint64_t r0 = (uint64_t)rd32(chunk + 4ull * t) * 16, r1 = (uint64_t)rd32(chunk + 4ull * (t + 1)) * 16;
    if (r1 < r0 + ZO_REC_HEAD + 128 || r1 > chunk_bytes || (r1 - r0 - ZO_REC_HEAD) % 128) return ZO_ERR_CORRUPT;
    const uint8_t *rec = chunk + r0;
    uint64_t W = (r1 - r0 - ZO_REC_HEAD) / 128;
    if (W > ZO_MAX_ROWS) return ZO_ERR_CORRUPT;
    /* bcol must be a permutation: every column holds exactly one backward stream */
    uint32_t owner[32]; /* the lane whose backward stream lives in column c */
    for (uint32_t c = 0; c < 32; ++c) owner[c] = 32;
    for (uint32_t lane = 0; lane < 32; ++lane) {
      uint32_t c = rec[lane];
      if (c >= 32 || owner[c] != 32) return ZO_ERR_CORRUPT;
      owner[c] = lane;
    }
    uint64_t fwd_end[32], bwd_end[32]; /* per lane: bits its forward stream used; first bit its backward stream used */
    for (uint32_t lane = 0; lane < 32; ++lane) {
      uint32_t bc = rec[lane];
      uint64_t fwd = 0, bwd = 32 * W;
      for (uint32_t i = 0; i < I; ++i)
        for (uint32_t j = 0; j < 8; ++j) {
          uint32_t pos = (i * 32 + lane) * 8 + j;
          uint64_t f = elem_of(&h, q, pos);
          if (f == UINT64_MAX) continue;
          uint32_t c = 0;
          int L = 0, found = 0;
          while (L < (int)h.max_code_len) {
            uint32_t bit;
            if (i % 2 == 0) {
              if (fwd >= 32 * W) return ZO_ERR_CORRUPT; /* the column is used up */
              bit = get_bit(rec, lane, fwd++);
            } else {
              if (bwd == 0) return ZO_ERR_CORRUPT;
              bit = get_bit(rec, bc, --bwd);
            }
            c = (c << 1) | bit;
            ++L;
            if (c >= first[L] && c - first[L] < count[L]) { found = 1; break; }
          }
          if (!found) return ZO_ERR_CORRUPT;
          uint8_t e = order[base[L] + (c - first[L])];
          uint8_t sb = smsec[q * h.tile_elems + pos];
          zo_merge(&e, &sb, 1, &out[f]);
        }
      fwd_end[lane] = fwd;
      bwd_end[lane] = bwd;
    }
    /* the two streams of a column must not overlap, and what lies between them is zero */
    for (uint32_t c = 0; c < 32; ++c) {
      uint64_t lo = fwd_end[c], hi = bwd_end[owner[c]];
      if (lo > hi) return ZO_ERR_CORRUPT;
      for (uint64_t g = lo; g < hi; ++g)
        if (get_bit(rec, c, g)) return ZO_ERR_CORRUPT;
    }
  }
  return ZO_OK;
}

int zo_decode(const uint8_t *blob, uint64_t bytes, uint16_t *out) {
  zo_header h;
  int rc = parse_header(blob, bytes, &h);
  if (rc != ZO_OK) return rc;
  for (uint32_t k = 0; k < h.n_chunks; ++k) {
    rc = zo_decode_chunk(blob, bytes, k, out);
    if (rc != ZO_OK) return rc;
  }
  return ZO_OK;
}

/* header fields, for tests: fills 12 u64 values
 * {n_elems, rows, cols, layout, chunk_elems, tile_elems, max_code_len,
 *  n_chunks, n_tiles, payload_bytes, sm_bytes, payload_off} */
int zo_info(const uint8_t *blob, uint64_t bytes, uint64_t *v) {
  zo_header h;
  int rc = parse_header(blob, bytes, &h);
  if (rc != ZO_OK) return rc;
  v[0] = h.n_elems; v[1] = h.rows; v[2] = h.cols; v[3] = h.layout; v[4] = h.chunk_elems; v[5] = h.tile_elems;
  v[6] = h.max_code_len; v[7] = h.n_chunks; v[8] = h.n_tiles; v[9] = h.payload_bytes; v[10] = h.sm_bytes;
  v[11] = h.payload_off;
  return ZO_OK;
}
