/* A caller of include/zipmoe.h that knows no Python: encodes two tensors, validates the blobs, lays them out for
 * one launch with zipmoe_launch_plan and checks what came back.  Host functions only (no GPU needed). */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "zipmoe.h"

#define CHECK(cond)                                              \
  do {                                                           \
    if (!(cond)) {                                               \
      printf("line %d: %s\n", __LINE__, #cond);                  \
      return 1;                                                  \
    }                                                            \
  } while (0)

static uint32_t lcg(uint32_t *s) { return *s = *s * 1664525u + 1013904223u; }

int main(void) {
  enum { N0 = 5 * 4099, ROWS1 = 32, COLS1 = 512 };
  uint16_t *x0 = malloc(2 * N0), *x1 = malloc(2 * ROWS1 * COLS1);
  uint32_t seed = 7;
  for (int i = 0; i < N0; ++i) x0[i] = (uint16_t)(((lcg(&seed) >> 31) << 15) | ((118 + (lcg(&seed) >> 30)) << 7) | (lcg(&seed) >> 25));
  for (int i = 0; i < ROWS1 * COLS1; ++i) x1[i] = (uint16_t)(((120 + (lcg(&seed) >> 29)) << 7) | (lcg(&seed) >> 25));

  zipmoe_encode_opts o0 = {16384, 0, ZIPMOE_LAYOUT_LINEAR, 1}, o1 = {8192, 12, ZIPMOE_LAYOUT_BLOCKED, 2};
  uint64_t cap0 = 0, cap1 = 0, n0 = 0, n1 = 0;
  CHECK(zipmoe_encode_bound(1, N0, &o0, &cap0) == ZIPMOE_OK && zipmoe_encode_bound(ROWS1, COLS1, &o1, &cap1) == ZIPMOE_OK);
  void *b0 = malloc(cap0), *b1 = malloc(cap1);
  CHECK(zipmoe_encode(x0, 1, N0, &o0, b0, cap0, &n0) == ZIPMOE_OK);
  CHECK(zipmoe_encode(x1, ROWS1, COLS1, &o1, b1, cap1, &n1) == ZIPMOE_OK);
  CHECK(zipmoe_blob_validate(b0, n0) == ZIPMOE_OK && zipmoe_blob_validate(b1, n1) == ZIPMOE_OK);
  CHECK(n0 < 2ull * N0 && n1 < 2ull * ROWS1 * COLS1);   /* smaller than the tensors */

  const void *blobs[2] = {b0, b1};
  uint64_t sizes[2] = {n0, n1};
  zipmoe_launch_info li;
  CHECK(zipmoe_launch_plan_size(blobs, sizes, 2, &li) == ZIPMOE_OK);
  CHECK(li.n_chunks == 2 + 2 && li.n_tiles == 6 + 4 && li.n_tables == 2);
  CHECK(li.out_elems == (uint64_t)((N0 + 7) / 8 * 8) + ROWS1 * COLS1 && li.sm_bytes == (uint64_t)((N0 + 15) / 16 * 16) + ROWS1 * COLS1);

  uint8_t *payload = malloc(li.payload_bytes + ZIPMOE_DEVICE_PAD_BYTES), *sm = malloc(li.sm_bytes + ZIPMOE_DEVICE_PAD_BYTES);
  zipmoe_chunk_desc *descs = calloc(li.n_chunks, sizeof *descs);
  zipmoe_table tables[2];
  uint32_t first[2];
  uint64_t out_base[2];
  zipmoe_launch_info full;
  CHECK(zipmoe_launch_plan(blobs, sizes, 2, payload, sm, descs, tables, first, out_base, &full) == ZIPMOE_OK);
  CHECK(full.payload_bytes == li.payload_bytes && full.n_tiles == li.n_tiles);
  CHECK(first[0] == 0 && first[1] == 2 && out_base[0] == 0 && out_base[1] == (uint64_t)((N0 + 7) / 8 * 8));
  CHECK(full.max_code_len >= 1 && full.max_code_len <= 12 && full.max_record_bytes >= 32 + 128);
  CHECK(full.flags == ((full.max_code_len <= 8 && full.max_record_bytes <= ZIPMOE_NARROW_RECORD_BYTES) ? ZIPMOE_DECODE_SHORT_CODES : 0u));
  uint32_t tiles = 0;
  for (uint32_t c = 0; c < full.n_chunks; ++c) {
    const zipmoe_chunk_desc *d = &descs[c];
    CHECK(d->tile_prefix == tiles && d->table_id == (c < 2 ? 0u : 1u) && d->run_first_chunk == (c < 2 ? 0u : 2u));
    CHECK(d->payload_off % 16 == 0 && d->sm_off % 16 == 0 && d->out_off == out_base[d->table_id]);
    CHECK(d->payload_off < full.payload_bytes && d->sm_off < full.sm_bytes);
    CHECK(d->row_pitch == (c < 2 ? 256u : (uint32_t)COLS1) && d->tiles_per_rowblk == (c < 2 ? 1u : 2u));
    tiles += d->n_tiles;
  }
  CHECK(tiles == full.n_tiles && descs[1].last_tile_elems == (uint32_t)(N0 - 5 * 4096));
  /* the sign+mantissa bytes of the linear tensor are in element order; the pad after the buffers is zero */
  for (int i = 0; i < N0; ++i) CHECK(sm[i] == (uint8_t)(((x0[i] >> 8) & 0x80) | (x0[i] & 0x7F)));
  for (uint32_t i = 0; i < ZIPMOE_DEVICE_PAD_BYTES; ++i) CHECK(payload[full.payload_bytes + i] == 0 && sm[full.sm_bytes + i] == 0);
  /* a damaged blob is refused by the planner too */
  ((uint8_t *)b1)[4] ^= 1;
  CHECK(zipmoe_launch_plan_size(blobs, sizes, 2, &li) == ZIPMOE_ERR_BAD_FORMAT);
  puts("ok");
  return 0;
}
