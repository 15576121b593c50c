// Internal view of the ZMOE v3 container shared by the library's host code
// (encoder, validator, planner).  Device code does not include this file: the
// kernels see only zipmoe_chunk_desc / zipmoe_table from the public header.
#pragma once
#include <cstdint>
#include <cstring>

#include "zipmoe.h"

namespace zipmoe {

constexpr uint32_t kMagic = 0x454F4D5Au;
constexpr uint32_t kVersion = 3;
constexpr uint64_t kHeaderBytes = 64;
constexpr uint64_t kTableOff = 64;
constexpr uint64_t kChunkOffOff = 320;
constexpr uint32_t kLanes = 32;
constexpr uint32_t kGroup = 8;          // elements per lane per iteration
constexpr uint32_t kIterElems = 256;    // kLanes * kGroup
constexpr uint32_t kRecordHeadBytes = 32;  // u8 bcol[32]: the column that holds each lane's backward stream
constexpr uint32_t kRowBytes = 128;        // one word of each of the 32 columns
constexpr uint32_t kMaxRows = 48;          // a column holds at most 128 codes of at most 12 bits

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

template <typename T>
inline T load_le(const uint8_t *p) {
  T v;
  std::memcpy(&v, p, sizeof(T));  // the library targets little-endian hosts only
  return v;
}
template <typename T>
inline void store_le(uint8_t *p, T v) {
  std::memcpy(p, &v, sizeof(T));
}

// Geometry derived from (rows, cols, layout, chunk_elems).
struct Geometry {
  uint64_t n_elems = 0;
  uint32_t rows = 0, cols = 0, layout = 0, chunk_elems = 0, tile_elems = 0;
  uint32_t iters = 0;            // tile_elems / 256
  uint32_t tiles_per_chunk = 0;
  uint32_t tiles_per_rowblk = 1; // cols / 256 for the blocked layout
  uint32_t n_tiles = 0, n_chunks = 0;
  uint64_t sm_bytes = 0;
  uint64_t payload_off = 0;

  // existing elements in tile q (only the last tile of a linear tensor is short)
  uint32_t tile_valid(uint32_t q) const {
    if (layout == ZIPMOE_LAYOUT_BLOCKED) return tile_elems;
    uint64_t lo = (uint64_t)q * tile_elems;
    uint64_t left = n_elems - lo;
    return left < tile_elems ? (uint32_t)left : tile_elems;
  }
  uint32_t chunk_tiles(uint32_t k) const {
    uint32_t q0 = k * tiles_per_chunk;
    uint32_t left = n_tiles - q0;
    return left < tiles_per_chunk ? left : tiles_per_chunk;
  }
  // flat index of the first element of iteration i of tile q, and the pitch between iterations
  uint64_t tile_origin(uint32_t q) const {
    if (layout == ZIPMOE_LAYOUT_BLOCKED) {
      uint64_t rb = q / tiles_per_rowblk, cb = q % tiles_per_rowblk;
      return rb * 16 * (uint64_t)cols + cb * 256;
    }
    return (uint64_t)q * tile_elems;
  }
  uint64_t row_pitch() const { return layout == ZIPMOE_LAYOUT_BLOCKED ? cols : kIterElems; }
};

zipmoe_status make_geometry(uint64_t rows, uint64_t cols, uint32_t layout, uint32_t chunk_elems, Geometry *g);

}  // namespace zipmoe
