// Exhaustive host-side check of the piece arithmetic the decode kernels use for a tile's sign+mantissa bytes
// (paper_2601_21198_b200/csrc/tile_geometry.h): for every number of existing elements of a tile, the pieces
// cover exactly the tile's round16(valid) bytes, none is empty, and none reaches past them.
#include <cstdio>

#include "tile_geometry.h"

int main() {
  using namespace zipmoe_dev;
  for (uint32_t valid = 1; valid <= 4096; ++valid) {
    const uint32_t all = (valid + 15u) / 16u * 16u;
    const uint32_t n = sm_pieces_of_tile(valid);
    if (n < 1 || n > kSmPieces) return std::printf("valid %u: %u pieces\n", valid, n), 1;
    uint32_t sum = 0;
    for (uint32_t p = 0; p < n; ++p) {
      const uint32_t b = sm_piece_bytes(valid, p);
      if (b == 0 || b % 16 || b > kSmPieceBytes) return std::printf("valid %u piece %u: %u bytes\n", valid, p, b), 1;
      if (p * kSmPieceBytes + b > all) return std::printf("valid %u piece %u overruns\n", valid, p), 1;
      sum += b;
    }
    if (sum != all || sm_piece_bytes(valid, n) != 0) return std::printf("valid %u: pieces sum to %u of %u\n", valid, sum, all), 1;
  }
  std::puts("ok");
  return 0;
}
