// Sizes of the pieces in which a tile's sign+mantissa bytes travel from global to shared memory.
// Plain C++ that compiles for the host and for the device, so that the arithmetic the kernels rely on can
// be checked exhaustively on a CPU.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define ZIPMOE_HD __host__ __device__ __forceinline__
#else
#define ZIPMOE_HD inline
#endif

namespace zipmoe_dev {

constexpr uint32_t kPieceIters = 8;                 // iterations (rows of 256 elements) served by one piece
constexpr uint32_t kSmPieceBytes = kPieceIters * 256;
constexpr uint32_t kSmPieces = 16 / kPieceIters;    // pieces of a full tile = sign+mantissa slots of a warp

// A tile with `valid` existing elements (1..4096) has round16(valid) sign+mantissa bytes in its section
// (the section of a tensor is zero-padded to 16 bytes); they travel in pieces of kSmPieceBytes.
ZIPMOE_HD uint32_t sm_bytes_of_tile(uint32_t valid) { return (valid + 15u) & ~15u; }
ZIPMOE_HD uint32_t sm_pieces_of_tile(uint32_t valid) { return (sm_bytes_of_tile(valid) + kSmPieceBytes - 1) / kSmPieceBytes; }
// bytes of piece p (p < sm_pieces_of_tile(valid)): never zero, never past the tile's own bytes
ZIPMOE_HD uint32_t sm_piece_bytes(uint32_t valid, uint32_t p) {
  const uint32_t all = sm_bytes_of_tile(valid), at = p * kSmPieceBytes;
  if (at >= all) return 0;
  return all - at < kSmPieceBytes ? all - at : kSmPieceBytes;
}

}  // namespace zipmoe_dev
