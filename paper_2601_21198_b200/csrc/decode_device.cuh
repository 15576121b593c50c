// Device-side building blocks of the decoder, shared by the bulk decode kernel
// and the fused decode+FFN kernels: PTX wrappers (mbarrier, bulk async copy,
// shared-memory loads), the per-table lookup-table builder, and the warp-level
// tile decoder.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdint>
#include <type_traits>

#include "zipmoe.h"
#include "tile_geometry.h"

namespace zipmoe_dev {

// One of two lookup tables per Huffman code, in the same shared-memory region:
//  * a code whose longest length is at most 8 bits gets the lane table: indexed
//    by the next 8 code bits and replicated for each of the 32 lanes, entry
//    (v, lane) at word v*32 + lane, so that lane l only ever touches bank l and
//    the data-dependent lookups of a warp are free of bank conflicts;
//  * any other code gets the wide table: one copy, indexed by the next 12 bits.
// Entry = (symbol << 23) | length in both: the symbol sits where the exponent
// field of the upper bf16 of a pair goes, the length in the low bits, and the
// bits between are zero, so that sums of entries carry the sum of the lengths
// in their low 23 bits whatever the symbols are.
constexpr int kLaneLutBits = 8;
constexpr int kLaneLutBytes = (1 << kLaneLutBits) * 32 * 4;   // 32 KB
constexpr int kWideLutBits = ZIPMOE_MAX_CODE_LEN;
constexpr int kWideLutEntries = 1 << kWideLutBits;
constexpr int kWideLutBytes = kWideLutEntries * 4;            // 16 KB
constexpr int kLutBytes = kLaneLutBytes;                      // the wide table overlays the lane table
constexpr int kLutScratchBytes = 256 + 16 * 4 + 8 * 16 * 4 + 256 * 2 + 256 * 4 + 16;
constexpr uint32_t kEntrySymShift = 23;
constexpr uint32_t kPosMask = (1u << kEntrySymShift) - 1;     // the bits of a sum of entries that count code bits

constexpr uint32_t kStatusBadDescriptor = 1;  // a descriptor, offset or table points outside the buffers
constexpr uint32_t kStatusBadRecord = 2;      // a tile record is not a column table and whole rows, or too high
constexpr uint32_t kStatusWaitTimeout = 3;    // an asynchronous copy did not complete in time
constexpr uint32_t kStatusBadTable = 4;       // code lengths do not form a complete prefix code
constexpr uint32_t kStatusBrokenPromise = 5;  // ZIPMOE_DECODE_SHORT_CODES was given, yet a tile has longer codes or a longer record
constexpr uint32_t kStatusCounterShared = 6;  // the work counter of a dynamically distributed launch is in use by another launch

constexpr uint32_t kRecHead = 32;    // a record starts with the column of each lane's backward stream
constexpr uint32_t kRowBytes = 128;  // then rows of one word per column
constexpr uint32_t kMaxRows = 48;    // 128 codes of at most 12 bits per column
constexpr int kPayBuf = kRecHead + 16 * kRowBytes;   // record bytes staged in shared memory by the narrow kernels (16 rows)
constexpr int kPaySlack = kRowBytes; // readable bytes after a staged record (a lane reads the word under its position and the next)
constexpr int kPayStage = kPayBuf + kPaySlack;

__device__ __forceinline__ void report(uint32_t *status, uint32_t code) {
  if (status) atomicCAS(status, 0u, code);
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier + bulk asynchronous copy ------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// Wait with an iteration limit: returns false instead of spinning forever if the copy never lands.  A try that
// fails is followed by a short sleep (growing to a quarter of a microsecond), so that a warp that waits -- the
// helper warps of the fused kernel wait most of the time -- leaves its scheduler's issue slots to the warps
// that decode.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t tries = 1u << 20) {
  if (mbar_try_wait(bar, parity)) return true;
  uint32_t ns = 32;
  for (uint32_t it = 0; it < tries; ++it) {
    __nanosleep(ns);
    if (mbar_try_wait(bar, parity)) return true;
    if (ns < 256) ns += ns;
  }
  return false;
}
// global -> shared, bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  // the compressed streams are read exactly once: their lines may leave the second-level cache first
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar), "l"(policy)
               : "memory");
}
// arm the barrier for `bytes` and start the copy (called by one lane)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  mbar_expect_tx(bar, bytes);
  bulk_g2s(dst, src, bytes, bar);
}

// ---- shared-memory loads ---------------------------------------------------
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

// ---- lookup tables -----------------------------------------------------------
// Builds the tables of one canonical Huffman code from its 256 code lengths.
// Canonical rule: symbols ordered by (length, symbol value) take consecutive
// code values; the first code of length L+1 is (first code of length L + count
// of length L) * 2.  Called by all THREADS threads of the CTA (a multiple of 32, >= 256);
// the caller synchronises before the call, and the call ends with a barrier.
// Returns the longest code length (0 for an invalid table).  An incomplete or
// over-full code is reported and leaves zero entries in the holes: decoding
// then yields garbage but stays in bounds.
// lut_raw holds the lane table when the result is <= 8, the wide table otherwise.
// A barrier of the whole CTA (id 0) or of `threads` threads that share a named barrier (a team of warps with a
// table of its own).
__device__ __forceinline__ void group_sync(uint32_t bar_id, uint32_t threads) {
  if (bar_id == 0) __syncthreads();
  else asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(threads) : "memory");
}

// (tid: the thread's index among the THREADS that call, bar_id: their barrier -- by default the whole CTA)
__device__ __forceinline__ uint32_t build_lut(const uint32_t THREADS, const uint8_t *code_len, uint8_t *lut_raw,
                                              uint8_t *scratch, uint32_t *status, const uint32_t tid_in = 0xFFFFFFFFu,
                                              const uint32_t bar_id = 0) {
  uint8_t *s_len = scratch;                                           // [256]
  uint32_t *s_first = reinterpret_cast<uint32_t *>(scratch + 256);    // [16] left-aligned 12-bit start of each length
  uint32_t *s_wcnt = s_first + 16;                                    // [8][16] per-warp symbol counts by length
  uint16_t *s_start = reinterpret_cast<uint16_t *>(s_wcnt + 8 * 16);  // [256] left-aligned start of each symbol
  uint32_t *s_short = reinterpret_cast<uint32_t *>(s_start + 256);    // [256] lane-table entry of each 8-bit prefix
  uint32_t *s_max = s_short + 256;                                    // [1] longest length
  uint32_t *lane_lut = reinterpret_cast<uint32_t *>(lut_raw);
  uint32_t *wide_lut = reinterpret_cast<uint32_t *>(lut_raw);
  const uint32_t tid = tid_in == 0xFFFFFFFFu ? threadIdx.x : tid_in, warp = tid >> 5, lane = tid & 31;

  uint32_t len = 0;
  if (tid < 256) {
    len = __ldg(code_len + tid);
    if (len > ZIPMOE_MAX_CODE_LEN) len = 0;
    s_len[tid] = (uint8_t)len;
    s_short[tid] = 0;
  }
  uint32_t rank_in_warp = 0;
  if (warp < 8) {
    for (uint32_t L = 1; L <= ZIPMOE_MAX_CODE_LEN; ++L) {
      uint32_t b = __ballot_sync(0xFFFFFFFFu, len == L);
      if (len == L) rank_in_warp = __popc(b & ((1u << lane) - 1));
      if (lane == 0) s_wcnt[warp * 16 + L] = __popc(b);
    }
  }
  group_sync(bar_id, THREADS);
  if (tid == 0) {
    uint32_t code = 0, longest = 0;
    for (uint32_t L = 1; L <= ZIPMOE_MAX_CODE_LEN; ++L) {
      uint32_t cnt = 0;
      for (uint32_t w = 0; w < 8; ++w) cnt += s_wcnt[w * 16 + L];
      if (cnt) longest = L;
      s_first[L] = code << (kWideLutBits - L);
      code = (code + cnt) << 1;
    }
    // a complete code ends with code == 2^(Lmax+1) after the last doubling
    if (code != (2u << ZIPMOE_MAX_CODE_LEN)) {
      report(status, kStatusBadTable);
      longest = ZIPMOE_MAX_CODE_LEN;   // take the general path; holes decode as length 0
    }
    *s_max = longest;
  }
  group_sync(bar_id, THREADS);
  const uint32_t longest = *s_max;
  if (tid < 256 && len) {
    uint32_t rank = rank_in_warp;
    for (uint32_t w = 0; w < warp; ++w) rank += s_wcnt[w * 16 + len];
    uint32_t start = s_first[len] + (rank << (kWideLutBits - len));
    s_start[tid] = (uint16_t)(start < (uint32_t)kWideLutEntries ? start : 0xFFFF);
  }
  if (longest > (uint32_t)kLaneLutBits)
    for (uint32_t k = tid; k < (uint32_t)kWideLutEntries; k += THREADS) wide_lut[k] = 0;
  group_sync(bar_id, THREADS);
  // every symbol fills the range of windows its code is a prefix of
  for (uint32_t s = warp; s < 256; s += THREADS / 32) {
    const uint32_t L = s_len[s];
    if (!L) continue;
    const uint32_t start = s_start[s], n = 1u << (kWideLutBits - L);
    if (start == 0xFFFF || start + n > (uint32_t)kWideLutEntries) continue;
    const uint32_t entry = (s << kEntrySymShift) | L;
    if (L <= (uint32_t)kLaneLutBits) {
      const uint32_t n8 = n >> (kWideLutBits - kLaneLutBits), s8 = start >> (kWideLutBits - kLaneLutBits);
      for (uint32_t k = lane; k < n8; k += 32) s_short[s8 + k] = entry;
    }
    if (longest > (uint32_t)kLaneLutBits)
      for (uint32_t k = lane; k < n; k += 32) wide_lut[start + k] = entry;
  }
  group_sync(bar_id, THREADS);
  // replicate the 8-bit table once per lane
  if (longest <= (uint32_t)kLaneLutBits)
    for (uint32_t k = tid; k < (1u << kLaneLutBits) * 32; k += THREADS) lane_lut[k] = s_short[k >> 5];
  group_sync(bar_id, THREADS);
  return longest;
}

// ---- descriptors -> tiles --------------------------------------------------
struct TileWork {
  const uint8_t *rec;   // global address of the tile record
  const uint8_t *sm;    // global address of the tile's sign+mantissa bytes
  uint16_t *out;        // global address of the tile's first element
  uint32_t rec_bytes, pitch, valid, iters, pieces;
  uint32_t n_sub;       // 1, or the number of small consecutive tiles taken in one step (see decode_step): rec_bytes,
                        // valid, iters and pieces are then those of the whole step
  bool ok, staged;      // staged: the record fits a record stage of the calling kernel
};

struct LaunchArgs {
  const zipmoe_chunk_desc *chunks;
  const zipmoe_table *tables;
  const uint8_t *payload;
  const uint8_t *sm;
  uint16_t *out;
  uint32_t *status;
  uint64_t payload_bytes, sm_bytes, out_elems;
  uint32_t n_chunks, n_tiles, n_tables, tiles_per_cta;
  uint32_t *work_counter;   // two words zeroed before the launch (dynamic distribution only): the next tile not yet
                            // handed to a CTA, and the tag of the launch that uses the counter
  uint32_t work_tag;
  uint32_t wait_tries;      // tries of a wait on an asynchronous copy before the kernel gives up on it
  uint32_t extra_tx;        // 0; the library's own tests arm record barriers for this many bytes more than the
                            // copy delivers, so that the give-up path can be exercised without any fault
};

// Which descriptor holds global tile g: exact guess for launches whose chunks all hold the same number of tiles,
// else a search on tile_prefix in which the 32 lanes of the warp probe 32 evenly spaced descriptors per step
// (three or four dependent loads for any launch, where a binary search needs up to seventeen).  Called by whole
// warps; the result is the same in every lane.
__device__ inline uint32_t find_chunk(const LaunchArgs &a, uint32_t g) {
  uint32_t c = (uint32_t)(((uint64_t)g * a.n_chunks) / a.n_tiles);
  if (c >= a.n_chunks) c = a.n_chunks - 1;
  uint32_t p = __ldg(&a.chunks[c].tile_prefix), m = __ldg(&a.chunks[c].n_tiles);
  if (g >= p && g - p < m) return c;
  const uint32_t lane = threadIdx.x & 31u;
  uint32_t lo = 0, hi = a.n_chunks;  // invariant: prefix[lo] <= g (prefix[0] = 0), and g < prefix[hi] where hi exists
  while (hi - lo > 1) {
    const uint32_t step = (hi - lo + 31) / 32;
    const uint32_t at = lo + lane * step;
    const bool below = at < hi && __ldg(&a.chunks[at].tile_prefix) <= g;
    const uint32_t k = __popc(__ballot_sync(0xFFFFFFFFu, below));   // prefixes ascend: the lanes that are below come first
    const uint32_t first = lo + (k ? k - 1 : 0) * step;
    hi = min(hi, first + step);
    lo = first;
  }
  return lo;
}

static_assert(sizeof(zipmoe_chunk_desc) == 80, "descriptor is read as five 16-byte words");

// Everything the decoder needs about tile t of descriptor c, with every offset
// checked against the sizes of the buffers the launch was given.
__device__ __forceinline__ TileWork resolve_tile(const LaunchArgs &a, uint32_t c, uint32_t t, const uint32_t stage_buf,
                                                 const uint32_t table_id) {
  TileWork w;
  w.ok = false;
  w.staged = false;
  w.n_sub = 1;
  if (c >= a.n_chunks) return w;
  const uint4 *d = reinterpret_cast<const uint4 *>(a.chunks + c);
  const uint4 d0 = __ldg(d), d1 = __ldg(d + 1), d2 = __ldg(d + 2), d3 = __ldg(d + 3);
  const uint64_t pay_off = ((uint64_t)d0.y << 32) | d0.x, sm_off = ((uint64_t)d0.w << 32) | d0.z;
  const uint64_t out_off = ((uint64_t)d1.y << 32) | d1.x;
  const uint32_t pitch = d1.z, tpr = d1.w, tile0 = d2.x, m = d2.y, tile_elems = d2.z, last = d2.w;
  if (d3.x != table_id) return w;   // every chunk of a run names the run's table
  if (t >= m || tpr == 0 || tile_elems == 0 || tile_elems > ZIPMOE_TILE_ELEMS_MAX || (tile_elems & 255) ||
      last == 0 || last > tile_elems || ((pitch & 7) | (pay_off & 15) | (sm_off & 15) | (out_off & 7)))
    return w;
  if (pay_off + 4ull * (t + 2) > a.payload_bytes) return w;
  const uint32_t *tab = reinterpret_cast<const uint32_t *>(a.payload + pay_off);
  const uint32_t o0 = __ldg(tab + t), o1 = __ldg(tab + t + 1);
  const uint64_t rec_off = pay_off + 16ull * o0;
  if (o1 <= o0) return w;
  w.rec_bytes = (o1 - o0) * 16u;
  // a record is the column table and 1..kMaxRows whole rows
  if (w.rec_bytes < kRecHead + kRowBytes || w.rec_bytes > kRecHead + kMaxRows * kRowBytes ||
      ((w.rec_bytes - kRecHead) & (kRowBytes - 1)) || rec_off + w.rec_bytes > a.payload_bytes)
    return w;
  w.iters = tile_elems >> 8;
  w.valid = (t == m - 1) ? last : tile_elems;
  w.pieces = sm_pieces_of_tile(w.valid);   // only the pieces that hold bytes of the tile are ever copied
  const uint32_t q = tile0 + t;
  uint64_t origin = out_off;
  if (tpr == 1) origin += (uint64_t)q * w.iters * pitch;   // linear layout: no division
  else origin += (uint64_t)(q / tpr) * w.iters * pitch + (uint64_t)(q % tpr) * 256;
  const uint32_t rows_used = (w.valid + 255) >> 8;
  if (origin + (uint64_t)(rows_used - 1) * pitch + (w.valid - (rows_used - 1) * 256) > a.out_elems) return w;
  const uint64_t sm_tile = sm_off + (uint64_t)t * tile_elems;
  if (sm_tile + w.valid > a.sm_bytes) return w;
  w.rec = a.payload + rec_off;
  w.sm = a.sm + sm_tile;
  w.out = a.out + origin;
  w.pitch = pitch;
  w.staged = w.rec_bytes <= stage_buf;
  w.ok = true;
  return w;
}

// ---- tile decoder -------------------------------------------------------------
// a*b + c on the multiply-add pipe (keeps pure integer adds and shifts-by-constant
// off the ALU pipe, which the variable shifts and logic ops of the decoder fill)
__device__ __forceinline__ uint32_t mad_u32(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// One lane's view of a tile record: the record is `rows` rows of 32 words (after a 32-byte column table); the
// lane's forward stream is column `lane` read downwards from row 0, its backward stream the column the table names
// read upwards from the last row.  Bit y of a column is bit 31 - y % 32 of its word in row y / 32; the forward
// stream's k-th bit is column bit k, the backward stream's k-th bit is column bit 32 * rows - 1 - k.
// A stream's whole state is the number of bits it has consumed.  For every batch of codes the lane loads the word
// under its position and the one after it afresh: word r of all columns is one 128-byte row, so these loads of a
// warp touch 32 different banks wherever the lanes are.  A batch takes the stream's next 32 bits into one register
// and decodes from its top:
//   FAST  (no code longer than 8 bits): four codes per batch, looked up in the lane table with the top 8 bits;
//   !FAST (codes up to 12 bits): two codes per batch, looked up in the wide table with the top 12 bits.
// Whole table entries, (symbol << 23) | length, are added to a position: the low 23 bits of the sum are the code
// bits consumed, the rest is masked off.
// STAGED: the record is in shared memory at rec_s; else it is read from global memory at rec_g (a record too
// high for the kernel's record stages: correct, slow).
template <bool STAGED, bool FAST>
struct LaneDecoder {
  uint32_t pos0, pos1;       // code bits consumed from the forward / backward stream
  uint32_t col0, top1;       // STAGED: shared address of the forward column's row 0 / of the backward column's last row
  const uint32_t *words_g;   // !STAGED: the record's rows in global memory
  uint32_t lane_g, bcol_g, last_row;
  uint32_t lut, my_lut;

  __device__ __forceinline__ void init(uint32_t rec_s, const uint8_t *rec_g, uint32_t rec_bytes, uint32_t lut_addr,
                                       uint32_t lane) {
    const uint32_t rows = (rec_bytes - kRecHead) / kRowBytes;
    uint32_t bcol;
    if (STAGED) bcol = lds_u8(rec_s + lane) & 31u;
    else bcol = __ldg(rec_g + lane) & 31u;
    col0 = rec_s + kRecHead + 4 * lane;
    top1 = rec_s + kRecHead + (rows - 1) * kRowBytes + 4 * bcol;
    words_g = reinterpret_cast<const uint32_t *>(rec_g + kRecHead);
    lane_g = lane;
    bcol_g = bcol;
    last_row = rows - 1;
    pos0 = pos1 = 0;
    lut = lut_addr;
    my_lut = lut_addr + 4 * lane;
  }
  // the next 32 bits of the forward stream, the first one in bit 31
  __device__ __forceinline__ uint32_t window0() const {
    const uint32_t r = pos0 >> 5;
    uint32_t c, n;
    if (STAGED) {
      const uint32_t a = mad_u32(r, kRowBytes, col0);
      c = lds_u32(a);
      n = lds_u32(a + kRowBytes);
    } else {
      c = __ldg(words_g + min(r, last_row) * 32 + lane_g);
      n = __ldg(words_g + min(r + 1, last_row) * 32 + lane_g);
    }
    return __funnelshift_l(n, c, pos0);
  }
  // the next 32 bits of the backward stream, the first one in bit 31
  __device__ __forceinline__ uint32_t window1() const {
    const uint32_t r = pos1 >> 5;
    uint32_t c, n;
    if (STAGED) {
      const uint32_t a = top1 - r * kRowBytes;
      c = lds_u32(a);
      n = lds_u32(a - kRowBytes);
    } else {
      c = __ldg(words_g + (last_row - min(r, last_row)) * 32 + bcol_g);
      n = __ldg(words_g + (last_row - min(r + 1, last_row)) * 32 + bcol_g);
    }
    return __brev(__funnelshift_r(c, n, pos1));
  }
  // The next 64 bits of a stream as two registers (hi = the next 32 bits, first one in bit 31; lo = the 32 after
  // them), from three words loaded at once: enough for two batches, so that only every other batch waits for
  // shared memory.  second(hi, lo, used) is the window after `used` (0..32) of hi's bits have been consumed.
  __device__ __forceinline__ void pair0(uint32_t &hi, uint32_t &lo) const {
    const uint32_t r = pos0 >> 5;
    uint32_t c, n, m;
    if (STAGED) {
      const uint32_t a = mad_u32(r, kRowBytes, col0);
      c = lds_u32(a);
      n = lds_u32(a + kRowBytes);
      m = lds_u32(a + 2 * kRowBytes);
    } else {
      c = __ldg(words_g + min(r, last_row) * 32 + lane_g);
      n = __ldg(words_g + min(r + 1, last_row) * 32 + lane_g);
      m = __ldg(words_g + min(r + 2, last_row) * 32 + lane_g);
    }
    hi = __funnelshift_l(n, c, pos0);
    lo = __funnelshift_l(m, n, pos0);
  }
  __device__ __forceinline__ void pair1(uint32_t &hi, uint32_t &lo) const {   // (bit-reversed: first bit in bit 0)
    const uint32_t r = pos1 >> 5;
    uint32_t c, n, m;
    if (STAGED) {
      const uint32_t a = top1 - r * kRowBytes;
      c = lds_u32(a);
      n = lds_u32(a - kRowBytes);
      m = lds_u32(a - 2 * kRowBytes);
    } else {
      c = __ldg(words_g + (last_row - min(r, last_row)) * 32 + bcol_g);
      n = __ldg(words_g + (last_row - min(r + 1, last_row)) * 32 + bcol_g);
      m = __ldg(words_g + (last_row - min(r + 2, last_row)) * 32 + bcol_g);
    }
    hi = __funnelshift_r(c, n, pos1);
    lo = __funnelshift_r(n, m, pos1);
  }
  __device__ static __forceinline__ uint32_t second0(uint32_t hi, uint32_t lo, uint32_t used) {
    return __funnelshift_lc(lo, hi, used);
  }
  __device__ static __forceinline__ uint32_t second1(uint32_t hi, uint32_t lo, uint32_t used) {
    return __brev(__funnelshift_rc(hi, lo, used));
  }
  __device__ __forceinline__ uint32_t lookup(uint32_t w) const {   // (symbol << 23) | length of the code at the top of w
    if (FAST) return lds_u32(mad_u32(w >> (32 - kLaneLutBits), 128u, my_lut));
    return lds_u32(mad_u32(w >> (32 - kWideLutBits), 4u, lut));
  }
  __device__ static __forceinline__ uint32_t next(uint32_t w, uint32_t entry) {   // drop the code just decoded
    return __funnelshift_l(0u, w, entry);
  }
  // 8 table entries and 8 sign+mantissa bytes -> 8 bf16.  Bytes 2 and 3 of an entry are the symbol at the place
  // of a bf16's exponent; two entries are packed by one byte permutation, the sign+mantissa bytes are spread to
  // their places by another, and one logic operation joins them.
  __device__ static __forceinline__ uint4 merge(const uint2 smv, const uint32_t (&e)[8]) {
    constexpr uint32_t kKeep = 0x807F807Fu;   // sign and mantissa bits of two bf16
    uint4 o;
    o.x = (__byte_perm(smv.x, 0, 0x1100) & kKeep) | __byte_perm(e[0], e[1], 0x7632);
    o.y = (__byte_perm(smv.x, 0, 0x3322) & kKeep) | __byte_perm(e[2], e[3], 0x7632);
    o.z = (__byte_perm(smv.y, 0, 0x1100) & kKeep) | __byte_perm(e[4], e[5], 0x7632);
    o.w = (__byte_perm(smv.y, 0, 0x3322) & kKeep) | __byte_perm(e[6], e[7], 0x7632);
    return o;
  }
  // The next 8 elements of both streams (one group of an even iteration and one of the following odd
  // iteration) merged with their sign+mantissa bytes.  The two decode chains are written interleaved so that
  // each one's lookup latency is covered by the other's work.
  __device__ __forceinline__ void group2(const uint2 sm0, const uint2 sm1, uint4 &o0, uint4 &o1) {
    uint32_t e[8], f[8];
    if (FAST) {
      // two batches of four codes per stream from one pair of windows
      uint32_t whi, wlo, xhi, xlo;
      pair0(whi, wlo);
      pair1(xhi, xlo);
      uint32_t w = whi, x = __brev(xhi), used0 = 0, used1 = 0;
#pragma unroll
      for (int h = 0; h < 8; h += 4) {
        if (h) {
          w = second0(whi, wlo, used0);
          x = second1(xhi, xlo, used1);
        }
        e[h] = lookup(w);
        f[h] = lookup(x);
        w = next(w, e[h]);
        x = next(x, f[h]);
        e[h + 1] = lookup(w);
        f[h + 1] = lookup(x);
        w = next(w, e[h + 1]);
        x = next(x, f[h + 1]);
        e[h + 2] = lookup(w);
        f[h + 2] = lookup(x);
        w = next(w, e[h + 2]);
        x = next(x, f[h + 2]);
        e[h + 3] = lookup(w);
        f[h + 3] = lookup(x);
        used0 = ((e[h] + e[h + 1]) + (e[h + 2] + e[h + 3])) & kPosMask;
        used1 = ((f[h] + f[h + 1]) + (f[h + 2] + f[h + 3])) & kPosMask;
        pos0 += used0;
        pos1 += used1;
      }
    } else {
      // two batches of two codes per stream from one pair of windows, twice
#pragma unroll
      for (int h = 0; h < 8; h += 4) {
        uint32_t whi, wlo, xhi, xlo;
        pair0(whi, wlo);
        pair1(xhi, xlo);
        uint32_t w = whi, x = __brev(xhi);
        e[h] = lookup(w);
        f[h] = lookup(x);
        w = next(w, e[h]);
        x = next(x, f[h]);
        e[h + 1] = lookup(w);
        f[h + 1] = lookup(x);
        const uint32_t used0 = (e[h] + e[h + 1]) & kPosMask, used1 = (f[h] + f[h + 1]) & kPosMask;
        w = second0(whi, wlo, used0);
        x = second1(xhi, xlo, used1);
        e[h + 2] = lookup(w);
        f[h + 2] = lookup(x);
        w = next(w, e[h + 2]);
        x = next(x, f[h + 2]);
        e[h + 3] = lookup(w);
        f[h + 3] = lookup(x);
        pos0 = (pos0 + used0 + e[h + 2] + e[h + 3]) & kPosMask;
        pos1 = (pos1 + used1 + f[h + 2] + f[h + 3]) & kPosMask;
      }
    }
    o0 = merge(sm0, e);
    o1 = merge(sm1, f);
  }
  // one code of stream WHICH
  template <int WHICH>
  __device__ __forceinline__ uint32_t single() {
    uint32_t e;
    if (WHICH == 0) {
      e = lookup(window0());
      pos0 = (pos0 + e) & kPosMask;
    } else {
      e = lookup(window1());
      pos1 = (pos1 + e) & kPosMask;
    }
    return e;
  }
  // the next 8 elements of stream WHICH alone (the ragged end of a tensor)
  template <int WHICH>
  __device__ __forceinline__ uint4 group1(const uint2 smv) {
    uint32_t e[8];
#pragma unroll
    for (int h = 0; h < 8; h += 2) {
      uint32_t w = WHICH == 0 ? window0() : window1();
      e[h] = lookup(w);
      w = next(w, e[h]);
      e[h + 1] = lookup(w);
      if (WHICH == 0) pos0 = (pos0 + e[h] + e[h + 1]) & kPosMask;
      else pos1 = (pos1 + e[h] + e[h + 1]) & kPosMask;
    }
    return merge(smv, e);
  }
};

// Decodes one tile with the 32 lanes of a warp.
//   record  : in shared memory at rec_s (STAGED) or in global memory at rec_g;
//   lut     : shared address of the lane table (FAST) or the wide table (!FAST);
//   SM bytes: arrive in pieces of kPieceIters iterations; feed.begin(p) waits for piece
//             p and returns its shared address (0xFFFFFFFF when the wait ran
//             out), feed.end(p) tells that the warp is done reading it;
//   output  : sink.group(i, lane, v) takes the 8 bf16 of iteration i, lane;
//             sink.elem(i, lane, j, v) one bf16 of the short last group of a
//             linear tensor.
// Returns 0 on success, else a status code (warp-uniform).
// SMALL: also an unrolled path for small full tiles (kept out of the instantiation that never sees any: it would
// only lengthen its code).
template <bool STAGED, bool FAST, bool SMALL, class Feed, class Sink>
__device__ __forceinline__ uint32_t decode_tile(uint32_t rec_s, const uint8_t *rec_g, uint32_t rec_bytes,
                                                uint32_t lut, uint32_t valid, uint32_t iters,
                                                uint32_t lane, Feed &feed, Sink &sink) {
  LaneDecoder<STAGED, FAST> dec;
  dec.init(rec_s, rec_g, rec_bytes, lut, lane);
  static_assert(kPieceIters % 2 == 0, "a piece holds whole pairs of iterations");

  const uint32_t pieces = sm_pieces_of_tile(valid);   // pieces that exist: iterations past them hold no element
  if (SMALL && valid == iters * 256u && iters < kPieceIters && (iters & 1u) == 0) {
    // a small full tile (chunks of less than 2048 elements): one piece, a few pairs of iterations
    const uint32_t sm_s = feed.begin(0);
    if (sm_s == 0xFFFFFFFFu) return kStatusWaitTimeout;
    const uint32_t sm_lane = sm_s + lane * 8;
#pragma unroll
    for (uint32_t k = 0; k < kPieceIters - 2; k += 2) {
      if (k < iters) {
        uint4 o0, o1;
        dec.group2(lds_v2(sm_lane + k * 256), lds_v2(sm_lane + (k + 1) * 256), o0, o1);
        sink.group(k, lane, o0);
        sink.group(k + 1, lane, o1);
      }
    }
    feed.end(0);
    return 0;
  }
  if (valid == iters * 256u && (iters % kPieceIters) == 0) {
    // every group exists and pieces are whole: unrolled iterations, addresses are immediates
    for (uint32_t p = 0; p < pieces; ++p) {
      const uint32_t sm_s = feed.begin(p);
      if (sm_s == 0xFFFFFFFFu) return kStatusWaitTimeout;
      const uint32_t sm_lane = sm_s + lane * 8;
#pragma unroll
      for (uint32_t k = 0; k < kPieceIters; k += 2) {
        uint4 o0, o1;
        dec.group2(lds_v2(sm_lane + k * 256), lds_v2(sm_lane + (k + 1) * 256), o0, o1);
        sink.group(kPieceIters * p + k, lane, o0);
        sink.group(kPieceIters * p + k + 1, lane, o1);
      }
      feed.end(p);
    }
    return 0;
  }
  // one group of sub-stream WHICH that may be short or absent (decided per lane)
  auto ragged = [&](auto which, uint32_t i, uint32_t sm_s) {
    constexpr int WHICH = decltype(which)::value;
    const uint32_t pos_e = (i * 32 + lane) * 8;
    const uint32_t sm_at = sm_s + ((i % kPieceIters) * 32 + lane) * 8;
    if (pos_e + 8 <= valid) {
      sink.group(i, lane, dec.template group1<WHICH>(lds_v2(sm_at)));
    } else if (pos_e < valid) {   // the one short group at the end of a linear tensor
      const uint32_t cnt = valid - pos_e;
      for (uint32_t j = 0; j < cnt; ++j) {
        const uint32_t e = dec.template single<WHICH>();
        const uint32_t at = sm_at + j;
        const uint32_t smb = (lds_u32(at & ~3u) >> (8 * (at & 3u))) & 0xFFu;
        sink.elem(i, lane, j, (uint16_t)(((smb & 0x80u) << 8) | ((e >> 16) & 0x7F80u) | (smb & 0x7Fu)));
      }
    }
  };
  for (uint32_t p = 0; p < pieces; ++p) {
    const uint32_t sm_s = feed.begin(p);
    if (sm_s == 0xFFFFFFFFu) return kStatusWaitTimeout;
    const uint32_t i_end = min(iters, kPieceIters * (p + 1));
#pragma unroll 1
    for (uint32_t i = kPieceIters * p; i < i_end; i += 2) {
      if (i + 2 <= i_end && (i + 2) * 256u <= valid) {   // both iterations are complete for every lane
        uint4 o0, o1;
        const uint32_t sm_at = sm_s + ((i % kPieceIters) * 32 + lane) * 8;
        dec.group2(lds_v2(sm_at), lds_v2(sm_at + 256), o0, o1);
        sink.group(i, lane, o0);
        sink.group(i + 1, lane, o1);
      } else {
        ragged(std::integral_constant<int, 0>{}, i, sm_s);
        if (i + 1 < i_end) ragged(std::integral_constant<int, 1>{}, i + 1, sm_s);
      }
    }
    feed.end(p);
  }
  return 0;
}

// Decodes a step of n_sub small tiles with the 32 lanes of a warp: consecutive full tiles of one linear tensor, each
// of `sub_iters` (2, 4 or 8) iterations with a record of its own, whose records were staged by one copy (lane i holds
// the offset of record i in the stage and its size), whose sign+mantissa bytes are one contiguous run served in the
// usual pieces, and whose outputs are one contiguous run of rows.  The per-tile costs of the pipeline (copies,
// waits, bookkeeping) are paid once per step.  Codes of at most 8 bits only.
template <class Feed, class Sink>
__device__ __forceinline__ uint32_t decode_step(uint32_t rec_s, uint32_t sub_off, uint32_t sub_bytes, uint32_t n_sub,
                                                uint32_t sub_iters, uint32_t lut, uint32_t lane, Feed &feed, Sink &sink) {
  const uint32_t per_piece = kPieceIters / sub_iters;          // tiles served by one piece of sign+mantissa bytes
  const uint32_t pieces = (n_sub + per_piece - 1) / per_piece;
  for (uint32_t p = 0; p < pieces; ++p) {
    const uint32_t sm_s = feed.begin(p);
    if (sm_s == 0xFFFFFFFFu) return kStatusWaitTimeout;
    const uint32_t i_end = min(n_sub, (p + 1) * per_piece);
#pragma unroll 1
    for (uint32_t i = p * per_piece; i < i_end; ++i) {
      const uint32_t off = __shfl_sync(0xFFFFFFFFu, sub_off, i), bytes = __shfl_sync(0xFFFFFFFFu, sub_bytes, i);
      LaneDecoder<true, true> dec;
      dec.init(rec_s + off, nullptr, bytes, lut, lane);
      const uint32_t row0 = i * sub_iters;                     // first row of the tile within the step
      const uint32_t sm_lane = sm_s + (row0 % kPieceIters) * 256 + lane * 8;
#pragma unroll 1
      for (uint32_t k = 0; k < sub_iters; k += 2) {
        uint4 o0, o1;
        dec.group2(lds_v2(sm_lane + k * 256), lds_v2(sm_lane + (k + 1) * 256), o0, o1);
        sink.group(row0 + k, lane, o0);
        sink.group(row0 + k + 1, lane, o1);
      }
    }
    feed.end(p);
  }
  return 0;
}

}  // namespace zipmoe_dev

namespace zipmoe_host {
// A named range around an entry point's host work and launches, for timeline profilers (costs nothing unless a
// tool is attached).
struct TraceRange {
  explicit TraceRange(const char *name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
};
constexpr uint32_t kWaitTries = 1u << 20;
// what zipmoe_test_wait_fault last set (0 extra bytes and kWaitTries unless a test is running)
void wait_fault_setting(uint32_t *extra_tx, uint32_t *tries);
}  // namespace zipmoe_host
