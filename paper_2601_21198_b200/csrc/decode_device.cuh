// Device-side building blocks of the decoder, shared by the bulk decode kernel
// and the fused decode+FFN kernels: PTX wrappers (mbarrier, bulk async copy,
// shared-memory loads), the per-table lookup-table builder, and the warp-level
// tile decoder.  sm_100a only.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "zipmoe.h"

namespace zipmoe_dev {

// Two lookup tables per Huffman code:
//  * the lane table resolves codes of up to 8 bits.  It is indexed by the next
//    8 code bits and replicated for each of the 32 lanes, entry (v, lane) at
//    word v*32 + lane, so that lane l only ever touches bank l: the
//    data-dependent lookups of a warp are free of bank conflicts.  Entry =
//    (symbol << 7) | length, or 0 when the 8 bits are the prefix of a longer code;
//  * the wide table (u16 entries, indexed by the next 12 bits) resolves any
//    code.  It is only built, and only consulted after a 0 entry, for codes
//    whose longest length exceeds 8.
constexpr int kLaneLutBits = 8;
constexpr int kLaneLutBytes = (1 << kLaneLutBits) * 32 * 4;   // 32 KB
constexpr int kWideLutBits = ZIPMOE_MAX_CODE_LEN;
constexpr int kWideLutEntries = 1 << kWideLutBits;
constexpr int kWideLutBytes = kWideLutEntries * 2;            // 8 KB
constexpr int kLutBytes = kLaneLutBytes + kWideLutBytes;
constexpr int kLutScratchBytes = 256 + 16 * 4 + 8 * 16 * 4 + 256 * 2 + 256 * 4 + 16;

constexpr uint32_t kStatusBadDescriptor = 1;  // a descriptor, offset or table points outside the buffers
constexpr uint32_t kStatusBadBitCount = 2;    // a tile's lane bit counts overrun its record
constexpr uint32_t kStatusWaitTimeout = 3;    // an asynchronous copy did not complete in time
constexpr uint32_t kStatusBadTable = 4;       // code lengths do not form a complete prefix code

constexpr uint32_t kSmPieceBytes = 1024;      // sign+mantissa bytes of four iterations
constexpr uint32_t kSmPieces = 4;             // pieces of a full tile = slots of a warp's ring

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
// Wait with an iteration limit (each try blocks for a short, hardware-defined
// time): returns false instead of spinning forever if the copy never lands.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t tries = 1u << 20) {
  for (uint32_t it = 0; it < tries; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> shared, bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
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
// of length L) * 2.  Called by all THREADS threads of the CTA (THREADS >= 256);
// the caller synchronises before the call, and the call ends with a barrier.
// Returns the longest code length (0 for an invalid table).  An incomplete or
// over-full code is reported and leaves zero entries in the holes: decoding
// then yields garbage but stays in bounds.
// Layout of lut_raw: lane table (kLaneLutBytes) then wide table (kWideLutBytes).
template <int THREADS>
__device__ uint32_t build_lut(const uint8_t *code_len, uint8_t *lut_raw, uint8_t *scratch, uint32_t *status) {
  static_assert(THREADS >= 256 && THREADS % 32 == 0, "one thread per symbol");
  uint8_t *s_len = scratch;                                           // [256]
  uint32_t *s_first = reinterpret_cast<uint32_t *>(scratch + 256);    // [16] left-aligned 12-bit start of each length
  uint32_t *s_wcnt = s_first + 16;                                    // [8][16] per-warp symbol counts by length
  uint16_t *s_start = reinterpret_cast<uint16_t *>(s_wcnt + 8 * 16);  // [256] left-aligned start of each symbol
  uint32_t *s_short = reinterpret_cast<uint32_t *>(s_start + 256);    // [256] lane-table entry of each 8-bit prefix
  uint32_t *s_max = s_short + 256;                                    // [1] longest length
  uint32_t *lane_lut = reinterpret_cast<uint32_t *>(lut_raw);
  uint16_t *wide_lut = reinterpret_cast<uint16_t *>(lut_raw + kLaneLutBytes);
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

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
  __syncthreads();
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
  __syncthreads();
  const uint32_t longest = *s_max;
  if (tid < 256 && len) {
    uint32_t rank = rank_in_warp;
    for (uint32_t w = 0; w < warp; ++w) rank += s_wcnt[w * 16 + len];
    uint32_t start = s_first[len] + (rank << (kWideLutBits - len));
    s_start[tid] = (uint16_t)(start < (uint32_t)kWideLutEntries ? start : 0xFFFF);
  }
  if (longest > (uint32_t)kLaneLutBits) {
    uint32_t *w32 = reinterpret_cast<uint32_t *>(wide_lut);
    for (uint32_t k = tid; k < (uint32_t)kWideLutEntries / 2; k += THREADS) w32[k] = 0;
  }
  __syncthreads();
  // every symbol fills the range of windows its code is a prefix of
  for (uint32_t s = warp; s < 256; s += THREADS / 32) {
    const uint32_t L = s_len[s];
    if (!L) continue;
    const uint32_t start = s_start[s], n = 1u << (kWideLutBits - L);
    if (start == 0xFFFF || start + n > (uint32_t)kWideLutEntries) continue;
    const uint32_t entry = (s << 7) | L;
    if (L <= (uint32_t)kLaneLutBits) {
      const uint32_t n8 = n >> (kWideLutBits - kLaneLutBits), s8 = start >> (kWideLutBits - kLaneLutBits);
      for (uint32_t k = lane; k < n8; k += 32) s_short[s8 + k] = entry;
    }
    if (longest > (uint32_t)kLaneLutBits)
      for (uint32_t k = lane; k < n; k += 32) wide_lut[start + k] = (uint16_t)entry;
  }
  __syncthreads();
  // replicate the 8-bit table once per lane
  for (uint32_t k = tid; k < (1u << kLaneLutBits) * 32; k += THREADS) lane_lut[k] = s_short[k >> 5];
  __syncthreads();
  return longest;
}

// ---- tile decoder -------------------------------------------------------------
template <bool STAGED>
struct WordSource {
  uint32_t base_s;           // shared address of the bit area (STAGED)
  const uint32_t *base_g;    // global address of the bit area (!STAGED)
  __device__ __forceinline__ uint32_t word(uint32_t idx) const {
    if (STAGED) return lds_u32(base_s + 4 * idx);
    return __ldg(base_g + idx);
  }
};

// Decodes one tile with the 32 lanes of a warp.
//   record  : in shared memory at rec_s (STAGED) or in global memory at rec_g;
//   SM bytes: arrive in pieces of four iterations; feed.begin(p) waits for piece
//             p and returns its shared address (0xFFFFFFFF when the wait ran
//             out), feed.end(p) tells that the warp is done reading it;
//   output  : sink.group(i, lane, v) takes the 8 bf16 of iteration i, lane;
//             sink.elem(i, lane, j, v) one bf16 of the short last group of a
//             linear tensor.
// The code bits of a lane form a stream of u32 words consumed from bit 31 down.
// The lane keeps a 64-bit window (hi:lo) whose top bits are the next code bits.
// `used` counts, in its low 7 bits, the bits shifted out since the window was
// last full; whole table entries are added to it (their low 4 bits are the code
// length, bits 4..6 are zero), so bits 7 and up are meaningless.  A new word is
// shifted in whenever 32 bits are free, which is checked after every four codes:
// the window then holds at least 33 bits, enough for four codes of at most 8
// bits.  A code longer than 8 bits (ESCAPE only) shows as a zero entry of the
// lane table and is resolved through the wide table with its own checks.
// Returns 0 on success, else a status code (warp-uniform); on
// kStatusBadBitCount nothing has been written.
template <bool STAGED, bool ESCAPE, class Feed, class Sink>
__device__ __forceinline__ uint32_t decode_tile(uint32_t rec_s, const uint8_t *rec_g, uint32_t rec_bytes,
                                                uint32_t lane_lut, uint32_t wide_lut, uint32_t valid, uint32_t iters,
                                                uint32_t lane, Feed &feed, Sink &sink) {
  uint32_t my_bits;
  if (STAGED) my_bits = lds_u16(rec_s + 2 * lane);
  else my_bits = __ldg(reinterpret_cast<const uint16_t *>(rec_g) + lane);
  uint32_t incl = my_bits;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= (uint32_t)d) incl += t;
  }
  const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
  if (64u * 8u + total > rec_bytes * 8u) return kStatusBadBitCount;
  const uint32_t start = incl - my_bits;

  WordSource<STAGED> src;
  src.base_s = rec_s + 64;
  src.base_g = reinterpret_cast<const uint32_t *>(rec_g + 64);
  uint32_t next = start >> 5;
  uint32_t used = start & 31;
  const uint32_t w0 = src.word(next), w1 = src.word(next + 1);
  next += 2;
  uint32_t hi = __funnelshift_l(w1, w0, used);
  uint32_t lo = w1 << used;
  const uint32_t my_lut = lane_lut + 4 * lane;

  auto refill = [&]() {   // shift one word in when 32 bits are free
    if (used & 32u) {
      const uint32_t w = src.word(next++);
      used ^= 32u;
      hi |= __funnelshift_l(w, 0u, used);      // w >> (32 - used mod 32), 0 when used mod 32 == 0
      lo |= __funnelshift_l(0u, w, used);      // w << (used mod 32)
    }
  };
  auto consume = [&](uint32_t e) {   // shifts use the low 5 bits of e = the code length
    hi = __funnelshift_l(lo, hi, e);
    lo = __funnelshift_l(0u, lo, e);
    used += e;
  };
  auto take = [&]() -> uint32_t {   // decode one code: returns (symbol << 7) | length
    uint32_t e = lds_u32(my_lut + ((hi >> (32 - kLaneLutBits)) << 7));
    consume(e);
    if (ESCAPE) {
      if (e == 0) {
        refill();
        e = lds_u16(wide_lut + ((hi >> (32 - kWideLutBits)) << 1));
        consume(e);
        refill();
      }
    }
    return e;
  };

  constexpr uint32_t kKeep = 0x807F807Fu;   // sign and mantissa bits of two bf16
  const uint32_t pieces = (iters + 3) >> 2;
  for (uint32_t p = 0; p < pieces; ++p) {
    const uint32_t sm_s = feed.begin(p);
    if (sm_s == 0xFFFFFFFFu) return kStatusWaitTimeout;
    const uint32_t i_end = min(iters, 4 * p + 4);
#pragma unroll 1
    for (uint32_t i = 4 * p; i < i_end; ++i) {
      const uint32_t pos = (i * 32 + lane) * 8;
      if (pos + 8 <= valid) {
        const uint2 smv = lds_v2(sm_s + ((i & 3) * 32 + lane) * 8);
        const uint32_t e0 = take(), e1 = take(), e2 = take(), e3 = take();
        refill();
        const uint32_t e4 = take(), e5 = take(), e6 = take(), e7 = take();
        refill();
        uint4 o;
        o.x = (__byte_perm(smv.x, 0, 0x1100) & kKeep) | (__byte_perm(e0, e1, 0x5410) & ~kKeep);
        o.y = (__byte_perm(smv.x, 0, 0x3322) & kKeep) | (__byte_perm(e2, e3, 0x5410) & ~kKeep);
        o.z = (__byte_perm(smv.y, 0, 0x1100) & kKeep) | (__byte_perm(e4, e5, 0x5410) & ~kKeep);
        o.w = (__byte_perm(smv.y, 0, 0x3322) & kKeep) | (__byte_perm(e6, e7, 0x5410) & ~kKeep);
        sink.group(i, lane, o);
      } else if (pos < valid) {   // the one short group at the end of a linear tensor
        const uint32_t cnt = valid - pos;
        for (uint32_t j = 0; j < cnt; ++j) {
          const uint32_t e = take();
          refill();
          const uint32_t at = ((i & 3) * 32 + lane) * 8 + j;
          const uint32_t smb = (lds_u32(sm_s + (at & ~3u)) >> (8 * (at & 3u))) & 0xFFu;
          sink.elem(i, lane, j, (uint16_t)(((smb & 0x80u) << 8) | (e & 0x7F80u) | (smb & 0x7Fu)));
        }
      }
    }
    feed.end(p);
  }
  return 0;
}

}  // namespace zipmoe_dev
