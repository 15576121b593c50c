// Device-side building blocks of the decoder, shared by the bulk decode kernel
// and the fused decode+FFN kernels: PTX wrappers (mbarrier, bulk async copy,
// shared-memory loads), the per-table lookup-table builder, and the warp-level
// tile decoder.  sm_100a only.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "zipmoe.h"

namespace zipmoe_dev {

constexpr int kLutBits = ZIPMOE_MAX_CODE_LEN;  // one lookup resolves any code
constexpr int kLutEntries = 1 << kLutBits;
constexpr int kLutBytes = kLutEntries * 2;      // u16 entries: (symbol << 7) | length
constexpr int kLutScratchBytes = 256 + 16 * 4 + 8 * 16 * 4 + 256 * 2;

constexpr uint32_t kStatusBadDescriptor = 1;  // a descriptor, offset or table points outside the buffers
constexpr uint32_t kStatusBadBitCount = 2;    // a tile's lane bit counts overrun its record
constexpr uint32_t kStatusWaitTimeout = 3;    // an asynchronous copy did not complete in time
constexpr uint32_t kStatusBadTable = 4;       // code lengths do not form a complete prefix code

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
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < (1u << 22); ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> shared, bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// one lane arms the stage's barrier and starts the copies of a tile's record
// (skipped when rec_bytes == 0: the record is then read from global) and of
// its sign+mantissa bytes
__device__ __forceinline__ void issue_tile_copies(const uint8_t *rec, uint32_t rec_bytes, const uint8_t *sm,
                                                  uint32_t sm_bytes, uint32_t rec_dst, uint32_t sm_dst, uint32_t bar) {
  mbar_expect_tx(bar, rec_bytes + sm_bytes);
  if (rec_bytes) bulk_g2s(rec_dst, rec, rec_bytes, bar);
  bulk_g2s(sm_dst, sm, sm_bytes, bar);
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

// ---- lookup table ------------------------------------------------------------
// Builds the 4096-entry table of one canonical Huffman code from its 256 code
// lengths: entry[v] for a 12-bit window v is (symbol << 7) | length of the code
// that is a prefix of v.  Canonical rule: symbols ordered by (length, symbol
// value) take consecutive code values; the first code of length L+1 is
// (first code of length L + count of length L) * 2.  Called by all THREADS
// threads of the CTA (THREADS >= 256); the caller synchronises before and
// after.  An incomplete or over-full code leaves zero entries (length 0) in the
// holes and is reported: decoding then yields garbage but stays in bounds.
template <int THREADS>
__device__ void build_lut(const uint8_t *code_len, uint8_t *lut_raw, uint8_t *scratch, uint32_t *status) {
  static_assert(THREADS >= 256 && THREADS % 32 == 0, "one thread per symbol");
  uint8_t *s_len = scratch;                                          // [256]
  uint32_t *s_first = reinterpret_cast<uint32_t *>(scratch + 256);   // [16] left-aligned start of each length
  uint32_t *s_wcnt = s_first + 16;                                   // [8][16] per-warp symbol counts by length
  uint16_t *s_start = reinterpret_cast<uint16_t *>(s_wcnt + 8 * 16); // [256] left-aligned start of each symbol
  uint32_t *lut32 = reinterpret_cast<uint32_t *>(lut_raw);
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  for (uint32_t k = tid; k < kLutEntries / 2; k += THREADS) lut32[k] = 0;
  uint32_t len = 0;
  if (tid < 256) {
    len = __ldg(code_len + tid);
    if (len > ZIPMOE_MAX_CODE_LEN) len = 0;
    s_len[tid] = (uint8_t)len;
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
    uint32_t code = 0;
    for (uint32_t L = 1; L <= ZIPMOE_MAX_CODE_LEN; ++L) {
      uint32_t cnt = 0;
      for (uint32_t w = 0; w < 8; ++w) cnt += s_wcnt[w * 16 + L];
      s_first[L] = code << (kLutBits - L);   // left-aligned
      code = (code + cnt) << 1;
    }
    // a complete code ends with code == 2^(Lmax+1) after the last doubling
    if (code != (2u << ZIPMOE_MAX_CODE_LEN)) report(status, kStatusBadTable);
  }
  __syncthreads();
  if (tid < 256 && len) {
    uint32_t rank = rank_in_warp;
    for (uint32_t w = 0; w < warp; ++w) rank += s_wcnt[w * 16 + len];
    uint32_t start = s_first[len] + (rank << (kLutBits - len));
    s_start[tid] = (uint16_t)(start < kLutEntries ? start : 0xFFFF);
  }
  __syncthreads();
  uint16_t *lut16 = reinterpret_cast<uint16_t *>(lut_raw);
  for (uint32_t s = warp; s < 256; s += THREADS / 32) {
    const uint32_t L = s_len[s];
    if (!L) continue;
    const uint32_t start = s_start[s], n = 1u << (kLutBits - L);
    if (start == 0xFFFF || start + n > kLutEntries) continue;
    const uint16_t entry = (uint16_t)((s << 7) | L);
    for (uint32_t k = lane; k < n; k += 32) lut16[start + k] = entry;
  }
}

// ---- tile decoder -------------------------------------------------------------
// The code bits of a lane form a stream of u32 words consumed from bit 31 down.
// The lane keeps a 64-bit window (hi:lo) whose top bits are the next code bits;
// `used` counts bits shifted out since the window was last full.
template <bool STAGED>
struct WordSource {
  uint32_t base_s;           // shared address of the bit area (STAGED)
  const uint32_t *base_g;    // global address of the bit area (!STAGED)
  __device__ __forceinline__ uint32_t word(uint32_t idx) const {
    if (STAGED) return lds_u32(base_s + 4 * idx);
    return __ldg(base_g + idx);
  }
};

// Decodes one tile with the 32 lanes of a warp.  Record and SM bytes are in
// shared memory (record in global memory when !STAGED).  Writes bf16 to `out`
// (global): iteration i, lane l -> out[i*pitch + 8*l .. +8).  `valid` is the
// number of existing elements of the tile (< 256*iters only for the last tile
// of a linear tensor).  Returns false (warp-uniform), writing nothing, if the
// lane bit counts overrun the record.
template <bool STAGED>
__device__ __forceinline__ bool decode_tile(uint32_t rec_s, const uint8_t *rec_g, uint32_t rec_bytes, uint32_t sm_s,
                                            uint32_t lut, uint16_t *out, uint32_t pitch, uint32_t valid,
                                            uint32_t iters, uint32_t lane) {
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
  if (64u * 8u + total > rec_bytes * 8u) return false;
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

  auto take = [&]() -> uint32_t {   // decode one code: returns (symbol << 7) | length
    const uint32_t e = lds_u16(lut + ((hi >> (32 - kLutBits)) << 1));
    const uint32_t len = e & 15u;
    hi = __funnelshift_l(lo, hi, len);
    lo <<= len;
    used += len;
    return e;
  };
  auto refill = [&]() {             // after at most two codes: top up with one word when 32 bits are free
    if (used >= 32) {
      const uint32_t w = src.word(next++);
      used -= 32;
      hi |= __funnelshift_l(w, 0u, used);
      lo |= w << used;
    }
  };

  constexpr uint32_t kKeep = 0x807F807Fu;   // sign and mantissa bits of two bf16
  for (uint32_t i = 0; i < iters; ++i) {
    const uint32_t pos = (i * 32 + lane) * 8;
    if (pos + 8 <= valid) {
      const uint2 smv = lds_v2(sm_s + pos);
      const uint32_t e0 = take(), e1 = take();
      refill();
      const uint32_t e2 = take(), e3 = take();
      refill();
      const uint32_t e4 = take(), e5 = take();
      refill();
      const uint32_t e6 = take(), e7 = take();
      refill();
      uint4 o;
      o.x = (__byte_perm(smv.x, 0, 0x1100) & kKeep) | (__byte_perm(e0, e1, 0x5410) & ~kKeep);
      o.y = (__byte_perm(smv.x, 0, 0x3322) & kKeep) | (__byte_perm(e2, e3, 0x5410) & ~kKeep);
      o.z = (__byte_perm(smv.y, 0, 0x1100) & kKeep) | (__byte_perm(e4, e5, 0x5410) & ~kKeep);
      o.w = (__byte_perm(smv.y, 0, 0x3322) & kKeep) | (__byte_perm(e6, e7, 0x5410) & ~kKeep);
      __stcs(reinterpret_cast<uint4 *>(out + (size_t)i * pitch + lane * 8), o);
    } else if (pos < valid) {   // the one short group at the end of a linear tensor
      const uint32_t cnt = valid - pos;
      uint16_t *dst = out + (size_t)i * pitch + lane * 8;
      for (uint32_t j = 0; j < cnt; ++j) {
        const uint32_t e = take();
        refill();
        const uint32_t smb = lds_u32(sm_s + ((pos + j) & ~3u)) >> (8 * ((pos + j) & 3u)) & 0xFFu;
        dst[j] = (uint16_t)(((smb & 0x80u) << 8) | (e & 0x7F80u) | (smb & 0x7Fu));
      }
    }
  }
  return true;
}

}  // namespace zipmoe_dev
