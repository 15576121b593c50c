// Bulk decode kernel for sm_100a: E-chunk decompression and tensor recovery in
// one pass (paper Section 3.1 "Real-time Inference", Section 3.3
// "Memory-Coalesced Tensor Recovery Kernel").  The paper decompresses E-chunks
// on CPU threads and uses the GPU only for the bit merge; here a warp decodes
// a tile's 32 Huffman sub-streams by table lookup from shared memory and
// merges each exponent byte with its sign+mantissa byte in registers, so the
// decompressed exponents never reach global memory.
//
// Data movement per tile (256*I elements):
//   global -> shared : the tile record (column table + rows of code words) by
//                      one bulk asynchronous copy (cp.async.bulk, completion
//                      on an mbarrier), one tile ahead of the decode; the
//                      tile's sign+mantissa bytes as two 2 KB pieces through
//                      two slots, each refilled for the next tile as soon as
//                      the current tile is done with it;
//   shared -> regs   : 8 SM bytes per lane per iteration, code words on demand;
//   regs   -> global : one 16-byte store per lane per iteration; a warp writes
//                      512 contiguous bytes per iteration.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <type_traits>

#include "zipmoe.h"
#include "decode_device.cuh"

namespace zipmoe_dev {

#ifndef ZIPMOE_WARPS
#define ZIPMOE_WARPS 16
#endif
constexpr int kPayStages = 2;
constexpr int kBarsPerWarp = kPayStages + kSmPieces;   // two record stages, one barrier per sign+mantissa slot

// Two instantiations of the kernel, chosen by the host from the launch's largest tile record:
//   WIDE = false: record stages of kPayStage bytes (records of up to 16 rows: every tensor whose codes average
//                 less than ~4 bits), 16 warps per CTA;
//   WIDE = true : record stages for records of up to 32 rows (8-bit codes everywhere, e.g. tensors with
//                 near-uniform exponents), one warp fewer so that the stages still fit.
// A record higher than its stage is read from global memory word by word (correct, slow).
template <bool WIDE>
struct Cfg {
#ifndef ZIPMOE_CTAS_PER_SM
#define ZIPMOE_CTAS_PER_SM 1
#endif
  static constexpr int kCtasPerSm = WIDE ? 1 : ZIPMOE_CTAS_PER_SM;
  static constexpr int kWarps = WIDE ? ZIPMOE_WARPS - 1 : ZIPMOE_WARPS / kCtasPerSm;   // warps per CTA
  static constexpr int kThreads = kWarps * 32;
  // bytes of a record stage: 32 rows; or 16 rows and a little more, so that a step of four small tiles with four
  // rows each (and the tile tables of their chunks in between) still fits
  static constexpr int kStage = WIDE ? (int)(kRecHead + 32 * kRowBytes) + kPaySlack : 2432 + kPaySlack;
  static constexpr int kBuf = kStage - kPaySlack;                         // longest staged record
  static constexpr int kWarpBytes = kPayStages * kStage + kSmPieces * kSmPieceBytes;
  // lookup tables: one, or two where the narrow stages leave room and the launch is dynamically distributed (two
  // teams of warps, see decode_kernel); a launch asks for no more shared memory than it uses, because what it
  // leaves is first-level cache (the fixed-range launches are 2 % slower with 35 KB less of it)
  static constexpr int kMaxLuts = WIDE ? 1 : 2;
  static constexpr int smem_bytes(int luts) {
    return luts * (kLutBytes + kLutScratchBytes) + kWarps * kWarpBytes + kWarps * kBarsPerWarp * 8;
  }
  static_assert(kCtasPerSm * (smem_bytes(kMaxLuts) + 1024) <= 228 * 1024, "shared memory per SM");
};

// Per-warp asynchronous pipeline.  A warp decodes its tiles one after the other;
// the record of the next tile is copied into the other record stage while the
// current one is decoded, and piece p of the next tile's sign+mantissa bytes is
// copied into slot p as soon as the current tile is done with its piece p.
struct WarpPipe {
  uint32_t pay_addr, sm_addr, bar_addr;   // shared addresses: record stages, SM slots, barriers
  uint32_t stage_bytes;                   // bytes of a record stage
  uint32_t tries, extra_tx;               // wait limit; test-only surplus a record barrier is armed with
  uint32_t phase;                         // bit b = parity to wait for on barrier b
  uint32_t pending;                       // bit b = a copy on barrier b has been started and not waited for
  uint32_t lane;

  __device__ __forceinline__ uint32_t bar(uint32_t b) const { return bar_addr + 8 * b; }
  __device__ __forceinline__ bool wait(uint32_t b) {
    if (!mbar_wait_bounded(bar(b), (phase >> b) & 1u, tries)) return false;
    phase ^= 1u << b;
    pending &= ~(1u << b);
    return true;
  }
  // all lanes call these; one lane starts the copy
  __device__ __forceinline__ void load_record(const TileWork &t, uint32_t stage) {
    if (!t.staged) return;
    if (lane == 0) {
      mbar_expect_tx(bar(stage), t.rec_bytes + extra_tx);
      bulk_g2s(pay_addr + stage * stage_bytes, t.rec, t.rec_bytes, bar(stage));
    }
    pending |= 1u << stage;
  }
  __device__ __forceinline__ void load_sm_piece(const TileWork &t, uint32_t p) {
    const uint32_t bytes = sm_piece_bytes(t.valid, p);
    if (bytes == 0) return;   // (callers ask for p < t.pieces only)
    if (lane == 0) bulk_load(sm_addr + p * kSmPieceBytes, t.sm + p * kSmPieceBytes, bytes, bar(kPayStages + p));
    pending |= 1u << (kPayStages + p);
  }
  // after a wait ran out: give what is still in flight one short, bounded chance to land
  __device__ __forceinline__ void drain() {
    for (uint32_t b = 0; b < (uint32_t)kBarsPerWarp; ++b)
      if (pending & (1u << b)) mbar_wait_bounded(bar(b), (phase >> b) & 1u, min(tries, 1u << 14));
  }
};

struct SmFeed {
  WarpPipe &pipe;
  const TileWork &nxt;
  uint32_t &nxt_issued;   // pieces of the next tile already started
  __device__ __forceinline__ uint32_t begin(uint32_t p) {
    if (!pipe.wait(kPayStages + p)) return 0xFFFFFFFFu;
    return pipe.sm_addr + p * kSmPieceBytes;
  }
  __device__ __forceinline__ void end(uint32_t p) {
    __syncwarp();   // every lane has read the slot
    if (nxt.ok && p == nxt_issued && p < nxt.pieces) {
      pipe.load_sm_piece(nxt, p);
      ++nxt_issued;
    }
  }
};

// PITCH = 256: the rows of a tile follow one another (linear layout), so that a row's offset is a constant of the
// unrolled decode loop; PITCH = 0: the pitch is the tensor's (blocked layout).
template <uint32_t PITCH>
struct GlobalSink {
  uint16_t *out;
  uint32_t pitch;
  __device__ __forceinline__ void group(uint32_t i, uint32_t lane, const uint4 &v) const {
    __stcs(reinterpret_cast<uint4 *>(out + (size_t)i * (PITCH ? PITCH : pitch) + lane * 8), v);
  }
  __device__ __forceinline__ void elem(uint32_t i, uint32_t lane, uint32_t j, uint16_t v) const {
    out[(size_t)i * (PITCH ? PITCH : pitch) + lane * 8 + j] = v;
  }
};

// A resolved tile in five words, so that the 32 lanes of a warp can each resolve one of the warp's next 32 tiles at
// once and hand them out by shuffle: resolving a tile costs a warp ~100 instructions, fetching a resolved one ~15.
//   rec16  : record, 16-byte units from `payload`;  sm16 : sign+mantissa bytes, 16-byte units from `sm`;
//   out8   : first element, 8-element units from `out`;  pitch;
//   bits   : valid (13 bits) | iterations << 13 (5) | record size in 16-byte units << 18 (10) | staged << 30 | ok << 31
struct PackedTile {
  uint32_t rec16, sm16, out8, pitch, bits;
};
__device__ __forceinline__ PackedTile pack_tile(const LaunchArgs &a, const TileWork &w) {
  PackedTile p = {0, 0, 0, 0, 0};
  if (!w.ok) return p;
  const uint64_t r = (uint64_t)(w.rec - a.payload) >> 4, s = (uint64_t)(w.sm - a.sm) >> 4;
  const uint64_t o = (uint64_t)(w.out - a.out) >> 3;
  if ((r | s | o) >> 32) return p;   // beyond what the packed form addresses (64 GB of input, 32 G elements of output)
  p.rec16 = (uint32_t)r;
  p.sm16 = (uint32_t)s;
  p.out8 = (uint32_t)o;
  p.pitch = w.pitch;
  p.bits = w.valid | (w.iters << 13) | ((w.rec_bytes >> 4) << 18) | ((w.staged ? 1u : 0u) << 30) | (1u << 31);
  return p;
}
// lane `src`'s packed tile, unpacked in every lane
__device__ __forceinline__ TileWork fetch_tile(const LaunchArgs &a, const PackedTile &mine, uint32_t src) {
  // a warp-wide OR over "lane src's word, zero elsewhere" instead of a shuffle: the result of a warp reduction is
  // known to be the same in every lane, so the tile's addresses and sizes live in uniform registers
  const bool me = (threadIdx.x & 31u) == src;
  const uint32_t bits = __reduce_or_sync(0xFFFFFFFFu, me ? mine.bits : 0u);
  const uint32_t rec16 = __reduce_or_sync(0xFFFFFFFFu, me ? mine.rec16 : 0u);
  const uint32_t sm16 = __reduce_or_sync(0xFFFFFFFFu, me ? mine.sm16 : 0u);
  const uint32_t out8 = __reduce_or_sync(0xFFFFFFFFu, me ? mine.out8 : 0u);
  TileWork w;
  w.n_sub = 1;
  w.pitch = __reduce_or_sync(0xFFFFFFFFu, me ? mine.pitch : 0u);
  w.ok = bits >> 31;
  w.staged = (bits >> 30) & 1u;
  w.valid = bits & 0x1FFFu;
  w.iters = (bits >> 13) & 31u;
  w.pieces = sm_pieces_of_tile(w.valid);
  w.rec_bytes = ((bits >> 18) & 0x3FFu) << 4;
  w.rec = a.payload + ((size_t)rec16 << 4);
  w.sm = a.sm + ((size_t)sm16 << 4);
  w.out = a.out + ((size_t)out8 << 3);
  return w;
}

// Like fetch_tile, but small tiles are taken several at a time: if the tile of lane `at` is a full tile of 2, 4 or 8
// iterations of a linear tensor (a whole number of tiles per piece of sign+mantissa bytes, so that no tile lies
// across two pieces), the tiles of the following lanes join it as long as they
// are full tiles of the same size, their sign+mantissa bytes and outputs continue where the previous tile's end,
// their records ascend, the whole span of records fits the record stage and the step stays within 4096 elements.
// Lane i comes back with offset and size of the step's i-th record (sub_off, sub_bytes) and every lane with the tile
// size in iterations (sub_iters).
__device__ __forceinline__ TileWork fetch_step(const LaunchArgs &a, const PackedTile &mine, uint32_t at, uint32_t stage_buf,
                                               uint32_t &sub_off, uint32_t &sub_bytes, uint32_t &sub_iters) {
  TileWork w = fetch_tile(a, mine, at);
  sub_off = 0;
  sub_bytes = w.rec_bytes;
  sub_iters = w.iters;
  if (!w.ok || !w.staged || w.pitch != 256u || w.iters > kPieceIters || (w.iters & 1u) || kPieceIters % w.iters != 0 ||
      w.valid != w.iters * 256u)
    return w;
  const uint32_t lane = threadIdx.x & 31u, i = lane - at, most = 16u / w.iters;
  const uint32_t first_rec = __shfl_sync(0xFFFFFFFFu, mine.rec16, at), first_sm = __shfl_sync(0xFFFFFFFFu, mine.sm16, at);
  const uint32_t first_out = __shfl_sync(0xFFFFFFFFu, mine.out8, at);
  const uint32_t my_units = (mine.bits >> 18) & 0x3FFu, my_end = mine.rec16 + my_units;
  const uint32_t prev_end = __shfl_up_sync(0xFFFFFFFFu, my_end, 1);
  const bool joins = lane >= at && i < most && (mine.bits >> 30) == 3u /* ok and staged */ &&
                     ((mine.bits >> 13) & 31u) == w.iters && (mine.bits & 0x1FFFu) == w.valid && mine.pitch == 256u &&
                     mine.sm16 == first_sm + i * (w.valid >> 4) && mine.out8 == first_out + i * (w.valid >> 3) &&
                     (i == 0 || mine.rec16 >= prev_end) && mine.rec16 >= first_rec &&
                     (uint64_t)(my_end - first_rec) * 16u <= stage_buf;
  const uint32_t run = ~(__ballot_sync(0xFFFFFFFFu, joins) >> at);   // zero bits = consecutive tiles that join
  const uint32_t n = min(most, run ? (uint32_t)__ffs(run) - 1u : 32u - at);
  if (n < 2) return w;
  const uint32_t src = min(at + lane, 31u);
  sub_off = (__shfl_sync(0xFFFFFFFFu, mine.rec16, src) - first_rec) * 16u;
  sub_bytes = __shfl_sync(0xFFFFFFFFu, my_units, src) * 16u;
  w.n_sub = n;
  w.rec_bytes = (__shfl_sync(0xFFFFFFFFu, my_end, at + n - 1) - first_rec) * 16u;
  w.valid *= n;
  w.iters *= n;
  w.pieces = sm_pieces_of_tile(w.valid);
  return w;
}

// BATCHED: tiles are resolved 32 at a time, one per lane, instead of one by one by the whole warp.  That pays when
// tiles are small or tensors many; with few large tensors of full tiles the one-by-one form keeps the hot loop leaner
// and is 3 % faster.  The host picks by the launch's tiles per tensor.
// LEAN: only the common path is compiled in -- record staged in shared memory, codes of at most 8 bits -- on the
// caller's promise (ZIPMOE_DECODE_SHORT_CODES) that the launch has nothing else; a tile that does is reported and
// left undecoded.  The shorter code is worth 2-3 %.
template <bool WIDE, bool BATCHED, bool LEAN = false>
__global__ void __launch_bounds__(Cfg<WIDE>::kThreads, Cfg<WIDE>::kCtasPerSm) decode_kernel(const LaunchArgs a) {
  using C = Cfg<WIDE>;
  constexpr int kWarps = C::kWarps, kWarpBytes = C::kWarpBytes;
  constexpr uint32_t kBuf = C::kBuf;
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Teams: a dynamically distributed launch with narrow stages splits its warps into two teams, each with its own
  // table, its own ranges of tiles and its own barrier, so that while one team changes tensors (waits for its
  // last warp, builds the table, fetches the first records) the other keeps decoding, and a tensor of a few
  // tiles leaves half as many warps without work.  Otherwise the CTA is one team.
  constexpr int kTeams = (BATCHED && !WIDE) ? 2 : 1;
  constexpr int kTeamWarps = kWarps / kTeams, kTeamThreads = kTeamWarps * 32;
  static_assert(kTeams <= C::kMaxLuts && kWarps % kTeams == 0 && kTeamThreads >= 256, "teams");
  const uint32_t team = warp / kTeamWarps, tw = warp - team * kTeamWarps, ttid = tid - team * kTeamThreads;
  const uint32_t bar_id = kTeams > 1 ? team + 1 : 0;
  uint8_t *lut_raw = smem + team * kLutBytes;
  uint8_t *warp_base = smem + kTeams * kLutBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(warp_base + kWarps * kWarpBytes);
  uint8_t *lut_scratch = reinterpret_cast<uint8_t *>(bars + kWarps * kBarsPerWarp) + team * kLutScratchBytes;

  uint32_t g0 = blockIdx.x * a.tiles_per_cta;
  uint32_t g1 = min(g0 + a.tiles_per_cta, a.n_tiles);
  if (!BATCHED && g0 >= g1) return;
  __shared__ uint32_t s_grab[2][2];   // BATCHED: the range of tiles each team took last

  WarpPipe pipe;
  pipe.pay_addr = smem_addr(warp_base + warp * kWarpBytes);
  pipe.stage_bytes = C::kStage;
  pipe.sm_addr = pipe.pay_addr + kPayStages * C::kStage;
  pipe.bar_addr = smem_addr(bars + warp * kBarsPerWarp);
  pipe.tries = a.wait_tries;
  pipe.extra_tx = a.extra_tx;
  pipe.phase = 0;
  pipe.pending = 0;
  pipe.lane = lane;
  const uint32_t lut = smem_addr(lut_raw);
  if (lane == 0)
    for (int b = 0; b < kBarsPerWarp; ++b) mbar_init(pipe.bar(b), 1);
  fence_barrier_init();
  __syncthreads();

  bool dead = false;    // this warp gave up after a wait ran out
  uint32_t lut_table = 0xFFFFFFFFu;   // BATCHED: the table in shared memory
  bool fast = true;
  // BATCHED: the launch's tiles are handed out dynamically, in ranges that shrink as the work runs out (half of what
  // an even split of the rest would give, at least kMinGrab tiles: measured best among halves, thirds, quarters
  // and minima of 1..32 tiles per warp), because tiles and tensors of such launches differ too much in cost for
  // equal shares to finish together.  Otherwise the CTA has its one fixed range.
#ifndef ZIPMOE_GRAB_MIN
#define ZIPMOE_GRAB_MIN 8
#endif
#ifndef ZIPMOE_GRAB_DIV
#define ZIPMOE_GRAB_DIV 2
#endif
  constexpr uint32_t kMinGrab = ZIPMOE_GRAB_MIN * kTeamWarps;
  for (;;) {
  if (BATCHED) {
    group_sync(bar_id, kTeamThreads);   // s_grab of the previous round has been read by every thread of the team
    if (ttid == 0) {
      // The counter is one 64-bit word: the tag of the launch that owns it above the next tile not yet handed out.
      // It was zeroed on the stream before this kernel; the first CTA to arrive installs the launch's tag.  Should
      // two launches ever be given the same counter while both are in flight (more of them queued than the ring
      // has slots), a CTA that finds the other launch's tag reports that and takes no more tiles, so that
      // incomplete output does not go unnoticed.  (The tag is checked before the range is taken, not in the same
      // atomic step: a compare-and-swap loop would make the CTAs of a launch queue up behind one another.)
      unsigned long long *ctr = reinterpret_cast<unsigned long long *>(a.work_counter);
      const unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(ctr);
      uint32_t tag = (uint32_t)(old >> 32);
      const uint32_t seen = (uint32_t)old;
      if (tag == 0u) {
        const uint32_t prev = atomicCAS(a.work_counter + 1, 0u, a.work_tag);   // the upper word
        tag = prev ? prev : a.work_tag;
      }
      uint32_t first = a.n_tiles, take = 0;
      if (tag != a.work_tag) {
        report(a.status, kStatusCounterShared);
      } else if (seen < a.n_tiles) {
        take = (a.n_tiles - seen) / (ZIPMOE_GRAB_DIV * kTeams * gridDim.x);
        take = max(take, max(1u, min(kMinGrab, a.n_tiles / (kTeams * gridDim.x))));   // small launches: spread over all teams
        first = (uint32_t)atomicAdd(ctr, (unsigned long long)take);
        take = first < a.n_tiles ? min(a.n_tiles - first, take) : 0u;
        if (take == 0) first = a.n_tiles;
      }
      s_grab[team][0] = first;
      s_grab[team][1] = first + take;
    }
    group_sync(bar_id, kTeamThreads);
    g0 = s_grab[team][0];
    g1 = s_grab[team][1];
    if (g0 >= g1) break;
  }
  uint32_t c = find_chunk(a, g0);

  while (g0 < g1) {
    const zipmoe_chunk_desc *d = a.chunks + c;
    const uint32_t table_id = __ldg(&d->table_id), run_first_chunk = __ldg(&d->run_first_chunk);
    const uint32_t run_first_tile = __ldg(&d->run_first_tile), run_end_tile = __ldg(&d->run_end_tile);
    const uint32_t tpc = __ldg(&d->tiles_per_chunk);
    const uint32_t seg_end = min(g1, run_end_tile);
    if (seg_end <= g0 || run_first_tile > g0 || tpc == 0 || table_id >= a.n_tables) {
      report(a.status, kStatusBadDescriptor);
      break;
    }
    // Each warp takes a contiguous share of the segment's tiles: consecutive tiles sit in the same chunk, so the
    // descriptor and the tile-table entries of the next tile are usually in the first-level cache already.
    const uint32_t share = (seg_end - g0 + kTeamWarps - 1) / kTeamWarps;
    uint32_t g = g0 + tw * share;
    const uint32_t g_end = min(seg_end, g + share);
    uint32_t stage = 0;
    constexpr bool batched = BATCHED;
    uint32_t tc = 0, tt = 0;   // descriptor and tile-in-chunk of this warp's next tile, stepped without divisions
    if (g < g_end) {
      tc = run_first_chunk + (g - run_first_tile) / tpc;
      tt = (g - run_first_tile) % tpc;
    }
    // Lane L resolves tile `first + L` of the warp's share: descriptor, tile-table entry and every bounds check
    // for 32 tiles at the price of one.  (An unresolvable tile comes back with ok = false.)
    auto resolve_batch = [&](uint32_t first) -> PackedTile {
      TileWork w;
      w.ok = false;
      const uint32_t mine = first + lane;
      if (mine < g_end) {
        const uint32_t rel = mine - run_first_tile;
        w = resolve_tile(a, run_first_chunk + rel / tpc, rel % tpc, kBuf, table_id);
      }
      return pack_tile(a, w);
    };
    // the warp's first tile of the segment is fetched while the table is being built (its own stages and
    // slots are free: it has finished its tiles of the previous segment)
    PackedTile batch = {0, 0, 0, 0, 0};
    TileWork cur;
    cur.ok = false;
    cur.n_sub = 1;
    // small tiles are taken several at a time (only where codes of at most 8 bits are promised: decode_step)
    constexpr bool steps = BATCHED && LEAN;
    uint32_t cur_off = 0, cur_bytes = 0, cur_sub_iters = 0, nxt_off = 0, nxt_bytes = 0, nxt_sub_iters = 0;
    if (g < g_end && !dead) {
      if (batched) {
        batch = resolve_batch(g);
        cur = steps ? fetch_step(a, batch, 0, kBuf, cur_off, cur_bytes, cur_sub_iters) : fetch_tile(a, batch, 0);
      } else {
        cur = resolve_tile(a, tc, tt, kBuf, table_id);
      }
      if (!cur.ok) report(a.status, kStatusBadDescriptor);
      else {
        pipe.load_record(cur, stage);
        for (uint32_t p = 0; p < cur.pieces; ++p) pipe.load_sm_piece(cur, p);
      }
    }
    if (!BATCHED || table_id != lut_table) {
      group_sync(bar_id, kTeamThreads);  // every warp of the team is done with the previous table
      fast = build_lut(kTeamThreads, a.tables[table_id].code_len, lut_raw, lut_scratch, a.status, ttid, bar_id) <=
             (uint32_t)kLaneLutBits;
      lut_table = table_id;
    }

    uint32_t advance = 1;   // tiles of the step being decoded
    for (uint32_t in_batch = cur.n_sub; g < g_end && !dead; g += advance) {   // in_batch: tiles of the batch handed out
      TileWork nxt;
      nxt.ok = false;
      nxt.n_sub = 1;
      uint32_t nxt_issued = 0;
      advance = cur.n_sub;
      if (g + advance < g_end) {
        if (batched) {
          if (in_batch == 32) {   // the batch is used up
            batch = resolve_batch(g + advance);
            in_batch = 0;
          }
          nxt = steps ? fetch_step(a, batch, in_batch, kBuf, nxt_off, nxt_bytes, nxt_sub_iters) : fetch_tile(a, batch, in_batch);
          in_batch += nxt.n_sub;
        } else {
          if (++tt == tpc) {
            tt = 0;
            ++tc;
          }
          nxt = resolve_tile(a, tc, tt, kBuf, table_id);
        }
        if (!nxt.ok) report(a.status, kStatusBadDescriptor);
      }
      // the next record is fetched while this one is decoded
      if (nxt.ok) pipe.load_record(nxt, stage ^ 1);   // that stage was released by the __syncwarp below
      if (cur.ok) {
        uint32_t rc = 0;
        if (cur.staged && !pipe.wait(stage)) rc = kStatusWaitTimeout;
        if (rc == 0) {
          const uint32_t rec_s = pipe.pay_addr + stage * pipe.stage_bytes;
          SmFeed feed{pipe, nxt, nxt_issued};
          GlobalSink<0> sink{cur.out, cur.pitch};
          if (LEAN) {
            if (!(cur.staged && fast)) {
              rc = kStatusBrokenPromise;
            } else if (cur.pitch == 256u) {
              GlobalSink<256> rows{cur.out, 256u};
              if (steps && cur.n_sub > 1)
                rc = decode_step(rec_s, cur_off, cur_bytes, cur.n_sub, cur_sub_iters, lut, lane, feed, rows);
              else
                rc = decode_tile<true, true, BATCHED>(rec_s, nullptr, cur.rec_bytes, lut, cur.valid, cur.iters, lane, feed, rows);
            } else {
              rc = decode_tile<true, true, BATCHED>(rec_s, nullptr, cur.rec_bytes, lut, cur.valid, cur.iters, lane, feed, sink);
            }
          } else if (cur.staged) {
            rc = fast ? decode_tile<true, true, BATCHED>(rec_s, nullptr, cur.rec_bytes, lut, cur.valid,
                                                  cur.iters, lane, feed, sink)
                        : decode_tile<true, false, BATCHED>(rec_s, nullptr, cur.rec_bytes, lut, cur.valid,
                                                   cur.iters, lane, feed, sink);
          } else {
            rc = fast ? decode_tile<false, true, BATCHED>(0, cur.rec, cur.rec_bytes, lut, cur.valid,
                                                   cur.iters, lane, feed, sink)
                        : decode_tile<false, false, BATCHED>(0, cur.rec, cur.rec_bytes, lut, cur.valid,
                                                    cur.iters, lane, feed, sink);
          }
        }
        if (rc == kStatusWaitTimeout) {
          report(a.status, rc);
          pipe.drain();
          dead = true;
          break;
        }
        if (rc == kStatusBrokenPromise) {
          // nothing was decoded: take the tile's sign+mantissa pieces off the barriers
          report(a.status, rc);
          for (uint32_t p = 0; p < cur.pieces && !dead; ++p)
            if (!pipe.wait(kPayStages + p)) dead = true;
          if (dead) {
            report(a.status, kStatusWaitTimeout);
            pipe.drain();
            break;
          }
        }
      }
      __syncwarp();   // every lane is done with the current record stage and SM slots
      if (nxt.ok)
        for (; nxt_issued < nxt.pieces; ++nxt_issued) pipe.load_sm_piece(nxt, nxt_issued);
      cur = nxt;
      cur_off = nxt_off;
      cur_bytes = nxt_bytes;
      cur_sub_iters = nxt_sub_iters;
      stage ^= 1;
    }
    g0 = seg_end;
    c = run_first_chunk + (run_end_tile - run_first_tile + tpc - 1) / tpc;
    if (g0 < g1 && c >= a.n_chunks) {
      report(a.status, kStatusBadDescriptor);
      break;
    }
  }
  if (!BATCHED) break;
  }
}

}  // namespace zipmoe_dev

namespace {
// Work counters of the dynamically distributed launches: a small ring in the library's own device memory, one
// word per launch, zeroed on the launch's stream right before the kernel.  A slot comes round again after
// kCounterSlots launches of that kind; by then the launch that had it has long finished.
constexpr uint32_t kCounterSlots = 1024;
static __device__ unsigned long long g_work_counters[kCounterSlots];   // per slot: tag of the owning launch << 32 | next tile
std::atomic<uint32_t> g_next_slot{0};
std::atomic<uint32_t> g_test_extra_tx{0}, g_test_tries{zipmoe_host::kWaitTries}, g_test_foreign_counter{0};

struct DeviceInfo {
  int sm_count = 0;
  bool ready = false;
  uint32_t *counters = nullptr;   // device address of g_work_counters on this device
};
DeviceInfo g_dev[64];

zipmoe_status prepare_device(int *sm_count, uint32_t **counters) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ZIPMOE_ERR_CUDA;
  if (!g_dev[dev].ready) {
    int sms = 0, major = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return ZIPMOE_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ZIPMOE_ERR_CUDA;
    if (major != 10) return ZIPMOE_ERR_UNSUPPORTED;
    using namespace zipmoe_dev;
    const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
    if (cudaFuncSetAttribute(decode_kernel<true, true>, at, Cfg<true>::smem_bytes(1)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_kernel<true, false>, at, Cfg<true>::smem_bytes(1)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_kernel<false, true>, at, Cfg<false>::smem_bytes(2)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_kernel<false, false>, at, Cfg<false>::smem_bytes(1)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_kernel<false, true, true>, at, Cfg<false>::smem_bytes(2)) != cudaSuccess ||
        cudaFuncSetAttribute(decode_kernel<false, false, true>, at, Cfg<false>::smem_bytes(1)) != cudaSuccess)
      return ZIPMOE_ERR_CUDA;
    void *ptr = nullptr;   // (in host code the array's name is not a device address: ask for it)
    if (cudaGetSymbolAddress(&ptr, g_work_counters) != cudaSuccess || !ptr) return ZIPMOE_ERR_CUDA;
    g_dev[dev].counters = static_cast<uint32_t *>(ptr);
    g_dev[dev].sm_count = sms;
    g_dev[dev].ready = true;
  }
  *sm_count = g_dev[dev].sm_count;
  *counters = g_dev[dev].counters;
  return ZIPMOE_OK;
}
}  // namespace

void zipmoe_host::wait_fault_setting(uint32_t *extra_tx, uint32_t *tries) {
  *extra_tx = g_test_extra_tx.load();
  *tries = g_test_tries.load();
}

extern "C" void zipmoe_test_foreign_counter(uint32_t on) { g_test_foreign_counter.store(on ? 1u : 0u); }

extern "C" void zipmoe_test_wait_fault(uint32_t extra_tx_bytes, uint32_t tries) {
  g_test_extra_tx.store(extra_tx_bytes & ~15u);
  g_test_tries.store(tries ? tries : zipmoe_host::kWaitTries);
}

extern "C" zipmoe_status zipmoe_decode(const zipmoe_chunk_desc *chunks, uint32_t n_chunks, uint32_t n_tiles,
                                       const zipmoe_table *tables, uint32_t n_tables, const uint8_t *payload,
                                       uint64_t payload_bytes, const uint8_t *sm, uint64_t sm_bytes,
                                       uint16_t *out_bf16, uint64_t out_elems, uint32_t *status_word,
                                       zipmoe_stream stream, uint32_t max_record_bytes, uint32_t flags) {
  zipmoe_host::TraceRange trace("zipmoe_decode");
  if (n_chunks == 0 || n_tiles == 0) return (n_chunks == 0 && n_tiles == 0) ? ZIPMOE_OK : ZIPMOE_ERR_INVALID_ARG;
  if (!chunks || !tables || n_tables == 0 || !payload || !sm || !out_bf16) return ZIPMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(payload) | reinterpret_cast<uintptr_t>(sm) | reinterpret_cast<uintptr_t>(out_bf16) |
       reinterpret_cast<uintptr_t>(chunks)) & 15)
    return ZIPMOE_ERR_INVALID_ARG;
  if (status_word && (reinterpret_cast<uintptr_t>(status_word) & 3)) return ZIPMOE_ERR_INVALID_ARG;
  int sms = 0;
  uint32_t *counters = nullptr;
  zipmoe_status rc = prepare_device(&sms, &counters);
  if (rc != ZIPMOE_OK) return rc;

  zipmoe_dev::LaunchArgs a;
  a.chunks = chunks;
  a.tables = tables;
  a.payload = payload;
  a.sm = sm;
  a.out = out_bf16;
  a.status = status_word;
  a.payload_bytes = payload_bytes;
  a.sm_bytes = sm_bytes;
  a.out_elems = out_elems;
  a.n_chunks = n_chunks;
  a.n_tiles = n_tiles;
  a.n_tables = n_tables;
  zipmoe_host::wait_fault_setting(&a.extra_tx, &a.wait_tries);
  // CTAs to fill the SMs once, each with a contiguous range of tiles
  const bool narrow = max_record_bytes != 0 && max_record_bytes <= (uint32_t)zipmoe_dev::Cfg<false>::kBuf;
  uint32_t ctas = (uint32_t)sms * (narrow ? zipmoe_dev::Cfg<false>::kCtasPerSm : zipmoe_dev::Cfg<true>::kCtasPerSm);
  if (n_tiles < ctas) ctas = n_tiles;
  a.tiles_per_cta = (n_tiles + ctas - 1) / ctas;
  ctas = (n_tiles + a.tiles_per_cta - 1) / a.tiles_per_cta;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  using Narrow = zipmoe_dev::Cfg<false>;
  using Wide = zipmoe_dev::Cfg<true>;
  // few large tensors (at least 512 tiles each on average): tiles resolved one by one, an equal range of tiles per
  // CTA; else tiles resolved 32 at a time and handed to the CTAs dynamically (one CTA per SM either way)
  const bool batched = (uint64_t)n_tiles < 512ull * n_tables;
  a.work_counter = nullptr;
  a.work_tag = 0;
  if (batched) {
    const uint32_t seq = g_next_slot.fetch_add(1);
    a.work_counter = counters + 2 * (seq % kCounterSlots);
    a.work_tag = seq | 0x80000000u;   // never zero; differs between any two launches that can meet on a slot
    // (the library's own tests can have the counter filled with 0x7F7F7F7F, a tag no launch carries: tags have bit 31 set)
    if (cudaMemsetAsync(a.work_counter, g_test_foreign_counter.load() ? 0x7F : 0, 8, st) != cudaSuccess) return ZIPMOE_ERR_CUDA;
    ctas = (uint32_t)sms * (narrow ? zipmoe_dev::Cfg<false>::kCtasPerSm : 1u);
    const uint32_t most = (n_tiles + 15 - 1) / 15;   // a tile per warp at least
    if (ctas > most) ctas = most;
  }
  const bool lean = narrow && (flags & ZIPMOE_DECODE_SHORT_CODES);
  if (lean && batched)
    zipmoe_dev::decode_kernel<false, true, true><<<ctas, Narrow::kThreads, Narrow::smem_bytes(2), st>>>(a);
  else if (lean) zipmoe_dev::decode_kernel<false, false, true><<<ctas, Narrow::kThreads, Narrow::smem_bytes(1), st>>>(a);
  else if (narrow && batched)
    zipmoe_dev::decode_kernel<false, true><<<ctas, Narrow::kThreads, Narrow::smem_bytes(2), st>>>(a);
  else if (narrow) zipmoe_dev::decode_kernel<false, false><<<ctas, Narrow::kThreads, Narrow::smem_bytes(1), st>>>(a);
  else if (batched) zipmoe_dev::decode_kernel<true, true><<<ctas, Wide::kThreads, Wide::smem_bytes(1), st>>>(a);
  else zipmoe_dev::decode_kernel<true, false><<<ctas, Wide::kThreads, Wide::smem_bytes(1), st>>>(a);
  return cudaGetLastError() == cudaSuccess ? ZIPMOE_OK : ZIPMOE_ERR_CUDA;
}
