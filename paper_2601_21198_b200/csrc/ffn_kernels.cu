// Fused decode + routed expert FFN for sm_100a.  The paper's step is the GPU
// execution of the tokens routed to an expert once its tensors are recovered
// (Section 3.3, p_n in the scheduler's notation); here the recovery and the
// three projections are one pass: every weight tile is decoded from its E-chunk
// and SM-chunk straight into a shared-memory operand tile and consumed by
// tcgen05 tensor-core MMAs, so decoded weights never reach global memory.
//
// One kernel, ffn_matmul_kernel, computes  Y[slot, row] = sum_k W[row, k] * X[slot, k]
// for the token slots routed to the experts that have tokens.  A job is one
// expert, one compressed matrix W (blocked layout: tiles of 16 rows x 256 columns)
// and one group of 16-row strips; a job has K / 256 steps.  The kernel is
// persistent: the steps of all jobs form one sequence that is cut into equal,
// contiguous shares, one per CTA (one CTA per SM), so that every SM decodes the
// same number of tiles whatever the number of experts with tokens.  A CTA works
// through its share piece by piece (a piece = consecutive steps of one job);
// where a job is cut between CTAs each writes a partial sum, added later by the
// elementwise kernels.  Within a piece:
//   * each decode warp owns one strip and walks its tiles along K.  A tile is
//     decoded in two halves of 8 rows.  Eight warps form a group: their eight
//     half-tile buffers (8 rows x 256 columns each, K-major, no swizzle) are
//     the eight 8-row groups of one A operand of M = 64.  A half is decoded
//     into registers first and stored once the MMAs that read the previous
//     half are done, so decode and MMA overlap;
//   * one MMA warp per group waits for the group's half to be complete and
//     issues its 16 MMAs (K = 16 each; B = the activations, N = token rows);
//     accumulators live in tensor memory, one [64 x N] fp32 block per group and half;
//   * one loader warp stages the activations in half K steps (token rows x 128
//     bf16) in a three-stage ring shared by all groups;
//   * at the end four warps read the accumulators back (tcgen05.ld) and store Y.
// The host wrapper runs it for W1 and W3 (gate, up), applies SiLU(g)*u, runs it
// for W2, and combines the experts of every token.
// Every wait on a barrier is bounded; a wait that runs out is reported through
// the status word and the kernel still runs to its end and frees tensor memory.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

#include "zipmoe.h"
#include "decode_device.cuh"

namespace zipmoe_dev {

#ifndef ZIPMOE_FFN_WARPS
#define ZIPMOE_FFN_WARPS 16
#endif
constexpr int kFfnMaxWarps = ZIPMOE_FFN_WARPS;            // decode warps per CTA, a multiple of the group size
#ifndef ZIPMOE_FFN_GROUP
#define ZIPMOE_FFN_GROUP 16
#endif
constexpr int kGroupWarps = ZIPMOE_FFN_GROUP;            // decode warps whose half-tiles form one operand of M = 8 * kGroupWarps (64 or 128)
static_assert(kGroupWarps == 8 || kGroupWarps == 16, "M is 64 or 128");
constexpr int kFfnGroups = (kFfnMaxWarps + kGroupWarps - 1) / kGroupWarps;             // the last group may be incomplete
constexpr int kFfnMaxThreads = (kFfnMaxWarps + kFfnGroups + 1) * 32;                   // decode, one MMA warp per group, loader
constexpr uint32_t kBLbo = 144;                          // bytes between the 8x8 cores of a half-tile along K: 128 + 16 of
                                                         // padding, so that the 32 lanes' 16-byte stores spread over all banks
constexpr uint32_t kBBufBytes = 32 * kBLbo;              // one half-tile: 8 rows x 256 columns
constexpr uint32_t kXGroupBytes = 2048;                  // 8 token rows x 128 columns of bf16, cores 128 bytes apart
constexpr uint32_t kXStages = 3;                         // half K steps in the activation ring: one whole step and half of the next
constexpr uint32_t kFfnWarpBytes = 2 * kPayStage + kBBufBytes;   // two record stages, one half-tile buffer
constexpr uint32_t kFfnShortTries = 1u << 10;            // wait limit once something has already gone wrong

struct FfnArgs {
  LaunchArgs la;                       // descriptors, tables, payload and SM buffers of all expert tensors
  const uint32_t *tensor_first_chunk;  // [3E] first descriptor of tensor e*3 + {0 w1, 1 w3, 2 w2}
  const uint32_t *expert_offset;       // [E+1] first slot of each expert
  const uint32_t *active;              // [0] number of experts with tokens, [1..] their ids
  const uint32_t *slot_token;          // [S] token of each slot, or null when X rows are the slots themselves
  const uint16_t *x;                   // bf16 activations, row pitch K
  float *y;                            // [n_mats][max_parts][S][rows] partial sums
  uint32_t rows, K;                    // every matrix of the launch is [rows, K]
  uint32_t tensor_base, n_mats;        // tensors tensor_base .. tensor_base + n_mats - 1 of every active expert
  uint32_t n_groups;                   // strip groups (16 * n_warps rows each) per matrix
  uint32_t min_units, max_parts;       // smallest share of a CTA in steps; bound on the CTAs a job is cut between
  uint32_t n_warps, groups, S;         // decode warps, 8-row groups of token rows per stage, total slots
  uint32_t smem_bytes;                 // dynamic shared memory of the launch
};

// The kernels of one call are launched with programmatic stream serialization: each may be set up on the SMs while
// its predecessor is still running, waits here until that one has completed and its memory is visible, and then
// lets its own successor do the same.  (Launched the ordinary way, the wait returns at once.)
__device__ __forceinline__ void after_previous_kernel() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- how the steps of a launch are shared out --------------------------------------------------
// U units (steps of all jobs, job-major) go to P CTAs; CTA c takes [c*U/P, (c+1)*U/P).  P is chosen so that
// every CTA gets at least min_units units, hence a job of `steps` units is cut between at most
// ceil(steps / min_units) + 1 CTAs.
__host__ __device__ inline uint32_t ffn_ctas_in_use(uint64_t U, uint32_t grid, uint32_t min_units) {
  uint64_t p = U / (min_units ? min_units : 1);
  if (p < 1) p = 1;
  return p < grid ? (uint32_t)p : grid;
}
__host__ __device__ inline uint64_t ffn_first_unit(uint32_t c, uint64_t U, uint32_t P) { return (uint64_t)c * U / P; }
__host__ __device__ inline uint32_t ffn_cta_of_unit(uint64_t u, uint64_t U, uint32_t P) {
  return (uint32_t)(((u + 1) * P - 1) / U);
}
// the CTAs that share job `job`: the first one, and how many
__host__ __device__ inline void ffn_job_parts(uint64_t job, uint32_t steps, uint64_t U, uint32_t P, uint32_t *first_cta,
                                              uint32_t *parts) {
  const uint32_t c0 = ffn_cta_of_unit(job * steps, U, P), c1 = ffn_cta_of_unit(job * steps + steps - 1, U, P);
  *first_cta = c0;
  *parts = c1 - c0 + 1;
}

// shared-memory layout: [X stages][per-warp buffers][tables][table scratch][barriers][tmem slot]
__host__ __device__ inline uint32_t ffn_bar_count(uint32_t n_warps) {
  return 2 * n_warps + 2 * ((n_warps + kGroupWarps - 1) / kGroupWarps) + 2 * kXStages;   // the word after them is the CTA's give-up flag
}
__host__ __device__ inline uint32_t ffn_smem_bytes(uint32_t n_warps, uint32_t groups) {
  const uint32_t after_warps = (uint32_t)kLutBytes + kLutScratchBytes + ffn_bar_count(n_warps) * 8 + 16;
  return kXStages * groups * kXGroupBytes + n_warps * kFfnWarpBytes + after_warps;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void sts_v4(uint32_t addr, const uint4 &v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// ordered with the other volatile asm of the decoder, so the load is issued where it is written: early
__device__ __forceinline__ uint2 ldg_v2_early(const uint8_t *p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// K-major, no-swizzle shared-memory matrix descriptor: 8x8 cores (8 rows of 16
// bytes, contiguous), `lbo` bytes between cores along K, `sbo` bytes between
// 8-row groups.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, one CTA
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}
// the barrier gets one arrival once every MMA issued so far by this thread has completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__global__ void __launch_bounds__(kFfnMaxThreads, 1) ffn_matmul_kernel(const FfnArgs a) {
  constexpr uint32_t kMyLutBytes = kLutBytes;
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t NW = a.n_warps, G = a.groups, Q = (NW + kGroupWarps - 1) / kGroupWarps, NCOL = 8 * G;
  // accumulator columns per group and half = N of the MMAs: with M = 128, N is a multiple of 16 (for up to 8 token
  // rows the operand then also covers the 8 rows after the stage's, whose columns come out as garbage and are
  // never read back)
  const uint32_t NACC = kGroupWarps == 16 ? (NCOL + 15u) & ~15u : NCOL;
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  after_previous_kernel();

  // ---- this CTA's share of the launch's steps ----
  const uint32_t n_active = __ldg(a.active);   // experts that have tokens
  const uint32_t steps = a.K >> 8;
  const uint32_t U = n_active * a.n_mats * a.n_groups * steps;   // (the host made sure that this fits 32 bits)
  if (U == 0) return;
  const uint32_t P = ffn_ctas_in_use(U, gridDim.x, a.min_units);
  if (blockIdx.x >= P) return;
  uint32_t u = (uint32_t)ffn_first_unit(blockIdx.x, U, P);
  const uint32_t u_end = (uint32_t)ffn_first_unit(blockIdx.x + 1, U, P);

  uint8_t *x_raw = smem;                                   // [kXStages][G][2048]
  uint8_t *warp_raw = x_raw + kXStages * G * kXGroupBytes; // [NW][2 record stages | half-tile buffer]
  uint8_t *lut_raw = warp_raw + NW * kFfnWarpBytes;
  uint8_t *lut_scratch = lut_raw + kMyLutBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(lut_scratch + kLutScratchBytes);
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + ffn_bar_count(NW));
  volatile uint32_t *give_up = tmem_slot + 1;              // set once a wait ran out: the CTA stops after the piece
  // barriers: [NW][2] record stages, [Q] group's half written, [Q] group's MMAs done, [3] X full, [3] X empty
  const uint32_t bar0 = smem_addr(bars);
  const uint32_t quad_full = bar0 + 8 * (2 * NW), quad_done = quad_full + 8 * Q;
  const uint32_t x_full = quad_done + 8 * Q, x_empty = x_full + 8 * kXStages;
  const uint32_t x_addr = smem_addr(x_raw), lut = smem_addr(lut_raw);
  const bool is_decode = warp < NW, is_mma = warp >= NW && warp < NW + Q, is_loader = warp == NW + Q;

  uint32_t tmem_cols = 32;
  while (tmem_cols < 2 * Q * NACC) tmem_cols <<= 1;
  if (tid == 0) {
    for (uint32_t b = 0; b < 2 * NW; ++b) mbar_init(bar0 + 8 * b, 1);
    for (uint32_t q = 0; q < Q; ++q) {
      mbar_init(quad_full + 8 * q, min((uint32_t)kGroupWarps, NW - q * kGroupWarps));   // the group's decode warps
      mbar_init(quad_done + 8 * q, 1);
    }
    for (uint32_t b = 0; b < kXStages; ++b) {
      mbar_init(x_full + 8 * b, 1);
      mbar_init(x_empty + 8 * b, Q);
    }
    *give_up = 0;
  }
  fence_barrier_init();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // (an incomplete last group: the MMA operand then also covers the bytes after the last warp's buffer, which
  // are the lookup table's, inside the allocation; the accumulator rows they produce are never read)
  const bool shape_ok = 2 * Q * NACC <= 512 && (kGroupWarps * Q - NW) * kFfnWarpBytes <= kMyLutBytes && steps > 0 &&
                        steps <= 64 && a.n_mats > 0 && a.n_groups > 0;
  if (!shape_ok) report(a.la.status, kStatusBadDescriptor);

  // The barriers are initialised once; every role counts what it has put through them since the kernel began,
  // so that the parity to wait for carries over from one piece to the next.
  const uint32_t my = smem_addr(warp_raw + (is_decode ? warp : 0) * kFfnWarpBytes);
  const uint32_t rec_bar = bar0 + 8 * (2 * (is_decode ? warp : 0));
  uint32_t rec_phase = 0, stage = 0;   // decode warp: parity of its two record stages, the stage of its next tile
  uint32_t hn = 0;                     // decode and MMA warps: halves the group has handed over so far
  uint32_t xst = 0, xround = 0;        // loader and MMA warps: ring stage of the next half K step, times the ring has gone round
  uint32_t lut_tensor = 0xFFFFFFFFu;   // the tensor whose table is in shared memory
  bool fast = true;

  while (shape_ok && u < u_end) {
    // ---- the piece: steps [s0, s0 + n_steps) of one job ----
    const uint32_t job = u / steps;
    const uint32_t s0 = u - job * steps;
    const uint32_t n_steps = min(steps - s0, u_end - u);
    const uint32_t grp = job % a.n_groups;
    const uint32_t jm = job / a.n_groups, mat = jm % a.n_mats, a_idx = jm / a.n_mats;
    const uint32_t part = blockIdx.x - ffn_cta_of_unit((uint64_t)job * steps, U, P);   // which of the job's partial sums
    u += n_steps;
    const uint32_t e = __ldg(a.active + 1 + a_idx);
    const uint32_t off = __ldg(a.expert_offset + e);
    uint32_t Te = __ldg(a.expert_offset + e + 1) - off;
    if (Te > NCOL) {       // more slots than the stage holds (a token listing the same expert twice)
      report(a.la.status, kStatusBadDescriptor);
      Te = NCOL;
    }
    const uint32_t n_strips = a.rows >> 4, strip = grp * NW + warp;
    const bool has_strip = is_decode && strip < n_strips;
    const uint32_t tensor = e * 3 + a.tensor_base + mat;

    // the tensor: blocked layout, 16 x 256 tiles, one Huffman table
    const uint32_t c0 = __ldg(a.tensor_first_chunk + tensor);
    bool ok = c0 < a.la.n_chunks && part < a.max_parts && Te > 0;
    uint32_t table_id = 0, tpc = 1;
    if (ok) {
      const zipmoe_chunk_desc *d = a.la.chunks + c0;
      table_id = __ldg(&d->table_id);
      tpc = __ldg(&d->tiles_per_chunk);
      ok = table_id < a.la.n_tables && tpc != 0 && __ldg(&d->row_pitch) == a.K &&
           __ldg(&d->tiles_per_rowblk) == steps && __ldg(&d->tile_elems) == ZIPMOE_TILE_ELEMS_MAX &&
           __ldg(&d->tile0) == 0;
    }
    if (!ok) {   // the same for every thread of the CTA: the piece is skipped
      report(a.la.status, kStatusBadDescriptor);
      continue;
    }
    // ---- decode warps: where the strip's tiles are, and the first fetches, while the table is being built ----
    bool failed = !has_strip;

    // Where the strip's tiles are: lane i (and i + 32) looks up record start and length of the i-th tile of
    // the piece once, so that the loop below touches global memory only for the data itself.
    uint32_t rec_at[2] = {0, 0}, rec_len[2] = {0, 0};   // in 16-byte units from the start of the payload buffer
    const uint8_t *sm_strip = a.la.sm;                  // sign+mantissa bytes of the strip's first tile
    if (!failed) {
      const uint32_t tq0 = strip * steps + s0;
      bool bad = false;
      for (uint32_t r = 0; r < 2; ++r) {
        const uint32_t i = lane + 32 * r;
        if (i >= n_steps || bad) continue;
        const uint32_t tq = tq0 + i, c = c0 + tq / tpc, t = tq % tpc;
        if (c >= a.la.n_chunks) {
          bad = true;
          continue;
        }
        const zipmoe_chunk_desc *d = a.la.chunks + c;
        const uint64_t pay_off = __ldg(&d->payload_off);
        if (t >= __ldg(&d->n_tiles) || __ldg(&d->tile_elems) != ZIPMOE_TILE_ELEMS_MAX || (pay_off & 15) ||
            __ldg(&d->table_id) != table_id || pay_off + 4ull * (t + 2) > a.la.payload_bytes ||
            (t + 1 == __ldg(&d->n_tiles) && __ldg(&d->last_tile_elems) != ZIPMOE_TILE_ELEMS_MAX)) {
          bad = true;
          continue;
        }
        const uint32_t *tab = reinterpret_cast<const uint32_t *>(a.la.payload + pay_off);
        const uint32_t o0 = __ldg(tab + t), o1 = __ldg(tab + t + 1);
        // a record is the column table (2 units of 16 bytes) and 1..kMaxRows rows (8 units each)
        if (o1 <= o0 || o1 - o0 < 10 || o1 - o0 > 2 + 8 * kMaxRows || ((o1 - o0 - 2) & 7u) ||
            pay_off + 16ull * o1 > a.la.payload_bytes) {
          bad = true;
          continue;
        }
        rec_at[r] = (uint32_t)(pay_off >> 4) + o0;
        rec_len[r] = o1 - o0;
      }
      const uint64_t sm_first = __ldg(&a.la.chunks[c0].sm_off) + (uint64_t)tq0 * ZIPMOE_TILE_ELEMS_MAX;
      if ((sm_first & 15) || sm_first + (uint64_t)n_steps * ZIPMOE_TILE_ELEMS_MAX > a.la.sm_bytes) bad = true;
      sm_strip = a.la.sm + sm_first;
      if (__any_sync(0xFFFFFFFFu, bad)) {
        report(a.la.status, kStatusBadDescriptor);
        failed = true;
      }
    }
    struct Tile {
      const uint8_t *rec, *sm;
      uint32_t rec_bytes;
      bool staged;
    };
    auto tile = [&](uint32_t i) -> Tile {   // the i-th tile of the piece (all lanes call this)
      const uint32_t at = __shfl_sync(0xFFFFFFFFu, i < 32 ? rec_at[0] : rec_at[1], i & 31);
      const uint32_t len = __shfl_sync(0xFFFFFFFFu, i < 32 ? rec_len[0] : rec_len[1], i & 31);
      Tile t;
      t.rec = a.la.payload + (size_t)at * 16;
      t.rec_bytes = len * 16;
      t.sm = sm_strip + (size_t)i * ZIPMOE_TILE_ELEMS_MAX;
      t.staged = t.rec_bytes <= (uint32_t)kPayBuf;
      return t;
    };
    Tile cur = {a.la.payload, a.la.sm, 0, false};
    uint2 sm[8];   // sign+mantissa bytes of the lane's groups in the 8 rows of a half-tile
    if (!failed) {
      cur = tile(0);
      if (cur.staged && lane == 0) {
        mbar_expect_tx(rec_bar + 8 * stage, cur.rec_bytes + a.la.extra_tx);
        bulk_g2s(my + stage * kPayStage, cur.rec, cur.rec_bytes, rec_bar + 8 * stage);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) sm[k] = ldg_v2_early(cur.sm + k * 256 + lane * 8);
    }

    if (tensor != lut_tensor) {   // (every warp is done with the previous table: a piece ends with CTA barriers)
      fast = build_lut(blockDim.x, a.la.tables[table_id].code_len, lut_raw, lut_scratch, a.la.status) <=
             (uint32_t)kLaneLutBits;
      lut_tensor = tensor;
    }

    if (is_loader) {
      // ---- activations: half a K step (8G token rows x 128 columns) per stage ----
      for (uint32_t hs = 0; hs < 2 * n_steps; ++hs) {
        if (xround > 0 && !mbar_wait_bounded(x_empty + 8 * xst, (xround - 1) & 1)) {
          report(a.la.status, kStatusWaitTimeout);
          *give_up = 1;
          break;
        }
        const uint32_t xstage = x_addr + xst * G * kXGroupBytes;
        for (uint32_t row = lane; row < NCOL; row += 32) {
          const uint16_t *src = a.x;
          uint32_t src_bytes = 0;   // rows past the expert's last slot are filled with zeros
          if (row < Te) {
            const uint32_t xr = a.slot_token ? __ldg(a.slot_token + off + row) : off + row;
            src = a.x + (size_t)xr * a.K + (size_t)(2 * s0 + hs) * 128;
            src_bytes = 16;
          }
          const uint32_t dst = xstage + (row >> 3) * kXGroupBytes + (row & 7) * 16;
#pragma unroll 8
          for (uint32_t k8 = 0; k8 < 16; ++k8)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + k8 * 128),
                         "l"(src + (src_bytes ? k8 * 8 : 0)), "r"(src_bytes)
                         : "memory");
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(x_full + 8 * xst);
        if (++xst == kXStages) {
          xst = 0;
          ++xround;
        }
      }
    } else if (is_mma) {
      // ---- one MMA warp per group; one lane issues, per half-tile: D[64 x N] (+)= A[64 x 256] * X[N x 256]^T ----
      // instruction descriptor: bf16 x bf16 -> fp32, N = NACC, M = 8 * kGroupWarps
      const uint32_t idesc =
          (1u << 4) | (1u << 7) | (1u << 10) | ((NACC >> 3) << 17) | ((uint32_t)(kGroupWarps / 2) << 24);
      const uint32_t q = warp - NW;
      const uint32_t abuf = smem_addr(warp_raw) + 2 * kPayStage + kGroupWarps * q * kFfnWarpBytes;
      const uint64_t a_desc0 = smem_desc(abuf, kBLbo, kFfnWarpBytes);
      bool alive = true;
      for (uint32_t s = 0; s < n_steps && alive; ++s) {
        // the step's two half steps of activations: ring stages xst and the one after it
        const uint32_t st0 = xst, rd0 = xround;
        const uint32_t st1 = st0 + 1 == kXStages ? 0 : st0 + 1, rd1 = st0 + 1 == kXStages ? rd0 + 1 : rd0;
        xst = st1 + 1 == kXStages ? 0 : st1 + 1;
        xround = st1 + 1 == kXStages ? rd1 + 1 : rd1;
        const uint64_t b_desc0 = smem_desc(x_addr + st0 * G * kXGroupBytes, 128, kXGroupBytes);
        const uint64_t b_desc1 = smem_desc(x_addr + st1 * G * kXGroupBytes, 128, kXGroupBytes);
        if (!mbar_wait_bounded(x_full + 8 * st0, rd0 & 1) || !mbar_wait_bounded(x_full + 8 * st1, rd1 & 1)) alive = false;
        for (uint32_t half = 0; half < 2 && alive; ++half, ++hn) {
          if (!mbar_wait_bounded(quad_full + 8 * q, hn & 1)) {
            alive = false;
            break;
          }
          if (lane == 0) {
            tc_fence_after();
            const uint32_t d_tmem = tmem + (2 * q + half) * NACC;
            // the K slice j of an operand starts 2 cores further: the start-address field counts 16-byte units
#pragma unroll
            for (uint32_t j = 0; j < 16; ++j)
              mma_bf16(d_tmem, a_desc0 + j * (2 * kBLbo / 16), (j < 8 ? b_desc0 : b_desc1) + (j & 7) * (256 / 16), idesc,
                       (s > 0 || j > 0) ? 1u : 0u);
            mma_commit(quad_done + 8 * q);
            if (half == 1) {   // this group is done with the step's two X stages
              mma_commit(x_empty + 8 * st0);
              mma_commit(x_empty + 8 * st1);
            }
          }
          __syncwarp();
        }
      }
      if (!alive) {
        report(a.la.status, kStatusWaitTimeout);
        *give_up = 1;
      }
    } else if (is_decode) {
      // ---- one strip of 16 rows: decode tile after tile along K, hand half-tiles to the group's A operand ----
      const uint32_t buf = my + 2 * kPayStage;
      const uint32_t q = warp / kGroupWarps;
      // hand-over of one half in two moves: before the first store, wait until the MMAs of the previous half have
      // read the buffer; after the last store, make the stores visible to the tensor core and tell the MMA warp
      auto buffer_free = [&]() -> bool {
        if (hn == 0) return true;
        return mbar_wait_bounded(quad_done + 8 * q, (hn - 1) & 1, (failed || *give_up) ? kFfnShortTries : (1u << 20));
      };
      auto publish = [&]() {
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(quad_full + 8 * q);
        ++hn;
      };
      for (uint32_t s = 0; s < n_steps; ++s) {
        Tile nxt = cur;
        const bool have_next = !failed && s + 1 < n_steps;
        if (have_next) {
          nxt = tile(s + 1);
          if (nxt.staged && lane == 0) {
            mbar_expect_tx(rec_bar + 8 * (stage ^ 1), nxt.rec_bytes + a.la.extra_tx);
            bulk_g2s(my + (stage ^ 1) * kPayStage, nxt.rec, nxt.rec_bytes, rec_bar + 8 * (stage ^ 1));
          }
        }
        bool step_done = false;
        if (!failed) {
          bool good = true;
          if (cur.staged) {
            good = mbar_wait_bounded(rec_bar + 8 * stage, (rec_phase >> stage) & 1, a.la.wait_tries);
            rec_phase ^= 1u << stage;
            if (!good) {
              report(a.la.status, kStatusWaitTimeout);
              *give_up = 1;
            }
          }
          // both halves of the tile, for every combination of record location and table kind
          auto run = [&](auto staged_c, auto fast_c) -> bool {
            LaneDecoder<decltype(staged_c)::value, decltype(fast_c)::value> dec;
            dec.init(my + stage * kPayStage, cur.rec, cur.rec_bytes, lut, lane);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              // Sign+mantissa bytes: sm[k] holds row k of the half being decoded; as soon as a row has been
              // used its register is refilled with the same row of the half after this one (the tile's second
              // half, or the first half of the strip's next tile), a whole half ahead of its use.
              const uint8_t *ahead = half == 0 ? cur.sm + 8 * 256 + lane * 8 : nxt.sm + lane * 8;
              const bool more = half == 0 || have_next;
              // and the half after that one is asked into the second-level cache (2 KB = 16 lines, one per lane)
              if (have_next && lane < 16)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(nxt.sm + (half == 0 ? 0 : 8 * 256) + lane * 128));
              // the first four rows (two from each of the lane's sub-streams) are decoded into registers while
              // the previous half's MMAs may still run
              uint4 v[4];
#pragma unroll
              for (int k = 0; k < 4; k += 2) {
                dec.group2(sm[k], sm[k + 1], v[k], v[k + 1]);
                if (more) {
                  sm[k] = ldg_v2_early(ahead + k * 256);
                  sm[k + 1] = ldg_v2_early(ahead + (k + 1) * 256);
                }
              }
              if (!buffer_free()) {
                report(a.la.status, kStatusWaitTimeout);
                *give_up = 1;
                publish();
                if (half == 0) publish();   // keep the count of halves
                return false;
              }
#pragma unroll
              for (int k = 0; k < 4; ++k) sts_v4(buf + lane * kBLbo + k * 16, v[k]);
#pragma unroll
              for (int k = 4; k < 8; k += 2) {
                uint4 o0, o1;
                dec.group2(sm[k], sm[k + 1], o0, o1);
                if (more) {
                  sm[k] = ldg_v2_early(ahead + k * 256);
                  sm[k + 1] = ldg_v2_early(ahead + (k + 1) * 256);
                }
                sts_v4(buf + lane * kBLbo + k * 16, o0);
                sts_v4(buf + lane * kBLbo + (k + 1) * 16, o1);
              }
              publish();
            }
            return true;
          };
          if (good) {
            if (cur.staged) good = fast ? run(std::true_type{}, std::true_type{}) : run(std::true_type{}, std::false_type{});
            else good = fast ? run(std::false_type{}, std::true_type{}) : run(std::false_type{}, std::false_type{});
            step_done = true;   // run() publishes both halves even when it fails
          }
          if (!good) failed = true;
        }
        if (!step_done) {   // nothing to contribute: keep the group's hand-over going with whatever the buffer holds
          buffer_free();
          publish();
          buffer_free();
          publish();
        }
        cur = nxt;
        stage ^= 1;
      }
      // the accumulators are final once the MMAs of the last half are done
      if (hn > 0 && !mbar_wait_bounded(quad_done + 8 * q, (hn - 1) & 1, (failed || *give_up) ? kFfnShortTries : (1u << 20))) {
        report(a.la.status, kStatusWaitTimeout);
        *give_up = 1;
      }
    }

    // ---- accumulators -> Y ----
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp < 4 && !*give_up) {
      // With M = 64, D row 16j + i sits in tensor-memory lane 32j + i (i < 16): warp j reads rows 16j..16j+15,
      // the halves of the group's warps 2j and 2j + 1.
      // With M = 128, D row r sits in lane r: warp j reads rows 32j..32j+31, the halves of warps 4j..4j+3.
      const uint32_t wg = kGroupWarps == 8 ? 2 * warp + ((lane >> 3) & 1) : 4 * warp + (lane >> 3), r = lane & 7;
      const uint32_t live_lanes = kGroupWarps == 8 ? 16 : 32;   // (rows of warps the group does not have are skipped below)
      float *y = a.y + ((size_t)(mat * a.max_parts + part) * a.S + off) * a.rows;
      for (uint32_t q = 0; q < Q; ++q) {
        const uint32_t st = grp * NW + kGroupWarps * q + wg;
        for (uint32_t half = 0; half < 2; ++half) {
          const uint32_t row = 16 * st + 8 * half + r;
          for (uint32_t c = 0; c < G; ++c) {
            uint32_t v[8];
            const uint32_t taddr = tmem + ((32 * warp) << 16) + (2 * q + half) * NACC + 8 * c;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                         : "r"(taddr)
                         : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (lane < live_lanes && kGroupWarps * q + wg < NW && st < n_strips) {
#pragma unroll
              for (uint32_t n = 0; n < 8; ++n) {
                const uint32_t tokrow = 8 * c + n;
                if (tokrow < Te) y[(size_t)tokrow * a.rows + row] = __uint_as_float(v[n]);
              }
            }
          }
        }
      }
    }
    // the next piece's MMAs overwrite the accumulators: only once they have been read
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*give_up) break;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

// ---- routing: slots grouped by expert ---------------------------------------------------
// slot_of[t*k + j] = slot of the j-th choice of token t (0xFFFFFFFF for an id out of range);
// slots of an expert are consecutive, in token order.  active[0] = number of experts with
// tokens, active[1..] their ids in ascending order; slot_active[slot] = position of the slot's
// expert in that list.
__global__ void route_kernel(const int32_t *topk_ids, uint32_t S, uint32_t k, uint32_t E, uint32_t max_per_expert,
                             uint32_t *expert_offset, uint32_t *active, uint32_t *slot_token, uint32_t *slot_of,
                             uint32_t *slot_active, uint32_t *status) {
  extern __shared__ uint32_t sh[];   // [E] counts, [E] cursors, [E] position in the active list, [S] ids
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // (the first kernel of a call: launched the ordinary way)
  uint32_t *cnt = sh, *cursor = sh + E, *apos = sh + 2 * E;
  int32_t *ids = reinterpret_cast<int32_t *>(sh + 3 * E);
  for (uint32_t i = threadIdx.x; i < 3 * E; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < S; i += blockDim.x) {
    const int32_t ex = topk_ids[i];
    ids[i] = ex;
    if (ex >= 0 && (uint32_t)ex < E) atomicAdd(&cnt[ex], 1u);
    else report(status, kStatusBadDescriptor);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t run = 0, n_active = 0;
    for (uint32_t x = 0; x < E; ++x) {
      expert_offset[x] = run;
      cursor[x] = run;
      if (cnt[x] > max_per_expert) report(status, kStatusBadDescriptor);
      if (cnt[x]) {
        apos[x] = n_active;
        active[1 + n_active++] = x;
      }
      run += cnt[x];
    }
    expert_offset[E] = run;
    active[0] = n_active;
    for (uint32_t i = 0; i < S; ++i) {   // slots of an expert in token order
      const int32_t ex = ids[i];
      uint32_t slot = 0xFFFFFFFFu;
      if (ex >= 0 && (uint32_t)ex < E) {
        slot = cursor[ex]++;
        slot_token[slot] = i / k;
        slot_active[slot] = apos[ex];
      }
      slot_of[i] = slot;
    }
  }
}

// How a matmul launch shared out its steps, for the kernels that add its partial sums.
struct PartsOf {
  const uint32_t *active;       // [0] = experts with tokens
  const uint32_t *slot_active;  // [S]
  uint32_t n_mats, n_groups, steps, min_units, max_parts, grid, rows_per_group;
  // number of partial sums of (slot, matrix, row)
  __device__ __forceinline__ uint32_t parts(uint32_t slot, uint32_t mat, uint32_t row) const {
    const uint64_t U = (uint64_t)__ldg(active) * n_mats * n_groups * steps;
    if (U == 0) return 0;
    const uint32_t P = ffn_ctas_in_use(U, grid, min_units);
    const uint64_t job = ((uint64_t)__ldg(slot_active + slot) * n_mats + mat) * n_groups + row / rows_per_group;
    uint32_t c0, n;
    ffn_job_parts(job, steps, U, P, &c0, &n);
    return n < max_parts ? n : max_parts;
  }
};

// h = bf16(SiLU(g) * u) for the slots in use; g = sum of the partial blocks gu[0][p], u of gu[1][p], each block
// fp32 [S][I].  grid = (ceil(I / blockDim), S)
__global__ void swiglu_kernel(const float *gu, const PartsOf po, const uint32_t *expert_offset, uint32_t E, uint32_t S,
                              uint32_t I, uint16_t *h) {
  // the numbers of partial sums are the same for all rows of a strip group: looked up once for the group of the
  // block's first row, and again by the threads whose row lies in another group
  __shared__ uint32_t s_parts[2];
  const uint32_t slot = blockIdx.y, row0 = blockIdx.x * blockDim.x, row = row0 + threadIdx.x;
  after_previous_kernel();
  if (slot >= __ldg(expert_offset + E)) return;
  if (threadIdx.x < 2) s_parts[threadIdx.x] = po.parts(slot, threadIdx.x, row0);
  __syncthreads();
  if (row >= I) return;
  const bool same = row / po.rows_per_group == row0 / po.rows_per_group;
  const uint32_t pg = same ? s_parts[0] : po.parts(slot, 0, row), pu = same ? s_parts[1] : po.parts(slot, 1, row);
  const size_t at = (size_t)slot * I + row, block = (size_t)S * I;
  float gv = 0.f, uv = 0.f;
  for (uint32_t p = 0; p < pg; ++p) gv += gu[p * block + at];
  for (uint32_t p = 0; p < pu; ++p) uv += gu[(po.max_parts + p) * block + at];
  const float hv = gv / (1.0f + __expf(-gv)) * uv;
  h[at] = __bfloat16_as_ushort(__float2bfloat16_rn(hv));
}

// out[t] = bf16( sum_j w[t,j] * sum_p y[p][slot_of[t,j]] )
__global__ void combine_kernel(const float *y, const PartsOf po, const uint32_t *slot_of, const float *topk_weights,
                               uint32_t T, uint32_t k, uint32_t S, uint32_t H, uint16_t *out) {
  // grid = (ceil(H / blockDim), T); the numbers of partial sums of the token's k slots, for the strip group of the
  // block's first column, are looked up once per block
  __shared__ uint32_t s_parts[8];
  const uint32_t t = blockIdx.y, c0 = blockIdx.x * blockDim.x, c = c0 + threadIdx.x;
  after_previous_kernel();
  if (threadIdx.x < k && threadIdx.x < 8) {
    const uint32_t slot = slot_of[t * k + threadIdx.x];
    s_parts[threadIdx.x] = slot == 0xFFFFFFFFu ? 0u : po.parts(slot, 0, c0);
  }
  __syncthreads();
  if (c >= H) return;
  const bool same = c / po.rows_per_group == c0 / po.rows_per_group;
  float acc = 0.f;
  for (uint32_t j = 0; j < k; ++j) {
    const uint32_t slot = slot_of[t * k + j];
    if (slot == 0xFFFFFFFFu) continue;
    float v = 0.f;
    const uint32_t n = (same && j < 8) ? s_parts[j] : po.parts(slot, 0, c);
    for (uint32_t p = 0; p < n; ++p) v += y[((size_t)p * S + slot) * H + c];
    acc += (topk_weights ? topk_weights[t * k + j] : 1.0f) * v;
  }
  out[(size_t)t * H + c] = __bfloat16_as_ushort(__float2bfloat16_rn(acc));
}

}  // namespace zipmoe_dev

namespace {

struct FfnPlan {
  uint32_t S, groups, n_warps, smem, grid;
  uint32_t groups_gu, groups_dn;     // strip groups per matrix
  uint32_t min_gu, min_dn;           // smallest share of a CTA, in K steps
  uint32_t parts_gu, parts_dn;       // bound on the partial sums of a job
  uint64_t off_offsets, off_active, off_slot_token, off_slot_of, off_slot_active, off_gu, off_h, off_y, total;
};

// Smallest share of a CTA in K steps, for a launch whose jobs have `steps` steps each and that has at least
// `units_min` steps in all (one expert with tokens): as large as keeps `grid` CTAs busy even then, but never so
// small that a job is cut into more than nine partial sums.
uint32_t pick_min_units(uint64_t units_min, uint32_t steps, uint32_t grid) {
  uint64_t m = units_min / grid;
  if (m > steps) m = steps;
  const uint32_t floor_ = (steps + 7) / 8;
  return m < floor_ ? floor_ : (uint32_t)m;
}

int g_sm_count[64];

zipmoe_status make_plan(uint32_t T, uint32_t k, const zipmoe_compressed_experts *ex, uint32_t grid, FfnPlan *p) {
  if (!ex || T == 0 || k == 0 || T > 64 || k > 8 || ex->n_experts == 0 || ex->n_experts > 256) return ZIPMOE_ERR_UNSUPPORTED;
  if (ex->hidden == 0 || ex->inter == 0 || ex->hidden % 256 || ex->inter % 256) return ZIPMOE_ERR_UNSUPPORTED;
  if (ex->hidden > 64 * 256 || ex->inter > 64 * 256) return ZIPMOE_ERR_UNSUPPORTED;   // a strip's tiles are looked up by 64
                                                                                      // lanes; step counts stay in 32 bits
  p->S = T * k;
  p->groups = (T + 7) / 8;
  p->grid = grid;
  // as many decode warps as fit beside the activation ring and the lookup table
  uint32_t nw = zipmoe_dev::kFfnMaxWarps;
  while (nw > (uint32_t)zipmoe_dev::kGroupWarps && zipmoe_dev::ffn_smem_bytes(nw, p->groups) > 227u * 1024u)
    nw -= nw % zipmoe_dev::kGroupWarps ? nw % zipmoe_dev::kGroupWarps : zipmoe_dev::kGroupWarps;   // first the incomplete group
  if (zipmoe_dev::ffn_smem_bytes(nw, p->groups) > 227u * 1024u) return ZIPMOE_ERR_UNSUPPORTED;
  p->n_warps = nw;
  p->smem = zipmoe_dev::ffn_smem_bytes(nw, p->groups);
  const uint32_t steps_gu = ex->hidden / 256, steps_dn = ex->inter / 256;
  p->groups_gu = (ex->inter / 16 + nw - 1) / nw;
  p->groups_dn = (ex->hidden / 16 + nw - 1) / nw;
  p->min_gu = pick_min_units(2ull * p->groups_gu * steps_gu, steps_gu, grid);
  p->min_dn = pick_min_units(1ull * p->groups_dn * steps_dn, steps_dn, grid);
  p->parts_gu = (steps_gu + p->min_gu - 1) / p->min_gu + 1;
  p->parts_dn = (steps_dn + p->min_dn - 1) / p->min_dn + 1;
  auto up = [](uint64_t v) { return (v + 255) / 256 * 256; };
  uint64_t at = 0;
  p->off_offsets = at; at = up(at + 4ull * (ex->n_experts + 1));
  p->off_active = at; at = up(at + 4ull * (ex->n_experts + 1));
  p->off_slot_token = at; at = up(at + 4ull * p->S);
  p->off_slot_of = at; at = up(at + 4ull * p->S);
  p->off_slot_active = at; at = up(at + 4ull * p->S);
  p->off_gu = at; at = up(at + 2ull * p->parts_gu * p->S * ex->inter * 4);
  p->off_h = at; at = up(at + (uint64_t)p->S * ex->inter * 2);
  p->off_y = at; at = up(at + (uint64_t)p->parts_dn * p->S * ex->hidden * 4);
  p->total = at;
  return ZIPMOE_OK;
}

// The workspace is sized for a grid of this many CTAs when no device is there to ask (a host-only size query);
// with a device, its number of SMs is used.  Fewer CTAs never need more partial sums.
constexpr uint32_t kPlanGridDefault = 148;

uint32_t plan_grid() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
    if (g_sm_count[dev] > 0) return (uint32_t)g_sm_count[dev];
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
      g_sm_count[dev] = sms;
      return (uint32_t)sms;
    }
  }
  (void)cudaGetLastError();   // no device: not an error for a size query
  return kPlanGridDefault;
}

bool g_ffn_ready[64];

}  // namespace

extern "C" zipmoe_status zipmoe_ffn_workspace_bytes(uint32_t T, uint32_t k, const zipmoe_compressed_experts *experts,
                                                    uint64_t *workspace_bytes) {
  if (!workspace_bytes) return ZIPMOE_ERR_INVALID_ARG;
  FfnPlan p;
  zipmoe_status rc = make_plan(T, k, experts, plan_grid(), &p);
  if (rc != ZIPMOE_OK) return rc;
  *workspace_bytes = p.total;
  return ZIPMOE_OK;
}

extern "C" zipmoe_status zipmoe_decode_expert_ffn(const uint16_t *tokens, uint32_t T, const int32_t *topk_ids,
                                                  const float *topk_weights, uint32_t k,
                                                  const zipmoe_compressed_experts *ex, uint16_t *out, void *workspace,
                                                  uint64_t workspace_bytes, uint32_t *status_word,
                                                  zipmoe_stream stream_) {
  using namespace zipmoe_dev;
  zipmoe_host::TraceRange trace("zipmoe_decode_expert_ffn");
  FfnPlan p;
  zipmoe_status rc = make_plan(T, k, ex, plan_grid(), &p);
  if (rc != ZIPMOE_OK) return rc;
  if (!tokens || !topk_ids || !out || !workspace || !ex->chunks || !ex->tensor_first_chunk || !ex->tables ||
      !ex->payload || !ex->sm || ex->n_chunks == 0 || ex->n_tables == 0)
    return ZIPMOE_ERR_INVALID_ARG;
  if (workspace_bytes < p.total) return ZIPMOE_ERR_BUFFER_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(tokens) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(workspace) |
       reinterpret_cast<uintptr_t>(ex->payload) | reinterpret_cast<uintptr_t>(ex->sm) |
       reinterpret_cast<uintptr_t>(ex->chunks)) & 15)
    return ZIPMOE_ERR_INVALID_ARG;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ZIPMOE_ERR_CUDA;
  if (!g_ffn_ready[dev]) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ZIPMOE_ERR_CUDA;
    if (major != 10) return ZIPMOE_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(ffn_matmul_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return ZIPMOE_ERR_CUDA;
    g_ffn_ready[dev] = true;
  }
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
  uint8_t *ws = static_cast<uint8_t *>(workspace);
  uint32_t *expert_offset = reinterpret_cast<uint32_t *>(ws + p.off_offsets);
  uint32_t *active = reinterpret_cast<uint32_t *>(ws + p.off_active);
  uint32_t *slot_token = reinterpret_cast<uint32_t *>(ws + p.off_slot_token);
  uint32_t *slot_of = reinterpret_cast<uint32_t *>(ws + p.off_slot_of);
  uint32_t *slot_active = reinterpret_cast<uint32_t *>(ws + p.off_slot_active);
  float *gu = reinterpret_cast<float *>(ws + p.off_gu);
  uint16_t *h = reinterpret_cast<uint16_t *>(ws + p.off_h);
  float *y = reinterpret_cast<float *>(ws + p.off_y);
  const uint32_t E = ex->n_experts, H = ex->hidden, I = ex->inter, S = p.S;

  route_kernel<<<1, 256, (3 * E + S) * sizeof(uint32_t), stream>>>(topk_ids, S, k, E, 8 * p.groups, expert_offset, active,
                                                                   slot_token, slot_of, slot_active, status_word);

  FfnArgs a;
  a.la.chunks = ex->chunks;
  a.la.tables = ex->tables;
  a.la.payload = ex->payload;
  a.la.sm = ex->sm;
  a.la.out = nullptr;
  a.la.status = status_word;
  a.la.payload_bytes = ex->payload_bytes;
  a.la.sm_bytes = ex->sm_bytes;
  a.la.out_elems = ~0ull;
  a.la.n_chunks = ex->n_chunks;
  a.la.n_tiles = 0;
  a.la.n_tables = ex->n_tables;
  a.la.tiles_per_cta = 0;
  a.la.work_counter = nullptr;
  a.la.work_tag = 0;
  zipmoe_host::wait_fault_setting(&a.la.extra_tx, &a.la.wait_tries);
  a.tensor_first_chunk = ex->tensor_first_chunk;
  a.expert_offset = expert_offset;
  a.active = active;
  a.n_warps = p.n_warps;
  a.groups = p.groups;
  a.S = S;
  a.smem_bytes = p.smem;
  const uint32_t threads = (p.n_warps + (p.n_warps + zipmoe_dev::kGroupWarps - 1) / zipmoe_dev::kGroupWarps + 1) * 32;
  PartsOf po;
  po.active = active;
  po.slot_active = slot_active;
  po.grid = p.grid;
  po.rows_per_group = 16 * p.n_warps;

  // gate and up: partial sums of W_{1,3} X over the pieces of each job
  a.slot_token = slot_token;
  a.x = tokens;
  a.y = gu;
  a.rows = I;
  a.K = H;
  a.tensor_base = 0;
  a.n_mats = 2;
  a.n_groups = p.groups_gu;
  a.min_units = p.min_gu;
  a.max_parts = p.parts_gu;
  // every kernel after the first may start while its predecessor drains (it waits for it before it reads anything)
  cudaLaunchAttribute overlap;
  overlap.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  overlap.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = stream;
  cfg.attrs = &overlap;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3(p.grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = p.smem;
  if (cudaLaunchKernelEx(&cfg, ffn_matmul_kernel, a) != cudaSuccess) return ZIPMOE_ERR_CUDA;

  po.n_mats = 2;
  po.n_groups = p.groups_gu;
  po.steps = H / 256;
  po.min_units = p.min_gu;
  po.max_parts = p.parts_gu;
  cudaLaunchConfig_t small = cfg;
  small.gridDim = dim3((I + 255) / 256, S);
  small.blockDim = dim3(256);
  small.dynamicSmemBytes = 0;
  if (cudaLaunchKernelEx(&small, swiglu_kernel, (const float *)gu, po, (const uint32_t *)expert_offset, E, S, I, h) !=
      cudaSuccess)
    return ZIPMOE_ERR_CUDA;

  // down: partial sums of W_2 H
  a.slot_token = nullptr;
  a.x = h;
  a.y = y;
  a.rows = H;
  a.K = I;
  a.tensor_base = 2;
  a.n_mats = 1;
  a.n_groups = p.groups_dn;
  a.min_units = p.min_dn;
  a.max_parts = p.parts_dn;
  if (cudaLaunchKernelEx(&cfg, ffn_matmul_kernel, a) != cudaSuccess) return ZIPMOE_ERR_CUDA;

  po.n_mats = 1;
  po.n_groups = p.groups_dn;
  po.steps = I / 256;
  po.min_units = p.min_dn;
  po.max_parts = p.parts_dn;
  small.gridDim = dim3((H + 255) / 256, T);
  if (cudaLaunchKernelEx(&small, combine_kernel, (const float *)y, po, (const uint32_t *)slot_of, topk_weights, T, k, S,
                         H, out) != cudaSuccess)
    return ZIPMOE_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? ZIPMOE_OK : ZIPMOE_ERR_CUDA;
}

// ---- the same call for callers that cannot allocate device memory ------------------------------
namespace {
// Scratch for zipmoe_decode_expert_ffn_noalloc.  It is part of the library image: every GPU that loads the
// library sets these bytes aside until the process exits, whether or not the entry point is ever called.
constexpr uint64_t kNoAllocScratchBytes = ZIPMOE_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];
// Device address of g_noalloc_scratch per device.  In host code the symbol itself is only a stand-in, not an
// address the GPU can use, so the address is asked for once per device and kept here.
void *g_noalloc_ptr[64];
}  // namespace

extern "C" zipmoe_status zipmoe_decode_expert_ffn_noalloc(const uint16_t *tokens, uint32_t T, const int32_t *topk_ids,
                                                          const float *topk_weights, uint32_t k,
                                                          const zipmoe_compressed_experts *experts, uint16_t *out,
                                                          uint32_t *status_word, zipmoe_stream stream) {
  uint64_t need = 0;
  zipmoe_status rc = zipmoe_ffn_workspace_bytes(T, k, experts, &need);
  if (rc != ZIPMOE_OK) return rc;
  if (need > kNoAllocScratchBytes) return ZIPMOE_ERR_BUFFER_TOO_SMALL;   // the call does not fit the built-in scratch
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ZIPMOE_ERR_CUDA;
  if (!g_noalloc_ptr[dev]) {   // first call on this device, with this device current
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return ZIPMOE_ERR_CUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  return zipmoe_decode_expert_ffn(tokens, T, topk_ids, topk_weights, k, experts, out, g_noalloc_ptr[dev],
                                  kNoAllocScratchBytes, status_word, stream);
}
