/*
 * zipmoe.h -- C ABI of the B200-native ZipMoE decode library.
 *
 * The library implements the compute-centric step of ZipMoE: expert weights
 * are kept losslessly compressed and the required bf16 tensors are computed
 * on demand instead of being transferred (paper Section 1, last paragraph).
 * Offline, each bf16 tensor is split into an exponent stream and a
 * sign+mantissa byte stream; the exponent stream is cut into K shards that
 * are entropy-coded independently ("E-chunks") while the sign+mantissa bytes
 * are stored raw ("SM-chunks") (Section 3.1, "Offline Initialization").
 * Online, E-chunks are decompressed and re-assembled with the SM-chunks into
 * exact bf16 (Section 3.1, "Real-time Inference"; Section 3.3,
 * "Memory-Coalesced Tensor Recovery Kernel").  The paper runs the
 * decompression on CPU threads with LZ4/ZSTD and leaves the compressor slot
 * open (Section 6, "Other Compressors"); here the slot holds an order-0
 * canonical Huffman code over exponent bytes and both steps run in one CUDA
 * kernel for sm_100a.
 *
 * Conventions for every entry point
 *   - Plain C, no exceptions, no aborts: the return value is a zipmoe_status.
 *   - The library never allocates or frees device memory and never
 *     synchronises a stream, except where an entry point says otherwise.
 *     Device buffers and streams belong to the caller.
 *   - "host" / "device" in an argument's comment says where the pointer must
 *     point.  Sizes are in the unit named in the comment.
 *   - The container ("blob") produced by zipmoe_encode is self-describing,
 *     little-endian, and documented in the repository's design notes; its
 *     payload and sign+mantissa sections are copied verbatim to the device.
 */
#ifndef ZIPMOE_H
#define ZIPMOE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int zipmoe_status;
#define ZIPMOE_OK 0
#define ZIPMOE_ERR_INVALID_ARG (-1)      /* null pointer, bad size, bad alignment, bad option  */
#define ZIPMOE_ERR_BAD_FORMAT (-2)       /* blob fails validation                               */
#define ZIPMOE_ERR_BUFFER_TOO_SMALL (-3) /* caller's output buffer can not hold the result      */
#define ZIPMOE_ERR_CUDA (-4)             /* a CUDA runtime call failed (launch, attribute, ...) */
#define ZIPMOE_ERR_DECODE_CORRUPT (-5)   /* reported through the device status word only        */
#define ZIPMOE_ERR_UNSUPPORTED (-6)      /* shape or option outside what the kernels handle     */

#define ZIPMOE_LAYOUT_LINEAR 0u  /* a tile is tile_elems consecutive elements of the flat tensor  */
#define ZIPMOE_LAYOUT_BLOCKED 1u /* a tile is a 16 x 256 block of the rows x cols matrix         */
#define ZIPMOE_MAX_CODE_LEN 12u
#define ZIPMOE_TILE_ELEMS_MAX 4096u
/* bytes the caller must keep readable after the end of the device payload and
 * sign+mantissa buffers (the kernels read whole 16-byte units and look a few
 * words past the last code) */
#define ZIPMOE_DEVICE_PAD_BYTES 256u

typedef struct CUstream_st *zipmoe_stream; /* a cudaStream_t; NULL is the default stream */

/* ---- encoding (host) ---------------------------------------------------- */

typedef struct {
  uint32_t chunk_elems;  /* elements per independently decodable chunk (the paper's shard): a multiple
                            of 256, and a multiple of 4096 when larger than 4096.  0 selects 65536.    */
  uint32_t max_code_len; /* longest Huffman code, 8..12.  0 selects 8: the decoder's fastest path (codes of
                            at most 8 bits resolve in a bank-conflict-free table, four per 32-bit window);
                            12 gives ~0.06-0.1 bit/element smaller output and decodes ~20 % slower.      */
  uint32_t layout;       /* ZIPMOE_LAYOUT_LINEAR or ZIPMOE_LAYOUT_BLOCKED (needs rows % 16 == 0,
                            cols % 256 == 0, chunk_elems >= 4096)                                       */
  uint32_t n_threads;    /* host threads for the encoder (chunks are independent). 0 selects 1.         */
} zipmoe_encode_opts;

typedef struct {
  uint64_t n_elems;       /* rows * cols                                                         */
  uint32_t rows, cols;
  uint32_t layout, chunk_elems, tile_elems, max_code_len;
  uint32_t n_chunks;      /* K = ceil(n_tiles / (chunk_elems / tile_elems))                      */
  uint32_t n_tiles;
  uint64_t table_off;     /* byte offset in the blob of the 256 code lengths                     */
  uint64_t chunk_off_off; /* byte offset of the n_chunks + 1 per-chunk bit offsets (u64)         */
  uint64_t payload_off;   /* byte offset and size of the E-chunk section (16-byte aligned)       */
  uint64_t payload_bytes;
  uint64_t sm_off;        /* byte offset and size of the SM-chunk section (16-byte aligned)      */
  uint64_t sm_bytes;
  uint64_t total_bytes;
} zipmoe_blob_info;

/* Upper bound on the blob size for a rows x cols tensor.  (Section 3.1: the
 * serialised form of one tensor: E-chunks, SM-chunks and metadata.)
 * host in: opts (NULL = defaults); host out: *blob_bytes_max. */
zipmoe_status zipmoe_encode_bound(uint64_t rows, uint64_t cols, const zipmoe_encode_opts *opts,
                                  uint64_t *blob_bytes_max);

/* Offline initialisation of one tensor (Section 3.1, "Offline Initialization"):
 * bit-field decomposition of each bf16 into exponent byte and sign+mantissa
 * byte, one canonical Huffman code per tensor over the exponent bytes, the
 * exponent stream cut into chunks of chunk_elems elements with per-chunk bit
 * offsets, sign+mantissa bytes stored raw.  Synchronous, host only, no CUDA.
 * host in : bf16 (rows*cols bit patterns, row-major), opts (NULL = defaults)
 * host out: blob[0 .. *blob_bytes), written only if blob_cap is large enough
 *           (ZIPMOE_ERR_BUFFER_TOO_SMALL otherwise; *blob_bytes is then the bound). */
zipmoe_status zipmoe_encode(const uint16_t *bf16, uint64_t rows, uint64_t cols, const zipmoe_encode_opts *opts,
                            void *blob, uint64_t blob_cap, uint64_t *blob_bytes);

/* Parse the header of a blob.  host in: blob; host out: *info. */
zipmoe_status zipmoe_blob_info_get(const void *blob, uint64_t blob_bytes, zipmoe_blob_info *info);

/* Full structural check of a blob on the host: header, complete prefix code
 * (Kraft sum exactly 1, lengths <= max_code_len), monotone 128-bit-aligned
 * chunk offsets, tile tables, record sizes and the records' column tables (a permutation each).
 * A blob that passes can be handed to the device decoder safely. */
zipmoe_status zipmoe_blob_validate(const void *blob, uint64_t blob_bytes);

/* ---- decode (device) ---------------------------------------------------- */

/* One descriptor per chunk of a launch.  A "run" is the consecutive
 * descriptors of one tensor (same table, consecutive chunks). */
typedef struct {
  uint64_t payload_off;     /* bytes from `payload` to this chunk's E-chunk (multiple of 16): its
                               per-chunk bit offset / 8 plus where the blob's payload section sits */
  uint64_t sm_off;          /* bytes from `sm` to the SM bytes of this chunk's first tile (mult. of 16) */
  uint64_t out_off;         /* elements from `out_bf16` to the tensor's element 0 (multiple of 8)  */
  uint32_t row_pitch;       /* elements between the 256-element rows of a tile: cols (blocked), 256 (linear) */
  uint32_t tiles_per_rowblk;/* cols / 256 (blocked), 1 (linear)                                    */
  uint32_t tile0;           /* index within the tensor of this chunk's first tile                 */
  uint32_t n_tiles;         /* tiles in this chunk                                                 */
  uint32_t tile_elems;      /* 256 * I, I = 1..16                                                  */
  uint32_t last_tile_elems; /* existing elements in this chunk's last tile (1..tile_elems)         */
  uint32_t table_id;        /* index into `tables`                                                 */
  uint32_t tile_prefix;     /* tiles in all earlier descriptors of the launch                      */
  uint32_t run_first_chunk; /* index in `chunks` of the run's first descriptor                     */
  uint32_t run_first_tile;  /* tile_prefix of that descriptor                                      */
  uint32_t run_end_tile;    /* tile_prefix + n_tiles of the run's last descriptor                  */
  uint32_t tiles_per_chunk; /* tiles in every chunk of the run but possibly the last               */
  uint32_t max_record_bytes;/* largest tile record of the run, in bytes (0 = unknown); a hint that lets the
                               kernel skip its wide-record handling for tensors that never need it  */
  uint32_t reserved;        /* zero; pads the descriptor to 80 bytes (five 16-byte loads)          */
} zipmoe_chunk_desc;

typedef struct {
  uint8_t code_len[256];    /* canonical Huffman code lengths, 0 = unused symbol */
} zipmoe_table;

/* Fill the descriptors and the table for one blob whose payload section will
 * sit at payload_base bytes into the device payload buffer, whose SM section
 * at sm_base bytes into the device SM buffer, and whose tensor at out_base
 * elements into the output (all three multiples of 16 bytes).  chunk_base and
 * tile_base are the number of descriptors and tiles already planned for this
 * launch.  Host only.
 * host in : blob;  host out: descs[0 .. info.n_chunks), *table. */
zipmoe_status zipmoe_blob_plan(const void *blob, uint64_t blob_bytes, uint64_t payload_base, uint64_t sm_base,
                               uint64_t out_base, uint32_t table_id, uint32_t chunk_base, uint32_t tile_base,
                               zipmoe_chunk_desc *descs, zipmoe_table *table);

/* One decode launch over several blobs: where every blob's E-chunk section, SM section and tensor sit in the
 * launch's three buffers, and what zipmoe_decode / zipmoe_decode_expert_ffn need to know about the whole. */
typedef struct {
  uint64_t payload_bytes;    /* E-chunk sections of all blobs, back to back                                   */
  uint64_t sm_bytes;         /* their SM sections, each rounded up to 16 bytes                                */
  uint64_t out_elems;        /* their tensors, each rounded up to 8 elements                                  */
  uint32_t n_chunks, n_tiles, n_tables;
  uint32_t max_record_bytes; /* largest tile record of the launch: zipmoe_decode's argument of that name      */
  uint32_t max_code_len;     /* longest code of any table of the launch                                       */
  uint32_t flags;            /* ZIPMOE_DECODE_SHORT_CODES if the launch may promise it, else 0                */
} zipmoe_launch_info;

/* Sizes only (the first call of the two-call pattern).  host in: blobs[n_blobs], blob_bytes[n_blobs];
 * host out: *info with the three sizes and the counts (max_record_bytes, max_code_len and flags are zero). */
zipmoe_status zipmoe_launch_plan_size(const void *const *blobs, const uint64_t *blob_bytes, uint32_t n_blobs,
                                      zipmoe_launch_info *info);

/* Lays the blobs out for one launch (Section 3.1: what "Real-time Inference" finds in memory -- E-chunks,
 * SM-chunks and metadata -- arranged for the decoder): copies every blob's E-chunk section into `payload` and
 * its SM section into `sm`, one after the other, zero-fills the ZIPMOE_DEVICE_PAD_BYTES after each, and writes
 * the chunk descriptors (zipmoe_blob_plan with table_id = index of the blob) and tables.  The caller copies the
 * four arrays to the device as they are.
 * host in : blobs, blob_bytes
 * host out: payload[info.payload_bytes + PAD], sm[info.sm_bytes + PAD], descs[info.n_chunks], tables[n_blobs],
 *           tensor_first_chunk[n_blobs] (may be NULL: first descriptor of each blob, as
 *           zipmoe_compressed_experts wants it), out_base[n_blobs] (may be NULL: element offset of each tensor
 *           in the output buffer of info.out_elems elements), *info (complete). */
zipmoe_status zipmoe_launch_plan(const void *const *blobs, const uint64_t *blob_bytes, uint32_t n_blobs, uint8_t *payload,
                                 uint8_t *sm, zipmoe_chunk_desc *descs, zipmoe_table *tables, uint32_t *tensor_first_chunk,
                                 uint64_t *out_base, zipmoe_launch_info *info);

/* Real-time reconstruction (Section 3.1 "Real-time Inference", steps 6-7;
 * Section 3.3 "Memory-Coalesced Tensor Recovery Kernel"): decode every
 * chunk's exponent bytes from its E-chunk and merge them with the SM bytes
 * into bf16, written once, in place, to out_bf16.  Chunks are independent and
 * may belong to any number of tensors.  One kernel launch on `stream`;
 * asynchronous; the exponent bytes never reach global memory.
 *
 * device in : chunks[n_chunks] (in launch order, tile_prefix ascending),
 *             tables[n_tables], payload[payload_bytes + PAD], sm[sm_bytes + PAD]
 * device out: out_bf16[out_elems]; status_word (nullable): left untouched on
 *             success, set to a non-zero code when a descriptor, offset or
 *             bit count points outside the given buffers or a wait ran out;
 *             the kernel skips the offending tile and always terminates.
 * n_tiles   : total tiles of the launch (sum of chunks[].n_tiles).
 * max_record_bytes : the largest chunks[].max_record_bytes of the launch, or 0 if unknown.  A host-side hint
 *             only: when no record exceeds ZIPMOE_NARROW_RECORD_BYTES (16 rows: every tensor but
 *             near-incompressible ones) a kernel variant with smaller record stages and one more warp runs, about
 *             3 % faster.  A wrong hint costs speed, never correctness.
 * flags     : 0, or ZIPMOE_DECODE_SHORT_CODES: the caller promises that no table of the launch has a code longer
 *             than 8 bits and that max_record_bytes is a true upper bound of at most ZIPMOE_NARROW_RECORD_BYTES (zipmoe_blob_plan's
 *             descriptors and the blobs' tables say both).  The kernel variant chosen then carries only the common
 *             path and is 2-3 % faster.  A tile that breaks the promise is not decoded: its output is left as it
 *             was and status_word is set (code 5), so a false promise is loud, never silent.
 * Work distribution: launches of few large tensors (n_tiles >= 512 * n_tables) give every CTA an equal range of
 *             tiles; all others hand the tiles out dynamically through an 8-byte counter.  The counters are a
 *             ring of 1024 in the library's own device memory (nothing is allocated); a launch zeroes its
 *             counter on `stream` before the kernel (one cudaMemsetAsync) and its first CTA tags it as the
 *             launch's own.  More than 1024 such launches in flight at once on one device would share counters:
 *             a launch that finds another launch's tag on its counter stops taking tiles and sets status_word
 *             (code 6), so that incomplete output does not go unnoticed.  The same holds for a captured graph
 *             that replays such a launch while a later launch owns its counter.
 * All device pointers 16-byte aligned.  Errors found on the host (null or
 * misaligned pointers, zero table count with non-zero chunks) are returned
 * before anything is launched. */
zipmoe_status zipmoe_decode(const zipmoe_chunk_desc *chunks, uint32_t n_chunks, uint32_t n_tiles,
                            const zipmoe_table *tables, uint32_t n_tables, const uint8_t *payload,
                            uint64_t payload_bytes, const uint8_t *sm, uint64_t sm_bytes, uint16_t *out_bf16,
                            uint64_t out_elems, uint32_t *status_word, zipmoe_stream stream,
                            uint32_t max_record_bytes, uint32_t flags);
#define ZIPMOE_DECODE_SHORT_CODES 1u
#define ZIPMOE_NARROW_RECORD_BYTES 2080u /* a tile record of 16 rows: 32 + 16 * 128 bytes */

/* The recovery step alone (Section 3.3, "Memory-Coalesced Tensor Recovery Kernel"): exponent bytes that
 * are already decompressed and sign+mantissa bytes, both in element order, are merged into bf16:
 *     out[i] = (sm[i] & 0x80) << 8 | exp[i] << 7 | (sm[i] & 0x7F).
 * One launch on `stream`, asynchronous, 2 bytes read and 2 written per element.
 * device in : exp[n_elems], sm[n_elems];  device out: out_bf16[n_elems]; all three 16-byte aligned. */
zipmoe_status zipmoe_recover(const uint8_t *exp, const uint8_t *sm, uint64_t n_elems, uint16_t *out_bf16,
                             zipmoe_stream stream);

/* ---- fused decode + routed expert FFN (device) ----------------------------- */

/* The compressed experts of one MoE layer.  A HOST struct holding DEVICE
 * pointers.  Expert e has three tensors, encoded with ZIPMOE_LAYOUT_BLOCKED:
 * tensor 3e+0 = w1 (gate) [inter, hidden], 3e+1 = w3 (up) [inter, hidden],
 * 3e+2 = w2 (down) [hidden, inter], all [out, in] row-major before encoding.
 * `chunks` holds the descriptors zipmoe_blob_plan wrote for the 3E blobs (their
 * out_off is not used), `tensor_first_chunk[3e+j]` the index of each tensor's
 * first descriptor, `tables` the code lengths its table_id refers to. */
typedef struct {
  uint32_t n_experts, hidden, inter, n_chunks;   /* hidden, inter: multiples of 256                           */
  const zipmoe_chunk_desc *chunks;               /* device [n_chunks]                                          */
  const uint32_t *tensor_first_chunk;            /* device [3 * n_experts]                                     */
  const zipmoe_table *tables;                    /* device [n_tables]                                          */
  uint32_t n_tables, reserved;
  const uint8_t *payload;                        /* device, payload_bytes + ZIPMOE_DEVICE_PAD_BYTES            */
  uint64_t payload_bytes;
  const uint8_t *sm;                             /* device, sm_bytes + ZIPMOE_DEVICE_PAD_BYTES                 */
  uint64_t sm_bytes;
} zipmoe_compressed_experts;

/* Scratch the fused call needs for T tokens with k experts each (routing lists,
 * fp32 gate/up activations, bf16 intermediate, fp32 partial outputs).  Host only. */
zipmoe_status zipmoe_ffn_workspace_bytes(uint32_t T, uint32_t k, const zipmoe_compressed_experts *experts,
                                         uint64_t *workspace_bytes);

/* Expert execution on compressed weights (Section 3.3: the GPU work p_n for the
 * tokens routed to expert n, here without ever materialising the expert): for
 * every token t and choice j with e = topk_ids[t, j]:
 *     g = W1_e x_t,  u = W3_e x_t,  h = bf16(SiLU(g) * u),  y = W2_e h
 *     out[t] = bf16( sum_j topk_weights[t, j] * y )
 * bf16 inputs, fp32 accumulation on the tensor cores (tcgen05, accumulators in
 * tensor memory), weights decoded tile by tile into shared memory.  The paper
 * does not define the expert network; this is the gated FFN of the models it
 * evaluates.  Five kernels on `stream`, asynchronous; the last four are launched
 * with programmatic stream serialization (each is set up while its predecessor
 * drains and waits for it before it reads anything), so work queued on `stream`
 * before and after the call is ordered against it as against one kernel.
 * device in : tokens [T, hidden] bf16 patterns; topk_ids [T, k] (each token's ids
 *             distinct); topk_weights [T, k] fp32 or NULL (= 1.0)
 * device out: out [T, hidden] bf16 patterns; workspace: scratch of at least
 *             zipmoe_ffn_workspace_bytes, 16-byte aligned; status_word as for
 *             zipmoe_decode.
 * Limits: T <= 64, k <= 8, n_experts <= 256 (ZIPMOE_ERR_UNSUPPORTED otherwise). */
zipmoe_status zipmoe_decode_expert_ffn(const uint16_t *tokens, uint32_t T, const int32_t *topk_ids,
                                       const float *topk_weights, uint32_t k,
                                       const zipmoe_compressed_experts *experts, uint16_t *out, void *workspace,
                                       uint64_t workspace_bytes, uint32_t *status_word, zipmoe_stream stream);

/* Size of the scratch built into the library for zipmoe_decode_expert_ffn_noalloc. */
#define ZIPMOE_NOALLOC_SCRATCH_BYTES (8u << 20)

/* The fused expert FFN for callers that have no way to obtain device memory.  (The paper has no
 * counterpart: this entry point exists for the embedding program's sake, not for the method's.)
 *
 * zipmoe_decode_expert_ffn needs a scratch buffer, and somebody has to allocate it.  Some callers
 * cannot: a plug-in inside a serving process whose host framework owns the whole device-memory pool
 * and hands out none of it, or a latency-critical decode loop in which cudaMalloc is off limits because
 * it synchronises the device and may fail late.  This variant takes no workspace argument.  It computes
 * exactly what zipmoe_decode_expert_ffn computes, with the same kernels, using a fixed array of
 * ZIPMOE_NOALLOC_SCRATCH_BYTES (8 MiB) that is part of the library image: every GPU that loads the
 * library keeps those 8 MiB reserved until the process exits.  It calls no allocation or free routine
 * of any kind.
 *
 *   - Calls whose scratch need (zipmoe_ffn_workspace_bytes) exceeds the built-in array are refused
 *     with ZIPMOE_ERR_BUFFER_TOO_SMALL before anything is launched; use zipmoe_decode_expert_ffn with
 *     a buffer of your own for those.
 *   - The first call on each device looks up the device address of the array (the device must be
 *     current).  Make that first call outside any stream capture; later calls do no set-up.
 *   - Every call on a device uses the same array, which keeps the previous call's contents.  Nothing
 *     in it has to be cleared: each call writes every word it later reads.  Two calls that overlap on
 *     the GPU (different streams, no ordering between them) race on the array and give wrong results;
 *     order them, or give all but one a workspace of their own through zipmoe_decode_expert_ffn.
 *
 * Arguments, limits and errors otherwise as for zipmoe_decode_expert_ffn. */
zipmoe_status zipmoe_decode_expert_ffn_noalloc(const uint16_t *tokens, uint32_t T, const int32_t *topk_ids,
                                               const float *topk_weights, uint32_t k,
                                               const zipmoe_compressed_experts *experts, uint16_t *out,
                                               uint32_t *status_word, zipmoe_stream stream);

/* ---- cache-pool planning (host only, no CUDA) ------------------------------
 * The paper's planner sizes four cache pools for experts in different compression states -- F full
 * tensors, C compressed (E-chunks and SM-chunks), S SM-chunks only, E E-chunks only -- from a
 * rank-based activation model (Section 3.4 "Compression-Aware Cache Management", Appendix
 * "Hierarchical Cache Pool Planning": Algorithms 2-4, and the iterative proportional fitting of the
 * appendix on the maximum-entropy property).  The delays c, v, u it takes are measured by the caller,
 * e.g. from zipmoe_decode timings.  Pool order everywhere: 0 = F, 1 = C, 2 = S, 3 = E. */

/* Algorithm 2: distribution of the number of experts selected among n ranks that are selected
 * independently with probabilities q[0..n): phi[h] = P(exactly h), h = 0..n (Poisson binomial).
 * host in: q (each in [0, 1]); host out: phi[n + 1]. */
zipmoe_status zipmoe_plan_hit_distribution(const double *q, uint32_t n, double *phi);

/* Selection probabilities q from marginal inclusion probabilities f (0 < f[i] < 1, sum = k) by the
 * modified iterative proportional fitting of the appendix: weights w start at f and are multiplied
 * by f[i] / f_t[i], f_t[i] = w[i] R(k-1, N \ {i}) / R(k, N) with R the elementary symmetric
 * polynomial, until max |f_t - f| <= tol or max_iters passes; q[i] = w[i] / (1 + w[i]).  Choosing
 * k of the n ranks with probability proportional to the product of their w then includes rank i
 * with probability f[i].
 * host in: f[n], k (1 <= k < n <= 512); host out: q[n], *iters_done (may be NULL).
 * Returns ZIPMOE_ERR_INVALID_ARG if f is not feasible (some f outside (0, 1), or sum != k within 1e-6). */
zipmoe_status zipmoe_plan_selection_probs(const double *f, uint32_t n, uint32_t k, uint32_t max_iters, double tol,
                                          double *q, uint32_t *iters_done);

typedef struct {
  double c;           /* decompression delay of one E-chunk                         */
  double v;           /* read delay of one E-chunk                                  */
  double u;           /* read delay of one SM-chunk (one tensor's sign+mantissa)    */
  uint32_t L;         /* decompression workers                                      */
  uint32_t K;         /* E-chunks (exponent shards) per tensor                      */
  uint32_t n_tensors; /* tensors per expert                                         */
} zipmoe_plan_costs;

/* Algorithm 3: estimated makespan of a sparse layer (without token execution) when k experts are
 * activated and hits[p] of them are found in pool p: max(T_IO, T_decomp) with
 *   n_SM = n_tensors (k - h_F - h_C - h_S),  n_E = n_tensors K (k - h_F - h_C - h_E),
 *   n_D = n_tensors K (k - h_F),  T_IO = n_SM u + n_E v,  T_decomp = (n_E v + n_D c) / L.
 * host in: k, hits[4] (sum <= k), costs; host out: *makespan. */
zipmoe_status zipmoe_plan_makespan(uint32_t k, const uint32_t hits[4], const zipmoe_plan_costs *costs, double *makespan);

/* Expected makespan of a cache partition: pools of capacity[p] experts (0 = pool not used) laid on
 * the popularity ranks in the order F, C, S, E, the remaining ranks being misses; the probability of
 * a hit pattern h given that exactly k experts are selected is
 *   Phi_M(k - sum h) / Phi_N(k) * prod_p Phi_p(h_p)      (Section 3.4),
 * each Phi from Algorithm 2 on the pool's rank interval.
 * host in: q[n] (selection probabilities by rank), k, capacity[4] (sum <= n), costs; host out: *expected. */
zipmoe_status zipmoe_plan_expected_makespan(const double *q, uint32_t n, uint32_t k, const uint32_t capacity[4],
                                            const zipmoe_plan_costs *costs, double *expected);

/* Algorithm 4: grid search over the memory ratios of the pools named in pool_mask (bit p = pool p may
 * be used; the others get ratio 0), step `step` (0 < step <= 1, 1 / step an integer up to 100).  A
 * pool with ratio g holds floor(g * budget / expert_size[p]) experts, `budget` and expert_size[p]
 * (memory of one expert in state p) in the same unit; capacities are cut, in the order F, C, S, E,
 * so that they sum to at most n.  Returns the ratios with the smallest expected makespan (ties: the
 * first one in the enumeration order, ratios of F varying slowest) and that makespan.
 * host in: f[n] inclusion probabilities by rank (as for zipmoe_plan_selection_probs), k, pool_mask,
 * budget, expert_size[4], costs, step; host out: ratios[4], capacity[4], *expected. */
zipmoe_status zipmoe_plan_cache_pools(const double *f, uint32_t n, uint32_t k, uint32_t pool_mask, double budget,
                                      const double expert_size[4], const zipmoe_plan_costs *costs, double step,
                                      double ratios[4], uint32_t capacity[4], double *expected);

/* ---- cache-affinity scheduling (host only, no CUDA) ---------------------------
 * The paper's scheduler (Section 3.3 "Cache-Affinity Scheduler"; appendix, Algorithm "Cache-Affinity
 * Scheduling") as a simulator.  One reconstruction task per tensor of every selected expert; a task's
 * compression state says what has to be read: 0 = M missed (E-chunks and SM-chunk), 1 = C compressed in memory
 * (nothing), 2 = S SM-chunk in memory (E-chunks), 3 = E E-chunks in memory (SM-chunk).  Costs: u = read of one
 * SM-chunk, rho * u / K = read of one of a tensor's K E-chunks, c = its decompression; p[n] = GPU time of the
 * tokens routed to expert n.  One I/O thread, L decompression workers, one GPU stream, all work-conserving:
 * the I/O thread reads, block by block, the E-chunks of the block's tasks and then their SM-chunks; a free
 * worker takes the first decompression in priority order whose E-chunk has arrived; the GPU runs an expert
 * once all its tensors are recovered.  Makespan = completion of the last expert. */
typedef struct {
  uint32_t expert; /* index into p                                   */
  uint32_t state;  /* 0 M, 1 C, 2 S, 3 E                             */
} zipmoe_sched_task;

typedef struct {
  double c, u, rho; /* delays as above; rho = compressed size of the exponent bits relative to their raw size */
  uint32_t K, L;    /* E-chunks per tensor; decompression workers                                             */
} zipmoe_sched_costs;

/* Makespan, and total idle time of the workers directly before their operations (the appendix's "charge"), of
 * the priority order order[0 .. n_tasks) cut into blocks: block_of[i] = block of order[i], non-decreasing.
 * host in: tasks, p[n_experts], costs, order (a permutation), block_of; host out: *makespan, *charge (may be NULL). */
zipmoe_status zipmoe_plan_simulate(const zipmoe_sched_task *tasks, uint32_t n_tasks, const double *p, uint32_t n_experts,
                                   const zipmoe_sched_costs *costs, const uint32_t *order, const uint32_t *block_of,
                                   double *makespan, double *charge);

/* Algorithm "Cache-Affinity Scheduling": tasks that must read an SM-chunk (Type-I) and the others (Type-II) are
 * sorted by non-increasing expert time; every block starts from the first unscheduled Type-I task and takes
 * candidates (Type-II first) at the earliest position that adds no worker idle time -- else after the last task
 * of its kind with at least its expert time -- until the block is compute-dominant: the l-th earliest worker
 * completes at least l * rho * u / K after the block's reads, for l = 1 .. min(L, K) (Eq. "compute_dominate").
 * Type-II tasks that no block took form a last block.
 * host out: order[n_tasks], block_of[n_tasks], *n_blocks and *makespan (either may be NULL). */
zipmoe_status zipmoe_plan_schedule(const zipmoe_sched_task *tasks, uint32_t n_tasks, const double *p, uint32_t n_experts,
                                   const zipmoe_sched_costs *costs, uint32_t *order, uint32_t *block_of,
                                   uint32_t *n_blocks, double *makespan);

/* For the library's own tests (the paper has no counterpart).  Every wait of a kernel on an asynchronous copy is
 * bounded: when it runs out the kernel sets status_word (code 3), skips the work that depended on the copy, and
 * still terminates.  That path cannot be reached with sound inputs, so this switch provokes it without a fault:
 * from now on zipmoe_decode and zipmoe_decode_expert_ffn arm the barrier of every tile-record copy for
 * extra_tx_bytes more than the copy delivers (so that the barrier never completes although the copy does) and give
 * up after `tries` tries.  (0, 0) restores normal operation.  Process-wide; not for concurrent use. */
void zipmoe_test_wait_fault(uint32_t extra_tx_bytes, uint32_t tries);

/* For the library's own tests (the paper has no counterpart).  A launch that hands its tiles out dynamically owns
 * a work counter of the library's ring for its duration; should it ever find the tag of another launch there, it
 * stops, decodes nothing more and sets status_word to code 6.  With more than a thousand such launches in flight
 * that could happen; a test cannot bring it about on purpose.  While this switch is on, zipmoe_decode therefore
 * fills the counter of such a launch with a tag that no launch carries instead of zeroing it.  0 restores normal
 * operation.  Process-wide; not for concurrent use. */
void zipmoe_test_foreign_counter(uint32_t on);

/* Name of a status code (static string). */
const char *zipmoe_status_string(zipmoe_status s);

/* Library version, for the binding's sanity check. */
uint32_t zipmoe_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ZIPMOE_H */
