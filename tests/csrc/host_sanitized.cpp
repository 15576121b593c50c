// The library's host code (encoder, validator, planners, scheduler) compiled with the address and undefined-
// behaviour sanitizers and driven over ragged, tiny, blocked and damaged inputs.  Any out-of-bounds access,
// misaligned store or overflow aborts the program; a clean run prints "ok".
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "zipmoe.h"

static uint32_t lcg(uint32_t &s) { return s = s * 1664525u + 1013904223u; }

#define CHECK(cond)                                        \
  do {                                                     \
    if (!(cond)) {                                         \
      std::printf("line %d: %s\n", __LINE__, #cond);       \
      return 1;                                            \
    }                                                      \
  } while (0)

int main() {
  uint32_t seed = 3;
  struct Case { uint64_t rows, cols; uint32_t chunk, layout, mcl, threads; bool uniform; };
  const Case cases[] = {{1, 1, 256, 0, 0, 1, false},     {1, 257, 1024, 0, 12, 2, false}, {3, 4099, 4096, 0, 8, 3, false},
                        {1, 70001, 16384, 0, 10, 4, true}, {32, 768, 8192, 1, 0, 2, false}, {16, 256, 4096, 1, 12, 1, true},
                        {0, 0, 4096, 0, 0, 1, false},    {1, 4096 + 2048, 4096, 0, 0, 1, false}};
  std::vector<std::vector<uint8_t>> blobs;
  for (const Case &c : cases) {
    const uint64_t n = c.rows * c.cols;
    std::vector<uint16_t> x(n + 1);
    for (uint64_t i = 0; i < n; ++i)
      x[i] = c.uniform ? (uint16_t)(lcg(seed) >> 16)
                       : (uint16_t)(((lcg(seed) >> 31) << 15) | ((112 + (lcg(seed) >> 28)) << 7) | (lcg(seed) >> 25));
    zipmoe_encode_opts o = {c.chunk, c.mcl, c.layout, c.threads};
    uint64_t cap = 0, got = 0;
    CHECK(zipmoe_encode_bound(c.rows, c.cols, &o, &cap) == ZIPMOE_OK);
    std::vector<uint8_t> blob(cap);                        // exactly the bound: an overrun is caught
    CHECK(zipmoe_encode(x.data(), c.rows, c.cols, &o, blob.data(), cap, &got) == ZIPMOE_OK && got <= cap);
    blob.resize(got);
    blob.shrink_to_fit();
    CHECK(zipmoe_blob_validate(blob.data(), blob.size()) == ZIPMOE_OK);
    zipmoe_blob_info info;
    CHECK(zipmoe_blob_info_get(blob.data(), blob.size(), &info) == ZIPMOE_OK && info.n_elems == n);
    // damage: every validator path must stay inside the blob
    for (int trial = 0; trial < 200 && got > 0; ++trial) {
      std::vector<uint8_t> bad(blob);
      for (int k = 0; k <= trial % 3; ++k) bad[lcg(seed) % bad.size()] ^= (uint8_t)(1u << (lcg(seed) % 8));
      (void)zipmoe_blob_validate(bad.data(), bad.size());
      std::vector<zipmoe_chunk_desc> d(info.n_chunks + 1);
      zipmoe_table t;
      (void)zipmoe_blob_plan(bad.data(), bad.size(), 0, 0, 0, 0, 0, 0, d.data(), &t);
      bad.resize(lcg(seed) % (bad.size() + 1));            // and truncation
      std::vector<uint8_t> cut(bad);
      (void)zipmoe_blob_validate(cut.data(), cut.size());
    }
    blobs.push_back(blob);
  }
  // one launch over all of them
  std::vector<const void *> ptrs;
  std::vector<uint64_t> sizes;
  for (auto &b : blobs) {
    ptrs.push_back(b.data());
    sizes.push_back(b.size());
  }
  zipmoe_launch_info li;
  CHECK(zipmoe_launch_plan_size(ptrs.data(), sizes.data(), (uint32_t)ptrs.size(), &li) == ZIPMOE_OK);
  std::vector<uint8_t> payload(li.payload_bytes + ZIPMOE_DEVICE_PAD_BYTES), sm(li.sm_bytes + ZIPMOE_DEVICE_PAD_BYTES);
  std::vector<zipmoe_chunk_desc> descs(li.n_chunks);
  std::vector<zipmoe_table> tables(ptrs.size());
  std::vector<uint32_t> first(ptrs.size());
  std::vector<uint64_t> out_base(ptrs.size());
  CHECK(zipmoe_launch_plan(ptrs.data(), sizes.data(), (uint32_t)ptrs.size(), payload.data(), sm.data(), descs.data(),
                           tables.data(), first.data(), out_base.data(), &li) == ZIPMOE_OK);
  // the planners
  const double f[6] = {0.9, 0.6, 0.3, 0.1, 0.06, 0.04};
  double q[6], expected = 0, ratios[4];
  uint32_t iters = 0, cap4[4];
  CHECK(zipmoe_plan_selection_probs(f, 6, 2, 500, 1e-12, q, &iters) == ZIPMOE_OK);
  zipmoe_plan_costs pc = {1.0, 0.2, 2.0, 2, 3, 3};
  const double sizes4[4] = {6, 4, 3, 1};
  CHECK(zipmoe_plan_cache_pools(f, 6, 2, 0xF, 12.0, sizes4, &pc, 0.25, ratios, cap4, &expected) == ZIPMOE_OK);
  const zipmoe_sched_task tasks[5] = {{0, 0}, {0, 0}, {1, 1}, {2, 2}, {3, 3}};
  const double p[4] = {1.0, 0.5, 2.0, 0.3};
  zipmoe_sched_costs sc = {0.7, 1.5, 0.4, 3, 2};
  uint32_t order[5], block_of[5], nb = 0;
  double mk = 0, mk2 = 0, charge = 0;
  CHECK(zipmoe_plan_schedule(tasks, 5, p, 4, &sc, order, block_of, &nb, &mk) == ZIPMOE_OK && nb >= 1);
  CHECK(zipmoe_plan_simulate(tasks, 5, p, 4, &sc, order, block_of, &mk2, &charge) == ZIPMOE_OK && mk == mk2);
  std::puts("ok");
  return 0;
}
