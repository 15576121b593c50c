// Host-side cache-affinity scheduler (no CUDA): the paper's Section 3.3 "Cache-Affinity Scheduler" and the
// appendix's Algorithm "Cache-Affinity Scheduling", as a simulator.  Reconstruction tasks (one per tensor of every
// selected expert) are partitioned into Type-I (an SM-chunk has to be read) and Type-II, sorted by expert time,
// and grouped into blocks around Type-I bases until a block is compute-dominant (Eq. "compute_dominate"); the
// blocks' priority order is then turned into a schedule on one I/O thread, L decompression workers and one GPU
// stream, all work-conserving.  Task states: 0 = M missed (E-chunks and SM-chunk read), 1 = C compressed in
// memory, 2 = S SM-chunk in memory (E-chunks read), 3 = E E-chunks in memory (SM-chunk read).
#include <algorithm>
#include <cstdint>
#include <limits>
#include <vector>

#include "zipmoe.h"

namespace {

constexpr double kEps = 1e-12;

struct Model {
  const zipmoe_sched_task *tasks;
  uint32_t n_tasks;
  const double *p;
  uint32_t n_experts;
  zipmoe_sched_costs k;
  bool reads_e(uint32_t j) const { return tasks[j].state == 0 || tasks[j].state == 2; }
  bool reads_sm(uint32_t j) const { return tasks[j].state == 0 || tasks[j].state == 3; }   // Type-I
  double p_of(uint32_t j) const { return p[tasks[j].expert]; }
};

struct Outcome {
  double makespan = 0, charge = 0;
  double io_end_last = 0;              // completion of the last block's reads
  std::vector<double> worker_end;      // per worker, completion of its last operation (all blocks)
};

// The schedule of a priority order: order[i] = task, block_of[i] = its block (non-decreasing).
Outcome simulate(const Model &m, const std::vector<uint32_t> &order, const std::vector<uint32_t> &block_of) {
  const uint32_t n = (uint32_t)order.size(), K = m.k.K, L = m.k.L;
  const double e_read = m.k.rho * m.k.u / K;
  std::vector<double> arrive((size_t)n * K, 0.0), sm_at(n, 0.0);
  Outcome out;
  // I/O thread: per block, E-chunk reads in task order, then SM-chunk reads in task order
  double t = 0;
  for (uint32_t a = 0; a < n;) {
    uint32_t b = a;
    while (b < n && block_of[b] == block_of[a]) ++b;
    for (uint32_t i = a; i < b; ++i)
      if (m.reads_e(order[i]))
        for (uint32_t v = 0; v < K; ++v) arrive[(size_t)i * K + v] = (t += e_read);
    for (uint32_t i = a; i < b; ++i)
      if (m.reads_sm(order[i])) sm_at[i] = (t += m.k.u);
    a = b;
  }
  out.io_end_last = t;
  // workers: the one that frees up first takes the first operation (in priority order) whose chunk has arrived
  const size_t n_ops = (size_t)n * K;
  std::vector<char> done(n_ops, 0);
  std::vector<double> finish(n_ops, 0.0), free_at(L, 0.0);
  size_t first_open = 0;
  double now = 0;
  for (size_t left = n_ops; left > 0;) {
    uint32_t w = 0;
    for (uint32_t x = 1; x < L; ++x)
      if (free_at[x] < free_at[w]) w = x;
    now = std::max(now, free_at[w]);
    while (first_open < n_ops && done[first_open]) ++first_open;
    size_t pick = n_ops;
    double next_arrival = std::numeric_limits<double>::infinity();
    for (size_t o = first_open; o < n_ops; ++o) {
      if (done[o]) continue;
      if (arrive[o] <= now + kEps) {
        pick = o;
        break;
      }
      next_arrival = std::min(next_arrival, arrive[o]);
    }
    if (pick == n_ops) {   // nothing has arrived yet: wait
      now = next_arrival;
      continue;
    }
    out.charge += now - free_at[w];
    free_at[w] = now + m.k.c;
    finish[pick] = free_at[w];
    done[pick] = 1;
    --left;
  }
  out.worker_end = free_at;
  std::sort(out.worker_end.begin(), out.worker_end.end());
  // experts: ready once all their tasks are recovered; the GPU runs the ready expert that comes first in the order
  std::vector<double> ready(m.n_experts, -1.0);
  std::vector<uint32_t> first_pos(m.n_experts, n);
  for (uint32_t i = 0; i < n; ++i) {
    const uint32_t e = m.tasks[order[i]].expert;
    double r = sm_at[i];
    for (uint32_t v = 0; v < K; ++v) r = std::max(r, finish[(size_t)i * K + v]);
    ready[e] = std::max(ready[e], r);
    first_pos[e] = std::min(first_pos[e], i);
  }
  double gpu = 0;
  for (;;) {
    uint32_t pick = m.n_experts;
    double soonest = std::numeric_limits<double>::infinity();
    bool any = false;
    for (uint32_t e = 0; e < m.n_experts; ++e) {
      if (first_pos[e] == n) continue;   // not requested, or already run
      any = true;
      if (ready[e] <= gpu + kEps) {
        if (pick == m.n_experts || first_pos[e] < first_pos[pick]) pick = e;
      } else {
        soonest = std::min(soonest, ready[e]);
      }
    }
    if (!any) break;
    if (pick == m.n_experts) {
      gpu = soonest;
      continue;
    }
    gpu += m.p[pick];
    first_pos[pick] = n;
  }
  out.makespan = gpu;
  return out;
}

// The blocks built so far followed by the candidate block, as one priority order.
struct Plan {
  std::vector<uint32_t> order, block_of;
  void append(const std::vector<uint32_t> &block, uint32_t id) {
    for (uint32_t j : block) {
      order.push_back(j);
      block_of.push_back(id);
    }
  }
};

Outcome with_block(const Model &m, const Plan &fixed, const std::vector<uint32_t> &block, uint32_t id) {
  Plan p = fixed;
  p.append(block, id);
  return simulate(m, p.order, p.block_of);
}

// Eq. "compute_dominate" with the rank of the worker in the place of the printed k: the l-th earliest worker
// completes at least l * rho * u / K after the block's reads, for l = 1 .. min(L, K).
bool compute_dominant(const Model &m, const Outcome &o) {
  const double step = m.k.rho * m.k.u / m.k.K;
  const uint32_t top = std::min(m.k.L, m.k.K);
  for (uint32_t l = 1; l <= top; ++l)
    if (o.worker_end[l - 1] - o.io_end_last < l * step - kEps) return false;
  return true;
}

std::vector<uint32_t> sorted_by_expert_time(const Model &m, bool type_one) {
  std::vector<uint32_t> js;
  for (uint32_t j = 0; j < m.n_tasks; ++j)
    if (m.reads_sm(j) == type_one) js.push_back(j);
  std::stable_sort(js.begin(), js.end(), [&](uint32_t a, uint32_t b) {
    if (m.p_of(a) != m.p_of(b)) return m.p_of(a) > m.p_of(b);
    return m.tasks[a].expert < m.tasks[b].expert;   // tasks of an expert together; then by task index (stable)
  });
  return js;
}

bool model_ok(const zipmoe_sched_task *tasks, uint32_t n_tasks, const double *p, uint32_t n_experts,
              const zipmoe_sched_costs *k) {
  if (!tasks || !p || !k || n_tasks == 0 || n_experts == 0 || k->K < 1 || k->L < 1) return false;
  if (!(k->c >= 0) || !(k->u >= 0) || !(k->rho >= 0)) return false;
  if ((uint64_t)n_tasks * k->K > (1u << 22)) return false;
  for (uint32_t j = 0; j < n_tasks; ++j)
    if (tasks[j].expert >= n_experts || tasks[j].state > 3 || !(p[tasks[j].expert] >= 0)) return false;
  return true;
}

}  // namespace

extern "C" zipmoe_status zipmoe_plan_simulate(const zipmoe_sched_task *tasks, uint32_t n_tasks, const double *p,
                                              uint32_t n_experts, const zipmoe_sched_costs *costs, const uint32_t *order,
                                              const uint32_t *block_of, double *makespan, double *charge) {
  if (!model_ok(tasks, n_tasks, p, n_experts, costs) || !order || !block_of || !makespan) return ZIPMOE_ERR_INVALID_ARG;
  std::vector<char> seen(n_tasks, 0);
  for (uint32_t i = 0; i < n_tasks; ++i) {
    if (order[i] >= n_tasks || seen[order[i]] || (i > 0 && block_of[i] < block_of[i - 1])) return ZIPMOE_ERR_INVALID_ARG;
    seen[order[i]] = 1;
  }
  const Model m{tasks, n_tasks, p, n_experts, *costs};
  const Outcome o = simulate(m, std::vector<uint32_t>(order, order + n_tasks), std::vector<uint32_t>(block_of, block_of + n_tasks));
  *makespan = o.makespan;
  if (charge) *charge = o.charge;
  return ZIPMOE_OK;
}

extern "C" zipmoe_status zipmoe_plan_schedule(const zipmoe_sched_task *tasks, uint32_t n_tasks, const double *p,
                                              uint32_t n_experts, const zipmoe_sched_costs *costs, uint32_t *order,
                                              uint32_t *block_of, uint32_t *n_blocks, double *makespan) {
  if (!model_ok(tasks, n_tasks, p, n_experts, costs) || !order || !block_of) return ZIPMOE_ERR_INVALID_ARG;
  const Model m{tasks, n_tasks, p, n_experts, *costs};
  std::vector<uint32_t> sig1 = sorted_by_expert_time(m, true), sig2 = sorted_by_expert_time(m, false);
  Plan plan;
  uint32_t id = 0;
  while (!sig1.empty()) {
    std::vector<uint32_t> block{sig1.front()};
    sig1.erase(sig1.begin());
    Outcome cur = with_block(m, plan, block, id);
    while (!(sig1.empty() && sig2.empty()) && !compute_dominant(m, cur)) {
      // the candidate: Type-II tasks first, then the remaining Type-I tasks
      std::vector<uint32_t> &from = sig2.empty() ? sig1 : sig2;
      const uint32_t j = from.front();
      from.erase(from.begin());
      bool placed = false;
      for (size_t pos = 0; pos <= block.size() && !placed; ++pos) {   // earliest position that adds no idle time
        std::vector<uint32_t> cand = block;
        cand.insert(cand.begin() + (std::ptrdiff_t)pos, j);
        const Outcome o = with_block(m, plan, cand, id);
        if (o.charge <= cur.charge + 1e-9) {
          block.swap(cand);
          cur = o;
          placed = true;
        }
      }
      if (!placed) {
        // after the last Type-II task with at least its expert time; after such a Type-I task if the block has
        // no Type-II task; at the end if there is none
        bool has_two = false;
        for (uint32_t t : block) has_two = has_two || !m.reads_sm(t);
        size_t pos = block.size();
        bool found = false;
        for (size_t i = 0; i < block.size(); ++i)
          if (m.reads_sm(block[i]) == !has_two && m.p_of(block[i]) >= m.p_of(j)) {
            pos = i + 1;
            found = true;
          }
        if (!found) pos = block.size();
        block.insert(block.begin() + (std::ptrdiff_t)pos, j);
        cur = with_block(m, plan, block, id);
      }
    }
    plan.append(block, id++);
  }
  if (!sig2.empty()) plan.append(sig2, id++);   // Type-II tasks that no block took
  for (uint32_t i = 0; i < n_tasks; ++i) {
    order[i] = plan.order[i];
    block_of[i] = plan.block_of[i];
  }
  if (n_blocks) *n_blocks = id;
  if (makespan) *makespan = simulate(m, plan.order, plan.block_of).makespan;
  return ZIPMOE_OK;
}
