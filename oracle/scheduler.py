"""CPU oracle for the cache-affinity scheduler (paper Section 3.3 "Cache-Affinity Scheduler"; Appendix
"ZipMoE's Scheduler", Algorithm "Cache-Affinity Scheduling"; Appendix "Theoretical Analysis", Definitions
"Charge" and "Critical-Path", Lemma 1, Theorem 1).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests may import this module.  Plain Python, written for reading,
shares nothing with the library's planner.

The model, in the paper's notation.  A request set Q holds one reconstruction task per tensor of every selected
expert.  Task j belongs to expert n(j) and has a compression state:
    "M" missed   : E-chunks and SM-chunk must be read        "C" compressed expert: both are cached
    "S" SM-expert: SM-chunk cached, E-chunks must be read     "E" E-expert         : E-chunks cached, SM-chunk read
Costs: u = read of one SM-chunk; one of the K E-chunks of a tensor reads in rho * u / K and decompresses in c;
p[n] = GPU time of all tokens routed to expert n.  Resources: one I/O thread, L decompression workers, one GPU
stream.  A tensor is recovered once its K E-chunks are decompressed and its SM-chunk is in memory (the recovery
kernel itself is taken as free: Section 3.3 calls it negligible); an expert executes once all its tensors in Q
are recovered; the GPU runs one expert at a time.  Makespan = completion of the last expert.

How a priority order becomes a schedule (Appendix "ZipMoE's Scheduler": the workers and the I/O thread fetch the
first available operation in a work-conserving manner, following the priority order of the blocks; Section 3.3:
within a block E-chunks are loaded before SM-chunks, each kind in the order of the block's tasks; blocks run one
after the other):
  * I/O thread: for every block in turn, the E-chunk reads of its tasks in task order, then its SM-chunk reads
    in task order, back to back from time 0;
  * workers: whenever a worker is free it takes, among the decompression operations whose E-chunk is in memory,
    the one highest in priority (block, position in the block, chunk index); with none ready it waits for the
    next arrival;
  * GPU: whenever free it runs, among the experts whose tensors are all recovered, the one whose first task is
    highest in priority.

Readings where the paper is silent or garbled (listed in the design notes as well):
  * Eq. "compute_dominate" prints `k * rho / K * u` with an unbound k; the text of Section 3.3 says "the l-th
    earliest decompression thread lags behind the I/O thread by at least l * rho / K * u" for 1 <= l <= min(L, K):
    k is read as l, the rank of the thread by completion time.
  * "no additional idle period on any thread" is measured by the total charge of Definition "Charge" (idle time
    of a worker directly before an operation) over the schedule of all blocks built so far plus the candidate.
  * A candidate with no such position goes directly after the last task of the preferred type whose expert time is
    at least its own; with none of those, to the end of the block.
  * Type-II tasks left over when the Type-I list runs empty form a last block in their sorted order.
  * The critical path z_j of Definition "Critical-Path" adds the E-chunk reads and the decompression as if they
    did not overlap; in this model they pipeline (Section 3.1: decompression overlaps loading), so for L < K a
    single task can finish earlier than the printed z_j.  With L >= K the two agree exactly (pinned in the tests).
"""
import itertools

NEEDS_E_READ = {"M": True, "S": True, "C": False, "E": False}
NEEDS_SM_READ = {"M": True, "E": True, "C": False, "S": False}


class Instance:
    """tasks: list of (expert, state); p: dict or list expert -> GPU time; costs c, u, rho, K, L."""

    def __init__(self, tasks, p, c, u, rho, K, L):
        self.tasks = [(int(n), str(s)) for n, s in tasks]
        self.p = p
        self.c, self.u, self.rho, self.K, self.L = float(c), float(u), float(rho), int(K), int(L)
        assert self.K >= 1 and self.L >= 1 and all(s in NEEDS_E_READ for _, s in self.tasks)

    def type_one(self, j):
        """Type-I: the task's reconstruction has to load an SM-chunk (Section 3.3, "Task Partition")."""
        return NEEDS_SM_READ[self.tasks[j][1]]

    def p_of(self, j):
        return self.p[self.tasks[j][0]]


def simulate(inst, blocks):
    """Schedule of the priority order `blocks` (list of lists of task indices, every task once).  Returns a dict:
    makespan, charge (Definition "Charge", summed), io_end[b] (completion of block b's last read; its start
    if it reads nothing), worker_end (completion time of every worker's last operation so far, per block:
    worker_end[b] is the sorted list after block b's operations), ready[j] (recovery time of task j)."""
    K, L, c = inst.K, inst.L, inst.c
    e_read = inst.rho * inst.u / K
    arrive = {}                    # (task, chunk) -> time its E-chunk is in memory
    sm_at = {}
    t = 0.0
    io_end = []
    for B in blocks:
        for j in B:
            for v in range(K):
                if NEEDS_E_READ[inst.tasks[j][1]]:
                    t += e_read
                    arrive[(j, v)] = t
                else:
                    arrive[(j, v)] = 0.0
        for j in B:
            if NEEDS_SM_READ[inst.tasks[j][1]]:
                t += inst.u
                sm_at[j] = t
            else:
                sm_at[j] = 0.0
        io_end.append(t)
    ops = [(b, i, v, j) for b, B in enumerate(blocks) for i, j in enumerate(B) for v in range(K)]   # priority order
    free_at = [0.0] * L
    done_at = {}
    charge = 0.0
    block_of_op_end = [[0.0] * L for _ in blocks]
    pending = list(ops)
    now = 0.0
    while pending:
        w = min(range(L), key=lambda k: (free_at[k], k))       # the worker that frees up first
        now = max(now, free_at[w])
        ready = [op for op in pending if arrive[(op[3], op[2])] <= now + 1e-12]
        if not ready:                                          # wait for the next E-chunk
            now = min(arrive[(op[3], op[2])] for op in pending)
            continue
        op = ready[0]                                          # pending is kept in priority order
        pending.remove(op)
        charge += now - free_at[w]
        free_at[w] = now + c
        done_at[(op[3], op[2])] = free_at[w]
        block_of_op_end[op[0]][w] = free_at[w]
    worker_end, run = [], [0.0] * L
    for b in range(len(blocks)):
        run = [max(r, x) for r, x in zip(run, block_of_op_end[b])]
        worker_end.append(sorted(run))
    ready_at = {j: max([sm_at[j]] + [done_at[(j, v)] for v in range(K)]) for B in blocks for j in B}
    # GPU: one expert at a time, in priority order among those that are ready
    first_pos, exp_ready = {}, {}
    for rank, j in enumerate(j for B in blocks for j in B):
        n = inst.tasks[j][0]
        first_pos.setdefault(n, rank)
        exp_ready[n] = max(exp_ready.get(n, 0.0), ready_at[j])
    left = set(exp_ready)
    gpu = 0.0
    while left:
        can = [n for n in left if exp_ready[n] <= gpu + 1e-12]
        if not can:
            gpu = min(exp_ready[n] for n in left)
            continue
        n = min(can, key=lambda m: first_pos[m])
        gpu += inst.p[n]
        left.remove(n)
    return {"makespan": gpu, "charge": charge, "io_end": io_end, "worker_end": worker_end, "ready": ready_at}


def compute_dominant(inst, blocks):
    """Eq. "compute_dominate" for the last block of `blocks`: the l-th earliest worker completes at least
    l * rho * u / K after the block's I/O, for every l up to min(L, K)."""
    s = simulate(inst, blocks)
    f_io, ends = s["io_end"][-1], s["worker_end"][-1]
    step = inst.rho * inst.u / inst.K
    return all(ends[l - 1] - f_io >= l * step - 1e-12 for l in range(1, min(inst.L, inst.K) + 1))


def sorted_tasks(inst, type_one):
    """sigma_I / sigma_II: non-increasing expert time, tasks of an expert together (then by task index)."""
    js = [j for j in range(len(inst.tasks)) if inst.type_one(j) == type_one]
    return sorted(js, key=lambda j: (-inst.p_of(j), inst.tasks[j][0], j))


def cache_affinity_blocks(inst):
    """Algorithm "Cache-Affinity Scheduling": the ordered list of blocks."""
    sig1, sig2 = sorted_tasks(inst, True), sorted_tasks(inst, False)
    blocks = []
    while sig1:
        B = [sig1.pop(0)]
        U = sig2 + sig1                                         # Type-II candidates first
        while U and not compute_dominant(inst, blocks + [B]):
            j = U.pop(0)
            (sig2 if j in sig2 else sig1).remove(j)
            before = simulate(inst, blocks + [B])["charge"]
            for pos in range(len(B) + 1):                       # earliest position that adds no idle time
                cand = B[:pos] + [j] + B[pos:]
                if simulate(inst, blocks + [cand])["charge"] <= before + 1e-9:
                    B = cand
                    break
            else:
                same = [i for i, t in enumerate(B) if not inst.type_one(t) and inst.p_of(t) >= inst.p_of(j)]
                if not any(not inst.type_one(t) for t in B):
                    same = [i for i, t in enumerate(B) if inst.type_one(t) and inst.p_of(t) >= inst.p_of(j)]
                pos = same[-1] + 1 if same else len(B)
                B = B[:pos] + [j] + B[pos:]
        blocks.append(B)
    if sig2:
        blocks.append(list(sig2))
    return blocks


def lower_bound(inst):
    """Lemma 1's bound on any schedule in this model: total I/O, total decompression over L workers, total GPU
    time, and the longest single-task path.  (The single-task term uses what every schedule must respect here:
    a task's last E-chunk cannot be in memory before all its K reads, its K decompressions spread over at most
    min(K, L) workers, and its reads share one I/O thread.)"""
    c, u, rho, K, L = inst.c, inst.u, inst.rho, inst.K, inst.L
    io = sum((rho * u if NEEDS_E_READ[s] else 0.0) + (u if NEEDS_SM_READ[s] else 0.0) for _, s in inst.tasks)
    comp = len(inst.tasks) * K * c / L
    gpu = sum(inst.p[n] for n in {n for n, _ in inst.tasks})
    z = 0.0
    for n, s in inst.tasks:
        e, m = (rho * u if NEEDS_E_READ[s] else 0.0), (u if NEEDS_SM_READ[s] else 0.0)
        z = max(z, max(e + c, K * c / min(K, L), e + m) + inst.p[n])
    return max(io, comp, gpu, z)


def critical_path_as_printed(inst, j):
    """z_j of Definition "Critical-Path", as the paper prints it."""
    n, s = inst.tasks[j]
    return (inst.rho * inst.u if s in "MS" else 0.0) + max(inst.K * inst.c / min(inst.K, inst.L),
                                                             inst.u if s in "ME" else 0.0) + inst.p[n]


def best_blocks(inst):
    """Brute force over every priority order of the tasks and every way of cutting it into blocks (tiny
    instances only): the smallest makespan any of them reaches, and blocks that reach it."""
    n = len(inst.tasks)
    best, arg = float("inf"), None
    for perm in itertools.permutations(range(n)):
        for cuts in itertools.product((False, True), repeat=max(0, n - 1)):
            blocks, cur = [], [perm[0]] if n else []
            for k in range(1, n):
                if cuts[k - 1]:
                    blocks.append(cur)
                    cur = []
                cur.append(perm[k])
            if cur:
                blocks.append(cur)
            m = simulate(inst, blocks)["makespan"]
            if m < best - 1e-12:
                best, arg = m, blocks
    return best, arg
