#!/usr/bin/env python
"""Benchmark of the ZipMoE decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the decode path over one MoE layer of compressed
expert weights: a single zipmoe_decode launch that decompresses every E-chunk
and re-assembles every bf16 tensor of the layer.  Prints ONE JSON line.

* value      : decoded bf16 GB/s, whole job, compressed inputs resident in HBM, on the
               largest single-GPU configuration (8 experts of 14336x4096, 2.8 GB of bf16).
               The loop of K launches is repeated until at least a second of device time
               has passed; `value` is taken from the median loop, `best` from the fastest.
* configs    : the same measurement (shorter) on every other decode configuration.
* e2e        : the same through the C ABI with HOST buffers: compressed streams
               copied host->device from pinned memory, decode, decoded tensors
               copied device->host, all inside the timed region.
* roofline   : algorithmic bytes of one launch (E-chunk section + sign/mantissa
               bytes read + bf16 written) / launch duration, against the
               measured HBM copy bandwidth of this machine's B200s.
* cpu_baseline: the CPU oracle (test infrastructure; plain C, bit-by-bit
               decoder) on a bounded sample of the same workload: one thread,
               and one thread per host core over chunks.
* --impl reference: the oracle alone, timed on the host cores; loads nothing of the CUDA library.
"""
import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decoded bf16 GB/s (lossless decode of compressed MoE expert weights), 1 B200, bit-exact"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "large_layer"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


def build_workload(name, keep_originals, experts=None, max_code_len=0):
    from paper_2601_21198_b200 import workloads
    if name == "small_layer":
        return workloads.small_layer(n_experts=experts or 64, keep_originals=keep_originals, max_code_len=max_code_len)
    if name == "large_layer":
        return workloads.large_layer(n_experts=experts or 8, keep_originals=keep_originals, max_code_len=max_code_len)
    if name == "single_matrix":
        return workloads.single_matrix(keep_originals=keep_originals, max_code_len=max_code_len)
    if name.startswith("stress"):      # stress1024 / stress16384 / stress262144: the stress-set tensors of one chunk size
        return workloads.stress_set(chunk_elems=int(name[6:]), keep_originals=keep_originals)[0]
    raise SystemExit("unknown workload %s" % name)


# ----------------------------------------------------------------------------- CPU oracle leg
# Everything here uses the seeded generators and the oracle only: the tensors are encoded by the oracle's own
# encoder and decoded by its bit-by-bit decoder, chunk by chunk.
ORACLE_SAMPLE = {
    # workload -> (description, thunk giving the sample tensor, chunk_elems)
    "large_layer": ("the first 8192 rows of expert 0's w1 (14336x4096 bf16, outlier channels), 256K-element chunks",
                    lambda inputs: inputs.outlier_matrix(8192, 4096, 0.015, 300), 262144),
    "small_layer": ("expert 0's gate matrix (1408x2048 bf16), 64K-element chunks",
                    lambda inputs: inputs.small_expert_tensor(0, 0), 65536),
    "single_matrix": ("the 2048x1408 matrix, 4096-element chunks", lambda inputs: inputs.single_expert_matrix(0), 4096),
}


def oracle_sample(workload):
    from paper_2601_21198_b200 import inputs      # seeded draws only: no codec arithmetic, no CUDA library
    from oracle import codec
    key = workload if workload in ORACLE_SAMPLE else "small_layer"
    text, thunk, chunk = ORACLE_SAMPLE[key]
    x = thunk(inputs)
    blob = codec.encode(x, chunk_elems=chunk, max_code_len=12)
    return {"text": text, "x": x, "blob": blob, "n_chunks": codec.info(blob)["n_chunks"]}


def oracle_decode_pass(sample, n_threads):
    """One pass over the sample: every chunk decoded by the oracle, chunks spread over n_threads host threads
    (ctypes releases the GIL; the chunks are independent, which is how the paper spreads E-chunk decompression
    over its L workers).  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import codec
    out = np.empty(sample["x"].size, np.uint16)
    out.fill(0)      # pages touched before the clock starts
    ks = list(range(sample["n_chunks"]))
    t0 = time.perf_counter()
    if n_threads == 1:
        for k in ks:
            codec.decode_chunk(sample["blob"], k, out)
    else:
        with ThreadPoolExecutor(n_threads) as pool:
            list(pool.map(lambda k: codec.decode_chunk(sample["blob"], k, out), ks))
    dt = time.perf_counter() - t0
    assert np.array_equal(out, sample["x"].ravel()), "the oracle's round trip is not the identity"
    return dt


def oracle_rates(sample, budget_s):
    """(single-thread GB/s, all-cores GB/s, threads used, passes) within about budget_s seconds of wall time."""
    cores = os.cpu_count() or 1
    threads = max(1, min(cores, sample["n_chunks"]))
    nbytes = 2.0 * sample["x"].size
    t1 = oracle_decode_pass(sample, 1)
    passes = int(max(1, min(50, (budget_s - t1) / max(t1 / threads * 1.3, 1e-3))))
    tn = min(oracle_decode_pass(sample, threads) for _ in range(passes))
    return nbytes / t1 / 1e9, nbytes / tn / 1e9, threads, passes


def run_reference(args):
    """The oracle as it stands, on the host cores; rank 0 only.  Each step decodes a bounded sample of the
    workload (all of its chunks, one thread per core), sized so that the whole run stays within minutes."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    workload = args.workload or HEADLINE
    sample = oracle_sample(workload)
    cores = os.cpu_count() or 1
    threads = max(1, min(cores, sample["n_chunks"]))
    single = 2.0 * sample["x"].size / oracle_decode_pass(sample, 1) / 1e9
    for _ in range(args.warmup):
        oracle_decode_pass(sample, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_decode_pass(sample, threads)
    dt_all = time.perf_counter() - t0
    value = args.steps * 2.0 * sample["x"].size / dt_all / 1e9
    text = "%s; encoded by the oracle's encoder (12-bit code limit); %d chunks over %d threads per step" % (
        sample["text"], sample["n_chunks"], threads)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt_all / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
        "config": {"workload": WORKLOAD_LABELS.get(workload, workload) + " (bounded sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": text,
                         "single_thread_gbs": single},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


WORKLOAD_LABELS = {"large_layer": "moe8_14336x4096_chunk256K", "small_layer": "moe64_2048x1408_chunk64K",
                   "single_matrix": "single_2048x1408_chunk4096"}


# ----------------------------------------------------------------------------- ranks
def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group (a no-op without one)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_gbs(world, bytes_per_rank_step, steps, ms_max):
    """Every rank decodes its own copy of the layer (weak scaling): aggregate GB/s over the slowest rank's time."""
    return world * bytes_per_rank_step * steps / (ms_max / 1e3) / 1e9


def loops_for(target_s, loop_ms, lo=1, hi=4000):
    """How many loops of loop_ms milliseconds reach target_s seconds."""
    return int(max(lo, min(hi, np.ceil(target_s * 1e3 / max(loop_ms, 1e-3)))))


# ----------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock, power and clock-event reasons through NVML (read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index, period=0.004):
        super().__init__(daemon=True)
        self.period, self.samples, self.stop_flag, self.ok = period, [], False, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.max_mhz = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed"
        if not inside:
            inside, window = self.samples, "warmup+timed"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "window": "none"}
        bits = 0
        for s in inside:
            bits |= s[2]
        reasons = sorted(name for bit, name in self.REASONS.items() if bits & bit)
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_min_mhz": float(min(s[1] for s in inside)),
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(inside), "window": window}


# ----------------------------------------------------------------------------- one decode configuration
def expected_output(w):
    """The launch's whole output buffer as the encoder's inputs say it must be (zero between tensors)."""
    plan = w.plan
    want = np.zeros(plan.out_elems, np.uint16)
    for i, x in enumerate(w.originals):
        want[plan.out_base[i]: plan.out_base[i] + x.size] = x.ravel()
    return want


def measure_decode(w, dev, steps, warmup, target_s, sampler=None, world=1, barrier=None):
    """Times loops of `steps` zipmoe_decode launches of workload w until target_s seconds of device time have
    passed.  Launches whose inputs and outputs would fit the second-level cache rotate through enough copies of
    the buffers to exceed it.  Returns a dict; `verified` means: status word clean and every element of the
    output equal to what the encoder was given."""
    import torch
    plan = w.plan
    alg = plan.algorithmic_bytes()
    copies = 1 if alg > 512e6 else int(np.ceil(512e6 / alg))
    dplans = [plan.to_device(dev) for _ in range(copies)]
    outs = [d.new_output() for d in dplans]
    stream = torch.cuda.current_stream(dev)

    dplans[0].decode(outs[0])
    torch.cuda.synchronize(dev)
    verified = int(dplans[0].status.item()) == 0
    if w.originals is not None:
        want = torch.from_numpy(expected_output(w).view(np.int16)).to(dev)
        verified = verified and bool(torch.equal(outs[0], want))
        del want

    def loop():
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(steps):
            dplans[i % copies].decode(outs[i % copies])
        b.record(stream)
        return a, b

    for i in range(warmup):
        dplans[i % copies].decode(outs[i % copies])
    if barrier:
        barrier()
    a, b = loop()
    torch.cuda.synchronize(dev)
    first = max_over_ranks([a.elapsed_time(b)], dev)[0]
    n_loops = loops_for(target_s, first)
    if barrier:
        barrier()
    t0 = time.perf_counter()
    evs = [loop() for _ in range(n_loops)]
    if barrier:
        barrier()
    else:
        torch.cuda.synchronize(dev)
    t1 = time.perf_counter()
    times = max_over_ranks([a.elapsed_time(b) for a, b in evs], dev)
    verified = verified and all(int(d.status.item()) == 0 for d in dplans)
    med, best = float(np.median(times)), float(min(times))
    # small launches with fixed ranges (nothing but the kernel on the stream): also replayed from a CUDA graph that
    # holds one launch per buffer copy, which takes the host's launch cost out of the figure
    in_graph = None
    if copies > 1 and barrier is None and plan.n_tiles >= 512 * plan.n_tables:
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(copies):
                    dplans[i].decode(outs[i])
            for _ in range(3):
                g.replay()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(side)
            for _ in range(20):
                g.replay()
            b.record(side)
        torch.cuda.synchronize(dev)
        in_graph = a.elapsed_time(b) / (20 * copies)
        verified = verified and all(int(d.status.item()) == 0 for d in dplans)
        del g
    peaks, _ = measured_peaks()
    res = {
        "workload": w.label, "tensors": len(w.blobs), "elements": w.n_elems,
        "chunk_elems": int(plan.infos[0].chunk_elems), "max_code_len": int(max(i.max_code_len for i in plan.infos)),
        "tiles": plan.n_tiles, "compressed_over_bf16": w.compressed_bytes() / w.bf16_bytes(),
        "ms_per_launch": med / steps, "ms_per_launch_best": best / steps, "loops": n_loops, "launches_per_loop": steps,
        "decoded_gbs": whole_job_gbs(world, w.bf16_bytes(), steps, med),
        "decoded_gbs_best": whole_job_gbs(world, w.bf16_bytes(), steps, best),
        "algorithmic_bytes_per_launch": alg,
        "frac": alg * steps / (med / 1e3) / 1e9 / peaks["hbm_gbs"],
        "frac_best": alg * steps / (best / 1e3) / 1e9 / peaks["hbm_gbs"],
        "buffer_copies_rotated": copies, "status_clean": all(int(d.status.item()) == 0 for d in dplans),
        "ms_per_launch_in_cuda_graph": in_graph,
        "verified_bit_exact": verified, "timed_seconds": sum(times) / 1e3,
    }
    if sampler is not None:
        res["clocks"] = sampler.summary(t0, t1)
    return res


def launch_floor_us(dev, n=200):
    """Microseconds per launch of a kernel that does next to nothing (a 1-element fill), back to back on the
    stream: what any single-launch measurement of a tiny workload cannot go below."""
    import torch
    x = torch.zeros(1, device=dev)
    stream = torch.cuda.current_stream(dev)
    for _ in range(20):
        x.fill_(1.0)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(n):
        x.fill_(1.0)
    b.record(stream)
    torch.cuda.synchronize(dev)
    return a.elapsed_time(b) / n * 1e3


# ----------------------------------------------------------------------------- DRAM traffic of the profiled kernel
def kernel_source_hash():
    """Identifies the decode kernel's source: a profile taken on other source does not describe this kernel."""
    h = hashlib.sha256()
    for name in ("decode_kernel.cu", "decode_device.cuh", "tile_geometry.h"):
        with open(os.path.join(ROOT, "paper_2601_21198_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(label, elements):
    """dram__bytes_read.sum + dram__bytes_write.sum of one decode_kernel launch on this workload, from the text
    record of the ncu capture kept with the profile summaries; None when there is no capture of this workload
    at this size or the kernel's source has changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    now = kernel_source_hash()
    with open(path) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            kv = dict(item.split("=", 1) for item in ln.split())
            if kv.get("workload") == label and int(kv.get("elements", 0)) == elements and kv.get("source") == now:
                return int(kv["dram_read"]) + int(kv["dram_write"])
    return None


# ----------------------------------------------------------------------------- fused expert FFN
def bench_ffn(dev, iters=20, cpu_tokens=2, token_counts=(1, 16, 64), config="large"):
    """Fused decode + expert SwiGLU FFN against decode-then-GEMM (zipmoe_decode of the routed experts into bf16
    followed by torch matmuls on the same stream), Zipf(1.2) expert popularity.
      config "large": 8 experts of 4096 -> 14336 -> 4096, top-2, T = 1, 16, 64 tokens; also times the CPU oracle's
                      FFN on a few tokens;
      config "small": the 64 experts of the paper's own model shape, 2048 -> 1408 -> 2048 (intermediate size
                      zero-padded to 1536 before encoding), top-6, T = 1, 16 tokens."""
    import torch
    from paper_2601_21198_b200 import binding, inputs, workloads
    if config == "large":
        w = workloads.large_layer(layout=binding.LAYOUT_BLOCKED, keep_originals=True)
        E, H, I, k = 8, 4096, 14336, 2
        label = "8 experts 4096->14336->4096 bf16 (blocked layout, 256K-element chunks), top-2, Zipf(1.2)"
    else:
        w = workloads.small_layer_ffn(keep_originals=False)
        E, H, I, k = 64, w.hidden, w.inter, 6
        label = "64 experts 2048->1408->2048 bf16, intermediate size zero-padded to 1536 (blocked layout, 64K-element chunks), top-6, Zipf(1.2)"
        token_counts = tuple(t for t in token_counts if t <= 16)
        cpu_tokens = 0
    ex = binding.DeviceExperts(w.blobs, H, I, dev)
    per_expert = [binding.DecodePlan(w.blobs[3 * e: 3 * e + 3]).to_device(dev) for e in range(E)]
    dense = [p.new_output() for p in per_expert]
    expert_bytes = [sum(i.payload_bytes + i.n_elems for i in p.plan.infos) for p in per_expert]
    stream = torch.cuda.current_stream(dev)
    out = {}
    for T in token_counts:
        tok = inputs.tokens(T, H, seed=100 + T)
        ids, wts = inputs.routing(T, n_experts=E, k=k, seed=T)
        d_tok = torch.from_numpy(tok.view(np.int16)).to(dev)
        d_ids = torch.from_numpy(ids).to(dev)
        d_wts = torch.from_numpy(wts).to(dev)
        active = sorted(set(ids.ravel().tolist()))
        y = ex.ffn(d_tok, d_ids, d_wts)

        def fused():
            ex.ffn(d_tok, d_ids, d_wts, out=y)

        x_bf = d_tok.view(torch.bfloat16)
        sel = {e: (torch.from_numpy(np.nonzero(ids == e)[0]).to(dev), torch.from_numpy(wts[ids == e]).to(dev))
               for e in active}
        acc = torch.zeros(T, H, dtype=torch.float32, device=dev)

        def unfused():
            acc.zero_()
            for e in active:
                per_expert[e].decode(dense[e])
                p = per_expert[e].plan
                w1 = p.tensor_slice(dense[e], 0).view(torch.bfloat16).view(I, H)
                w3 = p.tensor_slice(dense[e], 1).view(torch.bfloat16).view(I, H)
                w2 = p.tensor_slice(dense[e], 2).view(torch.bfloat16).view(H, I)
                rows, wt = sel[e]
                xe = x_bf[rows]
                h = torch.nn.functional.silu(xe @ w1.T) * (xe @ w3.T)
                acc.index_add_(0, rows, (h @ w2.T).float() * wt[:, None])
            return acc.to(torch.bfloat16)

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize(dev)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(iters):
                fn()
            b.record(stream)
            torch.cuda.synchronize(dev)
            return a.elapsed_time(b) / iters * 1e3      # microseconds

        ref = unfused().float()
        diff = (y.view(torch.bfloat16).float() - ref).abs().max().item()
        us_f, us_u = timed(fused), timed(unfused)
        # the same call replayed from a CUDA graph (what a decode loop would do with it)
        side = torch.cuda.Stream(dev)
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                fused()
            for _ in range(3):
                g.replay()
            ga, gb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ga.record(side)
            for _ in range(iters):
                g.replay()
            gb.record(side)
        torch.cuda.synchronize(dev)
        us_g = ga.elapsed_time(gb) / iters * 1e3
        del g
        nbytes = sum(expert_bytes[e] for e in active)
        out["T%d" % T] = {"us": us_f, "us_in_cuda_graph": us_g, "tokens_per_s": T / us_f * 1e6, "active_experts": len(active),
                          "compressed_gbs": nbytes / us_f / 1e3,
                          # the fused call must at least read the routed experts' compressed bytes once
                          "frac_of_hbm_roofline": nbytes / us_f / 1e3 / measured_peaks()[0]["hbm_gbs"],
                          "decode_then_gemm_us": us_u,
                          "speedup_vs_decode_then_gemm": us_u / us_f, "max_abs_diff_vs_decode_then_gemm": diff,
                          "status": int(ex.dev.status.item())}
    out["config"] = label
    if not cpu_tokens:
        return out
    # CPU oracle FFN on a few tokens of the T = 16 case (fp64 numpy)
    from oracle import ffn as offn
    tok = inputs.tokens(16, 4096, seed=116)
    ids, wts = inputs.routing(16, n_experts=8, k=2, seed=16)
    t0 = time.perf_counter()
    offn.expert_ffn(tok[:cpu_tokens], ids[:cpu_tokens], wts[:cpu_tokens], {e: w.originals[3 * e] for e in range(8)},
                    {e: w.originals[3 * e + 1] for e in range(8)}, {e: w.originals[3 * e + 2] for e in range(8)})
    dt = time.perf_counter() - t0
    out["cpu_oracle"] = {"tokens_per_s": cpu_tokens / dt, "sample": "%d tokens of the T=16 case, fp64 numpy" % cpu_tokens,
                         "cores": os.cpu_count() or 1}
    return out


# ----------------------------------------------------------------------------- end to end with host buffers
def measure_e2e(w, dev, n_slices, steps, barrier, weights_to_host=True):
    """pinned host -> device, decode, device -> pinned host, every step.  The layer is cut into slices of tensors,
    each with its own zipmoe_decode call, spread over a few streams, so that one slice's copy to the host overlaps
    the next slice's copy to the device (the host link is full duplex) and its decode.
    weights_to_host: the decoded bf16 goes back to the host every step (the strict reading of "end to end"); else
    it stays on the device, where an expert would use it, and what the host reads back per slice is the status
    word and a 64-bit sum of the decoded patterns (checked against the sum of the encoder's input)."""
    import torch
    from paper_2601_21198_b200 import binding
    stream = torch.cuda.current_stream(dev)
    n_slices = max(1, min(n_slices, len(w.blobs)))
    bounds = [len(w.blobs) * i // n_slices for i in range(n_slices + 1)]
    slices = []
    for i in range(n_slices):
        sp = binding.DecodePlan(w.blobs[bounds[i]:bounds[i + 1]])
        sd = sp.to_device(dev)
        slices.append({
            "plan": sp, "dev": sd, "out": sd.new_output(), "first": bounds[i],
            "h": [(sd.payload, torch.from_numpy(sp.payload).pin_memory()), (sd.sm, torch.from_numpy(sp.sm).pin_memory()),
                  (sd.descs, torch.from_numpy(sp.descs.view(np.uint8).copy()).pin_memory()),
                  (sd.tables, torch.from_numpy(sp.tables).pin_memory())],
            "h_out": torch.empty(sp.out_elems if weights_to_host else 0, dtype=torch.int16).pin_memory(),
            "sum": torch.zeros(1, dtype=torch.int64, device=dev), "h_sum": torch.zeros(1, dtype=torch.int64).pin_memory(),
            "h_status": torch.zeros(1, dtype=torch.int32).pin_memory()})
    side = [torch.cuda.Stream(dev) for _ in range(min(3, n_slices))]
    h2d_bytes = sum(h.numel() * h.element_size() for sl in slices for _, h in sl["h"])
    d2h_bytes = sum(sl["h_out"].numel() * 2 for sl in slices) if weights_to_host else 12 * len(slices)

    def e2e_step():
        for i, sl in enumerate(slices):
            st = side[i % len(side)]
            with torch.cuda.stream(st):
                for d_t, h_t in sl["h"]:
                    d_t.copy_(h_t, non_blocking=True)
                sl["dev"].decode(sl["out"], stream=st)
                if weights_to_host:
                    sl["h_out"].copy_(sl["out"], non_blocking=True)
                else:
                    sl["sum"].copy_(torch.sum(sl["out"], dtype=torch.int64))
                    sl["h_sum"].copy_(sl["sum"], non_blocking=True)
                    sl["h_status"].copy_(sl["dev"].status, non_blocking=True)

    def e2e_run(n):
        start = torch.cuda.Event(enable_timing=True)
        end = torch.cuda.Event(enable_timing=True)
        start.record(stream)
        for st in side:
            st.wait_event(start)
        for _ in range(n):
            e2e_step()
        for st in side:
            done = torch.cuda.Event()
            done.record(st)
            stream.wait_event(done)
        end.record(stream)
        return start, end

    e2e_run(2)
    barrier()
    f0, f1 = e2e_run(steps)
    barrier()
    ms = f0.elapsed_time(f1)
    ok = all(int(sl["dev"].status.item()) == 0 for sl in slices)
    if w.originals is not None and weights_to_host:      # every tensor, as it arrived on the host
        for sl in slices:
            host = sl["h_out"].numpy().view(np.uint16)
            for j in range(len(sl["plan"].infos)):
                ok = ok and bool(np.array_equal(sl["plan"].tensor_slice(host, j), w.originals[sl["first"] + j].ravel()))
    elif w.originals is not None:                         # the sums and status words that arrived on the host
        for sl in slices:
            want = sum(int(w.originals[sl["first"] + j].view(np.int16).sum(dtype=np.int64)) for j in range(len(sl["plan"].infos)))
            ok = ok and int(sl["h_sum"].item()) == want and int(sl["h_status"].item()) == 0
    return ms, ok, int(h2d_bytes), int(d2h_bytes), n_slices, len(side)


# ----------------------------------------------------------------------------- GPU leg
def run_ours(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    from paper_2601_21198_b200 import binding, build
    build.build()
    if args.ffn_only:      # profiling captures of the fused kernels on one token count
        res = bench_ffn(dev, iters=args.ffn_iters, cpu_tokens=0, token_counts=tuple(int(t) for t in args.ffn_only.split(",")),
                        config=args.ffn_config)
        print(json.dumps({"ffn": res}))
        return
    profiling = args.experts is not None or args.quick     # a small case for a profiler: no side sections
    name = args.workload or HEADLINE
    w = build_workload(name, keep_originals=not profiling, experts=args.experts, max_code_len=args.max_code_len)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    sampler = ClockSampler(local)
    sampler.start()
    head = measure_decode(w, dev, args.steps, args.warmup, 0.0 if profiling else args.min_seconds, sampler, world, barrier)
    verified = head["verified_bit_exact"]
    e2e_steps = max(1, min(args.steps, 6))
    if profiling:
        e2e_ms, e2e_ok, h2d_bytes, d2h_bytes, n_slices, n_side = None, True, 0, 0, 0, 0
        dev_ms, dev_ok, dev_d2h = None, True, 0
    else:
        e2e_ms, e2e_ok, h2d_bytes, d2h_bytes, n_slices, n_side = measure_e2e(w, dev, args.e2e_slices, e2e_steps, barrier)
        e2e_ms = max_over_ranks([e2e_ms], dev)[0]
        dev_ms, dev_ok, _, dev_d2h, _, _ = measure_e2e(w, dev, args.e2e_slices, e2e_steps, barrier, weights_to_host=False)
        dev_ms = max_over_ranks([dev_ms], dev)[0]
    verified = verified and e2e_ok and dev_ok
    sampler.stop_flag = True

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        bf16_bytes = w.bf16_bytes()
        plan = w.plan
        alg = head["algorithmic_bytes_per_launch"]
        per_launch_s = head["ms_per_launch"] / 1e3
        achieved = alg / per_launch_s / 1e9
        line = {
            "metric": METRIC, "value": head["decoded_gbs"], "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": head["ms_per_launch"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": w.label, "tensors": len(w.blobs), "elements": w.n_elems,
                       "chunk_elems": head["chunk_elems"], "max_code_len": head["max_code_len"], "chunks": plan.n_chunks,
                       "tiles": plan.n_tiles, "compressed_over_bf16": head["compressed_over_bf16"],
                       "l2": "inputs and outputs of one step (%.2f GB) exceed L2; no flush" % (alg / 1e9),
                       "sharding": "every rank decodes its own copy of the layer; no collective",
                       "timing": "loops of `steps` launches repeated for >= %.1f s of device time; value from the median "
                                 "loop, best from the fastest" % args.min_seconds},
            "timed": {"loops": head["loops"], "seconds": head["timed_seconds"], "ms_per_step_median": head["ms_per_launch"],
                      "ms_per_step_best": head["ms_per_launch_best"], "value_best": head["decoded_gbs_best"]},
            "clocks": head.get("clocks"),
            "e2e": {"value": None if e2e_ms is None else whole_job_gbs(world, bf16_bytes, e2e_steps, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes, "steps": e2e_steps,
                    "slices": n_slices, "streams": n_side,
                    "weights_stay_on_device": {
                        "value": None if dev_ms is None else whole_job_gbs(world, bf16_bytes, e2e_steps, dev_ms),
                        "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": dev_d2h,
                        "what": "same copies to the device and decodes; the host reads back each slice's status word "
                                "and a 64-bit sum of the decoded patterns instead of the bf16 weights"}},
            "gpu_launches": args.steps * head["loops"],
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "frac_best": head["frac_best"],
                         "traffic": recorded_traffic(w.label, w.n_elems),
                         "peak_kind": "of " + peak_kind, "algorithmic_bytes_per_launch": alg,
                         "kernel": "zipmoe_dev::decode_kernel", "launch_ms": head["ms_per_launch"]},
            "verified_bit_exact": verified,
        }
        del w
        torch.cuda.empty_cache()
        if world == 1 and not profiling:
            line["configs"] = other_configs(dev, args, name, head)
            line["launch_floor_us"] = launch_floor_us(dev)
            side_sections(line, dev, args)
            sample = oracle_sample(name)
            one, many, threads, passes = oracle_rates(sample, 20.0)
            line["cpu_baseline"] = {"value": many, "unit": UNIT, "cores": threads, "kind": "oracle",
                                    "single_thread_gbs": one,
                                    "sample": "%s, encoded and decoded by the oracle; best of %d passes over its %d "
                                              "chunks on %d threads" % (sample["text"], passes, sample["n_chunks"], threads)}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def other_configs(dev, args, headline_name, head):
    """Every other decode configuration, each timed for about half a second of device time."""
    import torch
    out = {headline_name: {k: v for k, v in head.items() if k != "clocks"}}
    todo = [("single_matrix", 0), ("small_layer", 0), ("small_layer_12bit", 12), ("large_layer", 0), ("stress1024", 0),
            ("stress16384", 0), ("stress262144", 0)]
    for key, mcl in todo:
        name = key.replace("_12bit", "")
        if key == headline_name:
            continue
        w = build_workload(name, keep_originals=True, max_code_len=mcl)
        r = measure_decode(w, dev, min(args.steps, 20), 3, args.min_seconds / 2)
        out[key] = r
        del w
        torch.cuda.empty_cache()
    return out


def side_sections(line, dev, args):
    """The paper's recovery step alone, the compression-state variants, and the fused expert FFN."""
    import torch
    from paper_2601_21198_b200 import binding
    peaks, _ = measured_peaks()
    stream = torch.cuda.current_stream(dev)
    w = build_workload("small_layer", keep_originals=False)
    plan = w.plan
    dplan = plan.to_device(dev)
    out = dplan.new_output()
    bf16_bytes = w.bf16_bytes()
    # the paper's own GPU step alone (merge of decompressed exponent bytes and SM bytes), same element count
    n = w.n_elems
    d_e = torch.randint(0, 256, (n,), dtype=torch.uint8, device=dev)
    d_s = torch.randint(0, 256, (n,), dtype=torch.uint8, device=dev)
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(105):
        if it == 5:
            r0.record(stream)
        binding.zipmoe_recover(d_e, d_s, n, out, stream.cuda_stream)
    r1.record(stream)
    torch.cuda.synchronize(dev)
    rms = r0.elapsed_time(r1) / 100
    line["recover_kernel"] = {"workload": w.label, "decoded_bf16_gbs": 2 * n / rms / 1e6, "traffic_gbs": 4 * n / rms / 1e6,
                              "frac_of_peak": 4 * n / rms / 1e6 / peaks["hbm_gbs"], "ms": rms,
                              "note": "exponent bytes already decompressed: 2 B read + 2 B written per element"}
    del d_e, d_s
    # compression states: one stream stays in pinned host memory and is read in place over the host link
    states = {"workload": w.label}
    h_pay = torch.from_numpy(plan.payload).pin_memory()
    h_sm = torch.from_numpy(plan.sm).pin_memory()
    d_pay, d_sm = dplan.payload, dplan.sm
    for name, (pay, smb, moved) in {"sm_chunks_on_host": (d_pay, h_sm, int(h_sm.numel())),
                                    "e_chunks_on_host": (h_pay, d_sm, int(h_pay.numel()))}.items():
        dplan.payload, dplan.sm = pay, smb
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dplan.decode(out)
        c0.record(stream)
        for _ in range(3):
            dplan.decode(out)
        c1.record(stream)
        torch.cuda.synchronize(dev)
        cms = c0.elapsed_time(c1) / 3
        states[name] = {"decoded_bf16_gbs": bf16_bytes / cms / 1e6, "ms": cms,
                        "host_bytes_read_per_step": moved, "host_link_gbs": moved / cms / 1e6}
    dplan.payload, dplan.sm = d_pay, d_sm
    line["compression_states"] = states
    del dplan, out, h_pay, h_sm, w
    torch.cuda.empty_cache()
    if not args.no_ffn:
        line["ffn"] = bench_ffn(dev)
        line["ffn_small_experts"] = bench_ffn(dev, config="small")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None,
                    choices=["small_layer", "large_layer", "single_matrix", "stress1024", "stress16384", "stress262144"],
                    help="the configuration of the headline figure (default: the 8-expert 14336x4096 layer)")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="device time the timed loops of the headline configuration must add up to")
    ap.add_argument("--ffn-only", default="", metavar="T[,T...]",
                    help="run only the fused expert-FFN section for T tokens (profiling captures)")
    ap.add_argument("--ffn-iters", type=int, default=20)
    ap.add_argument("--e2e-slices", type=int, default=8,
                    help="slices of tensors the end-to-end leg pipelines over its streams (1 = one call per step)")
    ap.add_argument("--ffn-config", default="large", choices=["large", "small"],
                    help="expert shapes of --ffn-only: 8 x 4096->14336->4096 top-2, or 64 x 2048->1408->2048 top-6")
    ap.add_argument("--no-ffn", action="store_true", help="skip the fused expert-FFN section of the report")
    ap.add_argument("--quick", action="store_true",
                    help="one timed loop of the chosen workload and nothing else (profiling captures)")
    ap.add_argument("--max-code-len", type=int, default=0, help="longest Huffman code the encoder may use (8..12)")
    ap.add_argument("--experts", type=int, default=None,
                    help="fewer experts than the configuration names (profiling captures on a small case only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
