#!/usr/bin/env python
"""Benchmark of the ZipMoE decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the decode path over one MoE layer of compressed
expert weights: a single zipmoe_decode launch that decompresses every E-chunk
and re-assembles every bf16 tensor of the layer.  Prints ONE JSON line.

* value      : decoded bf16 GB/s, whole job, compressed inputs resident in HBM.
* e2e        : the same through the C ABI with HOST buffers: compressed streams
               copied host->device from pinned memory, decode, decoded tensors
               copied device->host, all inside the timed region.
* roofline   : algorithmic bytes of one launch (E-chunk section + sign/mantissa
               bytes read + bf16 written) / mean launch duration, against the
               measured HBM copy bandwidth of this machine's B200s.
* cpu_baseline: the CPU oracle (test infrastructure; plain C, bit-by-bit
               decoder), one thread per host core over whole tensors, on a
               bounded sample of the same workload.
* --impl reference: the oracle alone, timed on the host cores.
"""
import argparse
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
def oracle_seconds_per_tensor(blob):
    from oracle import codec
    codec.lib()
    t0 = time.perf_counter()
    codec.decode(blob)
    return max(time.perf_counter() - t0, 1e-4)


def oracle_decode_rate(blobs, n_threads, count):
    """Decodes `count` whole tensors (cycling through blobs) with the CPU oracle on
    n_threads threads (ctypes releases the GIL).  Returns (decoded bf16 GB/s, seconds)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import codec
    sample = [blobs[i % len(blobs)] for i in range(count)]
    t0 = time.perf_counter()
    with ThreadPoolExecutor(min(n_threads, count)) as pool:
        sizes = list(pool.map(lambda b: codec.decode(b).size, sample))
    dt = time.perf_counter() - t0
    return 2.0 * sum(sizes) / dt / 1e9, dt


def run_reference(args):
    """The oracle as it stands, on the host cores; rank 0 only.  Each step decodes a
    bounded sample of the layer, sized so that the whole run stays near two minutes."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2601_21198_b200 import workloads
    cores = os.cpu_count() or 1
    w = workloads.small_layer(n_experts=max(1, min(64, (cores + 2) // 3)), keep_originals=False)
    per = oracle_seconds_per_tensor(w.blobs[0])
    wall_per_step = 120.0 / max(1, args.steps + args.warmup)
    count = int(max(1, min(4 * len(w.blobs), wall_per_step * cores / per)))
    threads = min(cores, count)
    for _ in range(args.warmup):
        oracle_decode_rate(w.blobs, threads, count)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_decode_rate(w.blobs, threads, count)
    dt_all = time.perf_counter() - t0
    value = args.steps * count * 2.0 * 2048 * 1408 / dt_all / 1e9
    sample = "%d tensors (2048x1408 bf16 each, 64K-element chunks) of the 64-expert layer per step" % count
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt_all / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
        "config": {"workload": "moe64_2048x1408_chunk64K (bounded sample)", "chunk_elems": 65536},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


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
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "window": window}


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
        nbytes = sum(expert_bytes[e] for e in active)
        out["T%d" % T] = {"us": us_f, "tokens_per_s": T / us_f * 1e6, "active_experts": len(active),
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
        res = bench_ffn(dev, iters=args.ffn_iters, cpu_tokens=0, token_counts=(args.ffn_only,), config=args.ffn_config)
        print(json.dumps({"ffn": res}))
        return
    w = build_workload(args.workload, keep_originals=False, experts=args.experts, max_code_len=args.max_code_len)
    plan = w.plan
    dplan = plan.to_device(dev)
    out = dplan.new_output()
    stream = torch.cuda.current_stream(dev)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(dev)

    # correctness before timing: status word clean and one tensor equal to what the encoder was given
    dplan.decode(out)
    torch.cuda.synchronize(dev)
    verified = int(dplan.status.item()) == 0
    from paper_2601_21198_b200 import inputs
    probe = inputs.small_expert_tensor(0, 0) if args.workload == "small_layer" else None
    if probe is not None:
        ref = torch.from_numpy(probe.view(np.int16).ravel()).to(dev)
        verified = verified and bool(torch.equal(plan.tensor_slice(out, 0), ref))
        del ref

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        dplan.decode(out)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    for _ in range(args.steps):
        dplan.decode(out)
    e1.record(stream)
    barrier()
    t1 = time.perf_counter()
    ms = e0.elapsed_time(e1)
    clocks = sampler.summary(t0, t1)
    verified = verified and int(dplan.status.item()) == 0

    # end to end: pinned host -> device, decode, device -> pinned host, every step.  The layer is cut into slices of
    # tensors, each with its own zipmoe_decode call, spread over a few streams, so that one slice's copy to the host
    # overlaps the next slice's copy to the device (the host link is full duplex) and its decode.
    n_slices = max(1, min(args.e2e_slices, len(w.blobs)))
    bounds = [len(w.blobs) * i // n_slices for i in range(n_slices + 1)]
    slices = []
    for i in range(n_slices):
        sp = binding.DecodePlan(w.blobs[bounds[i]:bounds[i + 1]])
        sd = sp.to_device(dev)
        slices.append({
            "plan": sp, "dev": sd, "out": sd.new_output(),
            "h": [(sd.payload, torch.from_numpy(sp.payload).pin_memory()), (sd.sm, torch.from_numpy(sp.sm).pin_memory()),
                  (sd.descs, torch.from_numpy(sp.descs.view(np.uint8).copy()).pin_memory()),
                  (sd.tables, torch.from_numpy(sp.tables).pin_memory())],
            "h_out": torch.empty(sp.out_elems, dtype=torch.int16).pin_memory()})
    side = [torch.cuda.Stream(dev) for _ in range(min(3, n_slices))]
    h2d_bytes = sum(h.numel() * h.element_size() for sl in slices for _, h in sl["h"])
    d2h_bytes = sum(sl["h_out"].numel() * 2 for sl in slices)
    e2e_steps = max(1, min(args.steps, 10))

    def e2e_step():
        for i, sl in enumerate(slices):
            st = side[i % len(side)]
            with torch.cuda.stream(st):
                for d_t, h_t in sl["h"]:
                    d_t.copy_(h_t, non_blocking=True)
                sl["dev"].decode(sl["out"], stream=st)
                sl["h_out"].copy_(sl["out"], non_blocking=True)

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
    f0, f1 = e2e_run(e2e_steps)
    barrier()
    e2e_ms = f0.elapsed_time(f1)
    e2e_ok = all(int(sl["dev"].status.item()) == 0 for sl in slices)
    if probe is not None:      # the first tensor of the first slice, as it arrived on the host
        e2e_ok = e2e_ok and bool(np.array_equal(slices[0]["plan"].tensor_slice(slices[0]["h_out"].numpy().view(np.uint16), 0),
                                                probe.ravel()))
    verified = verified and e2e_ok
    sampler.stop_flag = True

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], dev)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        bf16_bytes = w.bf16_bytes()
        per_launch_s = ms / 1e3 / args.steps
        alg = plan.algorithmic_bytes()
        achieved = alg / per_launch_s / 1e9
        line = {
            "metric": METRIC, "value": whole_job_gbs(world, bf16_bytes, args.steps, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_launch_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": w.label, "tensors": len(w.blobs), "elements": w.n_elems,
                       "chunk_elems": int(plan.infos[0].chunk_elems),
                       "max_code_len": int(plan.infos[0].max_code_len), "chunks": plan.n_chunks, "tiles": plan.n_tiles,
                       "compressed_over_bf16": w.compressed_bytes() / bf16_bytes,
                       "l2": "inputs and outputs of one step (%.2f GB) exceed L2; no flush" % (alg / 1e9),
                       "sharding": "every rank decodes its own copy of the layer; no collective"},
            "clocks": clocks,
            "e2e": {"value": whole_job_gbs(world, bf16_bytes, e2e_steps, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": int(h2d_bytes), "d2h_bytes_per_step": int(d2h_bytes), "steps": e2e_steps,
                    "slices": n_slices, "streams": len(side)},
            "gpu_launches": args.steps,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": TRAFFIC_BYTES.get(w.label),
                         "peak_kind": "of " + peak_kind, "algorithmic_bytes_per_launch": alg,
                         "kernel": "zipmoe_dev::decode_kernel", "launch_ms": per_launch_s * 1e3},
            "verified_bit_exact": verified,
        }
        if world == 1:
            # the paper's own GPU step alone (merge of decompressed exponent bytes and SM bytes), same element count
            n = w.n_elems
            d_e = torch.randint(0, 256, (n,), dtype=torch.uint8, device=dev)
            d_s = torch.randint(0, 256, (n,), dtype=torch.uint8, device=dev)
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for it in range(25):
                if it == 5:
                    r0.record(stream)
                binding.zipmoe_recover(d_e, d_s, n, out, stream.cuda_stream)
            r1.record(stream)
            torch.cuda.synchronize(dev)
            rms = r0.elapsed_time(r1) / 20
            line["recover_kernel"] = {"decoded_bf16_gbs": 2 * n / rms / 1e6, "traffic_gbs": 4 * n / rms / 1e6,
                                      "frac_of_peak": 4 * n / rms / 1e6 / peaks["hbm_gbs"], "ms": rms,
                                      "note": "exponent bytes already decompressed: 2 B read + 2 B written per element"}
            del d_e, d_s
        if world == 1:
            # compression states: one stream stays in pinned host memory and is read in place over PCIe
            states = {}
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
        if world == 1 and not args.no_ffn:
            del dplan, out, slices, h_pay, h_sm
            torch.cuda.empty_cache()
            line["ffn"] = bench_ffn(dev)
            line["ffn_small_experts"] = bench_ffn(dev, config="small")
        if world == 1:
            cores = os.cpu_count() or 1
            count = int(max(cores, 20.0 / oracle_seconds_per_tensor(w.blobs[0])))   # ~20 s of CPU work
            rate, dt = oracle_decode_rate(w.blobs, cores, count)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": "%d whole-tensor decodes cycling over the layer's %d tensors, %.1f s wall" % (
                                        count, len(w.blobs), dt)}
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of one decode_kernel launch, from the ncu capture summarised
# under profiles/ (null until a capture of the current kernel exists)
TRAFFIC_BYTES = {
    # 408.0 MB measured on 16 of the 64 experts (profiles/decode_kernel_moe16_2048x1408.md), scaled by 4:
    # traffic grows in proportion to the number of tiles
    "moe64_2048x1408_chunk64K": 4 * 407_956_992,
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="small_layer", choices=["small_layer", "large_layer", "single_matrix", "stress1024", "stress16384", "stress262144"])
    ap.add_argument("--ffn-only", type=int, default=0, metavar="T",
                    help="run only the fused expert-FFN section for T tokens (profiling captures)")
    ap.add_argument("--ffn-iters", type=int, default=20)
    ap.add_argument("--e2e-slices", type=int, default=8,
                    help="slices of tensors the end-to-end leg pipelines over its streams (1 = one call per step)")
    ap.add_argument("--ffn-config", default="large", choices=["large", "small"],
                    help="expert shapes of --ffn-only: 8 x 4096->14336->4096 top-2, or 64 x 2048->1408->2048 top-6")
    ap.add_argument("--no-ffn", action="store_true", help="skip the fused expert-FFN section of the report")
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
