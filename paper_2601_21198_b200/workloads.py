"""The benchmark workloads: seeded synthetic expert tensors (inputs.py) encoded
with zipmoe_encode and laid out for one decode launch.  Used by bench.py and by
the GPU parity tests so that both run the same launch configuration."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from . import binding, inputs


def host_threads():
    return max(1, min(32, (os.cpu_count() or 1)))


def _encode_all(named_tensors, chunk_elems, layout, keep_originals, max_code_len=0):
    """named_tensors: iterable of (name, thunk -> uint16 array).  Tensors are
    drawn and encoded on a small thread pool (numpy and the encoder release the
    GIL); returns (names, blobs, originals or None)."""
    items = list(named_tensors)
    nt = host_threads()
    outer = max(1, min(len(items), nt // 2 if len(items) > 1 else 1))
    inner = max(1, nt // outer)

    def work(item):
        name, thunk = item
        x = thunk()
        rows, cols = (x.shape if x.ndim == 2 else (1, x.size))
        lay = layout if (layout == binding.LAYOUT_LINEAR or (rows % 16 == 0 and cols % 256 == 0)) else 0
        blob = binding.zipmoe_encode(x, rows, cols, chunk_elems=chunk_elems, layout=lay, n_threads=inner,
                                     max_code_len=max_code_len)
        return name, blob, (x if keep_originals else None)

    with ThreadPoolExecutor(outer) as pool:
        res = list(pool.map(work, items))
    names = [r[0] for r in res]
    blobs = [r[1] for r in res]
    originals = [r[2] for r in res] if keep_originals else None
    return names, blobs, originals


class Workload:
    def __init__(self, label, names, blobs, originals):
        self.label = label
        self.names = names
        self.blobs = blobs
        self.originals = originals
        self.plan = binding.DecodePlan(blobs)
        self.n_elems = sum(i.n_elems for i in self.plan.infos)

    def bf16_bytes(self):
        return 2 * self.n_elems

    def compressed_bytes(self):
        return sum(b.size for b in self.blobs)


def single_matrix(keep_originals=True, max_code_len=0):
    """One 2048x1408 expert matrix, 4096-element chunks."""
    items = [("expert0", lambda: inputs.single_expert_matrix(0))]
    return Workload("single_2048x1408_chunk4096", *_encode_all(items, 4096, 0, keep_originals, max_code_len))


def small_layer(n_experts=64, keep_originals=True, layout=0, max_code_len=0):
    """64 experts x {gate, up [1408,2048]; down [2048,1408]}, 64K-element chunks (~1.1 GB bf16)."""
    items = []
    for e in range(n_experts):
        for j, (name, _) in enumerate(inputs.SMALL_EXPERT_TENSORS):
            items.append(("e%d.%s" % (e, name), lambda e=e, j=j: inputs.small_expert_tensor(e, j)))
    return Workload("moe%d_2048x1408_chunk64K" % n_experts, *_encode_all(items, 65536, layout, keep_originals, max_code_len))


def small_layer_ffn(n_experts=64, keep_originals=True, max_code_len=0):
    """The 64-expert layer for the fused FFN: every expert's intermediate size 1408 is padded to 1536 with zero
    units (binding.pad_expert_inter) and its three matrices are encoded with the blocked layout.  `originals`
    keeps the unpadded matrices; `inter` is the padded size."""
    def padded(e, j):
        ws = [inputs.small_expert_tensor(e, t) for t in range(3)]
        return binding.pad_expert_inter(*ws)[j]

    items = []
    for e in range(n_experts):
        for j, (name, _) in enumerate(inputs.SMALL_EXPERT_TENSORS):
            items.append(("e%d.%s" % (e, name), lambda e=e, j=j: padded(e, j)))
    w = Workload("moe%d_ffn_2048x1408_pad1536" % n_experts,
                 *_encode_all(items, 65536, binding.LAYOUT_BLOCKED, False, max_code_len))
    w.hidden, w.inter = 2048, 1536
    if keep_originals:
        w.originals = [inputs.small_expert_tensor(e, j) for e in range(n_experts) for j in range(3)]
    return w


def large_layer(n_experts=8, keep_originals=True, layout=0, hidden=4096, inter=14336, chunk_elems=262144,
                max_code_len=0):
    """8 experts x {w1, w3 [14336,4096]; w2 [4096,14336]} with outlier channels, 256K-element chunks (~2.8 GB bf16)."""
    items = []
    for e in range(n_experts):
        for j, name in enumerate(inputs.LARGE_EXPERT_TENSORS):
            items.append(("e%d.%s" % (e, name),
                          lambda e=e, j=j: inputs.large_expert_tensor(e, j, hidden=hidden, inter=inter)))
    label = "moe%d_%dx%d_chunk%dK" % (n_experts, inter, hidden, chunk_elems // 1024)
    return Workload(label, *_encode_all(items, chunk_elems, layout, keep_originals, max_code_len))


def stress_set(n_tensors=4096, chunk_elems=None, keep_originals=True, max_elems=4 << 20):
    """Codec stress tensors; with chunk_elems given, only the tensors of that chunk size."""
    items = []
    for i in range(n_tensors):
        fam = inputs.STRESS_FAMILIES[i % 4]
        chunk = inputs.STRESS_CHUNKS[(i // 4) % 3]
        if chunk_elems is not None and chunk != chunk_elems:
            continue
        items.append(("t%d.%s.c%d" % (i, fam, chunk), (i, chunk)))
    groups = {}
    for name, (i, chunk) in items:
        groups.setdefault(chunk, []).append((name, (lambda i=i: inputs.stress_tensor(i, max_elems=max_elems)[0])))
    out = []
    for chunk, its in sorted(groups.items()):
        out.append(Workload("stress_chunk%d" % chunk, *_encode_all(its, chunk, 0, keep_originals)))
    return out
