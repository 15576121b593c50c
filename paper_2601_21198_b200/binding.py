"""Thin ctypes binding over the C ABI in include/zipmoe.h.

Every function here has the name of the C entry point it forwards to and does
argument marshalling only (numpy arrays / torch tensors -> pointers and sizes).
`DecodePlan` holds what zipmoe_launch_plan wrote for several blobs (buffers,
descriptors, tables); it computes nothing of the codec or of the layout.

There is no fallback: if the CUDA library has not been built, importing this
module raises.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzipmoe.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "CUDA library %s not found: build it with `python -m paper_2601_21198_b200.build` "
        "(there is no CPU fallback)" % LIB_PATH)

_lib = ctypes.CDLL(LIB_PATH)

DECODE_SHORT_CODES = 1      # zipmoe_decode flag: no code above 8 bits, max_record_bytes exact and <= NARROW_RECORD_BYTES
NARROW_RECORD_BYTES = 2080  # a tile record of 16 rows
OK = 0
ERR_INVALID_ARG, ERR_BAD_FORMAT, ERR_BUFFER_TOO_SMALL, ERR_CUDA, ERR_DECODE_CORRUPT, ERR_UNSUPPORTED = -1, -2, -3, -4, -5, -6
LAYOUT_LINEAR, LAYOUT_BLOCKED = 0, 1
DEVICE_PAD_BYTES = 256

_u64, _u32, _vp, _int = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_int


class EncodeOpts(ctypes.Structure):
    _fields_ = [("chunk_elems", _u32), ("max_code_len", _u32), ("layout", _u32), ("n_threads", _u32)]


class BlobInfo(ctypes.Structure):
    _fields_ = [("n_elems", _u64), ("rows", _u32), ("cols", _u32), ("layout", _u32), ("chunk_elems", _u32),
                ("tile_elems", _u32), ("max_code_len", _u32), ("n_chunks", _u32), ("n_tiles", _u32),
                ("table_off", _u64), ("chunk_off_off", _u64), ("payload_off", _u64), ("payload_bytes", _u64),
                ("sm_off", _u64), ("sm_bytes", _u64), ("total_bytes", _u64)]


CHUNK_DESC_DTYPE = np.dtype([
    ("payload_off", "<u8"), ("sm_off", "<u8"), ("out_off", "<u8"), ("row_pitch", "<u4"), ("tiles_per_rowblk", "<u4"),
    ("tile0", "<u4"), ("n_tiles", "<u4"), ("tile_elems", "<u4"), ("last_tile_elems", "<u4"), ("table_id", "<u4"),
    ("tile_prefix", "<u4"), ("run_first_chunk", "<u4"), ("run_first_tile", "<u4"), ("run_end_tile", "<u4"),
    ("tiles_per_chunk", "<u4"), ("max_record_bytes", "<u4"), ("reserved", "<u4")], align=True)
assert CHUNK_DESC_DTYPE.itemsize == 80
TABLE_BYTES = 256

class CompressedExperts(ctypes.Structure):
    _fields_ = [("n_experts", _u32), ("hidden", _u32), ("inter", _u32), ("n_chunks", _u32), ("chunks", _vp),
                ("tensor_first_chunk", _vp), ("tables", _vp), ("n_tables", _u32), ("reserved", _u32),
                ("payload", _vp), ("payload_bytes", _u64), ("sm", _vp), ("sm_bytes", _u64)]


_lib.zipmoe_version.restype = _u32
_lib.zipmoe_status_string.restype = ctypes.c_char_p
_lib.zipmoe_status_string.argtypes = [_int]
_lib.zipmoe_encode_bound.argtypes = [_u64, _u64, ctypes.POINTER(EncodeOpts), ctypes.POINTER(_u64)]
_lib.zipmoe_encode.argtypes = [_vp, _u64, _u64, ctypes.POINTER(EncodeOpts), _vp, _u64, ctypes.POINTER(_u64)]
_lib.zipmoe_blob_info_get.argtypes = [_vp, _u64, ctypes.POINTER(BlobInfo)]
_lib.zipmoe_blob_validate.argtypes = [_vp, _u64]
_lib.zipmoe_blob_plan.argtypes = [_vp, _u64, _u64, _u64, _u64, _u32, _u32, _u32, _vp, _vp]
_lib.zipmoe_decode.argtypes = [_vp, _u32, _u32, _vp, _u32, _vp, _u64, _vp, _u64, _vp, _u64, _vp, _vp, _u32, _u32]
_lib.zipmoe_recover.argtypes = [_vp, _vp, _u64, _vp, _vp]
_lib.zipmoe_recover.restype = _int
_lib.zipmoe_ffn_workspace_bytes.argtypes = [_u32, _u32, ctypes.POINTER(CompressedExperts), ctypes.POINTER(_u64)]
_lib.zipmoe_decode_expert_ffn.argtypes = [_vp, _u32, _vp, _vp, _u32, ctypes.POINTER(CompressedExperts), _vp, _vp, _u64,
                                          _vp, _vp]
_lib.zipmoe_decode_expert_ffn_noalloc.argtypes = [_vp, _u32, _vp, _vp, _u32, ctypes.POINTER(CompressedExperts), _vp, _vp,
                                                  _vp]
_lib.zipmoe_decode_expert_ffn_noalloc.restype = _int
NOALLOC_SCRATCH_BYTES = 8 << 20
for _f in ("zipmoe_ffn_workspace_bytes", "zipmoe_decode_expert_ffn", "zipmoe_encode_bound", "zipmoe_encode", "zipmoe_blob_info_get", "zipmoe_blob_validate",
           "zipmoe_blob_plan", "zipmoe_decode"):
    getattr(_lib, _f).restype = _int


class ZipMoEError(RuntimeError):
    def __init__(self, where, status):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, zipmoe_status_string(status), status))


def _check(where, status):
    if status != OK:
        raise ZipMoEError(where, status)


def _ptr(a):
    """Address of a numpy array, a torch tensor, an int, or None."""
    if a is None:
        return None
    if isinstance(a, int):
        return a
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()


_lib.zipmoe_test_wait_fault.argtypes = [_u32, _u32]
_lib.zipmoe_test_wait_fault.restype = None


def zipmoe_test_wait_fault(extra_tx_bytes, tries):
    """Test switch: record barriers armed for extra_tx_bytes too many, waits limited to `tries`; (0, 0) = normal."""
    _lib.zipmoe_test_wait_fault(int(extra_tx_bytes), int(tries))


_lib.zipmoe_test_foreign_counter.argtypes = [_u32]
_lib.zipmoe_test_foreign_counter.restype = None


def zipmoe_test_foreign_counter(on):
    """Test switch: dynamically distributed launches find another launch's tag in their work counter; 0 = normal."""
    _lib.zipmoe_test_foreign_counter(int(on))


def zipmoe_version():
    return int(_lib.zipmoe_version())


def zipmoe_status_string(status):
    return _lib.zipmoe_status_string(int(status)).decode()


def _opts(chunk_elems, max_code_len, layout, n_threads):
    return EncodeOpts(int(chunk_elems), int(max_code_len), int(layout), int(n_threads))


def zipmoe_encode_bound(rows, cols, chunk_elems=0, max_code_len=0, layout=LAYOUT_LINEAR, n_threads=0):
    out = _u64(0)
    o = _opts(chunk_elems, max_code_len, layout, n_threads)
    _check("zipmoe_encode_bound", _lib.zipmoe_encode_bound(rows, cols, ctypes.byref(o), ctypes.byref(out)))
    return out.value


def zipmoe_encode(bf16, rows=None, cols=None, chunk_elems=0, max_code_len=0, layout=LAYOUT_LINEAR, n_threads=0):
    """bf16 bit patterns (numpy uint16, row-major) -> blob (numpy uint8)."""
    x = np.ascontiguousarray(bf16, dtype=np.uint16)
    if rows is None:
        rows, cols = (x.shape if x.ndim == 2 else (1, x.size))
    if rows * cols != x.size:
        raise ValueError("rows * cols != number of elements")
    cap = zipmoe_encode_bound(rows, cols, chunk_elems, max_code_len, layout, n_threads)
    blob = np.empty(cap, np.uint8)
    n = _u64(0)
    o = _opts(chunk_elems, max_code_len, layout, n_threads)
    _check("zipmoe_encode", _lib.zipmoe_encode(_ptr(x), rows, cols, ctypes.byref(o), _ptr(blob), cap, ctypes.byref(n)))
    return blob[: n.value].copy()


def zipmoe_blob_info_get(blob):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    info = BlobInfo()
    _check("zipmoe_blob_info_get", _lib.zipmoe_blob_info_get(_ptr(blob), blob.size, ctypes.byref(info)))
    return info


def zipmoe_blob_validate(blob):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    return int(_lib.zipmoe_blob_validate(_ptr(blob), blob.size))


def zipmoe_blob_plan(blob, payload_base, sm_base, out_base, table_id, chunk_base, tile_base):
    """Returns (descs: numpy structured array [n_chunks], table: numpy uint8 [256])."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    info = zipmoe_blob_info_get(blob)
    descs = np.zeros(info.n_chunks, CHUNK_DESC_DTYPE)
    table = np.zeros(TABLE_BYTES, np.uint8)
    _check("zipmoe_blob_plan", _lib.zipmoe_blob_plan(_ptr(blob), blob.size, payload_base, sm_base, out_base, table_id,
                                                     chunk_base, tile_base, _ptr(descs), _ptr(table)))
    return descs, table


def zipmoe_decode(chunks, n_chunks, n_tiles, tables, n_tables, payload, payload_bytes, sm, sm_bytes, out_bf16,
                  out_elems, status_word=None, stream=None, max_record_bytes=0, flags=0):
    """All pointer arguments are device tensors (or raw device addresses)."""
    _check("zipmoe_decode", _lib.zipmoe_decode(_ptr(chunks), n_chunks, n_tiles, _ptr(tables), n_tables, _ptr(payload),
                                                payload_bytes, _ptr(sm), sm_bytes, _ptr(out_bf16), out_elems,
                                                _ptr(status_word), _ptr(stream), int(max_record_bytes), int(flags)))


def zipmoe_recover(exp, sm, n_elems, out_bf16, stream=None):
    """Merge decompressed exponent bytes and sign+mantissa bytes (device tensors) into bf16."""
    _check("zipmoe_recover", _lib.zipmoe_recover(_ptr(exp), _ptr(sm), n_elems, _ptr(out_bf16), _ptr(stream)))


# ---- cache-pool planning (host only) ------------------------------------------------------------
class PlanCosts(ctypes.Structure):
    """zipmoe_plan_costs: delays c (decompress one E-chunk), v (read one E-chunk), u (read one SM-chunk),
    L decompression workers, K E-chunks per tensor, n_tensors per expert."""
    _fields_ = [("c", ctypes.c_double), ("v", ctypes.c_double), ("u", ctypes.c_double), ("L", _u32), ("K", _u32),
                ("n_tensors", _u32)]


_dp = ctypes.POINTER(ctypes.c_double)
_lib.zipmoe_plan_hit_distribution.argtypes = [_dp, _u32, _dp]
_lib.zipmoe_plan_selection_probs.argtypes = [_dp, _u32, _u32, _u32, ctypes.c_double, _dp, ctypes.POINTER(_u32)]
_lib.zipmoe_plan_makespan.argtypes = [_u32, ctypes.POINTER(_u32), ctypes.POINTER(PlanCosts), _dp]
_lib.zipmoe_plan_expected_makespan.argtypes = [_dp, _u32, _u32, ctypes.POINTER(_u32), ctypes.POINTER(PlanCosts), _dp]
_lib.zipmoe_plan_cache_pools.argtypes = [_dp, _u32, _u32, _u32, ctypes.c_double, _dp, ctypes.POINTER(PlanCosts),
                                         ctypes.c_double, _dp, ctypes.POINTER(_u32), _dp]
for _f in ("zipmoe_plan_hit_distribution", "zipmoe_plan_selection_probs", "zipmoe_plan_makespan",
           "zipmoe_plan_expected_makespan", "zipmoe_plan_cache_pools"):
    getattr(_lib, _f).restype = _int


def _dbl(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_dp)


def _u32x4(v):
    return (_u32 * 4)(*[int(x) for x in v])


def zipmoe_plan_hit_distribution(q):
    q, qp = _dbl(q)
    phi = np.zeros(q.size + 1)
    _check("zipmoe_plan_hit_distribution", _lib.zipmoe_plan_hit_distribution(qp, q.size, phi.ctypes.data_as(_dp)))
    return phi


def zipmoe_plan_selection_probs(f, k, max_iters=1000, tol=1e-12):
    f, fp = _dbl(f)
    q = np.zeros(f.size)
    it = _u32(0)
    _check("zipmoe_plan_selection_probs",
           _lib.zipmoe_plan_selection_probs(fp, f.size, k, max_iters, tol, q.ctypes.data_as(_dp), ctypes.byref(it)))
    return q, int(it.value)


def zipmoe_plan_makespan(k, hits, costs):
    out = ctypes.c_double(0)
    _check("zipmoe_plan_makespan", _lib.zipmoe_plan_makespan(k, _u32x4(hits), ctypes.byref(costs), ctypes.byref(out)))
    return out.value


def zipmoe_plan_expected_makespan(q, k, capacity, costs):
    q, qp = _dbl(q)
    out = ctypes.c_double(0)
    _check("zipmoe_plan_expected_makespan",
           _lib.zipmoe_plan_expected_makespan(qp, q.size, k, _u32x4(capacity), ctypes.byref(costs), ctypes.byref(out)))
    return out.value


def zipmoe_plan_cache_pools(f, k, pool_mask, budget, expert_size, costs, step):
    """Returns (ratios[4], capacity[4], expected makespan)."""
    f, fp = _dbl(f)
    size, sp = _dbl(expert_size)
    ratios = np.zeros(4)
    cap = (_u32 * 4)()
    out = ctypes.c_double(0)
    _check("zipmoe_plan_cache_pools",
           _lib.zipmoe_plan_cache_pools(fp, f.size, k, pool_mask, budget, sp, ctypes.byref(costs), step,
                                        ratios.ctypes.data_as(_dp), cap, ctypes.byref(out)))
    return ratios, [int(c) for c in cap], out.value


# ---- cache-affinity scheduling (host only) --------------------------------------------------------
class SchedTask(ctypes.Structure):
    _fields_ = [("expert", _u32), ("state", _u32)]


class SchedCosts(ctypes.Structure):
    _fields_ = [("c", ctypes.c_double), ("u", ctypes.c_double), ("rho", ctypes.c_double), ("K", _u32), ("L", _u32)]


SCHED_STATES = {"M": 0, "C": 1, "S": 2, "E": 3}
_lib.zipmoe_plan_simulate.argtypes = [ctypes.POINTER(SchedTask), _u32, _dp, _u32, ctypes.POINTER(SchedCosts),
                                      ctypes.POINTER(_u32), ctypes.POINTER(_u32), _dp, _dp]
_lib.zipmoe_plan_schedule.argtypes = [ctypes.POINTER(SchedTask), _u32, _dp, _u32, ctypes.POINTER(SchedCosts),
                                      ctypes.POINTER(_u32), ctypes.POINTER(_u32), ctypes.POINTER(_u32), _dp]
_lib.zipmoe_plan_simulate.restype = _int
_lib.zipmoe_plan_schedule.restype = _int


def _sched_args(tasks, p, costs):
    arr = (SchedTask * len(tasks))(*[SchedTask(int(n), SCHED_STATES[s] if isinstance(s, str) else int(s)) for n, s in tasks])
    pv, pp = _dbl(p)
    return arr, pv, pp, SchedCosts(*costs)


def zipmoe_plan_simulate(tasks, p, costs, blocks):
    """tasks: [(expert, state)], p: expert times, costs: (c, u, rho, K, L), blocks: lists of task indices.
    Returns (makespan, charge)."""
    arr, pv, pp, cs = _sched_args(tasks, p, costs)
    order = [j for B in blocks for j in B]
    block_of = [b for b, B in enumerate(blocks) for _ in B]
    n = len(tasks)
    mk, ch = ctypes.c_double(0), ctypes.c_double(0)
    _check("zipmoe_plan_simulate",
           _lib.zipmoe_plan_simulate(arr, n, pp, pv.size, ctypes.byref(cs), (_u32 * n)(*order), (_u32 * n)(*block_of),
                                     ctypes.byref(mk), ctypes.byref(ch)))
    return mk.value, ch.value


def zipmoe_plan_schedule(tasks, p, costs):
    """Returns (blocks: lists of task indices in priority order, makespan)."""
    arr, pv, pp, cs = _sched_args(tasks, p, costs)
    n = len(tasks)
    order, block_of, nb, mk = (_u32 * n)(), (_u32 * n)(), _u32(0), ctypes.c_double(0)
    _check("zipmoe_plan_schedule",
           _lib.zipmoe_plan_schedule(arr, n, pp, pv.size, ctypes.byref(cs), order, block_of, ctypes.byref(nb),
                                     ctypes.byref(mk)))
    blocks = [[] for _ in range(nb.value)]
    for j, b in zip(order, block_of):
        blocks[b].append(int(j))
    return blocks, mk.value


def zipmoe_ffn_workspace_bytes(T, k, experts):
    out = _u64(0)
    _check("zipmoe_ffn_workspace_bytes", _lib.zipmoe_ffn_workspace_bytes(T, k, ctypes.byref(experts), ctypes.byref(out)))
    return out.value


def zipmoe_decode_expert_ffn(tokens, T, topk_ids, topk_weights, k, experts, out, workspace, workspace_bytes,
                             status_word=None, stream=None):
    """Pointer arguments are device tensors (or raw device addresses); `experts` is a CompressedExperts."""
    _check("zipmoe_decode_expert_ffn",
           _lib.zipmoe_decode_expert_ffn(_ptr(tokens), T, _ptr(topk_ids), _ptr(topk_weights), k, ctypes.byref(experts),
                                         _ptr(out), _ptr(workspace), workspace_bytes, _ptr(status_word), _ptr(stream)))


def zipmoe_decode_expert_ffn_noalloc(tokens, T, topk_ids, topk_weights, k, experts, out, status_word=None, stream=None):
    """zipmoe_decode_expert_ffn without a workspace argument: the library's built-in scratch is used, so the
    caller (and this binding) allocates nothing.  Raises ZipMoEError(ERR_BUFFER_TOO_SMALL) when the call needs
    more than NOALLOC_SCRATCH_BYTES of scratch."""
    _check("zipmoe_decode_expert_ffn_noalloc",
           _lib.zipmoe_decode_expert_ffn_noalloc(_ptr(tokens), T, _ptr(topk_ids), _ptr(topk_weights), k,
                                                 ctypes.byref(experts), _ptr(out), _ptr(status_word), _ptr(stream)))


class LaunchInfo(ctypes.Structure):
    _fields_ = [("payload_bytes", _u64), ("sm_bytes", _u64), ("out_elems", _u64), ("n_chunks", _u32), ("n_tiles", _u32),
                ("n_tables", _u32), ("max_record_bytes", _u32), ("max_code_len", _u32), ("flags", _u32)]


_lib.zipmoe_launch_plan_size.argtypes = [ctypes.POINTER(_vp), ctypes.POINTER(_u64), _u32, ctypes.POINTER(LaunchInfo)]
_lib.zipmoe_launch_plan.argtypes = [ctypes.POINTER(_vp), ctypes.POINTER(_u64), _u32, _vp, _vp, _vp, _vp, _vp, _vp,
                                    ctypes.POINTER(LaunchInfo)]
_lib.zipmoe_launch_plan_size.restype = _int
_lib.zipmoe_launch_plan.restype = _int


class DecodePlan:
    """One decode launch over several blobs, as zipmoe_launch_plan lays it out: the three contiguous host
    buffers, the chunk descriptors and the tables.  Marshalling only: the layout is the library's."""

    def __init__(self, blobs):
        blobs = [np.ascontiguousarray(b, dtype=np.uint8) for b in blobs]
        n = len(blobs)
        ptrs = (_vp * max(n, 1))(*[b.ctypes.data for b in blobs])
        sizes = (_u64 * max(n, 1))(*[b.size for b in blobs])
        info = LaunchInfo()
        _check("zipmoe_launch_plan_size", _lib.zipmoe_launch_plan_size(ptrs, sizes, n, ctypes.byref(info)))
        self.payload = np.empty(info.payload_bytes + DEVICE_PAD_BYTES, np.uint8)
        self.sm = np.empty(info.sm_bytes + DEVICE_PAD_BYTES, np.uint8)
        self.descs = np.zeros(info.n_chunks, CHUNK_DESC_DTYPE)
        self.tables = np.zeros(n * TABLE_BYTES, np.uint8)
        self.tensor_first_chunk = np.zeros(n, np.uint32)
        out_base = np.zeros(n, np.uint64)
        _check("zipmoe_launch_plan",
               _lib.zipmoe_launch_plan(ptrs, sizes, n, _ptr(self.payload), _ptr(self.sm), _ptr(self.descs),
                                       _ptr(self.tables), _ptr(self.tensor_first_chunk), _ptr(out_base), ctypes.byref(info)))
        self.infos = [zipmoe_blob_info_get(b) for b in blobs]
        self.out_base = [int(v) for v in out_base]
        self.payload_base = [int(self.descs["payload_off"][int(c)]) if inf.n_chunks else 0
                             for c, inf in zip(self.tensor_first_chunk, self.infos)]
        self.sm_base = [int(self.descs["sm_off"][int(c)]) if inf.n_chunks else 0
                        for c, inf in zip(self.tensor_first_chunk, self.infos)]
        self.payload_bytes, self.sm_bytes, self.out_elems = info.payload_bytes, info.sm_bytes, info.out_elems
        self.n_chunks, self.n_tiles, self.n_tables = info.n_chunks, info.n_tiles, info.n_tables
        self.max_record_bytes, self.max_code_len, self.flags = info.max_record_bytes, info.max_code_len, info.flags

    def algorithmic_bytes(self):
        """Bytes one decode must move: E-chunk section + SM bytes read, bf16 written."""
        n = sum(inf.n_elems for inf in self.infos)
        return self.payload_bytes + n + 2 * n

    def to_device(self, device="cuda"):
        import torch
        return DevicePlan(self, torch.device(device))

    def tensor_slice(self, out, i):
        inf = self.infos[i]
        return out[self.out_base[i]: self.out_base[i] + inf.n_elems]


class DevicePlan:
    """Device copies of a DecodePlan's buffers (torch owns the memory)."""

    def __init__(self, plan, device):
        import torch
        self.plan = plan
        self.device = device
        self.descs = torch.from_numpy(plan.descs.view(np.uint8).copy()).to(device)
        self.tables = torch.from_numpy(plan.tables).to(device)
        self.payload = torch.from_numpy(plan.payload).to(device)
        self.sm = torch.from_numpy(plan.sm).to(device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def new_output(self):
        import torch
        return torch.zeros(self.plan.out_elems, dtype=torch.int16, device=self.device)

    def decode(self, out, stream=None):
        """One zipmoe_decode launch on `stream` (a torch stream or None = current)."""
        import torch
        p = self.plan
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        zipmoe_decode(self.descs, p.n_chunks, p.n_tiles, self.tables, p.n_tables, self.payload, p.payload_bytes,
                      self.sm, p.sm_bytes, out, p.out_elems, self.status, s.cuda_stream, p.max_record_bytes, p.flags)


def pad_expert_inter(w1, w3, w2, multiple=256):
    """The fused expert FFN takes experts whose hidden and intermediate sizes are multiples of 256.  An expert with
    another intermediate size (w1, w3 [inter, hidden]; w2 [hidden, inter], uint16 bf16 patterns) is padded with zero
    rows (w1, w3) and zero columns (w2) up to the next multiple: the added units compute SiLU(0) * 0 = 0 and feed
    zero weights, so the FFN's result is unchanged.  Returns (w1, w3, w2, padded inter)."""
    inter, hidden = w1.shape
    assert w3.shape == (inter, hidden) and w2.shape == (hidden, inter)
    padded = -(-inter // multiple) * multiple
    if padded == inter:
        return w1, w3, w2, inter
    a = np.zeros((padded, hidden), np.uint16)
    b = np.zeros((padded, hidden), np.uint16)
    c = np.zeros((hidden, padded), np.uint16)
    a[:inter], b[:inter], c[:, :inter] = w1, w3, w2
    return a, b, c, padded


class DeviceExperts:
    """The compressed experts of one layer on the device: blobs[3*e + j] (j: 0 w1, 1 w3, 2 w2, blocked
    layout) laid out by DecodePlan, plus the CompressedExperts struct the fused call takes."""

    def __init__(self, blobs, hidden, inter, device="cuda"):
        import torch
        assert len(blobs) % 3 == 0
        self.plan = DecodePlan(blobs)
        self.dev = self.plan.to_device(device)
        self.tensor_first_chunk = torch.from_numpy(self.plan.tensor_first_chunk.view(np.int32).copy()).to(self.dev.device)
        p, d = self.plan, self.dev
        self.struct = CompressedExperts(len(blobs) // 3, hidden, inter, p.n_chunks, d.descs.data_ptr(),
                                        self.tensor_first_chunk.data_ptr(), d.tables.data_ptr(), p.n_tables, 0,
                                        d.payload.data_ptr(), p.payload_bytes, d.sm.data_ptr(), p.sm_bytes)
        self.hidden, self.inter = hidden, inter
        self._ws = {}

    def ffn(self, tokens, topk_ids, topk_weights, out=None, stream=None):
        """tokens [T, hidden] int16 (bf16 patterns), topk_ids [T, k] int32, topk_weights [T, k] float32 or None:
        device tensors.  Returns out [T, hidden] int16."""
        import torch
        T, k = topk_ids.shape
        key = (T, k)
        if key not in self._ws:
            n = zipmoe_ffn_workspace_bytes(T, k, self.struct)
            self._ws[key] = torch.empty(n, dtype=torch.uint8, device=self.dev.device)
        ws = self._ws[key]
        if out is None:
            out = torch.empty(T, self.hidden, dtype=torch.int16, device=self.dev.device)
        s = torch.cuda.current_stream(self.dev.device) if stream is None else stream
        zipmoe_decode_expert_ffn(tokens, T, topk_ids, topk_weights, k, self.struct, out, ws, ws.numel(),
                                 self.dev.status, s.cuda_stream)
        return out
