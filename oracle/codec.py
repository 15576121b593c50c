"""ctypes access to the C oracle (oracle/zipmoe_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It holds no arithmetic
of its own: every function forwards to the C oracle, which is compiled with
gcc on first use.  Nothing here touches the CUDA library.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zipmoe_oracle.c")
_LIB = os.path.join(_HERE, "libzipmoe_oracle.so")

OK = 0


def build(force=False):
    """Compile the C oracle into oracle/libzipmoe_oracle.so (gcc -O2)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, u32, vp, ci = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p, ctypes.c_int
        L.zo_split.argtypes = [vp, u64, vp, vp]
        L.zo_split.restype = None
        L.zo_merge.argtypes = [vp, vp, u64, vp]
        L.zo_merge.restype = None
        L.zo_histogram.argtypes = [vp, u64, vp]
        L.zo_histogram.restype = None
        L.zo_code_lengths.argtypes = [vp, ci, vp]
        L.zo_code_lengths.restype = ci
        L.zo_canonical_codes.argtypes = [vp, vp]
        L.zo_canonical_codes.restype = ci
        L.zo_encode_bound.argtypes = [u64, u64, u32, u32]
        L.zo_encode_bound.restype = u64
        L.zo_encode.argtypes = [vp, u64, u64, u32, u32, ci, vp, u64, ctypes.POINTER(u64)]
        L.zo_encode.restype = ci
        L.zo_decode_chunk.argtypes = [vp, u64, u32, vp]
        L.zo_decode_chunk.restype = ci
        L.zo_decode.argtypes = [vp, u64, vp]
        L.zo_decode.restype = ci
        L.zo_info.argtypes = [vp, u64, vp]
        L.zo_info.restype = ci
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def split(x):
    x = np.ascontiguousarray(x, dtype=np.uint16).ravel()
    e = np.empty(x.size, np.uint8)
    s = np.empty(x.size, np.uint8)
    lib().zo_split(_p(x), x.size, _p(e), _p(s))
    return e, s


def merge(e, s):
    e = np.ascontiguousarray(e, dtype=np.uint8).ravel()
    s = np.ascontiguousarray(s, dtype=np.uint8).ravel()
    assert e.size == s.size
    x = np.empty(e.size, np.uint16)
    lib().zo_merge(_p(e), _p(s), e.size, _p(x))
    return x


def histogram(e):
    e = np.ascontiguousarray(e, dtype=np.uint8).ravel()
    h = np.zeros(256, np.uint64)
    lib().zo_histogram(_p(e), e.size, _p(h))
    return h


def code_lengths(hist, max_len=12):
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    assert hist.size == 256
    out = np.zeros(256, np.uint8)
    rc = lib().zo_code_lengths(_p(hist), int(max_len), _p(out))
    if rc != OK:
        raise ValueError("zo_code_lengths failed: %d" % rc)
    return out


def canonical_codes(lengths):
    lengths = np.ascontiguousarray(lengths, dtype=np.uint8)
    assert lengths.size == 256
    out = np.zeros(256, np.uint32)
    rc = lib().zo_canonical_codes(_p(lengths), _p(out))
    if rc != OK:
        raise ValueError("zo_canonical_codes failed: %d" % rc)
    return out


def encode(x, rows=None, cols=None, layout=0, chunk_elems=4096, max_code_len=12):
    """bf16 bit patterns (uint16) -> ZMOE v2 blob (uint8 array)."""
    x = np.ascontiguousarray(x, dtype=np.uint16)
    if rows is None:
        rows, cols = (x.shape if x.ndim == 2 else (1, x.size))
    assert rows * cols == x.size
    cap = lib().zo_encode_bound(rows, cols, layout, chunk_elems)
    if cap == 0:
        raise ValueError("bad geometry")
    blob = np.zeros(cap, np.uint8)
    n = ctypes.c_uint64(0)
    rc = lib().zo_encode(_p(x), rows, cols, layout, chunk_elems, max_code_len, _p(blob), cap, ctypes.byref(n))
    if rc != OK:
        raise ValueError("zo_encode failed: %d" % rc)
    return blob[: n.value].copy()


def info(blob):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    v = np.zeros(12, np.uint64)
    rc = lib().zo_info(_p(blob), blob.size, _p(v))
    if rc != OK:
        raise ValueError("zo_info failed: %d" % rc)
    keys = ["n_elems", "rows", "cols", "layout", "chunk_elems", "tile_elems", "max_code_len", "n_chunks",
            "n_tiles", "payload_bytes", "sm_bytes", "payload_off"]
    return {k: int(x) for k, x in zip(keys, v)}


def decode(blob):
    """ZMOE v2 blob -> bf16 bit patterns (uint16, flat, row-major)."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    n = info(blob)["n_elems"]
    out = np.zeros(n, np.uint16)
    rc = lib().zo_decode(_p(blob), blob.size, _p(out))
    if rc != OK:
        raise ValueError("zo_decode failed: %d" % rc)
    return out


def decode_chunk(blob, k, out):
    """Decode chunk k alone into its place in `out` (uint16, n_elems)."""
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    assert out.dtype == np.uint16 and out.flags.c_contiguous
    rc = lib().zo_decode_chunk(_p(blob), blob.size, int(k), _p(out))
    if rc != OK:
        raise ValueError("zo_decode_chunk failed: %d" % rc)
    return out
