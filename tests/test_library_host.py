"""Host side of the CUDA library without a GPU: the shared object loads and
exports every symbol the header declares; its encoder's blobs are decoded by
the oracle and the oracle's blobs pass its validator; the planner's
descriptors are consistent with the container."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import codec
from paper_2601_21198_b200 import build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(zb):
    header = open(os.path.join(ROOT, "include", "zipmoe.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(zipmoe_[a-z_0-9]+)\s*\(", header))
    assert {"zipmoe_encode", "zipmoe_decode", "zipmoe_blob_plan", "zipmoe_blob_validate"} <= names
    lib = ctypes.CDLL(zb.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), n
    assert zb.zipmoe_version() >= 100
    assert zb.zipmoe_status_string(0) == "ok" and "argument" in zb.zipmoe_status_string(-1)


def test_struct_layouts_match_the_header(zb):
    assert zb.CHUNK_DESC_DTYPE.itemsize == 80
    assert zb.CHUNK_DESC_DTYPE.fields["row_pitch"][1] == 24
    assert zb.CHUNK_DESC_DTYPE.fields["tiles_per_chunk"][1] == 68
    assert ctypes.sizeof(zb.BlobInfo) == 96


CASES = [
    (1, 1, 0, 256), (1, 7, 0, 256), (1, 255, 0, 256), (1, 257, 0, 1024), (3, 1000, 0, 1024), (1, 4096, 0, 4096),
    (1, 4097, 0, 4096), (5, 4099, 0, 16384), (64, 1408, 0, 4096), (100, 1408, 0, 65536), (16, 256, 1, 4096),
    (48, 768, 1, 8192), (32, 4096, 1, 65536), (16, 14336, 1, 262144),
]


@pytest.mark.parametrize("rows,cols,layout,chunk", CASES)
def test_library_blobs_are_decoded_by_the_oracle(zb, rows, cols, layout, chunk):
    x = inputs.gaussian((rows, cols), 0.02, rows * 31 + cols)
    blob = zb.zipmoe_encode(x, layout=layout, chunk_elems=chunk, n_threads=3)
    assert zb.zipmoe_blob_validate(blob) == zb.OK
    assert np.array_equal(codec.decode(blob), x.ravel())
    info = zb.zipmoe_blob_info_get(blob)
    o = codec.info(blob)
    assert (info.n_chunks, info.n_tiles, info.payload_bytes, info.sm_bytes) == \
           (o["n_chunks"], o["n_tiles"], o["payload_bytes"], o["sm_bytes"])
    assert info.total_bytes == blob.size


@pytest.mark.parametrize("rows,cols,layout,chunk", CASES[:12])
def test_oracle_blobs_pass_the_library_validator(zb, rows, cols, layout, chunk):
    x = inputs.gaussian((rows, cols), 0.02, rows * 37 + cols)
    blob = codec.encode(x, layout=layout, chunk_elems=chunk)
    assert zb.zipmoe_blob_validate(blob) == zb.OK
    # same sign+mantissa section from both encoders (that section has no freedom)
    mine = zb.zipmoe_encode(x, layout=layout, chunk_elems=chunk)
    a, b = zb.zipmoe_blob_info_get(blob), zb.zipmoe_blob_info_get(mine)
    assert np.array_equal(blob[a.sm_off: a.sm_off + a.sm_bytes], mine[b.sm_off: b.sm_off + b.sm_bytes])


def test_library_encoder_on_stress_families_specials_and_length_limits(zb):
    for idx in range(8):
        x, fam, chunk = inputs.stress_tensor(idx, max_elems=40000)
        for mcl in (0, 12, 10):
            blob = zb.zipmoe_encode(x, chunk_elems=chunk, max_code_len=mcl)
            assert zb.zipmoe_blob_validate(blob) == zb.OK
            assert blob[64:320].max() <= (mcl or 8)
            assert np.array_equal(codec.decode(blob), x), (fam, mcl)
    allp = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    assert np.array_equal(codec.decode(zb.zipmoe_encode(allp, chunk_elems=1024)), allp)
    empty = zb.zipmoe_encode(np.zeros(0, np.uint16), rows=0, cols=0)
    assert zb.zipmoe_blob_validate(empty) == zb.OK and codec.decode(empty).size == 0
    one = np.full(777, 0x3F80, np.uint16)
    assert np.array_equal(codec.decode(zb.zipmoe_encode(one, chunk_elems=256)), one)


def test_library_code_is_close_to_optimal(zb):
    x = inputs.single_expert_matrix(0)
    mine = zb.zipmoe_encode(x, chunk_elems=4096, n_threads=4, max_code_len=12)
    ref = codec.encode(x, chunk_elems=4096)
    hist = codec.histogram(codec.split(x)[0])
    cost_mine = int((hist * mine[64:320]).sum())
    cost_ref = int((hist * ref[64:320]).sum())
    assert cost_ref <= cost_mine <= cost_ref * 1.002      # the oracle's code is optimal under the limit
    assert mine.size / (2 * x.size) < 0.68


def test_bad_arguments_and_corrupt_blobs(zb):
    x = inputs.gaussian((10, 300), 0.02, 1)
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_encode(x, chunk_elems=1000)                   # not a multiple of 256
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_encode(x, chunk_elems=8192 + 256)             # above 4096 but not a multiple of 4096
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_encode(x, layout=1, chunk_elems=4096)         # blocked layout needs rows % 16, cols % 256
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_encode(x, max_code_len=7)
    blob = zb.zipmoe_encode(x, chunk_elems=1024)
    info = zb.zipmoe_blob_info_get(blob)
    for at, val in [(0, 0), (36, 13), (64 + int(np.flatnonzero(blob[64:320])[0]), 0), (328, blob[328] ^ 0x10),
                    (info.payload_off + 4, blob[info.payload_off + 4] + 1),
                    (info.payload_off + 17, 0xFF),             # a column that does not exist
                    (info.payload_off + 18, blob[info.payload_off + 19])]:   # two backward streams in one column
        b = blob.copy()
        b[at] = val
        assert zb.zipmoe_blob_validate(b) == zb.ERR_BAD_FORMAT, at
    assert zb.zipmoe_blob_validate(blob[:-1]) == zb.ERR_BAD_FORMAT


def test_random_corruptions_are_rejected_or_decode_in_bounds(zb):
    """Random byte damage anywhere in a blob: the validator either rejects it, or the blob is still structurally
    sound, in which case the oracle decodes it (to other data) or reports the damage itself -- never a crash.
    Damage to the header, the code table, the chunk offsets or a tile table must never pass the validator
    unnoticed when it changes the structure."""
    from oracle import codec
    x = inputs.stress_tensor(1, max_elems=30000)[0]
    blob = zb.zipmoe_encode(x, chunk_elems=1024)
    info = zb.zipmoe_blob_info_get(blob)
    rng = np.random.default_rng(17)
    accepted = rejected = 0
    for trial in range(400):
        b = blob.copy()
        region = trial % 4       # header + table, chunk offsets, payload, anywhere
        lo, hi = [(0, 320), (320, info.payload_off), (info.payload_off, info.sm_off), (0, b.size)][region]
        for _ in range(1 + trial % 3):
            at = int(rng.integers(lo, hi))
            b[at] ^= np.uint8(1 << int(rng.integers(0, 8)))
        if zb.zipmoe_blob_validate(b) != zb.OK:
            rejected += 1
            continue
        accepted += 1
        try:
            y = codec.decode(b)
            assert y.size == x.size
        except ValueError:
            pass
    assert accepted > 20 and rejected > 100, (accepted, rejected)


def test_plan_descriptors(zb):
    a = inputs.gaussian((5, 4099), 0.02, 3)          # linear, 2 chunks of 16384, short last tile
    b = inputs.gaussian((32, 512), 0.02, 4)          # blocked, 4 tiles, chunks of 8192 (2 tiles)
    blobs = [zb.zipmoe_encode(a, chunk_elems=16384), zb.zipmoe_encode(b, layout=1, chunk_elems=8192)]
    plan = zb.DecodePlan(blobs)
    d = plan.descs
    assert plan.n_chunks == 4 and plan.n_tiles == 6 + 4 and plan.n_tables == 2
    assert d["tile_prefix"].tolist() == [0, 4, 6, 8]
    assert d["n_tiles"].tolist() == [4, 2, 2, 2]
    assert d["table_id"].tolist() == [0, 0, 1, 1]
    assert d["run_first_chunk"].tolist() == [0, 0, 2, 2] and d["run_end_tile"].tolist() == [6, 6, 10, 10]
    assert d["last_tile_elems"].tolist() == [4096, 5 * 4099 - 5 * 4096, 4096, 4096]
    assert d["row_pitch"].tolist() == [256, 256, 512, 512] and d["tiles_per_rowblk"].tolist() == [1, 1, 2, 2]
    assert d["out_off"].tolist() == [0, 0, plan.out_base[1], plan.out_base[1]] and plan.out_base[1] % 8 == 0
    assert d["sm_off"].tolist() == [0, 16384, plan.sm_base[1], plan.sm_base[1] + 8192]
    assert (d["payload_off"] % 16 == 0).all() and d["payload_off"][2] == plan.payload_base[1]
    assert plan.payload.size == plan.payload_bytes + zb.DEVICE_PAD_BYTES
    assert plan.algorithmic_bytes() == plan.payload_bytes + 3 * (a.size + b.size)


def test_ffn_planning_on_the_host(zb):
    """zipmoe_ffn_workspace_bytes needs no GPU: limits and sizes of the fused call."""
    ok = zb.CompressedExperts(8, 4096, 14336, 1, 16, 16, 16, 1, 0, 16, 0, 16, 0)
    sizes = [zb.zipmoe_ffn_workspace_bytes(T, 2, ok) for T in (1, 8, 16, 64)]
    assert sizes == sorted(sizes) and sizes[0] > 0
    # fp32 gate/up partials dominate: at least 2 * S * inter * 4 bytes
    assert sizes[-1] >= 2 * 128 * 14336 * 4
    for bad in (dict(T=0), dict(T=65), dict(k=0), dict(k=9), dict(hidden=1000), dict(inter=100), dict(n_experts=0),
                dict(n_experts=257)):
        ex = zb.CompressedExperts(bad.get("n_experts", 8), bad.get("hidden", 4096), bad.get("inter", 14336), 1, 16, 16,
                                  16, 1, 0, 16, 0, 16, 0)
        with pytest.raises(zb.ZipMoEError) as err:
            zb.zipmoe_ffn_workspace_bytes(bad.get("T", 4), bad.get("k", 2), ex)
        assert err.value.status == zb.ERR_UNSUPPORTED, bad
    assert ctypes.sizeof(zb.CompressedExperts) == 80


def test_records_are_level_columns(zb):
    """A record is as high as its fullest column.  Fixed-length codes (all 256 exponents equally frequent) give 32
    rows and leave every lane in its own column; on Gaussian weights the library pairs long forward streams with
    short backward streams, so that the record is within a row of the mean need of its columns -- and the oracle,
    which reads the pairing from the record, decodes it."""
    from oracle import codec
    rng = np.random.default_rng(3)
    e = np.tile(np.arange(256, dtype=np.uint16), 40)
    rng.shuffle(e)
    x = (e << 7 | 0x0033).astype(np.uint16)                   # 10240 elements: two full tiles and a half one
    blob = zb.zipmoe_encode(x, chunk_elems=4096)
    assert (blob[64:320] == 8).all() and zb.zipmoe_blob_validate(blob) == zb.OK
    info = zb.zipmoe_blob_info_get(blob)
    table = blob[info.payload_off: info.payload_off + 8].view(np.uint32)
    assert (int(table[1]) - int(table[0])) * 16 == 32 + 32 * 128
    assert blob[info.payload_off + 16: info.payload_off + 48].tolist() == list(range(32))
    assert np.array_equal(codec.decode(blob), x)

    g = inputs.gaussian((64, 4096), 0.02, 12)
    blob = zb.zipmoe_encode(g, chunk_elems=65536, max_code_len=12)
    info = zb.zipmoe_blob_info_get(blob)
    L = blob[64:320].astype(np.int64)
    mean_rows = L[(g.ravel() >> 7) & 0xFF].sum() / 64 / 32 / 32   # code bits per column, in rows of 32 bits
    offs = blob[info.payload_off: info.payload_off + 4 * 17].view(np.uint32).astype(np.int64)   # 16 tiles in the chunk
    rows = ((offs[1:] - offs[:-1]) * 16 - 32) / 128
    assert (rows == rows.astype(np.int64)).all() and rows.min() >= mean_rows - 0.5 and rows.max() <= mean_rows + 2
    assert np.median(rows) <= mean_rows + 1
    assert any(blob[info.payload_off + int(offs[0]) * 16: info.payload_off + int(offs[0]) * 16 + 32].tolist()[k] != k
               for k in range(32))                            # a real pairing, not the identity
    assert np.array_equal(codec.decode(blob), g.ravel())


def test_plan_reports_the_largest_tile_record(zb):
    x = inputs.gaussian((64, 1408), 0.02, 5)
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=4096)])
    assert 1300 < plan.max_record_bytes < 1700
    u = np.random.default_rng(0).integers(0, 1 << 16, 20000, dtype=np.uint16)
    plan = zb.DecodePlan([zb.zipmoe_encode(u, chunk_elems=4096)])
    assert plan.max_record_bytes == 32 + 32 * 128        # 8-bit codes everywhere: 128 codes per column, 32 rows


def test_plan_rejects_a_damaged_tile_table(zb):
    """The planner's record-size hint picks the kernel variant, so a tile table whose entries would wrap the 32-bit
    size computation into a small number must be refused, not planned."""
    x = inputs.gaussian((8, 4096), 0.02, 6)
    blob = zb.zipmoe_encode(x, chunk_elems=16384)
    info = zb.zipmoe_blob_info_get(blob)
    assert zb.zipmoe_blob_plan(blob, 0, 0, 0, 0, 0, 0)[0]["max_record_bytes"][0] > 0
    for entry, value in [(1, 0x10000001), (2, 0xFFFFFFF0), (1, 0)]:
        b = blob.copy()
        b[info.payload_off + 4 * entry: info.payload_off + 4 * entry + 4] = np.frombuffer(np.uint32(value).tobytes(), np.uint8)
        with pytest.raises(zb.ZipMoEError) as err:
            zb.zipmoe_blob_plan(b, 0, 0, 0, 0, 0, 0)
        assert err.value.status == zb.ERR_BAD_FORMAT, (entry, value)
