"""Pins for the CPU oracle's codec (oracle/zipmoe_oracle.c): closed forms, values
the paper prints, textbook special cases, brute force on tiny inputs and the
container layout written out by hand.  No GPU, no CUDA library."""
import heapq
import itertools
import os

import numpy as np
import pytest

from oracle import codec
from paper_2601_21198_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, *v = line.split()
                out[k] = v
    return out


def entropy_bits(hist):
    p = hist[hist > 0].astype(np.float64)
    p /= p.sum()
    return float(-(p * np.log2(p)).sum())


# ---------------------------------------------------------------- bit fields

def test_split_fields_reproduce_the_value_formula():
    """(-1)^s * 2^(e-127) * 1.m over every normal pattern equals the number the
    pattern denotes (numpy's float32 view of pattern << 16)."""
    g = golden()
    assert [int(v) for v in g["bf16_field_bits"]] == [1, 8, 7]
    bias = int(g["bf16_exponent_bias"][0])
    x = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    e, sm = codec.split(x)
    normal = (e > 0) & (e < 255)
    sign = (sm >> 7).astype(np.float64)
    mant = (sm & 0x7F).astype(np.float64)
    val = (-1.0) ** sign * np.exp2(e.astype(np.float64) - bias) * (1.0 + mant / 128.0)
    ref = inputs.bf16_bits_to_f32(x).astype(np.float64)
    assert np.array_equal(val[normal], ref[normal])
    # the extremes the paper quotes
    big = val[normal].max()
    small = np.abs(val[normal]).min()
    assert abs(big / float(g["bf16_max_magnitude"][0]) - 1) < 5e-3
    assert abs(small / float(g["bf16_min_normal"][0]) - 1) < 5e-3


def test_split_merge_identity_on_every_pattern():
    x = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    e, sm = codec.split(x)
    assert np.array_equal(codec.merge(e, sm), x)
    # each of the two streams is one byte per element: half of the tensor each
    assert e.nbytes * 2 == x.nbytes and sm.nbytes * 2 == x.nbytes
    assert int(golden()["sm_share_percent"][0]) == 50


def test_special_values_are_just_patterns():
    sp = inputs.special_patterns()
    e, sm = codec.split(sp)
    assert np.array_equal(codec.merge(e, sm), sp)
    assert set(e.tolist()) == {0, 255}


# ---------------------------------------------------------------- code lengths

def kraft_scaled(lengths, scale=12):
    L = lengths[lengths > 0].astype(np.int64)
    return int((1 << (scale - L)).sum())


def huffman_cost(weights):
    """Textbook Huffman: total cost = sum of the weights of all merged nodes."""
    h = list(weights)
    heapq.heapify(h)
    cost = 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        cost += a + b
        heapq.heappush(h, a + b)
    return cost


def random_hist(rng, m, skew):
    hist = np.zeros(256, np.uint64)
    syms = rng.choice(256, size=m, replace=False)
    w = np.maximum(1, (rng.random(m) ** skew * 1e6)).astype(np.uint64)
    hist[syms] = w
    return hist


@pytest.mark.parametrize("m", [2, 3, 5, 17, 36, 100, 256])
@pytest.mark.parametrize("max_len", [8, 10, 12])
def test_kraft_equality_and_length_limit(m, max_len):
    rng = np.random.default_rng(m * 100 + max_len)
    for skew in (1.0, 4.0, 12.0):
        hist = random_hist(rng, m, skew)
        L = codec.code_lengths(hist, max_len)
        assert ((L > 0) == (hist > 0)).all()
        assert L.max() <= max_len
        assert kraft_scaled(L) == 1 << 12


@pytest.mark.parametrize("m", [2, 3, 8, 36, 256])
def test_cost_equals_textbook_huffman_when_limit_is_slack(m):
    """With near-equal weights an unrestricted Huffman tree is no deeper than
    ceil(log2 m) + 1 <= 12, so the limit does not bind and the cost is unique."""
    rng = np.random.default_rng(m)
    for _ in range(5):
        hist = np.zeros(256, np.uint64)
        syms = rng.choice(256, size=m, replace=False)
        hist[syms] = rng.integers(1000, 2000, m).astype(np.uint64)
        L = codec.code_lengths(hist, 12)
        cost = int((hist * L).sum())
        assert cost == huffman_cost([int(w) for w in hist[hist > 0]])
        n, H = int(hist.sum()), entropy_bits(hist)
        assert n * H <= cost < n * (H + 1)


def test_gaussian_weights_cost_between_entropy_and_entropy_plus_one():
    x = inputs.gaussian((256, 1024), 0.02, 3)
    hist = codec.histogram(codec.split(x)[0])
    L = codec.code_lengths(hist, 12)
    n, H = int(hist.sum()), entropy_bits(hist)
    cost = int((hist * L).sum())
    assert n * H <= cost < n * (H + 1)
    # the synthetic stand-in sits where the paper's models do (Fig. 2: 2.55-2.65 bits)
    ents = [float(v) for v in golden()["exponent_entropy_bits"]]
    assert min(ents) - 0.1 < H < max(ents) + 0.1


def brute_force_min_cost(weights, max_len):
    best = None
    m = len(weights)
    for lens in itertools.product(range(1, max_len + 1), repeat=m):
        if sum(2 ** (max_len - l) for l in lens) <= 2 ** max_len:
            c = sum(w * l for w, l in zip(weights, lens))
            best = c if best is None else min(best, c)
    return best


@pytest.mark.parametrize("weights,max_len", [
    ([1, 1], 3), ([5, 1, 1], 3), ([10, 3, 2, 1], 3), ([10, 3, 2, 1], 2), ([100, 50, 20, 5, 1], 3),
    ([100, 50, 20, 5, 1], 4), ([1, 1, 2, 3, 5, 8], 3), ([1, 1, 2, 3, 5, 8], 4), ([1, 1, 2, 3, 5, 8], 5),
    ([7, 7, 7, 7, 7, 7], 3), ([1000, 1, 1, 1, 1, 1], 3), ([1000, 1, 1, 1, 1, 1], 5),
])
def test_length_limited_cost_is_minimal_by_enumeration(weights, max_len):
    hist = np.zeros(256, np.uint64)
    syms = [3, 40, 77, 130, 200, 255][: len(weights)]
    hist[syms] = weights
    L = codec.code_lengths(hist, max_len)
    assert L.max() <= max_len and kraft_scaled(L) == 1 << 12
    assert int((hist * L).sum()) == brute_force_min_cost(weights, max_len)


def test_degenerate_histograms():
    assert codec.code_lengths(np.zeros(256, np.uint64)).max() == 0
    for s in (0, 17, 255):
        hist = np.zeros(256, np.uint64)
        hist[s] = 1234
        L = codec.code_lengths(hist)
        assert L[s] == 1 and L[(s + 1) % 256] == 1 and L.sum() == 2


def test_canonical_codes_are_ordered_and_prefix_free():
    rng = np.random.default_rng(5)
    hist = random_hist(rng, 40, 6.0)
    L = codec.code_lengths(hist, 12)
    C = codec.canonical_codes(L)
    used = [(int(L[s]), s, int(C[s])) for s in range(256) if L[s]]
    used.sort()
    # consecutive in (length, symbol) order, left-aligned values strictly increasing
    left = [c << (12 - l) for l, _, c in used]
    assert all(a < b for a, b in zip(left, left[1:]))
    for (l0, _, c0), (l1, _, c1) in zip(used, used[1:]):
        assert c1 == (c0 + 1) << (l1 - l0)
    words = [format(c, "0%db" % l) for l, _, c in used]
    for a in words:
        for b in words:
            assert a is b or not b.startswith(a)
    assert words[0] == "0" * used[0][0]
    with pytest.raises(ValueError):
        bad = L.copy()
        bad[np.flatnonzero(L)[0]] += 1      # Kraft sum drops below 1: not a complete code
        codec.canonical_codes(bad)


# ---------------------------------------------------------------- container

def _bits_of_bytes(values):
    """MSB-first bits of a list of 8-bit codes."""
    return [(v >> b) & 1 for v in values for b in range(7, -1, -1)]


def _record_of_columns(bcol, columns):
    """A tile record written out from the format's definition: 32 bytes naming the column of each lane's backward
    stream, then W rows of 32 words; bit y of column c is bit 31 - y % 32 of the word in row y // 32, column c."""
    W = len(columns[0]) // 32
    words = np.zeros((W, 32), np.uint32)
    for c, bits in enumerate(columns):
        assert len(bits) == 32 * W
        for y, bit in enumerate(bits):
            if bit:
                words[y // 32, c] |= np.uint32(1 << (31 - y % 32))
    return np.concatenate([np.array(bcol, np.uint8), words.astype("<u4").ravel().view(np.uint8)])


def _column(forward_bits, backward_bits, W):
    """Forward stream from bit 0 upwards, backward stream from bit 32 W - 1 downwards, zeros between."""
    col = [0] * (32 * W)
    assert len(forward_bits) + len(backward_bits) <= 32 * W
    col[:len(forward_bits)] = forward_bits
    for k, bit in enumerate(backward_bits):
        col[32 * W - 1 - k] = bit
    return col


def test_uniform_exponents_store_the_raw_exponent_bytes():
    """All 256 exponents equally frequent -> every code is the 8-bit symbol itself, so column c of a tile's
    record is: the exponent bytes of lane c's even iterations from the top, and those of its odd iterations
    written upwards from the bottom (all streams are equally long, so every lane keeps its own column).
    Needs no Huffman."""
    rng = np.random.default_rng(11)
    e = np.tile(np.arange(256, dtype=np.uint16), 32)
    rng.shuffle(e)
    sm = rng.integers(0, 256, e.size).astype(np.uint16)
    x = ((sm & 0x80) << 8 | e << 7 | sm & 0x7F).astype(np.uint16)
    blob = codec.encode(x, chunk_elems=4096)
    assert (blob[64:320] == 8).all()
    hdr = codec.info(blob)
    assert hdr["n_chunks"] == 2 and hdr["n_tiles"] == 2 and hdr["tile_elems"] == 4096
    pay = hdr["payload_off"]
    offs = blob[320:320 + 8 * 3].view(np.uint64)
    rec_bytes = 32 + 32 * 128          # 128 codes of 8 bits per column: 32 rows
    assert offs.tolist() == [0, (16 + rec_bytes) * 8, 2 * (16 + rec_bytes) * 8]
    for q in range(2):
        chunk = blob[pay + q * (16 + rec_bytes): pay + (q + 1) * (16 + rec_bytes)]
        assert chunk[:8].view(np.uint32).tolist() == [1, 1 + rec_bytes // 16]
        tile = e[q * 4096:(q + 1) * 4096].astype(np.uint8).reshape(16, 32, 8)   # [i, lane, j]
        cols = [_column(_bits_of_bytes(tile[0::2, lane, :].ravel().tolist()),
                        _bits_of_bytes(tile[1::2, lane, :].ravel().tolist()), 32) for lane in range(32)]
        assert np.array_equal(chunk[16:], _record_of_columns(range(32), cols))
    # sign+mantissa section: raw bytes in element order for the linear layout
    smsec = blob[pay + hdr["payload_bytes"]:]
    assert np.array_equal(smsec, ((x >> 8) & 0x80 | x & 0x7F).astype(np.uint8))
    assert np.array_equal(codec.decode(blob), x)


def test_uniform_exponents_odd_iteration_count_and_ragged_tail():
    """Three iterations per tile (chunk of 768 elements) and a tensor that ends in the middle of a lane's
    group: the forward stream holds iterations 0 and 2, the backward stream iteration 1, and elements past
    the end are not coded.  The longest column needs 16 + 8 codes of 8 bits: six rows."""
    n = 256 * 5 + 13
    rng = np.random.default_rng(5)
    e = np.concatenate([np.tile(np.arange(256, dtype=np.uint16), 5), np.arange(13, dtype=np.uint16)])
    rng.shuffle(e)
    x = (e << 7 | 0x0055).astype(np.uint16)
    blob = codec.encode(x, chunk_elems=768)
    assert (blob[64:320] == 8).all()            # counts of 5 or 6: still a balanced tree
    hdr = codec.info(blob)
    assert hdr["tile_elems"] == 768 and hdr["n_tiles"] == 2 and hdr["n_chunks"] == 2
    pay = hdr["payload_off"]
    offs = (blob[320:320 + 8 * 3].view(np.uint64) // 8).tolist()
    for q in range(2):
        chunk = blob[pay + offs[q]: pay + offs[q + 1]]
        first, end = chunk[:8].view(np.uint32).tolist()
        rec = chunk[16 * first: 16 * end]
        assert rec.size == 32 + 6 * 128
        cols = []
        for lane in range(32):
            sub = [[int(e[f]) for i in range(h, 3, 2) for j in range(8)
                    for f in [q * 768 + (i * 32 + lane) * 8 + j] if f < n] for h in range(2)]
            cols.append(_column(_bits_of_bytes(sub[0]), _bits_of_bytes(sub[1]), 6))
        # the lanes with the longest forward streams come first already (tile 1: lanes 0 and 1), every
        # backward stream is equally long: each lane keeps its own column
        assert np.array_equal(rec, _record_of_columns(range(32), cols))
    assert np.array_equal(codec.decode(blob), x)


def test_streams_are_paired_into_columns_longest_forward_with_shortest_backward():
    """Three exponents A, B, C with codes 0, 10, 11 (A far more frequent).  One tile of two iterations: the
    forward streams code iteration 0, the backward streams iteration 1.  Lane 3 has the longest forward stream
    (four B), lane 7 the shortest backward stream (no C; every other lane has one), so lane 7's backward stream
    goes to column 3, and the lanes between move up by one column.  One row holds everything."""
    A, B, C = 120, 121, 122
    e = np.full((2, 32, 8), A, np.uint16)
    e[0, 3, [1, 2, 5, 6]] = B
    for lane in range(32):
        if lane != 7:
            e[1, lane, lane % 8] = C
    x = (e.ravel() << 7 | 0x0011).astype(np.uint16)
    blob = codec.encode(x, chunk_elems=512)
    L = blob[64:320]
    assert (L[A], L[B], L[C]) == (1, 2, 2) and L.sum() == 5
    code = {A: [0], B: [1, 0], C: [1, 1]}
    hdr = codec.info(blob)
    assert hdr["n_tiles"] == 1 and hdr["payload_bytes"] == 16 + 32 + 128
    rec = blob[hdr["payload_off"] + 16: hdr["payload_off"] + hdr["payload_bytes"]]
    bcol = [0, 1, 2, 4, 5, 6, 7, 3] + list(range(8, 32))
    assert rec[:32].tolist() == bcol
    fwd = [[b for s in e[0, lane] for b in code[int(s)]] for lane in range(32)]
    bwd = [[b for s in e[1, lane] for b in code[int(s)]] for lane in range(32)]
    assert len(fwd[3]) == 12 and len(bwd[7]) == 8 and len(bwd[0]) == 9
    cols = [_column(fwd[c], bwd[bcol.index(c)], 1) for c in range(32)]
    assert np.array_equal(rec, _record_of_columns(bcol, cols))
    assert np.array_equal(codec.decode(blob), x)
    # column 0 uses bits 0..7 (forward) and 23..31 (backward); a set bit between them is damage
    bad = blob.copy()
    bad[hdr["payload_off"] + 16 + 32 + 2] |= 1          # bit 15 of column 0 = bit 16 of its word
    with pytest.raises(ValueError):
        codec.decode(bad)


def test_round_trip_brute_force_tiny():
    """Every sequence of up to 6 elements over three exponent values."""
    pats = np.array([0x3C00, 0xBC80, 0x3D7F], dtype=np.uint16)   # exponents 120, 121, 122
    for n in range(1, 7):
        for seq in itertools.product(range(3), repeat=n):
            x = pats[list(seq)]
            assert np.array_equal(codec.decode(codec.encode(x, chunk_elems=256)), x)


@pytest.mark.parametrize("chunk", [256, 1024, 4096, 16384])
def test_round_trip_every_pattern(chunk):
    rng = np.random.default_rng(chunk)
    x = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    rng.shuffle(x)
    for n in (65536, 65535, 4097, 4095, 257, 255, 9, 8, 7, 1):
        y = x[:n]
        assert np.array_equal(codec.decode(codec.encode(y, chunk_elems=chunk)), y)


@pytest.mark.parametrize("max_len", [8, 9, 12])
def test_round_trip_with_binding_length_limit(max_len):
    x, _, _ = inputs.stress_tensor(1, max_elems=50000)          # heavy-tailed: many rare exponents
    blob = codec.encode(x, chunk_elems=1024, max_code_len=max_len)
    assert blob[64:320].max() <= max_len
    assert np.array_equal(codec.decode(blob), x)


def test_round_trip_stress_families_and_specials():
    for idx in range(8):
        x, fam, chunk = inputs.stress_tensor(idx, max_elems=30000)
        blob = codec.encode(x, chunk_elems=chunk)
        assert np.array_equal(codec.decode(blob), x), fam
    sp = inputs.special_patterns()
    assert np.array_equal(codec.decode(codec.encode(sp, chunk_elems=256)), sp)


def test_empty_and_single_symbol_tensors():
    blob = codec.encode(np.zeros(0, np.uint16), rows=0, cols=0, chunk_elems=4096)
    hdr = codec.info(blob)
    assert hdr["n_chunks"] == 0 and hdr["n_tiles"] == 0 and codec.decode(blob).size == 0
    x = np.full(1000, 0x3C12, np.uint16)
    blob = codec.encode(x, chunk_elems=1024)
    assert np.array_equal(codec.decode(blob), x)
    hdr = codec.info(blob)
    rec = blob[hdr["payload_off"] + 16: hdr["payload_off"] + hdr["payload_bytes"]]
    assert rec.size == 32 + 128 and not rec[32:].any()     # one bit per element (the code 0): at most 16 + 16 in a column


def test_chunks_decode_independently_and_in_any_order():
    x = inputs.gaussian((20000,), 0.02, 9)
    blob = codec.encode(x, chunk_elems=1024)
    K = codec.info(blob)["n_chunks"]
    assert K == 20
    out = np.zeros(x.size, np.uint16)
    for k in np.random.default_rng(0).permutation(K):
        before = out.copy()
        codec.decode_chunk(blob, int(k), out)
        lo, hi = k * 1024, min((k + 1) * 1024, x.size)
        assert np.array_equal(out[lo:hi], x[lo:hi])
        untouched = np.ones(x.size, bool)
        untouched[lo:hi] = False
        assert np.array_equal(out[untouched], before[untouched])
    assert np.array_equal(out, x)


def test_blocked_layout_round_trip_and_tile_order():
    rows, cols = 48, 768
    x = inputs.gaussian((rows, cols), 0.02, 21)
    blob = codec.encode(x, layout=1, chunk_elems=8192)
    hdr = codec.info(blob)
    assert hdr["layout"] == 1 and hdr["n_tiles"] == 3 * 3 and hdr["n_chunks"] == 5
    assert np.array_equal(codec.decode(blob).reshape(rows, cols), x)
    # sign+mantissa section is stored tile by tile: tile q = 16x256 block (q // 3, q % 3)
    smsec = blob[hdr["payload_off"] + hdr["payload_bytes"]:]
    sm = ((x >> 8) & 0x80 | x & 0x7F).astype(np.uint8)
    for q in range(9):
        rb, cb = divmod(q, 3)
        block = sm[rb * 16:(rb + 1) * 16, cb * 256:(cb + 1) * 256]
        assert np.array_equal(smsec[q * 4096:(q + 1) * 4096], block.ravel())
    # chunk 1 (tiles 2, 3) alone fills exactly blocks (0,2) and (1,0)
    out = np.zeros(x.size, np.uint16)
    codec.decode_chunk(blob, 1, out)
    out = out.reshape(rows, cols)
    mask = np.zeros((rows, cols), bool)
    mask[0:16, 512:768] = True
    mask[16:32, 0:256] = True
    assert np.array_equal(out[mask], x[mask]) and not out[~mask].any()


def test_compressed_size_against_the_entropy_bound():
    """Payload can not beat the order-0 entropy of the exponents; the whole
    blob can not beat (8 + H)/16 of the tensor -- the bound the paper computes
    -- and for Gaussian weights it lands between that bound and the paper's
    general-purpose compressors."""
    g = golden()
    for pair in g["entropy_bound_pairs"]:
        H, pct = (float(v) for v in pair.split(":"))
        assert round((8 + H) / 16 * 100, 2) == pct
    x = inputs.single_expert_matrix(0)
    hist = codec.histogram(codec.split(x)[0])
    H, n = entropy_bits(hist), x.size
    for chunk in (4096, 65536):
        blob = codec.encode(x, chunk_elems=chunk)
        hdr = codec.info(blob)
        assert hdr["sm_bytes"] == n
        assert hdr["payload_bytes"] * 8 >= n * H
        ratio = blob.size / (2 * n)
        assert (8 + H) / 16 <= ratio
        assert ratio < float(g["zstd_size_percent"][0]) / 100
    support = int((hist > 0).sum())
    assert support <= max(float(v) for v in g["exponent_support_percent"]) / 100 * 256


def test_corrupt_blobs_are_rejected_not_decoded():
    x = inputs.gaussian((5000,), 0.02, 2)
    blob = codec.encode(x, chunk_elems=1024)
    hdr = codec.info(blob)
    pay = hdr["payload_off"]

    def broken(mut):
        b = blob.copy()
        mut(b)
        with pytest.raises(ValueError):
            codec.decode(b)

    broken(lambda b: b.__setitem__(0, 0))                                  # magic
    broken(lambda b: b.__setitem__(8, b[8] ^ 1))                           # n_elems vs rows*cols
    broken(lambda b: b.__setitem__(64 + int(np.flatnonzero(b[64:320])[0]), 0))   # incomplete code
    broken(lambda b: b.__setitem__(328, b[328] ^ 0x10))                    # chunk offset not 128-bit aligned
    broken(lambda b: b.__setitem__(pay + 4, b[pay + 4] + 1))               # tile table end != chunk size
    broken(lambda b: b.__setitem__(pay + 16, b[pay + 16] ^ 1))             # two backward streams in one column
    broken(lambda b: b.__setitem__(pay + 17, 32))                          # a column that does not exist
    with pytest.raises(ValueError):
        codec.decode(blob[:-16])                                           # truncated
