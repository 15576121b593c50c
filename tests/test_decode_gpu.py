"""GPU parity: zipmoe_decode (through the C ABI) against the CPU oracle, bit for
bit, on the same seeded inputs.  Small cases are compared element by element
with the oracle's decode of the same blob; full-size configurations are
compared with the original tensor (the one correct answer of a lossless codec)
and, chunk by chunk on a sample, with the oracle's independent decode."""
import numpy as np
import pytest

from oracle import codec
from paper_2601_21198_b200 import build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def gpu_decode(zb, blobs):
    import torch
    plan = zb.DecodePlan(blobs)
    dev = plan.to_device()
    out = dev.new_output()
    out.fill_(0x5555)
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    host = out.cpu().numpy().view(np.uint16)
    return plan, [plan.tensor_slice(host, i) for i in range(len(blobs))], host


CASES = [
    (1, 1, 0, 256), (1, 7, 0, 256), (1, 8, 0, 256), (1, 9, 0, 256), (1, 255, 0, 256), (1, 256, 0, 256), (1, 257, 0, 1024),
    (3, 1000, 0, 1024), (1, 4095, 0, 4096), (1, 4096, 0, 4096), (1, 4097, 0, 4096), (5, 4099, 0, 16384),
    (64, 1408, 0, 4096), (100, 1408, 0, 65536), (16, 256, 1, 4096), (48, 768, 1, 8192), (32, 4096, 1, 65536),
    (16, 14336, 1, 262144), (333, 1031, 0, 262144),
    # a short last tile whose sign+mantissa bytes end in the first 2 KB piece, at its end, or just past it
    (1, 2000, 0, 4096), (1, 2048, 0, 4096), (1, 4096 + 100, 0, 4096), (1, 4096 + 2048, 0, 4096), (3, 4096 + 1365, 0, 16384),
    (1, 4096 + 2049, 0, 4096),
]


@pytest.mark.parametrize("max_code_len", [8, 12])
@pytest.mark.parametrize("rows,cols,layout,chunk", CASES)
def test_decode_matches_oracle_small(zb, rows, cols, layout, chunk, max_code_len):
    x = inputs.gaussian((rows, cols), 0.02, rows * 31 + cols)
    blob = zb.zipmoe_encode(x, layout=layout, chunk_elems=chunk, max_code_len=max_code_len)
    _, (got,), _ = gpu_decode(zb, [blob])
    want = codec.decode(blob)
    assert np.array_equal(got, want)
    assert np.array_equal(want, x.ravel())


def test_decode_of_oracle_encoded_blobs(zb):
    """The blob comes from the oracle's encoder (optimal length-limited code,
    different tie-breaks): the GPU must decode it all the same."""
    xs = [inputs.gaussian((40, 1000), 0.02, 5), inputs.gaussian((32, 512), 0.02, 6),
          inputs.stress_tensor(1, max_elems=60000)[0]]
    blobs = [codec.encode(xs[0], chunk_elems=4096), codec.encode(xs[1], layout=1, chunk_elems=8192),
             codec.encode(xs[2], chunk_elems=1024, max_code_len=9)]
    _, got, _ = gpu_decode(zb, blobs)
    for g, x in zip(got, xs):
        assert np.array_equal(g, x.ravel())


def test_many_tensors_mixed_tiles_layouts_and_tables_in_one_launch(zb):
    rng = np.random.default_rng(0)
    xs, blobs = [], []
    for i in range(40):
        kind = i % 4
        if kind == 0:
            x = inputs.gaussian((int(rng.integers(1, 30000)),), 0.02 * (1 + i), i)
            b = zb.zipmoe_encode(x, chunk_elems=1024)
        elif kind == 1:
            x = inputs.gaussian((int(rng.integers(1, 200000)),), 0.01, i)
            b = zb.zipmoe_encode(x, chunk_elems=16384)
        elif kind == 2:
            x = inputs.gaussian((16 * int(rng.integers(1, 5)), 256 * int(rng.integers(1, 7))), 0.05, i)
            b = zb.zipmoe_encode(x, layout=1, chunk_elems=8192)
        else:
            x = inputs.stress_tensor(i, max_elems=50000)[0]
            b = zb.zipmoe_encode(x, chunk_elems=256)
        xs.append(x)
        blobs.append(b)
    plan, got, host = gpu_decode(zb, blobs)
    for g, x, b in zip(got, xs, blobs):
        assert np.array_equal(g, codec.decode(b))
        assert np.array_equal(g, x.ravel())
    # the padding elements between tensors are never written
    mask = np.ones(plan.out_elems, bool)
    for i, inf in enumerate(plan.infos):
        mask[plan.out_base[i]: plan.out_base[i] + inf.n_elems] = False
    assert (host[mask] == 0x5555).all()


@pytest.mark.parametrize("chunk", [512, 768, 1024, 1536, 2048])
def test_small_tiles_taken_several_at_a_time(zb, chunk):
    """Tiles of 512, 1024 or 2048 elements (chunks below 4096) are decoded several per step when they follow one
    another in a tensor and a warp is handed several of them: sixty tensors of about 400 tiles make the ranges of
    tiles long enough for that (a launch of a few hundred tiles hands them out one by one) while the launch still
    counts as one of many tensors, and next to them, in the same launch: whole multiples of a step, one tile more,
    one tile fewer, a ragged last tile, a tensor of a single tile, a tensor with wide records (near-uniform
    exponents: fewer tiles fit the stage).  Tiles of 768 or 1536
    elements would lie across two pieces of sign+mantissa bytes and must go one by one."""
    rng = np.random.default_rng(chunk)
    sizes = [8 * 4096, 8 * 4096 + chunk, 8 * 4096 - chunk, 5 * 4096 + chunk // 2 + 3, chunk, chunk - 1, 3 * chunk + 1,
             40 * chunk]
    sizes += [(400 + k % 5) * chunk + (k % 7) * (chunk // 3 + 1) for k in range(60)]
    xs = [inputs.gaussian((n,), 0.02 * (1 + k % 9), 1000 * chunk + k) for k, n in enumerate(sizes)]
    xs.append(rng.integers(0, 1 << 16, 100 * 4096 + 77, dtype=np.uint16))    # 8-bit codes everywhere
    xs.append(inputs.stress_tensor(5, max_elems=50000)[0])
    blobs = [zb.zipmoe_encode(x, chunk_elems=chunk) for x in xs]
    plan, got, host = gpu_decode(zb, blobs)
    assert plan.flags == zb.DECODE_SHORT_CODES and plan.n_tiles < 512 * plan.n_tables
    assert plan.n_tiles > 148 * 16 * 8                                        # several tiles per warp and range
    for g, x, b in zip(got, xs, blobs):
        assert np.array_equal(g, x.ravel())
    for i in (3, 6, 9, len(xs) - 2):
        assert np.array_equal(got[i], codec.decode(blobs[i]))
    mask = np.ones(plan.out_elems, bool)
    for i, inf in enumerate(plan.infos):
        mask[plan.out_base[i]: plan.out_base[i] + inf.n_elems] = False
    assert (host[mask] == 0x5555).all()                                       # nothing written between the tensors


def test_every_bit_pattern_and_special_values(zb):
    rng = np.random.default_rng(1)
    allp = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    rng.shuffle(allp)
    sp = np.tile(inputs.special_patterns(), 7)
    blobs = [zb.zipmoe_encode(allp, chunk_elems=c) for c in (256, 1024, 4096, 65536)] + \
            [zb.zipmoe_encode(sp, chunk_elems=256)]
    _, got, _ = gpu_decode(zb, blobs)
    for g in got[:4]:
        assert np.array_equal(g, allp)
    assert np.array_equal(got[4], sp)


def test_long_records_of_near_uniform_exponents(zb):
    """Near-uniform exponents: 8-bit codes, tile records of 32 rows, decoded by the kernel instantiation with
    the larger record stages."""
    x = np.random.default_rng(2).integers(0, 1 << 16, 50021, dtype=np.uint16)
    blob = zb.zipmoe_encode(x, chunk_elems=16384)
    assert blob[64:320].min() >= 7
    _, (got,), _ = gpu_decode(zb, [blob])
    assert np.array_equal(got, codec.decode(blob)) and np.array_equal(got, x)


def _mostly_one_exponent(n_tiles, rare_tiles, layout, seed):
    """bf16 patterns with one exponent nearly everywhere and, in the given tiles (4096 consecutive elements; in the
    blocked layout 16 rows x 256 columns of a matrix 4096 wide), exponents drawn from 200 other values: at a
    code-length limit of 12 those get codes of 9 bits or more, so the records of these tiles are higher than 32
    rows."""
    rng = np.random.default_rng(seed)
    n = n_tiles * 4096
    e = np.full(n, 120, np.uint16)
    rare = np.array([v for v in range(1, 202) if v != 120], np.uint16)
    if layout:
        e = e.reshape(-1, 4096)
    for t in rare_tiles:
        if layout:
            e[16 * (t // 16):16 * (t // 16) + 16, 256 * (t % 16):256 * (t % 16) + 256] = rng.choice(rare, (16, 256))
        else:
            e[t * 4096:(t + 1) * 4096] = rng.choice(rare, 4096)
    sm = (rng.integers(0, 2, n, dtype=np.uint16) << 15) | rng.integers(0, 128, n, dtype=np.uint16)
    return ((e << 7) | sm.reshape(e.shape)).astype(np.uint16)


@pytest.mark.parametrize("n_tiles,layout", [(64, 0), (64, 1), (600, 0), (640, 1)])
def test_records_too_high_for_a_stage_are_read_from_global_memory(zb, n_tiles, layout):
    """Tiles whose codes average above 8 bits have records of more than 32 rows, which no record stage holds: the
    decoder reads them from global memory.  With few tiles the launch hands tiles out dynamically, with 600 it
    gives every CTA a fixed range; both layouts."""
    x = _mostly_one_exponent(n_tiles, (0, 5, 6, n_tiles // 2, n_tiles - 1), layout, n_tiles + layout)
    blob = zb.zipmoe_encode(x, layout=layout, chunk_elems=16384, max_code_len=12)
    plan, (got,), _ = gpu_decode(zb, [blob])
    assert plan.max_record_bytes > 32 + 32 * 128 and plan.max_code_len > 8 and plan.flags == 0
    assert (plan.n_tiles >= 512) == (n_tiles >= 600)
    assert np.array_equal(got, x.ravel())
    assert np.array_equal(got, codec.decode(blob))


def test_fixed_ranges_with_wide_records(zb):
    """A single large tensor of near-uniform exponents (8-bit codes, records of 32 rows): fixed ranges of tiles per
    CTA in the kernel instantiation with the larger record stages, linear and blocked layout."""
    rng = np.random.default_rng(77)
    for layout, shape in ((0, (700 * 4096 + 1234,)), (1, (176, 16384))):
        x = rng.integers(0, 1 << 16, shape, dtype=np.uint16)
        blob = zb.zipmoe_encode(x, layout=layout, chunk_elems=65536)
        plan, (got,), _ = gpu_decode(zb, [blob])
        assert plan.n_tiles >= 512 * plan.n_tables and plan.max_record_bytes > zb.NARROW_RECORD_BYTES
        assert np.array_equal(got, x.ravel())


def test_stress_set_sample(zb):
    xs, blobs = [], []
    for i in range(0, 96):
        x, fam, chunk = inputs.stress_tensor(i, max_elems=1 << 18)
        xs.append(x)
        blobs.append(zb.zipmoe_encode(x, chunk_elems=chunk, max_code_len=(8, 12, 10)[i % 3]))
    _, got, _ = gpu_decode(zb, blobs)
    for i, (g, x) in enumerate(zip(got, xs)):
        assert np.array_equal(g, x), i
    for i in (0, 1, 2, 3, 50):
        assert np.array_equal(got[i], codec.decode(blobs[i]))


def test_dynamic_distribution_many_launches_in_a_row(zb):
    """Launches of small or many tensors hand their tiles out through a work counter taken from a ring of 1024 in
    the library's device memory: more launches than the ring has slots, two plans alternating on two streams, every
    output bit-exact at the end and on the way."""
    import torch
    xs = [inputs.stress_tensor(i, max_elems=1 << 17)[0] for i in (0, 1, 5, 9, 12)]          # a few tiles to ~30 each
    plans = [zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=c) for x in xs]) for c in (1024, 16384)]
    assert all(p.n_tiles < 512 * p.n_tables for p in plans)                                 # dynamically distributed
    devs = [p.to_device() for p in plans]
    outs = [d.new_output() for d in devs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    want = np.concatenate(xs)
    torch.cuda.synchronize()
    for it in range(1100):
        k = it & 1
        with torch.cuda.stream(streams[k]):
            if it % 97 == 0:
                outs[k].fill_(0x5555)
            devs[k].decode(outs[k], stream=streams[k])
        if it % 97 == 1 or it == 1099:
            torch.cuda.synchronize()
            for d, o, p in zip(devs, outs, plans):
                assert int(d.status.item()) == 0
                host = o.cpu().numpy().view(np.uint16)
                got = np.concatenate([p.tensor_slice(host, i) for i in range(len(xs))])
                assert np.array_equal(got, want), it


def test_launch_that_finds_its_work_counter_taken_says_so(zb):
    """A dynamically distributed launch that finds another launch's tag in its work counter (possible only with
    more than a thousand such launches in flight) must stop, leave the output alone and set status 6; the library's
    test switch fills the counter with a tag no launch carries.  Launches with fixed ranges use no counter; the next
    ordinary launch is exact."""
    import torch
    xs = [inputs.gaussian((n,), 0.02, n) for n in (30000, 5000, 70000)]
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=1024) for x in xs])
    assert plan.n_tiles < 512 * plan.n_tables
    dev = plan.to_device()
    out = dev.new_output()
    out.fill_(0x5555)
    zb.zipmoe_test_foreign_counter(1)
    try:
        dev.decode(out)
        torch.cuda.synchronize()
    finally:
        zb.zipmoe_test_foreign_counter(0)
    assert int(dev.status.item()) == 6
    assert bool((out == 0x5555).all())
    dev.status.zero_()
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    host = out.cpu().numpy().view(np.uint16)
    for i, x in enumerate(xs):
        assert np.array_equal(plan.tensor_slice(host, i), x)


def test_short_codes_promise_kept_and_broken(zb):
    """ZIPMOE_DECODE_SHORT_CODES selects the kernel variant that carries only the common path.  The plan gives the
    promise exactly when it holds; a launch that gives it falsely must leave the offending tiles undecoded and say
    so in the status word, never write wrong data."""
    import torch
    x = inputs.stress_tensor(1, max_elems=200000)[0]                 # heavy-tailed: needs codes above 8 bits at limit 12
    short = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=16384, max_code_len=8)])
    long_ = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=16384, max_code_len=12)])
    assert short.flags == zb.DECODE_SHORT_CODES and short.max_code_len <= 8
    assert long_.max_code_len > 8 and long_.flags == 0
    for plan in (short, long_):                                     # both decode exactly with the plan's own flags
        dev = plan.to_device()
        out = dev.new_output()
        dev.decode(out)
        torch.cuda.synchronize()
        assert int(dev.status.item()) == 0
        assert np.array_equal(plan.tensor_slice(out.cpu().numpy().view(np.uint16), 0), x)
    long_.flags = zb.DECODE_SHORT_CODES                             # the false promise
    dev = long_.to_device()
    out = dev.new_output()
    out.fill_(0x5555)
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 5
    assert bool((out == 0x5555).all())                              # nothing was written


@pytest.mark.parametrize("damage", ["incomplete", "overfull", "length 13"])
@pytest.mark.parametrize("promise", [False, True])
def test_code_lengths_that_are_no_prefix_code_set_status_4(zb, damage, promise):
    """A table whose 256 code lengths do not form a complete prefix code (one code dropped, one code too many, a
    length above 12) is reported in the status word; what is decoded with it is garbage but every access stays
    inside the call's buffers (the elements between and after the tensors keep their fill), and with the
    short-codes promise nothing is decoded at all.  The same launch with the sound table is exact afterwards."""
    import torch
    xs = [inputs.gaussian((n,), 0.02, n) for n in (50000, 4096, 9000)]
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=4096) for x in xs])
    sound = plan.tables.copy()
    used = np.nonzero(sound[:256])[0]
    if damage == "incomplete":
        plan.tables[used[0]] = 0                                     # a code of the first tensor's table goes missing
    elif damage == "overfull":
        plan.tables[int(np.flatnonzero(sound[:256] == 0)[0])] = 2    # a short code more than the code space holds
    else:
        plan.tables[used[0]] = 13
    if not promise:
        plan.flags = 0
    dev = plan.to_device()
    out = dev.new_output()
    out.fill_(0x5555)
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 4
    host = out.cpu().numpy().view(np.uint16)
    mask = np.ones(plan.out_elems, bool)
    for i, inf in enumerate(plan.infos):
        mask[plan.out_base[i]: plan.out_base[i] + inf.n_elems] = False
    assert (host[mask] == 0x5555).all()
    if promise:
        assert (plan.tensor_slice(host, 0) == 0x5555).all()          # the tensor with the bad table: left alone
    for i in (1, 2):                                                 # the other tensors have sound tables
        assert np.array_equal(plan.tensor_slice(host, i), xs[i])
    dev.tables.copy_(torch.from_numpy(sound))
    dev.status.zero_()
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    host = out.cpu().numpy().view(np.uint16)
    for i, x in enumerate(xs):
        assert np.array_equal(plan.tensor_slice(host, i), x)


@pytest.mark.parametrize("chunk,max_code_len", [(1024, 8), (4096, 8), (16384, 12)])
def test_damaged_code_streams_decode_to_other_data_but_stay_in_bounds(zb, chunk, max_code_len):
    """Bytes of the payload buffer (tile tables, column tables, code words) are overwritten at random.  The kernel
    cannot know the right data any more, but it must stay inside the call's buffers: a tile table entry that no
    longer describes a record is reported (status 1) and the tile skipped, everything else decodes to something, the
    elements between and after the tensors keep their fill, and the launch after it, on sound data, is exact."""
    import torch
    rng = np.random.default_rng(chunk + max_code_len)
    xs = [inputs.gaussian((n,), 0.02, n) for n in (70000, 33000, 4096 * 9 + 5)] + [inputs.stress_tensor(3, max_elems=60000)[0]]
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=chunk, max_code_len=max_code_len) for x in xs])
    dev = plan.to_device()
    sound = dev.payload.clone()
    out = dev.new_output()
    mask = np.ones(plan.out_elems, bool)
    for i, inf in enumerate(plan.infos):
        mask[plan.out_base[i]: plan.out_base[i] + inf.n_elems] = False
    for n_bytes in (1, 30, 3000):
        bad = plan.payload.copy()
        at = rng.integers(0, plan.payload_bytes, n_bytes)
        bad[at] = rng.integers(0, 256, n_bytes).astype(np.uint8)
        dev.payload.copy_(torch.from_numpy(bad))
        dev.status.zero_()
        out.fill_(0x5555)
        dev.decode(out)
        torch.cuda.synchronize()
        assert int(dev.status.item()) in (0, 1)
        assert (out.cpu().numpy().view(np.uint16)[mask] == 0x5555).all()
    dev.payload.copy_(sound)
    dev.status.zero_()
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    host = out.cpu().numpy().view(np.uint16)
    for i, x in enumerate(xs):
        assert np.array_equal(plan.tensor_slice(host, i), x.ravel())


def test_status_word_is_optional(zb):
    """A caller that passes no status word gets the same decode (errors would then go unreported: its choice)."""
    import torch
    xs = [inputs.gaussian((n,), 0.02, n) for n in (100000, 3000)]
    for chunk in (1024, 65536):
        plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=chunk) for x in xs])
        dev = plan.to_device()
        out = dev.new_output()
        zb.zipmoe_decode(dev.descs, plan.n_chunks, plan.n_tiles, dev.tables, plan.n_tables, dev.payload, plan.payload_bytes,
                         dev.sm, plan.sm_bytes, out, plan.out_elems, None, None, plan.max_record_bytes, plan.flags)
        torch.cuda.synchronize()
        host = out.cpu().numpy().view(np.uint16)
        for i, x in enumerate(xs):
            assert np.array_equal(plan.tensor_slice(host, i), x)


def test_empty_launch_and_bad_arguments(zb):
    import torch
    zb.zipmoe_decode(None, 0, 0, None, 0, None, 0, None, 0, None, 0)       # nothing to do: OK
    t = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_decode(t, 1, 1, None, 1, t, 16, t, 16, t, 8)               # null tables
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_decode(t, 1, 1, t, 1, t.data_ptr() + 4, 16, t, 16, t, 8)   # misaligned payload


def test_out_of_range_descriptors_set_the_status_word_and_write_nothing(zb):
    """The kernel checks every offset against the buffer sizes it was given: a
    descriptor that points outside is reported and its tiles are skipped."""
    import torch
    x = inputs.gaussian((3, 5000), 0.02, 8)
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=4096)])
    for field, value in [("payload_off", plan.payload_bytes + 4096), ("sm_off", plan.sm_bytes),
                         ("out_off", plan.out_elems), ("table_id", 5)]:
        bad = zb.DecodePlan.__new__(zb.DecodePlan)
        bad.__dict__.update(plan.__dict__)
        bad.descs = plan.descs.copy()
        bad.descs[field][1] = value
        dev = bad.to_device()
        out = dev.new_output()
        out.fill_(0x5555)
        dev.decode(out)
        torch.cuda.synchronize()
        assert int(dev.status.item()) != 0, field
        host = out.cpu().numpy().view(np.uint16)
        assert (host[4096:8192] == 0x5555).all(), field


def test_single_matrix_config_full(zb):
    from paper_2601_21198_b200 import workloads
    w = workloads.single_matrix()
    dev = w.plan.to_device()
    out = dev.new_output()
    dev.decode(out)
    got = out.cpu().numpy().view(np.uint16)
    assert int(dev.status.item()) == 0
    assert np.array_equal(got, codec.decode(w.blobs[0]))
    assert np.array_equal(got, w.originals[0].ravel())


def _check_full_workload(zb, w, n_sample_chunks):
    """Whole output against the originals on the device; sampled chunks against
    the oracle's independent decode of the same blob."""
    import torch
    dev = w.plan.to_device()
    out = dev.new_output()
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    for i, x in enumerate(w.originals):
        ref = torch.from_numpy(x.view(np.int16).ravel()).cuda()
        assert torch.equal(w.plan.tensor_slice(out, i), ref), w.names[i]
        del ref
    rng = np.random.default_rng(123)
    for _ in range(n_sample_chunks):
        i = int(rng.integers(len(w.blobs)))
        inf = w.plan.infos[i]
        k = int(rng.integers(inf.n_chunks))
        want = np.zeros(inf.n_elems, np.uint16)
        codec.decode_chunk(w.blobs[i], k, want)
        got = w.plan.tensor_slice(out, i).cpu().numpy().view(np.uint16)
        touched = want != 0
        assert touched.sum() > 0.9 * min(inf.chunk_elems, inf.n_elems - k * inf.chunk_elems)
        assert np.array_equal(got[touched], want[touched])


def test_small_expert_layer_config_full(zb):
    from paper_2601_21198_b200 import workloads
    _check_full_workload(zb, workloads.small_layer(), 24)


@pytest.mark.parametrize("max_code_len", [8, 12])
def test_large_expert_layer_config_full(zb, max_code_len):
    from paper_2601_21198_b200 import workloads
    _check_full_workload(zb, workloads.large_layer(max_code_len=max_code_len), 8)


def test_large_expert_layer_blocked_layout(zb):
    from paper_2601_21198_b200 import workloads
    _check_full_workload(zb, workloads.large_layer(n_experts=1, layout=1), 6)


def test_codec_stress_set_full(zb):
    """All 4096 tensors of the stress set (sizes 1K-4M, four value families, chunk sizes 1K / 16K / 256K): one
    launch per chunk size, whole output against the originals, sampled tensors against the oracle's decode."""
    import torch
    from paper_2601_21198_b200 import workloads
    rng = np.random.default_rng(5)
    seen = 0
    for w in workloads.stress_set():
        dev = w.plan.to_device()
        out = dev.new_output()
        dev.decode(out)
        torch.cuda.synchronize()
        assert int(dev.status.item()) == 0, w.label
        host = out.cpu().numpy().view(np.uint16)
        for i, x in enumerate(w.originals):
            assert np.array_equal(w.plan.tensor_slice(host, i), x), (w.label, w.names[i])
        small = [i for i, x in enumerate(w.originals) if x.size < 200000]
        for i in rng.choice(small, 6, replace=False):
            assert np.array_equal(w.plan.tensor_slice(host, int(i)), codec.decode(w.blobs[int(i)]))
        seen += len(w.blobs)
        del dev, out, host
    assert seen == 4096


@pytest.mark.parametrize("n", [1, 15, 16, 17, 4097, 1 << 20, (1 << 22) + 5])
def test_recovery_kernel_matches_oracle_merge(zb, n):
    """zipmoe_recover against the oracle's bit-field merge (pinned on the CPU by the value formula)."""
    import torch
    rng = np.random.default_rng(n)
    e = rng.integers(0, 256, n, dtype=np.uint8)
    s = rng.integers(0, 256, n, dtype=np.uint8)
    pad = (-n) % 16
    de = torch.from_numpy(np.concatenate([e, np.zeros(pad, np.uint8)])).cuda()
    ds = torch.from_numpy(np.concatenate([s, np.zeros(pad, np.uint8)])).cuda()
    out = torch.full((n + pad,), 0x5555, dtype=torch.int16, device="cuda")
    zb.zipmoe_recover(de, ds, n, out, torch.cuda.current_stream().cuda_stream)
    got = out.cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:n], codec.merge(e, s))
    assert (got[n:] == 0x5555).all()


@pytest.mark.parametrize("on_host", ["sm", "payload", "both"])
def test_streams_in_pinned_host_memory(zb, on_host):
    """Compression states: the E-chunks and the SM-chunks of a tensor may live in different memories.  Either
    stream (or both) stays in pinned host memory, which the device reads in place during the decode."""
    import torch
    x = inputs.gaussian((700, 1031), 0.02, 77)
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=65536)])
    dev = plan.to_device()
    if on_host in ("sm", "both"):
        dev.sm = torch.from_numpy(plan.sm).pin_memory()
    if on_host in ("payload", "both"):
        dev.payload = torch.from_numpy(plan.payload).pin_memory()
    out = dev.new_output()
    dev.decode(out)
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    assert np.array_equal(out.cpu().numpy().view(np.uint16)[: x.size], x.ravel())
