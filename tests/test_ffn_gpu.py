"""GPU parity of the fused decode + expert FFN (zipmoe_decode_expert_ffn through
the C ABI) against the CPU oracle's FFN on the oracle's decoded weights.
Tolerance (bf16 inputs, fp32 accumulation): every element within 1e-2 of the
oracle -- or within one bf16 spacing of it where that spacing is larger (an
output of magnitude >= 2 is 2^-6 = 0.0156 away from its neighbours, so a single
rounding flip of the final bf16 already exceeds 1e-2) -- and relative Frobenius
error <= 2e-2."""
import numpy as np
import pytest

from oracle import codec, ffn as offn
from paper_2601_21198_b200 import build, inputs

pytestmark = pytest.mark.gpu

MAX_ABS, REL_FRO = 1e-2, 2e-2


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def make_layer(zb, E, H, I, seed, std=0.03, max_code_len=0):
    ws, blobs = [], []
    for e in range(E):
        for j in range(3):
            shape = (I, H) if j < 2 else (H, I)
            w = inputs.gaussian(shape, std * (1 + 0.3 * ((e + j) % 3)), seed + 3 * e + j)
            ws.append(w)
            blobs.append(zb.zipmoe_encode(w, layout=zb.LAYOUT_BLOCKED, chunk_elems=65536, max_code_len=max_code_len))
    return ws, blobs


def oracle_out(ws_decoded, tok, ids, wts, rows):
    w1 = {e: ws_decoded[3 * e] for e in set(ids[rows].ravel().tolist())}
    w3 = {e: ws_decoded[3 * e + 1] for e in w1}
    w2 = {e: ws_decoded[3 * e + 2] for e in w1}
    return offn.expert_ffn(tok[rows], ids[rows], None if wts is None else wts[rows], w1, w3, w2)


def check(got_bits, want_bits, want_exact, label):
    """want_bits: the oracle's bf16 output; want_exact: its fp64 value before the last rounding.  Every element
    must lie within 1e-2 of the oracle's output -- except that an element of magnitude >= 1.28, whose bf16
    neighbours are more than 1e-2 apart, may be the neighbouring bf16 value (one rounding flip of the final
    conversion: fp32 against fp64 accumulation); such elements are counted, must be exactly one bf16 step away,
    and must be rare."""
    got, want = offn.bf16_to_f64(got_bits), offn.bf16_to_f64(want_bits)
    err = np.abs(got - want)
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    assert rel <= REL_FRO, (label, rel)
    wide = err > MAX_ABS
    n_wide = int(wide.sum())
    if n_wide:
        g, w = got_bits[wide].astype(np.int64), want_bits[wide].astype(np.int64)
        assert (np.abs(want[wide]) >= 1.28).all(), (label, "an error above 1e-2 on a small output", err.max())
        assert (np.abs(g - w) == 1).all(), (label, "more than one bf16 step from the oracle")   # same sign, adjacent patterns
        # a flip needs the exact value to sit near the midpoint of the two candidates
        assert (np.abs(got[wide] - want_exact[wide]) <= 0.75 * err[wide]).all(), label
        assert n_wide <= max(2, got.size // 500), (label, n_wide)
    print("%s: %d of %d outputs one bf16 step from the oracle (|value| >= 1.28), max abs err %.3g, rel Frobenius %.3g"
          % (label, n_wide, got.size, err.max(), rel))


@pytest.mark.parametrize("T", [1, 5, 16, 64])
@pytest.mark.parametrize("max_code_len", [8, 12])
def test_small_experts_match_oracle(zb, T, max_code_len):
    import torch
    E, H, I, k = 4, 512, 1024, 2
    ws, blobs = make_layer(zb, E, H, I, seed=50, max_code_len=max_code_len)
    decoded = [codec.decode(b).reshape(w.shape) for b, w in zip(blobs, ws)]
    for d, w in zip(decoded, ws):
        assert np.array_equal(d, w)
    ex = zb.DeviceExperts(blobs, H, I)
    tok = inputs.tokens(T, H, seed=T)
    ids, wts = inputs.routing(T, n_experts=E, k=k, seed=T)
    for weights in (wts, None):
        out = ex.ffn(torch.from_numpy(tok.view(np.int16)).cuda(), torch.from_numpy(ids).cuda(),
                     None if weights is None else torch.from_numpy(weights).cuda())
        torch.cuda.synchronize()
        assert int(ex.dev.status.item()) == 0
        want, y = oracle_out(decoded, tok, ids, weights, np.arange(T))
        check(out.cpu().numpy().view(np.uint16), want, y, (T, max_code_len, weights is None))


@pytest.mark.parametrize("long_codes", [False, True])
def test_experts_whose_records_do_not_fit_the_record_stage(zb, long_codes):
    """Weights with forty equally likely exponents take more than 5 bits per code: tile records of about 22 rows,
    more than the fused kernel's record stages hold, so the decode warps read them from global memory.  With a
    thin tail of forty more (tiny) exponents and a code-length limit of 12 the tail's codes are longer than 8 bits
    and the wide table is used as well."""
    import torch
    E, H, I, k, T = 2, 512, 1024, 2, 5
    rng = np.random.default_rng(123)
    ws, blobs = [], []
    for j in range(3 * E):
        shape = (I, H) if j % 3 < 2 else (H, I)
        e = rng.integers(84, 124, shape, dtype=np.uint16)
        if long_codes:
            e = np.where(rng.random(shape) < 2e-3, rng.integers(40, 80, shape, dtype=np.uint16), e)
        w = ((rng.integers(0, 2, shape, dtype=np.uint16) << 15) | (e << 7) |
             rng.integers(0, 128, shape, dtype=np.uint16)).astype(np.uint16)
        ws.append(w)
        blobs.append(zb.zipmoe_encode(w, layout=zb.LAYOUT_BLOCKED, chunk_elems=65536, max_code_len=12 if long_codes else 8))
    plan = zb.DecodePlan(blobs)
    assert plan.max_record_bytes > 2432 and (plan.max_code_len > 8) == long_codes
    ex = zb.DeviceExperts(blobs, H, I)
    tok = inputs.tokens(T, H, seed=9)
    ids, wts = inputs.routing(T, n_experts=E, k=k, seed=9)
    out = ex.ffn(torch.from_numpy(tok.view(np.int16)).cuda(), torch.from_numpy(ids).cuda(), torch.from_numpy(wts).cuda())
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    want, y = oracle_out(ws, tok, ids, wts, np.arange(T))
    check(out.cpu().numpy().view(np.uint16), want, y, ("records read from global memory", long_codes))


def test_single_expert_k1_and_unused_experts(zb):
    import torch
    E, H, I = 3, 256, 1024
    ws, blobs = make_layer(zb, E, H, I, seed=80)
    ex = zb.DeviceExperts(blobs, H, I)
    tok = inputs.tokens(7, H, seed=3)
    ids = np.full((7, 1), 1, np.int32)            # every token to expert 1; experts 0 and 2 idle
    out = ex.ffn(torch.from_numpy(tok.view(np.int16)).cuda(), torch.from_numpy(ids).cuda(), None)
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    want, y = oracle_out(ws, tok, ids, None, np.arange(7))
    check(out.cpu().numpy().view(np.uint16), want, y, "k1")


def test_status_word_is_optional(zb):
    import torch
    E, H, I = 2, 256, 512
    ws, blobs = make_layer(zb, E, H, I, seed=70)
    ex = zb.DeviceExperts(blobs, H, I)
    tok = torch.from_numpy(inputs.tokens(3, H, seed=4).view(np.int16)).cuda()
    ids_np, wts_np = inputs.routing(3, n_experts=E, k=2, seed=4)
    ids, wts = torch.from_numpy(ids_np).cuda(), torch.from_numpy(wts_np).cuda()
    want = ex.ffn(tok, ids, wts).clone()
    n = zb.zipmoe_ffn_workspace_bytes(3, 2, ex.struct)
    wsp = torch.empty(n, dtype=torch.uint8, device="cuda")
    out = torch.zeros(3, H, dtype=torch.int16, device="cuda")
    zb.zipmoe_decode_expert_ffn(tok, 3, ids, wts, 2, ex.struct, out, wsp, n, None, None)
    torch.cuda.synchronize()
    assert torch.equal(out, want)


def test_bad_arguments(zb):
    import torch
    E, H, I = 1, 256, 1024
    ws, blobs = make_layer(zb, E, H, I, seed=90)
    ex = zb.DeviceExperts(blobs, H, I)
    tok = torch.zeros(65, H, dtype=torch.int16, device="cuda")
    ids = torch.zeros(65, 1, dtype=torch.int32, device="cuda")
    with pytest.raises(zb.ZipMoEError):
        ex.ffn(tok, ids, None)                     # T > 64
    bad = zb.CompressedExperts.from_buffer_copy(ex.struct)
    bad.inter = 1000
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_ffn_workspace_bytes(4, 2, bad)   # inter not a multiple of 256


@pytest.mark.parametrize("T", [1, 16, 64])
def test_large_experts_config(zb, T):
    """8 experts of 4096 -> 14336 -> 4096 (256K-element chunks), top-2 of 8 with Zipf(1.2) popularity.
    Every token row is compared with the oracle for T = 1 and 16; for T = 64 (which also selects the kernel's
    other shared-memory plan) 16 rows chosen so that every expert that has tokens is covered."""
    import torch
    from paper_2601_21198_b200 import workloads
    w = _large_layer(workloads)
    ex = _large_experts(zb, w)
    tok = inputs.tokens(T, 4096, seed=100 + T)
    ids, wts = inputs.routing(T, n_experts=8, k=2, seed=T)
    out = ex.ffn(torch.from_numpy(tok.view(np.int16)).cuda(), torch.from_numpy(ids).cuda(),
                 torch.from_numpy(wts).cuda())
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    rows = np.arange(T) if T <= 16 else _rows_covering_all_experts(ids, 16, seed=T)
    assert set(ids[rows].ravel().tolist()) == set(ids.ravel().tolist())
    want, y = oracle_out(w.originals, tok, ids, wts, rows)
    check(out.cpu().numpy().view(np.uint16)[rows], want, y, ("large", T))


@pytest.mark.parametrize("T", [1, 16])
def test_paper_shape_experts_with_padded_intermediate_size(zb, T):
    """Experts of the paper's own models, 2048 -> 1408 -> 2048, top-6: the intermediate size is not a multiple of
    256, so the experts are zero-padded to 1536 before they are encoded.  The oracle FFN runs on the unpadded
    matrices: the padding must not change the result.  16 of the 64 experts keep the test short."""
    import torch
    from paper_2601_21198_b200 import workloads
    E, k = 16, 6
    w = workloads.small_layer_ffn(n_experts=E)
    assert w.inter == 1536 and all(i.rows % 16 == 0 and i.cols % 256 == 0 for i in w.plan.infos)
    ex = zb.DeviceExperts(w.blobs, w.hidden, w.inter)
    tok = inputs.tokens(T, w.hidden, seed=300 + T)
    ids, wts = inputs.routing(T, n_experts=E, k=k, seed=300 + T)
    out = ex.ffn(torch.from_numpy(tok.view(np.int16)).cuda(), torch.from_numpy(ids).cuda(), torch.from_numpy(wts).cuda())
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    want, y = oracle_out(w.originals, tok, ids, wts, np.arange(T))
    check(out.cpu().numpy().view(np.uint16), want, y, ("paper shape", T))


def _rows_covering_all_experts(ids, n, seed):
    """n token rows: first one row for every expert that appears in ids (the first token that names it), then
    seeded random rows."""
    rows = []
    for e in sorted(set(ids.ravel().tolist())):
        t = int(np.nonzero((ids == e).any(axis=1))[0][0])
        if t not in rows:
            rows.append(t)
    rest = [int(t) for t in np.random.default_rng(seed).permutation(ids.shape[0]) if int(t) not in rows]
    return np.array(sorted(rows + rest[: max(0, n - len(rows))]))


_cache = {}


def _large_layer(workloads):
    if "w" not in _cache:
        _cache["w"] = workloads.large_layer(layout=1)
    return _cache["w"]


def _large_experts(zb, w):
    if "ex" not in _cache:
        _cache["ex"] = zb.DeviceExperts(w.blobs, 4096, 14336)
    return _cache["ex"]
