"""The device entry points inside CUDA graphs.  A launch with fixed ranges of tiles per CTA and the fused FFN call
(five kernels, the last four with programmatic dependencies) are captured once and replayed on new inputs: what a
serving loop does to get rid of the launch overhead of small calls.  Every replay must be bit-exact (decode) or
bit-identical to the ordinary call (FFN, itself checked against the oracle elsewhere)."""
import numpy as np
import pytest

from paper_2601_21198_b200 import build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def test_decode_replayed_from_a_graph(zb):
    import torch
    x = inputs.single_expert_matrix(seed=4)                      # 704 tiles, one table: fixed ranges, no work counter
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=65536)])
    assert plan.n_tiles >= 512 * plan.n_tables
    dev = plan.to_device()
    out = dev.new_output()
    dev.decode(out)                                              # the first call does the one-time set-up: not captured
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        dev.decode(out)
    for _ in range(3):
        out.fill_(0x5555)
        g.replay()
        torch.cuda.synchronize()
        assert int(dev.status.item()) == 0
        assert np.array_equal(plan.tensor_slice(out.cpu().numpy().view(np.uint16), 0), x.ravel())
    # other compressed bytes in the same buffers: the graph decodes what is there at replay time
    y = inputs.single_expert_matrix(seed=5)
    other = zb.DecodePlan([zb.zipmoe_encode(y, chunk_elems=65536)])
    if other.payload_bytes <= plan.payload_bytes and other.n_chunks == plan.n_chunks:
        dev.payload[:other.payload.size].copy_(torch.from_numpy(other.payload))
        dev.sm.copy_(torch.from_numpy(other.sm))
        dev.descs.copy_(torch.from_numpy(other.descs.view(np.uint8).copy()))
        dev.tables.copy_(torch.from_numpy(other.tables))
        g.replay()
        torch.cuda.synchronize()
        assert int(dev.status.item()) == 0
        assert np.array_equal(plan.tensor_slice(out.cpu().numpy().view(np.uint16), 0), y.ravel())


def test_fused_ffn_replayed_from_a_graph(zb):
    import torch
    E, H, I, k, T = 4, 512, 1024, 2, 6
    blobs = []
    for e in range(E):
        for j in range(3):
            blobs.append(zb.zipmoe_encode(inputs.gaussian((I, H) if j < 2 else (H, I), 0.03, 300 + 3 * e + j),
                                          layout=zb.LAYOUT_BLOCKED, chunk_elems=65536))
    ex = zb.DeviceExperts(blobs, H, I)
    tok = torch.from_numpy(inputs.tokens(T, H, seed=1).view(np.int16)).cuda()
    ids_np, wts_np = inputs.routing(T, n_experts=E, k=k, seed=1)
    ids, wts = torch.from_numpy(ids_np).cuda(), torch.from_numpy(wts_np).cuda()
    out = torch.empty(T, H, dtype=torch.int16, device="cuda")
    want = ex.ffn(tok, ids, wts).clone()                         # ordinary call (and the one-time set-up)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        ex.ffn(tok, ids, wts, out=out)
    for _ in range(3):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert int(ex.dev.status.item()) == 0
        assert torch.equal(out, want)
    # new tokens and routing in the captured buffers
    tok2 = torch.from_numpy(inputs.tokens(T, H, seed=2).view(np.int16)).cuda()
    ids2_np, wts2_np = inputs.routing(T, n_experts=E, k=k, seed=2)
    want2 = ex.ffn(tok2, torch.from_numpy(ids2_np).cuda(), torch.from_numpy(wts2_np).cuda()).clone()
    tok.copy_(tok2)
    ids.copy_(torch.from_numpy(ids2_np))
    wts.copy_(torch.from_numpy(wts2_np))
    g.replay()
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    assert torch.equal(out, want2)
