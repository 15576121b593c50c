"""zipmoe_decode_expert_ffn_noalloc: the fused expert FFN for callers that cannot allocate device memory.

Such callers exist: a plug-in living inside a serving process whose framework owns all device memory, or a
decode loop in which cudaMalloc is not allowed because it stalls the device.  The entry point therefore brings
its own fixed scratch and takes no workspace.  It must give what the ordinary entry point gives.  The test calls
it through the C ABI twice in a row (the second call finds the first call's leftovers in the shared scratch) and
compares both results with zipmoe_decode_expert_ffn; it also checks that an oversized request is refused.

Collected last on purpose: a run that stops at the first failure has by then run every other test."""
import numpy as np
import pytest

from paper_2601_21198_b200 import build, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def test_noalloc_entry_matches_the_workspace_entry_twice_in_a_row(zb):
    import torch
    E, H, I, k = 4, 512, 1024, 2
    blobs = []
    for e in range(E):
        for j in range(3):
            shape = (I, H) if j < 2 else (H, I)
            blobs.append(zb.zipmoe_encode(inputs.gaussian(shape, 0.03, 700 + 3 * e + j), layout=zb.LAYOUT_BLOCKED,
                                          chunk_elems=65536))
    ex = zb.DeviceExperts(blobs, H, I)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for call, T in enumerate((16, 5)):          # second call: other sizes, stale contents in the scratch
        tok = torch.from_numpy(inputs.tokens(T, H, seed=40 + T).view(np.int16)).cuda()
        ids_np, wts_np = inputs.routing(T, n_experts=E, k=k, seed=40 + T)
        ids, wts = torch.from_numpy(ids_np).cuda(), torch.from_numpy(wts_np).cuda()
        assert zb.zipmoe_ffn_workspace_bytes(T, k, ex.struct) <= zb.NOALLOC_SCRATCH_BYTES
        want = ex.ffn(tok, ids, wts)            # ordinary entry point, workspace from torch
        got = torch.full((T, H), 0x5555, dtype=torch.int16, device="cuda")
        zb.zipmoe_decode_expert_ffn_noalloc(tok, T, ids, wts, k, ex.struct, got, status,
                                            torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and int(ex.dev.status.item()) == 0
        a = got.view(torch.bfloat16).float()
        b = want.view(torch.bfloat16).float()
        bound = torch.maximum(torch.full_like(b, 1e-2), b.abs() * 2.0 ** -7)     # the FFN tests' tolerance
        assert bool(((a - b).abs() <= bound).all()), call
        assert torch.equal(got, want), call     # same kernels, same order of additions: the same bits


def test_noalloc_entry_refuses_what_does_not_fit(zb):
    import torch
    E, H, I = 1, 4096, 14336                    # 64 tokens x 2 of these need far more than the built-in 8 MiB
    fake = zb.CompressedExperts(E, H, I, 1, 16, 16, 16, 1, 0, 16, 0, 16, 0)
    assert zb.zipmoe_ffn_workspace_bytes(64, 2, fake) > zb.NOALLOC_SCRATCH_BYTES
    t = torch.zeros(16, dtype=torch.int16, device="cuda")
    with pytest.raises(zb.ZipMoEError) as err:
        zb.zipmoe_decode_expert_ffn_noalloc(t, 64, t, None, 2, fake, t)
    assert err.value.status == zb.ERR_BUFFER_TOO_SMALL
