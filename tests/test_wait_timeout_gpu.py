"""The kernels' bounded waits.  Every wait on an asynchronous copy has a limit; when it runs out the kernel sets
the status word (code 3), leaves undone what depended on the copy, and still terminates with tensor memory
freed.  Sound inputs never get there, so the library's test switch arms each tile-record barrier for 16 bytes
more than the copy delivers: the copy completes, nothing faults, the barrier never does, and the wait gives up
after 1024 tries.  The next ordinary call on the same stream must work as if nothing had happened."""
import numpy as np
import pytest

from paper_2601_21198_b200 import build, inputs

pytestmark = pytest.mark.gpu
WAIT_TIMEOUT = 3


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


@pytest.mark.parametrize("n,chunk", [(4096, 4096), (3 * 4096 + 100, 16384), (40 * 1024, 1024)])
def test_decode_gives_up_reports_and_recovers(zb, n, chunk):
    import torch
    x = inputs.gaussian((1, n), 0.02, n)
    plan = zb.DecodePlan([zb.zipmoe_encode(x, chunk_elems=chunk)])
    dev = plan.to_device()
    out = dev.new_output()
    out.fill_(0x5555)
    zb.zipmoe_test_wait_fault(16, 1024)
    try:
        dev.decode(out)
        torch.cuda.synchronize()
    finally:
        zb.zipmoe_test_wait_fault(0, 0)
    assert int(dev.status.item()) == WAIT_TIMEOUT
    assert bool((out == 0x5555).all())                       # nothing was written
    dev.status.zero_()
    dev.decode(out)                                          # the same stream, the ordinary way
    torch.cuda.synchronize()
    assert int(dev.status.item()) == 0
    assert np.array_equal(out.cpu().numpy().view(np.uint16)[:n], x.ravel())


def test_fused_ffn_gives_up_frees_tensor_memory_and_recovers(zb):
    import torch
    E, H, I, k, T = 3, 512, 1024, 2, 9
    blobs = []
    for e in range(E):
        for j in range(3):
            blobs.append(zb.zipmoe_encode(inputs.gaussian((I, H) if j < 2 else (H, I), 0.03, 900 + 3 * e + j),
                                          layout=zb.LAYOUT_BLOCKED, chunk_elems=65536))
    ex = zb.DeviceExperts(blobs, H, I)
    tok = torch.from_numpy(inputs.tokens(T, H, seed=5).view(np.int16)).cuda()
    ids_np, wts_np = inputs.routing(T, n_experts=E, k=k, seed=5)
    ids, wts = torch.from_numpy(ids_np).cuda(), torch.from_numpy(wts_np).cuda()
    want = ex.ffn(tok, ids, wts).clone()
    torch.cuda.synchronize()
    assert int(ex.dev.status.item()) == 0
    zb.zipmoe_test_wait_fault(16, 1024)
    try:
        ex.ffn(tok, ids, wts)
        torch.cuda.synchronize()
    finally:
        zb.zipmoe_test_wait_fault(0, 0)
    assert int(ex.dev.status.item()) == WAIT_TIMEOUT
    ex.dev.status.zero_()
    for _ in range(2):                                       # tensor memory was freed: the kernels run again
        got = ex.ffn(tok, ids, wts)
        torch.cuda.synchronize()
        assert int(ex.dev.status.item()) == 0
        assert torch.equal(got, want)
