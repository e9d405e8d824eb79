"""The failure path behind SD_ATTN_ERR_DEVICE_TIMEOUT, exercised on purpose and without any fault.

Every wait inside the tensor-core kernels is bounded: a waiter that runs out of polls raises its block's abort
flag, records where it gave up in the handle's device status block, and the block drains, releases its tensor
memory and returns.  ``sd_attn_selftest_wait_timeout`` runs those steps in a one-block kernel whose first waiter has
a budget of a few thousand polls on a barrier nothing ever arrives on (nothing traps, faults or spins without a
limit).  Checked here: the status block's contents, that the query reports the time-out exactly once, and that the
handle and the context go on working -- an ordinary forward afterwards matches the oracle.
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_an_expired_wait_is_reported_once_and_the_handle_stays_usable():
    from paper_2304_11267_b200 import binding as bd
    from paper_2304_11267_b200 import build
    build.build()
    bd.load()
    a = bd.Attention()
    side = torch.cuda.Stream()
    s = side.cuda_stream
    rc, detail = bd.sd_attn_query_status(a.handle, s)
    assert rc == bd.OK and detail[0] == 0
    assert bd.sd_attn_selftest_wait_timeout(a.handle, s) == bd.OK
    rc, detail = bd.sd_attn_query_status(a.handle, s)          # synchronises the stream: the kernel has returned
    assert rc == bd.ERR_DEVICE_TIMEOUT
    assert detail == [1, 0, 99, 7]                              # code, block, wait site, tile of the waiter that gave up
    rc, detail = bd.sd_attn_query_status(a.handle, s)          # read and cleared: reported once
    assert rc == bd.OK and detail[0] == 0
    # two in a row before a query: the first record is kept
    assert bd.sd_attn_selftest_wait_timeout(a.handle, s) == bd.OK
    assert bd.sd_attn_selftest_wait_timeout(a.handle, s) == bd.OK
    assert bd.sd_attn_query_status(a.handle, s)[0] == bd.ERR_DEVICE_TIMEOUT
    assert bd.sd_attn_query_status(a.handle, s)[0] == bd.OK
    # the context and the handle work as before: the three tensor-core kernels against the oracle
    g = np.random.default_rng(3)
    for mode, (B, H, Nq, Nk, d) in ((bd.MODE_FUSED, (1, 2, 300, 500, 40)), (bd.MODE_CROSS, (1, 2, 300, 77, 40)),
                                    (bd.MODE_TWOPASS, (1, 2, 256, 256, 80))):
        q = g.standard_normal((B, H, Nq, d), dtype=np.float32).astype(np.float16)
        k = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
        v = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
        scale = float(np.float32(d ** -0.5))
        ref, _, _ = oracle.forward(q, k, v, scale)
        a.set_mode(mode)
        with torch.cuda.stream(side):
            out = a.forward(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), scale=scale,
                            stream=s)
        a.check(s)
        err = float(np.abs(out.cpu().numpy().astype(np.float64) - ref).max())
        assert err <= 2e-3 * float(np.abs(v.astype(np.float64)).max())
    assert bd.sd_attn_selftest_wait_timeout(None, s) == bd.ERR_INVALID_VALUE
    a.close()
