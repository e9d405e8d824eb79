"""The allocation-free two-pass entry point (collected last on purpose: see the file name).

Some users of the library cannot call cudaMalloc -- the device heap belongs to a host framework, or
allocations are banned on their latency path -- so they can neither create a handle nor lend a
workspace.  ``sd_attn_forward_twopass_static`` serves them from a scratch array built into the library.
This test drives it through the C ABI, twice in a row (the second call reuses the array the first one
dirtied, with a different shape).  The handle-based two-pass path runs the same two kernels on the same
bytes, so the two results must be EQUAL bit for bit; the result is also held against the oracle within the
tolerance of the parity tests, the device's free memory must not move across a call, and the status word
beside the array must read "ok".
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F16_ABS = 2e-3   # the fp16 tolerance of the parity tests: max |err| <= 2e-3 * max|V|


def rand_qkv(seed, B, H, Nq, Nk, d, qmult=1.0):
    g = np.random.default_rng(seed)
    q = (g.standard_normal((B, H, Nq, d), dtype=np.float32) * qmult).astype(np.float16)
    k = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
    v = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
    return q, k, v


def test_static_scratch_entry_point_matches_the_workspace_path_twice_in_a_row():
    from paper_2304_11267_b200 import binding as bd
    from paper_2304_11267_b200 import build
    build.build()
    bd.load()
    att = bd.Attention(bd.MODE_TWOPASS)
    stream = torch.cuda.current_stream().cuda_stream
    # first a large call that fills most of the built-in array, then a small ragged one on top of its leftovers
    shapes = [(1, 8, 1024, 1024, 40, 1.0), (2, 3, 200, 333, 80, 4.0)]
    for n, (B, H, Nq, Nk, d, qmult) in enumerate(shapes):
        assert bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, B, H, Nq, Nk, d, bd.F16) <= bd.STATIC_MAX_SCRATCH
        q, k, v = rand_qkv(77 + n, B, H, Nq, Nk, d, qmult)
        tq, tk, tv = (torch.from_numpy(x).cuda() for x in (q, k, v))
        scale = float(np.float32(1.0 / np.sqrt(d)))
        expect = att.forward(tq, tk, tv, scale=scale)
        att.check()
        got = torch.full_like(tq, float("nan"))
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        rc = bd.sd_attn_forward_twopass_static(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), got.data_ptr(),
                                               B, H, Nq, Nk, d, scale, bd.F16, stream)
        assert rc == bd.OK, bd.status_string(rc)
        rc, detail = bd.sd_attn_static_query_status(stream)      # synchronises the stream
        assert rc == bd.OK, detail
        if n > 0:   # (the first call on a device loads the kernels and looks the array up: see the header)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert torch.equal(got, expect), "call %d differs from the workspace path, which runs the same kernels" % n
        a = got.cpu().numpy().astype(np.float64)
        ref, _, _ = oracle.forward(q, k, v, scale)
        assert np.all(np.isfinite(a))
        vmax = float(np.abs(v.astype(np.float64)).max())
        assert np.abs(a - ref).max() <= F16_ABS * vmax, "call %d differs from the oracle" % n
    att.close()


def test_static_scratch_entry_point_rejects_oversized_and_unsupported_calls():
    from paper_2304_11267_b200 import binding as bd
    bd.load()
    q = torch.zeros(16, dtype=torch.float16, device="cuda")
    p = q.data_ptr()
    # 16 heads x 4096 x 4096 scores need 1 GiB: far beyond the built-in array -> refused, nothing enqueued
    assert bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, 2, 8, 4096, 4096, 40, bd.F16) > bd.STATIC_MAX_SCRATCH
    assert bd.sd_attn_forward_twopass_static(p, p, p, p, 2, 8, 4096, 4096, 40, 0.1, bd.F16) == bd.ERR_WORKSPACE
    assert bd.sd_attn_forward_twopass_static(p, p, p, p, 1, 1, 64, 64, 40, 0.1, bd.F32) == bd.ERR_UNSUPPORTED
    assert bd.sd_attn_forward_twopass_static(p, p, p, p, 1, 1, 64, 64, 36, 0.1, bd.F16) == bd.ERR_UNSUPPORTED
    assert bd.sd_attn_forward_twopass_static(0, p, p, p, 1, 1, 64, 64, 40, 0.1, bd.F16) == bd.ERR_INVALID_VALUE
    assert bd.sd_attn_forward_twopass_static(p, p, p, p, 1, 1, 0, 64, 40, 0.1, bd.F16) == bd.OK
    torch.cuda.synchronize()
