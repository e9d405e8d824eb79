"""GPU parity for sd_attn_forward_batch: independent problems of Eq. 3 spread over the library's streams.

Every problem of a batch is compared with the oracle element by element, and with the same problem run alone
(bitwise: the batch call launches the same kernels, only on other streams).
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F16_ABS = 2e-3
F16_REL_L2 = 2e-3

# a UNet step's mix at a quarter of the tokens: (B, H, Nq, Nk, d)
SHAPES = [(2, 8, 1024, 1024, 40), (2, 8, 1024, 77, 40), (2, 8, 256, 256, 80), (2, 8, 256, 77, 80),
          (2, 8, 64, 64, 160), (2, 8, 64, 77, 160), (2, 8, 16, 16, 160), (2, 8, 16, 77, 160),
          (2, 8, 1024, 1024, 40), (2, 8, 1024, 77, 40), (1, 3, 200, 50, 24)]


@pytest.fixture(scope="module")
def bd():
    from paper_2304_11267_b200 import binding
    from paper_2304_11267_b200 import build
    build.build()
    binding.load()
    return binding


def make(seed, shapes):
    g = np.random.default_rng(seed)
    host, dev = [], []
    for (B, H, Nq, Nk, d) in shapes:
        q = g.standard_normal((B, H, Nq, d), dtype=np.float32).astype(np.float16)
        k = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
        v = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(np.float16)
        host.append((q, k, v))
        tq, tk, tv = (torch.from_numpy(x).cuda() for x in (q, k, v))
        dev.append((tq, tk, tv, torch.zeros_like(tq)))
    return host, dev


def problems_of(bd, shapes, dev):
    return bd.make_problems([(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), B, H, Nq, Nk, d, d ** -0.5)
                             for (B, H, Nq, Nk, d), (tq, tk, tv, to) in zip(shapes, dev)])


def check(got, ref, v, what):
    got = got.astype(np.float64)
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    vmax = float(np.abs(v.astype(np.float64)).max())
    err = float(np.abs(got - ref).max())
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    assert err <= F16_ABS * vmax, "%s: max abs err %.3e > %.3e" % (what, err, F16_ABS * vmax)
    assert rel <= F16_REL_L2, "%s: rel L2 err %.3e" % (what, rel)


def test_batch_against_the_oracle_and_the_single_calls(bd):
    host, dev = make(21, SHAPES)
    a = bd.Attention()
    s = torch.cuda.current_stream().cuda_stream
    n0 = a.launch_count
    assert bd.sd_attn_forward_batch(a.handle, problems_of(bd, SHAPES, dev), bd.F16, s) == bd.OK
    a.check()
    assert a.launch_count - n0 == len(SHAPES)
    for shape, (q, k, v), (tq, tk, tv, to) in zip(SHAPES, host, dev):
        ref, _, _ = oracle.forward(q, k, v, shape[4] ** -0.5)
        check(to.cpu().numpy(), ref, v, "batch %s" % (shape,))
        alone = a.forward(tq, tk, tv)
        a.check()
        assert torch.equal(alone, to), "batch and single call differ for %s" % (shape,)
    a.close()


def test_batch_in_a_cuda_graph(bd):
    host, dev = make(22, SHAPES[:6])
    a = bd.Attention()
    probs = problems_of(bd, SHAPES[:6], dev)
    side = torch.cuda.Stream()
    assert bd.sd_attn_forward_batch(a.handle, probs, bd.F16, side.cuda_stream) == bd.OK   # warm the tensor-map cache
    a.check(side.cuda_stream)
    for (_, _, _, to) in dev:
        to.zero_()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            assert bd.sd_attn_forward_batch(a.handle, probs, bd.F16, side.cuda_stream) == bd.OK
    for (_, _, _, to) in dev:
        assert float(to.abs().max()) == 0.0     # captured, not run
    g.replay()
    torch.cuda.synchronize()
    a.check()
    for shape, (q, k, v), (_, _, _, to) in zip(SHAPES[:6], host, dev):
        ref, _, _ = oracle.forward(q, k, v, shape[4] ** -0.5)
        check(to.cpu().numpy(), ref, v, "graph batch %s" % (shape,))
    a.close()


def test_batch_edges(bd):
    a = bd.Attention()
    s = torch.cuda.current_stream().cuda_stream
    assert bd.sd_attn_forward_batch(a.handle, bd.make_problems([]), bd.F16, s) == bd.OK
    assert bd.load().sd_attn_forward_batch(a.handle, None, 2, bd.F16, None) == bd.ERR_INVALID_VALUE
    assert bd.load().sd_attn_forward_batch(a.handle, None, -1, bd.F16, None) == bd.ERR_INVALID_VALUE
    # one bad problem among good ones: its error comes back, the good ones before it have run, the stream is usable
    host, dev = make(23, SHAPES[:3])
    items = [(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), B, H, Nq, Nk, d, d ** -0.5)
             for (B, H, Nq, Nk, d), (tq, tk, tv, to) in zip(SHAPES[:3], dev)]
    bad = list(items[1])
    bad[8] = 1000          # head dim beyond the maximum
    rc = bd.sd_attn_forward_batch(a.handle, bd.make_problems([items[0], tuple(bad), items[2]]), bd.F16, s)
    assert rc == bd.ERR_UNSUPPORTED
    a.check()
    ref, _, _ = oracle.forward(*host[0], SHAPES[0][4] ** -0.5)
    check(dev[0][3].cpu().numpy(), ref, host[0][2], "the problem before the bad one")
    assert float(dev[2][3].abs().max()) == 0.0   # the one after it was not enqueued
    # a problem with no query rows is an OK no-op inside a batch as well
    empty = list(items[2])
    empty[6] = 0
    assert bd.sd_attn_forward_batch(a.handle, bd.make_problems([tuple(empty), items[2]]), bd.F16, s) == bd.OK
    a.check()
    ref, _, _ = oracle.forward(*host[2], SHAPES[2][4] ** -0.5)
    check(dev[2][3].cpu().numpy(), ref, host[2][2], "beside an empty problem")
    a.close()


def test_batch_twopass_runs_in_order(bd):
    """TWOPASS lends one workspace to every problem: the batch must not overlap them."""
    shapes = [(1, 4, 256, 256, 40), (1, 4, 256, 77, 40), (1, 4, 128, 128, 80)]
    host, dev = make(24, shapes)
    a = bd.Attention(mode=bd.MODE_TWOPASS)
    need = max(bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, B, H, Nq, Nk, d, bd.F16) for (B, H, Nq, Nk, d) in shapes)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert bd.sd_attn_set_workspace(a.handle, ws.data_ptr(), need) == bd.OK
    s = torch.cuda.current_stream().cuda_stream
    assert bd.sd_attn_forward_batch(a.handle, problems_of(bd, shapes, dev), bd.F16, s) == bd.OK
    a.check()
    for shape, (q, k, v), (_, _, _, to) in zip(shapes, host, dev):
        ref, _, _ = oracle.forward(q, k, v, shape[4] ** -0.5)
        check(to.cpu().numpy(), ref, v, "two-pass batch %s" % (shape,))
    a.close()
