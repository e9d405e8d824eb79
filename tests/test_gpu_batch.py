"""GPU parity for sd_attn_forward_batch: independent problems of Eq. 3, those of one shape as ONE launch, the
launches spread over the library's streams.

Every problem of a batch is compared with the oracle element by element, and with the same problem run alone
(bitwise: a grouped launch does the same arithmetic in the same order for every problem, whatever else is in it).
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
    assert a.launch_count - n0 == len(SHAPES) - 2          # the two repeated shapes ride along in their twins' launches
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
    # one bad problem among good ones: its error comes back and NOTHING was enqueued (all are checked first)
    host, dev = make(23, SHAPES[:3])
    items = [(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), B, H, Nq, Nk, d, d ** -0.5)
             for (B, H, Nq, Nk, d), (tq, tk, tv, to) in zip(SHAPES[:3], dev)]
    bad = list(items[1])
    bad[8] = 1000          # head dim beyond the maximum
    rc = bd.sd_attn_forward_batch(a.handle, bd.make_problems([items[0], tuple(bad), items[2]]), bd.F16, s)
    assert rc == bd.ERR_UNSUPPORTED
    a.check()
    assert float(dev[0][3].abs().max()) == 0.0 and float(dev[2][3].abs().max()) == 0.0
    # ... and the handle is as usable as before
    assert bd.sd_attn_forward_batch(a.handle, bd.make_problems([items[0]]), bd.F16, s) == bd.OK
    a.check()
    ref, _, _ = oracle.forward(*host[0], SHAPES[0][4] ** -0.5)
    check(dev[0][3].cpu().numpy(), ref, host[0][2], "after a refused batch")
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


@pytest.mark.parametrize("opts", [{}, {"fused_shares": 1}, {"fused_shares": 1, "fused_tiles": 3}],
                         ids=lambda e: "-".join("%s=%s" % kv for kv in e.items()) or "default")
def test_groups_of_one_shape_with_different_scales(bd, opts):
    """Five problems of one self-attention shape and five of one 77-key shape, every one with its own scale (one of
    them negative, one zero): two launches, and every problem bitwise equal to the same problem run alone -- also
    when the single-pass kernel deals the key range of its units out among all SMs and combines pieces (shares)."""
    shapes = [(2, 4, 640, 1100, 40)] * 5 + [(2, 4, 640, 77, 40)] * 5 + [(1, 2, 300, 700, 80)] * 2
    scales = [40 ** -0.5, -0.2, 0.0, 0.5, 0.05, 40 ** -0.5, -0.3, 0.0, 0.4, 0.02, 80 ** -0.5, -0.1]
    host, dev = make(25, shapes)
    a = bd.Attention(options=bd.Options(**opts))
    s = torch.cuda.current_stream().cuda_stream
    items = [(tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), to.data_ptr(), B, H, Nq, Nk, d, sc)
             for (B, H, Nq, Nk, d), (tq, tk, tv, to), sc in zip(shapes, dev, scales)]
    n0 = a.launch_count
    assert bd.sd_attn_forward_batch(a.handle, bd.make_problems(items), bd.F16, s) == bd.OK
    a.check()
    assert a.launch_count - n0 == 3
    for shape, sc, (q, k, v), (tq, tk, tv, to) in zip(shapes, scales, host, dev):
        ref, _, _ = oracle.forward(q, k, v, float(np.float32(sc)))
        check(to.cpu().numpy(), ref, v, "grouped %s scale %g %s" % (shape, sc, opts))
        alone = a.forward(tq, tk, tv, scale=sc)
        a.check()
        assert torch.equal(alone, to), "grouped and single call differ for %s scale %g" % (shape, sc)
    a.close()


def test_more_problems_of_a_shape_than_one_launch_takes(bd):
    """Eleven problems of one shape: launches of eight and three (single-pass kernel), of five, five and one (77 keys)."""
    for shape, launches in (((1, 2, 200, 300, 40), 2), ((1, 2, 200, 77, 40), 3)):
        shapes = [shape] * 11
        host, dev = make(26, shapes)
        a = bd.Attention()
        s = torch.cuda.current_stream().cuda_stream
        n0 = a.launch_count
        assert bd.sd_attn_forward_batch(a.handle, problems_of(bd, shapes, dev), bd.F16, s) == bd.OK
        a.check()
        assert a.launch_count - n0 == launches
        for (q, k, v), (_, _, _, to) in zip(host, dev):
            ref, _, _ = oracle.forward(q, k, v, shape[4] ** -0.5)
            check(to.cpu().numpy(), ref, v, "eleven of %s" % (shape,))
        a.close()
