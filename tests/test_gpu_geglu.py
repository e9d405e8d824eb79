"""GPU parity of the fused GEGLU step (Sec. 3.1, Eq. 2): sd_geglu_forward through the C ABI against the fp64 oracle on
the same seeded bytes, element by element.

Tolerance, derived from the arithmetic: the kernel evaluates a * (g/2 * erfc(z')), z' = -g / sqrt 2, in binary32 and
rounds once to the output type.  erfc comes from a fitted form t * exp2(p(t) - z^2 log2 e) (6e-7 relative for z <= 2 in
binary32, `ex2.approx` and `rcp.approx` included within 1e-6 more) and three products round; the rounding of z and of
z^2 log2 e in the exponent is amplified by |z d(erfc)/dz / erfc| <= 2 z^2 = g^2 in the tail.  With
amp = 2e-6 + 2.6e-7 g^2:
  fp16:  |err| <= (2^-11 + amp) * |exact| + 2^-25      (half an ulp of binary16, half a subnormal step near zero)
  fp32:  |err| <= amp * |exact| + 1e-37
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bd():
    from paper_2304_11267_b200 import binding
    from paper_2304_11267_b200 import build
    build.build()
    binding.load()
    return binding


def check(got, x, what=""):
    want = oracle.geglu_forward(x)
    got = got.astype(np.float64)
    assert got.shape == want.shape
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    C = x.shape[-1] // 2
    gate = x[..., C:].astype(np.float64)
    amp = 2e-6 + 2.6e-7 * gate * gate
    if x.dtype == np.float16:
        tol = (2.0 ** -11 + amp) * np.abs(want) + 2.0 ** -25
    else:
        tol = amp * np.abs(want) + 1e-37
    bad = np.abs(got - want) > tol
    assert not bad.any(), "%s: %d of %d elements off, worst |err| %.3e at exact %.3e" % (
        what, int(bad.sum()), bad.size, float(np.abs(got - want)[bad].max()), float(np.abs(want)[bad].max()))


def make(seed, rows, C, dtype, spread=1.5):
    g = np.random.default_rng(seed)
    x = (g.standard_normal((rows, 2 * C), dtype=np.float32) * spread).astype(dtype)
    return x


# the feed-forward blocks of the UNet at 512 x 512, batch 2: (tokens, channels of one half)
SD_SHAPES = [(8192, 1280), (2048, 2560), (512, 5120), (128, 5120)]


@pytest.mark.parametrize("rows,C", SD_SHAPES)
@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_unet_shapes_every_element(bd, rows, C, dtype):
    if dtype == np.float32 and rows > 2048:
        rows = 2048                      # the oracle's time, not the kernel's
    x = make(100 + C, rows, C, dtype)
    out = bd.geglu(torch.from_numpy(x).cuda()).cpu().numpy()
    check(out, x, what="%d x %d" % (rows, C))


@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_awkward_sizes(bd, dtype):
    """One channel, channel counts that are not multiples of the 16-byte piece (the scalar kernel), fewer elements than
    a block, more blocks than the grid cap (grid-stride loop with a ragged tail), one row."""
    for i, (rows, C) in enumerate([(1, 1), (3, 7), (5, 8), (1, 24), (77, 12), (1000, 36), (4097, 40), (9, 100003),
                                   (3001, 1288), (70000, 16)]):
        x = make(300 + i, rows, C, dtype)
        out = bd.geglu(torch.from_numpy(x).cuda()).cpu().numpy()
        check(out, x, what="%d x %d" % (rows, C))


@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_tails_zeros_and_signs(bd, dtype):
    """Gates from far negative (GELU -> -0, where 1 + erf cancels) to far positive (GELU -> g), exact zeros of both
    signs, and the sign pattern of the product."""
    gate = np.concatenate([np.linspace(-13.0, 13.0, 4001), [0.0, -0.0, 1e-4, -1e-4, 5.5, -5.5, 9.0, -9.0]])
    gate = np.resize(gate, 4016).astype(dtype)
    for a_val in (1.0, -1.0, 0.0, 3.5, -0.013):
        x = np.empty((2, 2 * 4016), dtype=dtype)
        x[:, :4016] = dtype(a_val)
        x[:, 4016:] = gate
        out = bd.geglu(torch.from_numpy(x).cuda()).cpu().numpy()
        check(out, x, what="a = %g" % a_val)
    # GELU(g) - GELU(-g) = g holds to output rounding
    x = np.empty((1, 2 * 4016), dtype=dtype)
    x[:, :4016] = dtype(1.0)
    x[:, 4016:] = gate
    pos = bd.geglu(torch.from_numpy(x).cuda()).cpu().numpy().astype(np.float64)
    x[:, 4016:] = -gate
    neg = bd.geglu(torch.from_numpy(x).cuda()).cpu().numpy().astype(np.float64)
    eps = 2.0 ** -10 if dtype == np.float16 else 4e-6
    assert np.all(np.abs((pos - neg) - gate.astype(np.float64)) <= eps * np.maximum(np.abs(gate.astype(np.float64)), 1e-3) + 1e-7)


def test_does_not_touch_memory_around_its_output_and_is_deterministic(bd):
    rows, C = 333, 200
    x = make(7, rows, C, np.float16)
    tx = torch.from_numpy(x).cuda()
    guard = 4096
    buf = torch.full((rows * C + 2 * guard,), 123.0, dtype=torch.float16, device="cuda")
    out = buf[guard:guard + rows * C].view(rows, C)
    bd.geglu(tx, out=out)
    again = bd.geglu(tx)
    torch.cuda.synchronize()
    assert torch.equal(out, again)
    assert bool((buf[:guard] == 123.0).all()) and bool((buf[guard + rows * C:] == 123.0).all())
    check(out.cpu().numpy(), x, what="guarded output")


def test_runs_on_a_side_stream_and_in_a_cuda_graph(bd):
    x = make(8, 2048, 2560, np.float16)
    tx = torch.from_numpy(x).cuda()
    out = torch.zeros((2048, 2560), dtype=torch.float16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        assert bd.sd_geglu_forward(tx.data_ptr(), out.data_ptr(), 2048, 2560, bd.F16, side.cuda_stream) == bd.OK
    g.replay()
    torch.cuda.synchronize()
    check(out.cpu().numpy(), x, what="graph replay")


def test_argument_errors_enqueue_nothing(bd):
    x = torch.zeros((4, 32), dtype=torch.float16, device="cuda")
    out = torch.full((4, 16), 7.0, dtype=torch.float16, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    assert bd.sd_geglu_forward(x.data_ptr(), out.data_ptr(), 0, 16, bd.F16, s) == bd.OK            # no rows: no-op
    assert bd.sd_geglu_forward(0, out.data_ptr(), 4, 16, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert bd.sd_geglu_forward(x.data_ptr(), 0, 4, 16, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert bd.sd_geglu_forward(x.data_ptr(), out.data_ptr(), -1, 16, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert bd.sd_geglu_forward(x.data_ptr(), out.data_ptr(), 4, 0, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert bd.sd_geglu_forward(x.data_ptr(), out.data_ptr(), 4, 16, 5, s) == bd.ERR_UNSUPPORTED
    assert bd.sd_geglu_forward(x.data_ptr() + 2, out.data_ptr(), 4, 8, bd.F16, s) == bd.ERR_ALIGNMENT
    assert bd.sd_geglu_forward(x.data_ptr(), out.data_ptr() + 8, 4, 8, bd.F16, s) == bd.ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
