"""GPU parity of the fused group normalisation (Sec. 3.1, Eq. 1): sd_groupnorm_forward through the C ABI against the
fp64 oracle on the same seeded bytes, element by element.

Tolerance, derived from the arithmetic: the kernel takes the mean and the centred sum of squares in binary32 (512
partial sums of n/512 terms each, then a tree: relative error below 4e-6 for the group sizes here), forms
scale = rstd * gamma and shift = beta - mu * scale and writes y = x * scale + shift with one rounding to the output
type.  With r = 1 / sqrt(var + eps) of the group and X = max |x| of the group:
  |err| <= (u + 2e-5) * |exact| + 1e-5 * (X r + 1) * |gamma_c| + tiny,   u = 2^-11 (fp16) or 0 (fp32)
(the second term covers the error of the mean and the cancellation in x * scale - mu * scale when |mu| >> sigma).
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


def check(got, x, groups, eps, gamma, beta, what=""):
    want, _, rstd = oracle.groupnorm_forward(x, groups, eps, gamma, beta)
    got = got.astype(np.float64)
    assert got.shape == want.shape and np.all(np.isfinite(got)), what
    N, C = x.shape[0], x.shape[1]
    xg = np.abs(x.astype(np.float64)).reshape(N, groups, -1).max(axis=2)             # [N, G]
    per_group = 1e-5 * (xg * rstd + 1.0)                                             # [N, G]
    ga = np.abs(gamma.astype(np.float64)) if gamma is not None else np.ones(C)
    per_chan = np.repeat(per_group, C // groups, axis=1) * ga[None, :]               # [N, C]
    u = 2.0 ** -11 if x.dtype == np.float16 else 0.0
    tol = (u + 2e-5) * np.abs(want) + per_chan.reshape((N, C) + (1,) * (x.ndim - 2)) + (2.0 ** -25 if u else 1e-30)
    bad = np.abs(got - want) > tol
    assert not bad.any(), "%s: %d of %d elements off, worst |err| %.3e" % (what, int(bad.sum()), bad.size,
                                                                           float(np.abs(got - want)[bad].max()))


def make(seed, shape, dtype, scale=1.0, shift=0.0):
    g = np.random.default_rng(seed)
    x = (g.standard_normal(shape, dtype=np.float32) * scale + shift).astype(dtype)
    C = shape[1]
    gamma = (1.0 + 0.3 * g.standard_normal(C, dtype=np.float32)).astype(dtype)
    beta = (0.2 * g.standard_normal(C, dtype=np.float32)).astype(dtype)
    return x, gamma, beta


def run(bd, x, groups, eps, gamma, beta):
    t = lambda a: torch.from_numpy(a).cuda() if a is not None else None
    return bd.groupnorm(t(x), groups, eps, t(gamma), t(beta)).cpu().numpy()


# the normalisation layers of the UNet at 512 x 512, batch 2, 32 groups: (channels, height = width)
SD_SHAPES = [(320, 64), (640, 32), (1280, 16), (1280, 8), (960, 64), (1920, 32), (2560, 16), (2560, 8)]


@pytest.mark.parametrize("C,side", SD_SHAPES)
@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_unet_shapes_every_element(bd, C, side, dtype):
    x, gamma, beta = make(10 + C + side, (2, C, side, side), dtype, scale=1.7, shift=0.4)
    check(run(bd, x, 32, 1e-5, gamma, beta), x, 32, 1e-5, gamma, beta, what="%d x %d x %d" % (C, side, side))


@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_awkward_sizes_and_the_streaming_form(bd, dtype):
    """Channels that are not multiples of 16 bytes, one value per channel, one channel per group, one group, groups
    that do not fit shared memory (1 MB and 4 MB), a batch of one and of seven."""
    cases = [((1, 6, 5, 3), 3), ((7, 8, 1), 4), ((2, 32, 3, 3), 32), ((3, 12, 10, 10), 1), ((1, 64, 128, 128), 2),
             ((1, 4, 1024, 512), 1), ((2, 10, 9), 5), ((1, 2, 65536), 2)]
    for i, (shape, groups) in enumerate(cases):
        x, gamma, beta = make(40 + i, shape, dtype)
        check(run(bd, x, groups, 1e-5, gamma, beta), x, groups, 1e-5, gamma, beta, what=str(shape))


@pytest.mark.parametrize("dtype", [np.float16, np.float32], ids=["f16", "f32"])
def test_large_means_small_variances_and_optional_arguments(bd, dtype):
    # mean far from zero (cancellation in x * scale - mu * scale), tiny variance against epsilon, constant groups
    x, gamma, beta = make(60, (2, 64, 16, 16), dtype, scale=0.5, shift=30.0)
    check(run(bd, x, 32, 1e-5, gamma, beta), x, 32, 1e-5, gamma, beta, what="shifted")
    x2 = x.copy()
    x2[:, :2] = dtype(3.0)                       # one constant group per sample: xhat = 0, y = beta
    out = run(bd, x2, 32, 1e-6, gamma, beta)
    check(out, x2, 32, 1e-6, gamma, beta, what="constant group")
    for ga, be in ((None, None), (gamma, None), (None, beta)):
        check(run(bd, x, 32, 1e-3, ga, be), x, 32, 1e-3, ga, be, what="optional affine")
    check(run(bd, x, 32, 0.0, gamma, beta), x, 32, 0.0, gamma, beta, what="eps = 0")


def test_in_place_side_stream_graph_and_guard_bytes(bd):
    x, gamma, beta = make(70, (2, 320, 32, 32), np.float16)
    want_x = x.copy()
    guard = 4096
    buf = torch.full((x.size + 2 * guard,), 99.0, dtype=torch.float16, device="cuda")
    t = buf[guard:guard + x.size].view(x.shape)
    t.copy_(torch.from_numpy(x))
    tg, tb = torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda()
    side = torch.cuda.Stream()
    bd.groupnorm(t, 32, 1e-5, tg, tb)            # first call outside the capture (it raises the shared-memory limit)
    t.copy_(torch.from_numpy(x))
    torch.cuda.synchronize()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        assert bd.sd_groupnorm_forward(t.data_ptr(), tg.data_ptr(), tb.data_ptr(), t.data_ptr(), 2, 320, 1024, 32, 1e-5,
                                       bd.F16, side.cuda_stream) == bd.OK          # in place
    t.copy_(torch.from_numpy(x))                 # (the capture did not run the kernel)
    g.replay()
    torch.cuda.synchronize()
    check(t.cpu().numpy(), want_x, 32, 1e-5, gamma, beta, what="in place, graph replay")
    assert bool((buf[:guard] == 99.0).all()) and bool((buf[guard + x.size:] == 99.0).all())


def test_argument_errors_enqueue_nothing(bd):
    x = torch.zeros((2, 8, 16), dtype=torch.float16, device="cuda")
    y = torch.full((2, 8, 16), 7.0, dtype=torch.float16, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    f = bd.sd_groupnorm_forward
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 0, 8, 16, 4, 1e-5, bd.F16, s) == bd.OK                  # no samples
    assert f(0, 0, 0, y.data_ptr(), 2, 8, 16, 4, 1e-5, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), 0, 0, 0, 2, 8, 16, 4, 1e-5, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 2, 8, 16, 3, 1e-5, bd.F16, s) == bd.ERR_INVALID_VALUE    # 8 % 3
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 2, 8, 0, 4, 1e-5, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 2, 8, 16, 4, -1.0, bd.F16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 2, 8, 16, 4, float("nan"), bd.F16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), 0, 0, y.data_ptr(), 2, 8, 16, 4, 1e-5, 9, s) == bd.ERR_UNSUPPORTED
    assert f(x.data_ptr() + 2, 0, 0, y.data_ptr(), 2, 8, 8, 4, 1e-5, bd.F16, s) == bd.ERR_ALIGNMENT
    assert f(x.data_ptr(), x.data_ptr() + 1, 0, y.data_ptr(), 2, 8, 16, 4, 1e-5, bd.F16, s) == bd.ERR_ALIGNMENT
    torch.cuda.synchronize()
    assert bool((y == 7.0).all())
