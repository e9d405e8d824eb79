"""GPU parity of the Winograd 3x3 convolution (Sec. 3.3) against the oracle: the directly evaluated convolution
in double precision on the same fp16 values.

Tolerance, from the arithmetic (binary16 U and V, binary32 accumulation, binary16 output).  Rounding the transformed
input V and filter U to binary16 puts a relative error of at most 2^-11 (uniform: 2.8e-4 r.m.s.) on each factor of
each of the 36 * C products of an output tile; the output transform A^T . A weighs the 36 partial sums with
coefficients up to 64 (the tile's last row and column take 8 x 8 on one of them) while the wanted output is their
heavily cancelling sum.  For independent inputs that comes to an error of about 1e-3 (first rows and columns) to
9e-3 (last corner) of the output's r.m.s. per element, 3e-3 in relative L2 (emulated in double precision with
rounded U and V; the transformed values of standard-normal inputs reach 190, of the filter 1/16 of the weights').
The output's own rounding adds 2^-11 |y|.  Bounds used: relative L2 <= 6e-3 (twice the estimate) and
max |err| <= 0.065 * rms(y) + 2^-11 |y| (seven sigma of the worst position; measured at most 0.054); measured values are printed.
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL_L2 = 6e-3
MAX_ABS_OF_RMS = 0.065


@pytest.fixture(scope="module")
def bd():
    from paper_2304_11267_b200 import binding
    from paper_2304_11267_b200 import build
    build.build()
    binding.load()
    return binding


def make(seed, N, H, W, C, K, bias=True):
    g = np.random.default_rng(seed)
    x = g.standard_normal((N, H, W, C), dtype=np.float32).astype(np.float16)
    w = (g.standard_normal((K, 3, 3, C), dtype=np.float32) / np.sqrt(9.0 * C)).astype(np.float16)
    b = (0.1 * g.standard_normal((K,), dtype=np.float32)).astype(np.float16) if bias else None
    return x, w, b


def run(bd, x, w, b):
    layer = bd.WinogradConv3x3(torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda() if b is not None else None)
    y = layer(torch.from_numpy(x).cuda())
    rc, detail = bd.sd_winograd_query_status()
    assert rc == bd.OK, detail
    return y.cpu().numpy()


def check(got, ref, what):
    got = got.astype(np.float64)
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(got - ref)
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    bound = MAX_ABS_OF_RMS * rms + 2.0 ** -11 * np.abs(ref)
    assert np.all(err <= bound), "%s: max err %.3e (rms of y %.3e)" % (what, float(err.max()), rms)
    assert rel <= REL_L2, "%s: rel L2 %.3e" % (what, rel)
    print("winograd %-34s max|err|/rms(y) %.2e  rel L2 %.2e" % (what, float(err.max()) / rms, rel))


# The UNet's 3x3 layer sizes at reduced resolution, ragged images (H, W not multiples of 4: partial tiles), one tile,
# a single-row image, channel counts that leave partial 64-column chunks (C = 40, 200) and partial 16-column
# accumulator groups (K = 24, 328), K above one accumulator (320 -> 2 x 160, 640 -> 3 x 224), more tiles than one
# 128-row GEMM tile and a ragged last one.
@pytest.mark.parametrize("N,H,W,C,K", [
    (2, 32, 32, 320, 320), (1, 16, 16, 640, 640), (1, 8, 8, 1280, 1280), (1, 32, 32, 8, 320),
    (1, 13, 10, 40, 24), (3, 7, 9, 200, 328), (1, 4, 4, 64, 64), (1, 1, 5, 16, 16), (1, 3, 3, 8, 8),
    (1, 50, 46, 64, 32), (5, 12, 12, 128, 256),
])
def test_against_the_direct_convolution(bd, N, H, W, C, K):
    x, w, b = make(100 + H + C + K, N, H, W, C, K)
    ref = oracle.conv3x3_forward(x, w, b)
    check(run(bd, x, w, b), ref, str((N, H, W, C, K)))


def test_without_bias_and_with_a_delta_filter(bd):
    """A centre-tap filter makes the convolution the identity: the transformed domain must give x back (to the
    stated error), including the zero border's effect on edge tiles."""
    N, H, W, C = 1, 10, 14, 16
    x, _, _ = make(7, N, H, W, C, C, bias=False)
    w = np.zeros((C, 3, 3, C), dtype=np.float16)
    for c in range(C):
        w[c, 1, 1, c] = 1.0
    ref = oracle.conv3x3_forward(x, w)
    np.testing.assert_array_equal(ref, x.astype(np.float64))
    check(run(bd, x, w, None), ref, "identity filter")


def test_small_weights_stay_out_of_the_subnormals(bd):
    """Weights of size 1e-3: the transformed filter's smallest entries (x 1/576) would be binary16 subnormals without
    the factor the filter transform carries."""
    x, w, b = make(9, 1, 16, 16, 64, 64)
    w = (w.astype(np.float32) * 0.02).astype(np.float16)
    ref = oracle.conv3x3_forward(x, w, b)
    got = run(bd, x, w, b).astype(np.float64)
    ref0 = oracle.conv3x3_forward(x, w)            # the bias is exact: measure the convolution part against its own scale
    err = np.abs((got - ref))
    rms = float(np.sqrt(np.mean(ref0 ** 2)))
    assert np.all(err <= MAX_ABS_OF_RMS * rms + 2.0 ** -10 * np.abs(ref)), (float(err.max()), rms)


def test_arguments(bd):
    s = torch.cuda.current_stream().cuda_stream
    x = torch.zeros(1, 8, 8, 16, dtype=torch.float16, device="cuda")
    U = torch.zeros(bd.sd_winograd_filter_elems(16, 16), dtype=torch.float16, device="cuda")
    y = torch.zeros(1, 8, 8, 16, dtype=torch.float16, device="cuda")
    need = bd.sd_winograd_workspace_bytes(1, 8, 8, 16, 16)
    assert need == 36 * 4 * 16 * 2 + 36 * 4 * 16 * 4
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    f = bd.sd_winograd_conv3x3_forward
    assert f(x.data_ptr(), U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need, 1, 8, 8, 16, 16, s) == bd.OK
    assert f(x.data_ptr(), U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need - 1, 1, 8, 8, 16, 16, s) == bd.ERR_WORKSPACE
    assert f(x.data_ptr(), U.data_ptr(), 0, y.data_ptr(), 0, 0, 1, 8, 8, 16, 16, s) == bd.ERR_WORKSPACE
    assert f(x.data_ptr(), U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need, 1, 8, 8, 12, 16, s) == bd.ERR_UNSUPPORTED
    assert f(0, U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need, 1, 8, 8, 16, 16, s) == bd.ERR_INVALID_VALUE
    assert f(x.data_ptr(), U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need, 0, 8, 8, 16, 16, s) == bd.OK
    assert f(x.data_ptr() + 2, U.data_ptr(), 0, y.data_ptr(), ws.data_ptr(), need, 1, 8, 8, 16, 16, s) == bd.ERR_ALIGNMENT
    assert bd.sd_winograd_transform_filter(0, U.data_ptr(), 16, 16, s) == bd.ERR_INVALID_VALUE
    assert bd.sd_winograd_workspace_bytes(1, 0, 8, 16, 16) == 0
    rc, _ = bd.sd_winograd_query_status()
    assert rc == bd.OK
