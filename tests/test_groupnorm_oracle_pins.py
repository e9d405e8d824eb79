"""Pins for the group-normalisation oracle (no GPU needed).

Eq. 1 of the paper is the textbook operation, so the oracle is pinned to numpy's mean and variance on the reshaped
tensor (a library routine, another formulation: one-pass reshape instead of the oracle's loops), to closed forms
(a ramp's mean and variance, constant input, a two-valued group), to the invariances the operation has (shift and
scale of the input, independence of groups and samples), and to where gamma and beta apply (per CHANNEL, not per
group).  A variance with the wrong divisor, a group made of strided instead of consecutive channels, an epsilon outside
the root or an affine per group each fail at least one of them.
"""
import numpy as np
import pytest

import oracle


def rand(seed, shape, dtype=np.float32, scale=1.0, shift=0.0):
    g = np.random.default_rng(seed)
    return (g.standard_normal(shape) * scale + shift).astype(dtype)


@pytest.mark.parametrize("dtype", [np.float16, np.float32])
@pytest.mark.parametrize("shape,groups", [((2, 8, 5, 3), 4), ((3, 12, 7), 3), ((1, 32, 4, 4), 32), ((2, 6, 1), 1)])
def test_against_numpy_mean_and_variance_of_the_reshaped_tensor(dtype, shape, groups):
    x = rand(1, shape, dtype, scale=2.0, shift=0.7)
    C = shape[1]
    gamma, beta = rand(2, (C,), dtype), rand(3, (C,), dtype)
    eps = 1e-5
    y, mean, rstd = oracle.groupnorm_forward(x, groups, eps, gamma, beta)
    xd = x.astype(np.float64).reshape(shape[0], groups, -1)
    mu = xd.mean(axis=2)
    var = xd.var(axis=2)                       # numpy's default: the biased variance
    np.testing.assert_allclose(mean, mu, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(rstd, 1.0 / np.sqrt(var + eps), rtol=1e-13)
    xhat = ((xd - mu[..., None]) / np.sqrt(var + eps)[..., None]).reshape(x.shape)
    bshape = (1, C) + (1,) * (x.ndim - 2)
    want = xhat * gamma.astype(np.float64).reshape(bshape) + beta.astype(np.float64).reshape(bshape)
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-14)


def test_closed_forms():
    # a ramp 0..n-1 in one group: mean (n-1)/2, biased variance (n^2-1)/12
    n = 48
    x = np.arange(n, dtype=np.float32).reshape(1, 4, 12)
    y, mean, rstd = oracle.groupnorm_forward(x, 1, 0.0)
    assert mean[0, 0] == pytest.approx((n - 1) / 2, rel=1e-15)
    assert rstd[0, 0] == pytest.approx(1.0 / np.sqrt((n * n - 1) / 12.0), rel=1e-14)
    assert y.ravel()[0] == pytest.approx(-(n - 1) / 2 / np.sqrt((n * n - 1) / 12.0), rel=1e-14)
    # constant input: xhat = 0 whatever epsilon is (as long as it is positive), output = beta
    x = np.full((2, 4, 9), 3.25, dtype=np.float16)
    beta = np.array([1.0, -2.0, 0.5, 0.0], dtype=np.float16)
    y, mean, rstd = oracle.groupnorm_forward(x, 2, 1e-5, None, beta)
    assert np.all(mean == 3.25) and np.allclose(rstd, 1.0 / np.sqrt(1e-5))
    np.testing.assert_array_equal(y, np.broadcast_to(beta.astype(np.float64)[None, :, None], y.shape))
    # a group of +1 and -1 in equal numbers: mean 0, variance 1, xhat = x / sqrt(1 + eps)
    x = np.tile(np.array([1.0, -1.0], dtype=np.float32), 8).reshape(1, 2, 8)
    y, mean, rstd = oracle.groupnorm_forward(x, 1, 0.21)
    assert mean[0, 0] == 0.0 and rstd[0, 0] == pytest.approx(1 / np.sqrt(1.21), rel=1e-15)
    np.testing.assert_allclose(y, x / np.sqrt(1.21), rtol=1e-15)


def test_invariances():
    x = rand(5, (2, 8, 6, 6), np.float32)
    y0, _, _ = oracle.groupnorm_forward(x, 4, 0.0)
    # shifting and scaling the input leaves xhat alone (epsilon 0; powers of two so the stored values shift exactly)
    y1, _, _ = oracle.groupnorm_forward((x * np.float32(4.0)).astype(np.float32), 4, 0.0)
    np.testing.assert_allclose(y1, y0, rtol=1e-12, atol=1e-13)
    # every group has mean 0 and variance 1
    yg = y0.reshape(2, 4, -1)
    np.testing.assert_allclose(yg.mean(axis=2), 0.0, atol=1e-14)
    np.testing.assert_allclose(yg.var(axis=2), 1.0, rtol=1e-12)
    # groups and samples are independent: changing one group changes only that group
    x2 = x.copy()
    x2[1, 2:4] += np.float32(5.0)            # channels 2, 3 of sample 1 = group 1 (consecutive channels)
    y2, _, _ = oracle.groupnorm_forward(x2, 4, 0.0)
    same = np.ones(y0.shape, dtype=bool)
    same[1, 2:4] = False
    np.testing.assert_array_equal(y2[same], y0[same])
    # (a shift of the whole group leaves its xhat alone, up to the binary32 rounding of the shifted inputs)
    np.testing.assert_allclose(y2[1, 2:4], y0[1, 2:4], rtol=1e-5, atol=2e-6)


def test_affine_is_per_channel_and_epsilon_is_inside_the_root():
    x = rand(6, (1, 4, 10), np.float32)
    gamma = np.array([1.0, 2.0, 3.0, 4.0], dtype=np.float32)
    beta = np.array([0.5, 0.0, -0.5, 1.0], dtype=np.float32)
    plain, _, _ = oracle.groupnorm_forward(x, 2, 1e-3)
    y, _, _ = oracle.groupnorm_forward(x, 2, 1e-3, gamma, beta)
    for c in range(4):
        np.testing.assert_allclose(y[0, c], plain[0, c] * float(gamma[c]) + float(beta[c]), rtol=1e-15, atol=1e-16)
    # epsilon: rstd = 1 / sqrt(var + eps), not 1 / (sqrt(var) + eps)
    _, _, r = oracle.groupnorm_forward(x, 2, 0.5)
    var = x.astype(np.float64).reshape(1, 2, -1).var(axis=2)
    np.testing.assert_allclose(r, 1 / np.sqrt(var + 0.5), rtol=1e-14)
    assert not np.allclose(r, 1 / (np.sqrt(var) + 0.5), rtol=1e-3)


def test_arguments():
    x = np.zeros((2, 6, 4), dtype=np.float16)
    with pytest.raises(ValueError):
        oracle.groupnorm_forward(x, 4, 1e-5)                        # 6 channels do not divide into 4 groups
    with pytest.raises(ValueError):
        oracle.groupnorm_forward(x, 3, 1e-5, np.zeros(5, dtype=np.float16))
    with pytest.raises(TypeError):
        oracle.groupnorm_forward(x.astype(np.float64), 3, 1e-5)
    y, m, r = oracle.groupnorm_forward(np.zeros((0, 6, 4), dtype=np.float16), 3, 1e-5)
    assert y.shape == (0, 6, 4) and m.shape == (0, 3)
