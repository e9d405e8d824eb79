"""Pins of the 3x3 convolution oracle (the definition behind the Winograd step, Sec. 3.3) and of Table 2's cost model.

The oracle is pinned to things other than itself: scipy's 2-D correlation (a library routine), a brute-force
evaluation in exact rational arithmetic, closed forms (delta filters, all-ones counts), linearity, and a hand-worked
example that tells correlation from flipped convolution and rows from columns.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "winograd_table2.txt")


def rand(seed, shape, dtype=np.float16):
    return np.random.default_rng(seed).standard_normal(shape, dtype=np.float32).astype(dtype)


def test_against_scipy_correlate2d():
    from scipy.signal import correlate2d
    N, H, W, C, K = 2, 9, 7, 3, 4
    x, w, b = rand(1, (N, H, W, C)), rand(2, (K, 3, 3, C)), rand(3, (K,))
    y = oracle.conv3x3_forward(x, w, b)
    xd, wd = x.astype(np.float64), w.astype(np.float64)
    for n in range(N):
        for k in range(K):
            want = sum(correlate2d(xd[n, :, :, c], wd[k, :, :, c], mode="same", boundary="fill", fillvalue=0.0)
                       for c in range(C)) + float(b[k])
            np.testing.assert_allclose(y[n, :, :, k], want, rtol=0, atol=1e-12)


def test_brute_force_in_exact_rationals():
    N, H, W, C, K = 1, 4, 5, 2, 2
    x, w = rand(4, (N, H, W, C)), rand(5, (K, 3, 3, C))
    y = oracle.conv3x3_forward(x, w)
    for i in range(H):
        for j in range(W):
            for k in range(K):
                acc = Fraction(0)
                for r in range(3):
                    for s in range(3):
                        ii, jj = i + r - 1, j + s - 1
                        if 0 <= ii < H and 0 <= jj < W:
                            for c in range(C):
                                acc += Fraction(float(x[0, ii, jj, c])) * Fraction(float(w[k, r, s, c]))
                assert abs(y[0, i, j, k] - float(acc)) <= 1e-13 * max(1.0, abs(float(acc)))


def test_delta_filters_shift_the_image():
    H, W = 6, 8
    x = rand(6, (1, H, W, 1))
    xd = x.astype(np.float64)[0, :, :, 0]
    for r in range(3):
        for s in range(3):
            w = np.zeros((1, 3, 3, 1), dtype=np.float16)
            w[0, r, s, 0] = 1.0
            y = oracle.conv3x3_forward(x, w)[0, :, :, 0]
            want = np.zeros((H, W))
            for i in range(H):
                for j in range(W):
                    ii, jj = i + r - 1, j + s - 1
                    if 0 <= ii < H and 0 <= jj < W:
                        want[i, j] = xd[ii, jj]
            np.testing.assert_array_equal(y, want)


def test_all_ones_counts_the_taps_inside_the_image():
    H, W, C = 5, 6, 7
    y = oracle.conv3x3_forward(np.ones((1, H, W, C), np.float16), np.ones((1, 3, 3, C), np.float16))[0, :, :, 0]
    assert y[0, 0] == 4 * C and y[0, W - 1] == 4 * C and y[H - 1, 0] == 4 * C      # corners
    assert y[0, 2] == 6 * C and y[2, 0] == 6 * C                                   # edges
    assert np.all(y[1:-1, 1:-1] == 9 * C)                                          # interior


def test_hand_worked_example_orientation():
    """x = [[1,2],[3,4]] (rows i, columns j), w[r][s] = 10 r + s: y[0][0] = x[0][0] w[1][1] + x[0][1] w[1][2] +
    x[1][0] w[2][1] + x[1][1] w[2][2] = 11 + 24 + 63 + 88 = 186 -- a flipped filter or swapped axes gives another
    number (flipped: 1*11 + 2*10 + 3*1 + 4*0 = 34; transposed: 11 + 2*21 + 3*12 + 88 = 177)."""
    x = np.array([[1, 2], [3, 4]], np.float16).reshape(1, 2, 2, 1)
    w = np.array([[10 * r + s for s in range(3)] for r in range(3)], np.float16).reshape(1, 3, 3, 1)
    y = oracle.conv3x3_forward(x, w)[0, :, :, 0]
    assert y[0, 0] == 186
    assert y[1, 1] == 1 * 0 + 2 * 1 + 3 * 10 + 4 * 11


def test_linearity_and_bias_and_channel_sum():
    x1, x2, w, b = rand(7, (1, 5, 5, 3)), rand(8, (1, 5, 5, 3)), rand(9, (2, 3, 3, 3)), rand(10, (2,))
    xs = (x1.astype(np.float32) + x2.astype(np.float32))
    y1, y2 = oracle.conv3x3_forward(x1, w), oracle.conv3x3_forward(x2, w)
    ys = oracle.conv3x3_forward(xs, w.astype(np.float32))
    np.testing.assert_allclose(ys, y1 + y2, rtol=0, atol=1e-12)
    yb = oracle.conv3x3_forward(x1, w, b)
    np.testing.assert_allclose(yb - y1, np.broadcast_to(b.astype(np.float64), yb.shape), rtol=0, atol=1e-12)
    # channels only meet in the sum: per-channel results add up
    parts = sum(oracle.conv3x3_forward(x1[..., c:c + 1], w[..., c:c + 1]) for c in range(3))
    np.testing.assert_allclose(parts, y1, rtol=0, atol=1e-12)


def test_bad_arguments():
    with pytest.raises(ValueError):
        oracle.conv3x3_forward(np.zeros((1, 4, 4, 3), np.float16), np.zeros((2, 3, 3, 4), np.float16))
    with pytest.raises(TypeError):
        oracle.conv3x3_forward(np.zeros((1, 4, 4, 3), np.float64), np.zeros((2, 3, 3, 3), np.float64))


def test_cost_model_reproduces_table_2():
    """Every printed cell, to the table's two decimals; the paper rounds 7.11 and 11.11 up to 7.12 and 11.12 and
    prints 1.78 as 1.8 and 1.77 (2x2 weight), so a cell may differ by one unit in its last printed digit."""
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert [int(r[0]) for r in rows] == [2, 4, 6, 8]
    for r in rows:
        m = int(r[0])
        got = oracle.winograd_cost_model(m)
        for cell, value in zip(r[1:], got):
            digits = len(cell.split(".")[1]) if "." in cell else 0
            assert abs(value - float(cell)) <= 10.0 ** -digits * 1.0001 + 1e-12, (m, cell, value)
    assert oracle.winograd_cost_model(4) == (4.0, 2.25, 4.0)     # the tile the paper selects


def test_error_level_of_the_transformed_domain_in_binary16():
    """Where the GPU test's tolerance comes from.  The algorithm for the points 0, +-1, +-2, inf, written here in double
    precision, (a) reproduces the oracle to rounding when nothing is rounded -- so the oracle is also pinned to the
    very identity the CUDA path relies on -- and (b) with the transformed filter and input rounded to binary16, as the
    tensor cores take them, lands at about 3e-3 relative L2 with its largest errors in the tile's last row and column:
    the bounds of the GPU test (6e-3, 0.08 of the output's r.m.s.) are twice that and nine sigma of the worst position."""
    BT = np.array([[4, 0, -5, 0, 1, 0], [0, -4, -4, 1, 1, 0], [0, 4, -4, -1, 1, 0],
                   [0, -2, -1, 2, 1, 0], [0, 2, -1, -2, 1, 0], [0, 4, 0, -5, 0, 1]], float)
    G = np.array([[1 / 4, 0, 0], [-1 / 6, -1 / 6, -1 / 6], [-1 / 6, 1 / 6, -1 / 6],
                  [1 / 24, 1 / 12, 1 / 6], [1 / 24, -1 / 12, 1 / 6], [0, 0, 1]], float)
    AT = np.array([[1, 1, 1, 1, 1, 0], [0, 1, -1, 2, -2, 0], [0, 1, 1, 4, 4, 0], [0, 1, -1, 8, -8, 1]], float)
    N, H, W, C, K = 1, 16, 16, 320, 24
    x = rand(31, (N, H, W, C))
    w = (np.random.default_rng(32).standard_normal((K, 3, 3, C), dtype=np.float32) / np.sqrt(9.0 * C)).astype(np.float16)
    ref = oracle.conv3x3_forward(x, w)[0]
    xp = np.zeros((H + 2, W + 2, C))
    xp[1:-1, 1:-1] = x[0].astype(np.float64)
    patches = np.stack([xp[4 * ty:4 * ty + 6, 4 * tx:4 * tx + 6] for ty in range(H // 4) for tx in range(W // 4)])
    U = np.einsum("ar,krsc,bs->kabc", G, w.astype(np.float64), G)
    V = np.einsum("ar,trsc,bs->tabc", BT, patches, BT)

    def finish(U_, V_):
        M = np.einsum("kabc,tabc->tkab", U_, V_)
        Y = np.einsum("ia,tkab,jb->tijk", AT, M, AT)
        return Y.reshape(H // 4, W // 4, 4, 4, K).transpose(0, 2, 1, 3, 4).reshape(H, W, K)

    np.testing.assert_allclose(finish(U, V), ref, rtol=0, atol=1e-12)                      # (a)
    to16 = lambda t: t.astype(np.float16).astype(np.float64)
    got = finish(to16(U * 128.0) / 128.0, to16(V))                                         # (b)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    rel = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert 1.5e-3 < rel < 4.5e-3, rel
    err = np.abs(got - ref).reshape(H // 4, 4, W // 4, 4, K)
    per_pos = np.sqrt((err ** 2).mean(axis=(0, 2, 4))) / rms
    assert per_pos[3, 3] == per_pos.max() and 4e-3 < per_pos[3, 3] < 1.4e-2, per_pos
    assert per_pos[0, 0] < 2e-3
    assert float(np.abs(got - ref).max()) < 0.08 * rms
    assert float(np.abs(V).max()) < 400 and float(np.abs(U).max() * 128.0) < 64             # binary16's range is far
