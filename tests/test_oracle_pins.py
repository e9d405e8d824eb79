"""Pins for the CPU oracle (no GPU needed).

The paper prints no worked numeric example of an attention output (its figures are
schematic), so the oracle is pinned to what the definition (Eq. 3, Eq. 4) and mathematics
fix instead: closed forms, a brute-force evaluation in another formulation and another
arithmetic (50-digit decimals, no max subtraction), invariants of softmax attention, and
scipy's softmax as an independent library routine.  Each pin is chosen so that a dropped
term, a wrong sign, a missing scale or a transposed operand fails at least one of them.
"""
import math
import os
from decimal import Decimal, getcontext

import numpy as np
import pytest
import scipy.special

import oracle
from paper_2304_11267_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def rand_qkv(seed, B, H, Nq, Nk, d, dtype=np.float16, qmult=1.0):
    g = rng(seed)
    q = (g.standard_normal((B, H, Nq, d), dtype=np.float32) * qmult).astype(dtype)
    k = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(dtype)
    v = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(dtype)
    return q, k, v


# ---------------------------------------------------------------- the binary16 decoder

def test_half_decoder_matches_numpy_on_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    mine = oracle.half_to_double(bits)
    ref = bits.view(np.float16).astype(np.float64)
    finite = np.isfinite(ref)
    assert np.array_equal(mine[finite], ref[finite])
    assert np.array_equal(np.signbit(mine[finite]), np.signbit(ref[finite]))
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    assert np.array_equal(np.isinf(mine), np.isinf(ref))
    assert np.array_equal(mine[np.isinf(ref)], ref[np.isinf(ref)])


# ---------------------------------------------------------------- closed forms

def read_golden_closed_forms():
    cases = []
    with open(os.path.join(GOLDEN, "closed_forms.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, scale, qs, ks, vs, expect = [p.strip() for p in line.split("|")]
            cases.append((name, float(scale),
                          [float(x) for x in qs.split()], [float(x) for x in ks.split()],
                          [float(x) for x in vs.split()], float(expect)))
    return cases


@pytest.mark.parametrize("case", read_golden_closed_forms(), ids=lambda c: c[0])
def test_golden_closed_forms_d1(case):
    """d = 1, one query: out = sum_j exp(s q k_j) v_j / sum_j exp(s q k_j), worked by hand."""
    _, scale, qs, ks, vs, expect = case
    q = np.array(qs, dtype=np.float32).reshape(1, 1, 1, 1)
    k = np.array(ks, dtype=np.float32).reshape(1, 1, -1, 1)
    v = np.array(vs, dtype=np.float32).reshape(1, 1, -1, 1)
    out, L, S = oracle.forward(q, k, v, scale)
    assert out.shape == (1, 1, 1, 1)
    # inputs are binary32 roundings of ln 2, ln 3: agreement to 1e-6 relative is all they allow
    assert out[0, 0, 0, 0] == pytest.approx(expect, rel=1e-6, abs=1e-7)


def test_two_keys_is_a_sigmoid_mixture():
    g = rng(11)
    for _ in range(20):
        d = int(g.integers(1, 9))
        q = g.standard_normal((1, 1, 1, d)).astype(np.float32)
        k = g.standard_normal((1, 1, 2, d)).astype(np.float32)
        v = g.standard_normal((1, 1, 2, d)).astype(np.float32)
        s = np.float32(g.uniform(-2, 2))
        a = [float(s) * sum(float(q[0, 0, 0, c]) * float(k[0, 0, j, c]) for c in range(d))
             for j in range(2)]
        w = 1.0 / (1.0 + math.exp(-(a[0] - a[1])))
        expect = w * v[0, 0, 0].astype(np.float64) + (1 - w) * v[0, 0, 1].astype(np.float64)
        out, L, S = oracle.forward(q, k, v, s)
        np.testing.assert_allclose(out[0, 0, 0], expect, rtol=1e-13, atol=1e-14)
        assert L[0, 0, 0] == pytest.approx(max(a), rel=1e-15)
        assert S[0, 0, 0] == pytest.approx(1.0 + math.exp(-abs(a[0] - a[1])), rel=1e-14)


def test_zero_queries_give_the_column_mean_of_v():
    _, k, v = rand_qkv(3, 2, 3, 5, 37, 8)
    q = np.zeros((2, 3, 5, 8), dtype=np.float16)
    out, L, S = oracle.forward(q, k, v, 0.7)
    mean = v.astype(np.float64).mean(axis=2, keepdims=True)
    np.testing.assert_allclose(out, np.broadcast_to(mean, out.shape), rtol=1e-14, atol=1e-15)
    assert np.all(L == 0.0)
    np.testing.assert_allclose(S, 37.0, rtol=0, atol=0)


def test_single_key_returns_its_value_row_exactly():
    q, k, v = rand_qkv(4, 2, 2, 9, 1, 40)
    out, L, S = oracle.forward(q, k, v, workloads.Call("x", 2, 2, 9, 1, 40, 0).scale())
    assert np.array_equal(out, np.broadcast_to(v.astype(np.float64), out.shape))
    assert np.all(S == 1.0)


# ---------------------------------------------------------------- brute force, other formulation

def brute_force_decimal(q, k, v, scale):
    """o = sum_j exp(a_j) v_j / sum_j exp(a_j): no max shift, 50-digit decimals, c outermost."""
    getcontext().prec = 50
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    s = Decimal(float(np.float32(scale)))
    out = np.zeros((B, H, Nq, d))
    for c in range(d):
        for i in range(Nq):
            for h in range(H):
                for b in range(B):
                    num, den = Decimal(0), Decimal(0)
                    for j in reversed(range(Nk)):
                        dot = Decimal(0)
                        for t in reversed(range(d)):
                            dot += Decimal(float(q[b, h, i, t])) * Decimal(float(k[b, h, j, t]))
                        w = (s * dot).exp()
                        num += w * Decimal(float(v[b, h, j, c]))
                        den += w
                    out[b, h, i, c] = float(num / den)
    return out


@pytest.mark.parametrize("dtype", [np.float16, np.float32])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1), (2, 1, 3, 5, 2), (1, 2, 8, 7, 4), (2, 2, 4, 8, 3)])
def test_matches_decimal_brute_force(shape, dtype):
    B, H, Nq, Nk, d = shape
    q, k, v = rand_qkv(100 + sum(shape), B, H, Nq, Nk, d, dtype, qmult=2.0)
    scale = np.float32(0.61)
    out, _, _ = oracle.forward(q, k, v, scale)
    np.testing.assert_allclose(out, brute_force_decimal(q, k, v, scale), rtol=1e-13, atol=1e-14)


def test_large_logits_do_not_overflow_and_match_decimal():
    """Logits near +-200: exp(a) alone overflows nothing in decimals; the shifted form must agree."""
    q = np.full((1, 1, 2, 2), 16.0, dtype=np.float16)
    q[0, 0, 1] = -16.0
    k = np.array([[[[6.0, 6.5], [5.5, 6.0], [-6.0, -6.0], [0.0, 0.0]]]], dtype=np.float16)
    v = np.array([[[[1.0, -2.0], [3.0, 0.5], [-7.0, 4.0], [0.25, 8.0]]]], dtype=np.float16)
    out, L, S = oracle.forward(q, k, v, 1.0)
    np.testing.assert_allclose(out, brute_force_decimal(q, k, v, 1.0), rtol=1e-13)
    assert L[0, 0, 0] == 200.0 and L[0, 0, 1] == 192.0


# ---------------------------------------------------------------- invariants of the definition

def test_rows_of_p_sum_to_one_and_reproduce_the_output():
    q, k, v = rand_qkv(5, 2, 2, 6, 19, 5, qmult=3.0)
    out, L, S, P = oracle.forward(q, k, v, 0.5, want_probs=True)
    np.testing.assert_allclose(P.sum(axis=-1), 1.0, rtol=0, atol=1e-15)
    assert np.all(P >= 0)
    np.testing.assert_allclose(np.einsum("bhij,bhjc->bhic", P, v.astype(np.float64)), out,
                               rtol=1e-13, atol=1e-15)
    # the largest weight of each row sits where the logit is largest and equals 1/S
    np.testing.assert_allclose(P.max(axis=-1), 1.0 / S, rtol=1e-15)


def test_identical_keys_give_the_mean_of_v():
    q, k, v = rand_qkv(6, 1, 2, 7, 13, 40)
    k[:] = k[:, :, :1, :]
    out, _, S = oracle.forward(q, k, v, 0.158)
    mean = v.astype(np.float64).mean(axis=2, keepdims=True)
    np.testing.assert_allclose(out, np.broadcast_to(mean, out.shape), rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(S, 13.0)


def test_one_dominant_logit_selects_its_value_row():
    g = rng(7)
    d, Nk = 8, 33
    q = np.zeros((1, 1, 4, d), dtype=np.float32)
    q[0, 0, :, 0] = 1.0
    k = np.zeros((1, 1, Nk, d), dtype=np.float32)
    v = g.standard_normal((1, 1, Nk, d)).astype(np.float32)
    for j_star in (0, 17, 32):
        kk = k.copy()
        kk[0, 0, j_star, 0] = 64.0     # logit 64 against zeros: other weights are e^-64
        out, L, S = oracle.forward(q, kk, v, 1.0)
        np.testing.assert_allclose(out[0, 0], np.broadcast_to(v[0, 0, j_star].astype(np.float64),
                                                              (4, d)), rtol=0, atol=1e-12)
        assert np.all(L == 64.0)


def test_constant_logit_shift_leaves_the_output_unchanged():
    q, k, v = rand_qkv(8, 1, 2, 6, 21, 8, np.float32)
    # keep everything on a coarse binary grid so that k + u is exact in binary32
    q = np.round(q * 8) / 8
    k = np.round(k * 8) / 8
    u = (np.round(rng(9).standard_normal((1, 2, 1, 8)) * 8) / 8).astype(np.float32)
    out0, L0, S0 = oracle.forward(q, k, v, 0.25)
    out1, L1, S1 = oracle.forward(q, (k + u).astype(np.float32), v, 0.25)
    np.testing.assert_allclose(out1, out0, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(S1, S0, rtol=1e-13)
    shift = 0.25 * np.einsum("bhic,bhjc->bhi", q.astype(np.float64), u.astype(np.float64))
    np.testing.assert_allclose(L1 - L0, shift, rtol=0, atol=1e-12)


def test_joint_permutation_of_keys_and_values():
    q, k, v = rand_qkv(10, 2, 2, 5, 77, 40)
    perm = rng(12).permutation(77)
    out0, L0, S0 = oracle.forward(q, k, v, 0.158)
    out1, L1, S1 = oracle.forward(q, k[:, :, perm], v[:, :, perm], 0.158)
    np.testing.assert_allclose(out1, out0, rtol=1e-12, atol=1e-15)
    assert np.array_equal(L0, L1)
    np.testing.assert_allclose(S1, S0, rtol=1e-13)
    # permuting K alone must change the result (guards against V being ignored)
    out2, _, _ = oracle.forward(q, k[:, :, perm], v, 0.158)
    assert np.abs(out2 - out0).max() > 1e-3


def test_query_permutation_permutes_output_rows():
    q, k, v = rand_qkv(13, 1, 3, 9, 11, 4)
    perm = rng(14).permutation(9)
    out0, _, _ = oracle.forward(q, k, v, 0.5)
    out1, _, _ = oracle.forward(q[:, :, perm], k, v, 0.5)
    assert np.array_equal(out1, out0[:, :, perm])


def test_batch_and_head_are_independent_problems():
    q, k, v = rand_qkv(15, 2, 3, 4, 6, 5)
    out, L, S = oracle.forward(q, k, v, 0.4)
    for b in range(2):
        for h in range(3):
            o1, l1, s1 = oracle.forward(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1],
                                        v[b:b + 1, h:h + 1], 0.4)
            assert np.array_equal(o1[0, 0], out[b, h])
            assert np.array_equal(l1[0, 0], L[b, h])


def test_scaling_v_scales_the_output_and_output_stays_in_the_hull_of_v():
    q, k, v = rand_qkv(16, 1, 2, 8, 30, 6, qmult=2.0)
    out, _, _ = oracle.forward(q, k, v, 0.3)
    out4, _, _ = oracle.forward(q, k, (v * np.float16(4)).astype(np.float16), 0.3)
    np.testing.assert_allclose(out4, 4 * out, rtol=1e-15)
    vmin = v.astype(np.float64).min(axis=2, keepdims=True)
    vmax = v.astype(np.float64).max(axis=2, keepdims=True)
    assert np.all(out >= vmin - 1e-15) and np.all(out <= vmax + 1e-15)


def test_scale_is_used_as_given_not_recomputed_from_d():
    q, k, v = rand_qkv(17, 1, 1, 5, 9, 16)
    a, _, _ = oracle.forward(q, k, v, 0.25)          # 1/sqrt(16)
    b, _, _ = oracle.forward(q, k, v, 0.5)
    c, _, _ = oracle.forward(q, k, v, -0.25)
    z, _, _ = oracle.forward(q, k, v, 0.0)
    assert np.abs(a - b).max() > 1e-3 and np.abs(a - c).max() > 1e-3
    np.testing.assert_allclose(z, np.broadcast_to(v.astype(np.float64).mean(axis=2, keepdims=True),
                                                  z.shape), rtol=1e-14)
    # negative scale equals positive scale with negated queries
    d, _, _ = oracle.forward((-q).astype(np.float16), k, v, 0.25)
    np.testing.assert_allclose(c, d, rtol=1e-15)


# ---------------------------------------------------------------- library special case

def numpy_reference(q, k, v, scale):
    q64, k64, v64 = (x.astype(np.float64) for x in (q, k, v))
    a = float(np.float32(scale)) * np.einsum("bhic,bhjc->bhij", q64, k64)
    p = scipy.special.softmax(a, axis=-1)
    return p @ v64, a


@pytest.mark.parametrize("dtype", [np.float16, np.float32])
@pytest.mark.parametrize("shape", [(1, 2, 33, 77, 40), (2, 1, 70, 129, 80), (1, 1, 17, 64, 160),
                                   (1, 3, 128, 128, 40)])
def test_matches_scipy_softmax(shape, dtype):
    B, H, Nq, Nk, d = shape
    q, k, v = rand_qkv(200 + Nq, B, H, Nq, Nk, d, dtype, qmult=4.0)
    scale = np.float32(1.0 / np.sqrt(d))
    out, L, S = oracle.forward(q, k, v, scale)
    ref, a = numpy_reference(q, k, v, scale)
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(L, a.max(axis=-1), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(np.log(S) + L, scipy.special.logsumexp(a, axis=-1), rtol=1e-12)


def test_row_subset_equals_the_same_rows_of_the_full_result():
    q, k, v = rand_qkv(18, 2, 3, 50, 77, 40)
    out, L, S, P = oracle.forward(q, k, v, 0.158, want_probs=True)
    rows = rng(19).choice(2 * 3 * 50, size=41, replace=False)
    o2, l2, s2, p2 = oracle.forward(q, k, v, 0.158, rows=rows, want_probs=True)
    assert np.array_equal(o2, out.reshape(-1, 40)[rows])
    assert np.array_equal(l2, L.reshape(-1)[rows])
    assert np.array_equal(s2, S.reshape(-1)[rows])
    assert np.array_equal(p2, P.reshape(-1, 77)[rows])


def test_thread_count_does_not_change_any_bit():
    q, k, v = rand_qkv(20, 1, 2, 300, 200, 40)
    n = oracle.max_threads()
    try:
        oracle.set_threads(1)
        a = oracle.forward(q, k, v, 0.158)
        oracle.set_threads(max(2, n))
        b = oracle.forward(q, k, v, 0.158)
    finally:
        oracle.set_threads(n)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_bad_arguments_are_rejected():
    q, k, v = rand_qkv(21, 1, 1, 2, 3, 4)
    with pytest.raises(TypeError):
        oracle.forward(q.astype(np.float32), k, v, 1.0)
    with pytest.raises(ValueError):
        oracle.forward(q, k[:, :, :, :3], v, 1.0)
    with pytest.raises(RuntimeError):
        oracle.forward(q, k, v, 1.0, rows=np.array([2]))      # only rows 0..1 exist
    with pytest.raises(RuntimeError):
        oracle.forward(q, k[:, :, :0], v[:, :, :0], 1.0)      # softmax over no keys


# ---------------------------------------------------------------- workload statistics

def test_synthetic_self_attention_statistics_at_1024_tokens():
    """N(0,1) inputs with s = 1/sqrt(d) give unit-variance logits; a missing or squared scale
    would move the row sums S by orders of magnitude."""
    call = workloads.config1()[0]
    q, k, v = workloads.make_inputs(call)
    rows = np.arange(0, call.B * call.H * call.Nq, 37)
    out, L, S = oracle.forward(q, k, v, call.scale(), rows=rows)
    assert 2.3 < L.mean() < 4.2          # max of 1024 unit normals is about 3.2
    assert 40 < S.mean() < 120           # about N * exp(1/2 - L)
    assert 0.03 < out.std() < 0.07       # about sqrt(e / N)


def test_padded_text_rows_share_one_weight():
    call = workloads.config3()[1]
    q, k, v = workloads.make_inputs(call)
    assert np.array_equal(k[:, :, 57:], np.broadcast_to(k[:, :, 57:58], k[:, :, 57:].shape))
    rows = np.arange(0, call.B * call.H * call.Nq, 211)
    out, L, S, P = oracle.forward(q, k, v, call.scale(), rows=rows, want_probs=True)
    assert np.array_equal(P[:, 57:], np.broadcast_to(P[:, 57:58], P[:, 57:].shape))
    # distinct V rows under identical keys: only their mean matters
    v2 = v.copy()
    v2[:, :, 57:] = rng(22).standard_normal(v2[:, :, 57:].shape).astype(np.float16)
    v3 = v2.copy()
    v3[:, :, 57:] = v2[:, :, 57:][:, :, ::-1]
    o2, _, _ = oracle.forward(q, k, v2, call.scale(), rows=rows)
    o3, _, _ = oracle.forward(q, k, v3, call.scale(), rows=rows)
    np.testing.assert_allclose(o3, o2, rtol=1e-12, atol=1e-14)
