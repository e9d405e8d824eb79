"""GPU parity for token-major tensors (q, out [B,Nq,H,d]; k, v [B,Nk,H,d]): the head split before and the head merge
after the attention (Sec. 3.2) as views of the projections' [B,N,H*d] tensors, with no copy.

The oracle knows one layout only, [B,H,N,d].  The test generates the inputs in that layout, hands the oracle exactly
those arrays and the library the SAME values transposed into token-major memory, and transposes the library's
result back before the element-by-element comparison (tolerances as in test_gpu_parity.py).
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

F16_ABS = 2e-3
F16_REL_L2 = 2e-3
F32_TOL = 1e-5


@pytest.fixture(scope="module")
def bd():
    from paper_2304_11267_b200 import binding
    from paper_2304_11267_b200 import build
    build.build()
    binding.load()
    return binding


@pytest.fixture()
def att(bd):
    a = bd.Attention(layout=bd.LAYOUT_BNHD)
    yield a
    a.check()
    a.close()


def rand_qkv(seed, B, H, Nq, Nk, d, dtype=np.float16):
    g = np.random.default_rng(seed)
    q = g.standard_normal((B, H, Nq, d), dtype=np.float32).astype(dtype)
    k = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(dtype)
    v = g.standard_normal((B, H, Nk, d), dtype=np.float32).astype(dtype)
    return q, k, v


def token_major(x):
    return torch.from_numpy(np.ascontiguousarray(x.transpose(0, 2, 1, 3))).cuda()


def run_token_major(att, q, k, v, scale):
    """q, k, v head-major numpy arrays -> the library's result, brought back to head-major."""
    out = att.forward(token_major(q), token_major(k), token_major(v), scale=float(scale))
    att.check()
    assert out.shape == (q.shape[0], q.shape[2], q.shape[1], q.shape[3])
    return out.cpu().numpy().transpose(0, 2, 1, 3)


def check(got, ref, v, dtype, what):
    got = got.astype(np.float64)
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    vmax = float(np.abs(v.astype(np.float64)).max())
    err = float(np.abs(got - ref).max())
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    if dtype == np.float16:
        assert err <= F16_ABS * vmax, "%s: max abs err %.3e > %.3e" % (what, err, F16_ABS * vmax)
        assert rel <= F16_REL_L2, "%s: rel L2 err %.3e" % (what, rel)
    else:
        assert err <= F32_TOL * vmax, "%s: max abs err %.3e > %.3e" % (what, err, F32_TOL * vmax)
        assert rel <= F32_TOL, "%s: rel L2 err %.3e" % (what, rel)


# Self-attention through the single-pass kernel: four tiles per CTA (1024 x 40), one tile in four parts (a ragged 200),
# two-chunk and three-chunk rows (d = 80, 160), one tile in two parts, more than one batch entry, a lone head.
@pytest.mark.parametrize("B,H,N,d", [(2, 8, 1024, 40), (2, 8, 200, 40), (2, 8, 640, 80), (2, 8, 256, 160),
                                     (3, 5, 333, 64), (1, 1, 129, 40), (4, 1, 130, 24)])
def test_self_attention_token_major(att, bd, B, H, N, d):
    q, k, v = rand_qkv(100 + N + d, B, H, N, N, d)
    scale = d ** -0.5
    ref, _, _ = oracle.forward(q, k, v, scale)
    got = run_token_major(att, q, k, v, scale)
    assert att.last_mode == bd.MODE_FUSED
    check(got, ref, v, np.float16, "token-major self %s" % ((B, H, N, d),))


# Cross-attention over the 77 text tokens (the persistent kernel: four groups with Q and the output as unswizzled
# row tiles at d <= 48 -- full and ragged last tiles --, three and two groups above), and over fewer keys (the
# one-tile kernel).
@pytest.mark.parametrize("B,H,Nq,Nk,d", [(2, 8, 1024, 77, 40), (2, 8, 300, 77, 80), (2, 8, 256, 77, 160),
                                         (2, 8, 4096, 77, 40), (2, 4, 200, 33, 40), (1, 3, 64, 16, 160),
                                         (2, 8, 333, 77, 40), (1, 3, 200, 70, 24), (3, 5, 129, 77, 48)])
def test_cross_attention_token_major(att, bd, B, H, Nq, Nk, d):
    q, k, v = rand_qkv(200 + Nq + d, B, H, Nq, Nk, d)
    scale = d ** -0.5
    ref, _, _ = oracle.forward(q, k, v, scale)
    got = run_token_major(att, q, k, v, scale)
    assert att.last_mode == bd.MODE_CROSS
    check(got, ref, v, np.float16, "token-major cross %s" % ((B, H, Nq, Nk, d),))


@pytest.mark.parametrize("dtype,d", [(np.float32, 40), (np.float32, 37), (np.float16, 20)])
def test_cuda_core_path_token_major(att, bd, dtype, d):
    B, H, Nq, Nk = 2, 3, 150, 77
    q, k, v = rand_qkv(300 + d, B, H, Nq, Nk, d, dtype)
    scale = d ** -0.5
    ref, _, _ = oracle.forward(q, k, v, scale)
    got = run_token_major(att, q, k, v, scale)
    assert att.last_mode == bd.MODE_SIMT
    check(got, ref, v, dtype, "token-major cuda-core %s d=%d" % (np.dtype(dtype).name, d))


def test_same_values_in_either_layout(bd):
    """The two layouts run the same kernel on the same values in the same order: the results are bitwise equal."""
    B, H, N, d = 2, 8, 512, 40
    q, k, v = rand_qkv(7, B, H, N, N, d)
    a = bd.Attention()
    o1 = a.forward(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), scale=d ** -0.5)
    a.check()
    a.set_layout(bd.LAYOUT_BNHD)
    o2 = a.forward(token_major(q), token_major(k), token_major(v), scale=d ** -0.5)
    a.check()
    a.set_layout(bd.LAYOUT_BHND)
    o3 = a.forward(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), scale=d ** -0.5)
    a.check()
    a.close()
    assert torch.equal(o1, o2.permute(0, 2, 1, 3))
    assert torch.equal(o1, o3)
    # the 77-key kernel: only the way a Q tile reaches shared memory and the output leaves it differs
    q, k, v = rand_qkv(8, 2, 8, 300, 77, 40)
    a = bd.Attention()
    c1 = a.forward(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda(), scale=40 ** -0.5)
    a.check()
    a.set_layout(bd.LAYOUT_BNHD)
    c2 = a.forward(token_major(q), token_major(k), token_major(v), scale=40 ** -0.5)
    a.check()
    a.close()
    assert torch.equal(c1, c2.permute(0, 2, 1, 3))


def test_neighbouring_heads_do_not_leak(att, bd):
    """d = 40 rows are 80 bytes inside 128-byte tile rows: the 24 columns after a head's 40 belong to the next head in
    token-major memory and must read as zero, not as that head's values.  Huge values in every other head would
    show."""
    B, H, N, d = 1, 4, 256, 40
    q, k, v = rand_qkv(11, B, H, N, N, d)
    q[:, 1::2] *= 30.0
    k[:, 1::2] *= 30.0
    ref, _, _ = oracle.forward(q, k, v, d ** -0.5)
    got = run_token_major(att, q, k, v, d ** -0.5)
    check(got, ref, v, np.float16, "token-major, loud neighbours")


def test_host_call_token_major(att, bd):
    B, H, Nq, Nk, d = 2, 8, 256, 77, 40
    q, k, v = rand_qkv(13, B, H, Nq, Nk, d)
    ref, _, _ = oracle.forward(q, k, v, d ** -0.5)
    hq, hk, hv = (np.ascontiguousarray(x.transpose(0, 2, 1, 3)) for x in (q, k, v))
    tq, tk, tv = (torch.from_numpy(x).pin_memory() for x in (hq, hk, hv))
    out = torch.empty_like(tq).pin_memory()
    need = bd.sd_attn_host_staging_bytes(B, H, Nq, Nk, d, bd.F16)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    rc = bd.sd_attn_forward_host(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), out.data_ptr(),
                                 staging.data_ptr(), need, B, H, Nq, Nk, d, d ** -0.5, bd.F16, s)
    assert rc == bd.OK
    att.check()
    check(out.numpy().transpose(0, 2, 1, 3), ref, v, np.float16, "token-major host call")


def test_modes_without_the_layout_say_so(bd):
    B, H, N, d = 1, 2, 128, 40
    a = bd.Attention(layout=bd.LAYOUT_BNHD)
    x = torch.zeros(B, N, H, d, dtype=torch.float16, device="cuda")
    a.set_mode(bd.MODE_TWOPASS)
    need = bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, B, H, N, N, d, bd.F16)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert bd.sd_attn_set_workspace(a.handle, ws.data_ptr(), need) == bd.OK
    s = torch.cuda.current_stream().cuda_stream
    rc = bd.sd_attn_forward(a.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), B, H, N, N, d, 1.0, bd.F16, s)
    assert rc == bd.ERR_UNSUPPORTED
    assert bd.sd_attn_set_layout(a.handle, 7) == bd.ERR_INVALID_VALUE
    a.close()
