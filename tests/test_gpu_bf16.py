"""GPU parity for bfloat16 tensors (dtype SD_ATTN_BF16) against the fp64 oracle.

The inputs are seeded normals rounded to bfloat16; the oracle receives exactly those values (as binary32 arrays,
which hold every bfloat16 exactly) and works in double precision as always.

Tolerance, derived from the arithmetic: bfloat16 keeps 8 significant bits, so rounding to nearest is off by at most
2^-8 relative, against binary16's 2^-11 -- 8 times coarser.  Two roundings matter, as for binary16: the weights
(each 2^-8 relative, signs independent; coherent worst case 2^-8 * max|V|) and the output (2^-8 * |o|, |o| <=
max|V|); everything else (binary32 accumulation, the exponential) is far below.  Worst case 2 * 2^-8 * max|V| =
7.8e-3 * max|V|; the bounds used: 8e-3 * max|V| (that worst case; measured 3.7e-4 ... 1.6e-3) and 5e-3 relative L2
(the output's rounding alone is 2^-8 / sqrt(3) = 2.3e-3 relative, measured 1.6e-3 ... 2.5e-3: a scale error of one percent fails).
"""
import numpy as np
import pytest

import oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

BF16_ABS = 8e-3
BF16_REL_L2 = 5e-3


@pytest.fixture(scope="module")
def bd():
    from paper_2304_11267_b200 import binding
    from paper_2304_11267_b200 import build
    build.build()
    binding.load()
    return binding


@pytest.fixture()
def att(bd):
    a = bd.Attention()
    yield a
    a.check()
    a.close()


def rand_bf16(seed, B, H, Nq, Nk, d):
    """Head-major bfloat16 tensors (torch, on the CPU) and the same values as binary32 numpy arrays."""
    g = np.random.default_rng(seed)
    ts = [torch.from_numpy(g.standard_normal(shape, dtype=np.float32)).to(torch.bfloat16)
          for shape in ((B, H, Nq, d), (B, H, Nk, d), (B, H, Nk, d))]
    return ts, [t.to(torch.float32).numpy() for t in ts]


def check(got, ref, v, what):
    got = got.astype(np.float64)
    assert np.all(np.isfinite(got)), "%s: non-finite output" % what
    vmax = float(np.abs(v.astype(np.float64)).max())
    err = float(np.abs(got - ref).max())
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))
    assert err <= BF16_ABS * vmax, "%s: max abs err %.3e > %.3e" % (what, err, BF16_ABS * vmax)
    assert rel <= BF16_REL_L2, "%s: rel L2 err %.3e" % (what, rel)
    return err / vmax, rel


@pytest.mark.parametrize("B,H,Nq,Nk,d,mode", [
    (2, 8, 1024, 1024, 40, "fused"),    # four tiles per CTA, the polynomial share of the exponentials
    (2, 8, 200, 200, 40, "fused"),      # one tile per CTA in four parts, ragged
    (1, 8, 640, 640, 80, "fused"),      # two chunks per row
    (2, 8, 256, 256, 160, "fused"),     # three chunks per row, two parts
    (3, 5, 333, 333, 64, "fused"),
    (2, 8, 1024, 77, 40, "cross"),      # persistent 77-key kernel, four groups (raw Q tiles rewritten in shared memory)
    (2, 8, 300, 77, 80, "cross"),       # three groups
    (2, 8, 256, 77, 160, "cross"),      # two groups
    (2, 4, 200, 33, 40, "cross"),       # the one-tile kernel
    (2, 3, 150, 77, 20, "simt"),        # d % 8 != 0: the CUDA-core kernel
])
def test_bf16_against_the_oracle(att, bd, B, H, Nq, Nk, d, mode):
    (q, k, v), (q32, k32, v32) = rand_bf16(500 + Nq + Nk + d, B, H, Nq, Nk, d)
    scale = d ** -0.5
    ref, _, _ = oracle.forward(q32, k32, v32, scale)
    out = att.forward(q.cuda(), k.cuda(), v.cuda(), scale=scale)
    att.check()
    assert out.dtype == torch.bfloat16
    assert bd.MODE_NAMES[att.last_mode] == mode
    err, rel = check(out.to(torch.float32).cpu().numpy(), ref, v32, "bf16 %s %s" % (mode, (B, H, Nq, Nk, d)))
    print("bf16 %-5s %-24s max|err|/max|V| %.2e  rel L2 %.2e" % (mode, (B, H, Nq, Nk, d), err, rel))


def test_bf16_config2_sampled_rows(att, bd):
    """The 4096-token shape in the launch configuration the bench times, on sampled rows."""
    B, H, N, d = 2, 8, 4096, 40
    (q, k, v), (q32, k32, v32) = rand_bf16(77, B, H, N, N, d)
    rows = np.unique(np.concatenate([np.arange(128), np.arange(B * H * N - 128, B * H * N),
                                     np.random.default_rng(3).choice(B * H * N, 384, replace=False)]))
    ref, _, _ = oracle.forward(q32, k32, v32, d ** -0.5, rows=rows)
    out = att.forward(q.cuda(), k.cuda(), v.cuda())
    att.check()
    got = out.to(torch.float32).cpu().numpy().reshape(-1, d)[rows]
    check(got, ref, v32, "bf16 4096 x 40")


def test_bf16_token_major(bd):
    a = bd.Attention(layout=bd.LAYOUT_BNHD)
    for (B, H, Nq, Nk, d) in [(2, 8, 384, 384, 40), (2, 8, 300, 77, 80)]:
        (q, k, v), (q32, k32, v32) = rand_bf16(900 + Nq + d, B, H, Nq, Nk, d)
        ref, _, _ = oracle.forward(q32, k32, v32, d ** -0.5)
        tm = [t.permute(0, 2, 1, 3).contiguous().cuda() for t in (q, k, v)]
        out = a.forward(*tm)
        a.check()
        check(out.permute(0, 2, 1, 3).to(torch.float32).cpu().numpy(), ref, v32, "bf16 token-major %s" % ((B, H, Nq, Nk, d),))
    a.close()


def test_bf16_is_not_fp16_with_the_bits_reinterpreted(att, bd):
    """The same bytes read as binary16 are different numbers: the dtype must reach the tensor core's descriptor."""
    (q, k, v), (q32, k32, v32) = rand_bf16(5, 1, 2, 256, 256, 40)
    ref, _, _ = oracle.forward(q32, k32, v32, 40 ** -0.5)
    wrong = att.forward(q.cuda().view(torch.float16), k.cuda().view(torch.float16), v.cuda().view(torch.float16),
                        scale=40 ** -0.5)
    att.check()
    got = wrong.view(torch.bfloat16).to(torch.float32).cpu().numpy().astype(np.float64)
    vmax = float(np.abs(v32).max())
    assert not (np.all(np.isfinite(got)) and np.abs(got - ref).max() <= BF16_ABS * vmax)


def test_bf16_host_call(att, bd):
    B, H, Nq, Nk, d = 2, 8, 256, 77, 40
    (q, k, v), (q32, k32, v32) = rand_bf16(13, B, H, Nq, Nk, d)
    ref, _, _ = oracle.forward(q32, k32, v32, d ** -0.5)
    tq, tk, tv = (t.contiguous().pin_memory() for t in (q, k, v))
    out = torch.empty_like(tq).pin_memory()
    need = bd.sd_attn_host_staging_bytes(B, H, Nq, Nk, d, bd.BF16)
    staging = torch.empty(need, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    rc = bd.sd_attn_forward_host(att.handle, tq.data_ptr(), tk.data_ptr(), tv.data_ptr(), out.data_ptr(),
                                 staging.data_ptr(), need, B, H, Nq, Nk, d, d ** -0.5, bd.BF16, s)
    assert rc == bd.OK
    att.check()
    check(out.to(torch.float32).numpy(), ref, v32, "bf16 host call")


def test_modes_without_bf16_say_so(bd):
    B, H, N, d = 1, 2, 128, 40
    a = bd.Attention(mode=bd.MODE_TWOPASS)
    x = torch.zeros(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    need = bd.sd_attn_workspace_bytes(bd.MODE_TWOPASS, B, H, N, N, d, bd.F16)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert bd.sd_attn_set_workspace(a.handle, ws.data_ptr(), need) == bd.OK
    s = torch.cuda.current_stream().cuda_stream
    rc = bd.sd_attn_forward(a.handle, x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), B, H, N, N, d, 1.0, bd.BF16, s)
    assert rc == bd.ERR_UNSUPPORTED
    a.close()
