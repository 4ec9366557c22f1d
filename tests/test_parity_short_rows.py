"""GPU parity on short rows (8 to 1024 columns), where the row kernels switch to 2 - 32 lanes of a warp per row
and the elementwise kernels to tiles that cross rows: every lane count, row counts that leave part of the last
warp or tile without data, in-place use, strided rows. Tolerances as everywhere: 1e-5 fp32, 2e-2 bf16, 2e-3
fp16, relative to max(1, |ref|)."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_bf16_tight, assert_close, to_f64, tol_of

pytestmark = pytest.mark.gpu
F32, BF16, F16 = torch.float32, torch.bfloat16, torch.float16
# (rows, cols, dtype): vectors per row 1, 2, 3, 4, 8, 12, 16, 17, 31, 32, 33, 64, 96, 128 across the data types
SHAPES = [(1031, 8, BF16), (517, 16, BF16), (259, 24, F16), (1000, 32, BF16), (403, 64, BF16), (77, 96, F16),
          (2051, 128, BF16), (129, 136, BF16), (65, 248, F16), (300, 256, BF16), (33, 264, BF16), (131, 512, F16),
          (67, 768, BF16), (259, 1024, BF16), (1025, 4, F32), (999, 20, F32), (257, 64, F32), (63, 132, F32),
          (515, 256, F32), (35, 512, F32)]


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


@pytest.mark.parametrize("rows,cols,dtype", SHAPES)
def test_short_row_norms_and_softmax(kop, rows, cols, dtype):
    seed = rows + cols
    x, r, b, g, be = synth.layernorm_inputs(rows, cols, dtype, seed, "cuda")
    tol = tol_of(dtype)
    # RMSNorm, with and without the residual add
    y = Guarded((rows, cols), dtype)
    kop.kop_rmsnorm(x, g, 1e-6, out=y.t)
    assert_close(y.t, kopref.rmsnorm(host(x), host(g), 1e-6, threads=None), tol, "rmsnorm")
    y.check("rmsnorm")
    h = Guarded((rows, cols), dtype)
    y2 = Guarded((rows, cols), dtype)
    kop.kop_residual_rmsnorm(x, r, g, 1e-6, h_out=h.t, out=y2.t)
    rh, ry = kopref.residual_rmsnorm(host(x), host(r), host(g), 1e-6, threads=None)
    assert_close(h.t, rh, tol, "residual_rmsnorm h")
    assert_close(y2.t, ry, tol, "residual_rmsnorm y")
    h.check("h")
    y2.check("y")
    # LayerNorm: the benchmark prologue, and plain
    y3 = Guarded((rows, cols), dtype)
    _, mean, rstd = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5, out=y3.t)
    ref, rmean, rrstd = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5, threads=None)
    assert_close(y3.t, ref, tol, "layernorm")
    assert_close(mean, rmean, 1e-5, "mean")
    if cols > 1:
        assert_close(rstd, rrstd, 1e-4, "rstd")
    y3.check("layernorm")
    y4, _, _ = kop.kop_residual_layernorm(x, None, g, be, 1e-5)
    assert_close(y4, kopref.residual_layernorm(host(x), None, host(g), host(be), 1e-5, threads=None)[0], tol, "plain layernorm")
    if dtype != F32:                                       # 16-bit parameters
        y5, _, _ = kop.kop_layernorm_ex(x, r, b.to(dtype), g.to(dtype), be.to(dtype), 1e-5, "residual")
        assert_close(y5, kopref.residual_layernorm(host(x), host(r), host(g.to(dtype)), host(be.to(dtype)), 1e-5, threads=None)[0],
                     tol, "layernorm 16-bit params")
    # softmax with bias, and in place without
    s = Guarded((rows, cols), dtype)
    kop.kop_softmax_scale_bias(x, b, 0.5, out=s.t)
    assert_close(s.t, kopref.softmax_scale_bias(host(x), host(b), 0.5, threads=None), tol, "softmax")
    s.check("softmax")
    xi = x.clone()
    kop.kop_softmax_scale_bias(xi, None, 1.0, out=xi)
    ref = kopref.softmax_scale_bias(host(x), None, 1.0, threads=None)
    assert_close(xi, ref, tol, "softmax in place")
    assert np.all(np.abs(to_f64(xi).sum(axis=1) - 1.0) <= (1e-5 if dtype == F32 else 2e-2))


@pytest.mark.parametrize("rows,cols,dtype", SHAPES)
def test_short_row_elementwise(kop, rows, cols, dtype):
    seed = rows * 3 + cols
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    res, _ = synth.softmax_inputs(rows, cols, dtype, seed + 1, "cuda")
    tol = tol_of(dtype)
    y = Guarded((rows, cols), dtype)
    kop.kop_bias_act(x, bias, "gelu_tanh", out=y.t)
    ref = kopref.bias_act(host(x), host(bias), "gelu_tanh", threads=None)
    assert_close(y.t, ref, tol, "bias_act")
    if dtype == BF16:
        assert_bf16_tight(y.t, ref, "bias_act")
    y.check("bias_act")
    big = torch.zeros((rows, cols + 24), dtype=dtype, device="cuda")        # strided rows keep their row stride
    big[:, :cols] = x
    assert_close(kop.kop_bias_act(big[:, :cols], bias, "silu"), kopref.bias_act(host(x), host(bias), "silu", threads=None),
                 tol, "bias_act strided")
    c = Guarded((rows, cols), dtype)
    kop.kop_epilogue_chain(x, bias, res, 0.5, 2.0, -1.0, 1.5, "mish", out=c.t)
    assert_close(c.t, kopref.epilogue_chain(host(x), host(bias), host(res), 0.5, 2.0, -1.0, 1.5, "mish", threads=None), tol, "chain")
    c.check("chain")
    if cols % 2 == 0:
        o = Guarded((rows, cols // 2), dtype)
        kop.kop_silu_mul(x, out=o.t)
        assert_close(o.t, kopref.silu_mul(host(x)), tol, "silu_mul")
        o.check("silu_mul")
        o2 = Guarded((rows, cols // 2), dtype)
        kop.kop_silu_mul_interleaved(x, out=o2.t)
        assert_close(o2.t, kopref.silu_mul_interleaved(host(x)), tol, "silu_mul_interleaved")
        o2.check("silu_mul_interleaved")


@pytest.mark.parametrize("rows,cols,dtype", SHAPES)
def test_short_row_scale_matvec_and_strided_add(kop, rows, cols, dtype):
    seed = rows * 5 + cols
    tol = tol_of(dtype)
    a, b = synth.row_scale_inputs(rows, cols, dtype, seed, "cuda")
    y = Guarded((rows, cols), dtype)
    kop.kop_row_scale(a, b, out=y.t)
    assert_close(y.t, kopref.row_scale(host(a), host(b)), tol, "row_scale")
    y.check("row_scale")
    xv, wv, bs = synth.matvec_inputs(rows, cols, dtype, seed, "cuda")
    o = Guarded((rows,), F32)
    kop.kop_matvec_bias(xv, wv, bs, out=o.t)
    ref = kopref.matvec_bias(host(xv), host(wv), bs)
    mag = (host(xv).double().abs() @ host(wv).double().abs()).numpy() + abs(bs)
    assert np.all(np.abs(to_f64(o.t) - ref) <= 1e-5 * np.maximum(1.0, mag)), "matvec"
    o.check("matvec")
    p, q = synth.pair_inputs(rows, cols, dtype, seed, "cuda")
    pad = 8 if dtype != F32 else 4
    bp = torch.zeros((rows, cols + pad), dtype=dtype, device="cuda")          # strided rows: no collapse to one long row
    bq = torch.zeros((rows, cols + 2 * pad), dtype=dtype, device="cuda")
    bp[:, :cols] = p
    bq[:, :cols] = q
    outb = torch.full((rows, cols + pad), 7.0, dtype=dtype, device="cuda")
    kop.kop_residual_add(bp[:, :cols], bq[:, :cols], out=outb[:, :cols])
    assert_close(outb[:, :cols], kopref.residual_add(host(p), host(q)), tol, "strided residual_add")
    assert bool((outb[:, cols:] == 7.0).all())


def test_matvec_long_rows(kop):
    for rows, cols, dtype in ((37, 16384, BF16), (9, 65536, F32), (5, 40008, BF16)):
        xv, wv, bs = synth.matvec_inputs(rows, cols, dtype, 3, "cuda")
        ref = kopref.matvec_bias(host(xv), host(wv), bs)
        mag = (host(xv).double().abs() @ host(wv).double().abs()).numpy() + abs(bs)
        got = to_f64(kop.kop_matvec_bias(xv, wv, bs))
        assert np.all(np.abs(got - ref) <= 1e-5 * np.maximum(1.0, mag)), f"matvec [{rows},{cols}]"
