"""GPU parity: every libkop segment, called through the C ABI, against the float64 CPU oracle on
the same seeded inputs. Five seeds at sizes that span several CTAs / tiles plus ragged tails, the
full benchmark shapes on seed 0, edge cases (empty, one element, odd lengths, misaligned bases,
strided rows, in-place, masked columns, bad labels), guard bands around every output, and
run-to-run bit equality.

Tolerance: |got - ref| <= tol * max(1, |ref|), tol = 1e-5 for fp32 data and 2e-2 for bf16 data;
bf16 outputs are additionally held to about two bf16 steps of the float64 value."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_bf16_tight, assert_close, to_f64, tol_of

pytestmark = pytest.mark.gpu

SEEDS = synth.SEEDS
F32, BF16 = torch.float32, torch.bfloat16


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return t.detach().cpu()


# ------------------------------------------------------------------------------------------ softmax

SOFTMAX_SHAPES = [
    (128, 512, F32),       # benchmark small config: warp-per-row
    (1000, 512, F32),
    (333, 96, F32),        # partial last vector group in the warp
    (257, 2048, F32),      # CTA-per-row, row in registers
    (19, 16384, F32),      # longest register-resident row
    (7, 20000, F32),       # beyond one CTA's registers: two sweeps with vector loads
    (5, 40000, BF16),
    (3, 131072, BF16),
    (2, 100000, F32),
    (3, 128256, BF16),     # a vocabulary size
    (2, 140008, BF16),
    (9, 12288, F32),       # fp32 rows beyond 32 KB: two sweeps although the row would fit the registers
    (3, 20001, BF16),      # odd length: edge elements around two sweeps of aligned vectors
    (37, 513, F32),        # odd length: edge elements, the row in a warp's registers
    (64, 1, F32),
    (515, 1000, BF16),
    (129, 4096, BF16),
    (33, 777, BF16),
]


@pytest.mark.parametrize("rows,cols,dtype", SOFTMAX_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_softmax_parity(kop, rows, cols, dtype, seed):
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    out = Guarded((rows, cols), dtype)
    kop.kop_softmax_scale_bias(x, bias, 0.125, out=out.t)
    ref = kopref.softmax_scale_bias(host(x), host(bias), 0.125, threads=None)
    assert_close(out.t, ref, tol_of(dtype), "softmax")
    out.check("softmax")
    sums = to_f64(out.t).sum(axis=1)
    assert np.all(np.abs(sums - 1.0) <= (1e-5 if dtype == F32 else 2e-2))


@pytest.mark.parametrize("rows,cols,dtype", [(257, 2048, F32), (129, 4096, BF16), (19, 8192, F32), (33, 16384, BF16),
                                             (65, 3072, torch.float16), (40, 2056, BF16), (1500, 1032, F32)])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_softmax_no_bias_block_rows(kop, rows, cols, dtype, seed):
    """Rows in one CTA's registers without a bias: exact rows take the predicate-free variant (32 values a thread from
    2048 columns, fp32 rows up to 32 KB), ragged ones the general form."""
    x, _ = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    out = Guarded((rows, cols), dtype)
    kop.kop_softmax_scale_bias(x, None, 0.5, out=out.t)
    ref = kopref.softmax_scale_bias(host(x), None, 0.5, threads=None)
    assert_close(out.t, ref, tol_of(dtype), "softmax no bias")
    out.check("softmax no bias")
    assert torch.equal(out.t, kop.kop_softmax_scale_bias(x, None, 0.5))


@pytest.mark.parametrize("rows,cols,dtype", [(2364, 197, BF16), (1000, 77, F32), (900, 49, torch.float16), (333, 257, BF16),
                                             (100, 577, F32), (40, 1025, BF16), (64, 1001, F32), (7, 50257, BF16),
                                             (5, 50257, F32), (130, 7, BF16), (50, 3, F32), (21, 2051, torch.float16),
                                             (3, 70001, F32)])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_softmax_ragged_rows(kop, rows, cols, dtype, seed):
    """Rows that are not a whole number of aligned 16-byte vectors (attention scores of 197 or 77 keys, a 50257-wide
    vocabulary): head elements, aligned vectors and tail elements, with the row in a half warp's or a warp's registers
    up to 128 vectors and in two sweeps beyond; with and without a bias, plain and log form, in place, from a base that
    is off a boundary, and (x and y at different offsets) through the element-wise kernel."""
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    tol = tol_of(dtype)
    for use_bias in (False, True):
        b = bias if use_bias else None
        hb = host(b) if use_bias else None
        ref = kopref.softmax_scale_bias(host(x), hb, 0.25, threads=None)
        out = Guarded((rows, cols), dtype)
        kop.kop_softmax_scale_bias(x, b, 0.25, out=out.t)
        assert_close(out.t, ref, tol, f"ragged softmax bias={use_bias}")
        out.check("ragged softmax")
        lref = kopref.softmax_opts(host(x), hb, 0.25, True, 0, threads=None)
        lout = Guarded((rows, cols), dtype)
        kop.kop_softmax_opts(x, b, 0.25, True, 0, out=lout.t)
        assert_close(lout.t, lref, tol, f"ragged log-softmax bias={use_bias}")
        lout.check("ragged log-softmax")
    ref = kopref.softmax_scale_bias(host(x), None, 0.25, threads=None)
    xi = x.clone()
    kop.kop_softmax_scale_bias(xi, None, 0.25, out=xi)
    assert_close(xi, ref, tol, "ragged softmax in place")
    # one element off the allocation's boundary, x and y alike; then y alone (different offsets)
    n = rows * cols
    xo = torch.zeros(n + 9, dtype=dtype, device="cuda")
    yo = torch.full((n + 9,), 3.0, dtype=dtype, device="cuda")
    xo[1:n + 1] = x.reshape(-1)
    kop.kop_softmax_scale_bias(xo[1:n + 1].view(rows, cols), None, 0.25, out=yo[1:n + 1].view(rows, cols))
    assert_close(yo[1:n + 1].view(rows, cols), ref, tol, "ragged softmax off the boundary")
    assert float(yo[0]) == 3.0 and bool((yo[n + 1:] == 3.0).all())
    yo.fill_(3.0)
    kop.kop_softmax_scale_bias(xo[1:n + 1].view(rows, cols), None, 0.25, out=yo[2:n + 2].view(rows, cols))
    assert_close(yo[2:n + 2].view(rows, cols), ref, tol, "softmax, x and y at different offsets")
    assert bool((yo[:2] == 3.0).all()) and bool((yo[n + 2:] == 3.0).all())
    # masked first and last column (-inf bias): exact zeros there; a NaN in an edge element poisons its row only
    b2 = bias.clone()
    b2[0] = float("-inf")
    b2[cols - 1] = float("-inf")
    if cols > 2:
        y = kop.kop_softmax_scale_bias(x, b2, 0.25)
        assert_close(y, kopref.softmax_scale_bias(host(x), host(b2), 0.25, threads=None), tol, "ragged softmax masked")
        assert bool((y[:, 0] == 0).all()) and bool((y[:, cols - 1] == 0).all())
    xn = x.clone()
    xn[rows // 2, 0] = float("nan")
    xn[rows - 1, cols - 1] = float("nan")
    y = kop.kop_softmax_scale_bias(xn, None, 0.25)
    bad = torch.isnan(y).any(dim=1)
    want = torch.zeros(rows, dtype=torch.bool, device="cuda")
    want[rows // 2] = True
    want[rows - 1] = True
    assert torch.equal(bad, want) and bool(torch.isnan(y[rows // 2]).all()) and bool(torch.isnan(y[rows - 1]).all())


def test_softmax_large_config_seed0(kop):
    c = synth.CONFIGS["softmax_large"]
    x, bias = synth.softmax_inputs(c["rows"], c["cols"], c["dtype"], 0, "cuda")
    y = kop.kop_softmax_scale_bias(x, bias, c["scale"])
    ref = kopref.softmax_scale_bias(host(x), host(bias), c["scale"], threads=None)
    assert_close(y, ref, 1e-5, "softmax large")


def test_softmax_options(kop):
    x, bias = synth.softmax_inputs(300, 512, F32, 1, "cuda")
    # no bias
    y = kop.kop_softmax_scale_bias(x, None, 0.5)
    assert_close(y, kopref.softmax_scale_bias(host(x), None, 0.5), 1e-5, "no bias")
    # masked columns (-inf bias) give exact zeros
    b2 = bias.clone()
    b2[::3] = float("-inf")
    y = kop.kop_softmax_scale_bias(x, b2, 0.125)
    assert_close(y, kopref.softmax_scale_bias(host(x), host(b2), 0.125), 1e-5, "masked")
    assert bool((y[:, ::3] == 0).all())
    # in place
    ref = kopref.softmax_scale_bias(host(x), host(bias), 0.125)
    xi = x.clone()
    kop.kop_softmax_scale_bias(xi, bias, 0.125, out=xi)
    assert_close(xi, ref, 1e-5, "in place")
    # strided rows (a column slice of a wider matrix), vector-aligned and not
    wide = torch.zeros((300, 1024), dtype=F32, device="cuda")
    wide[:, 256:768] = x
    ow = torch.full((300, 640), 7.0, dtype=F32, device="cuda")
    kop.kop_softmax_scale_bias(wide[:, 256:768], bias, 0.125, out=ow[:, 64:576])
    assert_close(ow[:, 64:576], ref, 1e-5, "strided")
    assert bool((ow[:, :64] == 7.0).all()) and bool((ow[:, 576:] == 7.0).all())
    wide[:, 257:769] = x
    y = kop.kop_softmax_scale_bias(wide[:, 257:769], bias, 0.125)         # misaligned base, y aligned: element-wise kernel
    assert_close(y, ref, 1e-5, "misaligned")
    # empty
    e = torch.empty((0, 512), dtype=F32, device="cuda")
    assert kop.kop_softmax_scale_bias(e, bias, 0.125).shape == (0, 512)
    # determinism
    a = kop.kop_softmax_scale_bias(x, bias, 0.125)
    b = kop.kop_softmax_scale_bias(x, bias, 0.125)
    assert torch.equal(a, b)


# ------------------------------------------------------------------------------------------ LayerNorm

LN_SHAPES = [
    (2048, 4096, BF16),    # benchmark row length, >= 4 waves of CTAs (two rows per CTA)
    (1185, 4096, BF16),    # odd row count on the two-rows-per-CTA kernel
    (1301, 2048, F32),     # the same kernel on fp32 rows
    (300, 4096, F32),
    (129, 1024, BF16),
    (65, 256, BF16),
    (33, 8192, BF16),
    (17, 16384, F32),      # longest register-resident row
    (9, 20480, BF16),      # beyond one CTA's registers: three sweeps with vector loads
    (5, 40004, F32),       # several batches, ragged last one
    (3, 20481, BF16),      # odd length: the scalar three-sweep kernel
    (21, 513, F32),        # scalar
    (40, 1000, BF16),      # 125 vectors: ragged CTA
    (5, 1, F32),
]


@pytest.mark.parametrize("rows,hidden,dtype", LN_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_layernorm_parity(kop, rows, hidden, dtype, seed):
    x, r, b, g, be = synth.layernorm_inputs(rows, hidden, dtype, seed, "cuda")
    out = Guarded((rows, hidden), dtype)
    mean = Guarded((rows,), F32)
    rstd = Guarded((rows,), F32)
    kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5, out=out.t, mean=mean.t, rstd=rstd.t)
    ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5,
                                                     threads=None)
    tol = tol_of(dtype)
    if hidden == 1:
        # var = 0: y = beta exactly, rstd = 1/sqrt(eps) ~ 316: only the relative rule applies there
        assert_close(out.t, ry, tol, "ln y (hidden 1)")
    else:
        assert_close(out.t, ry, tol, "ln y")
    assert_close(mean.t, rm, tol, "ln mean")
    assert_close(rstd.t, rr, tol, "ln rstd")
    # statistics are fp32 whatever the data dtype: hold them to a tighter, informational-grade bound
    assert_close(mean.t, rm, 1e-3 if dtype == BF16 else 1e-5, "ln mean (tight)")
    assert_close(rstd.t, rr, 1e-3 if dtype == BF16 else 1e-5, "ln rstd (tight)")
    if dtype == BF16:
        assert_bf16_tight(out.t, ry, "ln y", floor=8e-3)
    for gd in (out, mean, rstd):
        gd.check("ln")


@pytest.mark.parametrize("rows,hidden,dtype", [(2048, 4096, BF16), (1185, 4096, BF16), (300, 4096, F32), (65, 256, BF16),
                                               (9, 20480, F32), (33, 1001, F32), (7, 1, F32)])
@pytest.mark.parametrize("seed", SEEDS)
def test_layernorm_erf_gelu_parity(kop, rows, hidden, dtype, seed):
    """The error-function GELU variant: same kernels, other prologue."""
    x, r, b, g, be = synth.layernorm_inputs(rows, hidden, dtype, seed, "cuda")
    y = Guarded((rows, hidden), dtype)
    mean = Guarded((rows,), F32)
    rstd = Guarded((rows,), F32)
    kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5, out=y.t, mean=mean.t, rstd=rstd.t, erf_form=True)
    ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5, threads=None,
                                                     erf_form=True)
    tol = tol_of(dtype)
    assert_close(y.t, ry, tol, "erf-gelu layernorm y")
    assert_close(mean.t, rm, 1e-5 if dtype == F32 else 1e-3, "erf-gelu layernorm mean")
    if hidden > 1:
        assert_close(rstd.t, rr, 1e-5 if dtype == F32 else 1e-3, "erf-gelu layernorm rstd")
    if dtype == BF16:
        assert_bf16_tight(y.t, ry, "erf-gelu layernorm y")
    for gb in (y, mean, rstd):
        gb.check("erf-gelu layernorm")
    # and it is not the tanh form: the two differ by the approximation error of the tanh form
    if hidden >= 256 and dtype == F32:
        y0, _, _ = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
        assert float((y0 - y.t).abs().max()) > 1e-5


def test_layernorm_full_config_seed0(kop):
    c = synth.CONFIGS["layernorm"]
    x, r, b, g, be = synth.layernorm_inputs(c["rows"], c["hidden"], c["dtype"], 0, "cuda")
    y, mean, rstd = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, c["eps"])
    ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), c["eps"],
                                                     threads=None)
    assert_close(y, ry, 2e-2, "ln full y")
    assert_close(mean, rm, 2e-2, "ln full mean")
    assert_close(rstd, rr, 2e-2, "ln full rstd")
    assert_bf16_tight(y, ry, "ln full y", floor=8e-3)
    y2, m2, r2 = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, c["eps"])
    assert torch.equal(y, y2) and torch.equal(mean, m2) and torch.equal(rstd, r2)


def test_layernorm_options(kop):
    x, r, b, g, be = synth.layernorm_inputs(100, 4096, BF16, 3, "cuda")
    ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5)
    # no statistics outputs
    y, m, s = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5, want_stats=False)
    assert m is None and s is None
    assert_close(y, ry, 2e-2, "no stats")
    # in place over x, and over the residual
    xi = x.clone()
    kop.kop_bias_gelu_residual_layernorm(xi, r, b, g, be, 1e-5, out=xi)
    assert_close(xi, ry, 2e-2, "in place x")
    ri = r.clone()
    kop.kop_bias_gelu_residual_layernorm(x, ri, b, g, be, 1e-5, out=ri)
    assert_close(ri, ry, 2e-2, "in place residual")
    # strided inputs and output
    wx = torch.zeros((100, 8192), dtype=BF16, device="cuda")
    wx[:, 4096:] = x
    wr = torch.zeros((100, 4104), dtype=BF16, device="cuda")
    wr[:, :4096] = r
    wo = torch.zeros((100, 4096 + 64), dtype=BF16, device="cuda")
    kop.kop_bias_gelu_residual_layernorm(wx[:, 4096:], wr[:, :4096], b, g, be, 1e-5, out=wo[:, 64:])
    assert_close(wo[:, 64:], ry, 2e-2, "strided")
    assert bool((wo[:, :64] == 0).all())
    # misaligned base -> scalar kernel
    wx2 = torch.zeros((100, 4099), dtype=BF16, device="cuda")
    wx2[:, 3:] = x
    y, _, _ = kop.kop_bias_gelu_residual_layernorm(wx2[:, 3:], r, b, g, be, 1e-5)
    assert_close(y, ry, 2e-2, "misaligned")
    e = torch.empty((0, 4096), dtype=BF16, device="cuda")
    y, _, _ = kop.kop_bias_gelu_residual_layernorm(e, e, b, g, be, 1e-5)
    assert y.shape == (0, 4096)


# ------------------------------------------------------------------------------------------ BN + ReLU + pool

BN_SHAPES = [
    (8, 256, 56, 56, F32),     # benchmark plane
    (3, 5, 56, 56, BF16),
    (4, 16, 7, 7, F32),        # small odd plane: bundles of four planes
    (4, 16, 14, 14, F32),      # small plane: 16-byte loads
    (2, 3, 112, 112, F32),     # multi-trip plane
    (2, 7, 33, 35, F32),       # large odd plane: scalar CTA
    (5, 3, 1, 1, F32),
    (2, 8, 64, 64, BF16),
    (16, 2048, 7, 7, BF16),    # 98-byte planes: bundles of eight
    (3, 5, 7, 7, BF16),
    (3, 5, 14, 14, BF16),      # 392-byte planes: 8-byte loads
    (2, 3, 5, 9, torch.float16),
    (2, 6, 2, 3, F32),         # 24-byte planes: 8-byte loads of fp32
    (2, 3, 31, 31, F32),       # 961-element planes, four per run
    (7, 9, 3, 3, F32),
    (2, 1100, 1, 1, BF16),     # one element per plane, runs of 1024 planes
    # planes that are not whole vectors in bundles of 2, 4 or 8: planes left over after the last bundle, vectors that
    # straddle two planes and two channels, channel indices that wrap inside a bundle, 16 lanes a bundle
    (3, 5, 7, 7, F32),         # 15 planes: three bundles of four and three planes left over
    (1, 3, 7, 7, BF16),        # fewer planes than a bundle of eight: the lanes-per-plane kernel alone
    (5, 2, 7, 7, torch.float16),   # C = 2: the channel wraps four times inside a bundle
    (2, 9, 9, 9, F32),         # 81 vectors a bundle
    (3, 7, 9, 11, BF16),       # 198-byte planes: bundles of eight, 99 vectors each, 16 lanes a bundle
    (4, 6, 5, 5, F32),
    (2, 11, 3, 3, BF16),       # 9-element planes, eight a bundle
    (3, 1, 13, 13, torch.float16),
]


@pytest.mark.parametrize("N,C,H,W,dtype", BN_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_bn_relu_avgpool_parity(kop, N, C, H, W, dtype, seed):
    x, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
    out = Guarded((N, C, H, W), dtype)
    pooled = Guarded((N, C), F32)
    kop.kop_bn_relu_avgpool(x, scale, shift, out=out.t, pooled=pooled.t)
    ry, rp = kopref.bn_relu_avgpool(host(x), host(scale), host(shift), threads=None)
    tol = tol_of(dtype)
    assert_close(out.t, ry, tol, "bn y")
    assert_close(pooled.t, rp, tol, "bn pooled")
    assert_close(pooled.t, rp, 1e-5, "bn pooled (fp32-grade: pooled sums unrounded activations)")
    if dtype == BF16:
        assert_bf16_tight(out.t, ry, "bn y", floor=1e-6)
    out.check("bn y")
    pooled.check("bn pooled")


BN_NHWC_SHAPES = [
    (8, 256, 56, 56, F32),     # benchmark image, channels last: 16-vector tiles, rows split over a cluster of 8
    (120, 256, 24, 24, BF16),  # cluster of 2
    (3, 64, 28, 28, BF16),     # 8 channel vectors
    (2, 2048, 7, 7, F32),      # wide and shallow: 16-vector tiles
    (300, 32, 5, 5, BF16),     # many small images
    (2, 20, 9, 9, F32),        # 5 vectors: ragged tile
    (3, 24, 6, 6, BF16),       # 3 vectors
    (2, 7, 33, 35, F32),       # 7 channels: scalar kernel
    (2, 33, 4, 4, BF16),       # scalar kernel bf16, two lane tiles
    (5, 4, 1, 1, F32),
    (2, 1, 3, 3, F32),         # C == 1: both layouts coincide (takes the NCHW path)
]


@pytest.mark.parametrize("N,C,H,W,dtype", BN_NHWC_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_bn_relu_avgpool_channels_last_parity(kop, N, C, H, W, dtype, seed):
    x, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
    x = x.contiguous(memory_format=torch.channels_last)
    buf = Guarded((N, H, W, C), dtype)                       # NHWC memory ...
    out = buf.t.permute(0, 3, 1, 2)                          # ... addressed as NCHW
    pooled = Guarded((N, C), F32)
    kop.kop_bn_relu_avgpool(x, scale, shift, out=out, pooled=pooled.t)
    ry, rp = kopref.bn_relu_avgpool(host(x), host(scale), host(shift), threads=None)
    tol = tol_of(dtype)
    assert_close(out, ry, tol, "bn nhwc y")
    assert_close(pooled.t, rp, 1e-5, "bn nhwc pooled")
    if dtype == BF16:
        assert_bf16_tight(out, ry, "bn nhwc y", floor=1e-6)
    buf.check("bn nhwc y")
    pooled.check("bn nhwc pooled")


def test_bn_channels_last_full_config_in_place_and_nan(kop):
    c = synth.CONFIGS["bn_pool"]
    x, scale, shift = synth.bn_pool_inputs(c["N"], c["C"], c["H"], c["W"], c["dtype"], 0, "cuda")
    xl = x.contiguous(memory_format=torch.channels_last)
    y, p = kop.kop_bn_relu_avgpool(xl, scale, shift)
    assert y.is_contiguous(memory_format=torch.channels_last)
    # the NCHW kernel on the same logical tensor is an independent GPU path: same values up to sum order
    y0, p0 = kop.kop_bn_relu_avgpool(x, scale, shift)
    assert torch.equal(y.contiguous(), y0)
    assert float((p - p0).abs().max()) < 1e-5
    ry, rp = kopref.bn_relu_avgpool(host(x[:8]), host(scale), host(shift), threads=None)
    assert_close(y[:8], ry, 1e-5, "bn nhwc full y (first 8 images)")
    assert_close(p[:8], rp, 1e-5, "bn nhwc full pooled")
    y2, p2 = kop.kop_bn_relu_avgpool(xl, scale, shift)
    assert torch.equal(y, y2) and torch.equal(p, p2)
    xi = xl[:4].clone(memory_format=torch.channels_last)
    _, pi = kop.kop_bn_relu_avgpool(xi, scale, shift, out=xi)
    # (the tile width, hence the summation order, may differ with the batch size: values, not bits)
    assert torch.equal(xi, y[:4]) and float((pi - p[:4]).abs().max()) < 1e-5
    xn = xl[:1].clone(memory_format=torch.channels_last)
    xn[0, 3, 5, 7] = float("nan")
    yn, pn = kop.kop_bn_relu_avgpool(xn, scale, shift)
    assert bool(torch.isnan(yn[0, 3, 5, 7])) and bool(torch.isnan(pn[0, 3])) and int(torch.isnan(pn).sum()) == 1


def test_bn_full_config_seed0_and_options(kop):
    c = synth.CONFIGS["bn_pool"]
    x, scale, shift = synth.bn_pool_inputs(c["N"], c["C"], c["H"], c["W"], c["dtype"], 0, "cuda")
    y, p = kop.kop_bn_relu_avgpool(x, scale, shift)
    ry, rp = kopref.bn_relu_avgpool(host(x), host(scale), host(shift), threads=None)
    assert_close(y, ry, 1e-5, "bn full y")
    assert_close(p, rp, 1e-5, "bn full pooled")
    y2, p2 = kop.kop_bn_relu_avgpool(x, scale, shift)
    assert torch.equal(y, y2) and torch.equal(p, p2)
    # in place
    xi = x[:4].clone()
    _, pi = kop.kop_bn_relu_avgpool(xi, scale, shift, out=xi)
    assert_close(xi, ry[:4], 1e-5, "bn in place")
    assert_close(pi, rp[:4], 1e-5, "bn in place pooled")
    # NaN propagates through ReLU into the activation and the pooled mean
    xn = x[:1].clone()
    xn[0, 3, 5, 7] = float("nan")
    yn, pn = kop.kop_bn_relu_avgpool(xn, scale, shift)
    assert bool(torch.isnan(yn[0, 3, 5, 7])) and bool(torch.isnan(pn[0, 3]))
    assert int(torch.isnan(pn).sum()) == 1
    # x and y must share one layout: a channels-last input with an NCHW output is rejected, not misread,
    # and so is a tensor that is neither (a sliced width)
    with pytest.raises(kop.KopError) as ei:
        kop.kop_bn_relu_avgpool(x[:2].contiguous(memory_format=torch.channels_last), scale, shift,
                                out=torch.empty_like(x[:2]))
    assert ei.value.status == 3
    with pytest.raises(kop.KopError) as ei:
        kop.kop_bn_relu_avgpool(x[:2, :, :, :48], scale, shift, out=torch.empty_like(x[:2, :, :, :48]))
    assert ei.value.status == 3
    e = torch.empty((0, 256, 56, 56), dtype=F32, device="cuda")
    ye, pe = kop.kop_bn_relu_avgpool(e, scale, shift)
    assert ye.shape == e.shape and pe.shape == (0, 256)


# ------------------------------------------------------------------------------------------ softmax variants

def assert_close_with_neg_inf(got, ref, tol, what):
    g = to_f64(got)
    assert np.array_equal(np.isneginf(g), np.isneginf(ref)), what + ": masked positions"
    fin = ~np.isneginf(ref)
    err = np.abs(g[fin] - ref[fin])
    assert np.all(err <= tol * np.maximum(1.0, np.abs(ref[fin]))), f"{what}: max err {err.max():.3e}"


@pytest.mark.parametrize("rows,cols,dtype", [(96, 512, F32), (1024, 128, BF16), (130, 1000, F32), (66, 1001, F32),
                                             (20, 16384, BF16), (12, 20000, F32), (9, 1, F32), (4, 50000, BF16),
                                             (65, 4096, BF16), (33, 2048, F32)])
@pytest.mark.parametrize("seed", SEEDS)
def test_softmax_opts_parity(kop, rows, cols, dtype, seed):
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    tol = tol_of(dtype)
    period = cols if cols <= 512 else cols // 3
    for log_output in (False, True):
        for causal in (0, period):
            for use_bias in (True, False):
                y = Guarded((rows, cols), dtype)
                kop.kop_softmax_opts(x, bias if use_bias else None, 0.125, log_output, causal, out=y.t)
                ref = kopref.softmax_opts(host(x), host(bias) if use_bias else None, 0.125, log_output, causal, threads=None)
                what = f"softmax_opts log={log_output} causal={causal} bias={use_bias}"
                if log_output:
                    assert_close_with_neg_inf(y.t, ref, tol, what)
                else:
                    assert_close(y.t, ref, tol, what)
                y.check(what)
    # no options: the same values as the plain entry point (another kernel path for short rows)
    plain = kop.kop_softmax_scale_bias(x, bias, 0.125)
    assert_close(kop.kop_softmax_opts(x, bias, 0.125), to_f64(plain), 1e-6 if dtype == F32 else tol, "softmax_opts without options")


@pytest.mark.parametrize("rows,cols,period,dtype", [(300, 256, 64, BF16), (77, 768, 256, F32), (1000, 64, 64, torch.float16),
                                                    (515, 1024, 1, BF16), (131, 1000, 500, F32), (64, 32, 7, F32)])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_softmax_causal_short_rows(kop, rows, cols, period, dtype, seed):
    """Causal rows of up to 128 vectors (the lanes-per-row and warp-per-row kernels): periods that wrap within the
    rows, a visible range that starts inside the row (cols - period > 0), a period of one, with and without a bias."""
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    for use_bias in (False, True):
        y = Guarded((rows, cols), dtype)
        kop.kop_softmax_opts(x, bias if use_bias else None, 0.25, False, period, out=y.t)
        ref = kopref.softmax_opts(host(x), host(bias) if use_bias else None, 0.25, False, period, threads=None)
        assert_close(y.t, ref, tol_of(dtype), f"causal short rows bias={use_bias}")
        y.check("causal short rows")
        # masked columns are exact zeros
        g = to_f64(y.t)
        assert np.array_equal(g == 0.0, ref == 0.0) or np.all(g[ref == 0.0] == 0.0)


def test_softmax_opts_attention_shape_and_validation(kop):
    # attention scores of 4 heads x 256 queries over 256 keys, square causal mask, in place
    S = 256
    x, _ = synth.softmax_inputs(4 * S, S, BF16, 3, "cuda")
    ref = kopref.softmax_opts(host(x), None, 0.125, False, S, threads=None)
    xi = x.clone()
    kop.kop_softmax_opts(xi, None, 0.125, False, S, out=xi)
    assert_close(xi, ref, 2e-2, "causal attention softmax in place")
    assert bool((xi.view(4, S, S).triu(1) == 0).all())
    assert bool(torch.allclose(xi.float().sum(dim=1), torch.ones(4 * S, device="cuda"), atol=2e-2))
    with pytest.raises(kop.KopError) as ei:
        kop.kop_softmax_opts(x, None, 1.0, False, S + 1)
    assert ei.value.status == 2


# ------------------------------------------------------------------------------------------ cross-entropy

CE_SHAPES = [
    (2048, 32000, BF16),   # benchmark row length
    (300, 32000, F32),
    (257, 4096, BF16),
    (100, 50264, BF16),    # multi-batch rows (more than 16 vectors per thread)
    (64, 131072, BF16),
    (33, 1000, F32),
    (21, 32001, BF16),     # odd vocab: every row starts at another offset from a 16-byte boundary
    (37, 50257, BF16),     # head and tail elements around the aligned vectors, several batches a thread
    (19, 50257, F32),
    (300, 1001, BF16),     # odd and short: lanes per row with edge elements
    (523, 197, F32),
    (1000, 77, torch.float16),
    (200, 7, BF16),        # shorter than one vector: edge elements only
    (64, 4102, F32),       # every second row starts 8 bytes off a boundary
    (9, 1, F32),
    (5, 8, BF16),
    # small vocabularies (rows of at most 16 KB): 4, 8, 16 and 32 lanes of a warp per row; row counts that span
    # several ticket groups and leave part of the last warp without a row
    (3001, 16, BF16),
    (1025, 1000, BF16),
    (777, 1024, BF16),
    (515, 2048, BF16),
    (259, 4096, F32),
    (70, 8192, BF16),
    (1031, 100, F32),
    (600, 1000, torch.float16),
]


@pytest.mark.parametrize("rows,vocab,dtype", CE_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_ce_parity(kop, rows, vocab, dtype, seed):
    if rows * vocab > 40_000_000 and seed not in (0, 42):
        # every seed runs at this row length; the other three use fewer rows (rows are independent, so the
        # kernel variant is the same) to keep the CPU oracle's time bounded. 640 rows still span three ticket
        # groups with a ragged last one.
        rows = 640
    z, lab = synth.ce_inputs(rows, vocab, dtype, seed, "cuda")
    loss = Guarded((rows,), F32)
    mean = Guarded((1,), F32)
    bad = Guarded((1,), torch.int32)
    kop.kop_ce_loss_rowwise(z, lab, loss=loss.t, mean_loss=mean.t, bad_label_count=bad.t)
    rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab), threads=None)
    tol = tol_of(dtype)
    assert_close(loss.t, rl, tol, "ce loss")
    assert_close(mean.t, np.array([rmean]), tol, "ce mean")
    # the kernel computes in fp32 whatever the logits' dtype: hold it to fp32-grade accuracy too
    assert_close(loss.t, rl, 2e-5, "ce loss (fp32-grade)")
    assert_close(mean.t, np.array([rmean]), 2e-5, "ce mean (fp32-grade)")
    assert int(bad.t.item()) == rbad == 0
    for gd in (loss, mean, bad):
        gd.check("ce")


def test_ce_full_config_sampled_rows_and_mean(kop):
    c = synth.CONFIGS["ce_loss"]
    z, lab = synth.ce_inputs(c["rows"], c["vocab"], c["dtype"], 0, "cuda")
    loss, mean, bad = kop.kop_ce_loss_rowwise(z, lab)
    idx = torch.from_numpy(np.random.default_rng(0).choice(c["rows"], 1024, replace=False)).to("cuda")
    idx = torch.cat([idx, torch.tensor([0, c["rows"] - 1], device="cuda")])
    rl, _, _ = kopref.ce_loss_rowwise(host(z[idx]), host(lab[idx]), threads=None)
    assert_close(loss[idx], rl, 2e-2, "ce full sampled rows")
    assert_close(loss[idx], rl, 2e-5, "ce full sampled rows (fp32-grade)")
    # property that holds at any size: the mean output is the mean of the per-row losses
    assert abs(float(mean.item()) - to_f64(loss).mean()) <= 1e-5 * 13
    assert int(bad.item()) == 0
    # loss >= 0 and close to ln V + sigma^2/2 on average for N(0,2) logits
    assert float(loss.min().item()) >= 0.0
    assert abs(float(mean.item()) - (np.log(c["vocab"]) + 2.0)) < 0.1
    l2, m2, _ = kop.kop_ce_loss_rowwise(z, lab)
    assert torch.equal(loss, l2) and torch.equal(mean, m2)


def test_ce_options(kop):
    z, lab = synth.ce_inputs(200, 4096, BF16, 5, "cuda")
    # bad labels: NaN loss for those rows, counted, mean NaN
    lab2 = lab.clone()
    lab2[3] = -1
    lab2[77] = 4096
    loss, mean, bad = kop.kop_ce_loss_rowwise(z, lab2)
    rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab2))
    assert int(bad.item()) == rbad == 2
    assert bool(torch.isnan(loss[3])) and bool(torch.isnan(loss[77])) and bool(torch.isnan(mean[0]))
    assert_close(loss, rl, 2e-5, "ce with bad labels")
    # strided rows; workspace reuse across calls without clearing it
    wide = torch.zeros((200, 8192), dtype=BF16, device="cuda")
    wide[:, 4096:] = z
    ws = torch.full((64,), 0xFF, dtype=torch.uint8, device="cuda")     # garbage on entry
    for _ in range(3):
        loss, mean, bad = kop.kop_ce_loss_rowwise(wide[:, 4096:], lab, workspace=ws)
        rl, rmean, _ = kopref.ce_loss_rowwise(host(z), host(lab))
        assert_close(loss, rl, 2e-5, "ce strided")
        assert_close(mean, np.array([rmean]), 2e-5, "ce strided mean")
    # extreme logits: no overflow, -inf entries allowed
    zz = z.clone().float()
    zz[:, 0] = 3.0e4
    zz[:, 1] = float("-inf")
    zz = zz.to(BF16)
    lab_e = lab.clamp(min=2)                       # keep the label off the -inf column
    loss, _, _ = kop.kop_ce_loss_rowwise(zz, lab_e)
    rl, _, _ = kopref.ce_loss_rowwise(host(zz), host(lab_e))
    assert_close(loss, rl, 2e-2, "ce extreme")
    # uniform row -> ln V
    u = torch.full((4, 32000), -1.75, dtype=BF16, device="cuda")
    loss, mean, _ = kop.kop_ce_loss_rowwise(u, torch.tensor([0, 5, 31999, 16000], dtype=torch.int32, device="cuda"))
    assert torch.allclose(loss, torch.full_like(loss, float(np.log(32000))), rtol=0, atol=2e-5)
    e = torch.empty((0, 4096), dtype=BF16, device="cuda")
    l0, _, _ = kop.kop_ce_loss_rowwise(e, torch.empty((0,), dtype=torch.int32, device="cuda"))
    assert l0.shape == (0,)


# ------------------------------------------------------------------------------------------ MLP pieces

RMS_SHAPES = [(2048, 4096, BF16), (300, 4096, F32), (65, 512, BF16), (17, 16384, BF16),
              (9, 20480, F32), (5, 40008, BF16), (3, 20481, BF16), (21, 1001, BF16), (7, 1, F32),
              (19, 12288, BF16), (7, 10000, BF16)]       # packed rows with fp32 weights: 384 threads, and a ragged 320


@pytest.mark.parametrize("rows,hidden,dtype", RMS_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_rmsnorm_parity(kop, rows, hidden, dtype, seed):
    h, w, _, _ = synth.mlp_inputs(rows, hidden, 8, dtype, seed, "cuda")
    out = Guarded((rows, hidden), dtype)
    kop.kop_rmsnorm(h, w, 1e-6, out=out.t)
    ref = kopref.rmsnorm(host(h), host(w), 1e-6, threads=None)
    assert_close(out.t, ref, tol_of(dtype), "rmsnorm")
    if dtype == BF16:
        assert_bf16_tight(out.t, ref, "rmsnorm", floor=1e-6)
    out.check("rmsnorm")


@pytest.mark.parametrize("rows,hidden,dtype", [(2048, 4096, BF16), (300, 4096, F32), (65, 512, torch.float16), (17, 16384, BF16),
                                               (9, 20480, BF16), (33, 1001, F32), (5, 1, F32)])
@pytest.mark.parametrize("seed", SEEDS)
def test_residual_rmsnorm_parity(kop, rows, hidden, dtype, seed):
    h, w, _, _ = synth.mlp_inputs(rows, hidden, 1, dtype, seed, "cuda")
    _, d = synth.pair_inputs(rows, hidden, dtype, seed + 1, "cuda")
    hg, yg = Guarded((rows, hidden), dtype), Guarded((rows, hidden), dtype)
    kop.kop_residual_rmsnorm(h, d, w, 1e-6, h_out=hg.t, out=yg.t)
    rh, ry = kopref.residual_rmsnorm(host(h), host(d), host(w), 1e-6, threads=None)
    tol = tol_of(dtype)
    assert_close(hg.t, rh, tol, "residual_rmsnorm h")
    assert_close(yg.t, ry, tol, "residual_rmsnorm y")
    if dtype == BF16:
        assert_bf16_tight(yg.t, ry, "residual_rmsnorm y")
    hg.check("h")
    yg.check("y")
    # h equals the stand-alone residual add bit for bit; the residual stream updated in place
    assert torch.equal(hg.t, kop.kop_residual_add(h, d))
    hi = h.clone()
    _, yi = kop.kop_residual_rmsnorm(hi, d, w, 1e-6, h_out=hi)
    assert torch.equal(hi, hg.t) and torch.equal(yi, yg.t)
    with pytest.raises(kop.KopError) as ei:
        kop.kop_residual_rmsnorm(h, d, w, 1e-6, h_out=hg.t, out=hg.t)          # the two outputs must differ
    assert ei.value.status == 6


SILU_SHAPES = [(512, 14336, BF16), (100, 14336, F32), (33, 1000, BF16), (17, 1001, F32),
               (64, 8, BF16), (5, 1, F32)]


@pytest.mark.parametrize("rows,inter,dtype", SILU_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_silu_mul_parity(kop, rows, inter, dtype, seed):
    gu = synth.gate_up_inputs(rows, inter, dtype, seed, "cuda", std=3.0)
    out = Guarded((rows, inter), dtype)
    kop.kop_silu_mul(gu, out=out.t)
    ref = kopref.silu_mul(host(gu), threads=None)
    assert_close(out.t, ref, tol_of(dtype), "silu_mul")
    if dtype == BF16:
        assert_bf16_tight(out.t, ref, "silu_mul", floor=1e-6)
    out.check("silu_mul")


ADD_SHAPES = [(2048, 4096, BF16), (100, 4096, F32), (33, 1001, BF16), (1, 7, F32)]


@pytest.mark.parametrize("rows,cols,dtype", ADD_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_residual_add_parity(kop, rows, cols, dtype, seed):
    a, b = synth.pair_inputs(rows, cols, dtype, seed, "cuda")
    out = Guarded((rows, cols), dtype)
    kop.kop_residual_add(a, b, out=out.t)
    ref = kopref.residual_add(host(a), host(b), threads=None)
    if dtype == F32:
        # one fp32 add, correctly rounded: equal to the float64 sum rounded to fp32
        assert np.array_equal(to_f64(out.t), ref.astype(np.float32).astype(np.float64))
    else:
        assert_close(out.t, ref, 2e-2, "residual_add")
        assert_bf16_tight(out.t, ref, "residual_add", floor=1e-6)
    out.check("residual_add")


def test_mlp_pieces_options(kop):
    h, w, _, _ = synth.mlp_inputs(64, 4096, 8, BF16, 9, "cuda")
    ref = kopref.rmsnorm(host(h), host(w), 1e-6)
    hi = h.clone()
    kop.kop_rmsnorm(hi, w, 1e-6, out=hi)
    assert_close(hi, ref, 2e-2, "rmsnorm in place")
    wide = torch.zeros((64, 4096 + 72), dtype=BF16, device="cuda")
    wide[:, 72:] = h
    assert_close(kop.kop_rmsnorm(wide[:, 72:], w, 1e-6), ref, 2e-2, "rmsnorm strided")
    wide2 = torch.zeros((64, 4097), dtype=BF16, device="cuda")
    wide2[:, 1:] = h
    assert_close(kop.kop_rmsnorm(wide2[:, 1:], w, 1e-6), ref, 2e-2, "rmsnorm misaligned")
    # silu_mul on a strided view and residual add in place, with strided operands
    gu = synth.gate_up_inputs(50, 1024, BF16, 2, "cuda", std=3.0)
    wg = torch.zeros((50, 4096), dtype=BF16, device="cuda")
    wg[:, 1024:3072] = gu
    assert_close(kop.kop_silu_mul(wg[:, 1024:3072]), kopref.silu_mul(host(gu)), 2e-2, "silu strided")
    a, b = synth.pair_inputs(50, 1024, BF16, 2, "cuda")
    rs = kopref.residual_add(host(a), host(b))
    ai = a.clone()
    kop.kop_residual_add(ai, b, out=ai)
    assert_close(ai, rs, 2e-2, "add in place")
    wa = torch.zeros((50, 2048), dtype=BF16, device="cuda")
    wa[:, 8:1032] = a
    assert_close(kop.kop_residual_add(wa[:, 8:1032], b), rs, 2e-2, "add strided")
    for fn, args in ((kop.kop_rmsnorm, (torch.empty((0, 64), dtype=BF16, device="cuda"), w[:64].contiguous(), 1e-6)),
                     (kop.kop_silu_mul, (torch.empty((0, 64), dtype=BF16, device="cuda"),)),
                     (kop.kop_residual_add, (torch.empty((0, 64), dtype=BF16, device="cuda"),) * 2)):
        assert fn(*args).shape[0] == 0


# ------------------------------------------------------------------------------------------ row scale, mat-vec

ROW_SCALE_SHAPES = [(4096, 4096, F32), (1000, 4096, BF16), (33, 1001, F32), (257, 520, BF16), (1, 1, F32)]


@pytest.mark.parametrize("rows,cols,dtype", ROW_SCALE_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_row_scale_parity(kop, rows, cols, dtype, seed):
    a, b = synth.row_scale_inputs(rows, cols, dtype, seed, "cuda")
    out = Guarded((rows, cols), dtype)
    kop.kop_row_scale(a, b, out=out.t)
    ref = kopref.row_scale(host(a), host(b), threads=None)
    if dtype == F32:
        assert np.array_equal(to_f64(out.t), ref.astype(np.float32).astype(np.float64))    # one fp32 product
    else:
        assert_close(out.t, ref, 2e-2, "row_scale")
        assert_bf16_tight(out.t, ref, "row_scale", floor=1e-6)
    out.check("row_scale")


MATVEC_SHAPES = [(4096, 4096, BF16), (1000, 4096, F32), (37, 1000, BF16), (129, 257, F32), (9, 8, BF16), (3, 1, F32)]


@pytest.mark.parametrize("rows,k,dtype", MATVEC_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_matvec_bias_parity(kop, rows, k, dtype, seed):
    x, w, b_sum = synth.matvec_inputs(rows, k, dtype, seed, "cuda")
    out = Guarded((rows,), F32)
    kop.kop_matvec_bias(x, w, b_sum, out=out.t)
    ref = kopref.matvec_bias(host(x), host(w), np.float32(b_sum), threads=None)
    assert_close(out.t, ref, tol_of(dtype), "matvec_bias")
    assert_close(out.t, ref, 2e-5, "matvec_bias (fp32-grade: fp32 products and sums)")
    out.check("matvec_bias")


def test_row_ops_options_and_full_configs(kop):
    c = synth.CONFIGS["matvec_bias"]
    x, w, b_sum = synth.matvec_inputs(c["rows"], c["k"], c["dtype"], 0, "cuda")
    out = kop.kop_matvec_bias(x, w, b_sum)
    ref = kopref.matvec_bias(host(x), host(w), np.float32(b_sum), threads=None)
    assert_close(out, ref, 2e-5, "matvec full config")
    assert torch.equal(out, kop.kop_matvec_bias(x, w, b_sum))
    # strided rows
    wide = torch.zeros((100, 8192), dtype=BF16, device="cuda")
    wide[:, 4096:] = x[:100]
    assert_close(kop.kop_matvec_bias(wide[:, 4096:], w, b_sum), ref[:100], 2e-5, "matvec strided")
    wide2 = torch.zeros((100, 4097), dtype=BF16, device="cuda")
    wide2[:, 1:] = x[:100]
    assert_close(kop.kop_matvec_bias(wide2[:, 1:], w, b_sum), ref[:100], 2e-5, "matvec misaligned")
    # row scale in place and strided
    a, b = synth.row_scale_inputs(300, 4096, F32, 1, "cuda")
    rs = kopref.row_scale(host(a), host(b))
    bi = b.clone()
    kop.kop_row_scale(a, bi, out=bi)
    assert np.array_equal(to_f64(bi), rs.astype(np.float32).astype(np.float64))
    wb = torch.zeros((300, 8192), dtype=F32, device="cuda")
    wb[:, 1024:5120] = b
    assert np.array_equal(to_f64(kop.kop_row_scale(a, wb[:, 1024:5120])), rs.astype(np.float32).astype(np.float64))
    assert kop.kop_row_scale(a[:0], b[:0]).shape == (0, 4096)
    assert kop.kop_matvec_bias(x[:0], w, b_sum).shape == (0,)


# ------------------------------------------------------------------------------------------ coverage variants

RLN_SHAPES = [(2048, 4096, BF16), (1185, 4096, BF16), (300, 4096, F32), (65, 256, BF16), (9, 20480, BF16), (4, 33000, F32),
              (21, 513, F32),
              # plain LayerNorm of 16-bit rows: row pairs with 32 values a thread (64- and 160-thread CTAs, an odd row count)
              (1301, 2048, torch.float16), (1187, 5120, BF16), (1185, 6144, BF16), (1186, 8192, torch.float16)]


@pytest.mark.parametrize("rows,hidden,dtype", RLN_SHAPES)
@pytest.mark.parametrize("with_residual", [True, False])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_residual_layernorm_parity(kop, rows, hidden, dtype, with_residual, seed):
    x, r, _, g, be = synth.layernorm_inputs(rows, hidden, dtype, seed, "cuda")
    res = r if with_residual else None
    out = Guarded((rows, hidden), dtype)
    mean = Guarded((rows,), F32)
    rstd = Guarded((rows,), F32)
    kop.kop_residual_layernorm(x, res, g, be, 1e-5, out=out.t, mean=mean.t, rstd=rstd.t)
    ry, rm, rr = kopref.residual_layernorm(host(x), None if res is None else host(res), host(g), host(be), 1e-5,
                                           threads=None)
    assert_close(out.t, ry, tol_of(dtype), "rln y")
    assert_close(mean.t, rm, 1e-5, "rln mean (exact fp32 sums of the inputs)")
    assert_close(rstd.t, rr, 1e-5, "rln rstd")
    if dtype == BF16:
        assert_bf16_tight(out.t, ry, "rln y", floor=1e-6)
    for gd in (out, mean, rstd):
        gd.check("rln")


@pytest.mark.parametrize("rows,inter,dtype", [(512, 14336, BF16), (100, 4096, F32), (33, 1000, BF16), (17, 1001, F32), (5, 1, F32)])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_silu_mul_interleaved_parity(kop, rows, inter, dtype, seed):
    gu = synth.gate_up_inputs(rows, inter, dtype, seed, "cuda", std=3.0)
    out = Guarded((rows, inter), dtype)
    kop.kop_silu_mul_interleaved(gu, out=out.t)
    ref = kopref.silu_mul_interleaved(host(gu), threads=None)
    assert_close(out.t, ref, tol_of(dtype), "silu_mul_interleaved")
    if dtype == BF16:
        assert_bf16_tight(out.t, ref, "silu_mul_interleaved", floor=1e-6)
    out.check("silu_mul_interleaved")
    # same numbers as the split layout on the de-interleaved columns
    split = torch.cat([gu[:, 0::2], gu[:, 1::2]], dim=1).contiguous()
    assert torch.equal(out.t, kop.kop_silu_mul(split))


@pytest.mark.parametrize("rows,vocab,dtype", [(2048, 32000, BF16), (300, 4096, F32), (257, 50264, BF16), (21, 32001, BF16), (9, 8, F32),
                                              (1300, 1000, BF16), (523, 2048, BF16), (2051, 40, F32), (67, 8192, BF16),
                                              (37, 50257, BF16), (300, 197, F32), (129, 1001, torch.float16)])
@pytest.mark.parametrize("smoothing", [0.0, 0.1])
@pytest.mark.parametrize("seed", SEEDS[:3])
def test_ce_opts_parity(kop, rows, vocab, dtype, smoothing, seed):
    z, lab = synth.ce_inputs(rows, vocab, dtype, seed, "cuda")
    lab = lab.clone()
    lab[::5] = -100                                    # every fifth row is ignored
    loss = Guarded((rows,), F32)
    mean = Guarded((1,), F32)
    bad = Guarded((1,), torch.int32)
    cnt = Guarded((1,), torch.int32)
    total = Guarded((1,), F32)
    kop.kop_ce_loss_rowwise_opts(z, lab, -100, smoothing, loss=loss.t, mean_loss=mean.t, bad_label_count=bad.t,
                                 counted_rows=cnt.t, sum_loss=total.t)
    rl, rmean, rbad, rcnt = kopref.ce_loss_opts(host(z), host(lab), -100, smoothing, threads=None)
    assert_close(loss.t, rl, 2e-5, "ce opts loss")
    assert_close(mean.t, np.array([rmean]), 2e-5, "ce opts mean")
    # reduction "sum" against its own oracle function, to the same relative accuracy
    rsum = kopref.ce_loss_sum(host(z), host(lab), -100, smoothing, threads=None)
    assert_close(total.t, np.array([rsum]), 2e-5, "ce opts sum")
    # sum and mean come from one fixed-order total: mean is exactly that total divided by the count
    assert float(mean.t.item()) == float((total.t / cnt.t.float()).item())
    assert int(bad.t.item()) == rbad == 0 and int(cnt.t.item()) == rcnt
    assert bool((loss.t[::5] == 0).all())
    for gd in (loss, mean, bad, cnt, total):
        gd.check("ce opts")


def test_ce_opts_edge_cases(kop):
    z, lab = synth.ce_inputs(64, 4096, BF16, 3, "cuda")
    # no ignored row, no smoothing: bit-identical to the plain entry point
    a = kop.kop_ce_loss_rowwise_opts(z, lab, -100, 0.0)
    b = kop.kop_ce_loss_rowwise(z, lab)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and int(a[3].item()) == 64
    # everything ignored: zero losses, NaN mean, nothing counted
    allig = torch.full_like(lab, 7)
    l, m, bd, c = kop.kop_ce_loss_rowwise_opts(z, allig, 7, 0.2)
    assert bool((l == 0).all()) and bool(torch.isnan(m[0])) and int(c.item()) == 0 and int(bd.item()) == 0
    # a bad label next to ignored rows
    lab2 = lab.clone()
    lab2[1] = 4096
    lab2[2] = -100
    l, m, bd, c = kop.kop_ce_loss_rowwise_opts(z, lab2, -100, 0.0)
    assert bool(torch.isnan(l[1])) and float(l[2]) == 0.0 and int(bd.item()) == 1 and int(c.item()) == 63
    with pytest.raises(kop.KopError) as ei:
        kop.kop_ce_loss_rowwise_opts(z, lab, -100, 1.0)
    assert ei.value.status == 2
    # reduction "sum": nothing counted sums to 0 (the mean is NaN), a bad label makes it NaN, and it is
    # bit-identical run to run
    tot = torch.full((1,), -7.0, dtype=F32, device="cuda")
    kop.kop_ce_loss_rowwise_opts(z, allig, 7, 0.2, sum_loss=tot)
    assert float(tot.item()) == 0.0
    kop.kop_ce_loss_rowwise_opts(z, lab2, -100, 0.0, sum_loss=tot)
    assert bool(torch.isnan(tot[0]))
    t1, t2 = torch.empty_like(tot), torch.empty_like(tot)
    zz, ll = synth.ce_inputs(3000, 1000, BF16, 4, "cuda")
    kop.kop_ce_loss_rowwise_opts(zz, ll, -100, 0.1, sum_loss=t1)
    kop.kop_ce_loss_rowwise_opts(zz, ll, -100, 0.1, sum_loss=t2)
    assert torch.equal(t1, t2)
    assert_close(t1, np.array([kopref.ce_loss_sum(host(zz), host(ll), -100, 0.1, threads=None)]), 2e-5, "ce sum 3000 rows")


@pytest.mark.parametrize("vocab,dtype", [(32000, BF16),     # CTA per row, batches of four vectors
                                         (4096, BF16),      # 32 lanes per row
                                         (1024, F32),       # lanes-per-row kernel, 8-vector rows
                                         (64, BF16),        # four lanes per row
                                         (1001, F32),       # odd length: lanes per row with edge elements
                                         (197, BF16),
                                         (50257, BF16),     # odd and long: edge elements around the vector sweep
                                         (40000, F32)])
def test_ce_non_finite_logits(kop, vocab, dtype):
    """NaN and +inf logits make exactly their own row NaN, whichever kernel the shape selects and wherever in the
    row they sit (one element, a whole thread's batch, the whole row); -inf logits are ordinary. The oracle's
    max-shifted definition says the same (pinned against torch float64 on the CPU)."""
    rows = 12
    z, lab = synth.ce_inputs(rows, vocab, dtype, 8, "cuda")
    z = z.clone()
    z[1, vocab // 3] = float("nan")                     # one NaN
    z[2, : min(vocab, 64)] = float("nan")               # a run of NaNs: whole vectors / a thread's whole batch
    z[3, :] = float("nan")                              # nothing but NaNs
    z[4, vocab - 1] = float("inf")                      # +inf in the last column
    z[5, 0] = float("inf")
    z[5, vocab // 2] = float("inf")                     # two +inf
    z[6, 1::2] = float("-inf")                          # half the row masked: still a number
    z[7, :] = float("-inf")                             # empty row: NaN
    z[8, 0] = float("nan")
    z[8, 1:] = float("-inf")                            # a NaN among nothing
    lab = lab.clone()
    lab[6] = 0
    loss, mean, bad = kop.kop_ce_loss_rowwise(z, lab)
    rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab))
    want_nan = np.array([False, True, True, True, True, True, False, True, True, False, False, False])
    assert np.array_equal(np.isnan(rl), want_nan)
    assert np.array_equal(torch.isnan(loss).cpu().numpy(), want_nan), loss
    assert_close(loss, rl, 2e-5, "ce with non-finite logits")
    assert bool(torch.isnan(mean[0])) and np.isnan(rmean) and int(bad.item()) == 0
