"""GPU parity with fp16 (IEEE binary16) data: every entry point against the float64 oracle on the same
seeded inputs, five seeds, at shapes that take the vector kernels (several CTAs, ragged tails) and the
scalar ones. Tolerance |got - ref| <= 2e-3 * max(1, |ref|) (the RNE store is 2^-11 relative; see
tests/_util.py), fp32 statistics outputs at their usual fp32-grade bounds."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_close, to_f64

pytestmark = pytest.mark.gpu
F16 = torch.float16
TOL = 2e-3
SEEDS = synth.SEEDS


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


@pytest.mark.parametrize("rows,cols", [(300, 4096), (65, 1000), (33, 1001), (9, 20480), (5, 1)])
@pytest.mark.parametrize("seed", SEEDS)
def test_fp16_row_kernels(kop, rows, cols, seed):
    x, bias = synth.softmax_inputs(rows, cols, F16, seed, "cuda")
    y = Guarded((rows, cols), F16)
    kop.kop_softmax_scale_bias(x, bias, 0.125, out=y.t)
    assert_close(y.t, kopref.softmax_scale_bias(host(x), host(bias), 0.125, threads=None), TOL, "softmax")
    y.check("softmax")
    if cols >= 2:
        x, r, b, g, be = synth.layernorm_inputs(rows, cols, F16, seed, "cuda")
        y, mu, rs = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
        ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5, threads=None)
        assert_close(y, ry, TOL, "layernorm y")
        assert_close(mu, rm, 1e-3, "layernorm mean")
        assert_close(rs, rr, 1e-3, "layernorm rstd")
        y, _, _ = kop.kop_residual_layernorm(x, None, g, be, 1e-5)
        assert_close(y, kopref.residual_layernorm(host(x), None, host(g), host(be), 1e-5, threads=None)[0], TOL, "plain layernorm")
    h, w, _, _ = synth.mlp_inputs(rows, cols, 1, F16, seed, "cuda")
    assert_close(kop.kop_rmsnorm(h, w, 1e-6), kopref.rmsnorm(host(h), host(w), 1e-6, threads=None), TOL, "rmsnorm")
    z, lab = synth.ce_inputs(rows, cols, F16, seed, "cuda")
    loss, mean, bad = kop.kop_ce_loss_rowwise(z, lab)
    rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab), threads=None)
    assert_close(loss, rl, 2e-5, "ce loss (fp32 output)")
    assert abs(float(mean) - rmean) <= 2e-5 * max(1.0, abs(rmean)) and int(bad) == rbad
    loss, mean, bad, cnt = kop.kop_ce_loss_rowwise_opts(z, lab, -100, 0.1)
    rl, rmean, rbad, rcnt = kopref.ce_loss_opts(host(z), host(lab), -100, 0.1, threads=None)
    assert_close(loss, rl, 2e-5, "ce opts loss")
    gu = synth.gate_up_inputs(rows, cols, F16, seed, "cuda")
    assert_close(kop.kop_silu_mul(gu), kopref.silu_mul(host(gu), threads=None), TOL, "silu_mul")
    assert_close(kop.kop_silu_mul_interleaved(gu), kopref.silu_mul_interleaved(host(gu), threads=None), TOL, "silu_mul_interleaved")
    a, b2 = synth.pair_inputs(rows, cols, F16, seed, "cuda")
    assert_close(kop.kop_residual_add(a, b2), kopref.residual_add(host(a), host(b2), threads=None), TOL, "residual_add")
    av, bm = synth.row_scale_inputs(rows, cols, F16, seed, "cuda")
    assert_close(kop.kop_row_scale(av, bm), kopref.row_scale(host(av), host(bm), threads=None), TOL, "row_scale")
    xv, wv, bs = synth.matvec_inputs(rows, cols, F16, seed, "cuda")
    ref = kopref.matvec_bias(host(xv), host(wv), bs, threads=None)
    mag = (host(xv).double().abs() @ host(wv).double().abs()).numpy() + abs(bs)
    assert np.all(np.abs(to_f64(kop.kop_matvec_bias(xv, wv, bs)) - ref) <= 1e-5 * np.maximum(1.0, mag)), "matvec"
    xc, mask = synth.cumsum_inputs(rows, cols, F16, seed, "cuda")
    ref = kopref.cumsum_rows(host(xc), host(mask), False, True, threads=None)
    got = to_f64(kop.kop_cumsum_rows(xc, mask, False, True))
    assert np.all(np.abs(got - ref) <= TOL * np.maximum(1.0, np.abs(ref).max(axis=1, keepdims=True))), "cumsum"


@pytest.mark.parametrize("N,C,H,W,groups", [(3, 64, 56, 56, 8), (2, 12, 7, 7, 4), (2, 32, 28, 28, 32), (2, 6, 17, 19, 3)])
@pytest.mark.parametrize("seed", SEEDS)
def test_fp16_image_kernels(kop, N, C, H, W, groups, seed):
    x, scale, shift = synth.bn_pool_inputs(N, C, H, W, F16, seed, "cuda")
    y, p = kop.kop_bn_relu_avgpool(x, scale, shift)
    ry, rp = kopref.bn_relu_avgpool(host(x), host(scale), host(shift), threads=None)
    assert_close(y, ry, TOL, "bn y")
    assert_close(p, rp, 1e-5, "bn pooled")
    yl, pl = kop.kop_bn_relu_avgpool(x.contiguous(memory_format=torch.channels_last), scale, shift)
    assert_close(yl, ry, TOL, "bn nhwc y")
    assert_close(pl, rp, 1e-5, "bn nhwc pooled")
    xg, gamma, beta = synth.groupnorm_inputs(N, C, H, W, F16, seed, "cuda")
    y, mu, rs = kop.kop_groupnorm_act(xg, gamma, beta, groups, 1e-5, 2)
    ry, rm, rr = kopref.groupnorm_act(host(xg), host(gamma), host(beta), groups, 1e-5, 2, threads=None)
    assert_close(y, ry, TOL, "groupnorm y")
    assert_close(mu, rm, 1e-5, "groupnorm mean")
    assert_close(rs, rr, 1e-5, "groupnorm rstd")
    for kernel, stride, padding in (((3, 3), (2, 2), (1, 1)), ((2, 2), (2, 2), (0, 0)), ((3, 2), (1, 2), (1, 0))):
        for mode in ("max", "avg"):
            y = kop.kop_affine_relu_pool2d(x, scale, shift, kernel, stride, padding, mode, True)
            ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), kernel, stride, padding, mode, True, threads=None)
            assert_close(y, ref, TOL, f"pool2d {kernel} {mode}")


def test_fp16_mlp_segment_and_overflow(kop):
    M, H, I = 256, 512, 1792
    hdl = kop.MlpHandle()
    try:
        h, w, W1, W2 = synth.mlp_inputs(M, H, I, F16, 0, "cuda")
        out = kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6)
        ref = kopref.mlp_segment(host(h), host(w), host(W1), host(W2), 1e-6, threads=None)
        assert_close(out, ref, 4 * TOL, "mlp segment (four roundings along the chain)")
    finally:
        hdl.close()
    # results beyond the fp16 range are stored as infinity, not as garbage
    a = torch.full((4, 64), 60000.0, dtype=F16, device="cuda")
    s = kop.kop_residual_add(a, a)
    assert bool(torch.isinf(s).all()) and bool((s > 0).all())
