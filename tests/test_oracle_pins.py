"""Pins for the float64 CPU oracle: every oracle function is checked against something
other than itself — closed forms, invariants, special cases that reduce to a library
routine (torch / scipy in float64), and 50-digit mpmath brute force on tiny inputs.

The paper prints no worked numeric example for any of these segments (it only names the
segment classes), so there are no paper-printed golden values; the pins are what the
mathematics fixes.
"""
import math

import mpmath as mp
import numpy as np
import pytest
import scipy.special
import torch
import torch.nn.functional as F

from oracle import kopref

mp.mp.dps = 50
RNG = np.random.default_rng(20260930)


def f32(a):
    return np.asarray(a, dtype=np.float32)


def to_bf16_bits(a):
    """fp32 -> bf16 bit patterns through torch (an independent RNE implementation)."""
    t = torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


# --------------------------------------------------------------------------- bf16 helpers

def test_bf16_widening_exhaustive_round_trip():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    wide = kopref.bf16_to_f64(bits)
    via_torch = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    finite = np.isfinite(via_torch)
    assert np.array_equal(wide[finite], via_torch[finite])
    assert np.array_equal(np.isnan(wide), np.isnan(via_torch))
    back = kopref.f64_to_bf16_rne(wide)
    keep = ~np.isnan(wide)
    assert np.array_equal(back[keep], bits[keep])


def test_bf16_rne_ties_and_against_torch():
    # 1 + 2^-8 lies exactly between 1 (even mantissa) and 1 + 2^-7: ties-to-even gives 1.
    assert kopref.f64_to_bf16_rne([1.0 + 2.0 ** -8])[0] == 0x3F80
    # 1 + 3*2^-8 lies between 1+2^-7 (odd) and 1+2^-6 (even): rounds up.
    assert kopref.f64_to_bf16_rne([1.0 + 3 * 2.0 ** -8])[0] == 0x3F82
    # just above / below a tie (not representable in fp32: shows there is no double rounding)
    assert kopref.f64_to_bf16_rne([1.0 + 2.0 ** -8 + 2.0 ** -40])[0] == 0x3F81
    assert kopref.f64_to_bf16_rne([1.0 + 2.0 ** -8 - 2.0 ** -40])[0] == 0x3F80
    assert kopref.f64_to_bf16_rne([-0.0])[0] == 0x8000
    assert kopref.f64_to_bf16_rne([1e40])[0] == 0x7F80
    v = RNG.standard_normal(4096).astype(np.float32) * np.float32(37.0)
    assert np.array_equal(kopref.f64_to_bf16_rne(v.astype(np.float64)), to_bf16_bits(v))
    tiny = (RNG.standard_normal(512) * 1e-39).astype(np.float32)      # bf16 subnormals
    assert np.array_equal(kopref.f64_to_bf16_rne(tiny.astype(np.float64)), to_bf16_bits(tiny))


# --------------------------------------------------------------------------- softmax

def mp_softmax_row(x, b, s):
    z = [mp.mpf(float(xi)) * mp.mpf(float(s)) + mp.mpf(float(bi)) for xi, bi in zip(x, b)]
    e = [mp.exp(t) for t in z]
    S = mp.fsum(e)
    return [float(t / S) for t in e]


def test_softmax_invariants():
    x = f32(RNG.standard_normal((37, 513)))
    b = f32(RNG.standard_normal(513) * 0.1)
    y = kopref.softmax_scale_bias(x, b, 0.125)
    assert np.all(np.abs(y.sum(axis=1) - 1.0) <= 1e-13)
    assert np.all((y >= 0.0) & (y <= 1.0))
    # shift invariance: adding a constant to every bias entry changes nothing
    y2 = kopref.softmax_scale_bias(x, f32(b + np.float32(3.0)), 0.125)
    assert np.max(np.abs(y - y2)) <= 1e-7     # b+3 is re-rounded to fp32: not bit-exact
    # constant row -> exactly uniform; one column -> 1
    yc = kopref.softmax_scale_bias(f32(np.full((3, 16), 2.5)), None, 0.125)
    assert np.array_equal(yc, np.full((3, 16), 1.0 / 16))
    assert np.array_equal(kopref.softmax_scale_bias(f32([[7.0]]), None, 0.125), [[1.0]])
    # scale 0 and no bias -> uniform whatever x is
    assert np.array_equal(kopref.softmax_scale_bias(x[:2, :8], None, 0.0), np.full((2, 8), 0.125))


def test_softmax_scale_before_bias_and_two_element_closed_form():
    # z = x*s + b (scale applies to x only): with x=(8,0), s=0.125, b=(0,2): z=(1,2)
    y = kopref.softmax_scale_bias(f32([[8.0, 0.0]]), f32([0.0, 2.0]), 0.125)
    assert y[0, 0] == pytest.approx(1.0 / (1.0 + math.e), rel=1e-15)
    assert y[0, 1] == pytest.approx(math.e / (1.0 + math.e), rel=1e-15)


def test_softmax_masked_column_and_all_masked_row():
    x = f32(RNG.standard_normal((2, 6)))
    b = f32([0, -np.inf, 0, 0, -np.inf, 0])
    y = kopref.softmax_scale_bias(x, b, 1.0)
    assert np.all(y[:, [1, 4]] == 0.0)
    keep = [0, 2, 3, 5]
    assert np.allclose(y[:, keep], kopref.softmax_scale_bias(x[:, keep], None, 1.0), rtol=0, atol=1e-16)
    ynan = kopref.softmax_scale_bias(x, f32([-np.inf] * 6), 1.0)
    assert np.all(np.isnan(ynan))


def test_softmax_matches_library_and_mpmath():
    x = f32(RNG.standard_normal((5, 8)) * 3)
    b = f32(RNG.standard_normal(8))
    y = kopref.softmax_scale_bias(x, b, 0.125)
    lib = scipy.special.softmax(x.astype(np.float64) * 0.125 + b.astype(np.float64), axis=1)
    assert np.max(np.abs(y - lib)) <= 1e-15
    for i in range(5):
        assert np.max(np.abs(y[i] - np.array(mp_softmax_row(x[i], b, 0.125)))) <= 1e-15
    # bf16 data path: values are widened exactly
    xb = to_bf16_bits(x)
    yb = kopref.softmax_scale_bias(xb, b, 0.125)
    xw = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.max(np.abs(yb - scipy.special.softmax(xw * 0.125 + b.astype(np.float64), axis=1))) <= 1e-15


# --------------------------------------------------------------------------- GELU (tanh form)

def mp_gelu(u):
    u = mp.mpf(u)
    return 0.5 * u * (1 + mp.tanh(mp.sqrt(2 / mp.pi) * (u + mp.mpf("0.044715") * u ** 3)))


def test_gelu_tanh_points_identity_limits():
    assert kopref.gelu_tanh(0.0) == 0.0
    for u in [-6.0, -2.5, -1.0, -0.3, 0.1, 0.5, 1.0, 2.0, 3.7, 8.0]:
        assert kopref.gelu_tanh(u) == pytest.approx(float(mp_gelu(u)), rel=2e-15, abs=1e-15)  # 1 + tanh cancels near -1
        # g(u) - g(-u) = u exactly in real arithmetic (tanh is odd)
        assert kopref.gelu_tanh(u) - kopref.gelu_tanh(-u) == pytest.approx(u, rel=1e-15)
    assert kopref.gelu_tanh(12.0) == 12.0
    assert abs(kopref.gelu_tanh(-12.0)) <= 1e-30
    # library: torch's tanh-approximate GELU in float64
    u = torch.linspace(-5, 5, 41, dtype=torch.float64)
    ref = F.gelu(u, approximate="tanh").numpy()
    got = np.array([kopref.gelu_tanh(float(t)) for t in u])
    assert np.max(np.abs(got - ref)) <= 1e-15


# --------------------------------------------------------------------------- bias+GELU+residual+LayerNorm

def test_layernorm_zero_mean_unit_variance_before_affine():
    H = 96
    x = f32(RNG.standard_normal((9, H)))
    r = f32(RNG.standard_normal((9, H)))
    b = f32(RNG.standard_normal(H) * 0.1)
    eps = 1e-5
    y, mu, rstd = kopref.bias_gelu_residual_layernorm(x, r, b, f32(np.ones(H)), f32(np.zeros(H)), eps)
    assert np.all(np.abs(y.mean(axis=1)) <= 1e-12)
    var = 1.0 / rstd ** 2 - eps                       # sigma^2 recovered from rstd
    assert np.allclose(y.var(axis=1), var / (var + eps), rtol=1e-12, atol=0)
    # mean output is the mean of v = r + gelu(x + b)
    v = r.astype(np.float64) + F.gelu(torch.from_numpy(x.astype(np.float64) + b.astype(np.float64)),
                                      approximate="tanh").numpy()
    assert np.allclose(mu, v.mean(axis=1), rtol=0, atol=1e-14)
    assert np.allclose(rstd, 1.0 / np.sqrt(v.var(axis=1) + eps), rtol=1e-13, atol=0)


def test_layernorm_closed_forms():
    # x = 0, bias = 0 -> gelu term vanishes, so v = r: plain LayerNorm of r.
    H = 64
    zeros = f32(np.zeros((1, H)))
    ones, nul = f32(np.ones(H)), f32(np.zeros(H))
    r = f32(np.arange(H, dtype=np.float64)[None, :])              # arithmetic progression
    y, mu, rstd = kopref.bias_gelu_residual_layernorm(zeros, r, nul, ones, nul, 1e-5)
    assert mu[0] == pytest.approx((H - 1) / 2, rel=1e-15)
    assert rstd[0] == pytest.approx(1.0 / math.sqrt((H * H - 1) / 12.0 + 1e-5), rel=1e-14)
    # two-element row [-1, 1]: mu = 0, var = 1 -> y = -+ 1/sqrt(1+eps)
    y2, _, _ = kopref.bias_gelu_residual_layernorm(f32(np.zeros((1, 2))), f32([[-1.0, 1.0]]),
                                                   f32([0, 0]), f32([1, 1]), f32([0, 0]), 1e-5)
    assert y2[0, 0] == pytest.approx(-1.0 / math.sqrt(1 + 1e-5), rel=1e-15)
    assert y2[0, 1] == pytest.approx(+1.0 / math.sqrt(1 + 1e-5), rel=1e-15)
    # affine step is elementwise: gamma, beta applied per column
    g = f32(RNG.standard_normal(H))
    be = f32(RNG.standard_normal(H))
    ya, _, _ = kopref.bias_gelu_residual_layernorm(zeros, r, nul, g, be, 1e-5)
    assert np.allclose(ya, y * g.astype(np.float64) + be.astype(np.float64), rtol=1e-14, atol=1e-14)


def test_layernorm_op_order_and_library():
    # distinguishes bias->gelu->residual->LN from any other order: compare with torch float64
    H = 40
    x = f32(RNG.standard_normal((6, H)) * 2)
    r = f32(RNG.standard_normal((6, H)))
    b = f32(RNG.standard_normal(H))
    g = f32(1 + 0.02 * RNG.standard_normal(H))
    be = f32(0.02 * RNG.standard_normal(H))
    y, mu, rstd = kopref.bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
    tx, tr, tb, tg, tbe = (torch.from_numpy(a.astype(np.float64)) for a in (x, r, b, g, be))
    v = tr + F.gelu(tx + tb, approximate="tanh")
    ref = F.layer_norm(v, (H,), tg, tbe, 1e-5).numpy()
    assert np.max(np.abs(y - ref)) <= 1e-13
    # bf16 inputs are widened exactly and v is not rounded
    xb, rb = to_bf16_bits(x), to_bf16_bits(r)
    yb, _, _ = kopref.bias_gelu_residual_layernorm(xb, rb, b, g, be, 1e-5)
    txb = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64)
    trb = torch.from_numpy(r).to(torch.bfloat16).to(torch.float64)
    refb = F.layer_norm(trb + F.gelu(txb + tb, approximate="tanh"), (H,), tg, tbe, 1e-5).numpy()
    assert np.max(np.abs(yb - refb)) <= 1e-13


def test_layernorm_mpmath_tiny():
    x = f32([[0.5, -1.25, 2.0, 0.0]])
    r = f32([[1.0, 0.25, -0.5, 3.0]])
    b = f32([0.1, -0.2, 0.3, 0.0])
    g = f32([1.0, 0.5, 2.0, -1.0])
    be = f32([0.0, 0.1, -0.1, 0.2])
    y, mu, rstd = kopref.bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
    v = [mp.mpf(float(r[0, j])) + mp_gelu(mp.mpf(float(x[0, j])) + mp.mpf(float(b[j]))) for j in range(4)]
    m = mp.fsum(v) / 4
    var = mp.fsum([(t - m) ** 2 for t in v]) / 4
    rs = 1 / mp.sqrt(var + mp.mpf(1e-5))
    ref = [float((v[j] - m) * rs * mp.mpf(float(g[j])) + mp.mpf(float(be[j]))) for j in range(4)]
    assert np.max(np.abs(y[0] - np.array(ref))) <= 1e-14
    assert mu[0] == pytest.approx(float(m), rel=1e-15)
    assert rstd[0] == pytest.approx(float(rs), rel=1e-14)


def test_welford_chan_merge_equals_two_pass():
    # The merge formula a single-pass method relies on, checked against the oracle's
    # two-pass statistics: delta = mu_b - mu_a; mu = mu_a + delta n_b/n;
    # M2 = M2_a + M2_b + delta^2 n_a n_b / n.
    H = 200
    r = f32(RNG.standard_normal((1, H)) * 3 + 5)
    _, mu, rstd = kopref.bias_gelu_residual_layernorm(f32(np.zeros((1, H))), r, f32(np.zeros(H)),
                                                     f32(np.ones(H)), f32(np.zeros(H)), 0.0)
    v = r[0].astype(np.float64)
    for cut in (1, 37, 100, 199):
        a, b = v[:cut], v[cut:]
        na, nb = len(a), len(b)
        mua, mub = a.mean(), b.mean()
        M2a, M2b = ((a - mua) ** 2).sum(), ((b - mub) ** 2).sum()
        d = mub - mua
        n = na + nb
        m = mua + d * nb / n
        M2 = M2a + M2b + d * d * na * nb / n
        assert m == pytest.approx(mu[0], rel=1e-14)
        assert 1.0 / math.sqrt(M2 / n) == pytest.approx(rstd[0], rel=1e-13)


# --------------------------------------------------------------------------- BN + ReLU + avgpool

def test_bn_relu_avgpool_special_cases():
    N, Cc, H, W = 2, 3, 5, 4
    x = f32(RNG.standard_normal((N, Cc, H, W)))
    one, nul = f32(np.ones(Cc)), f32(np.zeros(Cc))
    y, p = kopref.bn_relu_avgpool(x, one, nul)
    assert np.array_equal(y, np.maximum(x.astype(np.float64), 0.0))      # scale 1, shift 0 = ReLU
    assert np.allclose(p, y.mean(axis=(2, 3)), rtol=1e-15, atol=0)
    # all-positive plane: pooling is linear, p = scale * mean(x) + shift
    xp = f32(np.abs(x) + 0.5)
    sc, sh = f32([0.5, 1.0, 1.5]), f32([0.1, 0.2, 0.3])
    _, pp = kopref.bn_relu_avgpool(xp, sc, sh)
    expect = xp.astype(np.float64).mean(axis=(2, 3)) * sc.astype(np.float64) + sh.astype(np.float64)
    assert np.allclose(pp, expect, rtol=1e-14, atol=0)
    # all-negative after affine -> zeros
    yn, pn = kopref.bn_relu_avgpool(f32(-xp), sc, f32(-sh))
    assert np.all(yn == 0.0) and np.all(pn == 0.0)
    # constant plane
    yc, pc = kopref.bn_relu_avgpool(f32(np.full((1, 3, 2, 2), 2.0)), sc, sh)
    assert np.allclose(pc[0], 2.0 * sc.astype(np.float64) + sh.astype(np.float64), rtol=1e-15)
    # channel index is the second axis (a transposed-operand mistake fails here)
    xs = f32(np.ones((2, 3, 2, 2)))
    _, ps = kopref.bn_relu_avgpool(xs, f32([1, 2, 3]), nul)
    assert np.array_equal(ps, np.array([[1.0, 2.0, 3.0], [1.0, 2.0, 3.0]]))


def test_bn_relu_nan_propagates_and_library():
    x = f32(RNG.standard_normal((2, 4, 3, 3)))
    x[0, 1, 1, 1] = np.nan
    sc = f32(RNG.uniform(0.5, 1.5, 4))
    sh = f32(RNG.standard_normal(4) * 0.1)
    y, p = kopref.bn_relu_avgpool(x, sc, sh)
    assert np.isnan(y[0, 1, 1, 1]) and np.isnan(p[0, 1])
    assert not np.isnan(p[1]).any()
    # library: eval-mode batch_norm with mean 0 / var 1-eps folded, then relu, then adaptive pool
    xc = torch.from_numpy(np.nan_to_num(x).astype(np.float64))
    ref_y = F.relu(xc * torch.from_numpy(sc.astype(np.float64))[None, :, None, None]
                   + torch.from_numpy(sh.astype(np.float64))[None, :, None, None])
    ref_p = F.adaptive_avg_pool2d(ref_y, 1)[:, :, 0, 0].numpy()
    yy, ppp = kopref.bn_relu_avgpool(np.nan_to_num(x), sc, sh)
    assert np.max(np.abs(yy - ref_y.numpy())) <= 1e-15
    assert np.max(np.abs(ppp - ref_p)) <= 1e-15


# --------------------------------------------------------------------------- cross-entropy

def test_ce_closed_forms():
    V = 32000
    z = f32(np.full((3, V), -1.75))
    loss, mean, bad = kopref.ce_loss_rowwise(z, np.array([0, 17, V - 1], dtype=np.int32))
    assert np.all(np.abs(loss - math.log(V)) <= 1e-12)                  # uniform row -> ln V
    assert mean == pytest.approx(math.log(V), rel=1e-14) and bad == 0
    # two classes: loss = log1p(exp(z_other - z_label))
    z2 = f32([[1.5, -0.25], [1.5, -0.25]])
    l2, m2, _ = kopref.ce_loss_rowwise(z2, np.array([0, 1], dtype=np.int32))
    assert l2[0] == pytest.approx(math.log1p(math.exp(-1.75)), rel=1e-14)
    assert l2[1] == pytest.approx(math.log1p(math.exp(+1.75)), rel=1e-14)
    assert m2 == pytest.approx((l2[0] + l2[1]) / 2, rel=1e-15)          # mean divides by M


def test_ce_invariants_and_library():
    M, V = 11, 257
    z = f32(RNG.standard_normal((M, V)) * 2)
    lab = RNG.integers(0, V, M).astype(np.int32)
    loss, mean, bad = kopref.ce_loss_rowwise(z, lab)
    assert np.all(loss >= 0) and bad == 0
    # loss = logsumexp - label logit
    lse = scipy.special.logsumexp(z.astype(np.float64), axis=1)
    assert np.allclose(loss, lse - z[np.arange(M), lab].astype(np.float64), rtol=0, atol=1e-13)
    # library
    ref = F.cross_entropy(torch.from_numpy(z.astype(np.float64)), torch.from_numpy(lab.astype(np.int64)),
                          reduction="none").numpy()
    assert np.max(np.abs(loss - ref)) <= 1e-13
    assert mean == pytest.approx(ref.mean(), rel=1e-14)
    # sum over all possible labels of exp(-loss) is 1 (the softmax is a distribution)
    row = np.repeat(z[:1], V, axis=0)
    lall, _, _ = kopref.ce_loss_rowwise(row, np.arange(V, dtype=np.int32))
    assert abs(np.exp(-lall).sum() - 1.0) <= 1e-13
    # shift invariance (power-of-two shift keeps fp32 exact enough: use exact small ints)
    zi = f32(RNG.integers(-8, 8, (4, 33)))
    li = RNG.integers(0, 33, 4).astype(np.int32)
    a, _, _ = kopref.ce_loss_rowwise(zi, li)
    b, _, _ = kopref.ce_loss_rowwise(f32(zi + 100.0), li)
    assert np.max(np.abs(a - b)) <= 1e-12
    # large logits do not overflow (max subtraction)
    big, _, _ = kopref.ce_loss_rowwise(f32([[1000.0, 999.0]]), np.array([1], dtype=np.int32))
    assert big[0] == pytest.approx(math.log1p(math.exp(-1.0)) + 1.0, rel=1e-14)


def test_ce_online_merge_equals_two_pass_and_mpmath():
    V = 300
    z = f32(RNG.standard_normal((1, V)) * 4)
    lab = np.array([123], dtype=np.int32)
    loss, _, _ = kopref.ce_loss_rowwise(z, lab)
    zz = z[0].astype(np.float64)
    for cut in (1, 64, 299):
        # (m, s) (+) (m', s') = (max, s e^{m - max} + s' e^{m' - max})
        ma, mb = zz[:cut].max(), zz[cut:].max()
        sa, sb = np.exp(zz[:cut] - ma).sum(), np.exp(zz[cut:] - mb).sum()
        m = max(ma, mb)
        s = sa * math.exp(ma - m) + sb * math.exp(mb - m)
        assert m + math.log(s) - zz[123] == pytest.approx(loss[0], rel=1e-13)
    ref = mp.log(mp.fsum([mp.exp(mp.mpf(float(t))) for t in z[0]])) - mp.mpf(float(z[0, 123]))
    assert loss[0] == pytest.approx(float(ref), rel=1e-14)


def test_ce_bad_labels_and_bf16():
    z = f32(RNG.standard_normal((4, 10)))
    loss, mean, bad = kopref.ce_loss_rowwise(z, np.array([0, -1, 10, 9], dtype=np.int32))
    assert bad == 2 and np.isnan(loss[1]) and np.isnan(loss[2]) and np.isnan(mean)
    assert np.isfinite(loss[0]) and np.isfinite(loss[3])
    zb = to_bf16_bits(z)
    lb, _, _ = kopref.ce_loss_rowwise(zb, np.array([0, 1, 2, 3], dtype=np.int32))
    zw = torch.from_numpy(z).to(torch.bfloat16).to(torch.float64)
    ref = F.cross_entropy(zw, torch.tensor([0, 1, 2, 3]), reduction="none").numpy()
    assert np.max(np.abs(lb - ref)) <= 1e-14


# --------------------------------------------------------------------------- RMSNorm

def test_rmsnorm_closed_forms_and_library():
    H = 48
    one = f32(np.ones(H))
    eps = 1e-6
    x = f32(RNG.standard_normal((7, H)))
    y = kopref.rmsnorm(x, one, eps)
    ms = (x.astype(np.float64) ** 2).mean(axis=1)
    assert np.allclose((y ** 2).mean(axis=1), ms / (ms + eps), rtol=1e-13, atol=0)
    c = 3.0
    yc = kopref.rmsnorm(f32(np.full((1, H), c)), one, eps)
    assert np.allclose(yc, c / math.sqrt(c * c + eps), rtol=1e-15, atol=0)
    alt = f32([[1.0, -1.0] * (H // 2)])
    ya = kopref.rmsnorm(alt, one, eps)
    assert np.allclose(ya, alt.astype(np.float64) / math.sqrt(1 + eps), rtol=1e-15, atol=0)
    # f(a x) = sign(a) f(x) when eps = 0
    y0 = kopref.rmsnorm(x, one, 0.0)
    ym = kopref.rmsnorm(f32(x * np.float32(-4.0)), one, 0.0)
    assert np.allclose(ym, -y0, rtol=1e-14, atol=0)
    # weight is applied per column; library rms_norm in float64
    w = f32(1 + 0.02 * RNG.standard_normal(H))
    yw = kopref.rmsnorm(x, w, eps)
    ref = F.rms_norm(torch.from_numpy(x.astype(np.float64)), (H,),
                     torch.from_numpy(w.astype(np.float64)), eps).numpy()
    assert np.max(np.abs(yw - ref)) <= 1e-14
    # mpmath on one row
    row = x[0]
    msq = mp.fsum([mp.mpf(float(t)) ** 2 for t in row]) / H
    refm = [float(mp.mpf(float(row[j])) / mp.sqrt(msq + mp.mpf(eps)) * mp.mpf(float(w[j]))) for j in range(H)]
    assert np.max(np.abs(yw[0] - np.array(refm))) <= 1e-14


# --------------------------------------------------------------------------- SiLU * up, residual add

def test_silu_mul_identities_layout_library():
    inter = 6
    g = f32(RNG.standard_normal((3, inter)) * 3)
    u = f32(RNG.standard_normal((3, inter)))
    gu = np.concatenate([g, u], axis=1)                         # [gate | up] halves
    out = kopref.silu_mul(gu)
    ref = (F.silu(torch.from_numpy(g.astype(np.float64))) * torch.from_numpy(u.astype(np.float64))).numpy()
    assert np.max(np.abs(out - ref)) <= 1e-15
    # up = 1 -> silu(gate); silu(0) = 0; silu(g) - silu(-g) = g
    ones = f32(np.ones((3, inter)))
    s_pos = kopref.silu_mul(np.concatenate([g, ones], axis=1))
    s_neg = kopref.silu_mul(np.concatenate([-g, ones], axis=1))
    assert np.allclose(s_pos - s_neg, g.astype(np.float64), rtol=1e-14, atol=1e-15)
    assert kopref.silu_mul(f32([[0.0, 5.0]]))[0, 0] == 0.0
    # large gate -> gate * up
    big = kopref.silu_mul(f32([[40.0, 0.5]]))
    assert big[0, 0] == pytest.approx(20.0, rel=1e-15)
    # swapping the halves changes the answer (SiLU applies to the first half)
    assert np.max(np.abs(kopref.silu_mul(np.concatenate([u, g], axis=1)) - out)) > 1e-3
    for gv, uv in [(0.5, 2.0), (-3.0, 1.5), (7.25, -0.125)]:
        refm = mp.mpf(gv) / (1 + mp.exp(-mp.mpf(gv))) * mp.mpf(uv)
        assert kopref.silu_mul(f32([[gv, uv]]))[0, 0] == pytest.approx(float(refm), rel=1e-15)


def test_residual_add_exact():
    a = f32(RNG.standard_normal((5, 9)))
    b = f32(RNG.standard_normal((5, 9)))
    assert np.array_equal(kopref.residual_add(a, b), a.astype(np.float64) + b.astype(np.float64))
    ab, bb = to_bf16_bits(a), to_bf16_bits(b)
    wa = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    wb = torch.from_numpy(b).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(kopref.residual_add(ab, bb), wa + wb)


# --------------------------------------------------------------------------- GEMM helper and the chain

def test_gemm_nt_exact_cases():
    M, K, N = 4, 6, 5
    A = f32(RNG.integers(-5, 6, (M, K)))
    Wm = f32(RNG.integers(-5, 6, (N, K)))
    Cm = kopref.gemm_nt(A, Wm)
    assert np.array_equal(Cm, A.astype(np.float64) @ Wm.astype(np.float64).T)   # small ints: exact
    eye = f32(np.eye(K))
    assert np.array_equal(kopref.gemm_nt(A, eye), A.astype(np.float64))
    perm = f32(np.eye(K)[[2, 0, 1, 5, 4, 3]])           # row n of W selects column perm[n] of A
    assert np.array_equal(kopref.gemm_nt(A, perm), A.astype(np.float64)[:, [2, 0, 1, 5, 4, 3]])
    Ar = RNG.standard_normal((M, K))
    Wr = RNG.standard_normal((N, K))
    assert np.allclose(kopref.gemm_nt(Ar, Wr), Ar @ Wr.T, rtol=1e-14, atol=1e-14)


def test_mlp_chain_selector_weights_collapse_to_elementwise():
    # W1 = [I; I] (gate and up both copy the normed row), W2 = I:
    # out_j = h_j + silu(n_j) * n_j with n = rmsnorm(h).
    Hd = 16
    h = f32(RNG.standard_normal((5, Hd)))
    w = f32(1 + 0.02 * RNG.standard_normal(Hd))
    W1 = f32(np.concatenate([np.eye(Hd), np.eye(Hd)], axis=0))
    W2 = f32(np.eye(Hd))
    out = kopref.mlp_segment(h, w, W1, W2, 1e-6)
    hd = h.astype(np.float64)
    n = hd / np.sqrt((hd ** 2).mean(axis=1, keepdims=True) + 1e-6) * w.astype(np.float64)
    assert np.allclose(out, hd + n / (1 + np.exp(-n)) * n, rtol=1e-13, atol=1e-14)


def test_mlp_chain_reduced_shape_vs_numpy():
    M, Hd, I = 12, 32, 56
    h = to_bf16_bits(RNG.standard_normal((M, Hd)))
    w = f32(1 + 0.02 * RNG.standard_normal(Hd))
    W1 = to_bf16_bits(RNG.standard_normal((2 * I, Hd)) * 0.02)
    W2 = to_bf16_bits(RNG.standard_normal((Hd, I)) * 0.02)
    out = kopref.mlp_segment(h, w, W1, W2, 1e-6)

    def wide(bits):
        return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    hd, W1d, W2d = wide(h), wide(W1), wide(W2)
    n = hd / np.sqrt((hd ** 2).mean(axis=1, keepdims=True) + 1e-6) * w.astype(np.float64)
    gu = n @ W1d.T
    act = gu[:, :I] / (1 + np.exp(-gu[:, :I])) * gu[:, I:]
    ref = hd + act @ W2d.T
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-14)


# --------------------------------------------------------------------------- residual+LN, interleaved SwiGLU, CE options

def test_residual_layernorm_library_and_invariants():
    H = 72
    x = f32(RNG.standard_normal((8, H)) * 2 + 1)
    r = f32(RNG.standard_normal((8, H)))
    g = f32(1 + 0.1 * RNG.standard_normal(H))
    be = f32(0.1 * RNG.standard_normal(H))
    tx, tr, tg, tbe = (torch.from_numpy(a.astype(np.float64)) for a in (x, r, g, be))
    y, mu, rstd = kopref.residual_layernorm(x, r, g, be, 1e-5)
    assert np.max(np.abs(y - F.layer_norm(tx + tr, (H,), tg, tbe, 1e-5).numpy())) <= 1e-13
    assert np.allclose(mu, (tx + tr).mean(dim=1).numpy(), rtol=0, atol=1e-14)
    # no residual: plain LayerNorm; zero mean and sigma^2/(sigma^2+eps) variance before the affine step
    y0, mu0, rstd0 = kopref.residual_layernorm(x, None, f32(np.ones(H)), f32(np.zeros(H)), 1e-5)
    assert np.max(np.abs(y0 - F.layer_norm(tx, (H,), None, None, 1e-5).numpy())) <= 1e-13
    assert np.all(np.abs(y0.mean(axis=1)) <= 1e-12)
    var = x.astype(np.float64).var(axis=1)
    assert np.allclose(y0.var(axis=1), var / (var + 1e-5), rtol=1e-12, atol=0)
    # consistent with the full bias+GELU+residual oracle when the GELU term is switched off by x = 0, b = 0
    yf, _, _ = kopref.bias_gelu_residual_layernorm(f32(np.zeros((8, H))), r, f32(np.zeros(H)), g, be, 1e-5)
    yr, _, _ = kopref.residual_layernorm(r, None, g, be, 1e-5)
    assert np.array_equal(yf, yr)


def test_silu_mul_interleaved_is_a_column_permutation_of_the_split_layout():
    inter = 7
    g = f32(RNG.standard_normal((4, inter)) * 3)
    u = f32(RNG.standard_normal((4, inter)))
    inter_l = np.empty((4, 2 * inter), dtype=np.float32)
    inter_l[:, 0::2] = g
    inter_l[:, 1::2] = u
    assert np.array_equal(kopref.silu_mul_interleaved(inter_l), kopref.silu_mul(np.concatenate([g, u], axis=1)))
    ref = (F.silu(torch.from_numpy(g.astype(np.float64))) * torch.from_numpy(u.astype(np.float64))).numpy()
    assert np.max(np.abs(kopref.silu_mul_interleaved(inter_l) - ref)) <= 1e-15


def test_ce_options_against_library_and_base_oracle():
    M, V = 13, 101
    z = f32(RNG.standard_normal((M, V)) * 2)
    lab = RNG.integers(0, V, M).astype(np.int32)
    lab[[2, 7]] = -100
    tz, tl = torch.from_numpy(z.astype(np.float64)), torch.from_numpy(lab.astype(np.int64))
    for s in (0.0, 0.1, 0.35):
        loss, mean, bad, cnt = kopref.ce_loss_opts(z, lab, ignore_index=-100, smoothing=s)
        ref = F.cross_entropy(tz, tl, reduction="none", ignore_index=-100, label_smoothing=s).numpy()
        assert np.max(np.abs(loss - ref)) <= 1e-13
        assert mean == pytest.approx(float(F.cross_entropy(tz, tl, ignore_index=-100, label_smoothing=s)), rel=1e-13)
        assert bad == 0 and cnt == M - 2 and loss[2] == 0.0 and loss[7] == 0.0
    # no ignored rows and no smoothing: identical to the plain oracle
    lab2 = RNG.integers(0, V, M).astype(np.int32)
    a, ma, _, c = kopref.ce_loss_opts(z, lab2, ignore_index=-100, smoothing=0.0)
    b, mb, _ = kopref.ce_loss_rowwise(z, lab2)
    assert np.array_equal(a, b) and ma == mb and c == M
    # smoothing on a uniform row changes nothing (both terms equal ln V); all rows ignored -> NaN mean
    zu = f32(np.full((2, V), 0.5))
    lu, mu_, _, _ = kopref.ce_loss_opts(zu, np.array([3, 4], dtype=np.int32), smoothing=0.3)
    assert np.all(np.abs(lu - math.log(V)) <= 1e-13)
    _, mn, _, cn = kopref.ce_loss_opts(zu, np.array([-100, -100], dtype=np.int32))
    assert cn == 0 and math.isnan(mn)
    # an out-of-range label that is not ignore_index is bad, not ignored
    l3, m3, b3, c3 = kopref.ce_loss_opts(zu, np.array([V, 1], dtype=np.int32))
    assert b3 == 1 and c3 == 2 and math.isnan(l3[0]) and math.isnan(m3)


def test_ce_sum_reduction_against_library_and_closed_forms():
    M, V = 17, 53
    z = f32(RNG.standard_normal((M, V)) * 2)
    lab = RNG.integers(0, V, M).astype(np.int32)
    lab[[0, 9]] = -100
    tz, tl = torch.from_numpy(z.astype(np.float64)), torch.from_numpy(lab.astype(np.int64))
    for s in (0.0, 0.2):
        total = kopref.ce_loss_sum(z, lab, ignore_index=-100, smoothing=s)
        ref = float(F.cross_entropy(tz, tl, reduction="sum", ignore_index=-100, label_smoothing=s))
        assert total == pytest.approx(ref, rel=1e-13)
        # sum = mean * counted rows, and = the sum of the per-row output
        loss, mean, _, cnt = kopref.ce_loss_opts(z, lab, ignore_index=-100, smoothing=s)
        assert total == pytest.approx(mean * cnt, rel=1e-13)
        assert total == pytest.approx(math.fsum(loss), rel=1e-13)
    # another ignore_index: label 5 no longer counts, -100 becomes a bad label (NaN sum)
    lab5 = RNG.integers(0, V, M).astype(np.int32)
    lab5[3] = 5
    t5 = kopref.ce_loss_sum(z, lab5, ignore_index=5)
    keep = lab5 != 5
    ref5 = float(F.cross_entropy(tz[keep], torch.from_numpy(lab5[keep].astype(np.int64)), reduction="sum"))
    assert t5 == pytest.approx(ref5, rel=1e-13)
    assert math.isnan(kopref.ce_loss_sum(z, lab, ignore_index=5))
    # closed forms: n uniform rows sum to n ln V whatever the smoothing; nothing counted sums to 0, not NaN
    zu = f32(np.full((6, V), -0.25))
    assert kopref.ce_loss_sum(zu, np.arange(6, dtype=np.int32), smoothing=0.4) == pytest.approx(6 * math.log(V), rel=1e-14)
    assert kopref.ce_loss_sum(zu, np.full(6, -100, dtype=np.int32)) == 0.0
    # two-class rows: loss = log1p(exp(-(z_label - z_other)))
    z2 = f32(np.array([[1.5, -0.5], [0.25, 2.0]]))
    want = math.log1p(math.exp(-2.0)) + math.log1p(math.exp(1.75))
    assert kopref.ce_loss_sum(z2, np.array([0, 0], dtype=np.int32)) == pytest.approx(want, rel=1e-14)


def test_ce_non_finite_logits_follow_the_shifted_definition():
    # A NaN anywhere in a row, or a +inf logit (inf - inf in the max-shifted form), makes that row's loss NaN and
    # leaves the other rows alone; -inf logits are ordinary (exp gives 0). torch's cross_entropy in float64 agrees.
    V = 40
    z = f32(RNG.standard_normal((6, V)))
    z[1, 7] = np.nan
    z[2, :] = np.nan
    z[3, 0] = np.inf
    z[4, 5] = -np.inf
    lab = np.array([1, 2, 3, 4, 6, 39], dtype=np.int32)
    loss, mean, bad = kopref.ce_loss_rowwise(z, lab)
    ref = F.cross_entropy(torch.from_numpy(z.astype(np.float64)), torch.from_numpy(lab.astype(np.int64)),
                          reduction="none").numpy()
    assert np.array_equal(np.isnan(loss), [False, True, True, True, False, False])
    assert np.array_equal(np.isnan(loss), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.max(np.abs(loss[ok] - ref[ok])) <= 1e-13
    assert math.isnan(mean) and bad == 0


# --------------------------------------------------------------------------- GroupNorm / InstanceNorm + activation

def test_groupnorm_library_invariants_and_instance_norm():
    N, Cc, H, W, G = 3, 12, 5, 7, 4
    x = f32(RNG.standard_normal((N, Cc, H, W)) * 2 + 0.5)
    g = f32(1 + 0.1 * RNG.standard_normal(Cc))
    b = f32(0.1 * RNG.standard_normal(Cc))
    tx, tg, tb = (torch.from_numpy(a.astype(np.float64)) for a in (x, g, b))
    y, mu, rstd = kopref.groupnorm_act(x, g, b, G, 1e-5)
    assert np.max(np.abs(y - F.group_norm(tx, G, tg, tb, 1e-5).numpy())) <= 1e-13
    xs = x.astype(np.float64).reshape(N, G, -1)
    assert np.allclose(mu, xs.mean(axis=2), rtol=0, atol=1e-14)
    assert np.allclose(rstd, 1 / np.sqrt(xs.var(axis=2) + 1e-5), rtol=1e-13, atol=0)
    # no affine: every group has zero mean and variance var/(var+eps)
    y0, _, _ = kopref.groupnorm_act(x, None, None, G, 1e-5)
    ys = y0.reshape(N, G, -1)
    assert np.all(np.abs(ys.mean(axis=2)) <= 1e-12)
    assert np.allclose(ys.var(axis=2), xs.var(axis=2) / (xs.var(axis=2) + 1e-5), rtol=1e-12, atol=0)
    # groups == C is InstanceNorm; groups == 1 normalises the whole image (LayerNorm over C,H,W)
    yi, _, _ = kopref.groupnorm_act(x, None, None, Cc, 1e-5)
    assert np.max(np.abs(yi - F.instance_norm(tx, eps=1e-5).numpy())) <= 1e-13
    y1, _, _ = kopref.groupnorm_act(x, None, None, 1, 1e-5)
    assert np.max(np.abs(y1 - F.layer_norm(tx, (Cc, H, W), eps=1e-5).numpy())) <= 1e-13
    # the affine step indexes the channel, not the group (a group-indexed gamma fails this)
    gsel = f32(np.arange(1, Cc + 1))
    ysel, _, _ = kopref.groupnorm_act(x, gsel, None, G, 1e-5)
    assert np.allclose(ysel, y0 * gsel.astype(np.float64)[None, :, None, None], rtol=1e-14, atol=1e-14)
    # activations act on the normalised, affine-transformed value
    yr, _, _ = kopref.groupnorm_act(x, g, b, G, 1e-5, act=1)
    ysl, _, _ = kopref.groupnorm_act(x, g, b, G, 1e-5, act=2)
    assert np.array_equal(yr, np.maximum(y, 0.0))
    assert np.max(np.abs(ysl - F.silu(torch.from_numpy(y)).numpy())) <= 1e-14
    # bf16 input widened exactly; constant group -> zeros (var 0, rstd = 1/sqrt(eps))
    xb = to_bf16_bits(x)
    yb, _, _ = kopref.groupnorm_act(xb, g, b, G, 1e-5)
    txb = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64)
    assert np.max(np.abs(yb - F.group_norm(txb, G, tg, tb, 1e-5).numpy())) <= 1e-13
    yc, muc, rc = kopref.groupnorm_act(f32(np.full((1, 4, 2, 2), 3.0)), None, None, 2, 1e-5)
    assert np.all(yc == 0.0) and np.all(muc == 3.0) and np.allclose(rc, 1 / math.sqrt(1e-5), rtol=1e-15)


# --------------------------------------------------------------------------- row scale, mat-vec + bias sum

def test_row_scale_is_diag_times_matrix():
    n = 7
    a = f32(RNG.standard_normal(n))
    B = f32(RNG.standard_normal((n, 5)))
    out = kopref.row_scale(a, B)
    # the O(N^3) form the case study starts from: diag(a) @ B, in float64
    assert np.array_equal(out, np.diag(a.astype(np.float64)) @ B.astype(np.float64))
    assert np.array_equal(kopref.row_scale(f32(np.ones(n)), B), B.astype(np.float64))
    ai = f32(RNG.integers(-4, 5, n))
    Bi = f32(RNG.integers(-4, 5, (n, 5)))
    assert np.array_equal(kopref.row_scale(ai, Bi), ai[:, None].astype(np.float64) * Bi)      # exact on integers
    ab, Bb = to_bf16_bits(a), to_bf16_bits(B)
    wa = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    wB = torch.from_numpy(B).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(kopref.row_scale(ab, Bb), wa[:, None] * wB)


def test_matvec_bias_equals_linear_then_sum_and_later_reductions_are_identities():
    # sum_j (sum_k X_ik W_jk + b_j) = sum_k X_ik (sum_j W_jk) + sum_j b_j
    M, K, N = 9, 13, 6
    X = f32(RNG.standard_normal((M, K)))
    Wm = f32(RNG.standard_normal((N, K)))
    b = f32(RNG.standard_normal(N))
    w_colsum = f32(Wm.astype(np.float64).sum(axis=0))           # rounded to fp32 as the caller would pass it
    b_sum = float(b.astype(np.float64).sum())
    out = kopref.matvec_bias(X, w_colsum, b_sum)
    lin = kopref.gemm_nt(X, Wm) + b.astype(np.float64)[None, :]
    assert np.allclose(out, lin.sum(axis=1), rtol=0, atol=1e-5)      # fp32 rounding of the column sums only
    exact = X.astype(np.float64) @ w_colsum.astype(np.float64) + b_sum
    assert np.allclose(out, exact, rtol=1e-14, atol=1e-14)
    # max, mean and logsumexp over a singleton dimension return the element itself
    col = out[:, None]
    assert np.array_equal(col.max(axis=1), out) and np.array_equal(col.mean(axis=1), out)
    assert np.allclose(scipy.special.logsumexp(col, axis=1), out, rtol=1e-15, atol=1e-15)
    # integer case is exact; a transposed weight would fail it
    Xi = f32(RNG.integers(-3, 4, (4, 5)))
    wi = f32([1, -2, 3, 0, 5])
    assert np.array_equal(kopref.matvec_bias(Xi, wi, 2.0), Xi.astype(np.float64) @ wi.astype(np.float64) + 2.0)


def test_threads_do_not_change_results():
    x = f32(RNG.standard_normal((64, 100)))
    b = f32(RNG.standard_normal(100))
    assert np.array_equal(kopref.softmax_scale_bias(x, b, 0.125, threads=1),
                          kopref.softmax_scale_bias(x, b, 0.125, threads=4))
    lab = RNG.integers(0, 100, 64).astype(np.int32)
    l1, m1, _ = kopref.ce_loss_rowwise(x, lab, threads=1)
    l4, m4, _ = kopref.ce_loss_rowwise(x, lab, threads=4)
    assert np.array_equal(l1, l4) and m1 == m4


# --------------------------------------------------------------------------- row-wise cumulative sums

def test_cumsum_closed_forms_library_and_identities():
    # closed forms: integers are exact in float64
    n = 257
    ones = np.ones((2, n), dtype=np.float32)
    k = np.arange(1, n + 1, dtype=np.float64)
    assert np.array_equal(kopref.cumsum_rows(ones)[0], k)                          # 1, 2, ..., n
    assert np.array_equal(kopref.cumsum_rows(ones, exclusive=True)[1], k - 1)      # 0, 1, ..., n-1
    assert np.array_equal(kopref.cumsum_rows(ones, reverse=True)[0], k[::-1])      # n, ..., 1
    assert np.array_equal(kopref.cumsum_rows(ones, exclusive=True, reverse=True)[0], k[::-1] - 1)
    ramp = np.tile(np.arange(1, n + 1, dtype=np.float32), (3, 1))
    assert np.array_equal(kopref.cumsum_rows(ramp)[2], k * (k + 1) / 2)            # triangular numbers
    alt = np.tile(np.where(np.arange(n) % 2 == 0, 1.0, -1.0).astype(np.float32), (1, 1))
    assert np.array_equal(kopref.cumsum_rows(alt)[0], (np.arange(n) % 2 == 0).astype(np.float64))
    geo = np.tile((0.5 ** np.arange(40)).astype(np.float32), (1, 1))              # exact powers of two
    assert np.array_equal(kopref.cumsum_rows(geo)[0], 2.0 - 0.5 ** np.arange(40))
    # library routine in float64 on random data, every variant, fp32 and bf16 inputs
    x = f32(RNG.normal(0, 1, (7, 301)))
    m = RNG.random((7, 301)) < 0.6
    xd = x.astype(np.float64)
    inc = np.cumsum(xd, axis=1)
    np.testing.assert_allclose(kopref.cumsum_rows(x), inc, rtol=0, atol=1e-12)
    np.testing.assert_allclose(kopref.cumsum_rows(x, exclusive=True), inc - xd, rtol=0, atol=1e-12)
    rev = np.cumsum(xd[:, ::-1], axis=1)[:, ::-1]
    np.testing.assert_allclose(kopref.cumsum_rows(x, reverse=True), rev, rtol=0, atol=1e-12)
    np.testing.assert_allclose(kopref.cumsum_rows(x, exclusive=True, reverse=True), rev - xd, rtol=0, atol=1e-12)
    np.testing.assert_allclose(kopref.cumsum_rows(x, mask=m), np.cumsum(xd * m, axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(kopref.cumsum_rows(x, mask=m, reverse=True),
                               np.cumsum((xd * m)[:, ::-1], axis=1)[:, ::-1], rtol=0, atol=1e-12)
    tb = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_allclose(kopref.cumsum_rows(tb), torch.cumsum(tb.to(torch.float64), dim=1).numpy(),
                               rtol=0, atol=1e-12)
    # identities: inclusive forward + exclusive reverse = row total; the last column is the row sum;
    # an all-ones mask changes nothing, an all-zero mask gives zeros; differences recover the input
    total = xd.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(kopref.cumsum_rows(x) + kopref.cumsum_rows(x, exclusive=True, reverse=True),
                               np.broadcast_to(total, x.shape), rtol=0, atol=1e-11)
    np.testing.assert_allclose(kopref.cumsum_rows(x)[:, -1], math_fsum_rows(xd), rtol=0, atol=1e-12)
    assert np.array_equal(kopref.cumsum_rows(x, mask=np.ones_like(m)), kopref.cumsum_rows(x))
    assert np.array_equal(kopref.cumsum_rows(x, mask=np.zeros_like(m)), np.zeros_like(xd))
    np.testing.assert_allclose(np.diff(kopref.cumsum_rows(x), axis=1), xd[:, 1:], rtol=0, atol=1e-12)
    # one column: inclusive is x, exclusive is 0
    c1 = f32(RNG.normal(0, 1, (5, 1)))
    assert np.array_equal(kopref.cumsum_rows(c1), c1.astype(np.float64))
    assert np.array_equal(kopref.cumsum_rows(c1, exclusive=True), np.zeros((5, 1)))
    # threads do not change the result
    assert np.array_equal(kopref.cumsum_rows(x, mask=m, threads=4), kopref.cumsum_rows(x, mask=m, threads=1))


def math_fsum_rows(a):
    return np.array([math.fsum(r) for r in a])


def test_bn_oracle_is_layout_agnostic():
    """The oracle is defined over (n, c, h, w) indices: a channels-last tensor gives the same values, and
    both agree with torch in float64 evaluated directly on the NHWC-permuted data."""
    x = torch.from_numpy(f32(RNG.normal(0, 1, (3, 6, 5, 4))))
    scale = torch.from_numpy(f32(RNG.uniform(0.5, 1.5, 6)))
    shift = torch.from_numpy(f32(RNG.normal(0, 0.1, 6)))
    y0, p0 = kopref.bn_relu_avgpool(x, scale, shift)
    y1, p1 = kopref.bn_relu_avgpool(x.contiguous(memory_format=torch.channels_last), scale, shift)
    assert np.array_equal(y0, y1) and np.array_equal(p0, p1)
    nhwc = x.permute(0, 2, 3, 1).to(torch.float64)                       # [n, h, w, c]
    a = torch.relu(nhwc * scale.to(torch.float64) + shift.to(torch.float64))
    np.testing.assert_allclose(y0, a.permute(0, 3, 1, 2).numpy(), rtol=0, atol=1e-15)
    np.testing.assert_allclose(p0, a.mean(dim=(1, 2)).numpy(), rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- affine + ReLU + windowed pooling

def test_pool2d_library_closed_forms_and_special_cases():
    x = torch.from_numpy(f32(RNG.normal(0, 1, (2, 3, 11, 13))))
    scale = torch.from_numpy(f32(RNG.uniform(0.5, 1.5, 3)))
    shift = torch.from_numpy(f32(RNG.normal(0, 0.3, 3)))
    xd = x.to(torch.float64)
    a = torch.relu(xd * scale.to(torch.float64)[None, :, None, None] + shift.to(torch.float64)[None, :, None, None])
    for k, s, p in [((3, 3), (2, 2), (1, 1)), ((2, 2), (2, 2), (0, 0)), ((3, 2), (1, 3), (1, 0)), ((5, 5), (1, 1), (2, 2)),
                    ((1, 1), (1, 1), (0, 0)), ((11, 13), (1, 1), (0, 0))]:
        # library routines in float64 (torch pads max pooling with -inf and averages with padding counted)
        np.testing.assert_allclose(kopref.affine_relu_pool2d(x, scale, shift, k, s, p, "max", True),
                                   F.max_pool2d(a, k, s, p).numpy(), rtol=0, atol=1e-15)
        np.testing.assert_allclose(kopref.affine_relu_pool2d(x, scale, shift, k, s, p, "avg", True),
                                   F.avg_pool2d(a, k, s, p, count_include_pad=True).numpy(), rtol=0, atol=1e-14)
        # no affine, no ReLU: plain pooling of x
        np.testing.assert_allclose(kopref.affine_relu_pool2d(x, None, None, k, s, p, "max", False),
                                   F.max_pool2d(xd, k, s, p).numpy(), rtol=0, atol=0)
        np.testing.assert_allclose(kopref.affine_relu_pool2d(x, None, None, k, s, p, "avg", False),
                                   F.avg_pool2d(xd, k, s, p, count_include_pad=True).numpy(), rtol=0, atol=1e-14)
    # special cases: a 1x1 window is the activation itself; a window covering the image is the global pool
    one = kopref.affine_relu_pool2d(x, scale, shift, (1, 1), (1, 1), (0, 0), "max", True)
    np.testing.assert_allclose(one, a.numpy(), rtol=0, atol=1e-15)
    _, pooled = kopref.bn_relu_avgpool(x, scale, shift)
    full = kopref.affine_relu_pool2d(x, scale, shift, (11, 13), (1, 1), (0, 0), "avg", True)
    np.testing.assert_allclose(full[:, :, 0, 0], pooled, rtol=0, atol=1e-14)
    # closed forms: a ramp along w, 2x2 windows of stride 2: max picks the right column, avg the midpoint
    ramp = torch.arange(16, dtype=torch.float32).repeat(1, 1, 4, 1)                  # [1,1,4,16], value = column
    assert np.array_equal(kopref.affine_relu_pool2d(ramp, None, None, (2, 2), (2, 2), (0, 0), "max", False)[0, 0, 0],
                          np.arange(1, 16, 2, dtype=np.float64))
    assert np.array_equal(kopref.affine_relu_pool2d(ramp, None, None, (2, 2), (2, 2), (0, 0), "avg", False)[0, 0, 1],
                          np.arange(0.5, 16, 2))
    # padding never wins a max (all-negative input keeps its own maximum) and counts as zeros in an average
    neg = torch.full((1, 1, 4, 4), -3.0)
    assert np.array_equal(kopref.affine_relu_pool2d(neg, None, None, (3, 3), (2, 2), (1, 1), "max", False),
                          np.full((1, 1, 2, 2), -3.0))
    corner = kopref.affine_relu_pool2d(torch.ones((1, 1, 4, 4)), None, None, (3, 3), (2, 2), (1, 1), "avg", False)
    assert corner[0, 0, 0, 0] == 4.0 / 9.0 and corner[0, 0, 1, 1] == 1.0
    # NaN: poisons exactly the windows that contain it
    xn = x.clone()
    xn[0, 1, 4, 6] = float("nan")
    ym = kopref.affine_relu_pool2d(xn, scale, shift, (3, 3), (2, 2), (1, 1), "max", True)
    assert {tuple(t) for t in np.argwhere(np.isnan(ym))} == {(0, 1, 2, 3)}      # rows 3..5, columns 5..7
    ref_nan = torch.isnan(F.max_pool2d(torch.relu(xn.double() * scale.double()[None, :, None, None]
                                                  + shift.double()[None, :, None, None]), 3, 2, 1)).numpy()
    assert np.array_equal(np.isnan(ym), ref_nan)
    # bf16 input and threads
    xb = x.to(torch.bfloat16)
    np.testing.assert_allclose(kopref.affine_relu_pool2d(xb, None, None, (3, 3), (2, 2), (1, 1), "max", False, threads=3),
                               F.max_pool2d(xb.double(), 3, 2, 1).numpy(), rtol=0, atol=0)


# --------------------------------------------------------------------------- fp16 inputs

def test_f16_widening_exhaustive_and_one_function_end_to_end():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    wide = kopref.f16_to_f64(bits)
    via_numpy = bits.view(np.float16).astype(np.float64)              # an independent implementation
    finite = np.isfinite(via_numpy)
    assert np.array_equal(wide[finite], via_numpy[finite])
    assert np.array_equal(np.isnan(wide), np.isnan(via_numpy)) and np.array_equal(np.isinf(wide), np.isinf(via_numpy))
    assert np.array_equal(np.signbit(wide[~np.isnan(wide)]), np.signbit(via_numpy[~np.isnan(via_numpy)]))
    # through a whole oracle function: fp16 tensors are widened exactly, so the result equals the one on
    # the same values given as float64
    x = torch.from_numpy(f32(RNG.normal(0, 1, (5, 37)))).to(torch.float16)
    b = torch.from_numpy(f32(RNG.normal(0, 0.1, 37)))
    assert np.array_equal(kopref.softmax_scale_bias(x, b, 0.3), kopref.softmax_scale_bias(x.to(torch.float64), b, 0.3))
    assert np.array_equal(kopref.softmax_scale_bias(x.numpy(), b, 0.3), kopref.softmax_scale_bias(x, b, 0.3))
    h = torch.from_numpy(f32(RNG.normal(0, 1, (4, 16)))).to(torch.float16)
    w = torch.from_numpy(f32(RNG.normal(1, 0.02, 16)))
    W1 = torch.from_numpy(f32(RNG.normal(0, 0.1, (24, 16)))).to(torch.float16)
    W2 = torch.from_numpy(f32(RNG.normal(0, 0.1, (16, 12)))).to(torch.float16)
    np.testing.assert_allclose(kopref.mlp_segment(h, w, W1, W2, 1e-6),
                               kopref.mlp_segment(h.double(), w, W1.double(), W2.double(), 1e-6), rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- error-function GELU

def test_gelu_erf_and_the_erf_form_of_the_layernorm_segment():
    # the scalar against 50-digit arithmetic, a library routine and its closed-form points
    for u in [-8.0, -3.0, -1.0, -0.3, 0.0, 1e-8, 0.5, 1.0, 2.5, 6.0, 12.0]:
        exact = float(mp.mpf(u) / 2 * (1 + mp.erf(mp.mpf(u) / mp.sqrt(2))))
        assert kopref.gelu_erf(u) == pytest.approx(exact, rel=1e-14, abs=1e-15)      # 1 + erf cancels for u << 0
        assert kopref.gelu_erf(u) == pytest.approx(0.5 * u * (1.0 + scipy.special.erf(u / math.sqrt(2.0))), rel=1e-14, abs=1e-15)
    assert kopref.gelu_erf(0.0) == 0.0
    assert kopref.gelu_erf(40.0) == 40.0 and kopref.gelu_erf(-40.0) == 0.0          # saturation
    # gelu(u) - gelu(-u) = u for every u (erf is odd)
    for u in [0.1, 0.7, 3.3]:
        assert kopref.gelu_erf(u) - kopref.gelu_erf(-u) == pytest.approx(u, rel=1e-15)
    # it differs from the tanh form where that approximation is off (about 1e-4 around |u| = 2)
    assert 5e-5 < abs(kopref.gelu_erf(2.0) - kopref.gelu_tanh(2.0)) < 5e-4
    # the whole segment against torch in float64 (gelu approximate='none' is the erf form)
    x = torch.from_numpy(f32(RNG.normal(0, 1, (6, 48))))
    r = torch.from_numpy(f32(RNG.normal(0, 1, (6, 48))))
    b = torch.from_numpy(f32(RNG.normal(0, 0.1, 48)))
    g = torch.from_numpy(f32(RNG.normal(1, 0.02, 48)))
    be = torch.from_numpy(f32(RNG.normal(0, 0.02, 48)))
    y, mu, rs = kopref.bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5, erf_form=True)
    v = r.double() + F.gelu(x.double() + b.double(), approximate="none")
    ref = F.layer_norm(v, (48,), g.double(), be.double(), 1e-5)
    np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(mu, v.mean(dim=1).numpy(), rtol=0, atol=1e-14)
    np.testing.assert_allclose(rs, 1.0 / torch.sqrt(v.var(dim=1, unbiased=False) + 1e-5).numpy(), rtol=1e-13)
    # and the tanh form is untouched by the refactoring
    y0, _, _ = kopref.bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
    v0 = r.double() + F.gelu(x.double() + b.double(), approximate="tanh")
    np.testing.assert_allclose(y0, F.layer_norm(v0, (48,), g.double(), be.double(), 1e-5).numpy(), rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- row reductions

def test_reduce_rows_library_closed_forms_and_specials():
    x = f32(RNG.normal(0, 2, (9, 203)))
    xd = x.astype(np.float64)
    np.testing.assert_allclose(kopref.reduce_rows(x, "sum")[0], [math.fsum(r) for r in xd], rtol=0, atol=1e-11)
    np.testing.assert_allclose(kopref.reduce_rows(x, "mean")[0], [math.fsum(r) / 203 for r in xd], rtol=0, atol=1e-13)
    v, i = kopref.reduce_rows(x, "max")
    assert np.array_equal(v, xd.max(axis=1)) and np.array_equal(i, xd.argmax(axis=1))
    v, i = kopref.reduce_rows(x, "min")
    assert np.array_equal(v, xd.min(axis=1)) and np.array_equal(i, xd.argmin(axis=1))
    np.testing.assert_allclose(kopref.reduce_rows(x, "logsumexp")[0], scipy.special.logsumexp(xd, axis=1), rtol=1e-14)
    np.testing.assert_allclose(kopref.reduce_rows(x, "logsumexp")[0],
                               torch.logsumexp(torch.from_numpy(xd), dim=1).numpy(), rtol=1e-14)
    # closed forms
    n = 1000
    ramp = np.tile(np.arange(1, n + 1, dtype=np.float32), (2, 1))
    assert kopref.reduce_rows(ramp, "sum")[0][0] == n * (n + 1) / 2 and kopref.reduce_rows(ramp, "mean")[0][1] == (n + 1) / 2
    const = np.full((1, n), 0.75, dtype=np.float32)
    assert kopref.reduce_rows(const, "logsumexp")[0][0] == pytest.approx(0.75 + math.log(n), rel=1e-15)
    # ties: the first position wins; the logsumexp of huge values does not overflow
    ties = np.array([[1, 5, 5, 2, 5], [3, 0, 0, 3, 3]], dtype=np.float32)
    assert list(kopref.reduce_rows(ties, "max")[1]) == [1, 0] and list(kopref.reduce_rows(ties, "min")[1]) == [0, 1]
    big = np.array([[1e30, 1e30]], dtype=np.float32)
    assert kopref.reduce_rows(big, "logsumexp")[0][0] == pytest.approx(float(np.float32(1e30)) + math.log(2.0), rel=1e-15)
    # NaN and infinities
    xn = x.copy()
    xn[3, 17] = np.nan
    xn[3, 90] = np.nan
    for op in ("sum", "mean", "max", "min", "logsumexp"):
        v, i = kopref.reduce_rows(xn, op)
        assert np.isnan(v[3]) and not np.isnan(np.delete(v, 3)).any()
        if i is not None:
            assert i[3] == 17
    assert int(torch.from_numpy(xn[3]).argmax()) == 17                  # torch ranks NaN the same way
    ninf = np.full((1, 8), -np.inf, dtype=np.float32)
    assert kopref.reduce_rows(ninf, "logsumexp")[0][0] == -np.inf and kopref.reduce_rows(ninf, "max")[1][0] == 0
    pinf = np.array([[0.0, np.inf, 1.0]], dtype=np.float32)
    assert kopref.reduce_rows(pinf, "logsumexp")[0][0] == np.inf and kopref.reduce_rows(pinf, "max")[1][0] == 1
    # bf16 / fp16 inputs and threads
    tb = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(kopref.reduce_rows(tb, "max", threads=3)[0], tb.double().max(dim=1).values.numpy())
    th = torch.from_numpy(x).to(torch.float16)
    np.testing.assert_allclose(kopref.reduce_rows(th, "sum")[0], th.double().sum(dim=1).numpy(), rtol=0, atol=1e-11)


# --------------------------------------------------------------------------- bias + activation epilogue

def test_bias_act_against_torch_mpmath_and_identities():
    x = torch.from_numpy(f32(RNG.normal(0, 2.5, (6, 41))))
    b = torch.from_numpy(f32(RNG.normal(0, 0.5, 41)))
    u = x.double() + b.double()
    lib_ref = {
        "identity": u, "relu": torch.relu(u), "leaky_relu": F.leaky_relu(u, 0.2), "gelu_tanh": F.gelu(u, approximate="tanh"),
        "gelu_erf": F.gelu(u, approximate="none"), "silu": F.silu(u), "sigmoid": torch.sigmoid(u), "tanh": torch.tanh(u),
        "mish": F.mish(u), "hardswish": F.hardswish(u), "elu": F.elu(u, 0.2),
    }
    for act, ref in lib_ref.items():
        np.testing.assert_allclose(kopref.bias_act(x, b, act, alpha=0.2), ref.numpy(), rtol=1e-13, atol=1e-14, err_msg=act)
        # without bias it is the activation of x itself
        np.testing.assert_allclose(kopref.bias_act(x, None, act, alpha=0.2),
                                   kopref.bias_act(x.double(), torch.zeros(41), act, alpha=0.2), rtol=0, atol=0, err_msg=act)
    # 50-digit values of the transcendental ones
    for v in [-20.0, -3.0, -0.5, 0.0, 0.7, 4.0, 25.0, 60.0]:
        m = mp.mpf(v)
        assert kopref.act_value(v, "silu") == pytest.approx(float(m / (1 + mp.exp(-m))), rel=1e-14, abs=1e-300)
        assert kopref.act_value(v, "sigmoid") == pytest.approx(float(1 / (1 + mp.exp(-m))), rel=1e-14)
        assert kopref.act_value(v, "mish") == pytest.approx(float(m * mp.tanh(mp.log(1 + mp.exp(m)))), rel=1e-13, abs=1e-300)
        assert kopref.act_value(v, "elu", 1.5) == pytest.approx(float(m if v > 0 else 1.5 * mp.expm1(m)), rel=1e-14)
    # identities and closed-form points
    for v in [0.3, 1.7, 9.0]:
        assert kopref.act_value(v, "sigmoid") + kopref.act_value(-v, "sigmoid") == pytest.approx(1.0, rel=1e-15)
        assert kopref.act_value(v, "silu") - kopref.act_value(-v, "silu") == pytest.approx(v, rel=1e-14)
        assert kopref.act_value(v, "tanh") == -kopref.act_value(-v, "tanh")
    assert kopref.act_value(-3.0, "hardswish") == 0.0 and kopref.act_value(3.0, "hardswish") == 3.0
    assert kopref.act_value(1.0, "hardswish") == pytest.approx(4.0 / 6.0, rel=1e-15)
    assert kopref.act_value(-2.0, "leaky_relu", 0.25) == -0.5 and kopref.act_value(2.0, "leaky_relu", 0.25) == 2.0
    assert kopref.act_value(0.0, "sigmoid") == 0.5 and kopref.act_value(0.0, "mish") == 0.0
    assert math.isnan(kopref.act_value(float("nan"), "relu")) and kopref.act_value(-1.0, "relu") == 0.0
    # bf16 / fp16 inputs are widened exactly
    xb = x.to(torch.bfloat16)
    np.testing.assert_allclose(kopref.bias_act(xb, b, "mish"), F.mish(xb.double() + b.double()).numpy(), rtol=1e-13, atol=1e-14)


# --------------------------------------------------------------------------- softmax variants

def test_softmax_opts_log_and_causal():
    x = torch.from_numpy(f32(RNG.normal(0, 2, (12, 37))))
    b = torch.from_numpy(f32(RNG.normal(0, 0.5, 37)))
    z = x.double() * 0.7 + b.double()
    # without options it is the plain oracle; the log form is its logarithm and torch's log_softmax
    assert np.array_equal(kopref.softmax_opts(x, b, 0.7), kopref.softmax_scale_bias(x, b, 0.7))
    np.testing.assert_allclose(kopref.softmax_opts(x, b, 0.7, log_output=True), F.log_softmax(z, dim=1).numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(np.exp(kopref.softmax_opts(x, b, 0.7, log_output=True)), kopref.softmax_scale_bias(x, b, 0.7),
                               rtol=1e-13)
    # log-softmax of a constant row of n entries is -ln n; it survives huge logits
    const = torch.full((2, 50), 3.0)
    np.testing.assert_allclose(kopref.softmax_opts(const, None, 1.0, log_output=True), np.full((2, 50), -math.log(50)), rtol=1e-15)
    big = torch.tensor([[1000.0, 999.0]])
    np.testing.assert_allclose(kopref.softmax_opts(big, None, 1.0, log_output=True)[0],
                               [-math.log1p(math.exp(-1.0)), -1.0 - math.log1p(math.exp(-1.0))], rtol=1e-14)
    # causal, square (period == cols): equals torch softmax over the masked scores, row by row within each block
    S = 9
    sc = torch.from_numpy(f32(RNG.normal(0, 1, (3 * S, S))))
    mask = torch.tril(torch.ones(S, S, dtype=torch.bool)).repeat(3, 1)
    zm = (sc.double() * 0.5).masked_fill(~mask, float("-inf"))
    np.testing.assert_allclose(kopref.softmax_opts(sc, None, 0.5, causal_period=S), torch.softmax(zm, dim=1).numpy(), rtol=0, atol=1e-15)
    got = kopref.softmax_opts(sc, None, 0.5, log_output=True, causal_period=S)
    ref = F.log_softmax(zm, dim=1).numpy()
    assert np.array_equal(np.isneginf(got), np.isneginf(ref)) and np.array_equal(np.isneginf(got), ~mask.numpy())
    np.testing.assert_allclose(got[mask.numpy()], ref[mask.numpy()], rtol=0, atol=1e-13)
    # first row of every block sees one column: probability 1 there; the last row sees all: the plain softmax
    p = kopref.softmax_opts(sc, None, 0.5, causal_period=S)
    assert np.array_equal(p[0::S, 0], np.ones(3)) and np.array_equal(p[0, 1:], np.zeros(S - 1))
    np.testing.assert_allclose(p[S - 1::S], kopref.softmax_scale_bias(sc[S - 1::S], None, 0.5), rtol=0, atol=0)
    # a period shorter than the row leaves a prefix visible to every row (4 queries over 9 keys: 5 + r + 1 visible)
    q = kopref.softmax_opts(sc[:8], None, 1.0, causal_period=4)
    for r in range(8):
        vis = 5 + (r % 4) + 1
        assert np.all(q[r, vis:] == 0) and q[r, :vis].sum() == pytest.approx(1.0, rel=1e-14) and np.all(q[r, :vis] > 0)


# --------------------------------------------------------------------------- pointwise epilogue chain

def test_epilogue_chain_composition_and_special_cases():
    x = torch.from_numpy(f32(RNG.normal(0, 2, (5, 33))))
    r = torch.from_numpy(f32(RNG.normal(0, 2, (5, 33))))
    b = torch.from_numpy(f32(RNG.normal(0, 0.5, 33)))
    u = (x.double() + b.double()) * 0.7 + r.double() * 1.5
    # the composition written with library operations in float64
    np.testing.assert_allclose(kopref.epilogue_chain(x, b, r, 0.7, 1.5, -1.0, 2.0, "gelu_tanh"),
                               F.gelu(torch.clamp(u, -1.0, 2.0), approximate="tanh").numpy(), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(kopref.epilogue_chain(x, b, r, 0.7, 1.5, act="mish"), F.mish(u).numpy(), rtol=1e-13, atol=1e-14)
    # special cases reduce to the other oracles: no residual, unit scale, no clamp = bias_act; x + r = residual_add
    assert np.array_equal(kopref.epilogue_chain(x, b, None, act="silu"), kopref.bias_act(x, b, "silu"))
    assert np.array_equal(kopref.epilogue_chain(x, None, r), kopref.residual_add(x, r))
    # hardtanh is the clamp alone; relu6 is clamp(0, 6)
    np.testing.assert_allclose(kopref.epilogue_chain(x, None, None, 3.0, lo=-1.0, hi=1.0), F.hardtanh(x.double() * 3.0).numpy(),
                               rtol=0, atol=0)
    np.testing.assert_allclose(kopref.epilogue_chain(x, None, None, 3.0, lo=0.0, hi=6.0), F.relu6(x.double() * 3.0).numpy(),
                               rtol=0, atol=0)
    # the order matters: the bias is added before the scale, the clamp comes before the activation
    one = torch.tensor([[2.0]])
    assert kopref.epilogue_chain(one, torch.tensor([1.0]), None, 10.0)[0, 0] == 30.0
    assert kopref.epilogue_chain(one, None, None, 1.0, lo=-1.0, hi=1.0, act="sigmoid")[0, 0] == pytest.approx(1 / (1 + math.exp(-1.0)))
    # NaN passes through the clamp
    assert math.isnan(kopref.epilogue_chain(torch.tensor([[float("nan")]]), None, None, lo=0.0, hi=1.0)[0, 0])


# --------------------------------------------------------------------------- residual + RMSNorm

def test_residual_rmsnorm_composition_against_torch():
    x = torch.from_numpy(f32(RNG.normal(0, 1, (6, 40))))
    r = torch.from_numpy(f32(RNG.normal(0, 1, (6, 40))))
    w = torch.from_numpy(f32(RNG.normal(1, 0.02, 40)))
    h, y = kopref.residual_rmsnorm(x, r, w, 1e-6)
    v = x.double() + r.double()
    assert np.array_equal(h, v.numpy())
    np.testing.assert_allclose(y, F.rms_norm(v, (40,), w.double(), 1e-6).numpy(), rtol=1e-14, atol=1e-15)
    # the norm sees the unrounded sum: with bf16 inputs it differs from rounding h first
    xb, rb = x.to(torch.bfloat16), r.to(torch.bfloat16)
    hb, yb = kopref.residual_rmsnorm(xb, rb, w, 1e-6)
    assert np.array_equal(hb, (xb.double() + rb.double()).numpy())
    rounded_first = kopref.rmsnorm((xb.float() + rb.float()).to(torch.bfloat16), w, 1e-6)
    assert np.abs(yb - rounded_first).max() > 1e-4
    # zero residual: plain RMSNorm
    assert np.array_equal(kopref.residual_rmsnorm(x, torch.zeros_like(x), w, 1e-6)[1], kopref.rmsnorm(x, w, 1e-6))


# --------------------------------------------------------------------------- LSTM cell (pointwise part)

def test_lstm_cell_against_torch_lstmcell_and_closed_forms():
    B, I, H = 5, 7, 6
    cell = torch.nn.LSTMCell(I, H).double()
    xin = torch.from_numpy(RNG.normal(0, 1, (B, I)))
    h0 = torch.from_numpy(RNG.normal(0, 1, (B, H)))
    c0 = torch.from_numpy(RNG.normal(0, 1, (B, H)))
    with torch.no_grad():
        h1, c1 = cell(xin, (h0, c0))                                   # the library routine fixes the gate order i, f, g, o
        ig = xin @ cell.weight_ih.t()                                  # the two preserved GEMMs
        hg = h0 @ cell.weight_hh.t()
        bias = (cell.bias_ih + cell.bias_hh).float()
    h, c = kopref.lstm_cell(ig, c0, gates2=hg, bias=bias)
    b64 = bias.double()
    href, cref = kopref.lstm_cell(ig + hg + b64, c0)                   # the same with the sum formed outside
    np.testing.assert_allclose(h, href, rtol=0, atol=1e-15)
    tol = 1e-7                                                         # the bias went through fp32
    np.testing.assert_allclose(h, h1.numpy(), rtol=0, atol=tol)
    np.testing.assert_allclose(c, c1.numpy(), rtol=0, atol=tol)
    hx, cx = kopref.lstm_cell(ig + hg + (cell.bias_ih + cell.bias_hh).detach(), c0)
    np.testing.assert_allclose(hx, h1.numpy(), rtol=0, atol=1e-14)
    np.testing.assert_allclose(cx, c1.numpy(), rtol=0, atol=1e-14)
    # closed forms: all-zero gates halve the cell state; saturated gates pass or block it
    z = np.zeros((1, 8))
    h, c = kopref.lstm_cell(z, np.array([[2.0, -4.0]]))
    assert np.array_equal(c, [[1.0, -2.0]]) and h[0, 0] == pytest.approx(0.5 * math.tanh(1.0), rel=1e-15)
    big = np.array([[-40.0, -40.0, 40.0, 40.0, 0.3, -0.7, 40.0, 40.0]])   # i closed, f open, o open, H = 2
    h, c = kopref.lstm_cell(big, np.array([[0.25, -1.5]]))
    np.testing.assert_allclose(c, [[0.25, -1.5]], rtol=1e-15)
    np.testing.assert_allclose(h, np.tanh([[0.25, -1.5]]), rtol=1e-15)
    big = np.array([[40.0, 40.0, -40.0, -40.0, 0.3, -0.7, 40.0, 40.0]])   # i open, f closed: c = tanh(g)
    h, c = kopref.lstm_cell(big, np.array([[9.0, 9.0]]))
    np.testing.assert_allclose(c, np.tanh([[0.3, -0.7]]), rtol=1e-15)


def test_gru_cell_against_torch_grucell_and_closed_forms():
    B, I, H = 5, 7, 6
    cell = torch.nn.GRUCell(I, H).double()
    xin = torch.from_numpy(RNG.normal(0, 1, (B, I)))
    h0 = torch.from_numpy(RNG.normal(0, 1, (B, H)))
    with torch.no_grad():
        h1 = cell(xin, h0)                         # the library routine fixes the block order r, z, n and the n-gate form
        gi = xin @ cell.weight_ih.t()              # the two preserved GEMMs
        gh = h0 @ cell.weight_hh.t()
        bi, bh = cell.bias_ih.detach(), cell.bias_hh.detach()
    got = kopref.gru_cell(gi + bi, gh + bh, h0)                        # biases added outside, in float64
    np.testing.assert_allclose(got, h1.numpy(), rtol=0, atol=1e-14)
    got32 = kopref.gru_cell(gi, gh, h0, bias_i=bi.float(), bias_h=bh.float())
    np.testing.assert_allclose(got32, h1.numpy(), rtol=0, atol=1e-6)   # the biases went through fp32
    same = kopref.gru_cell(gi + bi.float().double(), gh + bh.float().double(), h0)
    np.testing.assert_allclose(got32, same, rtol=0, atol=1e-15)
    # the hidden bias of the candidate sits inside the reset gate: moving it to the input side changes the result
    moved = kopref.gru_cell(gi + bi + torch.cat([torch.zeros(2 * H, dtype=torch.float64), bh[2 * H:]]),
                            gh + torch.cat([bh[:2 * H], torch.zeros(H, dtype=torch.float64)]), h0)
    assert np.abs(moved - h1.numpy()).max() > 1e-3
    # closed forms (H = 2): zero gates average tanh(0) = 0 and h; z saturated keeps h; z closed and r closed give tanh(gi_n)
    z6 = np.zeros((1, 6))
    assert np.array_equal(kopref.gru_cell(z6, z6, np.array([[2.0, -4.0]])), [[1.0, -2.0]])
    keep = np.array([[0.0, 0.0, 40.0, 40.0, 0.3, -0.7]])
    np.testing.assert_allclose(kopref.gru_cell(keep, z6, np.array([[0.25, -1.5]])), [[0.25, -1.5]], rtol=1e-15)
    gi_c = np.array([[-40.0, -40.0, -40.0, -40.0, 0.3, -0.7]])         # r = 0, z = 0
    gh_c = np.array([[0.0, 0.0, 0.0, 0.0, 5.0, 5.0]])                  # blocked by r
    np.testing.assert_allclose(kopref.gru_cell(gi_c, gh_c, np.array([[9.0, 9.0]])), np.tanh([[0.3, -0.7]]), rtol=1e-12)
    gi_o = np.array([[40.0, 40.0, -40.0, -40.0, 0.3, -0.7]])           # r = 1, z = 0: n = tanh(gi_n + gh_n)
    np.testing.assert_allclose(kopref.gru_cell(gi_o, gh_c, np.array([[9.0, 9.0]])), np.tanh([[5.3, 4.3]]), rtol=1e-12)
    # 16-bit inputs are widened exactly
    g16 = torch.from_numpy(RNG.normal(0, 1, (3, 12))).to(torch.bfloat16)
    h16 = torch.from_numpy(RNG.normal(0, 1, (3, 4))).to(torch.bfloat16)
    np.testing.assert_array_equal(kopref.gru_cell(g16, g16, h16), kopref.gru_cell(g16.double(), g16.double(), h16.double()))


def test_16_bit_parameters_widen_exactly_and_match_the_float64_library_norms():
    """Parameters stored in bf16 / fp16: the oracle widens them to fp32 before use. Every one of the 65,536 bit
    patterns of each format must come out as the value the format defines (checked against the oracle's own
    bit-field decoder for data tensors, a separate implementation), and LayerNorm / RMSNorm with such
    parameters must equal the float64 library routine given the same parameters widened by torch."""
    bits = torch.arange(65536, dtype=torch.int32).to(torch.int16)
    for tdt in (torch.bfloat16, torch.float16):
        t = bits.view(tdt)
        with np.errstate(invalid="ignore"):                       # signalling NaN patterns
            via_param = kopref.as_param(t).astype(np.float64)
        decoded = kopref.residual_add(t.reshape(1, -1), torch.zeros((1, 65536), dtype=tdt))[0]   # the C decoder, + 0
        ref = t.double().numpy()
        ok = ~np.isnan(ref)
        assert np.array_equal(via_param[ok], ref[ok]) and np.array_equal(np.isnan(via_param), np.isnan(ref))
        assert np.array_equal(via_param[ok], decoded[ok]) and np.array_equal(np.isnan(via_param), np.isnan(decoded))
    H = 96
    x = torch.from_numpy(RNG.normal(0, 1, (7, H))).to(torch.bfloat16)
    g16 = torch.from_numpy(RNG.normal(1, 0.1, H)).to(torch.bfloat16)
    b16 = torch.from_numpy(RNG.normal(0, 0.1, H)).to(torch.bfloat16)
    y, _, _ = kopref.residual_layernorm(x, None, g16, b16, 1e-5)
    ref = torch.nn.functional.layer_norm(x.double(), (H,), g16.double(), b16.double(), 1e-5).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)
    yr = kopref.rmsnorm(x, g16, 1e-6)
    refr = torch.nn.functional.rms_norm(x.double(), (H,), g16.double(), 1e-6).numpy()
    np.testing.assert_allclose(yr, refr, rtol=0, atol=1e-13)
    # rounding the parameters to bf16 is visible: the fp32 originals give a different result
    g32 = torch.from_numpy(RNG.normal(1, 0.1, H)).float()
    assert np.abs(kopref.rmsnorm(x, g32, 1e-6) - kopref.rmsnorm(x, g32.to(torch.bfloat16), 1e-6)).max() > 1e-4


def test_lp_normalize_rows_against_torch_and_closed_forms():
    x = torch.from_numpy(RNG.normal(0, 2, (9, 37)))
    for p in (1, 2):
        y, n = kopref.lp_normalize_rows(x, p, 1e-12)
        np.testing.assert_allclose(y, torch.nn.functional.normalize(x, p=float(p), dim=1, eps=1e-12).numpy(), rtol=1e-14, atol=0)
        np.testing.assert_allclose(n, torch.linalg.vector_norm(x, ord=p, dim=1).numpy(), rtol=1e-14)
        # the result has unit p-norm, and scaling the row by c only changes the sign
        np.testing.assert_allclose(np.linalg.norm(y, ord=p, axis=1), 1.0, rtol=1e-13)
        y3, n3 = kopref.lp_normalize_rows(x * -3.0, p, 1e-12)
        np.testing.assert_allclose(y3, -y, rtol=1e-13, atol=0)
        np.testing.assert_allclose(n3, 3.0 * n, rtol=1e-13)
    # closed forms: the 3-4-5 triangle; p = 1 divides by the sum of magnitudes
    y, n = kopref.lp_normalize_rows(np.array([[3.0, -4.0]]), 2)
    assert n[0] == 5.0 and np.array_equal(y, [[0.6, -0.8]])
    y, n = kopref.lp_normalize_rows(np.array([[1.0, -2.0, 5.0]]), 1)
    assert n[0] == 8.0 and np.array_equal(y, [[0.125, -0.25, 0.625]])
    # eps: a zero row stays zero (0 / eps), a tiny row is divided by eps, not by its norm
    y, n = kopref.lp_normalize_rows(np.zeros((1, 4)), 2, 1e-6)
    assert n[0] == 0.0 and np.array_equal(y, np.zeros((1, 4)))
    y, _ = kopref.lp_normalize_rows(np.array([[1e-9, 0.0]]), 2, 1e-6)
    np.testing.assert_allclose(y, [[1e-3, 0.0]], rtol=1e-15)
    # p = 1 and p = 2 differ (a transposed switch would show here)
    a, _ = kopref.lp_normalize_rows(np.array([[1.0, 1.0]]), 1)
    b, _ = kopref.lp_normalize_rows(np.array([[1.0, 1.0]]), 2)
    assert a[0, 0] == 0.5 and b[0, 0] == pytest.approx(2 ** -0.5, rel=1e-15)
    # a NaN makes its whole row NaN; 16-bit data is widened exactly
    y, n = kopref.lp_normalize_rows(np.array([[1.0, float("nan")], [3.0, 4.0]]), 2)
    assert np.isnan(y[0]).all() and np.isnan(n[0]) and np.array_equal(y[1], [0.6, 0.8])
    h = torch.from_numpy(RNG.normal(0, 1, (3, 16))).to(torch.bfloat16)
    np.testing.assert_array_equal(kopref.lp_normalize_rows(h, 2)[0], kopref.lp_normalize_rows(h.double(), 2)[0])
