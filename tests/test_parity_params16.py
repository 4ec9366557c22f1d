"""GPU parity of kop_layernorm_ex / kop_rmsnorm_ex against the float64 CPU oracle with the parameter vectors
stored in the data type (bf16 / fp16) and in fp32: four LayerNorm prologues, RMSNorm with and without the
residual add, five seeds, register-row, row-pair and generic kernels, misaligned parameters. The oracle
receives the same 16-bit parameters and widens them exactly. Tolerance |got - ref| <= tol * max(1, |ref|),
tol = 2e-2 (bf16), 2e-3 (fp16), 1e-5 (fp32 data, fp32 parameters only)."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_bf16_tight, assert_close, tol_of

pytestmark = pytest.mark.gpu
SEEDS = synth.SEEDS
F32, BF16, F16 = torch.float32, torch.bfloat16, torch.float16


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


def ln_oracle(pro, x, r, b, g, be, eps):
    if pro == "bias_gelu_residual":
        return kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), eps, threads=None)
    if pro == "bias_erfgelu_residual":
        return kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), eps, threads=None, erf_form=True)
    return kopref.residual_layernorm(host(x), host(r) if pro == "residual" else None, host(g), host(be), eps, threads=None)


# 4096 x 600 rows: the row-pair kernel; 4096 x 40: one row per CTA; 1000: tail predicates; 1001: generic kernel
@pytest.mark.parametrize("rows,hidden,dtype", [(1300, 4096, BF16), (40, 4096, F16), (33, 1000, BF16), (17, 1001, F16),
                                               (9, 8192, BF16), (5, 24576, BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_layernorm_ex_16_bit_parameters(kop, rows, hidden, dtype, seed):
    x, r, b, g, be = synth.layernorm_inputs(rows, hidden, dtype, seed, "cuda")
    b16, g16, be16 = b.to(dtype), g.to(dtype), be.to(dtype)
    tol = tol_of(dtype)
    for pro in kop.LN_PROLOGUES:
        y = Guarded((rows, hidden), dtype)
        _, mean, rstd = kop.kop_layernorm_ex(x, r, b16, g16, be16, 1e-5, pro, out=y.t)
        ry, rmean, rrstd = ln_oracle(pro, x, r, b16, g16, be16, 1e-5)
        assert_close(y.t, ry, tol, f"layernorm_ex {pro} 16-bit params")
        if dtype == BF16:
            assert_bf16_tight(y.t, ry, f"layernorm_ex {pro}")
        assert_close(mean, rmean, 1e-5, f"{pro} mean")
        assert_close(rstd, rrstd, 1e-5, f"{pro} rstd")
        y.check(pro)
    # fp32 parameters through the same entry point give exactly what the fixed-type entry point gives
    ya, _, _ = kop.kop_layernorm_ex(x, r, b, g, be, 1e-5, "bias_gelu_residual")
    yb, _, _ = kop.kop_bias_gelu_residual_layernorm(x, r, b, g, be, 1e-5)
    assert torch.equal(ya, yb)


@pytest.mark.parametrize("rows,hidden,dtype", [(600, 4096, BF16), (40, 4096, F16), (33, 1000, BF16), (17, 1001, F16),
                                               (5, 24576, F16),
                                               # rows kept packed in registers: exact (384 / 512 threads) and ragged
                                               (19, 12288, BF16), (11, 16384, F16), (7, 10000, BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_rmsnorm_ex_16_bit_parameters(kop, rows, hidden, dtype, seed):
    x, r, _, g, _ = synth.layernorm_inputs(rows, hidden, dtype, seed, "cuda")
    w16 = g.to(dtype)
    tol = tol_of(dtype)
    y = Guarded((rows, hidden), dtype)
    kop.kop_rmsnorm_ex(x, w16, 1e-6, out=y.t)
    ref = kopref.rmsnorm(host(x), host(w16), 1e-6, threads=None)
    assert_close(y.t, ref, tol, "rmsnorm_ex 16-bit weight")
    if dtype == BF16:
        assert_bf16_tight(y.t, ref, "rmsnorm_ex")
    y.check("rmsnorm_ex")
    h = Guarded((rows, hidden), dtype)
    y2 = Guarded((rows, hidden), dtype)
    kop.kop_rmsnorm_ex(x, w16, 1e-6, residual=r, h_out=h.t, out=y2.t)
    rh, ry = kopref.residual_rmsnorm(host(x), host(r), host(w16), 1e-6, threads=None)
    assert_close(h.t, rh, tol, "rmsnorm_ex residual h")
    assert_close(y2.t, ry, tol, "rmsnorm_ex residual y")
    h.check("h")
    y2.check("y")
    assert torch.equal(kop.kop_rmsnorm_ex(x, g, 1e-6), kop.kop_rmsnorm(x, g, 1e-6))


def test_norm_ex_misaligned_parameters_and_fp32_data(kop):
    rows, hidden = 24, 2048
    x, r, b, g, be = synth.layernorm_inputs(rows, hidden, BF16, 4, "cuda")
    p = [t.to(BF16) for t in (b, g, be)]
    ref, _, _ = ln_oracle("bias_gelu_residual", x, r, *p, 1e-5)
    shifted = []
    for t in p:                                            # 2-byte aligned only: the generic kernel
        buf = torch.zeros(hidden + 1, dtype=BF16, device="cuda")
        buf[1:] = t
        shifted.append(buf[1:])
    y, _, _ = kop.kop_layernorm_ex(x, r, *shifted, 1e-5, "bias_gelu_residual")
    assert_close(y, ref, 2e-2, "misaligned 16-bit parameters")
    assert_close(kop.kop_rmsnorm_ex(x, shifted[1], 1e-6), kopref.rmsnorm(host(x), host(p[1]), 1e-6), 2e-2, "misaligned weight")
    xf, rf, bf, gf, bef = synth.layernorm_inputs(rows, hidden, F32, 4, "cuda")
    yf, _, _ = kop.kop_layernorm_ex(xf, rf, bf, gf, bef, 1e-5, "residual")
    assert_close(yf, kopref.residual_layernorm(host(xf), host(rf), host(gf), host(bef), 1e-5)[0], 1e-5, "fp32 data")
    with pytest.raises(Exception):
        kop.kop_layernorm_ex(xf, rf, bf.to(BF16), gf.to(BF16), bef.to(BF16), 1e-5)


def test_layernorm_ex_benchmark_shape_sampled_rows(kop):
    cfg = synth.CONFIGS["layernorm"]
    rows, hidden, dtype = cfg["rows"], cfg["hidden"], cfg["dtype"]
    x, r, b, g, be = synth.layernorm_inputs(rows, hidden, dtype, 0, "cuda")
    p = [t.to(dtype) for t in (b, g, be)]
    y, _, _ = kop.kop_layernorm_ex(x, r, *p, cfg["eps"], "bias_gelu_residual")
    idx = torch.tensor(sorted({0, 1, rows - 2, rows - 1} | set(np.random.default_rng(1).integers(0, rows, 60).tolist()))).cuda()
    ref, _, _ = ln_oracle("bias_gelu_residual", x[idx], r[idx], *p, cfg["eps"])
    assert_close(y[idx], ref, tol_of(dtype), "full-size sampled rows, 16-bit parameters")


# ------------------------------------------------------------------ the other entry points with 16-bit parameters

# vector kernels (lanes per row, warp per row, CTA per row, two sweeps), ragged and odd lengths (scalar kernel)
@pytest.mark.parametrize("rows,cols,dtype", [(700, 64, BF16), (333, 512, F16), (129, 4096, BF16), (5, 40000, BF16),
                                             (33, 777, F16), (9, 1000, BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_softmax_ex_16_bit_bias(kop, rows, cols, dtype, seed):
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    b16 = bias.to(dtype)
    tol = tol_of(dtype)
    y = Guarded((rows, cols), dtype)
    kop.kop_softmax_ex(x, b16, 0.125, out=y.t)
    assert_close(y.t, kopref.softmax_scale_bias(host(x), host(b16), 0.125, threads=None), tol, "softmax_ex")
    y.check("softmax_ex")
    for log_out, period in ((True, 0), (False, cols), (True, max(1, cols // 2))):
        got = kop.kop_softmax_ex(x, b16, 0.5, log_out, period).cpu().double().numpy()
        ref = kopref.softmax_opts(host(x), host(b16), 0.5, log_out, period, threads=None)
        fin = np.isfinite(ref)
        assert np.array_equal(np.isneginf(got), np.isneginf(ref))
        assert np.all(np.abs(got[fin] - ref[fin]) <= tol * np.maximum(1.0, np.abs(ref[fin]))), (log_out, period)
    # fp32 bias through the same entry point: bit for bit what the fixed-type entry points give; no bias at all
    assert torch.equal(kop.kop_softmax_ex(x, bias, 0.125), kop.kop_softmax_scale_bias(x, bias, 0.125))
    assert torch.equal(kop.kop_softmax_ex(x, bias, 0.125, True, cols), kop.kop_softmax_opts(x, bias, 0.125, True, cols))
    assert torch.equal(kop.kop_softmax_ex(x, None, 0.125), kop.kop_softmax_scale_bias(x, None, 0.125))


@pytest.mark.parametrize("shape,dtype", [((3, 40, 56, 56), BF16), ((2, 24, 7, 7), F16), ((5, 16, 14, 14), BF16),
                                         ((2, 9, 5, 3), F16), ((2, 64, 28, 28), BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_bn_relu_avgpool_ex_16_bit_scale_shift(kop, shape, dtype, seed):
    x, sc, sh = synth.bn_pool_inputs(*shape, dtype, seed, "cuda")
    sc16, sh16 = sc.to(dtype), sh.to(dtype)
    tol = tol_of(dtype)
    ry, rp = kopref.bn_relu_avgpool(host(x), host(sc16), host(sh16), threads=None)
    y, p = kop.kop_bn_relu_avgpool_ex(x, sc16, sh16)
    assert_close(y, ry, tol, "bn_ex y")
    assert_close(p, rp, 1e-5, "bn_ex pooled")
    xl = x.contiguous(memory_format=torch.channels_last)
    yl, pl = kop.kop_bn_relu_avgpool_ex(xl, sc16, sh16)
    assert_close(yl, ry, tol, "bn_ex channels-last y")
    assert_close(pl, rp, 1e-5, "bn_ex channels-last pooled")
    a = kop.kop_bn_relu_avgpool_ex(x, sc, sh)
    b = kop.kop_bn_relu_avgpool(x, sc, sh)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("shape,groups,dtype", [((3, 32, 28, 28), 8, BF16), ((2, 16, 56, 56), 16, F16), ((4, 12, 7, 7), 4, BF16),
                                                ((2, 6, 5, 3), 2, F16), ((1, 8, 112, 112), 1, BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_groupnorm_act_ex_16_bit_gamma_beta(kop, shape, groups, dtype, seed):
    x, g, b = synth.groupnorm_inputs(*shape, dtype, seed, "cuda")
    g16, b16 = g.to(dtype), b.to(dtype)
    tol = tol_of(dtype)
    for act in (0, 1, 2):
        y, mu, rs = kop.kop_groupnorm_act_ex(x, g16, b16, groups, 1e-5, act)
        ry, rm, rr = kopref.groupnorm_act(host(x), host(g16), host(b16), groups, 1e-5, act, threads=None)
        assert_close(y, ry, tol, f"groupnorm_ex act={act}")
        assert_close(mu, rm, 1e-3, "groupnorm_ex mean")
        assert_close(rs, rr, 1e-3, "groupnorm_ex rstd")
    y, _, _ = kop.kop_groupnorm_act_ex(x, g16, None, groups, 1e-5, 0)        # gamma only
    assert_close(y, kopref.groupnorm_act(host(x), host(g16), None, groups, 1e-5, 0, threads=None)[0], tol, "gamma only")
    a = kop.kop_groupnorm_act_ex(x, g, b, groups, 1e-5, 2)
    c = kop.kop_groupnorm_act(x, g, b, groups, 1e-5, 2)
    assert torch.equal(a[0], c[0]) and torch.equal(a[1], c[1]) and torch.equal(a[2], c[2])
    assert kop.kop_groupnorm_wait_timeouts() == 0


@pytest.mark.parametrize("rows,cols,dtype", [(300, 4096, BF16), (2000, 64, F16), (65, 1000, BF16), (17, 1001, F16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_bias_act_and_chain_ex_16_bit_bias(kop, rows, cols, dtype, seed):
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    r, _ = synth.softmax_inputs(rows, cols, dtype, seed + 7, "cuda")
    b16 = bias.to(dtype)
    tol = tol_of(dtype)
    for act in ("gelu_tanh", "silu", "relu", "mish"):
        y = Guarded((rows, cols), dtype)
        kop.kop_bias_act_ex(x, b16, act, out=y.t)
        assert_close(y.t, kopref.bias_act(host(x), host(b16), act, threads=None), tol, f"bias_act_ex {act}")
        y.check("bias_act_ex")
    y = kop.kop_epilogue_chain_ex(x, b16, r, 0.5, 2.0, -1.0, 1.5, "silu")
    assert_close(y, kopref.epilogue_chain(host(x), host(b16), host(r), 0.5, 2.0, -1.0, 1.5, "silu", threads=None), tol, "chain_ex")
    y = kop.kop_epilogue_chain_ex(x, b16, None, 1.25, 1.0, act="gelu_erf")
    assert_close(y, kopref.epilogue_chain(host(x), host(b16), None, 1.25, 1.0, act="gelu_erf", threads=None), tol, "chain_ex no residual")
    assert torch.equal(kop.kop_bias_act_ex(x, bias, "gelu_tanh"), kop.kop_bias_act(x, bias, "gelu_tanh"))
    assert torch.equal(kop.kop_epilogue_chain_ex(x, bias, r, 0.5, 2.0, -1.0, 1.5, "silu"),
                       kop.kop_epilogue_chain(x, bias, r, 0.5, 2.0, -1.0, 1.5, "silu"))
    assert torch.equal(kop.kop_bias_act_ex(x, None, "relu"), kop.kop_bias_act(x, None, "relu"))


# one geometry per pooling kernel: stride-2 strip, stride-1 strip, shared-memory walk, runs of small planes, generic
# tile, direct (rows too wide for a tile)
POOL_EX_CASES = [
    (2, 8, 112, 112, (3, 3), (2, 2), (1, 1), BF16),
    (1, 3, 57, 64, (3, 3), (1, 1), (1, 1), F16),
    (2, 3, 57, 57, (3, 3), (1, 1), (1, 1), BF16),
    (5, 37, 7, 7, (3, 3), (2, 2), (1, 1), F16),
    (3, 50, 14, 14, (3, 3), (2, 2), (1, 1), BF16),
    (2, 3, 30, 44, (5, 3), (2, 1), (2, 1), F16),
    (1, 2, 6, 5000, (3, 3), (2, 2), (1, 1), BF16),
    # 2x2 / stride 2: a thread per output (pairs), two outputs a thread (width divisible by four), scalar loads (odd width)
    (5, 37, 14, 14, (2, 2), (2, 2), (0, 0), F16),
    (3, 50, 28, 28, (2, 2), (2, 2), (0, 0), BF16),
    (6, 11, 7, 7, (2, 2), (2, 2), (0, 0), BF16),
]


@pytest.mark.parametrize("N,C,H,W,kernel,stride,padding,dtype", POOL_EX_CASES)
@pytest.mark.parametrize("seed", SEEDS)
def test_affine_relu_pool2d_ex_16_bit_scale_shift(kop, N, C, H, W, kernel, stride, padding, dtype, seed):
    x, sc, sh = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
    sc16, sh16 = sc.to(dtype), sh.to(dtype)
    tol = tol_of(dtype)
    OH = (H + 2 * padding[0] - kernel[0]) // stride[0] + 1
    OW = (W + 2 * padding[1] - kernel[1]) // stride[1] + 1
    for mode in ("max", "avg"):
        for relu in (True, False):
            y = Guarded((N, C, OH, OW), dtype)
            kop.kop_affine_relu_pool2d_ex(x, sc16, sh16, kernel, stride, padding, mode, relu, out=y.t)
            ref = kopref.affine_relu_pool2d(host(x), host(sc16), host(sh16), kernel, stride, padding, mode, relu, threads=None)
            assert_close(y.t, ref, tol, f"pool2d_ex {mode} relu={relu}")
            y.check("pool2d_ex")
        # fp32 parameters and no parameters through the new entry point: bit-equal to the base entry point
        assert torch.equal(kop.kop_affine_relu_pool2d_ex(x, sc, sh, kernel, stride, padding, mode, True),
                           kop.kop_affine_relu_pool2d(x, sc, sh, kernel, stride, padding, mode, True))
        assert torch.equal(kop.kop_affine_relu_pool2d_ex(x, None, None, kernel, stride, padding, mode, False),
                           kop.kop_affine_relu_pool2d(x, None, None, kernel, stride, padding, mode, False))


def test_ex_entry_points_misaligned_parameters_and_type_rules(kop):
    rows, cols = 40, 2048
    x, bias = synth.softmax_inputs(rows, cols, BF16, 2, "cuda")
    b16 = bias.to(BF16)
    buf = torch.zeros(cols + 1, dtype=BF16, device="cuda")
    buf[1:] = b16                                             # 2-byte aligned only: the scalar-load kernels
    ref = kopref.softmax_scale_bias(host(x), host(b16), 1.0)
    assert_close(kop.kop_softmax_ex(x, buf[1:], 1.0), ref, 2e-2, "misaligned 16-bit softmax bias")
    assert_close(kop.kop_bias_act_ex(x, buf[1:], "silu"), kopref.bias_act(host(x), host(b16), "silu"), 2e-2, "misaligned bias")
    # 16-bit parameters go with 16-bit data of the same type only
    xf = x.float()
    for call in (lambda: kop.kop_softmax_ex(xf, b16, 1.0), lambda: kop.kop_bias_act_ex(x, bias.half(), "relu")):
        with pytest.raises(Exception):
            call()
    L = kop.lib()
    P, Q, R = 0x10000, 0x20000, 0x30000
    assert L.kop_softmax_ex(P, Q, R, 4, 8, 8, 8, 1.0, 0, 0, 0, 1, None) == 4          # fp32 data, bf16 params
    assert L.kop_softmax_ex(P, Q, R, 4, 8, 8, 8, 1.0, 0, 0, 1, 2, None) == 4          # bf16 data, fp16 params
    assert L.kop_bias_act_ex(P, Q, R, 4, 8, 8, 8, 1, 0.0, 2, 1, None) == 4
    assert L.kop_epilogue_chain_ex(P, Q, None, R, 4, 8, 8, 8, 8, 1.0, 1.0, -1.0, 1.0, 0, 0.0, 1, 7, None) == 4
    assert L.kop_softmax_ex(P, Q + 1, R, 4, 8, 8, 8, 1.0, 0, 0, 1, 1, None) == 5      # bias not on a 2-byte boundary
    pool = (1, 2, 8, 8, 3, 3, 2, 2, 1, 1, 0, 1)
    assert L.kop_affine_relu_pool2d_ex(P, Q, Q, R, *pool, 0, 1, None) == 4            # fp32 data, bf16 params
    assert L.kop_affine_relu_pool2d_ex(P, Q, Q, R, *pool, 2, 1, None) == 4            # fp16 data, bf16 params
    assert L.kop_affine_relu_pool2d_ex(P, Q, Q + 1, R, *pool, 1, 1, None) == 5        # shift not on a 2-byte boundary
    assert L.kop_affine_relu_pool2d_ex(P, Q, Q + 2, R, *pool, 1, 0, None) == 5        # fp32 shift on a 2-byte boundary
    assert L.kop_affine_relu_pool2d_ex(P, Q, None, R, *pool, 1, 1, None) == 1         # scale without shift
