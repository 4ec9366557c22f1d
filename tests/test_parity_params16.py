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
                                               (5, 24576, F16)])
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
