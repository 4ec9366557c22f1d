"""GPU parity of kop_bias_act against the float64 CPU oracle: the eleven activations, three data types, five
seeds, with and without bias, vector and scalar paths, strided and in-place use, NaN / infinity behaviour,
guard bands. Tolerance |got - ref| <= tol * max(1, |ref|), tol = 1e-5 (fp32), 2e-2 (bf16), 2e-3 (fp16)."""
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
ACTS = ("identity", "relu", "leaky_relu", "gelu_tanh", "gelu_erf", "silu", "sigmoid", "tanh", "mish", "hardswish", "elu")


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


@pytest.mark.parametrize("rows,cols,dtype", [(512, 4096, BF16), (300, 4096, F32), (65, 1000, F16), (33, 1001, F32),
                                             (9, 20480, BF16), (7, 1, F32), (700, 197, BF16), (41, 5003, BF16),
                                             (300, 9, F16), (50, 3, F32)])
@pytest.mark.parametrize("seed", SEEDS)
def test_bias_act_parity(kop, rows, cols, dtype, seed):
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    x = x * 3.0                                            # reach the saturated ends of the activations
    bias = bias * 5.0
    tol = tol_of(dtype)
    for k, act in enumerate(ACTS):
        use_bias = (k + seed) % 3 != 0
        y = Guarded((rows, cols), dtype)
        kop.kop_bias_act(x, bias if use_bias else None, act, alpha=0.2, out=y.t)
        ref = kopref.bias_act(host(x), host(bias) if use_bias else None, act, alpha=0.2, threads=None)
        assert_close(y.t, ref, tol, f"bias_act {act} bias={use_bias}")
        if dtype == BF16:
            assert_bf16_tight(y.t, ref, f"bias_act {act}")
        y.check(act)


def test_bias_act_options(kop):
    rows, cols = 40, 2048
    x, bias = synth.softmax_inputs(rows, cols, F32, 9, "cuda")
    x = x * 4.0
    for act in ("gelu_erf", "mish", "elu"):
        ref = kopref.bias_act(host(x), host(bias), act, alpha=1.0)
        xi = x.clone()
        kop.kop_bias_act(xi, bias, act, alpha=1.0, out=xi)                       # in place
        assert_close(xi, ref, 1e-5, act + " in place")
        big = torch.zeros((rows, cols + 40), dtype=F32, device="cuda")            # strided rows
        big[:, :cols] = x
        outb = torch.full((rows, cols + 8), 5.0, dtype=F32, device="cuda")
        kop.kop_bias_act(big[:, :cols], bias, act, alpha=1.0, out=outb[:, :cols])
        assert_close(outb[:, :cols], ref, 1e-5, act + " strided")
        assert bool((outb[:, cols:] == 5.0).all())
        flat = torch.zeros(rows * cols + 1, dtype=F32, device="cuda")             # misaligned base, y aligned: element-wise kernel
        flat[1:] = x.reshape(-1)
        assert_close(kop.kop_bias_act(flat[1:].view(rows, cols), bias, act, alpha=1.0), ref, 1e-5, act + " misaligned")
    # rows that are not whole vectors, x and y one element off a 16-byte boundary alike (the span kernel's head and tail
    # elements) and at different offsets (element-wise kernel); nothing written outside y
    for dt, (r2, c2) in ((BF16, (300, 197)), (F32, (64, 1001)), (F16, (5, 7))):
        xs_, bs_ = synth.softmax_inputs(r2, c2, dt, 3, "cuda")
        n = r2 * c2
        ref = kopref.bias_act(host(xs_), host(bs_), "silu", threads=None)
        xo = torch.zeros(n + 16, dtype=dt, device="cuda")
        xo[1:n + 1] = xs_.reshape(-1)
        for yoff in (1, 2):
            yo = torch.full((n + 16,), 9.0, dtype=dt, device="cuda")
            kop.kop_bias_act(xo[1:n + 1].view(r2, c2), bs_, "silu", out=yo[yoff:n + yoff].view(r2, c2))
            assert_close(yo[yoff:n + yoff].view(r2, c2), ref, tol_of(dt), f"bias_act off the boundary, y offset {yoff}")
            assert bool((yo[:yoff] == 9.0).all()) and bool((yo[n + yoff:] == 9.0).all())
        ro = torch.zeros(n + 16, dtype=dt, device="cuda")
        ro[1:n + 1] = (xs_ * 0.5).reshape(-1)
        yo = torch.full((n + 16,), 9.0, dtype=dt, device="cuda")
        kop.kop_epilogue_chain(xo[1:n + 1].view(r2, c2), bs_, ro[1:n + 1].view(r2, c2), 0.7, 1.5, -1.0, 2.0, "gelu_tanh",
                               out=yo[1:n + 1].view(r2, c2))
        cref = kopref.epilogue_chain(host(xs_), host(bs_), host(xs_ * 0.5), 0.7, 1.5, -1.0, 2.0, "gelu_tanh", threads=None)
        assert_close(yo[1:n + 1].view(r2, c2), cref, tol_of(dt), "chain off the boundary")
        assert float(yo[0]) == 9.0 and bool((yo[n + 1:] == 9.0).all())
    # special values
    sp = torch.tensor([[float("nan"), float("inf"), float("-inf"), 0.0, -0.0, 100.0, -100.0, 1e-30]], device="cuda")
    for act in ACTS:
        got = kop.kop_bias_act(sp, None, act, alpha=0.5).cpu().double().numpy()
        ref = kopref.bias_act(host(sp), None, act, alpha=0.5)
        assert bool(np.isnan(got[0, 0])), act + ": NaN must stay NaN"
        finite = np.isfinite(ref[0])
        assert np.allclose(got[0][finite], ref[0][finite], rtol=1e-5, atol=1e-5), act + " special values"
        both_inf = np.isinf(ref[0])
        assert np.array_equal(got[0][both_inf], ref[0][both_inf]), act + " infinities"
    e = torch.empty((0, 8), dtype=F32, device="cuda")
    assert kop.kop_bias_act(e, None, "relu").shape == (0, 8)
    assert kop.lib().kop_bias_act(x.data_ptr(), None, x.data_ptr(), 4, 16, 16, 16, 11, 0.0, 0, None) == 2


@pytest.mark.parametrize("rows,cols,dtype", [(256, 4096, BF16), (300, 4096, F32), (65, 1000, F16), (33, 1001, F32), (7, 1, BF16),
                                             (700, 197, BF16), (21, 5003, F32), (300, 9, F16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_epilogue_chain_parity(kop, rows, cols, dtype, seed):
    """The general chain y = act(clamp((x + bias) * scale + residual * residual_scale, lo, hi))."""
    x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    r, _ = synth.softmax_inputs(rows, cols, dtype, seed + 1, "cuda")
    tol = tol_of(dtype)
    inf = float("inf")
    cases = [(bias, r, 0.7, 1.5, -1.0, 2.0, "gelu_tanh"), (bias, None, 2.0, 1.0, -inf, inf, "mish"),
             (None, r, 1.0, 1.0, -inf, inf, "identity"), (bias, r, 3.0, -0.5, 0.0, 6.0, "identity"),
             (None, None, 4.0, 1.0, -1.0, 1.0, "sigmoid"), (bias, r, 1.0, 1.0, -inf, 0.5, "elu")]
    for b, res, scale, rscale, lo, hi, act in cases:
        y = Guarded((rows, cols), dtype)
        kop.kop_epilogue_chain(x, b, res, scale, rscale, lo, hi, act, alpha=0.3, out=y.t)
        ref = kopref.epilogue_chain(host(x), host(b), host(res), scale, rscale, lo, hi, act, alpha=0.3, threads=None)
        assert_close(y.t, ref, tol, f"chain {act} bias={b is not None} res={res is not None}")
        y.check("chain")
    # in place over the residual, and NaN through the clamp
    ri = r.clone()
    kop.kop_epilogue_chain(x, bias, ri, 0.7, 1.5, -1.0, 2.0, "gelu_tanh", out=ri)
    assert_close(ri, kopref.epilogue_chain(host(x), host(bias), host(r), 0.7, 1.5, -1.0, 2.0, "gelu_tanh"), tol, "chain in place")
    xn = x.clone()
    xn[0, 0] = float("nan")
    assert bool(torch.isnan(kop.kop_epilogue_chain(xn, None, None, lo=0.0, hi=1.0)[0, 0]))
    with pytest.raises(kop.KopError) as ei:
        kop.kop_epilogue_chain(x, None, None, lo=1.0, hi=0.0)
    assert ei.value.status == 2
