"""GPU parity of kop_reduce_rows against the float64 CPU oracle: five seeds, the five operations, three data
types, rows for the CTA-per-row and the warp-per-row kernels (vector and scalar paths), strided and
misaligned inputs, ties, NaN / infinity rules, guard bands, run-to-run bit equality.

max / min values and argmax / argmin indices must be bit-exact. logsumexp is held to
tol * max(1, |ref|) with tol = 1e-5 whatever the data type (the output is fp32; the input is widened
exactly). A sum is not bounded by its own size (terms cancel): it is held to 1e-5 * max(1, sum_j |x_j|)
(an fp32 tree of `cols` terms rounds relative to the partial sums on the way), the mean to that over cols."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, to_f64

pytestmark = pytest.mark.gpu
SEEDS = synth.SEEDS
F32, BF16, F16 = torch.float32, torch.bfloat16, torch.float16
OPS = ("sum", "mean", "max", "min", "logsumexp")


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return t.detach().cpu()


def check_op(kop, x, xh, op, what):
    rows, cols = x.shape
    out = Guarded((rows,), F32)
    idx = Guarded((rows,), torch.int32)
    kop.kop_reduce_rows(x, op, out=out.t, index=idx.t)
    ref, ridx = kopref.reduce_rows(xh, op, threads=None)
    got = to_f64(out.t)
    if op in ("max", "min"):
        assert np.array_equal(got, ref, equal_nan=True), f"{what} {op}: values must be exact"
        assert np.array_equal(idx.t.cpu().numpy(), ridx), f"{what} {op}: indices must be exact"
    elif op == "logsumexp":
        with np.errstate(invalid="ignore"):
            ok = (np.abs(got - ref) <= 1e-5 * np.maximum(1.0, np.abs(ref))) | (got == ref) | (np.isnan(got) & np.isnan(ref))
        assert ok.all(), f"{what} logsumexp: max err {np.nanmax(np.abs(got - ref)):.3e}"
    else:
        mag = xh.double().abs().sum(dim=1).numpy()
        scale = np.maximum(1.0, mag) / (cols if op == "mean" else 1.0)
        ok = (np.abs(got - ref) <= 1e-5 * np.maximum(scale, 1e-30)) | (np.isnan(got) & np.isnan(ref))
        assert ok.all(), f"{what} {op}: max err {np.nanmax(np.abs(got - ref)):.3e}"
    out.check(what)
    idx.check(what)
    return out.t.clone(), idx.t.clone()


SHAPES = [(512, 8192, BF16), (300, 4096, F32), (65, 1000, F16), (33, 1001, F32), (9, 40000, BF16),
          (2000, 64, F32), (1000, 7, BF16), (257, 520, F16), (5, 1, F32),
          # 8, 16 and 32 lanes per row, row counts that leave part of the last warp without a row
          (67, 1024, BF16), (129, 2048, BF16), (35, 3072, F16), (131, 4096, BF16), (21, 600, F32),
          # rows that are not whole aligned vectors: edge elements before and after the aligned vectors, every lane count
          # and the CTA-per-row kernel
          (700, 197, BF16), (300, 77, F32), (41, 4097, BF16), (130, 2051, F16), (9, 50257, BF16), (7, 50257, F32),
          (50, 3, F16), (33, 8193, F32)]


@pytest.mark.parametrize("rows,cols,dtype", SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_reduce_parity(kop, rows, cols, dtype, seed):
    x, _ = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    x = x * 3.0                                           # a wider spread for the logsumexp
    xh = host(x)
    for op in OPS:
        a = check_op(kop, x, xh, op, f"reduce [{rows},{cols}] {dtype}")
        b = kop.kop_reduce_rows(x, op)
        assert torch.equal(a[0], b[0]) or bool(torch.isnan(a[0]).any()), "run-to-run bit equality"


def test_reduce_full_config_seed0(kop):
    c = synth.CONFIGS["reduce"]
    x, _ = synth.softmax_inputs(c["rows"], c["cols"], c["dtype"], 0, "cuda")
    xh = host(x)
    for op in ("sum", "max", "logsumexp"):
        check_op(kop, x, xh, op, "reduce full")


def test_reduce_ties_specials_and_layouts(kop):
    # ties: low-precision data has many equal maxima; the first position must win on every path
    for rows, cols in ((64, 4096), (64, 100)):
        x = torch.randint(-3, 4, (rows, cols), device="cuda").to(BF16)
        check_op(kop, x, host(x), "max", "ties")
        check_op(kop, x, host(x), "min", "ties")
    x, _ = synth.softmax_inputs(40, 2048, F32, 3, "cuda")
    # NaN: result NaN, index of the first NaN; other rows untouched
    xn = x.clone()
    xn[5, 1900] = float("nan")
    xn[5, 77] = float("nan")
    xn[9, 0] = float("nan")
    for op in OPS:
        v, i = check_op(kop, xn, host(xn), op, "nan")
        assert bool(torch.isnan(v[5])) and bool(torch.isnan(v[9])) and int(torch.isnan(v).sum()) == 2
        if op in ("max", "min"):
            assert int(i[5]) == 77 and int(i[9]) == 0
    # infinities
    xi = x.clone()
    xi[2] = float("-inf")
    xi[3, 100] = float("inf")
    xi[4, 7] = float("-inf")
    for op in ("max", "min", "logsumexp"):
        check_op(kop, xi, host(xi), op, "inf")
    v, i = kop.kop_reduce_rows(xi, "max")
    assert float(v[2]) == float("-inf") and int(i[2]) == 0 and float(v[3]) == float("inf") and int(i[3]) == 100
    assert float(kop.kop_reduce_rows(xi, "logsumexp")[0][2]) == float("-inf")
    # ties and NaNs that sit in the edge elements of rows that are not whole vectors: first position, whichever part holds it
    for rows, cols, dt in ((37, 197, BF16), (9, 20011, BF16), (21, 1001, F32)):
        xt = torch.randint(-2, 3, (rows, cols), device="cuda").to(dt)
        check_op(kop, xt, host(xt), "max", "edge ties")
        check_op(kop, xt, host(xt), "min", "edge ties")
        xe = xt.clone()
        xe[1, cols - 1] = float("nan")
        xe[2, 0] = float("nan")
        xe[2, cols // 2] = float("nan")
        xe[3, cols - 1] = 7.0                              # the maximum in the last element
        xe[4, 0] = -7.0                                    # the minimum in the first
        for op in OPS:
            v, i = check_op(kop, xe, host(xe), op, "edge specials")
            if op in ("max", "min"):
                assert int(i[1]) == cols - 1 and int(i[2]) == 0
        assert int(kop.kop_reduce_rows(xe, "max")[1][3]) == cols - 1 and int(kop.kop_reduce_rows(xe, "min")[1][4]) == 0
    # strided rows and a misaligned base (edge elements around the aligned vectors)
    big = torch.zeros((40, 2048 + 24), dtype=F32, device="cuda")
    big[:, :2048] = x
    for op in OPS:
        check_op(kop, big[:, :2048], host(x), op, "strided")
    flat = torch.zeros(40 * 2048 + 1, dtype=F32, device="cuda")
    flat[1:] = x.reshape(-1)
    for op in OPS:
        check_op(kop, flat[1:].view(40, 2048), host(x), op, "misaligned")
    # empty and bad op
    e = torch.empty((0, 16), dtype=F32, device="cuda")
    assert kop.kop_reduce_rows(e, "sum")[0].shape == (0,)
    assert kop.lib().kop_reduce_rows(x.data_ptr(), x.data_ptr(), None, 4, 16, 16, 9, 0, None) == 2
