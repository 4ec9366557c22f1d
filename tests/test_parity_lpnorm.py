"""GPU parity of kop_lp_normalize_rows against the float64 CPU oracle: p = 1 and 2, three data types, five seeds,
every kernel shape (lanes per row, CTA per row, two sweeps, scalar), in place, strided, eps and special values,
guard bands. Tolerance |got - ref| <= tol * max(1, |ref|), tol = 1e-5 (fp32), 2e-2 (bf16), 2e-3 (fp16); norms
to 1e-5 relative."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_bf16_tight, assert_close, to_f64, tol_of

pytestmark = pytest.mark.gpu
SEEDS = synth.SEEDS
F32, BF16, F16 = torch.float32, torch.bfloat16, torch.float16
SHAPES = [(2048, 4096, BF16), (300, 4096, F32), (1031, 64, BF16), (517, 128, F32), (259, 520, F16), (65, 1000, F32),
          (33, 1001, F32), (17, 16384, BF16), (9, 20480, F32), (5, 40008, BF16), (3, 20481, BF16), (7, 1, F32),
          (131, 768, BF16), (67, 1024, F16),
          # rows that are not whole aligned vectors: edge elements around the aligned vectors in all three kernels
          (700, 197, BF16), (300, 77, F32), (64, 1001, F32), (41, 4097, BF16), (9, 20011, BF16), (5, 70001, F32),
          (130, 7, torch.float16), (50, 3, F32), (33, 2051, torch.float16)]


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


@pytest.mark.parametrize("rows,cols,dtype", SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_lp_normalize_parity(kop, rows, cols, dtype, seed):
    x, _ = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
    tol = tol_of(dtype)
    for p in (1, 2):
        y = Guarded((rows, cols), dtype)
        n = Guarded((rows,), F32)
        kop.kop_lp_normalize_rows(x, p, 1e-12, out=y.t, norms=n.t)
        ry, rn = kopref.lp_normalize_rows(host(x), p, 1e-12, threads=None)
        assert_close(y.t, ry, tol, f"lp_normalize p={p}")
        if dtype == BF16:
            assert_bf16_tight(y.t, ry, f"lp_normalize p={p}", floor=1e-6)
        assert np.all(np.abs(to_f64(n.t) - rn) <= 1e-5 * np.maximum(1e-30, np.abs(rn))), f"norms p={p}"
        y.check("y")
        n.check("norms")


def test_lp_normalize_options_and_special_values(kop):
    rows, cols = 40, 2048
    x, _ = synth.softmax_inputs(rows, cols, F32, 9, "cuda")
    ref, rn = kopref.lp_normalize_rows(host(x), 2, 1e-12)
    xi = x.clone()
    out, norms = kop.kop_lp_normalize_rows(xi, 2, out=xi)                         # in place
    assert out is xi
    assert_close(xi, ref, 1e-5, "in place")
    big = torch.zeros((rows, cols + 40), dtype=F32, device="cuda")                # strided rows
    big[:, :cols] = x
    outb = torch.full((rows, cols + 8), 5.0, dtype=F32, device="cuda")
    kop.kop_lp_normalize_rows(big[:, :cols], 2, out=outb[:, :cols], want_norms=False)
    assert_close(outb[:, :cols], ref, 1e-5, "strided")
    assert bool((outb[:, cols:] == 5.0).all())
    flat = torch.zeros(rows * cols + 1, dtype=F32, device="cuda")                 # misaligned base: scalar kernel
    flat[1:] = x.reshape(-1)
    assert_close(kop.kop_lp_normalize_rows(flat[1:].view(rows, cols), 2)[0], ref, 1e-5, "misaligned")
    # eps: a zero row stays zero, a tiny row is divided by eps; NaN and infinity
    inf, nan = float("inf"), float("nan")
    sp = torch.tensor([[0.0, 0.0, 0.0, 0.0], [1e-9, 0.0, 0.0, 0.0], [3.0, -4.0, 0.0, 0.0], [1.0, nan, 2.0, 3.0],
                       [1.0, inf, 2.0, 3.0]], device="cuda")
    for p in (1, 2):
        got, gn = kop.kop_lp_normalize_rows(sp, p, 1e-6)
        ry, rn = kopref.lp_normalize_rows(host(sp), p, 1e-6)
        g, n = got.cpu().double().numpy(), gn.cpu().double().numpy()
        assert np.array_equal(np.isnan(g), np.isnan(ry)) and np.array_equal(np.isnan(n), np.isnan(rn))
        ok = ~np.isnan(ry)
        assert np.allclose(g[ok], ry[ok], rtol=1e-5, atol=1e-12)
        okn = np.isfinite(rn)
        assert np.allclose(n[okn], rn[okn], rtol=1e-6) and np.array_equal(np.isinf(n), np.isinf(rn))
    # a tensor as one row: its Frobenius norm
    t = x[:8].contiguous().view(1, -1)
    _, fn = kop.kop_lp_normalize_rows(t, 2)
    assert abs(float(fn[0]) - float(torch.linalg.matrix_norm(x[:8].double()))) <= 1e-5 * float(fn[0])


def test_lp_normalize_rows_off_the_vector_grid(kop):
    """x and y one element off a 16-byte boundary alike (the split kernels), in place, and at different offsets (the
    element-wise kernel); nothing outside y may change."""
    for dtype, (rows, cols) in ((BF16, (300, 197)), (F32, (64, 1001)), (torch.float16, (5, 20011))):
        x, _ = synth.softmax_inputs(rows, cols, dtype, 3, "cuda")
        n = rows * cols
        ry, rn = kopref.lp_normalize_rows(host(x), 2, 1e-12, threads=None)
        xo = torch.zeros(n + 16, dtype=dtype, device="cuda")
        xo[1:n + 1] = x.reshape(-1)
        for yoff in (1, 2):
            yo = torch.full((n + 16,), 9.0, dtype=dtype, device="cuda")
            _, norms = kop.kop_lp_normalize_rows(xo[1:n + 1].view(rows, cols), 2, 1e-12, out=yo[yoff:n + yoff].view(rows, cols))
            assert_close(yo[yoff:n + yoff].view(rows, cols), ry, tol_of(dtype), f"lp_normalize off the grid, y offset {yoff}")
            assert np.all(np.abs(to_f64(norms) - rn) <= 1e-5 * np.maximum(1e-30, np.abs(rn)))
            assert bool((yo[:yoff] == 9.0).all()) and bool((yo[n + yoff:] == 9.0).all())
        xi = xo[1:n + 1].view(rows, cols)
        kop.kop_lp_normalize_rows(xi, 2, 1e-12, out=xi)
        assert_close(xi, ry, tol_of(dtype), "lp_normalize off the grid, in place")
