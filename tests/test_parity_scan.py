"""GPU parity of kop_cumsum_rows against the float64 CPU oracle: five seeds, every variant (inclusive /
exclusive x forward / reverse x masked / unmasked), rows that fill one tile exactly, ragged last tiles,
rows longer than a tile (carry across tiles), the scalar kernel (row lengths that are not whole 16-byte
vectors, misaligned bases, odd mask strides), strided rows, in-place use, guard bands, NaN / infinity
placement and run-to-run bit equality.

Tolerance. A running sum is not bounded by its own value: after wandering to a partial sum of size P a
row can return to 0, and every fp32 addition on the way rounded relative to P. An output is reached
through at most ~25 additions (4 or 8 inside the vector, 5 shuffle levels twice, the carries), each
rounding by at most 2^-24 of the largest partial sum of its row, so the bound is
|got - ref| <= tol * max(1, max_k |ref[i, k]|) with the usual tol = 1e-5 (fp32 data) / 2e-2 (bf16 data)."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, to_f64, tol_of

pytestmark = pytest.mark.gpu

SEEDS = synth.SEEDS
F32, BF16 = torch.float32, torch.bfloat16


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


def assert_scan_close(got, ref, tol, what):
    g = to_f64(got)
    assert g.shape == ref.shape, what
    scale = np.maximum(1.0, np.nanmax(np.where(np.isfinite(ref), np.abs(ref), 0.0), axis=1, keepdims=True))
    same_special = (np.isnan(g) & np.isnan(ref)) | (np.isinf(ref) & (g == ref))
    with np.errstate(invalid="ignore"):
        ok = (np.abs(g - ref) <= tol * scale) | same_special
    if not ok.all():
        i = np.argwhere(~ok)[0]
        raise AssertionError(f"{what}: {(~ok).sum()} of {ok.size} outside tol={tol:g}; first at {tuple(i)}: "
                             f"got {g[tuple(i)]!r} ref {ref[tuple(i)]!r} row scale {scale[i[0], 0]:.3g}")


SCAN_SHAPES = [
    # rows, cols, dtype
    (512, 4096, F32),      # benchmark row: one tile of 256 threads x 4 vectors, exactly full
    (300, 4096, BF16),     # 512 vectors: 128 threads
    (65, 1000, F32),       # 250 vectors: ragged tile
    (33, 8, F32),          # two vectors
    (9, 20000, F32),       # 5000 vectors: two tiles of 1024 threads, carry, ragged second tile
    (5, 40000, BF16),      # 5000 vectors bf16
    (3, 131072, F32),      # 32768 vectors: eight full tiles
    (37, 1001, F32),       # scalar kernel (1001 % 4 != 0)
    (21, 1003, BF16),      # scalar kernel bf16
    (7, 1, F32),           # single column
    # short rows: 1, 2, 4, 8, 16 and 32 lanes of a warp per row; row counts that leave lanes without a row
    (1031, 16, F32), (515, 32, F32), (259, 64, BF16), (131, 136, BF16), (67, 256, F32), (35, 512, BF16),
    (19, 1024, BF16), (1025, 8, BF16), (77, 100, F32),
    (41, 1032, BF16), (13, 8192, BF16), (11, 16384, torch.float16), (9, 16392, BF16),   # a warp per row with a carry; just beyond it
    (4, 3, BF16),
]


@pytest.mark.parametrize("rows,cols,dtype", SCAN_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_cumsum_parity(kop, rows, cols, dtype, seed):
    x, mask = synth.cumsum_inputs(rows, cols, dtype, seed, "cuda")
    tol = tol_of(dtype)
    for use_mask in (False, True):
        for exclusive in (False, True):
            for reverse in (False, True):
                y = Guarded((rows, cols), dtype)
                kop.kop_cumsum_rows(x, mask if use_mask else None, exclusive, reverse, out=y.t)
                ref = kopref.cumsum_rows(host(x), host(mask) if use_mask else None, exclusive, reverse, threads=None)
                assert_scan_close(y.t, ref, tol, f"cumsum mask={use_mask} excl={exclusive} rev={reverse}")
                y.check("cumsum y")


def test_cumsum_full_config_seed0(kop):
    c = synth.CONFIGS["cumsum"]
    x, mask = synth.cumsum_inputs(c["rows"], c["cols"], c["dtype"], 0, "cuda")
    y = kop.kop_cumsum_rows(x)
    assert_scan_close(y, kopref.cumsum_rows(host(x), threads=None), 1e-5, "cumsum full")
    assert torch.equal(y, kop.kop_cumsum_rows(x))
    ym = kop.kop_cumsum_rows(x, mask, exclusive=True, reverse=True)
    assert_scan_close(ym, kopref.cumsum_rows(host(x), host(mask), True, True, threads=None), 1e-5, "cumsum full masked")


def test_cumsum_exact_integers(kop):
    """Small integers sum exactly in fp32 whatever the association: bit-exact against the closed forms."""
    n = 8192
    ones = torch.ones((3, n), dtype=F32, device="cuda")
    k = torch.arange(1, n + 1, dtype=F32, device="cuda")
    assert torch.equal(kop.kop_cumsum_rows(ones)[1], k)
    assert torch.equal(kop.kop_cumsum_rows(ones, exclusive=True)[2], k - 1)
    assert torch.equal(kop.kop_cumsum_rows(ones, reverse=True)[0], k.flip(0))
    assert torch.equal(kop.kop_cumsum_rows(ones, exclusive=True, reverse=True)[0], k.flip(0) - 1)
    ramp = torch.arange(1, 2049, dtype=F32, device="cuda").repeat(2, 1)          # triangular numbers < 2^24
    kk = torch.arange(1, 2049, dtype=torch.float64, device="cuda")
    assert torch.equal(kop.kop_cumsum_rows(ramp)[1].double(), kk * (kk + 1) / 2)
    odd = torch.ones((2, 1001), dtype=F32, device="cuda")                         # scalar kernel
    assert torch.equal(kop.kop_cumsum_rows(odd)[0], torch.arange(1, 1002, dtype=F32, device="cuda"))
    alt_mask = (torch.arange(n, device="cuda") % 2 == 0).repeat(3, 1)
    assert torch.equal(kop.kop_cumsum_rows(ones, alt_mask)[0], torch.div(torch.arange(n, device="cuda"), 2,
                                                                         rounding_mode="floor").float() + 1)


def test_cumsum_options(kop):
    rows, cols = 19, 2048
    x, mask = synth.cumsum_inputs(rows, cols, F32, 11, "cuda")
    ref = kopref.cumsum_rows(host(x))
    # in place
    xi = x.clone()
    kop.kop_cumsum_rows(xi, out=xi)
    assert_scan_close(xi, ref, 1e-5, "cumsum in place")
    xi = x.clone()
    kop.kop_cumsum_rows(xi, mask, True, True, out=xi)
    assert_scan_close(xi, kopref.cumsum_rows(host(x), host(mask), True, True), 1e-5, "cumsum in place masked")
    # strided rows (vector kernel: strides are multiples of four elements)
    big = torch.zeros((rows, cols + 64), dtype=F32, device="cuda")
    big[:, :cols] = x
    outb = torch.full((rows, cols + 32), 7.0, dtype=F32, device="cuda")
    kop.kop_cumsum_rows(big[:, :cols], out=outb[:, :cols])
    assert_scan_close(outb[:, :cols], ref, 1e-5, "cumsum strided")
    assert bool((outb[:, cols:] == 7.0).all())
    # misaligned base (4-byte but not 16-byte aligned): scalar kernel
    buf = torch.zeros(rows * cols + 1, dtype=F32, device="cuda")
    xo = buf[1:].view(rows, cols)
    xo.copy_(x)
    assert_scan_close(kop.kop_cumsum_rows(xo, reverse=True), kopref.cumsum_rows(host(x), reverse=True), 1e-5,
                      "cumsum misaligned base")
    # a mask whose row stride is odd forces the scalar kernel too
    mbig = torch.zeros((rows, cols + 1), dtype=torch.uint8, device="cuda")
    mbig[:, :cols] = mask
    assert_scan_close(kop.kop_cumsum_rows(x, mbig[:, :cols]), kopref.cumsum_rows(host(x), host(mask)), 1e-5,
                      "cumsum odd mask stride")
    # bool masks are accepted as they are
    assert torch.equal(kop.kop_cumsum_rows(x, mask.bool()), kop.kop_cumsum_rows(x, mask))
    # NaN / infinity: exactly the outputs whose sums include the element are affected; masked-out ones are not
    xn = x.clone()
    xn[2, 700] = float("nan")
    xn[3, 900] = float("inf")
    y = kop.kop_cumsum_rows(xn)
    assert not bool(torch.isnan(y[2, :700]).any()) and bool(torch.isnan(y[2, 700:]).all())
    assert bool(torch.isfinite(y[3, :900]).all()) and bool((y[3, 900:] == float("inf")).all())
    ye = kop.kop_cumsum_rows(xn, exclusive=True)
    assert not bool(torch.isnan(ye[2, :701]).any()) and bool(torch.isnan(ye[2, 701:]).all())
    yr = kop.kop_cumsum_rows(xn, reverse=True)
    assert bool(torch.isnan(yr[2, :701]).all()) and not bool(torch.isnan(yr[2, 701:]).any())
    m2 = torch.ones_like(mask)
    m2[2, 700] = 0
    m2[3, 900] = 0
    ym = kop.kop_cumsum_rows(xn, m2)
    assert bool(torch.isfinite(ym).all())
    x0 = x.clone()
    x0[2, 700] = 0
    x0[3, 900] = 0
    assert torch.equal(ym, kop.kop_cumsum_rows(x0))
    # empty
    e = torch.empty((0, cols), dtype=F32, device="cuda")
    assert kop.kop_cumsum_rows(e).shape == (0, cols)
