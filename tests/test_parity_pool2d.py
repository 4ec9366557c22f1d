"""GPU parity of kop_affine_relu_pool2d against the float64 CPU oracle: five seeds over max / average, with
and without the affine + ReLU prologue, the compile-time window shapes (3x3 s2, 2x2 s2, 3x3 s1) and generic
ones (rectangular, large, stride > kernel), planes that split into several bands, widths that are not whole
16-byte vectors (scalar staging and / or scalar stores), rows too wide for a shared-memory tile (direct
kernel), guard bands, NaN placement and run-to-run bit equality.

Tolerance: |got - ref| <= tol * max(1, |ref|), tol = 1e-5 for fp32 data and 2e-2 for bf16 data. Max pooling
of unmodified fp32 input must be bit-exact (it only selects)."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import Guarded, assert_bf16_tight, assert_close, tol_of

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


POOL_CASES = [
    # N, C, H, W, kernel, stride, padding, dtype
    (2, 8, 112, 112, (3, 3), (2, 2), (1, 1), F32),     # benchmark plane: two bands per plane
    (3, 5, 56, 56, (3, 3), (2, 2), (1, 1), BF16),
    (2, 6, 64, 64, (2, 2), (2, 2), (0, 0), F32),
    (2, 4, 32, 32, (3, 3), (1, 1), (1, 1), BF16),
    (2, 3, 224, 224, (3, 3), (2, 2), (1, 1), F32),     # eight bands per plane
    (2, 3, 30, 44, (5, 3), (2, 1), (2, 1), F32),       # rectangular generic window
    (2, 3, 17, 19, (3, 3), (2, 2), (1, 1), F32),       # odd sizes: scalar staging and scalar stores
    (2, 2, 16, 16, (2, 2), (3, 3), (0, 0), BF16),      # stride larger than the window
    (3, 4, 7, 7, (7, 7), (1, 1), (0, 0), F32),         # window = image (global pooling)
    (2, 2, 9, 8, (1, 1), (1, 1), (0, 0), BF16),        # identity window
    (1, 2, 6, 5000, (3, 3), (2, 2), (1, 1), F32),      # rows too wide for a tile: direct kernel
    # small planes: runs of planes per CTA, vectors crossing plane boundaries, a last run that ends inside a vector
    (5, 37, 7, 7, (3, 3), (2, 2), (1, 1), F32),
    (3, 50, 14, 14, (3, 3), (2, 2), (1, 1), BF16),
    (4, 9, 14, 14, (2, 2), (2, 2), (0, 0), torch.float16),
    (7, 11, 4, 4, (3, 3), (1, 1), (1, 1), F32),
    (2, 13, 28, 28, (3, 3), (2, 2), (1, 1), BF16),
    (3, 5, 5, 9, (2, 3), (1, 2), (1, 1), F32),         # generic window on a small plane
    (3, 3, 3, 3, (3, 3), (3, 3), (0, 0), BF16),        # 9-element planes
    (70, 64, 7, 7, (3, 3), (1, 1), (1, 1), BF16),      # several runs
    # stride-1 3x3 over whole 8-column segments: the register strip kernel (four bands; odd height, ragged last band)
    (2, 3, 56, 56, (3, 3), (1, 1), (1, 1), F32),
    (1, 2, 57, 64, (3, 3), (1, 1), (1, 1), BF16),
    (1, 1, 19, 8, (3, 3), (1, 1), (1, 1), torch.float16),          # one segment per row: both halos are padding
    # 2x2 / 3x3 at stride 1 / 2 out of a shared-memory tile: widths that are not whole segments or vectors, padding
    # in one direction only, a padded 2x2 window, one large plane in several bands, rows that start off a vector
    (2, 3, 60, 60, (3, 3), (2, 2), (1, 1), F32),
    (2, 3, 57, 57, (3, 3), (1, 1), (1, 1), BF16),
    (2, 3, 40, 44, (2, 2), (1, 1), (0, 0), F32),
    (2, 2, 33, 36, (3, 3), (1, 1), (1, 0), F32),
    (2, 2, 36, 33, (3, 3), (2, 2), (0, 1), BF16),
    (2, 2, 30, 30, (2, 2), (2, 2), (1, 1), torch.float16),
    (1, 1, 200, 204, (3, 3), (1, 1), (1, 1), F32),
    (1, 1, 301, 97, (3, 3), (2, 2), (1, 1), BF16),
    (3, 7, 28, 28, (3, 3), (1, 1), (1, 1), F32),                   # runs of whole small planes through the same kernel
    (5, 3, 23, 31, (2, 2), (1, 1), (0, 0), BF16),
    # 2x2 / stride 2 without padding, a thread per output: pair loads (even width), scalar loads (odd width), an odd
    # height (the last row is never read), one-output planes, a CTA's worth of outputs that ends inside a plane
    (5, 37, 14, 14, (2, 2), (2, 2), (0, 0), F32),
    (3, 50, 28, 28, (2, 2), (2, 2), (0, 0), BF16),
    (6, 11, 7, 7, (2, 2), (2, 2), (0, 0), F32),
    (2, 3, 57, 57, (2, 2), (2, 2), (0, 0), BF16),
    (3, 5, 15, 14, (2, 2), (2, 2), (0, 0), torch.float16),
    (9, 13, 2, 2, (2, 2), (2, 2), (0, 0), F32),
    (2, 3, 3, 2, (2, 2), (2, 2), (0, 0), BF16),
    (1, 2, 60, 60, (2, 2), (2, 2), (0, 0), F32),
    # widths that are a multiple of four: two adjacent outputs a thread (4 x 4 planes: one pair per output row)
    (3, 50, 28, 28, (2, 2), (2, 2), (0, 0), F32),
    (5, 7, 12, 20, (2, 2), (2, 2), (0, 0), torch.float16),
    (33, 17, 4, 4, (2, 2), (2, 2), (0, 0), BF16),
    (2, 3, 61, 60, (2, 2), (2, 2), (0, 0), BF16),
    # the window is the plane (global pooling): 16-, 8-, 4-byte and single-element loads, few and many lanes per plane
    (5, 37, 7, 7, (7, 7), (1, 1), (0, 0), F32),
    (5, 37, 7, 7, (7, 7), (7, 7), (0, 0), BF16),
    (3, 50, 14, 14, (14, 14), (1, 1), (0, 0), BF16),
    (2, 13, 28, 28, (28, 28), (1, 1), (0, 0), F32),
    (4, 9, 8, 8, (8, 8), (3, 3), (0, 0), torch.float16),
    (3, 5, 5, 9, (5, 9), (1, 1), (0, 0), BF16),
    (1, 2, 224, 224, (224, 224), (1, 1), (0, 0), F32),
    (70, 3, 2, 2, (2, 2), (1, 1), (0, 0), F32),
    (33, 7, 1, 1, (1, 1), (1, 1), (0, 0), BF16),
    # global pooling of planes that nothing wider than four bytes divides
    (2, 9, 9, 9, (9, 9), (1, 1), (0, 0), F32),
    (4, 6, 5, 5, (5, 5), (1, 1), (0, 0), torch.float16),
    (5, 2, 7, 7, (7, 7), (1, 1), (0, 0), BF16),
    (1, 3, 7, 7, (7, 7), (1, 1), (0, 0), F32),
    (3, 7, 9, 11, (9, 11), (1, 1), (0, 0), BF16),
    # 3 x 3 / stride 2 on rows that are not whole 8-column segments: the strip walk with aligned window loads, every
    # offset of a row from a 16-byte boundary (odd widths), a ragged last group of outputs, one band and several, a
    # bottom padding row (odd height with padding), planes from 256 elements
    (2, 3, 55, 55, (3, 3), (2, 2), (0, 0), F32),
    (3, 5, 27, 27, (3, 3), (2, 2), (0, 0), BF16),
    (1, 2, 147, 147, (3, 3), (2, 2), (0, 0), torch.float16),
    (2, 3, 35, 71, (3, 3), (2, 2), (0, 0), F32),
    (5, 7, 17, 17, (3, 3), (2, 2), (0, 0), BF16),
    (2, 2, 111, 109, (3, 3), (2, 2), (0, 0), BF16),
    (2, 3, 61, 60, (3, 3), (2, 2), (1, 1), F32),
    (3, 4, 30, 30, (3, 3), (2, 2), (1, 1), torch.float16),
    (2, 5, 16, 18, (3, 3), (2, 2), (1, 1), BF16),
    (2, 3, 57, 57, (3, 3), (2, 2), (1, 1), F32),                   # padded odd width: a padding column on the far side too
    (3, 2, 27, 33, (3, 3), (2, 2), (1, 1), BF16),
    (2, 3, 35, 35, (3, 3), (1, 1), (1, 1), F32),                   # stride 1 on odd widths: the same kernel
    (3, 5, 17, 17, (3, 3), (1, 1), (1, 1), BF16),
    (1, 2, 66, 57, (3, 3), (1, 1), (1, 1), torch.float16),
    # K x K windows at stride K without padding (K = 3, 4): a thread per output; sizes that leave unread rows / columns
    (2, 3, 113, 113, (3, 3), (3, 3), (0, 0), F32),
    (3, 5, 27, 28, (3, 3), (3, 3), (0, 0), BF16),
    (2, 4, 56, 56, (4, 4), (4, 4), (0, 0), torch.float16),
    (5, 7, 9, 10, (4, 4), (4, 4), (0, 0), F32),
    (1, 2, 256, 256, (3, 3), (3, 3), (0, 0), BF16),
    (70, 9, 4, 4, (4, 4), (4, 4), (0, 0), BF16),
]


@pytest.mark.parametrize("N,C,H,W,kernel,stride,padding,dtype", POOL_CASES)
@pytest.mark.parametrize("seed", SEEDS)
def test_pool2d_parity(kop, N, C, H, W, kernel, stride, padding, dtype, seed):
    x, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
    tol = tol_of(dtype)
    OH = (H + 2 * padding[0] - kernel[0]) // stride[0] + 1
    OW = (W + 2 * padding[1] - kernel[1]) // stride[1] + 1
    for mode in ("max", "avg"):
        for affine, relu in ((True, True), (False, False), (True, False)):
            sc, sf = (scale, shift) if affine else (None, None)
            y = Guarded((N, C, OH, OW), dtype)
            kop.kop_affine_relu_pool2d(x, sc, sf, kernel, stride, padding, mode, relu, out=y.t)
            ref = kopref.affine_relu_pool2d(host(x), host(sc), host(sf), kernel, stride, padding, mode, relu, threads=None)
            what = f"pool2d {mode} affine={affine} relu={relu}"
            assert_close(y.t, ref, tol, what)
            if dtype == BF16:
                assert_bf16_tight(y.t, ref, what, floor=1e-6)
            if mode == "max" and not affine:
                assert np.array_equal(y.t.cpu().to(torch.float64).numpy(), ref), what + " (selection is exact)"
            y.check(what)


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_pool2d_window_loads_at_the_tensor_ends(kop, dtype):
    """The aligned window loads of the any-width strip kernel where a whole 16-byte vector would cross the tensor's first
    or last byte: x starts one, two and three elements after a 16-byte boundary inside a larger buffer."""
    N, C, H, W = 2, 3, 33, 37
    x, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, 4, "cuda")
    ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), (3, 3), (2, 2), (0, 0), "max", True, threads=None)
    n = x.numel()
    for off in (1, 2, 3, 5):
        buf = torch.full((n + 16,), float("nan"), dtype=dtype, device="cuda")
        buf[off:off + n] = x.reshape(-1)
        y = Guarded((N, C, 16, 18), dtype)
        kop.kop_affine_relu_pool2d(buf[off:off + n].view(N, C, H, W), scale, shift, (3, 3), (2, 2), (0, 0), "max", True, out=y.t)
        assert_close(y.t, ref, tol_of(dtype), f"pool2d window loads, offset {off}")
        y.check("pool2d window loads")


def test_pool2d_full_config_seed0(kop):
    c = synth.CONFIGS["pool2d"]
    x, scale, shift = synth.bn_pool_inputs(c["N"], c["C"], c["H"], c["W"], c["dtype"], 0, "cuda")
    y = kop.kop_affine_relu_pool2d(x, scale, shift, c["kernel"], c["stride"], c["padding"], c["mode"], True)
    ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), c["kernel"], c["stride"], c["padding"],
                                    c["mode"], True, threads=None)
    assert_close(y, ref, 1e-5, "pool2d full")
    assert torch.equal(y, kop.kop_affine_relu_pool2d(x, scale, shift, c["kernel"], c["stride"], c["padding"], c["mode"], True))
    # a second GPU path for the same definition: the global-pool entry point equals a window covering the image
    xs = x[:4, :, :14, :14].contiguous()
    g = kop.kop_affine_relu_pool2d(xs, scale, shift, (14, 14), (1, 1), (0, 0), "avg", True)
    _, pooled = kop.kop_bn_relu_avgpool(xs, scale, shift)
    assert float((g[:, :, 0, 0] - pooled).abs().max()) < 1e-5


def test_pool2d_k2s2_unaligned_base(kop):
    """2x2 / stride 2 on a tensor that starts one element into its buffer: the pair loads are not aligned, the scalar
    loads take over; same results."""
    for dtype in (F32, BF16):
        x, scale, shift = synth.bn_pool_inputs(3, 5, 14, 14, dtype, 11, "cuda")
        buf = torch.empty(x.numel() + 1, dtype=dtype, device="cuda")
        xs = buf[1:].view(x.shape)
        xs.copy_(x)
        for mode in ("max", "avg"):
            a = kop.kop_affine_relu_pool2d(x, scale, shift, (2, 2), (2, 2), (0, 0), mode, True)
            b = kop.kop_affine_relu_pool2d(xs, scale, shift, (2, 2), (2, 2), (0, 0), mode, True)
            ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), (2, 2), (2, 2), (0, 0), mode, True)
            assert_close(a, ref, tol_of(dtype), f"k2s2 aligned {mode}")
            assert_close(b, ref, tol_of(dtype), f"k2s2 unaligned {mode}")
            assert torch.equal(a, b)


def test_pool2d_global_unaligned_and_nan(kop):
    """Global pooling on a tensor that starts one element into its buffer (narrower loads), and a NaN in one plane."""
    for dtype in (F32, BF16):
        x, scale, shift = synth.bn_pool_inputs(3, 5, 14, 14, dtype, 13, "cuda")
        buf = torch.empty(x.numel() + 1, dtype=dtype, device="cuda")
        xs = buf[1:].view(x.shape)
        xs.copy_(x)
        for mode in ("max", "avg"):
            a = kop.kop_affine_relu_pool2d(x, scale, shift, (14, 14), (1, 1), (0, 0), mode, True)
            b = kop.kop_affine_relu_pool2d(xs, scale, shift, (14, 14), (1, 1), (0, 0), mode, True)
            ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), (14, 14), (1, 1), (0, 0), mode, True)
            assert_close(a, ref, tol_of(dtype), f"global aligned {mode}")
            assert_close(b, ref, tol_of(dtype), f"global unaligned {mode}")
            if mode == "max":
                assert torch.equal(a, b)                       # a maximum does not depend on the order
    xn, scale, shift = synth.bn_pool_inputs(2, 4, 7, 7, F32, 3, "cuda")
    xn[1, 2, 3, 4] = float("nan")
    for mode in ("max", "avg"):
        y = kop.kop_affine_relu_pool2d(xn, scale, shift, (7, 7), (1, 1), (0, 0), mode, True)
        ref = kopref.affine_relu_pool2d(host(xn), host(scale), host(shift), (7, 7), (1, 1), (0, 0), mode, True)
        assert np.array_equal(np.isnan(y.cpu().numpy()), np.isnan(ref)) and np.isnan(ref).sum() == 1


def test_pool2d_options(kop):
    x, scale, shift = synth.bn_pool_inputs(2, 4, 20, 24, F32, 5, "cuda")
    # NaN poisons exactly the windows that contain it, in both modes
    xn = x.clone()
    xn[1, 2, 9, 13] = float("nan")
    for mode in ("max", "avg"):
        y = kop.kop_affine_relu_pool2d(xn, scale, shift, (3, 3), (2, 2), (1, 1), mode, True)
        ref = kopref.affine_relu_pool2d(host(xn), host(scale), host(shift), (3, 3), (2, 2), (1, 1), mode, True)
        assert np.array_equal(np.isnan(y.cpu().numpy()), np.isnan(ref)) and np.isnan(ref).sum() >= 1
    # all-negative input: padding (-inf) never wins a max; averages count the padding as zeros
    neg = -torch.rand((1, 2, 8, 8), device="cuda") - 1.0
    ym = kop.kop_affine_relu_pool2d(neg, None, None, (3, 3), (2, 2), (1, 1), "max", False)
    assert bool(torch.isfinite(ym).all()) and bool((ym <= -1.0).all())
    ones = torch.ones((1, 1, 4, 4), device="cuda")
    ya = kop.kop_affine_relu_pool2d(ones, None, None, (3, 3), (2, 2), (1, 1), "avg", False)
    assert abs(float(ya[0, 0, 0, 0]) - 4.0 / 9.0) < 1e-7 and abs(float(ya[0, 0, 1, 1]) - 1.0) < 1e-7
    # empty batch; bad geometry
    e = torch.empty((0, 4, 20, 24), dtype=F32, device="cuda")
    assert kop.kop_affine_relu_pool2d(e, scale, shift, (3, 3), (2, 2), (1, 1)).shape == (0, 4, 10, 12)
    with pytest.raises(kop.KopError) as ei:
        kop.kop_affine_relu_pool2d(x, scale, shift, (3, 3), (2, 2), (2, 2))       # padding > kernel / 2
    assert ei.value.status == 2
    with pytest.raises(kop.KopError) as ei:
        kop.kop_affine_relu_pool2d(x, scale, None, (3, 3), (2, 2), (1, 1))        # scale without shift
    assert ei.value.status == 1
