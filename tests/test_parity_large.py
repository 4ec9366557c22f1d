"""Tensors beyond 2^31 elements: element offsets must be 64-bit everywhere. One bf16 [70000, 32768] tensor
(2.29e9 elements, 4.6 GB) goes through several entry points; rows on both sides of the 2^31-element boundary
(row 65536) and the last rows are compared with the oracle computed on just those rows."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from tests._util import assert_close, to_f64

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16
ROWS, COLS = 70000, 32768
SAMPLE = [0, 1, 65535, 65536, 65537, 69998, 69999]


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def test_more_than_2_to_31_elements(kop):
    free, _ = torch.cuda.mem_get_info()
    if free < 24 << 30:
        pytest.skip("needs about 20 GB of free device memory")
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    x = torch.empty((ROWS, COLS), dtype=BF16, device="cuda")
    for r0 in range(0, ROWS, 10000):                       # generate in slabs: no fp32 temporary of the whole tensor
        r1 = min(ROWS, r0 + 10000)
        x[r0:r1] = torch.randn((r1 - r0, COLS), generator=g, device="cuda", dtype=torch.float32).to(BF16)
    assert x.numel() > 2 ** 31
    xs = x[SAMPLE].cpu()
    bias = torch.randn(COLS, generator=g, device="cuda", dtype=torch.float32) * 0.1
    # row reductions (read-only)
    v, i = kop.kop_reduce_rows(x, "max")
    rv, ri = kopref.reduce_rows(xs, "max", threads=None)
    assert np.array_equal(to_f64(v[SAMPLE]), rv) and np.array_equal(i[SAMPLE].cpu().numpy(), ri)
    v, _ = kop.kop_reduce_rows(x, "logsumexp")
    assert_close(v[SAMPLE], kopref.reduce_rows(xs, "logsumexp", threads=None)[0], 1e-5, "large logsumexp")
    # cross-entropy
    lab = torch.randint(0, COLS, (ROWS,), generator=g, device="cuda").to(torch.int32)
    loss, mean, bad = kop.kop_ce_loss_rowwise(x, lab)
    rl, _, _ = kopref.ce_loss_rowwise(xs, lab[SAMPLE].cpu(), threads=None)
    assert_close(loss[SAMPLE], rl, 2e-5, "large ce loss")
    assert int(bad) == 0 and abs(float(mean) - float(loss.double().mean())) < 1e-4
    # bias + activation into a second tensor, then residual add in place on it, then the running sum
    y = kop.kop_bias_act(x, bias, "silu")
    assert_close(y[SAMPLE], kopref.bias_act(xs, bias.cpu(), "silu", threads=None), 2e-2, "large bias_act")
    ys = y[SAMPLE].cpu()
    kop.kop_residual_add(x, y, out=y)
    assert_close(y[SAMPLE], kopref.residual_add(xs, ys, threads=None), 2e-2, "large residual add")
    del y
    torch.cuda.empty_cache()
    c = kop.kop_cumsum_rows(x, reverse=True)
    ref = kopref.cumsum_rows(xs, None, False, True, threads=None)
    got = to_f64(c[SAMPLE])
    assert np.all(np.abs(got - ref) <= 2e-2 * np.maximum(1.0, np.abs(ref).max(axis=1, keepdims=True))), "large cumsum"
    del c
    torch.cuda.empty_cache()
    # softmax in place (rows of 32768 bf16 elements take the multi-sweep kernel), RMSNorm into the same storage
    w = torch.randn(COLS, generator=g, device="cuda", dtype=torch.float32) * 0.02 + 1.0
    n = kop.kop_rmsnorm(x, w, 1e-6)
    assert_close(n[SAMPLE], kopref.rmsnorm(xs, w.cpu(), 1e-6, threads=None), 2e-2, "large rmsnorm")
    del n
    torch.cuda.empty_cache()
    kop.kop_softmax_scale_bias(x, bias, 0.5, out=x)
    assert_close(x[SAMPLE], kopref.softmax_scale_bias(xs, bias.cpu(), 0.5, threads=None), 2e-2, "large softmax in place")


def test_more_than_2_to_31_elements_ragged_rows(kop):
    """The same for rows that are not whole 16-byte vectors: bf16 [1100000, 1999] (2.2e9 elements): edge elements and
    aligned vectors of rows on both sides of the 2^31-element boundary (row 1074279), the span kernel's flat indices
    beyond 2^32 bytes, in-place softmax."""
    free, _ = torch.cuda.mem_get_info()
    if free < 16 << 30:
        pytest.skip("needs about 14 GB of free device memory")
    rows, cols = 1100000, 1999
    edge = (2 ** 31) // cols
    sample = [0, 1, 2, edge - 1, edge, edge + 1, rows - 2, rows - 1]
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    x = torch.empty((rows, cols), dtype=BF16, device="cuda")
    for r0 in range(0, rows, 100000):
        r1 = min(rows, r0 + 100000)
        x[r0:r1] = torch.randn((r1 - r0, cols), generator=g, device="cuda", dtype=torch.float32).to(BF16)
    assert x.numel() > 2 ** 31
    xs = x[sample].cpu()
    bias = torch.randn(cols, generator=g, device="cuda", dtype=torch.float32) * 0.1
    v, i = kop.kop_reduce_rows(x, "max")
    rv, ri = kopref.reduce_rows(xs, "max", threads=None)
    assert np.array_equal(to_f64(v[sample]), rv) and np.array_equal(i[sample].cpu().numpy(), ri)
    v, _ = kop.kop_reduce_rows(x, "sum")
    assert_close(v[sample], kopref.reduce_rows(xs, "sum", threads=None)[0], 1e-3, "large ragged sum")
    lab = torch.randint(0, cols, (rows,), generator=g, device="cuda").to(torch.int32)
    loss, mean, bad = kop.kop_ce_loss_rowwise(x, lab)
    rl, _, _ = kopref.ce_loss_rowwise(xs, lab[sample].cpu(), threads=None)
    assert_close(loss[sample], rl, 2e-5, "large ragged ce loss")
    assert int(bad) == 0 and abs(float(mean) - float(loss.double().mean())) < 1e-4
    y = kop.kop_bias_act(x, bias, "silu")
    assert_close(y[sample], kopref.bias_act(xs, bias.cpu(), "silu", threads=None), 2e-2, "large ragged bias_act")
    del y
    torch.cuda.empty_cache()
    kop.kop_softmax_scale_bias(x, bias, 0.5, out=x)
    assert_close(x[sample], kopref.softmax_scale_bias(xs, bias.cpu(), 0.5, threads=None), 2e-2, "large ragged softmax in place")


def test_more_than_2_to_31_elements_images(kop):
    free, _ = torch.cuda.mem_get_info()
    if free < 30 << 30:
        pytest.skip("needs about 25 GB of free device memory")
    N, C, H, W, G = 40, 512, 384, 384, 32
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    x = torch.empty((N, C, H, W), dtype=BF16, device="cuda")
    for n in range(N):
        x[n] = torch.randn((C, H, W), generator=g, device="cuda", dtype=torch.float32).to(BF16)
    assert x.numel() > 2 ** 31
    scale = torch.rand(C, generator=g, device="cuda") + 0.5
    shift = torch.randn(C, generator=g, device="cuda") * 0.1
    picks = [(0, 0), (28, 230), (29, 0), (39, 511)]            # element offsets on both sides of 2^31
    # BN + ReLU + global pool (planes are independent)
    y, p = kop.kop_bn_relu_avgpool(x, scale, shift)
    for n, c in picks:
        ry, rp = kopref.bn_relu_avgpool(x[n:n + 1, c:c + 1].cpu(), scale[c:c + 1].cpu(), shift[c:c + 1].cpu(), threads=None)
        assert_close(y[n:n + 1, c:c + 1], ry, 2e-2, f"large bn y {n},{c}")
        assert_close(p[n:n + 1, c:c + 1], rp, 1e-5, f"large bn pooled {n},{c}")
    del y
    torch.cuda.empty_cache()
    # windowed pooling (planes are independent)
    q = kop.kop_affine_relu_pool2d(x, scale, shift, (3, 3), (2, 2), (1, 1), "max", True)
    for n, c in picks:
        ref = kopref.affine_relu_pool2d(x[n:n + 1, c:c + 1].cpu(), scale[c:c + 1].cpu(), shift[c:c + 1].cpu(), (3, 3), (2, 2),
                                        (1, 1), "max", True, threads=None)
        assert_close(q[n:n + 1, c:c + 1], ref, 2e-2, f"large pool {n},{c}")
    del q
    torch.cuda.empty_cache()
    # GroupNorm: a group is C / G = 16 channels of one image
    gamma = torch.randn(C, generator=g, device="cuda") * 0.02 + 1.0
    beta = torch.randn(C, generator=g, device="cuda") * 0.02
    z, mu, rs = kop.kop_groupnorm_act(x, gamma, beta, G, 1e-5, 2)
    cpg = C // G
    for n, grp in [(0, 0), (28, 14), (29, 0), (39, 31)]:
        c0 = grp * cpg
        rz, rm, rr = kopref.groupnorm_act(x[n:n + 1, c0:c0 + cpg].cpu(), gamma[c0:c0 + cpg].cpu(), beta[c0:c0 + cpg].cpu(), 1,
                                          1e-5, 2, threads=None)
        assert_close(z[n:n + 1, c0:c0 + cpg], rz, 2e-2, f"large groupnorm {n},{grp}")
        assert_close(mu[n:n + 1, grp:grp + 1], rm, 1e-5, "large groupnorm mean")
        assert_close(rs[n:n + 1, grp:grp + 1], rr, 1e-5, "large groupnorm rstd")


def test_pool2d_k2s2_index_limits(kop):
    """The thread-per-output 2x2 / stride 2 kernel at the edge of what its multiply-shift divisions cover: just under
    2^24 planes of 4 x 4 (the largest quotient, 67 M outputs), sampled planes from both ends and the middle, and the
    same geometry with one plane too many, which must take another kernel and give the same values."""
    free, _ = torch.cuda.mem_get_info()
    if free < 6 << 30:
        pytest.skip("needs about 4 GB of free device memory")
    for N, C in ((256, 65535), (257, 65536)):                      # 16,776,960 planes (inside), 16,842,752 (outside)
        g = torch.Generator(device="cuda")
        g.manual_seed(5)
        x = torch.randn((N, C, 4, 4), generator=g, device="cuda", dtype=torch.float32)
        scale = torch.rand(C, generator=g, device="cuda") + 0.5
        shift = torch.randn(C, generator=g, device="cuda") * 0.1
        for mode in ("max", "avg"):
            y = kop.kop_affine_relu_pool2d(x, scale, shift, (2, 2), (2, 2), (0, 0), mode, True)
            for n, c in [(0, 0), (0, C - 1), (N // 2, 12345), (N - 1, 0), (N - 1, C - 1)]:
                ref = kopref.affine_relu_pool2d(x[n:n + 1, c:c + 1].cpu(), scale[c:c + 1].cpu(), shift[c:c + 1].cpu(), (2, 2),
                                                (2, 2), (0, 0), mode, True, threads=None)
                assert_close(y[n:n + 1, c:c + 1], ref, 1e-5, f"k2s2 limits {N}x{C} {mode} {n},{c}")
            # a whole contiguous block of planes at the far end against the oracle
            ref = kopref.affine_relu_pool2d(x[N - 1:, C - 4096:].cpu(), scale[C - 4096:].cpu(), shift[C - 4096:].cpu(), (2, 2),
                                            (2, 2), (0, 0), mode, True, threads=None)
            assert_close(y[N - 1:, C - 4096:], ref, 1e-5, f"k2s2 limits {N}x{C} {mode} last planes")
            del y
        del x
        torch.cuda.empty_cache()
