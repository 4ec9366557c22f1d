"""GPU parity of kop_groupnorm_act (GroupNorm / InstanceNorm with optional affine and activation)
against the float64 CPU oracle: five seeds over shapes that hit the register kernel (chunks up to 40 KB: teams of
8 lanes, of one warp and of several, every load width, units that straddle two channels), the
shared-memory-staged kernel (one and several parts, ragged last part, several waves of CTAs), the cluster and
two-sweep kernels (chunks beyond the staging budget) and the scalar kernel (long chunks that do not split into
16-byte vectors), all three activations, missing affine parameters, in-place use, misaligned bases, guard bands
and run-to-run bit equality.

Tolerance: |got - ref| <= tol * max(1, |ref|), tol = 1e-5 for fp32 data and 2e-2 for bf16 data;
the fp32 statistics are held to 1e-5 for both data types."""
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


GN_SHAPES = [
    # N, C, H, W, groups, dtype, act
    (4, 256, 56, 56, 32, F32, 2),      # benchmark chunk: 8 channels of 56x56, staged, 4 trips with a ragged last one
    (3, 64, 28, 28, 8, BF16, 2),       # staged bf16
    (2, 32, 56, 56, 32, F32, 0),       # InstanceNorm (groups == C)
    (2, 6, 40, 40, 1, F32, 1),         # groups == 1, chunk 38,400 B
    (2, 64, 64, 64, 2, F32, 2),        # chunk 512 KB: beyond one CTA's staging budget, a cluster of 8 CTAs
    (2, 128, 64, 64, 2, BF16, 1),      # chunk 1 MB bf16: beyond the cluster window, two sweeps
    (3, 8, 160, 160, 2, F32, 2),       # 400 KB: cluster of 7
    (2, 3, 290, 290, 1, BF16, 1),      # 493 KB, slices that do not divide evenly
    (1, 2, 600, 600, 1, F32, 0),       # one chunk of 2.9 MB: a cluster of 8 shares it, two sweeps
    (2, 12, 256, 256, 3, BF16, 2),     # six chunks of 512 KB bf16 (staged cluster); 1 MB fp32 below
    (2, 12, 256, 256, 3, F32, 1),      # six chunks of 1 MB: shared by clusters of 8, uneven slices
    (1, 6, 256, 256, 3, torch.float16, 2),   # 256 KB fp16: cluster of 4
    (3, 12, 7, 7, 4, F32, 2),          # plane 49, chunk of 147: 4-byte units
    (3, 12, 5, 6, 3, BF16, 0),         # plane 30 bf16: 16-byte units that straddle channels (30 % 8 != 0)
    (2, 8, 2, 2, 4, F32, 1),           # plane of one vector, chunk of two
    (5, 3, 1, 1, 3, F32, 0),           # one element per group: variance 0, y = beta
    (1, 16, 4, 4, 2, BF16, 2),
    (10, 256, 56, 56, 32, F32, 0),     # 320 chunks of 100 KB: more CTAs than fit the GPU at once
    (80, 64, 56, 56, 8, BF16, 1),      # 640 chunks of 50 KB
    # chunks held in registers: every team size and load width, the last CTA's idle teams
    (9, 37, 7, 7, 37, F32, 2),         # InstanceNorm 7 x 7: 49 units of 4 bytes, 8 lanes a chunk
    (5, 48, 14, 14, 48, BF16, 2),      # InstanceNorm 14 x 14 bf16: 49 units of 8 bytes
    (7, 30, 7, 7, 5, F32, 1),          # 6 channels of 49 a group: 8-byte units that straddle channels
    (3, 21, 5, 3, 7, torch.float16, 0),   # 45 elements: 2-byte units
    (11, 64, 4, 4, 32, BF16, 2),       # 2 channels of 16 a group: 4 units, two a lane
    (3, 16, 2, 2, 4, BF16, 2),         # plane of 4 bf16: the unit shrinks to 8 bytes to stay inside two channels
    (4, 6, 6, 6, 6, torch.float16, 1),    # 72 bytes a chunk: 8-byte units
    (2, 2048, 7, 7, 32, F32, 2),       # 64 channels of 49: 784 units of 16 bytes that straddle, four warps a chunk
    (3, 64, 14, 14, 4, BF16, 2),       # 16 channels of 14 x 14 bf16: 392 straddling units, two warps a chunk
    (5, 52, 14, 14, 13, F32, 1),       # 196 units: a warp a chunk, four chunks a CTA, 65 chunks (one idle team)
    (3, 40, 8, 8, 2, F32, 2),          # 320 units: three warps of four units a thread
    (7, 24, 10, 10, 12, BF16, 0),      # 25 units of 16 bytes: 8 lanes, four units a lane at most
    (3, 20, 32, 32, 2, F32, 2),        # 40 KB: ten warps a chunk, the longest register chunk
    (2, 22, 32, 32, 2, F32, 0),        # 44 KB: the first staged chunk
    (2, 256, 14, 14, 2, BF16, 2),      # 49 KB of planes that are not whole vectors: thirteen warps a chunk in registers
    (2, 330, 7, 7, 1, F32, 1),         # 63 KB, sixteen warps; one channel more would be the scalar kernel
    (2, 340, 7, 7, 1, F32, 1),         # 65 KB: the scalar kernel
    (6, 40, 7, 7, 1, F32, 0),          # groups == 1, chunk of 1960
]


@pytest.mark.parametrize("N,C,H,W,groups,dtype,act", GN_SHAPES)
@pytest.mark.parametrize("seed", SEEDS)
def test_groupnorm_parity(kop, N, C, H, W, groups, dtype, act, seed):
    x, gamma, beta = synth.groupnorm_inputs(N, C, H, W, dtype, seed, "cuda")
    eps = 1e-5
    y = Guarded((N, C, H, W), dtype)
    mean = Guarded((N, groups), F32)
    rstd = Guarded((N, groups), F32)
    kop.kop_groupnorm_act(x, gamma, beta, groups, eps, act, out=y.t, mean=mean.t, rstd=rstd.t)
    ry, rm, rr = kopref.groupnorm_act(host(x), host(gamma), host(beta), groups, eps, act, threads=None)
    tol = tol_of(dtype)
    assert_close(y.t, ry, tol, "groupnorm y")
    assert_close(mean.t, rm, 1e-5, "groupnorm mean")
    if H * W * (C // groups) > 1:
        assert_close(rstd.t, rr, 1e-5, "groupnorm rstd")
    else:
        # a single element: var = 0, rstd = eps^-1/2 = 316.2; relative comparison
        assert np.allclose(rstd.t.cpu().numpy(), rr, rtol=1e-5)
    if dtype == BF16:
        assert_bf16_tight(y.t, ry, "groupnorm y", floor=2e-3)
    y.check("groupnorm y")
    mean.check("groupnorm mean")
    rstd.check("groupnorm rstd")


def test_groupnorm_full_config_seed0(kop):
    c = synth.CONFIGS["groupnorm"]
    x, gamma, beta = synth.groupnorm_inputs(c["N"], c["C"], c["H"], c["W"], c["dtype"], 0, "cuda")
    y, m, r = kop.kop_groupnorm_act(x, gamma, beta, c["groups"], c["eps"], c["act"])
    ry, rm, rr = kopref.groupnorm_act(host(x), host(gamma), host(beta), c["groups"], c["eps"], c["act"], threads=None)
    assert_close(y, ry, 1e-5, "groupnorm full y")
    assert_close(m, rm, 1e-5, "groupnorm full mean")
    assert_close(r, rr, 1e-5, "groupnorm full rstd")
    y2, m2, r2 = kop.kop_groupnorm_act(x, gamma, beta, c["groups"], c["eps"], c["act"])
    assert torch.equal(y, y2) and torch.equal(m, m2) and torch.equal(r, r2)


def test_groupnorm_options(kop):
    N, C, H, W, G = 3, 32, 16, 16, 4
    x, gamma, beta = synth.groupnorm_inputs(N, C, H, W, F32, 7, "cuda")
    # no affine, no statistics
    y, m, r = kop.kop_groupnorm_act(x, None, None, G, 1e-5, 0, want_stats=False)
    assert m is None and r is None
    ry, _, _ = kopref.groupnorm_act(host(x), None, None, G, 1e-5, 0)
    assert_close(y, ry, 1e-5, "groupnorm no affine")
    # gamma only / beta only
    y, _, _ = kop.kop_groupnorm_act(x, gamma, None, G, 1e-5, 1)
    assert_close(y, kopref.groupnorm_act(host(x), host(gamma), None, G, 1e-5, 1)[0], 1e-5, "groupnorm gamma only")
    y, _, _ = kop.kop_groupnorm_act(x, None, beta, G, 1e-5, 2)
    assert_close(y, kopref.groupnorm_act(host(x), None, host(beta), G, 1e-5, 2)[0], 1e-5, "groupnorm beta only")
    # in place, staged and unstaged
    ry, rm, rr = kopref.groupnorm_act(host(x), host(gamma), host(beta), G, 1e-5, 2)
    xi = x.clone()
    kop.kop_groupnorm_act(xi, gamma, beta, G, 1e-5, 2, out=xi)
    assert_close(xi, ry, 1e-5, "groupnorm in place")
    xb, gb, bb = synth.groupnorm_inputs(1, 16, 128, 128, BF16, 3, "cuda")       # 2 groups of 256 KB
    rb = kopref.groupnorm_act(host(xb), host(gb), host(bb), 2, 1e-5, 2, threads=None)[0]
    kop.kop_groupnorm_act(xb, gb, bb, 2, 1e-5, 2, out=xb)
    assert_close(xb, rb, 2e-2, "groupnorm in place unstaged")
    # a base that is 4-byte but not 16-byte aligned: 4-byte units
    buf = torch.zeros(N * C * H * W + 1, dtype=F32, device="cuda")
    xo = buf[1:].view(N, C, H, W)
    xo.copy_(x)
    yo = torch.zeros(N * C * H * W + 1, dtype=F32, device="cuda")[1:].view(N, C, H, W)
    kop.kop_groupnorm_act(xo, gamma, beta, G, 1e-5, 2, out=yo)
    assert_close(yo, ry, 1e-5, "groupnorm misaligned base")
    # a bf16 base that is only 2-byte aligned (one-element units), short and long chunks
    for shp, grp in (((3, 8, 6, 6), 4), ((1, 4, 96, 96), 2)):
        xh, gh, bh = synth.groupnorm_inputs(*shp, BF16, 5, "cuda")
        n = xh.numel()
        xo = torch.zeros(n + 1, dtype=BF16, device="cuda")[1:].view(*shp)
        xo.copy_(xh)
        yo = torch.zeros(n + 1, dtype=BF16, device="cuda")[1:].view(*shp)
        kop.kop_groupnorm_act(xo, gh, bh, grp, 1e-5, 2, out=yo)
        assert_close(yo, kopref.groupnorm_act(host(xh), host(gh), host(bh), grp, 1e-5, 2, threads=None)[0], 2e-2,
                     "groupnorm bf16 misaligned base")
    # large offset, small spread: the one-sweep statistics must not lose the variance to cancellation
    xs = (x * 1e-2 + 100.0).contiguous()
    y, m, r = kop.kop_groupnorm_act(xs, gamma, beta, G, 1e-5, 0)
    ry2, rm2, rr2 = kopref.groupnorm_act(host(xs), host(gamma), host(beta), G, 1e-5, 0)
    assert_close(m, rm2, 1e-6, "groupnorm offset mean")
    assert np.allclose(r.cpu().numpy(), rr2, rtol=1e-4), "groupnorm offset rstd"
    assert_close(y, ry2, 2e-3, "groupnorm offset y (the fp32 mean's ulp at 100, times rstd = 100, dominates)")
    # constant input: variance exactly 0, y = beta
    xc = torch.full((2, 8, 8, 8), 3.25, dtype=F32, device="cuda")
    g8, b8 = gamma[:8].contiguous(), beta[:8].contiguous()
    y, m, r = kop.kop_groupnorm_act(xc, g8, b8, 2, 1e-5, 0)
    assert torch.equal(m, torch.full_like(m, 3.25))
    assert torch.equal(y, b8.view(1, 8, 1, 1).expand_as(y).contiguous())
    # NaN in one group poisons that group only; ReLU keeps it
    xn = x.clone()
    xn[1, 9, 3, 3] = float("nan")
    y, m, r = kop.kop_groupnorm_act(xn, gamma, beta, G, 1e-5, 1)
    cpg = C // G
    assert bool(torch.isnan(y[1, cpg:2 * cpg]).all()) and bool(torch.isnan(m[1, 1]))
    assert int(torch.isnan(m).sum()) == 1 and not bool(torch.isnan(y[0]).any()) and not bool(torch.isnan(y[1, :cpg]).any())
    # empty batch
    e = torch.empty((0, C, H, W), dtype=F32, device="cuda")
    ye, me, re_ = kop.kop_groupnorm_act(e, gamma, beta, G, 1e-5, 0)
    assert ye.shape == e.shape and me.shape == (0, G)
    # bad group count
    with pytest.raises(kop.KopError) as ei:
        kop.kop_groupnorm_act(x, gamma, beta, 5, 1e-5, 0)
    assert ei.value.status == 2


def test_groupnorm_no_copy_wait_ever_ran_out(kop):
    """Runs after the cases above in this module: the staged kernel's bounded waits all completed."""
    x, gamma, beta = synth.groupnorm_inputs(8, 64, 56, 56, F32, 1, "cuda")
    kop.kop_groupnorm_act(x, gamma, beta, 8, 1e-5, 2)
    assert kop.kop_groupnorm_wait_timeouts() == 0
