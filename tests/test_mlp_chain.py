"""The chained transformer-MLP segment (RMSNorm -> vendor GEMM -> SiLU*up -> vendor GEMM -> residual)
against the pure-float64 oracle chain, checked with the paper's model-level rule (Gate 3): strict
comparison first, else the float64 disambiguation with an unfused same-dtype chain as the
baseline (rho = d_opt / d_ref <= 10, scale-relative check when the baseline is exact, absolute
escape bound). Also: per-kernel parity on the actual device intermediates, CUDA-graph capture of
the five-node segment, and the sampled-row check at the full benchmark shape."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import assert_close, to_f64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


@pytest.fixture(scope="module")
def handle(kop):
    h = kop.MlpHandle()
    yield h
    h.close()


def unfused_chain(h, w, W1, W2, eps):
    """The same chain with stock torch ops, one op at a time, rounding to the data dtype after
    each one: the baseline r_low of the Gate-3 rule (a comparator, not part of the product)."""
    dt = h.dtype
    hf = h.float()
    n = (hf * torch.rsqrt(hf.pow(2).mean(dim=1, keepdim=True) + eps) * w).to(dt)
    gu = n @ W1.t()
    inter = W1.shape[0] // 2
    act = (F.silu(gu[:, :inter].float()) * gu[:, inter:].float()).to(dt)
    d = act @ W2.t()
    return (hf + d.float()).to(dt)


def gate3(o, r64, r_low, tol):
    """Returns (passed, tier, d_opt, d_ref)."""
    o64, low64 = to_f64(o), to_f64(r_low)
    err = np.abs(o64 - r64)
    if np.all(err <= tol * np.maximum(1.0, np.abs(r64))):
        return True, "strict", float(err.max()), float(np.abs(low64 - r64).max())
    d_opt = float(err.max())
    d_ref = float(np.abs(low64 - r64).max())
    scale = float(np.abs(low64).max())
    if d_ref >= 1e-8:
        ok = d_opt / d_ref <= 10.0
        tier = "rho"
    else:
        ok = d_opt / max(scale, 1e-12) <= 1e-4
        tier = "scale-relative"
    if not ok and d_opt <= max(5e-3, 1e-3 * scale):
        ok, tier = True, "absolute"
    return ok, tier, d_opt, d_ref


@pytest.mark.parametrize("seed", synth.SEEDS)
@pytest.mark.parametrize("dtype", [BF16, F32])
def test_chain_reduced_shape(kop, handle, seed, dtype):
    M, H, I = 256, 512, 1792
    h, w, W1, W2 = synth.mlp_inputs(M, H, I, dtype, seed, "cuda")
    out = kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, 1e-6)
    r64 = kopref.mlp_segment(h.cpu(), w.cpu(), W1.cpu(), W2.cpu(), 1e-6, threads=None)
    r_low = unfused_chain(h, w, W1, W2, 1e-6)
    ok, tier, d_opt, d_ref = gate3(out, r64, r_low, 2e-2 if dtype == BF16 else 1e-5)
    assert ok, f"chain failed Gate 3 ({tier}): d_opt={d_opt:.3e} d_ref={d_ref:.3e}"
    # the fused chain must not be worse than a few times the unfused baseline in any case
    assert d_opt <= 10 * max(d_ref, 1e-6)


def test_chain_in_place_and_graph_capture(kop, handle):
    M, H, I = 512, 1024, 3584
    h, w, W1, W2 = synth.mlp_inputs(M, H, I, BF16, 0, "cuda")
    need = kop.kop_rmsnorm_swiglu_residual_workspace_bytes(M, H, I, kop.KOP_BF16)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    eager = kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, 1e-6, workspace=ws)
    torch.cuda.synchronize()
    out = torch.empty_like(h)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, 1e-6, out=out, workspace=ws)   # warm-up
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, 1e-6, out=out, workspace=ws)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    # out may be h itself
    hi = h.clone()
    kop.kop_rmsnorm_swiglu_residual(handle, hi, w, W1, W2, 1e-6, out=hi, workspace=ws)
    assert torch.equal(hi, eager)


def test_chain_full_shape_sampled_rows_and_intermediates(kop, handle):
    c = synth.CONFIGS["mlp"]
    M, H, I = c["rows"], c["hidden"], c["inter"]
    h, w, W1, W2 = synth.mlp_inputs(M, H, I, BF16, 0, "cuda")
    out = kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, c["eps"])
    idx = torch.from_numpy(np.sort(np.random.default_rng(1).choice(M, 16, replace=False))).to("cuda")
    hs = h[idx].contiguous()
    # rows are independent through the whole chain: the oracle runs the sampled rows only
    r64 = kopref.mlp_segment(hs.cpu(), w.cpu(), W1.cpu(), W2.cpu(), c["eps"], threads=None)
    r_low = unfused_chain(hs, w, W1, W2, c["eps"])
    ok, tier, d_opt, d_ref = gate3(out[idx], r64, r_low, 2e-2)
    assert ok, f"full-shape chain failed Gate 3 ({tier}): d_opt={d_opt:.3e} d_ref={d_ref:.3e}"
    # per-kernel parity on the actual device intermediates of the same chain
    n = kop.kop_rmsnorm(h, w, c["eps"])
    assert_close(n[idx], kopref.rmsnorm(hs.cpu(), w.cpu(), c["eps"]), 2e-2, "chain rmsnorm")
    gu = n @ W1.t()                                   # preserved vendor GEMM
    act = kop.kop_silu_mul(gu)
    assert_close(act[idx], kopref.silu_mul(gu[idx].cpu()), 2e-2, "chain silu_mul")
    d = act @ W2.t()
    res = kop.kop_residual_add(h, d)
    assert_close(res[idx], kopref.residual_add(hs.cpu(), d[idx].cpu()), 2e-2, "chain residual")
    # the driver and the piecewise chain run the same kernels around the same vendor GEMM
    diff = (out.float() - res.float()).abs()
    assert bool((diff <= 2e-2 * res.float().abs().clamp(min=1.0)).all()), "driver vs pieces"


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_chain_with_residual_in_the_gemm_epilogue(kop, dtype):
    """The vendor-library configuration (residual folded into the down projection through cuBLASLt):
    same Gate-3 rule against the float64 chain, at most one rounding away from the default form,
    capturable in a CUDA graph, in place, and switchable back."""
    M, H, I = 256, 512, 1792
    hdl = kop.MlpHandle()
    try:
        for seed in synth.SEEDS[:3]:
            h, w, W1, W2 = synth.mlp_inputs(M, H, I, dtype, seed, "cuda")
            hdl.set_residual_in_gemm(False)
            base = kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6)
            hdl.set_residual_in_gemm(True)
            out = kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6)
            r64 = kopref.mlp_segment(h.cpu(), w.cpu(), W1.cpu(), W2.cpu(), 1e-6, threads=None)
            r_low = unfused_chain(h, w, W1, W2, 1e-6)
            ok, tier, d_opt, d_ref = gate3(out, r64, r_low, 2e-2 if dtype == BF16 else 1e-5)
            assert ok, f"epilogue chain failed Gate 3 ({tier}): d_opt={d_opt:.3e} d_ref={d_ref:.3e}"
            # one rounding fewer than the default form: never further from the float64 chain than it, up to noise
            d_base = float(np.abs(to_f64(base) - r64).max())
            assert d_opt <= 1.5 * d_base + 1e-6
            step = 2.0 ** -7 if dtype == BF16 else 2.0 ** -20
            diff = (out.float() - base.float()).abs()
            assert bool((diff <= step * (1.0 + base.float().abs())).all()), "more than one rounding apart"
        # graph capture, replay, in place, and back to the default form
        ws = torch.empty(kop.kop_rmsnorm_swiglu_residual_workspace_bytes(M, H, I, kop.KOP_BF16 if dtype == BF16 else kop.KOP_F32),
                         dtype=torch.uint8, device="cuda")
        eager = kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6, workspace=ws)
        torch.cuda.synchronize()
        out = torch.empty_like(h)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6, out=out, workspace=ws)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6, out=out, workspace=ws)
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
        hdl.set_residual_in_gemm(False)
        assert torch.equal(kop.kop_rmsnorm_swiglu_residual(hdl, h, w, W1, W2, 1e-6, workspace=ws), base)
        # in place the default form is used whatever the setting
        hdl.set_residual_in_gemm(True)
        hi = h.clone()
        kop.kop_rmsnorm_swiglu_residual(hdl, hi, w, W1, W2, 1e-6, out=hi, workspace=ws)
        assert torch.equal(hi, base)
    finally:
        hdl.close()
