"""GPU parity of kop_gru_cell against the float64 CPU oracle: three data types, five seeds, every combination
of the two biases, vector and scalar paths, the state updated in place, saturated gates, NaN / infinity
behaviour, guard bands. Tolerance |got - ref| <= tol * max(1, |ref|), tol = 1e-5 (fp32), 2e-2 (bf16),
2e-3 (fp16)."""
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


@pytest.mark.parametrize("rows,hidden,dtype", [(256, 1024, BF16), (130, 1024, F32), (65, 520, F16), (33, 1001, F32),
                                               (9, 4100, BF16), (7, 1, F32), (1, 7, F16), (3, 6, BF16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_gru_cell_parity(kop, rows, hidden, dtype, seed):
    gi, gh, bi, bh, h_prev = synth.gru_inputs(rows, hidden, dtype, seed, "cuda")
    gi = gi * 2.0                                          # reach the saturated ends of the gates
    tol = tol_of(dtype)
    for use_bi in (True, False):
        for use_bh in (True, False):
            h = Guarded((rows, hidden), dtype)
            kop.kop_gru_cell(gi, gh, h_prev, bi if use_bi else None, bh if use_bh else None, h_out=h.t)
            ref = kopref.gru_cell(host(gi), host(gh), host(h_prev), host(bi) if use_bi else None,
                                  host(bh) if use_bh else None, threads=None)
            what = f"gru bias_i={use_bi} bias_h={use_bh}"
            assert_close(h.t, ref, tol, what)
            if dtype == BF16:
                assert_bf16_tight(h.t, ref, what)
            h.check(what)


def test_gru_cell_in_place_and_steps(kop):
    rows, hidden = 48, 768
    for dtype in (F32, BF16):
        gi, gh, bi, bh, h = synth.gru_inputs(rows, hidden, dtype, 5, "cuda")
        tol = tol_of(dtype)
        for step in range(4):
            gk = torch.roll(gi, step, 1).contiguous()
            before = host(h).clone()
            out = kop.kop_gru_cell(gk, gh, h, bi, bh, h_out=h)
            assert out is h
            assert_close(h, kopref.gru_cell(host(gk), host(gh), before, host(bi), host(bh)), tol, f"in-place step {step}")


def test_gru_cell_misaligned_takes_the_scalar_path(kop):
    rows, hidden = 12, 256
    gi, gh, bi, bh, h_prev = synth.gru_inputs(rows, hidden, F32, 3, "cuda")
    ref = kopref.gru_cell(host(gi), host(gh), host(h_prev), host(bi), host(bh))
    flat = torch.zeros(rows * 3 * hidden + 1, dtype=F32, device="cuda")
    flat[1:] = gh.reshape(-1)
    assert_close(kop.kop_gru_cell(gi, flat[1:].view(rows, 3 * hidden), h_prev, bi, bh), ref, 1e-5, "misaligned gh")
    flat_b = torch.zeros(3 * hidden + 1, dtype=F32, device="cuda")
    flat_b[1:] = bi
    assert_close(kop.kop_gru_cell(gi, gh, h_prev, flat_b[1:], bh), ref, 1e-5, "misaligned bias")


def test_gru_cell_special_values(kop):
    inf, nan = float("inf"), float("nan")
    #         gi: r    z    n      gh: r    z    n      h_prev
    cases = [((0.0, 0.0, 0.0), (0.0, 0.0, 0.0), 1.0),
             ((0.0, 100.0, 0.5), (0.0, 0.0, 0.5), 0.75),    # z = 1: keep h
             ((-100.0, -100.0, 0.3), (0.0, 0.0, 5.0), 9.0),  # r = 0, z = 0: tanh(gi_n)
             ((inf, -inf, 1.0), (0.0, 0.0, 1.0), 2.0),        # r = 1, z = 0: tanh(2)
             ((0.0, 0.0, nan), (0.0, 0.0, 0.0), 1.0),
             ((0.0, nan, 0.0), (0.0, 0.0, 0.0), 1.0),
             ((0.0, 0.0, 0.0), (0.0, 0.0, 0.0), nan),
             ((0.0, 0.0, inf), (0.0, 0.0, 0.0), 0.5)]
    hidden = 4
    gi = torch.zeros((len(cases), 3 * hidden), dtype=F32)
    gh = torch.zeros_like(gi)
    hp = torch.zeros((len(cases), hidden), dtype=F32)
    for r, (a, b, h0) in enumerate(cases):
        for k in range(3):
            gi[r, k * hidden:(k + 1) * hidden] = a[k]
            gh[r, k * hidden:(k + 1) * hidden] = b[k]
        hp[r] = h0
    ref = kopref.gru_cell(gi, gh, hp)
    got = kop.kop_gru_cell(gi.cuda(), gh.cuda(), hp.cuda()).cpu().double().numpy()
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.allclose(got[ok], ref[ok], rtol=1e-5, atol=1e-5)
    assert np.all(got[1] == 0.75)


def test_gru_cell_benchmark_shape_sampled_rows(kop):
    cfg = synth.CONFIGS["gru_cell"]
    rows, hidden, dtype = cfg["rows"], cfg["hidden"], cfg["dtype"]
    gi, gh, bi, bh, h_prev = synth.gru_inputs(rows, hidden, dtype, 0, "cuda")
    h = kop.kop_gru_cell(gi, gh, h_prev, bi, bh)
    idx = torch.tensor(sorted({0, 1, rows // 2, rows - 2, rows - 1} | set(np.random.default_rng(0).integers(0, rows, 59).tolist()))).cuda()
    ref = kopref.gru_cell(host(gi[idx]), host(gh[idx]), host(h_prev[idx]), host(bi), host(bh))
    assert_close(h[idx], ref, tol_of(dtype), "full-size sampled rows")
    assert bool(torch.isfinite(h.float()).all()) and float(h.float().abs().max()) <= 1.0
