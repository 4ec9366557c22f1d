"""GPU parity of kop_lstm_cell against the float64 CPU oracle: three data types, five seeds, one or two gate
tensors, with and without bias, vector and scalar paths, the state updated in place, saturated gates, NaN /
infinity behaviour, guard bands. Tolerance |got - ref| <= tol * max(1, |ref|), tol = 1e-5 (fp32), 2e-2 (bf16),
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
                                               (9, 4100, BF16), (7, 1, F32), (1, 7, F16)])
@pytest.mark.parametrize("seed", SEEDS)
def test_lstm_cell_parity(kop, rows, hidden, dtype, seed):
    gates, gates2, bias, c_prev = synth.lstm_inputs(rows, hidden, dtype, seed, "cuda")
    gates = gates * 2.0                                    # reach the saturated ends of the gates
    tol = tol_of(dtype)
    for use_g2 in (True, False):
        for use_bias in (True, False):
            h = Guarded((rows, hidden), dtype)
            c = Guarded((rows, hidden), dtype)
            kop.kop_lstm_cell(gates, c_prev, gates2 if use_g2 else None, bias if use_bias else None, h_out=h.t, c_out=c.t)
            rh, rc = kopref.lstm_cell(host(gates), host(c_prev), host(gates2) if use_g2 else None,
                                      host(bias) if use_bias else None, threads=None)
            what = f"lstm g2={use_g2} bias={use_bias}"
            assert_close(h.t, rh, tol, what + " h")
            assert_close(c.t, rc, tol, what + " c")
            if dtype == BF16:
                assert_bf16_tight(h.t, rh, what + " h")
                assert_bf16_tight(c.t, rc, what + " c")
            h.check(what)
            c.check(what)


def test_lstm_cell_in_place_and_steps(kop):
    """Several steps with the state updated in place follow the oracle's step by step (each step's inputs
    are the product's own rounded outputs, so errors do not compound in the comparison)."""
    rows, hidden = 48, 768
    for dtype in (F32, BF16):
        gates, gates2, bias, c = synth.lstm_inputs(rows, hidden, dtype, 5, "cuda")
        tol = tol_of(dtype)
        for step in range(4):
            gk = torch.roll(gates, step, 1).contiguous()
            before = host(c).clone()
            h, c2 = kop.kop_lstm_cell(gk, c, gates2, bias, c_out=c)
            assert c2 is c
            rh, rc = kopref.lstm_cell(host(gk), before, host(gates2), host(bias))
            assert_close(c, rc, tol, f"in-place step {step} c")
            assert_close(h, rh, tol, f"in-place step {step} h")


def test_lstm_cell_misaligned_takes_the_scalar_path(kop):
    rows, hidden = 12, 256
    gates, gates2, bias, c_prev = synth.lstm_inputs(rows, hidden, F32, 3, "cuda")
    rh, rc = kopref.lstm_cell(host(gates), host(c_prev), host(gates2), host(bias))
    flat = torch.zeros(rows * 4 * hidden + 1, dtype=F32, device="cuda")
    flat[1:] = gates.reshape(-1)
    h, c = kop.kop_lstm_cell(flat[1:].view(rows, 4 * hidden), c_prev, gates2, bias)
    assert_close(h, rh, 1e-5, "misaligned gates h")
    assert_close(c, rc, 1e-5, "misaligned gates c")
    flat_c = torch.zeros(rows * hidden + 1, dtype=F32, device="cuda")
    h, c = kop.kop_lstm_cell(gates, c_prev, gates2, bias, c_out=flat_c[1:].view(rows, hidden))
    assert_close(h, rh, 1e-5, "misaligned c_out h")
    assert_close(c, rc, 1e-5, "misaligned c_out c")
    assert float(flat_c[0]) == 0.0


def test_lstm_cell_special_values(kop):
    inf, nan = float("inf"), float("nan")
    #            i     f     g     o
    cases = [((0.0, 0.0, 0.0, 0.0), 1.0),
             ((100.0, -100.0, 100.0, 100.0), 5.0),         # forget everything, write tanh(g) = 1
             ((-100.0, 100.0, 3.0, -100.0), 5.0),          # keep c, closed output gate: h = 0
             ((inf, inf, inf, inf), 2.0),
             ((-inf, -inf, -inf, -inf), 2.0),
             ((0.0, 0.0, nan, 0.0), 1.0),
             ((0.0, 0.0, 0.0, 0.0), nan),
             ((1.0, 100.0, 1.0, 1.0), 1e30)]
    hidden = 4
    g = torch.zeros((len(cases), 4 * hidden), dtype=F32)
    c = torch.zeros((len(cases), hidden), dtype=F32)
    for r, (a, cp) in enumerate(cases):
        for k in range(4):
            g[r, k * hidden:(k + 1) * hidden] = a[k]
        c[r] = cp
    rh, rc = kopref.lstm_cell(g, c)
    h, co = kop.kop_lstm_cell(g.cuda(), c.cuda())
    gh, gc = h.cpu().double().numpy(), co.cpu().double().numpy()
    assert np.array_equal(np.isnan(gh), np.isnan(rh)) and np.array_equal(np.isnan(gc), np.isnan(rc))
    ok = ~np.isnan(rh)
    assert np.allclose(gh[ok], rh[ok], rtol=1e-5, atol=1e-5) and np.allclose(gc[ok], rc[ok], rtol=1e-5, atol=1e-5)
    assert np.all(gh[2] == 0.0) and np.all(gc[1] == 1.0)


def test_lstm_cell_benchmark_shape_sampled_rows(kop):
    cfg = synth.CONFIGS["lstm_cell"]
    rows, hidden, dtype = cfg["rows"], cfg["hidden"], cfg["dtype"]
    gates, gates2, bias, c_prev = synth.lstm_inputs(rows, hidden, dtype, 0, "cuda")
    h, c = kop.kop_lstm_cell(gates, c_prev, gates2, bias)
    idx = torch.tensor(sorted({0, 1, rows // 2, rows - 2, rows - 1} | set(np.random.default_rng(0).integers(0, rows, 59).tolist())))
    rh, rc = kopref.lstm_cell(host(gates[idx.cuda()]), host(c_prev[idx.cuda()]), host(gates2[idx.cuda()]), host(bias))
    assert_close(h[idx.cuda()], rh, tol_of(dtype), "full-size sampled h")
    assert_close(c[idx.cuda()], rc, tol_of(dtype), "full-size sampled c")
    assert bool(torch.isfinite(h.float()).all()) and float(h.float().abs().max()) <= 1.0
