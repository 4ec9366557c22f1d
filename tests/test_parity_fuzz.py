"""Randomised GPU parity sweep: for every entry point, a few hundred small random shapes (seeded, so the
sweep is reproducible) with random dtypes, strides, alignments and options, each compared with the
float64 oracle under the usual rule |got - ref| <= tol * max(1, |ref|) (1e-5 fp32 data, 2e-2 bf16 data, 2e-3 fp16 data).
The hand-picked cases in the other parity files aim at known kernel boundaries; this sweep is for the
ones nobody thought of (odd lengths next to vector multiples, one-row and one-column tensors, sizes that
straddle the kernels' dispatch thresholds)."""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import assert_close, to_f64, tol_of

pytestmark = pytest.mark.gpu
F32, BF16, F16 = torch.float32, torch.bfloat16, torch.float16


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def host(t):
    return None if t is None else t.detach().cpu()


def pick_len(rng, hi):
    """Lengths biased towards the interesting neighbourhoods: tiny, around multiples of 4 / 8 / 32 / 256."""
    kind = rng.integers(0, 5)
    if kind == 0:
        return int(rng.integers(1, 12))
    if kind == 1:
        return int(min(hi, max(1, 8 * rng.integers(1, hi // 8 + 1) + rng.integers(-1, 2))))
    if kind == 2:
        return int(min(hi, max(1, 256 * rng.integers(1, max(2, hi // 256 + 1)) + rng.integers(-2, 3))))
    return int(rng.integers(1, hi + 1))


def strided(rng, t):
    """Sometimes re-home a 2-D tensor inside a wider buffer (row stride > cols) or at an odd offset."""
    mode = rng.integers(0, 4)
    rows, cols = t.shape
    if mode == 0:
        pad = int(rng.integers(1, 9)) * (8 if rng.integers(0, 2) else 1)
        big = torch.zeros((rows, cols + pad), dtype=t.dtype, device=t.device)
        big[:, :cols] = t
        return big[:, :cols]
    if mode == 1:
        flat = torch.zeros(rows * cols + 1, dtype=t.dtype, device=t.device)
        flat[1:] = t.reshape(-1)
        return flat[1:].view(rows, cols)
    return t


LN_ILL_CONDITIONED = 32.0      # rstd * max|gamma| above which a row's bound gets the conditioning term


def assert_close_ln(got, ref, rmean, rrstd, gamma, beta, tol, what):
    """LayerNorm outputs with the conditioning of the row taken into account. In fp32 the deviation v - mean carries
    an absolute error of about one ulp of max|v| (2^-24 * max|v|), which the normalisation multiplies by
    k = rstd * max|gamma|. With max|v| at most about 5 for these inputs the product stays below 1e-5 as long as
    k <= 32, so every such row is held to the plain rule. Only rows beyond that (a random two- or three-column row
    whose values differ by 1e-3 has rstd 300, and then no fp32 evaluation order reaches 1e-5) get the extra term
    8 ulp(fp32) * max|v| * k, with max|v| bounded from the oracle's own outputs."""
    g = to_f64(got)
    ga = gamma.detach().cpu().double().numpy()
    be = beta.detach().cpu().double().numpy()
    dev = np.abs((ref - be) / (rrstd[:, None] * np.where(ga == 0.0, 1.0, ga)))            # |v - mean| per element
    vmax = np.abs(rmean) + dev.max(axis=1)
    k = rrstd * np.abs(ga).max()
    extra = np.where(k > LN_ILL_CONDITIONED, 8.0 * 2.0 ** -24 * vmax * k, 0.0)
    err = np.abs(g - ref)
    bound = tol * np.maximum(1.0, np.abs(ref)) + extra[:, None]
    assert np.all(err <= bound), f"{what}: max err {err.max():.3e} (worst bound excess {np.max(err - bound):.3e})"


def test_fuzz_row_kernels(kop):
    rng = np.random.default_rng(2609_30059)
    for it in range(120):
        dtype = (F32, BF16, F16)[int(rng.integers(0, 3))]
        tol = tol_of(dtype)
        rows, cols = pick_len(rng, 70), pick_len(rng, 3000)
        seed = int(rng.integers(0, 1 << 30))
        what = f"it={it} rows={rows} cols={cols} {dtype}"
        # softmax
        x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
        xs = strided(rng, x)
        scale = float(rng.uniform(0.05, 2.0))
        use_bias = bool(rng.integers(0, 2))
        y = kop.kop_softmax_scale_bias(xs, bias if use_bias else None, scale)
        assert_close(y, kopref.softmax_scale_bias(host(x), host(bias) if use_bias else None, scale), tol, "softmax " + what)
        # bias + GELU + residual + LayerNorm and the plain / residual LayerNorm
        if cols >= 2:
            x, r, b, g, be = synth.layernorm_inputs(rows, cols, dtype, seed, "cuda")
            xs, rs_ = strided(rng, x), strided(rng, r)
            y, mu, rstd = kop.kop_bias_gelu_residual_layernorm(xs, rs_, b, g, be, 1e-5)
            ry, rm, rr = kopref.bias_gelu_residual_layernorm(host(x), host(r), host(b), host(g), host(be), 1e-5)
            assert_close_ln(y, ry, rm, rr, g, be, tol, "layernorm y " + what)
            assert_close(mu, rm, 1e-3, "layernorm mean " + what)
            with_res = bool(rng.integers(0, 2))
            y, mu, rstd = kop.kop_residual_layernorm(xs, rs_ if with_res else None, g, be, 1e-5)
            ry, rm, rr = kopref.residual_layernorm(host(x), host(r) if with_res else None, host(g), host(be), 1e-5)
            assert_close_ln(y, ry, rm, rr, g, be, tol, "residual layernorm y " + what)
        # RMSNorm
        h, w, _, _ = synth.mlp_inputs(rows, cols, 1, dtype, seed, "cuda")
        hs = strided(rng, h)
        assert_close(kop.kop_rmsnorm(hs, w, 1e-6), kopref.rmsnorm(host(h), host(w), 1e-6), tol, "rmsnorm " + what)
        # cross-entropy (plain and with options)
        z, lab = synth.ce_inputs(rows, cols, dtype, seed, "cuda")
        zs = strided(rng, z)
        loss, mean, bad = kop.kop_ce_loss_rowwise(zs, lab)
        rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab))
        assert_close(loss, rl, max(tol, 2e-5), "ce loss " + what)
        assert abs(float(mean) - rmean) <= max(tol, 2e-5) * max(1.0, abs(rmean)) and int(bad) == rbad, "ce mean " + what
        lab2 = lab.clone()
        lab2[rng.random(rows) < 0.3] = -100
        sm = float(rng.choice([0.0, 0.1, 0.3]))
        loss, mean, bad, cnt = kop.kop_ce_loss_rowwise_opts(zs, lab2, -100, sm)
        rl, rmean, rbad, rcnt = kopref.ce_loss_opts(host(z), host(lab2), -100, sm)
        assert_close(loss, rl, max(tol, 2e-5), "ce opts loss " + what)
        assert int(cnt) == rcnt and int(bad) == rbad, "ce opts counts " + what
        if rcnt > 0:
            assert abs(float(mean) - rmean) <= max(tol, 2e-5) * max(1.0, abs(rmean)), "ce opts mean " + what
        # SwiGLU epilogues, residual add, row scale, mat-vec
        gu = synth.gate_up_inputs(rows, cols, dtype, seed, "cuda")
        assert_close(kop.kop_silu_mul(strided(rng, gu)), kopref.silu_mul(host(gu)), tol, "silu_mul " + what)
        assert_close(kop.kop_silu_mul_interleaved(strided(rng, gu)), kopref.silu_mul_interleaved(host(gu)), tol,
                     "silu_mul_interleaved " + what)
        a, b2 = synth.pair_inputs(rows, cols, dtype, seed, "cuda")
        assert_close(kop.kop_residual_add(strided(rng, a), strided(rng, b2)), kopref.residual_add(host(a), host(b2)), tol,
                     "residual_add " + what)
        av, bm = synth.row_scale_inputs(rows, cols, dtype, seed, "cuda")
        assert_close(kop.kop_row_scale(av, strided(rng, bm)), kopref.row_scale(host(av), host(bm)), tol, "row_scale " + what)
        xv, wv, bs = synth.matvec_inputs(rows, cols, dtype, seed, "cuda")
        ref = kopref.matvec_bias(host(xv), host(wv), bs)
        got = to_f64(kop.kop_matvec_bias(strided(rng, xv), wv, bs))
        # fp32 accumulation of `cols` products against a float64 sum: scale by the sum of magnitudes
        mag = (host(xv).double().abs() @ host(wv).double().abs()).numpy() + abs(bs)
        assert np.all(np.abs(got - ref) <= 1e-5 * np.maximum(1.0, mag)), "matvec " + what
        # row reductions: extremes and their positions exactly, logsumexp to 1e-5
        xr = strided(rng, x)
        for op in ("max", "min"):
            v, i = kop.kop_reduce_rows(xr, op)
            rv, ri = kopref.reduce_rows(host(x), op)
            assert np.array_equal(to_f64(v), rv) and np.array_equal(i.cpu().numpy(), ri), f"reduce {op} " + what
        v, _ = kop.kop_reduce_rows(xr, "logsumexp")
        rv, _ = kopref.reduce_rows(host(x), "logsumexp")
        assert np.all(np.abs(to_f64(v) - rv) <= 1e-5 * np.maximum(1.0, np.abs(rv))), "reduce logsumexp " + what
        # bias + activation epilogue, a random activation
        act = ("identity", "relu", "leaky_relu", "gelu_tanh", "gelu_erf", "silu", "sigmoid", "tanh", "mish", "hardswish",
               "elu")[int(rng.integers(0, 11))]
        xa, ba = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
        assert_close(kop.kop_bias_act(strided(rng, xa), ba, act, alpha=0.3), kopref.bias_act(host(xa), host(ba), act, alpha=0.3),
                     tol, f"bias_act {act} " + what)
        # the same epilogue, the chain and the softmax with the bias stored in the data type (16-bit data only)
        if dtype != F32:
            b16 = ba.to(dtype)
            assert_close(kop.kop_bias_act_ex(strided(rng, xa), b16, act, alpha=0.3),
                         kopref.bias_act(host(xa), host(b16), act, alpha=0.3), tol, f"bias_act_ex {act} " + what)
            assert_close(kop.kop_epilogue_chain_ex(strided(rng, xa), b16, strided(rng, x), 0.75, 1.5, -2.0, 2.5, act, alpha=0.3),
                         kopref.epilogue_chain(host(xa), host(b16), host(x), 0.75, 1.5, -2.0, 2.5, act, alpha=0.3), tol,
                         f"epilogue_chain_ex {act} " + what)
            assert_close(kop.kop_softmax_ex(strided(rng, xa), b16, scale),
                         kopref.softmax_scale_bias(host(xa), host(b16), scale), tol, "softmax_ex " + what)
        # LSTM gate arithmetic (cols = hidden units, any length: vector and element kernels)
        hid = max(1, cols // 4)
        tg, tg2, tb, tc = synth.lstm_inputs(rows, hid, dtype, seed, "cuda")
        two, wb = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        gh, gc = kop.kop_lstm_cell(tg, tc, tg2 if two else None, tb if wb else None)
        rh, rc = kopref.lstm_cell(host(tg), host(tc), host(tg2) if two else None, host(tb) if wb else None)
        assert_close(gh, rh, tol, "lstm h " + what)
        assert_close(gc, rc, tol, "lstm c " + what)
        ui, uh, ubi, ubh, up = synth.gru_inputs(rows, hid, dtype, seed, "cuda")
        wi, wh = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        assert_close(kop.kop_gru_cell(ui, uh, up, ubi if wi else None, ubh if wh else None),
                     kopref.gru_cell(host(ui), host(uh), host(up), host(ubi) if wi else None, host(ubh) if wh else None),
                     tol, "gru " + what)
        # Lp normalisation of rows
        pn = int(rng.integers(1, 3))
        gy, gn = kop.kop_lp_normalize_rows(strided(rng, x), pn, 1e-12)
        ry, rn = kopref.lp_normalize_rows(host(x), pn, 1e-12)
        assert_close(gy, ry, tol, f"lp_normalize p={pn} " + what)
        assert np.all(np.abs(to_f64(gn) - rn) <= 1e-5 * np.maximum(1e-30, np.abs(rn))), "lp norms " + what
        # running sums
        xc, mask = synth.cumsum_inputs(rows, cols, dtype, seed, "cuda")
        ex, rv, um = bool(rng.integers(0, 2)), bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        got = to_f64(kop.kop_cumsum_rows(strided(rng, xc), mask if um else None, ex, rv))
        ref = kopref.cumsum_rows(host(xc), host(mask) if um else None, ex, rv)
        scale_rows = np.maximum(1.0, np.abs(ref).max(axis=1, keepdims=True))
        assert np.all(np.abs(got - ref) <= tol * scale_rows), "cumsum " + what


def test_fuzz_image_kernels(kop):
    rng = np.random.default_rng(30059_2609)
    for it in range(100):
        dtype = (F32, BF16, F16)[int(rng.integers(0, 3))]
        tol = tol_of(dtype)
        N, H, W = int(rng.integers(1, 5)), pick_len(rng, 40), pick_len(rng, 40)
        groups = int(rng.choice([1, 2, 3, 4, 8]))
        C = groups * int(rng.integers(1, 9))
        seed = int(rng.integers(0, 1 << 30))
        what = f"it={it} N={N} C={C} H={H} W={W} G={groups} {dtype}"
        x, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
        # BN + ReLU + global pool, NCHW and channels-last
        y, p = kop.kop_bn_relu_avgpool(x, scale, shift)
        ry, rp = kopref.bn_relu_avgpool(host(x), host(scale), host(shift))
        assert_close(y, ry, tol, "bn y " + what)
        assert_close(p, rp, 1e-5, "bn pooled " + what)
        xl = x.contiguous(memory_format=torch.channels_last)
        yl, pl = kop.kop_bn_relu_avgpool(xl, scale, shift)
        assert_close(yl, ry, tol, "bn nhwc y " + what)
        assert_close(pl, rp, 1e-5, "bn nhwc pooled " + what)
        # GroupNorm + activation
        xg, gamma, beta = synth.groupnorm_inputs(N, C, H, W, dtype, seed, "cuda")
        act = int(rng.integers(0, 3))
        aff = bool(rng.integers(0, 4))
        y, mu, rs = kop.kop_groupnorm_act(xg, gamma if aff else None, beta if aff else None, groups, 1e-5, act)
        ry, rm, rr = kopref.groupnorm_act(host(xg), host(gamma) if aff else None, host(beta) if aff else None, groups, 1e-5, act)
        assert_close(y, ry, tol, "groupnorm y " + what)
        assert_close(mu, rm, 1e-5, "groupnorm mean " + what)
        # windowed pooling with a random legal geometry
        kh, kw = int(rng.integers(1, min(H, 5) + 1)), int(rng.integers(1, min(W, 5) + 1))
        sh, sw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        ph, pw = int(rng.integers(0, kh // 2 + 1)), int(rng.integers(0, kw // 2 + 1))
        mode = "max" if rng.integers(0, 2) else "avg"
        aff, relu = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        y = kop.kop_affine_relu_pool2d(x, scale if aff else None, shift if aff else None, (kh, kw), (sh, sw), (ph, pw), mode, relu)
        ref = kopref.affine_relu_pool2d(host(x), host(scale) if aff else None, host(shift) if aff else None, (kh, kw),
                                        (sh, sw), (ph, pw), mode, relu)
        assert_close(y, ref, tol, f"pool2d k=({kh},{kw}) s=({sh},{sw}) p=({ph},{pw}) {mode} " + what)
        # the windows CNNs use (2 x 2 / 3 x 3, stride 1 / 2, pad 0 / 1) on larger planes: the strip and walk kernels,
        # widths that are and are not whole 8-column segments
        Hb = int(rng.choice([16, 24, 33, 40, 57, 64]))
        Wb = int(rng.choice([16, 24, 30, 33, 40, 56, 60, 63, 64, 72]))
        k = int(rng.integers(2, 4))
        st = int(rng.integers(1, 3))
        pd = (int(rng.integers(0, 2)), int(rng.integers(0, 2)))
        xb, scb, shb = synth.bn_pool_inputs(int(rng.integers(1, 3)), int(rng.integers(1, 5)), Hb, Wb, dtype, seed, "cuda")
        y = kop.kop_affine_relu_pool2d(xb, scb if aff else None, shb if aff else None, (k, k), (st, st), pd, mode, relu)
        ref = kopref.affine_relu_pool2d(host(xb), host(scb) if aff else None, host(shb) if aff else None, (k, k), (st, st),
                                        pd, mode, relu)
        assert_close(y, ref, tol, f"pool2d {Hb}x{Wb} k={k} s={st} p={pd} {mode} " + what)
        # 16-bit data: folded BatchNorm coefficients and GroupNorm weights stored in the data type
        if dtype != F32:
            s16, h16 = scale.to(dtype), shift.to(dtype)
            y, p = kop.kop_bn_relu_avgpool_ex(xl if rng.integers(0, 2) else x, s16, h16)
            ry, rp = kopref.bn_relu_avgpool(host(x), host(s16), host(h16))
            assert_close(y, ry, tol, "bn_ex y " + what)
            assert_close(p, rp, 1e-5, "bn_ex pooled " + what)
            g16, be16 = gamma.to(dtype), beta.to(dtype)
            y, _, _ = kop.kop_groupnorm_act_ex(xg, g16, be16, groups, 1e-5, act)
            assert_close(y, kopref.groupnorm_act(host(xg), host(g16), host(be16), groups, 1e-5, act)[0], tol, "groupnorm_ex y " + what)
    assert kop.kop_groupnorm_wait_timeouts() == 0


def rehome(rng, t, off, pad):
    """A copy of the 2-D tensor t whose first element sits `off` elements after a 16-byte boundary and whose rows are
    `pad` elements apart beyond their length (pad = 0: contiguous); surrounded by NaN so that a stray read shows."""
    rows, cols = t.shape
    stride = cols + pad
    buf = torch.full((rows * stride + 32,), float("nan"), dtype=t.dtype, device=t.device)
    view = buf[off:off + rows * stride].view(rows, stride)[:, :cols]
    view.copy_(t)
    return view


def test_fuzz_rows_off_the_vector_grid(kop):
    """Rows that are not whole aligned 16-byte vectors, input and output at the same random offset from a boundary and
    with the same random row pitch (the head / vectors / tail split of the softmax, cross-entropy, reduction and
    bias + activation kernels), in place as well; nothing outside the output rows may change."""
    rng = np.random.default_rng(197_50257)
    for it in range(150):
        dtype = (F32, BF16, F16)[int(rng.integers(0, 3))]
        tol = tol_of(dtype)
        rows = pick_len(rng, 40)
        cols = pick_len(rng, 2600) if rng.integers(0, 4) else int(rng.integers(8000, 20000))
        off = int(rng.integers(0, 8))
        pad = int(rng.integers(0, 2)) * int(rng.integers(1, 12))
        seed = int(rng.integers(0, 1 << 30))
        what = f"it={it} rows={rows} cols={cols} off={off} pad={pad} {dtype}"
        x, bias = synth.softmax_inputs(rows, cols, dtype, seed, "cuda")
        xs = rehome(rng, x, off, pad)
        use_bias = bool(rng.integers(0, 2))
        b, hb = (bias, host(bias)) if use_bias else (None, None)
        log_out = bool(rng.integers(0, 2))
        out = rehome(rng, torch.full_like(x, 7.0), off, pad)
        frame = out.untyped_storage()                       # the whole buffer, to check the pitch gaps afterwards
        kop.kop_softmax_opts(xs, b, 0.5, log_out, 0, out=out)
        ref = kopref.softmax_opts(host(x), hb, 0.5, log_out, 0)
        assert_close(out, ref, tol, "softmax " + what)
        if pad:
            gaps = torch.empty(0, dtype=dtype, device="cuda").set_(frame)[off:off + rows * (cols + pad)].view(rows, cols + pad)[:, cols:]
            assert bool(torch.isnan(gaps).all()), "softmax wrote between rows " + what
        xi = rehome(rng, x, off, pad)
        kop.kop_softmax_scale_bias(xi, b, 0.5, out=xi)
        assert_close(xi, kopref.softmax_scale_bias(host(x), hb, 0.5), tol, "softmax in place " + what)
        # reductions and cross-entropy read only
        op = ("sum", "max", "min", "logsumexp", "mean")[int(rng.integers(0, 5))]
        v, i = kop.kop_reduce_rows(xs, op)
        rv, ri = kopref.reduce_rows(host(x), op)
        if op in ("max", "min"):
            assert np.array_equal(to_f64(v), rv) and np.array_equal(i.cpu().numpy(), ri), f"reduce {op} " + what
        else:
            mag = np.maximum(1.0, host(x).double().abs().sum(dim=1).numpy()) / (cols if op == "mean" else 1.0)
            bound = 1e-5 * (mag if op != "logsumexp" else np.maximum(1.0, np.abs(rv)))
            assert np.all(np.abs(to_f64(v) - rv) <= bound), f"reduce {op} " + what
        z, lab = synth.ce_inputs(rows, cols, dtype, seed, "cuda")
        loss, mean, bad = kop.kop_ce_loss_rowwise(rehome(rng, z, off, pad), lab)
        rl, rmean, rbad = kopref.ce_loss_rowwise(host(z), host(lab))
        assert_close(loss, rl, max(tol, 2e-5), "ce loss " + what)
        # bias + activation and the chain: contiguous tensors take the span kernel, pitched ones the element-wise one
        act = ("silu", "gelu_tanh", "relu", "tanh")[int(rng.integers(0, 4))]
        out = rehome(rng, torch.full_like(x, 7.0), off, pad)
        kop.kop_bias_act(xs, b, act, out=out)
        assert_close(out, kopref.bias_act(host(x), hb, act), tol, f"bias_act {act} " + what)
        r, _ = synth.softmax_inputs(rows, cols, dtype, seed + 1, "cuda")
        rs_ = rehome(rng, r, off, pad)
        kop.kop_epilogue_chain(xs, b, rs_, 0.7, 1.5, -1.0, 2.0, act, out=rs_)
        assert_close(rs_, kopref.epilogue_chain(host(x), hb, host(r), 0.7, 1.5, -1.0, 2.0, act), tol, f"chain {act} " + what)


def test_fuzz_images_off_the_vector_grid(kop):
    """GroupNorm chunks in registers and the any-width pooling strips on tensors whose first element sits at a random offset
    from a 16-byte boundary, input and output alike."""
    rng = np.random.default_rng(55_27_13)
    for it in range(80):
        dtype = (F32, BF16, F16)[int(rng.integers(0, 3))]
        tol = tol_of(dtype)
        N, H, W = int(rng.integers(1, 4)), int(rng.integers(3, 60)), int(rng.integers(3, 60))
        groups = int(rng.choice([1, 2, 4, 8]))
        C = groups * int(rng.integers(1, 7))
        off = int(rng.integers(0, 8))
        seed = int(rng.integers(0, 1 << 30))
        what = f"it={it} N={N} C={C} H={H} W={W} G={groups} off={off} {dtype}"
        x, gamma, beta = synth.groupnorm_inputs(N, C, H, W, dtype, seed, "cuda")
        n = x.numel()
        xb = torch.full((n + 32,), float("nan"), dtype=dtype, device="cuda")
        xb[off:off + n] = x.reshape(-1)
        xv = xb[off:off + n].view(N, C, H, W)
        yb = torch.full((n + 32,), 5.0, dtype=dtype, device="cuda")
        yv = yb[off:off + n].view(N, C, H, W)
        act = int(rng.integers(0, 3))
        kop.kop_groupnorm_act(xv, gamma, beta, groups, 1e-5, act, out=yv)
        ry, rm, rr = kopref.groupnorm_act(host(x), host(gamma), host(beta), groups, 1e-5, act)
        assert_close(yv, ry, tol, "groupnorm " + what)
        assert bool((yb[:off] == 5.0).all()) and bool((yb[off + n:] == 5.0).all()), "groupnorm wrote outside " + what
        st = int(rng.integers(1, 3))
        pd = int(rng.integers(0, 2))
        if H + 2 * pd >= 3 and W + 2 * pd >= 3:
            _, scale, shift = synth.bn_pool_inputs(N, C, H, W, dtype, seed, "cuda")
            mode = "max" if rng.integers(0, 2) else "avg"
            y = kop.kop_affine_relu_pool2d(xv, scale, shift, (3, 3), (st, st), (pd, pd), mode, True)
            ref = kopref.affine_relu_pool2d(host(x), host(scale), host(shift), (3, 3), (st, st), (pd, pd), mode, True)
            assert_close(y, ref, tol, f"pool2d 3x3 s={st} p={pd} {mode} " + what)
