"""ctypes front end of the float64 CPU oracle (oracle/kopref.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's cpu_baseline / reference legs. The product package never imports it,
and this module imports nothing from the product package.

Data tensors may be numpy arrays (float32, float64, float16, or uint16 holding bf16
bit patterns) or CPU torch tensors (float32, float64, bfloat16, float16); they must be
contiguous in their last dimension. Every result is a float64 numpy array.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

F32, BF16, F64, F16 = 0, 1, 2, 3
_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        i64, dbl, vp = C.c_int64, C.c_double, C.c_void_p
        _lib.kopref_bf16_to_f64.restype = dbl
        _lib.kopref_bf16_to_f64.argtypes = [C.c_uint16]
        _lib.kopref_f16_to_f64.restype = dbl
        _lib.kopref_f16_to_f64.argtypes = [C.c_uint16]
        _lib.kopref_f64_to_bf16_rne.restype = C.c_uint16
        _lib.kopref_f64_to_bf16_rne.argtypes = [dbl]
        _lib.kopref_gelu_tanh.restype = dbl
        _lib.kopref_gelu_tanh.argtypes = [dbl]
        _lib.kopref_softmax_scale_bias.argtypes = [vp, vp, vp, i64, i64, i64, i64, dbl, C.c_int, C.c_int]
        _lib.kopref_bias_gelu_residual_layernorm.argtypes = [vp] * 8 + [i64] * 5 + [dbl, C.c_int, C.c_int]
        _lib.kopref_bias_erfgelu_residual_layernorm.argtypes = [vp] * 8 + [i64] * 5 + [dbl, C.c_int, C.c_int]
        _lib.kopref_gelu_erf.restype = dbl
        _lib.kopref_gelu_erf.argtypes = [dbl]
        _lib.kopref_bn_relu_avgpool.argtypes = [vp] * 5 + [i64] * 4 + [C.c_int, C.c_int]
        _lib.kopref_ce_loss_rowwise.argtypes = [vp] * 5 + [i64] * 3 + [C.c_int, C.c_int]
        _lib.kopref_rmsnorm.argtypes = [vp] * 3 + [i64] * 4 + [dbl, C.c_int, C.c_int]
        _lib.kopref_silu_mul.argtypes = [vp] * 2 + [i64] * 4 + [C.c_int, C.c_int]
        _lib.kopref_residual_add.argtypes = [vp] * 3 + [i64] * 5 + [C.c_int, C.c_int]
        _lib.kopref_gemm_nt.argtypes = [vp, C.c_int, vp, C.c_int, vp, i64, i64, i64, C.c_int]
        _lib.kopref_residual_layernorm.argtypes = [vp] * 7 + [i64] * 5 + [dbl, C.c_int, C.c_int]
        _lib.kopref_silu_mul_interleaved.argtypes = [vp] * 2 + [i64] * 4 + [C.c_int, C.c_int]
        _lib.kopref_ce_loss_opts.argtypes = [vp] * 6 + [i64] * 3 + [C.c_int32, dbl, C.c_int, C.c_int]
        _lib.kopref_ce_loss_sum.argtypes = [vp] * 4 + [i64] * 3 + [C.c_int32, dbl, C.c_int, C.c_int]
        _lib.kopref_groupnorm_act.argtypes = [vp] * 6 + [i64] * 5 + [dbl, C.c_int, C.c_int, C.c_int]
        _lib.kopref_row_scale.argtypes = [vp, vp, vp, i64, i64, i64, i64, C.c_int, C.c_int]
        _lib.kopref_affine_relu_pool2d.argtypes = [vp] * 4 + [i64] * 4 + [C.c_int] * 10
        _lib.kopref_reduce_rows.argtypes = [vp, vp, vp, i64, i64, i64, C.c_int, C.c_int, C.c_int]
        _lib.kopref_bias_act.argtypes = [vp, vp, vp, i64, i64, i64, i64, C.c_int, dbl, C.c_int, C.c_int]
        _lib.kopref_act_value.restype = dbl
        _lib.kopref_act_value.argtypes = [dbl, C.c_int, dbl]
        _lib.kopref_softmax_opts.argtypes = [vp, vp, vp, i64, i64, i64, i64, dbl, C.c_int, i64, C.c_int, C.c_int]
        _lib.kopref_epilogue_chain.argtypes = [vp, vp, vp, vp] + [i64] * 5 + [dbl] * 4 + [C.c_int, dbl, C.c_int, C.c_int]
        _lib.kopref_lstm_cell.argtypes = [vp] * 6 + [i64, i64, C.c_int, C.c_int]
        _lib.kopref_gru_cell.argtypes = [vp] * 6 + [i64, i64, C.c_int, C.c_int]
        _lib.kopref_lp_normalize_rows.argtypes = [vp, vp, vp, i64, i64, i64, i64, C.c_int, C.c_double, C.c_int, C.c_int]
        _lib.kopref_cumsum_rows.argtypes = [vp, vp, vp] + [i64] * 5 + [C.c_int] * 4
        _lib.kopref_matvec_bias.argtypes = [vp, vp, dbl, vp, i64, i64, i64, C.c_int, C.c_int]
    return _lib


def host_threads() -> int:
    """Host cores this process may use (what `threads=None` resolves to)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


def _nt(threads) -> int:
    return host_threads() if threads is None else int(threads)


def as_data(a):
    """Return (numpy array, dtype tag) for a data tensor without changing any bit."""
    if hasattr(a, "detach"):  # torch tensor
        import torch
        a = a.detach()
        assert a.device.type == "cpu", "oracle inputs live on the host"
        if a.dtype == torch.bfloat16:
            return a.contiguous().view(torch.int16).numpy().view(np.uint16), BF16
        if a.dtype == torch.float16:
            return a.contiguous().view(torch.int16).numpy().view(np.uint16), F16
        a = a.contiguous().numpy()
    a = np.asarray(a)
    if a.dtype == np.float32:
        return np.ascontiguousarray(a), F32
    if a.dtype == np.uint16:
        return np.ascontiguousarray(a), BF16
    if a.dtype == np.float16:
        return np.ascontiguousarray(a).view(np.uint16), F16
    if a.dtype == np.float64:
        return np.ascontiguousarray(a), F64
    raise TypeError(f"unsupported oracle data dtype {a.dtype}")


def as_param(a):
    """Parameter vector as a contiguous fp32 numpy array (None stays None). fp32 input is taken as is; a
    bf16 / fp16 torch tensor (parameters stored in the data type) is widened to fp32, which is exact: every
    value of either 16-bit format is an fp32 value."""
    if a is None:
        return None
    if hasattr(a, "detach"):
        a = a.detach().cpu()
        if str(a.dtype) in ("torch.bfloat16", "torch.float16"):
            a = a.float()
        a = a.numpy()
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float32, "parameter vectors are fp32, or 16-bit torch tensors"
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc, name):
    if rc != 0:
        raise ValueError(f"{name}: bad argument (rc={rc})")


def bf16_to_f64(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    f = lib().kopref_bf16_to_f64
    return np.array([f(int(b)) for b in bits.ravel()], dtype=np.float64).reshape(bits.shape)


def f16_to_f64(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    f = lib().kopref_f16_to_f64
    return np.array([f(int(b)) for b in bits.ravel()], dtype=np.float64).reshape(bits.shape)


def f64_to_bf16_rne(v) -> np.ndarray:
    v = np.asarray(v, dtype=np.float64)
    f = lib().kopref_f64_to_bf16_rne
    return np.array([f(float(t)) for t in v.ravel()], dtype=np.uint16).reshape(v.shape)


def gelu_tanh(u: float) -> float:
    return lib().kopref_gelu_tanh(float(u))


def softmax_scale_bias(x, bias, scale, threads=1) -> np.ndarray:
    xa, dt = as_data(x)
    rows, cols = xa.shape
    b = as_param(bias)
    y = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_softmax_scale_bias(_p(xa), _p(b), _p(y), rows, cols, cols, cols,
                                           float(scale), dt, _nt(threads)), "softmax_scale_bias")
    return y


def gelu_erf(u: float) -> float:
    return lib().kopref_gelu_erf(float(u))


def softmax_opts(x, bias, scale, log_output=False, causal_period=0, threads=1) -> np.ndarray:
    """Softmax or log-softmax of x * scale + bias per row, optionally causal (see kopref_softmax_opts)."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    b = as_param(bias)
    y = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_softmax_opts(_p(xa), _p(b), _p(y), rows, cols, cols, cols, float(scale), int(bool(log_output)),
                                     int(causal_period), dt, _nt(threads)), "softmax_opts")
    return y


def bias_gelu_residual_layernorm(x, residual, bias, gamma, beta, eps, threads=1, erf_form=False):
    """Returns (y, mean, rstd). erf_form: the error-function GELU instead of the tanh form."""
    xa, dt = as_data(x)
    ra, dt2 = as_data(residual)
    assert dt == dt2 and xa.shape == ra.shape
    rows, hidden = xa.shape
    b, g, be = as_param(bias), as_param(gamma), as_param(beta)
    y = np.empty((rows, hidden), dtype=np.float64)
    mean = np.empty(rows, dtype=np.float64)
    rstd = np.empty(rows, dtype=np.float64)
    fn = lib().kopref_bias_erfgelu_residual_layernorm if erf_form else lib().kopref_bias_gelu_residual_layernorm
    _check(fn(
        _p(xa), _p(ra), _p(b), _p(g), _p(be), _p(y), _p(mean), _p(rstd),
        rows, hidden, hidden, hidden, hidden, float(eps), dt, _nt(threads)),
        "bias_gelu_residual_layernorm")
    return y, mean, rstd


def bn_relu_avgpool(x, scale, shift, threads=1, want_y=True):
    """x is NCHW contiguous. Returns (y or None, pooled[N,C])."""
    xa, dt = as_data(x)
    N, Cc, H, W = xa.shape
    sc, sh = as_param(scale), as_param(shift)
    y = np.empty((N, Cc, H, W), dtype=np.float64) if want_y else None
    pooled = np.empty((N, Cc), dtype=np.float64)
    _check(lib().kopref_bn_relu_avgpool(_p(xa), _p(sc), _p(sh), _p(y), _p(pooled),
                                        N, Cc, H, W, dt, _nt(threads)), "bn_relu_avgpool")
    return y, pooled


def ce_loss_rowwise(logits, labels, threads=1):
    """Returns (loss[rows], mean, bad_label_count)."""
    za, dt = as_data(logits)
    rows, vocab = za.shape
    if hasattr(labels, "detach"):
        labels = labels.detach().cpu().numpy()
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    loss = np.empty(rows, dtype=np.float64)
    mean = C.c_double(0.0)
    bad = C.c_int64(0)
    _check(lib().kopref_ce_loss_rowwise(_p(za), _p(lab), _p(loss), C.addressof(mean),
                                        C.addressof(bad), rows, vocab, vocab, dt, _nt(threads)),
           "ce_loss_rowwise")
    return loss, mean.value, bad.value


def rmsnorm(x, weight, eps, threads=1) -> np.ndarray:
    xa, dt = as_data(x)
    rows, hidden = xa.shape
    w = as_param(weight)
    y = np.empty((rows, hidden), dtype=np.float64)
    _check(lib().kopref_rmsnorm(_p(xa), _p(w), _p(y), rows, hidden, hidden, hidden,
                                float(eps), dt, _nt(threads)), "rmsnorm")
    return y


def residual_rmsnorm(x, residual, weight, eps, threads=1):
    """The residual stream step of a pre-norm transformer block: h = x + residual, y = rmsnorm(h; weight, eps),
    both from the unrounded float64 sum. Returns (h, y). A composition of the two oracle functions above and
    below (residual_add, rmsnorm): nothing new is computed here."""
    h = residual_add(x, residual, threads)
    return h, rmsnorm(h, weight, eps, threads)


def lp_normalize_rows(x, p=2, eps=1e-12, threads=1):
    """y = x / max(||x||_p, eps) per row, p in (1, 2). Returns (y, norms)."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    y = np.empty((rows, cols), dtype=np.float64)
    n = np.empty((rows,), dtype=np.float64)
    _check(lib().kopref_lp_normalize_rows(_p(xa), _p(y), _p(n), rows, cols, cols, cols, int(p), float(eps), dt, _nt(threads)),
           "lp_normalize_rows")
    return y, n


def silu_mul(gate_up, threads=1) -> np.ndarray:
    ga, dt = as_data(gate_up)
    rows, two_i = ga.shape
    assert two_i % 2 == 0
    inter = two_i // 2
    out = np.empty((rows, inter), dtype=np.float64)
    _check(lib().kopref_silu_mul(_p(ga), _p(out), rows, inter, two_i, inter, dt, _nt(threads)),
           "silu_mul")
    return out


def residual_add(a, b, threads=1) -> np.ndarray:
    aa, dt = as_data(a)
    ba, dt2 = as_data(b)
    assert dt == dt2 and aa.shape == ba.shape
    rows, cols = aa.shape
    out = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_residual_add(_p(aa), _p(ba), _p(out), rows, cols, cols, cols, cols,
                                     dt, _nt(threads)), "residual_add")
    return out


def gemm_nt(a, w, threads=1) -> np.ndarray:
    """C = A @ W^T with A [M,K], W [N,K]; triple loop in float64."""
    aa, adt = as_data(a)
    wa, wdt = as_data(w)
    M, K = aa.shape
    N, K2 = wa.shape
    assert K == K2
    out = np.empty((M, N), dtype=np.float64)
    _check(lib().kopref_gemm_nt(_p(aa), adt, _p(wa), wdt, _p(out), M, N, K, _nt(threads)), "gemm_nt")
    return out


def residual_layernorm(x, residual, gamma, beta, eps, threads=1):
    """LayerNorm(x + residual) (residual may be None). Returns (y, mean, rstd)."""
    xa, dt = as_data(x)
    ra = None
    if residual is not None:
        ra, dt2 = as_data(residual)
        assert dt == dt2 and ra.shape == xa.shape
    rows, hidden = xa.shape
    g, be = as_param(gamma), as_param(beta)
    y = np.empty((rows, hidden), dtype=np.float64)
    mean = np.empty(rows, dtype=np.float64)
    rstd = np.empty(rows, dtype=np.float64)
    _check(lib().kopref_residual_layernorm(_p(xa), _p(ra), _p(g), _p(be), _p(y), _p(mean), _p(rstd), rows, hidden,
                                           hidden, hidden, hidden, float(eps), dt, _nt(threads)), "residual_layernorm")
    return y, mean, rstd


def silu_mul_interleaved(gate_up, threads=1) -> np.ndarray:
    ga, dt = as_data(gate_up)
    rows, two_i = ga.shape
    assert two_i % 2 == 0
    inter = two_i // 2
    out = np.empty((rows, inter), dtype=np.float64)
    _check(lib().kopref_silu_mul_interleaved(_p(ga), _p(out), rows, inter, two_i, inter, dt, _nt(threads)),
           "silu_mul_interleaved")
    return out


def ce_loss_opts(logits, labels, ignore_index=-100, smoothing=0.0, threads=1):
    """Returns (loss[rows], mean over counted rows, bad_label_count, counted_rows)."""
    za, dt = as_data(logits)
    rows, vocab = za.shape
    if hasattr(labels, "detach"):
        labels = labels.detach().cpu().numpy()
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    loss = np.empty(rows, dtype=np.float64)
    mean = C.c_double(0.0)
    bad = C.c_int64(0)
    cnt = C.c_int64(0)
    _check(lib().kopref_ce_loss_opts(_p(za), _p(lab), _p(loss), C.addressof(mean), C.addressof(bad),
                                     C.addressof(cnt), rows, vocab, vocab, int(ignore_index), float(smoothing),
                                     dt, _nt(threads)), "ce_loss_opts")
    return loss, mean.value, bad.value, cnt.value


def ce_loss_sum(logits, labels, ignore_index=-100, smoothing=0.0, threads=1) -> float:
    """Cross-entropy with reduction "sum": the per-row losses added over the rows whose label is not ignore_index."""
    za, dt = as_data(logits)
    rows, vocab = za.shape
    if hasattr(labels, "detach"):
        labels = labels.detach().cpu().numpy()
    lab = np.ascontiguousarray(labels, dtype=np.int32)
    loss = np.empty(rows, dtype=np.float64)
    total = C.c_double(0.0)
    _check(lib().kopref_ce_loss_sum(_p(za), _p(lab), _p(loss), C.addressof(total), rows, vocab, vocab,
                                    int(ignore_index), float(smoothing), dt, _nt(threads)), "ce_loss_sum")
    return total.value


def groupnorm_act(x, gamma, beta, groups, eps, act=0, threads=1):
    """x is NCHW contiguous; act 0 none / 1 relu / 2 silu. Returns (y, mean[N,groups], rstd[N,groups])."""
    xa, dt = as_data(x)
    N, Cc, H, W = xa.shape
    g, be = as_param(gamma), as_param(beta)
    y = np.empty((N, Cc, H, W), dtype=np.float64)
    mean = np.empty((N, groups), dtype=np.float64)
    rstd = np.empty((N, groups), dtype=np.float64)
    _check(lib().kopref_groupnorm_act(_p(xa), _p(g), _p(be), _p(y), _p(mean), _p(rstd), N, Cc, H, W, int(groups),
                                      float(eps), int(act), dt, _nt(threads)), "groupnorm_act")
    return y, mean, rstd


def row_scale(a, b, threads=1) -> np.ndarray:
    """out[i, :] = a[i] * b[i, :]."""
    aa, adt = as_data(a)
    ba, bdt = as_data(b)
    assert adt == bdt and aa.ndim == 1 and aa.shape[0] == ba.shape[0]
    rows, cols = ba.shape
    out = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_row_scale(_p(aa), _p(ba), _p(out), rows, cols, cols, cols, bdt, _nt(threads)), "row_scale")
    return out


def matvec_bias(x, w, b_sum, threads=1) -> np.ndarray:
    """out[i] = sum_k x[i, k] * w[k] + b_sum (w fp32)."""
    xa, dt = as_data(x)
    M, K = xa.shape
    wa = as_param(w)
    assert wa.shape == (K,)
    out = np.empty(M, dtype=np.float64)
    _check(lib().kopref_matvec_bias(_p(xa), _p(wa), float(b_sum), _p(out), M, K, K, dt, _nt(threads)), "matvec_bias")
    return out


def affine_relu_pool2d(x, scale, shift, kernel, stride, padding, mode="max", relu=True, threads=1) -> np.ndarray:
    """Per-channel affine (scale / shift both None: none) + optional ReLU + max / avg pooling over windows.
    kernel, stride, padding: (h, w) pairs. x is NCHW contiguous. Returns y[N, C, OH, OW]."""
    xa, dt = as_data(x)
    N, Cc, H, W = xa.shape
    sc, sh = as_param(scale), as_param(shift)
    (kh, kw), (sth, stw), (ph, pw) = kernel, stride, padding
    OH, OW = (H + 2 * ph - kh) // sth + 1, (W + 2 * pw - kw) // stw + 1
    y = np.empty((N, Cc, OH, OW), dtype=np.float64)
    _check(lib().kopref_affine_relu_pool2d(_p(xa), _p(sc), _p(sh), _p(y), N, Cc, H, W, kh, kw, sth, stw, ph, pw,
                                           {"max": 0, "avg": 1}[mode], int(bool(relu)), dt, _nt(threads)),
           "affine_relu_pool2d")
    return y


REDUCE_OPS = {"sum": 0, "mean": 1, "max": 2, "min": 3, "logsumexp": 4}


def reduce_rows(x, op, threads=1):
    """Reduction of each row of x [rows, cols]. Returns (values[rows] float64, index[rows] int32 or None);
    the index (first position of the result) exists for "max" and "min" only."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    out = np.empty(rows, dtype=np.float64)
    idx = np.empty(rows, dtype=np.int32) if op in ("max", "min") else None
    _check(lib().kopref_reduce_rows(_p(xa), _p(out), _p(idx), rows, cols, cols, REDUCE_OPS[op], dt, _nt(threads)),
           "reduce_rows")
    return out, idx


ACTS = {"identity": 0, "relu": 1, "leaky_relu": 2, "gelu_tanh": 3, "gelu_erf": 4, "silu": 5, "sigmoid": 6,
        "tanh": 7, "mish": 8, "hardswish": 9, "elu": 10}


def act_value(u: float, act: str, alpha: float = 0.01) -> float:
    return lib().kopref_act_value(float(u), ACTS[act], float(alpha))


def bias_act(x, bias, act, alpha=0.01, threads=1) -> np.ndarray:
    """y = act(x + bias) (bias None: act(x)); x [rows, cols], bias fp32 [cols]."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    b = as_param(bias)
    y = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_bias_act(_p(xa), _p(b), _p(y), rows, cols, cols, cols, ACTS[act], float(alpha), dt, _nt(threads)),
           "bias_act")
    return y


def epilogue_chain(x, bias, residual, scale=1.0, residual_scale=1.0, lo=-np.inf, hi=np.inf, act="identity", alpha=0.01,
                   threads=1) -> np.ndarray:
    """y = act(clamp((x + bias) * scale + residual * residual_scale, lo, hi)); bias / residual may be None."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    b = as_param(bias)
    ra = None
    if residual is not None:
        ra, dt2 = as_data(residual)
        assert dt2 == dt and ra.shape == xa.shape
    y = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_epilogue_chain(_p(xa), _p(b), _p(ra), _p(y), rows, cols, cols, cols, cols, float(scale),
                                       float(residual_scale), float(lo), float(hi), ACTS[act], float(alpha), dt, _nt(threads)),
           "epilogue_chain")
    return y


def lstm_cell(gates, c_prev, gates2=None, bias=None, threads=1):
    """Pointwise part of an LSTM step. gates (+ gates2 + bias): [rows, 4 * hidden] in the order i, f, g, o;
    c_prev: [rows, hidden]. Returns (h_out, c_out)."""
    ga, dt = as_data(gates)
    ca, dt2 = as_data(c_prev)
    rows, four_h = ga.shape
    hidden = four_h // 4
    assert dt == dt2 and four_h == 4 * hidden and ca.shape == (rows, hidden)
    g2 = None
    if gates2 is not None:
        g2, dt3 = as_data(gates2)
        assert dt3 == dt and g2.shape == ga.shape
    b = as_param(bias)
    h = np.empty((rows, hidden), dtype=np.float64)
    c = np.empty((rows, hidden), dtype=np.float64)
    _check(lib().kopref_lstm_cell(_p(ga), _p(g2), _p(b), _p(ca), _p(h), _p(c), rows, hidden, dt, _nt(threads)), "lstm_cell")
    return h, c


def gru_cell(gi, gh, h_prev, bias_i=None, bias_h=None, threads=1) -> np.ndarray:
    """Pointwise part of a GRU step. gi, gh: [rows, 3 * hidden] in the order r, z, n; h_prev: [rows, hidden];
    bias_i / bias_h are added to gi / gh. Returns h_out."""
    ia, dt = as_data(gi)
    ha, dt2 = as_data(gh)
    pa, dt3 = as_data(h_prev)
    rows, three_h = ia.shape
    hidden = three_h // 3
    assert dt == dt2 == dt3 and three_h == 3 * hidden and ha.shape == ia.shape and pa.shape == (rows, hidden)
    bi, bh = as_param(bias_i), as_param(bias_h)
    out = np.empty((rows, hidden), dtype=np.float64)
    _check(lib().kopref_gru_cell(_p(ia), _p(ha), _p(bi), _p(bh), _p(pa), _p(out), rows, hidden, dt, _nt(threads)), "gru_cell")
    return out


def cumsum_rows(x, mask=None, exclusive=False, reverse=False, threads=1) -> np.ndarray:
    """Running sum along each row of x [rows, cols]; mask (uint8 / bool, same shape, nonzero = keep) zeroes
    elements before they are summed. See kopref_cumsum_rows for the four variants."""
    xa, dt = as_data(x)
    rows, cols = xa.shape
    m = None
    if mask is not None:
        m = np.ascontiguousarray(np.asarray(mask.detach().cpu().numpy() if hasattr(mask, "detach") else mask)
                                 .astype(np.uint8))
        assert m.shape == (rows, cols)
    out = np.empty((rows, cols), dtype=np.float64)
    _check(lib().kopref_cumsum_rows(_p(xa), None if m is None else _p(m), _p(out), rows, cols, cols, cols, cols,
                                    int(bool(exclusive)), int(bool(reverse)), dt, _nt(threads)), "cumsum_rows")
    return out


def mlp_segment(h, rms_weight, w_gate_up, w_down, eps, threads=1) -> np.ndarray:
    """The chained segment in pure float64, no intermediate rounding:
    out = h + (silu(gate) * up) @ W2^T with [gate|up] = rmsnorm(h) @ W1^T."""
    n = rmsnorm(h, rms_weight, eps, threads)
    gu = gemm_nt(n, w_gate_up, threads)
    act = silu_mul(gu, threads)
    d = gemm_nt(act, w_down, threads)
    ha, tag = as_data(h)
    if tag == BF16:
        hd = (ha.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    elif tag == F16:
        hd = ha.view(np.float16).astype(np.float64)
    else:
        hd = ha.astype(np.float64)
    return residual_add(hd, d, threads)
