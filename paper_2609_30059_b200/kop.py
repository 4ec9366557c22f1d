"""Thin Python binding of libkop's C ABI (include/kop.h): argument marshalling only.

Every function has the name of the C entry point it calls, takes torch CUDA tensors (used purely as
device memory) and passes raw device pointers, shapes, element strides, the dtype tag and the
current CUDA stream to the library. Output tensors are allocated here when the caller passes none;
all arithmetic happens inside the CUDA kernels. There is no fallback: if libkop.so has not been
built (python -m paper_2609_30059_b200.build) importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkop.so")

KOP_OK = 0
KOP_F32, KOP_BF16, KOP_F16 = 0, 1, 2
STATUS_NAMES = [
    "KOP_OK", "KOP_ERR_NULL_POINTER", "KOP_ERR_BAD_SHAPE", "KOP_ERR_BAD_STRIDE",
    "KOP_ERR_UNSUPPORTED_DTYPE", "KOP_ERR_MISALIGNED", "KOP_ERR_BAD_ALIAS",
    "KOP_ERR_WORKSPACE_TOO_SMALL", "KOP_ERR_UNSUPPORTED_DEVICE", "KOP_ERR_CUDA", "KOP_ERR_CUBLAS",
]


class KopError(RuntimeError):
    """A libkop call returned a status other than KOP_OK."""

    def __init__(self, status: int, where: str):
        self.status = int(status)
        name = lib().kop_status_string(self.status).decode()
        super().__init__(f"{where}: {name} ({self.status})")


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library with argument types declared (raw C-ABI access)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_30059_b200.build`; "
                          "libkop has no fallback path")
    L = C.CDLL(LIB_PATH)
    vp, i64, f32, i32, sz = C.c_void_p, C.c_int64, C.c_float, C.c_int, C.c_size_t
    L.kop_version.restype = C.c_int
    L.kop_version.argtypes = []
    L.kop_status_string.restype = C.c_char_p
    L.kop_status_string.argtypes = [i32]
    L.kop_softmax_scale_bias.argtypes = [vp, vp, vp, i64, i64, i64, i64, f32, i32, vp]
    L.kop_softmax_opts.argtypes = [vp, vp, vp, i64, i64, i64, i64, f32, i32, i64, i32, vp]
    L.kop_softmax_opts.restype = i32
    L.kop_bias_gelu_residual_layernorm.argtypes = [vp] * 8 + [i64] * 5 + [f32, i32, vp]
    L.kop_bias_erfgelu_residual_layernorm.argtypes = [vp] * 8 + [i64] * 5 + [f32, i32, vp]
    L.kop_bias_erfgelu_residual_layernorm.restype = i32
    L.kop_bn_relu_avgpool.argtypes = [vp] * 5 + [i64] * 4 + [C.POINTER(i64), C.POINTER(i64), i32, vp]
    L.kop_ce_loss_rowwise.argtypes = [vp] * 5 + [i64] * 3 + [vp, sz, i32, vp]
    L.kop_ce_loss_rowwise_workspace_bytes.restype = sz
    L.kop_ce_loss_rowwise_workspace_bytes.argtypes = [i64, i64, i32]
    L.kop_ce_loss_rowwise_static.argtypes = [vp] * 5 + [i64] * 3 + [i32, vp]
    L.kop_ce_loss_rowwise_static.restype = i32
    L.kop_ce_loss_rowwise_static_max_rows.restype = i64
    L.kop_ce_loss_rowwise_static_max_rows.argtypes = []
    L.kop_rmsnorm.argtypes = [vp, vp, vp, i64, i64, i64, i64, f32, i32, vp]
    L.kop_residual_rmsnorm.argtypes = [vp] * 5 + [i64] * 6 + [f32, i32, vp]
    L.kop_residual_rmsnorm.restype = i32
    L.kop_layernorm_ex.argtypes = [vp] * 8 + [i64] * 5 + [f32, i32, i32, i32, vp]
    L.kop_layernorm_ex.restype = i32
    L.kop_rmsnorm_ex.argtypes = [vp] * 5 + [i64] * 6 + [f32, i32, i32, vp]
    L.kop_rmsnorm_ex.restype = i32
    L.kop_silu_mul.argtypes = [vp, vp, i64, i64, i64, i64, i32, vp]
    L.kop_residual_add.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i32, vp]
    L.kop_ce_loss_rowwise_opts.argtypes = [vp] * 7 + [i64] * 3 + [C.c_int32, f32, vp, sz, i32, vp]
    L.kop_ce_loss_rowwise_opts.restype = i32
    L.kop_residual_layernorm.argtypes = [vp] * 7 + [i64] * 5 + [f32, i32, vp]
    L.kop_residual_layernorm.restype = i32
    L.kop_silu_mul_interleaved.argtypes = [vp, vp, i64, i64, i64, i64, i32, vp]
    L.kop_silu_mul_interleaved.restype = i32
    L.kop_row_scale.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp]
    L.kop_row_scale.restype = i32
    L.kop_matvec_bias.argtypes = [vp, vp, f32, vp, i64, i64, i64, i32, vp]
    L.kop_matvec_bias.restype = i32
    L.kop_groupnorm_act.argtypes = [vp] * 6 + [i64] * 5 + [f32, i32, i32, vp]
    L.kop_groupnorm_act.restype = i32
    L.kop_affine_relu_pool2d.argtypes = [vp] * 4 + [i64] * 4 + [i32] * 9 + [vp]
    L.kop_affine_relu_pool2d.restype = i32
    L.kop_affine_relu_pool2d_ex.argtypes = [vp] * 4 + [i64] * 4 + [i32] * 10 + [vp]
    L.kop_affine_relu_pool2d_ex.restype = i32
    L.kop_reduce_rows.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, vp]
    L.kop_reduce_rows.restype = i32
    L.kop_bias_act.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, f32, i32, vp]
    L.kop_bias_act.restype = i32
    L.kop_epilogue_chain.argtypes = [vp, vp, vp, vp] + [i64] * 5 + [f32] * 4 + [i32, f32, i32, vp]
    L.kop_epilogue_chain.restype = i32
    L.kop_cumsum_rows.argtypes = [vp, vp, vp] + [i64] * 5 + [i32, i32, i32, vp]
    L.kop_cumsum_rows.restype = i32
    L.kop_lp_normalize_rows.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, f32, i32, vp]
    L.kop_lp_normalize_rows.restype = i32
    L.kop_lstm_cell.argtypes = [vp] * 6 + [i64, i64, i32, vp]
    L.kop_lstm_cell.restype = i32
    L.kop_gru_cell.argtypes = [vp] * 6 + [i64, i64, i32, vp]
    L.kop_gru_cell.restype = i32
    L.kop_groupnorm_wait_timeouts.argtypes = [C.POINTER(C.c_uint)]
    L.kop_groupnorm_wait_timeouts.restype = i32
    L.kop_rmsnorm_swiglu_residual.argtypes = [vp] * 6 + [i64] * 3 + [f32, vp, sz, i32, vp]
    L.kop_rmsnorm_swiglu_residual_workspace_bytes.restype = sz
    L.kop_rmsnorm_swiglu_residual_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.kop_mlp_handle_create.argtypes = [C.POINTER(vp)]
    L.kop_mlp_handle_destroy.argtypes = [vp]
    L.kop_softmax_ex.argtypes = [vp, vp, vp, i64, i64, i64, i64, f32, i32, i64, i32, i32, vp]
    L.kop_softmax_ex.restype = i32
    L.kop_bn_relu_avgpool_ex.argtypes = [vp] * 5 + [i64] * 4 + [C.POINTER(i64), C.POINTER(i64), i32, i32, vp]
    L.kop_bn_relu_avgpool_ex.restype = i32
    L.kop_groupnorm_act_ex.argtypes = [vp] * 6 + [i64] * 5 + [f32, i32, i32, i32, vp]
    L.kop_groupnorm_act_ex.restype = i32
    L.kop_bias_act_ex.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, f32, i32, i32, vp]
    L.kop_bias_act_ex.restype = i32
    L.kop_epilogue_chain_ex.argtypes = [vp, vp, vp, vp] + [i64] * 5 + [f32] * 4 + [i32, f32, i32, i32, vp]
    L.kop_epilogue_chain_ex.restype = i32
    L.kop_mlp_handle_wrap.argtypes = [vp, C.POINTER(vp)]
    L.kop_mlp_handle_wrap.restype = i32
    L.kop_mlp_handle_set_residual_in_gemm.argtypes = [vp, i32]
    L.kop_mlp_handle_set_residual_in_gemm.restype = i32
    for name in ("kop_softmax_scale_bias", "kop_bias_gelu_residual_layernorm", "kop_bn_relu_avgpool",
                 "kop_ce_loss_rowwise", "kop_rmsnorm", "kop_silu_mul", "kop_residual_add",
                 "kop_rmsnorm_swiglu_residual", "kop_mlp_handle_create", "kop_mlp_handle_destroy"):
        getattr(L, name).restype = i32
    _lib = L
    return L


def _dtype_tag(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return KOP_F32
    if t.dtype == torch.bfloat16:
        return KOP_BF16
    if t.dtype == torch.float16:
        return KOP_F16
    raise TypeError(f"libkop data tensors are float32, bfloat16 or float16, got {t.dtype}")


def _rows2d(t: torch.Tensor, name: str):
    sh, st = t.shape, t.stride()
    if len(sh) != 2 or (sh[1] > 1 and st[1] != 1):
        raise ValueError(f"{name}: expected a 2-D tensor with unit inner stride")
    if not t.is_cuda:
        raise ValueError(f"{name}: expected a CUDA tensor")
    return sh[0], sh[1], st[0] if sh[0] > 1 else max(st[0], sh[1])


def _param(t, name: str, n: int):
    if t is None:
        return None
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or t.numel() != n:
        raise ValueError(f"{name}: expected a contiguous fp32 CUDA vector of {n} elements")
    return t.data_ptr()


def _out1(t, name: str, dtype, device, n: int = 1):
    """A caller-owned output vector: contiguous, of `dtype`, on `device`, with at least n elements. Returns its pointer."""
    if (not isinstance(t, torch.Tensor) or t.dtype != dtype or not t.is_cuda or t.device != device
            or not t.is_contiguous() or t.numel() < n):
        raise ValueError(f"{name}: expected a contiguous {dtype} tensor of at least {n} element(s) on {device}")
    return t.data_ptr()


# torch.cuda.current_stream() builds a Stream object (about 3 us a call, a quarter of a small launch through this
# binding); the raw handle of the current device's current stream is the same value without the object.
_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream) -> int:
    if stream is None:
        if _raw_current_stream is not None:
            return _raw_current_stream(torch.cuda.current_device())
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(st: int, where: str):
    if st != KOP_OK:
        raise KopError(st, where)


def kop_version() -> int:
    return lib().kop_version()


def kop_softmax_scale_bias(x, bias, scale, out=None, stream=None):
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    _check(lib().kop_softmax_scale_bias(x.data_ptr(), _param(bias, "bias", cols), out.data_ptr(), rows,
                                        cols, xs, ys, float(scale), _dtype_tag(x), _stream(stream)),
           "kop_softmax_scale_bias")
    return out


def kop_softmax_opts(x, bias, scale, log_output=False, causal_period=0, out=None, stream=None):
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    _check(lib().kop_softmax_opts(x.data_ptr(), _param(bias, "bias", cols), out.data_ptr(), rows, cols, xs, ys,
                                  float(scale), int(bool(log_output)), int(causal_period), _dtype_tag(x),
                                  _stream(stream)), "kop_softmax_opts")
    return out


def kop_bias_gelu_residual_layernorm(x, residual, bias, gamma, beta, eps, out=None, mean=None,
                                     rstd=None, want_stats=True, stream=None, erf_form=False):
    """erf_form=True calls kop_bias_erfgelu_residual_layernorm (error-function GELU)."""
    rows, hidden, xs = _rows2d(x, "x")
    _, _, rs = _rows2d(residual, "residual")
    assert residual.shape == x.shape and residual.dtype == x.dtype
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    if want_stats:
        mean = torch.empty(rows, dtype=torch.float32, device=x.device) if mean is None else mean
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device) if rstd is None else rstd
    fn = lib().kop_bias_erfgelu_residual_layernorm if erf_form else lib().kop_bias_gelu_residual_layernorm
    _check(fn(
        x.data_ptr(), residual.data_ptr(), _param(bias, "bias", hidden), _param(gamma, "gamma", hidden),
        _param(beta, "beta", hidden), out.data_ptr(),
        None if mean is None else mean.data_ptr(), None if rstd is None else rstd.data_ptr(),
        rows, hidden, xs, rs, ys, float(eps), _dtype_tag(x), _stream(stream)),
        "kop_bias_gelu_residual_layernorm")
    return out, mean, rstd


def kop_bn_relu_avgpool(x, scale, shift, out=None, pooled=None, stream=None):
    if x.dim() != 4 or not x.is_cuda:
        raise ValueError("x: expected a 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    out = torch.empty_like(x) if out is None else out
    pooled = torch.empty((N, Cc), dtype=torch.float32, device=x.device) if pooled is None else pooled
    xs = (C.c_int64 * 4)(*x.stride())
    ys = (C.c_int64 * 4)(*out.stride())
    _check(lib().kop_bn_relu_avgpool(x.data_ptr(), _param(scale, "scale", Cc), _param(shift, "shift", Cc),
                                     out.data_ptr(), pooled.data_ptr(), N, Cc, H, W, xs, ys,
                                     _dtype_tag(x), _stream(stream)), "kop_bn_relu_avgpool")
    return out, pooled


def kop_ce_loss_rowwise_workspace_bytes(rows: int, vocab: int, dtype_tag: int) -> int:
    return lib().kop_ce_loss_rowwise_workspace_bytes(rows, vocab, dtype_tag)


def kop_ce_loss_rowwise(logits, labels, loss=None, mean_loss=None, bad_label_count=None,
                        workspace=None, stream=None):
    """Returns (loss[rows], mean_loss[1], bad_label_count[1]) as device tensors."""
    rows, vocab, zs = _rows2d(logits, "logits")
    if labels.dtype != torch.int32 or not labels.is_cuda or not labels.is_contiguous() or labels.numel() != rows:
        raise ValueError("labels: expected a contiguous int32 CUDA vector of `rows` elements")
    dev = logits.device
    loss = torch.empty(rows, dtype=torch.float32, device=dev) if loss is None else loss
    mean_loss = torch.empty(1, dtype=torch.float32, device=dev) if mean_loss is None else mean_loss
    bad_label_count = (torch.empty(1, dtype=torch.int32, device=dev)
                       if bad_label_count is None else bad_label_count)
    need = kop_ce_loss_rowwise_workspace_bytes(rows, vocab, _dtype_tag(logits))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    _check(lib().kop_ce_loss_rowwise(logits.data_ptr(), labels.data_ptr(), loss.data_ptr(),
                                     mean_loss.data_ptr(), bad_label_count.data_ptr(), rows, vocab, zs,
                                     workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                     _dtype_tag(logits), _stream(stream)), "kop_ce_loss_rowwise")
    return loss, mean_loss, bad_label_count


def kop_ce_loss_rowwise_static_max_rows() -> int:
    return lib().kop_ce_loss_rowwise_static_max_rows()


def kop_ce_loss_rowwise_static(logits, labels, loss, mean_loss, bad_label_count, stream=None):
    """kop_ce_loss_rowwise without a workspace argument, for callers that cannot allocate: the
    scratch is a fixed array inside the library (see include/kop.h for the row limit, the one-time
    per-device set-up on the first call, and why overlapping calls race). This wrapper allocates
    nothing either: the caller passes every output tensor."""
    rows, vocab, zs = _rows2d(logits, "logits")
    if labels.dtype != torch.int32 or not labels.is_cuda or not labels.is_contiguous() or labels.numel() != rows:
        raise ValueError("labels: expected a contiguous int32 CUDA vector of `rows` elements")
    # The caller owns every output here, so a short or wrongly typed one would be written out of bounds on the
    # device: refuse it on the host.
    dev = logits.device
    if loss is None or not isinstance(loss, torch.Tensor) or loss.numel() != rows:
        raise ValueError("loss: expected a contiguous float32 CUDA vector of `rows` elements")
    _check(lib().kop_ce_loss_rowwise_static(
        logits.data_ptr(), labels.data_ptr(), _out1(loss, "loss", torch.float32, dev, rows),
        None if mean_loss is None else _out1(mean_loss, "mean_loss", torch.float32, dev),
        None if bad_label_count is None else _out1(bad_label_count, "bad_label_count", torch.int32, dev),
        rows, vocab, zs, _dtype_tag(logits), _stream(stream)), "kop_ce_loss_rowwise_static")
    return loss, mean_loss, bad_label_count


def kop_rmsnorm(x, weight, eps, out=None, stream=None):
    rows, hidden, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    _check(lib().kop_rmsnorm(x.data_ptr(), _param(weight, "weight", hidden), out.data_ptr(), rows, hidden,
                             xs, ys, float(eps), _dtype_tag(x), _stream(stream)), "kop_rmsnorm")
    return out


def kop_residual_rmsnorm(x, residual, weight, eps, h_out=None, out=None, stream=None):
    """Returns (h, y): h = x + residual, y = rmsnorm(h)."""
    rows, hidden, xs = _rows2d(x, "x")
    _, _, rs = _rows2d(residual, "residual")
    assert residual.shape == x.shape and residual.dtype == x.dtype
    h_out = torch.empty_like(x) if h_out is None else h_out
    out = torch.empty_like(x) if out is None else out
    _, _, hs = _rows2d(h_out, "h_out")
    _, _, ys = _rows2d(out, "out")
    _check(lib().kop_residual_rmsnorm(x.data_ptr(), residual.data_ptr(), _param(weight, "weight", hidden), h_out.data_ptr(),
                                      out.data_ptr(), rows, hidden, xs, rs, hs, ys, float(eps), _dtype_tag(x),
                                      _stream(stream)), "kop_residual_rmsnorm")
    return h_out, out


LN_PROLOGUES = ("bias_gelu_residual", "residual", "none", "bias_erfgelu_residual")


def _param_any(t, name: str, n: int, data):
    """Parameter vector in fp32 or in the data tensor's own type. Returns (pointer, dtype tag)."""
    if t.dtype not in (torch.float32, data.dtype) or not t.is_cuda or not t.is_contiguous() or t.numel() != n:
        raise ValueError(f"{name}: expected a contiguous CUDA vector of {n} fp32 or {data.dtype} elements")
    return t.data_ptr(), (KOP_F32 if t.dtype == torch.float32 else _dtype_tag(data))


def _params_any(data, n, **named):
    """Optional parameter vectors that must share one type (fp32 or the data type). Returns (pointers, dtype tag)."""
    tag, ptrs = None, []
    for name, t in named.items():
        if t is None:
            ptrs.append(None)
            continue
        ptr, tg = _param_any(t, name, n, data)
        if tag is not None and tg != tag:
            raise ValueError("parameter vectors must share one dtype: " + ", ".join(named))
        tag = tg
        ptrs.append(ptr)
    return ptrs, (KOP_F32 if tag is None else tag)


def kop_softmax_ex(x, bias, scale, log_output=False, causal_period=0, out=None, stream=None):
    """kop_softmax_scale_bias / kop_softmax_opts with the bias in fp32 or in x.dtype."""
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    (bp,), ptag = _params_any(x, cols, bias=bias)
    _check(lib().kop_softmax_ex(x.data_ptr(), bp, out.data_ptr(), rows, cols, xs, ys, float(scale),
                                int(bool(log_output)), int(causal_period), _dtype_tag(x), ptag, _stream(stream)),
           "kop_softmax_ex")
    return out


def kop_bn_relu_avgpool_ex(x, scale, shift, out=None, pooled=None, stream=None):
    """kop_bn_relu_avgpool with scale / shift in fp32 or in x.dtype (both the same)."""
    if x.dim() != 4 or not x.is_cuda:
        raise ValueError("x: expected a 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    out = torch.empty_like(x) if out is None else out
    pooled = torch.empty((N, Cc), dtype=torch.float32, device=x.device) if pooled is None else pooled
    xs = (C.c_int64 * 4)(*x.stride())
    ys = (C.c_int64 * 4)(*out.stride())
    (sp, hp), ptag = _params_any(x, Cc, scale=scale, shift=shift)
    _check(lib().kop_bn_relu_avgpool_ex(x.data_ptr(), sp, hp, out.data_ptr(), pooled.data_ptr(), N, Cc, H, W, xs, ys,
                                        _dtype_tag(x), ptag, _stream(stream)), "kop_bn_relu_avgpool_ex")
    return out, pooled


def kop_groupnorm_act_ex(x, gamma, beta, groups, eps, act=0, out=None, mean=None, rstd=None, want_stats=True,
                         stream=None):
    """kop_groupnorm_act with gamma / beta in fp32 or in x.dtype (both the same; each may be None)."""
    if x.dim() != 4 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x: expected a contiguous 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    out = torch.empty_like(x) if out is None else out
    if out.shape != x.shape or out.dtype != x.dtype or not out.is_contiguous():
        raise ValueError("out: expected a contiguous tensor of x's shape and dtype")
    if want_stats:
        mean = torch.empty((N, groups), dtype=torch.float32, device=x.device) if mean is None else mean
        rstd = torch.empty((N, groups), dtype=torch.float32, device=x.device) if rstd is None else rstd
    (gp, bp), ptag = _params_any(x, Cc, gamma=gamma, beta=beta)
    _check(lib().kop_groupnorm_act_ex(x.data_ptr(), gp, bp, out.data_ptr(), None if mean is None else mean.data_ptr(),
                                      None if rstd is None else rstd.data_ptr(), N, Cc, H, W, int(groups), float(eps),
                                      int(act), _dtype_tag(x), ptag, _stream(stream)), "kop_groupnorm_act_ex")
    return out, mean, rstd


def kop_bias_act_ex(x, bias, act, alpha=0.01, out=None, stream=None):
    """kop_bias_act with the bias in fp32 or in x.dtype."""
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    (bp,), ptag = _params_any(x, cols, bias=bias)
    _check(lib().kop_bias_act_ex(x.data_ptr(), bp, out.data_ptr(), rows, cols, xs, ys, ACTS[act], float(alpha),
                                 _dtype_tag(x), ptag, _stream(stream)), "kop_bias_act_ex")
    return out


def kop_epilogue_chain_ex(x, bias, residual, scale=1.0, residual_scale=1.0, lo=float("-inf"), hi=float("inf"),
                          act="identity", alpha=0.01, out=None, stream=None):
    """kop_epilogue_chain with the bias in fp32 or in x.dtype."""
    rows, cols, xs = _rows2d(x, "x")
    rs = cols
    if residual is not None:
        _, _, rs = _rows2d(residual, "residual")
        assert residual.shape == x.shape and residual.dtype == x.dtype
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    (bp,), ptag = _params_any(x, cols, bias=bias)
    _check(lib().kop_epilogue_chain_ex(x.data_ptr(), bp, None if residual is None else residual.data_ptr(),
                                       out.data_ptr(), rows, cols, xs, rs, ys, float(scale), float(residual_scale),
                                       float(lo), float(hi), ACTS[act], float(alpha), _dtype_tag(x), ptag,
                                       _stream(stream)), "kop_epilogue_chain_ex")
    return out


def kop_layernorm_ex(x, residual, bias, gamma, beta, eps, prologue="bias_gelu_residual", out=None, mean=None,
                     rstd=None, want_stats=True, stream=None):
    """LayerNorm with a chosen prologue (LN_PROLOGUES) and parameters in fp32 or x.dtype (all the same type)."""
    pro = LN_PROLOGUES.index(prologue)
    rows, hidden, xs = _rows2d(x, "x")
    rs = xs
    if pro != 2:
        _, _, rs = _rows2d(residual, "residual")
        assert residual.shape == x.shape and residual.dtype == x.dtype
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    if want_stats:
        mean = torch.empty(rows, dtype=torch.float32, device=x.device) if mean is None else mean
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device) if rstd is None else rstd
    gp, ptag = _param_any(gamma, "gamma", hidden, x)
    bp, btag = _param_any(beta, "beta", hidden, x)
    ip, itag = _param_any(bias, "bias", hidden, x) if pro in (0, 3) else (None, ptag)
    if not (ptag == btag == itag):
        raise ValueError("bias, gamma and beta must share one dtype")
    _check(lib().kop_layernorm_ex(x.data_ptr(), None if pro == 2 else residual.data_ptr(), ip, gp, bp, out.data_ptr(),
                                  None if mean is None else mean.data_ptr(), None if rstd is None else rstd.data_ptr(),
                                  rows, hidden, xs, rs, ys, float(eps), pro, _dtype_tag(x), ptag, _stream(stream)),
           "kop_layernorm_ex")
    return out, mean, rstd


def kop_rmsnorm_ex(x, weight, eps, residual=None, h_out=None, out=None, stream=None):
    """RMSNorm with the weight in fp32 or x.dtype. With a residual returns (h, y), h = x + residual; else y."""
    rows, hidden, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    wp, ptag = _param_any(weight, "weight", hidden, x)
    rs = hs = 0
    if residual is not None:
        _, _, rs = _rows2d(residual, "residual")
        assert residual.shape == x.shape and residual.dtype == x.dtype
        h_out = torch.empty_like(x) if h_out is None else h_out
        _, _, hs = _rows2d(h_out, "h_out")
    _check(lib().kop_rmsnorm_ex(x.data_ptr(), None if residual is None else residual.data_ptr(), wp,
                                None if residual is None else h_out.data_ptr(), out.data_ptr(), rows, hidden, xs, rs, hs,
                                ys, float(eps), _dtype_tag(x), ptag, _stream(stream)), "kop_rmsnorm_ex")
    return (h_out, out) if residual is not None else out


def kop_silu_mul(gate_up, out=None, stream=None):
    rows, two_i, is_ = _rows2d(gate_up, "gate_up")
    if two_i % 2:
        raise ValueError("gate_up: the row length must be even ([gate | up])")
    inter = two_i // 2
    out = torch.empty((rows, inter), dtype=gate_up.dtype, device=gate_up.device) if out is None else out
    _, _, os_ = _rows2d(out, "out")
    _check(lib().kop_silu_mul(gate_up.data_ptr(), out.data_ptr(), rows, inter, is_, os_,
                              _dtype_tag(gate_up), _stream(stream)), "kop_silu_mul")
    return out


def kop_residual_add(a, b, out=None, stream=None):
    rows, cols, as_ = _rows2d(a, "a")
    _, _, bs = _rows2d(b, "b")
    assert a.shape == b.shape and a.dtype == b.dtype
    out = torch.empty_like(a) if out is None else out
    _, _, os_ = _rows2d(out, "out")
    _check(lib().kop_residual_add(a.data_ptr(), b.data_ptr(), out.data_ptr(), rows, cols, as_, bs, os_,
                                  _dtype_tag(a), _stream(stream)), "kop_residual_add")
    return out


def kop_ce_loss_rowwise_opts(logits, labels, ignore_index=-100, label_smoothing=0.0, loss=None, mean_loss=None,
                             bad_label_count=None, counted_rows=None, workspace=None, stream=None, sum_loss=None):
    """Returns (loss[rows], mean_loss[1], bad_label_count[1], counted_rows[1]) as device tensors; the "sum"
    reduction is written to `sum_loss` (fp32 [1]) when the caller passes one."""
    rows, vocab, zs = _rows2d(logits, "logits")
    if labels.dtype != torch.int32 or not labels.is_cuda or not labels.is_contiguous() or labels.numel() != rows:
        raise ValueError("labels: expected a contiguous int32 CUDA vector of `rows` elements")
    dev = logits.device
    loss = torch.empty(rows, dtype=torch.float32, device=dev) if loss is None else loss
    mean_loss = torch.empty(1, dtype=torch.float32, device=dev) if mean_loss is None else mean_loss
    bad_label_count = torch.empty(1, dtype=torch.int32, device=dev) if bad_label_count is None else bad_label_count
    counted_rows = torch.empty(1, dtype=torch.int32, device=dev) if counted_rows is None else counted_rows
    need = kop_ce_loss_rowwise_workspace_bytes(rows, vocab, _dtype_tag(logits))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    _check(lib().kop_ce_loss_rowwise_opts(logits.data_ptr(), labels.data_ptr(), loss.data_ptr(),
                                          mean_loss.data_ptr(),
                                          None if sum_loss is None else _out1(sum_loss, "sum_loss", torch.float32, dev),
                                          bad_label_count.data_ptr(),
                                          counted_rows.data_ptr(), rows, vocab, zs, int(ignore_index),
                                          float(label_smoothing), workspace.data_ptr(),
                                          workspace.numel() * workspace.element_size(), _dtype_tag(logits),
                                          _stream(stream)), "kop_ce_loss_rowwise_opts")
    return loss, mean_loss, bad_label_count, counted_rows


def kop_residual_layernorm(x, residual, gamma, beta, eps, out=None, mean=None, rstd=None, want_stats=True,
                           stream=None):
    rows, hidden, xs = _rows2d(x, "x")
    rs = xs
    if residual is not None:
        _, _, rs = _rows2d(residual, "residual")
        assert residual.shape == x.shape and residual.dtype == x.dtype
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    if want_stats:
        mean = torch.empty(rows, dtype=torch.float32, device=x.device) if mean is None else mean
        rstd = torch.empty(rows, dtype=torch.float32, device=x.device) if rstd is None else rstd
    _check(lib().kop_residual_layernorm(
        x.data_ptr(), None if residual is None else residual.data_ptr(), _param(gamma, "gamma", hidden),
        _param(beta, "beta", hidden), out.data_ptr(), None if mean is None else mean.data_ptr(),
        None if rstd is None else rstd.data_ptr(), rows, hidden, xs, rs, ys, float(eps), _dtype_tag(x),
        _stream(stream)), "kop_residual_layernorm")
    return out, mean, rstd


def kop_silu_mul_interleaved(gate_up, out=None, stream=None):
    rows, two_i, is_ = _rows2d(gate_up, "gate_up")
    if two_i % 2:
        raise ValueError("gate_up: the row length must be even ([g0, u0, g1, u1, ...])")
    inter = two_i // 2
    out = torch.empty((rows, inter), dtype=gate_up.dtype, device=gate_up.device) if out is None else out
    _, _, os_ = _rows2d(out, "out")
    _check(lib().kop_silu_mul_interleaved(gate_up.data_ptr(), out.data_ptr(), rows, inter, is_, os_,
                                          _dtype_tag(gate_up), _stream(stream)), "kop_silu_mul_interleaved")
    return out


def kop_row_scale(a, b, out=None, stream=None):
    rows, cols, bs = _rows2d(b, "b")
    if a.dtype != b.dtype or not a.is_cuda or not a.is_contiguous() or a.numel() != rows:
        raise ValueError("a: expected a contiguous CUDA vector of `rows` elements with b's dtype")
    out = torch.empty_like(b) if out is None else out
    _, _, os_ = _rows2d(out, "out")
    _check(lib().kop_row_scale(a.data_ptr(), b.data_ptr(), out.data_ptr(), rows, cols, bs, os_,
                               _dtype_tag(b), _stream(stream)), "kop_row_scale")
    return out


def kop_matvec_bias(x, w, b_sum, out=None, stream=None):
    rows, k, xs = _rows2d(x, "x")
    out = torch.empty(rows, dtype=torch.float32, device=x.device) if out is None else out
    _check(lib().kop_matvec_bias(x.data_ptr(), _param(w, "w", k), float(b_sum), out.data_ptr(), rows, k, xs,
                                 _dtype_tag(x), _stream(stream)), "kop_matvec_bias")
    return out


def kop_groupnorm_act(x, gamma, beta, groups, eps, act=0, out=None, mean=None, rstd=None, want_stats=True,
                      stream=None):
    """act: 0 identity, 1 ReLU, 2 SiLU. groups == C is InstanceNorm. Returns (y, mean[N, groups], rstd[N, groups])."""
    if x.dim() != 4 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x: expected a contiguous 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    out = torch.empty_like(x) if out is None else out
    if out.shape != x.shape or out.dtype != x.dtype or not out.is_contiguous():
        raise ValueError("out: expected a contiguous tensor of x's shape and dtype")
    if want_stats:
        mean = torch.empty((N, groups), dtype=torch.float32, device=x.device) if mean is None else mean
        rstd = torch.empty((N, groups), dtype=torch.float32, device=x.device) if rstd is None else rstd
    _check(lib().kop_groupnorm_act(x.data_ptr(), _param(gamma, "gamma", Cc), _param(beta, "beta", Cc),
                                   out.data_ptr(), None if mean is None else mean.data_ptr(),
                                   None if rstd is None else rstd.data_ptr(), N, Cc, H, W, int(groups),
                                   float(eps), int(act), _dtype_tag(x), _stream(stream)), "kop_groupnorm_act")
    return out, mean, rstd


def kop_affine_relu_pool2d(x, scale, shift, kernel, stride, padding, mode="max", relu=True, out=None, stream=None):
    """kernel, stride, padding: (h, w) pairs; mode "max" or "avg"; scale / shift both None for plain pooling."""
    if x.dim() != 4 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x: expected a contiguous 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    (kh, kw), (sh, sw), (ph, pw) = kernel, stride, padding
    OH, OW = (H + 2 * ph - kh) // sh + 1, (W + 2 * pw - kw) // sw + 1
    out = torch.empty((N, Cc, max(OH, 0), max(OW, 0)), dtype=x.dtype, device=x.device) if out is None else out
    if out.dtype != x.dtype or not out.is_contiguous():
        raise ValueError("out: expected a contiguous tensor of x's dtype")
    _check(lib().kop_affine_relu_pool2d(x.data_ptr(), _param(scale, "scale", Cc), _param(shift, "shift", Cc),
                                        out.data_ptr(), N, Cc, H, W, kh, kw, sh, sw, ph, pw,
                                        {"max": 0, "avg": 1}[mode], int(bool(relu)), _dtype_tag(x), _stream(stream)),
           "kop_affine_relu_pool2d")
    return out


def kop_affine_relu_pool2d_ex(x, scale, shift, kernel, stride, padding, mode="max", relu=True, out=None, stream=None):
    """kop_affine_relu_pool2d with scale / shift in fp32 or in x.dtype."""
    if x.dim() != 4 or not x.is_cuda or not x.is_contiguous():
        raise ValueError("x: expected a contiguous 4-D NCHW CUDA tensor")
    N, Cc, H, W = x.shape
    (kh, kw), (sh, sw), (ph, pw) = kernel, stride, padding
    OH, OW = (H + 2 * ph - kh) // sh + 1, (W + 2 * pw - kw) // sw + 1
    out = torch.empty((N, Cc, max(OH, 0), max(OW, 0)), dtype=x.dtype, device=x.device) if out is None else out
    if out.dtype != x.dtype or not out.is_contiguous():
        raise ValueError("out: expected a contiguous tensor of x's dtype")
    (sp, hp), ptag = _params_any(x, Cc, scale=scale, shift=shift)
    _check(lib().kop_affine_relu_pool2d_ex(x.data_ptr(), sp, hp, out.data_ptr(), N, Cc, H, W, kh, kw, sh, sw, ph, pw,
                                           {"max": 0, "avg": 1}[mode], int(bool(relu)), _dtype_tag(x), ptag,
                                           _stream(stream)), "kop_affine_relu_pool2d_ex")
    return out


ACTS = {"identity": 0, "relu": 1, "leaky_relu": 2, "gelu_tanh": 3, "gelu_erf": 4, "silu": 5, "sigmoid": 6,
        "tanh": 7, "mish": 8, "hardswish": 9, "elu": 10}


def kop_bias_act(x, bias, act, alpha=0.01, out=None, stream=None):
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    _check(lib().kop_bias_act(x.data_ptr(), _param(bias, "bias", cols), out.data_ptr(), rows, cols, xs, ys, ACTS[act],
                              float(alpha), _dtype_tag(x), _stream(stream)), "kop_bias_act")
    return out


def kop_epilogue_chain(x, bias, residual, scale=1.0, residual_scale=1.0, lo=float("-inf"), hi=float("inf"),
                       act="identity", alpha=0.01, out=None, stream=None):
    rows, cols, xs = _rows2d(x, "x")
    rs = cols
    if residual is not None:
        _, _, rs = _rows2d(residual, "residual")
        assert residual.shape == x.shape and residual.dtype == x.dtype
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    _check(lib().kop_epilogue_chain(x.data_ptr(), _param(bias, "bias", cols), None if residual is None else residual.data_ptr(),
                                    out.data_ptr(), rows, cols, xs, rs, ys, float(scale), float(residual_scale), float(lo),
                                    float(hi), ACTS[act], float(alpha), _dtype_tag(x), _stream(stream)), "kop_epilogue_chain")
    return out


REDUCE_OPS = {"sum": 0, "mean": 1, "max": 2, "min": 3, "logsumexp": 4}


def kop_reduce_rows(x, op, out=None, index=None, want_index=True, stream=None):
    """Returns (values fp32 [rows], index int32 [rows] or None); the index exists for "max" / "min" only."""
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty(rows, dtype=torch.float32, device=x.device) if out is None else out
    if op in ("max", "min") and want_index and index is None:
        index = torch.empty(rows, dtype=torch.int32, device=x.device)
    if op not in ("max", "min"):
        index = None
    _check(lib().kop_reduce_rows(x.data_ptr(), out.data_ptr(), None if index is None else index.data_ptr(), rows, cols,
                                 xs, REDUCE_OPS[op], _dtype_tag(x), _stream(stream)), "kop_reduce_rows")
    return out, index


def kop_cumsum_rows(x, mask=None, exclusive=False, reverse=False, out=None, stream=None):
    """mask: uint8 or bool CUDA tensor of x's shape (nonzero = keep), unit inner stride."""
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    assert out.shape == x.shape and out.dtype == x.dtype
    mp, ms = None, cols
    if mask is not None:
        if mask.dtype == torch.bool:
            mask = mask.view(torch.uint8)
        if mask.dtype != torch.uint8 or mask.shape != x.shape:
            raise ValueError("mask: expected a uint8 / bool tensor of x's shape")
        _, _, ms = _rows2d(mask, "mask")
        mp = mask.data_ptr()
    _check(lib().kop_cumsum_rows(x.data_ptr(), mp, out.data_ptr(), rows, cols, xs, ms, ys, int(bool(exclusive)),
                                 int(bool(reverse)), _dtype_tag(x), _stream(stream)), "kop_cumsum_rows")
    return out


def kop_lp_normalize_rows(x, p=2, eps=1e-12, out=None, norms=None, want_norms=True, stream=None):
    """y = x / max(||x||_p, eps) per row (p = 1 or 2). Returns (y, norms[rows] or None)."""
    rows, cols, xs = _rows2d(x, "x")
    out = torch.empty_like(x) if out is None else out
    _, _, ys = _rows2d(out, "out")
    if want_norms and norms is None:
        norms = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(lib().kop_lp_normalize_rows(x.data_ptr(), out.data_ptr(), None if norms is None else norms.data_ptr(), rows, cols,
                                       xs, ys, int(p), float(eps), _dtype_tag(x), _stream(stream)), "kop_lp_normalize_rows")
    return out, norms


def kop_lstm_cell(gates, c_prev, gates2=None, bias=None, h_out=None, c_out=None, stream=None):
    """gates (and gates2): contiguous [rows, 4H]; c_prev: contiguous [rows, H]; bias: fp32 [4H].
    Returns (h_out, c_out); pass c_out=c_prev to update the state in place."""
    if gates.dim() != 2 or c_prev.dim() != 2 or not gates.is_contiguous() or not c_prev.is_contiguous():
        raise ValueError("gates / c_prev: expected contiguous 2-D tensors")
    rows, hidden = c_prev.shape
    if gates.shape != (rows, 4 * hidden) or gates.dtype != c_prev.dtype:
        raise ValueError("gates: expected [rows, 4 * hidden] of c_prev's dtype")
    if gates2 is not None and (gates2.shape != gates.shape or gates2.dtype != gates.dtype or not gates2.is_contiguous()):
        raise ValueError("gates2: expected a contiguous tensor like gates")
    if bias is not None and (bias.dtype != torch.float32 or bias.shape != (4 * hidden,) or not bias.is_contiguous()):
        raise ValueError("bias: expected contiguous fp32 [4 * hidden]")
    h_out = torch.empty_like(c_prev) if h_out is None else h_out
    c_out = torch.empty_like(c_prev) if c_out is None else c_out
    for t in (h_out, c_out):
        assert t.shape == c_prev.shape and t.dtype == c_prev.dtype and t.is_contiguous()
    _check(lib().kop_lstm_cell(gates.data_ptr(), None if gates2 is None else gates2.data_ptr(),
                               None if bias is None else bias.data_ptr(), c_prev.data_ptr(), h_out.data_ptr(),
                               c_out.data_ptr(), rows, hidden, _dtype_tag(gates), _stream(stream)), "kop_lstm_cell")
    return h_out, c_out


def kop_gru_cell(gi, gh, h_prev, bias_i=None, bias_h=None, h_out=None, stream=None):
    """gi, gh: contiguous [rows, 3H] (blocks r, z, n); h_prev: contiguous [rows, H]; biases fp32 [3H].
    Returns h_out; pass h_out=h_prev to update the state in place."""
    if gi.dim() != 2 or h_prev.dim() != 2 or not gi.is_contiguous() or not h_prev.is_contiguous():
        raise ValueError("gi / h_prev: expected contiguous 2-D tensors")
    rows, hidden = h_prev.shape
    if gi.shape != (rows, 3 * hidden) or gi.dtype != h_prev.dtype:
        raise ValueError("gi: expected [rows, 3 * hidden] of h_prev's dtype")
    if gh.shape != gi.shape or gh.dtype != gi.dtype or not gh.is_contiguous():
        raise ValueError("gh: expected a contiguous tensor like gi")
    for b in (bias_i, bias_h):
        if b is not None and (b.dtype != torch.float32 or b.shape != (3 * hidden,) or not b.is_contiguous()):
            raise ValueError("bias: expected contiguous fp32 [3 * hidden]")
    h_out = torch.empty_like(h_prev) if h_out is None else h_out
    assert h_out.shape == h_prev.shape and h_out.dtype == h_prev.dtype and h_out.is_contiguous()
    _check(lib().kop_gru_cell(gi.data_ptr(), gh.data_ptr(), None if bias_i is None else bias_i.data_ptr(),
                              None if bias_h is None else bias_h.data_ptr(), h_prev.data_ptr(), h_out.data_ptr(),
                              rows, hidden, _dtype_tag(gi), _stream(stream)), "kop_gru_cell")
    return h_out


def kop_groupnorm_wait_timeouts() -> int:
    n = C.c_uint(0)
    _check(lib().kop_groupnorm_wait_timeouts(C.byref(n)), "kop_groupnorm_wait_timeouts")
    return int(n.value)


class MlpHandle:
    """Owner of the vendor-GEMM handle (kop_mlp_handle_create / kop_mlp_handle_destroy)."""

    def __init__(self):
        h = C.c_void_p()
        _check(lib().kop_mlp_handle_create(C.byref(h)), "kop_mlp_handle_create")
        self.ptr = h.value

    def set_residual_in_gemm(self, enable: bool):
        """Fold the residual add into the down projection's cuBLASLt epilogue (see kop.h)."""
        _check(lib().kop_mlp_handle_set_residual_in_gemm(self.ptr, int(bool(enable))),
               "kop_mlp_handle_set_residual_in_gemm")

    def close(self):
        if self.ptr:
            lib().kop_mlp_handle_destroy(self.ptr)
            self.ptr = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass


def kop_rmsnorm_swiglu_residual_workspace_bytes(rows, hidden, inter, dtype_tag) -> int:
    return lib().kop_rmsnorm_swiglu_residual_workspace_bytes(rows, hidden, inter, dtype_tag)


def kop_rmsnorm_swiglu_residual(handle: MlpHandle, h, rms_weight, w_gate_up, w_down, eps, out=None,
                                workspace=None, stream=None):
    rows, hidden, _ = _rows2d(h, "h")
    two_i, hid2, _ = _rows2d(w_gate_up, "w_gate_up")
    hid3, inter, _ = _rows2d(w_down, "w_down")
    if not (h.is_contiguous() and w_gate_up.is_contiguous() and w_down.is_contiguous()):
        raise ValueError("h, w_gate_up and w_down must be contiguous")
    if hid2 != hidden or hid3 != hidden or two_i != 2 * inter:
        raise ValueError("weight shapes must be [2*inter, hidden] and [hidden, inter]")
    out = torch.empty_like(h) if out is None else out
    tag = _dtype_tag(h)
    need = kop_rmsnorm_swiglu_residual_workspace_bytes(rows, hidden, inter, tag)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=h.device)
    _check(lib().kop_rmsnorm_swiglu_residual(handle.ptr, h.data_ptr(), _param(rms_weight, "rms_weight", hidden),
                                             w_gate_up.data_ptr(), w_down.data_ptr(), out.data_ptr(),
                                             rows, hidden, inter, float(eps), workspace.data_ptr(),
                                             workspace.numel(), tag, _stream(stream)),
           "kop_rmsnorm_swiglu_residual")
    return out
