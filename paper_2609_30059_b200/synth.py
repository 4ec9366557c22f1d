"""Seeded synthetic inputs for the fused segments: shapes and value distributions only.

This module holds none of the segments' arithmetic; it only draws tensors. Values are drawn in
fp32 with torch's generator on the requested device, in a fixed order per segment, and then cast
to the data dtype, so the CUDA path and the CPU oracle see identical bit patterns (the oracle gets
a host copy). In N(a, b) the second parameter is the standard deviation.
"""
from __future__ import annotations

import torch

SEEDS = (0, 42, 123, 1337, 2609)

# Full-size workloads (the benchmark configurations).
CONFIGS = {
    "softmax_small": dict(rows=128, cols=512, dtype=torch.float32, scale=0.125),
    "softmax_large": dict(rows=131072, cols=512, dtype=torch.float32, scale=0.125),
    "layernorm": dict(rows=8192, hidden=4096, dtype=torch.bfloat16, eps=1e-5),
    "bn_pool": dict(N=64, C=256, H=56, W=56, dtype=torch.float32),
    "ce_loss": dict(rows=32768, vocab=32000, dtype=torch.bfloat16),
    "mlp": dict(rows=16384, hidden=4096, inter=14336, dtype=torch.bfloat16, eps=1e-6),
    # beyond the five benchmark configs: the two kernels the paper's case studies print
    "row_scale": dict(rows=4096, cols=4096, dtype=torch.float32),          # the paper's 4096 x 4096 shape
    "matvec_bias": dict(rows=32768, k=4096, dtype=torch.bfloat16),         # shape not given in the paper
    # GroupNorm + SiLU as in a diffusion U-Net residual block: 32 groups over 256 channels of a 56 x 56 map
    "groupnorm": dict(N=64, C=256, H=56, W=56, groups=32, dtype=torch.float32, eps=1e-5, act=2),
    # running sum along rows (shape ours; the paper gives none)
    "cumsum": dict(rows=32768, cols=4096, dtype=torch.float32),
    # BatchNorm + ReLU + 3x3 / stride-2 max pool on a 112 x 112 map with 64 channels (a CNN stem)
    "pool2d": dict(N=64, C=64, H=112, W=112, kernel=(3, 3), stride=(2, 2), padding=(1, 1), mode="max",
                   dtype=torch.float32),
    # the same epilogue with a stride-1 3x3 window (an inception-style pooling branch) and on the 14 x 14 maps of a
    # CNN's later stages (shapes ours)
    "pool2d_s1": dict(N=64, C=64, H=112, W=112, kernel=(3, 3), stride=(1, 1), padding=(1, 1), mode="avg",
                      dtype=torch.float32),
    "pool2d_14": dict(N=256, C=512, H=14, W=14, kernel=(3, 3), stride=(2, 2), padding=(1, 1), mode="max",
                      dtype=torch.float32),
    # pointwise part of one LSTM step: batch 16384, hidden 1024 (shape ours)
    "lstm_cell": dict(rows=16384, hidden=1024, dtype=torch.bfloat16),
    "gru_cell": dict(rows=16384, hidden=1024, dtype=torch.bfloat16),
    # shapes away from the benchmark's row lengths (ours): per-head RMSNorm of 16384 tokens x 64 heads of 128, and a
    # softmax over a 128256-entry vocabulary
    "rmsnorm_head128": dict(rows=1048576, hidden=128, eps=1e-6, dtype=torch.bfloat16),
    "softmax_vocab": dict(rows=2048, cols=128256, scale=1.0, dtype=torch.bfloat16),
    "softmax_4096": dict(rows=32768, cols=4096, scale=1.0, dtype=torch.bfloat16),        # rows in one CTA's registers
    # attention scores of a ViT with a class token (12 heads x 197 queries x 128 images, 197 keys): rows that are not
    # whole 16-byte vectors
    "softmax_197": dict(rows=12 * 197 * 128, cols=197, scale=1.0, dtype=torch.bfloat16),
    # GroupNorm(32) + SiLU on a late-stage feature map: 16 channels of 14 x 14 bf16 a group, chunks held in registers
    "groupnorm_14": dict(N=512, C=512, H=14, W=14, groups=32, eps=1e-5, act=2, dtype=torch.bfloat16),
    # row reductions (shape ours)
    "reduce": dict(rows=32768, cols=8192, dtype=torch.bfloat16),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, mean, std, g, device):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std + mean


def _uniform(shape, lo, hi, g, device):
    return torch.rand(shape, generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo


def softmax_inputs(rows, cols, dtype=torch.float32, seed=0, device="cpu"):
    """x ~ N(0,1) [rows, cols]; bias fp32 ~ N(0,0.1) [cols]."""
    g = _gen(seed, device)
    x = _normal((rows, cols), 0.0, 1.0, g, device).to(dtype)
    bias = _normal((cols,), 0.0, 0.1, g, device)
    return x, bias


def layernorm_inputs(rows, hidden, dtype=torch.bfloat16, seed=0, device="cpu"):
    """x, residual ~ N(0,1); bias ~ N(0,0.1); gamma ~ N(1,0.02); beta ~ N(0,0.02) (params fp32)."""
    g = _gen(seed, device)
    x = _normal((rows, hidden), 0.0, 1.0, g, device).to(dtype)
    residual = _normal((rows, hidden), 0.0, 1.0, g, device).to(dtype)
    bias = _normal((hidden,), 0.0, 0.1, g, device)
    gamma = _normal((hidden,), 1.0, 0.02, g, device)
    beta = _normal((hidden,), 0.0, 0.02, g, device)
    return x, residual, bias, gamma, beta


def bn_pool_inputs(N, C, H, W, dtype=torch.float32, seed=0, device="cpu"):
    """x ~ N(0,1) NCHW; scale ~ U(0.5,1.5); shift ~ N(0,0.1) (params fp32)."""
    g = _gen(seed, device)
    x = _normal((N, C, H, W), 0.0, 1.0, g, device).to(dtype)
    scale = _uniform((C,), 0.5, 1.5, g, device)
    shift = _normal((C,), 0.0, 0.1, g, device)
    return x, scale, shift


def ce_inputs(rows, vocab, dtype=torch.bfloat16, seed=0, device="cpu"):
    """logits ~ N(0,2) [rows, vocab]; labels int32 ~ U[0, vocab)."""
    g = _gen(seed, device)
    logits = _normal((rows, vocab), 0.0, 2.0, g, device).to(dtype)
    labels = torch.randint(0, vocab, (rows,), generator=g, device=device, dtype=torch.int64).to(torch.int32)
    return logits, labels


def mlp_inputs(rows, hidden, inter, dtype=torch.bfloat16, seed=0, device="cpu"):
    """h ~ N(0,1); rms weight fp32 ~ N(1,0.02); W_gate_up [2*inter, hidden], W_down [hidden, inter] ~ N(0,0.02)."""
    g = _gen(seed, device)
    h = _normal((rows, hidden), 0.0, 1.0, g, device).to(dtype)
    rms_weight = _normal((hidden,), 1.0, 0.02, g, device)
    w_gate_up = _normal((2 * inter, hidden), 0.0, 0.02, g, device).to(dtype)
    w_down = _normal((hidden, inter), 0.0, 0.02, g, device).to(dtype)
    return h, rms_weight, w_gate_up, w_down


def gate_up_inputs(rows, inter, dtype=torch.bfloat16, seed=0, device="cpu", std=1.0):
    """A stand-in [rows, 2*inter] GEMM output ~ N(0, std) for testing the SwiGLU epilogue alone."""
    g = _gen(seed, device)
    return _normal((rows, 2 * inter), 0.0, std, g, device).to(dtype)


def pair_inputs(rows, cols, dtype=torch.bfloat16, seed=0, device="cpu"):
    """Two ~N(0,1) tensors for the residual add."""
    g = _gen(seed, device)
    a = _normal((rows, cols), 0.0, 1.0, g, device).to(dtype)
    b = _normal((rows, cols), 0.0, 1.0, g, device).to(dtype)
    return a, b


def row_scale_inputs(rows, cols, dtype=torch.float32, seed=0, device="cpu"):
    """a ~ N(0,1) [rows]; b ~ N(0,1) [rows, cols], both of the data dtype."""
    g = _gen(seed, device)
    a = _normal((rows,), 0.0, 1.0, g, device).to(dtype)
    b = _normal((rows, cols), 0.0, 1.0, g, device).to(dtype)
    return a, b


def matvec_inputs(rows, k, dtype=torch.bfloat16, seed=0, device="cpu"):
    """x ~ N(0,1) [rows, k]; w fp32 ~ N(0,0.16) [k] and b_sum ~ N(0,0.8) (a Python float): the spread
    that column sums over 64 outputs of a N(0,0.02) weight and a N(0,0.1) bias would have."""
    g = _gen(seed, device)
    x = _normal((rows, k), 0.0, 1.0, g, device).to(dtype)
    w = _normal((k,), 0.0, 0.16, g, device)
    b_sum = _normal((1,), 0.0, 0.8, g, device)
    return x, w, float(b_sum.item())


def groupnorm_inputs(N, C, H, W, dtype=torch.float32, seed=0, device="cpu"):
    """x NCHW with a per-channel offset and spread (x = m_c + s_c * N(0,1), m_c ~ N(0,1), s_c ~ U(0.5,2)), so the
    groups have non-zero means; gamma ~ N(1,0.02); beta ~ N(0,0.02) (params fp32)."""
    g = _gen(seed, device)
    m = _normal((1, C, 1, 1), 0.0, 1.0, g, device)
    s = _uniform((1, C, 1, 1), 0.5, 2.0, g, device)
    x = (_normal((N, C, H, W), 0.0, 1.0, g, device) * s + m).to(dtype)
    gamma = _normal((C,), 1.0, 0.02, g, device)
    beta = _normal((C,), 0.0, 0.02, g, device)
    return x, gamma, beta


def cumsum_inputs(rows, cols, dtype=torch.float32, seed=0, device="cpu", keep=0.7):
    """x ~ N(0,1) [rows, cols]; mask uint8, 1 with probability `keep`."""
    g = _gen(seed, device)
    x = _normal((rows, cols), 0.0, 1.0, g, device).to(dtype)
    mask = (torch.rand((rows, cols), generator=g, device=device, dtype=torch.float32) < keep).to(torch.uint8)
    return x, mask


def lstm_inputs(rows, hidden, dtype=torch.float32, seed=0, device="cpu"):
    """gates, gates2 ~ N(0,1) [rows, 4 * hidden]; c_prev ~ N(0,1) [rows, hidden]; bias fp32 ~ N(0,0.1) with
    +1 on the forget block (the usual initialisation)."""
    g = _gen(seed, device)
    gates = _normal((rows, 4 * hidden), 0.0, 1.0, g, device).to(dtype)
    gates2 = _normal((rows, 4 * hidden), 0.0, 1.0, g, device).to(dtype)
    c_prev = _normal((rows, hidden), 0.0, 1.0, g, device).to(dtype)
    bias = _normal((4 * hidden,), 0.0, 0.1, g, device)
    bias[hidden:2 * hidden] += 1.0
    return gates, gates2, bias, c_prev


def gru_inputs(rows, hidden, dtype=torch.float32, seed=0, device="cpu"):
    """gi, gh ~ N(0,1) [rows, 3 * hidden]; h_prev ~ U(-1,1) [rows, hidden] (a hidden state is a convex mix of
    tanh values); bias_i, bias_h fp32 ~ N(0,0.1)."""
    g = _gen(seed, device)
    gi = _normal((rows, 3 * hidden), 0.0, 1.0, g, device).to(dtype)
    gh = _normal((rows, 3 * hidden), 0.0, 1.0, g, device).to(dtype)
    h_prev = _uniform((rows, hidden), -1.0, 1.0, g, device).to(dtype)
    bias_i = _normal((3 * hidden,), 0.0, 0.1, g, device)
    bias_h = _normal((3 * hidden,), 0.0, 0.1, g, device)
    return gi, gh, bias_i, bias_h, h_prev
