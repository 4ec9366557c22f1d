"""Every compute entry point enqueues on the caller's stream without allocating or synchronising, so a whole
sequence of them can be captured into one CUDA graph and replayed: the replayed results must equal the eager
ones bit for bit, twice in a row (scratch that a call clears on the stream is cleared again in every replay)."""
import pytest
import torch

from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth

pytestmark = pytest.mark.gpu
F32, BF16 = torch.float32, torch.bfloat16


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def test_all_entry_points_in_one_graph(kop):
    dev = "cuda"
    rows, cols = 96, 2048
    x, bias = synth.softmax_inputs(rows, cols, BF16, 1, dev)
    lx, lr, lb, lg, lbe = synth.layernorm_inputs(rows, cols, BF16, 2, dev)
    z, lab = synth.ce_inputs(rows, cols, BF16, 3, dev)
    lab_ig = lab.clone()
    lab_ig[::4] = -100
    img, sc, sh = synth.bn_pool_inputs(3, 16, 28, 28, F32, 4, dev)
    img_cl = img.contiguous(memory_format=torch.channels_last)
    gx, gg, gb = synth.groupnorm_inputs(3, 16, 28, 28, F32, 5, dev)
    gu = synth.gate_up_inputs(rows, cols // 2, BF16, 6, dev)
    cx, cmask = synth.cumsum_inputs(rows, cols, F32, 7, dev)
    av, bm = synth.row_scale_inputs(rows, cols, F32, 8, dev)
    mx, mw, mb = synth.matvec_inputs(rows, cols, BF16, 9, dev)
    h, w, W1, W2 = synth.mlp_inputs(64, 256, 512, BF16, 10, dev)
    tg, tg2, tb, tc = synth.lstm_inputs(rows, 96, BF16, 11, dev)
    ui, uh, ubi, ubh, up = synth.gru_inputs(rows, 96, BF16, 12, dev)
    lb16, lg16, lbe16 = lb.to(lx.dtype), lg.to(lx.dtype), lbe.to(lx.dtype)
    bias16 = bias.to(x.dtype)
    img16, sc16, sh16 = img.to(BF16), sc.to(BF16), sh.to(BF16)
    handle = kop.MlpHandle()
    ws_ce = torch.empty(max(16, kop.kop_ce_loss_rowwise_workspace_bytes(rows, cols, kop.KOP_BF16)), dtype=torch.uint8, device=dev)
    ws_mlp = torch.empty(kop.kop_rmsnorm_swiglu_residual_workspace_bytes(64, 256, 512, kop.KOP_BF16), dtype=torch.uint8, device=dev)

    # every output is preallocated: nothing may allocate inside the captured region
    o = {
        "softmax": torch.empty_like(x), "softmax_opts": torch.empty_like(x), "ln": torch.empty_like(lx),
        "ln_mean": torch.empty(rows, device=dev), "ln_rstd": torch.empty(rows, device=dev), "ln_erf": torch.empty_like(lx),
        "rln": torch.empty_like(lx), "ce_loss": torch.empty(rows, device=dev), "ce_mean": torch.empty(1, device=dev),
        "ce_bad": torch.empty(1, dtype=torch.int32, device=dev), "ceo_loss": torch.empty(rows, device=dev),
        "ceo_mean": torch.empty(1, device=dev), "ceo_bad": torch.empty(1, dtype=torch.int32, device=dev),
        "ceo_cnt": torch.empty(1, dtype=torch.int32, device=dev), "bn": torch.empty_like(img),
        "bn_p": torch.empty((3, 16), device=dev), "bn_cl": torch.empty_like(img_cl), "bn_cl_p": torch.empty((3, 16), device=dev),
        "gn": torch.empty_like(gx), "gn_mean": torch.empty((3, 4), device=dev), "gn_rstd": torch.empty((3, 4), device=dev),
        "pool": torch.empty((3, 16, 14, 14), device=dev), "rms": torch.empty_like(lx), "silu": torch.empty((rows, cols // 2), dtype=BF16, device=dev),
        "silu_i": torch.empty((rows, cols // 2), dtype=BF16, device=dev), "add": torch.empty_like(lx), "cumsum": torch.empty_like(cx),
        "row_scale": torch.empty_like(bm), "matvec": torch.empty(rows, device=dev), "red": torch.empty(rows, device=dev),
        "red_i": torch.empty(rows, dtype=torch.int32, device=dev), "lse": torch.empty(rows, device=dev),
        "act": torch.empty_like(x), "chain": torch.empty_like(x), "mlp": torch.empty_like(h),
        "rr_h": torch.empty_like(lx), "rr_y": torch.empty_like(lx), "lstm_h": torch.empty_like(tc), "lstm_c": torch.empty_like(tc),
        "gru_h": torch.empty_like(up), "lpn": torch.empty_like(lx), "lpn_n": torch.empty(rows, device=dev),
        "ln_ex": torch.empty_like(lx), "rms_ex_h": torch.empty_like(lx), "rms_ex_y": torch.empty_like(lx),
        "ceo_sum": torch.empty(1, device=dev), "softmax_ex": torch.empty_like(x), "act_ex": torch.empty_like(x),
        "chain_ex": torch.empty_like(x), "bn_ex": torch.empty_like(img16), "bn_ex_p": torch.empty((3, 16), device=dev),
        "gn_ex": torch.empty_like(img16), "pool_s1": torch.empty((3, 16, 28, 28), device=dev),
        "pool_walk": torch.empty((3, 16, 27, 27), device=dev), "pool_ex": torch.empty((3, 16, 14, 14), dtype=BF16, device=dev),
    }

    def run():
        kop.kop_softmax_scale_bias(x, bias, 0.125, out=o["softmax"])
        kop.kop_softmax_opts(x, bias, 0.125, True, cols, out=o["softmax_opts"])
        kop.kop_bias_gelu_residual_layernorm(lx, lr, lb, lg, lbe, 1e-5, out=o["ln"], mean=o["ln_mean"], rstd=o["ln_rstd"])
        kop.kop_bias_gelu_residual_layernorm(lx, lr, lb, lg, lbe, 1e-5, out=o["ln_erf"], want_stats=False, erf_form=True)
        kop.kop_residual_layernorm(lx, lr, lg, lbe, 1e-5, out=o["rln"], want_stats=False)
        kop.kop_ce_loss_rowwise(z, lab, loss=o["ce_loss"], mean_loss=o["ce_mean"], bad_label_count=o["ce_bad"], workspace=ws_ce)
        kop.kop_ce_loss_rowwise_opts(z, lab_ig, -100, 0.1, loss=o["ceo_loss"], mean_loss=o["ceo_mean"],
                                     bad_label_count=o["ceo_bad"], counted_rows=o["ceo_cnt"], workspace=ws_ce,
                                     sum_loss=o["ceo_sum"])
        kop.kop_bn_relu_avgpool(img, sc, sh, out=o["bn"], pooled=o["bn_p"])
        kop.kop_bn_relu_avgpool(img_cl, sc, sh, out=o["bn_cl"], pooled=o["bn_cl_p"])
        kop.kop_groupnorm_act(gx, gg, gb, 4, 1e-5, 2, out=o["gn"], mean=o["gn_mean"], rstd=o["gn_rstd"])
        kop.kop_affine_relu_pool2d(img, sc, sh, (3, 3), (2, 2), (1, 1), "max", True, out=o["pool"])
        kop.kop_rmsnorm(lx, lg, 1e-6, out=o["rms"])
        kop.kop_silu_mul(gu, out=o["silu"])
        kop.kop_silu_mul_interleaved(gu, out=o["silu_i"])
        kop.kop_residual_add(lx, lr, out=o["add"])
        kop.kop_cumsum_rows(cx, cmask, True, True, out=o["cumsum"])
        kop.kop_row_scale(av, bm, out=o["row_scale"])
        kop.kop_matvec_bias(mx, mw, mb, out=o["matvec"])
        kop.kop_reduce_rows(x, "max", out=o["red"], index=o["red_i"])
        kop.kop_reduce_rows(x, "logsumexp", out=o["lse"])
        kop.kop_bias_act(x, bias, "mish", out=o["act"])
        kop.kop_epilogue_chain(x, bias, lx, 0.5, 2.0, -1.0, 1.0, "gelu_erf", out=o["chain"])
        kop.kop_residual_rmsnorm(lx, lr, lg, 1e-6, h_out=o["rr_h"], out=o["rr_y"])
        kop.kop_lstm_cell(tg, tc, tg2, tb, h_out=o["lstm_h"], c_out=o["lstm_c"])
        kop.kop_gru_cell(ui, uh, up, ubi, ubh, h_out=o["gru_h"])
        kop.kop_lp_normalize_rows(lx, 2, 1e-12, out=o["lpn"], norms=o["lpn_n"])
        kop.kop_layernorm_ex(lx, lr, lb16, lg16, lbe16, 1e-5, "bias_erfgelu_residual", out=o["ln_ex"], want_stats=False)
        kop.kop_rmsnorm_ex(lx, lg16, 1e-6, residual=lr, h_out=o["rms_ex_h"], out=o["rms_ex_y"])
        kop.kop_softmax_ex(x, bias16, 0.125, True, cols, out=o["softmax_ex"])
        kop.kop_bias_act_ex(x, bias16, "silu", out=o["act_ex"])
        kop.kop_epilogue_chain_ex(x, bias16, lx, 0.5, 2.0, -1.0, 1.0, "relu", out=o["chain_ex"])
        kop.kop_bn_relu_avgpool_ex(img16, sc16, sh16, out=o["bn_ex"], pooled=o["bn_ex_p"])
        kop.kop_groupnorm_act_ex(img16, sc16, sh16, 4, 1e-5, 1, out=o["gn_ex"], want_stats=False)
        kop.kop_affine_relu_pool2d(img, sc, sh, (3, 3), (1, 1), (1, 1), "avg", True, out=o["pool_s1"])
        kop.kop_affine_relu_pool2d(img, sc, sh, (2, 2), (1, 1), (0, 0), "max", False, out=o["pool_walk"])
        kop.kop_affine_relu_pool2d_ex(img16, sc16, sh16, (3, 3), (2, 2), (1, 1), "max", True, out=o["pool_ex"])
        kop.kop_rmsnorm_swiglu_residual(handle, h, w, W1, W2, 1e-6, out=o["mlp"], workspace=ws_mlp)

    try:
        run()                                              # eager pass: also does every one-time set-up
        torch.cuda.synchronize()
        eager = {k: v.clone() for k, v in o.items()}
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                run()
        for _ in range(2):
            for v in o.values():
                v.zero_()
            graph.replay()
            torch.cuda.synchronize()
            for k, v in o.items():
                same = torch.equal(v, eager[k]) or (v.is_floating_point() and torch.equal(torch.isnan(v), torch.isnan(eager[k]))
                                                    and torch.equal(torch.nan_to_num(v), torch.nan_to_num(eager[k])))
                assert same, f"{k}: replayed result differs from the eager one"
        assert kop.kop_groupnorm_wait_timeouts() == 0
    finally:
        handle.close()
