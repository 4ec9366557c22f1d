"""Host-thread safety of the C ABI: several threads, each on its own stream with its own outputs and
workspace, call a mix of entry points at the same time; every result must be bit-identical to the same call
made alone (the library keeps no per-call state, and its kernels' reduction orders do not depend on what else
is running)."""
import threading

import pytest
import torch

from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def one_pass(kop, inp, ws, stream):
    x, bias, lx, lr, lb, lg, lbe, z, lab, gx, gg, gb, tg, tg2, tb, tc = inp
    out = []
    with torch.cuda.stream(stream):
        out.append(kop.kop_softmax_scale_bias(x, bias, 0.125))
        out.extend(kop.kop_bias_gelu_residual_layernorm(lx, lr, lb, lg, lbe, 1e-5))
        out.extend(kop.kop_ce_loss_rowwise(z, lab, workspace=ws)[:2])
        out.append(kop.kop_rmsnorm(lx, lg, 1e-6))
        out.extend(kop.kop_reduce_rows(x, "max"))
        out.append(kop.kop_reduce_rows(x, "logsumexp")[0])
        out.append(kop.kop_cumsum_rows(x))
        out.extend(kop.kop_groupnorm_act(gx, gg, gb, 4, 1e-5, 2))
        out.extend(kop.kop_lstm_cell(tg, tc, tg2, tb))
    return out


def test_concurrent_host_threads_give_the_serial_results(kop):
    dev = "cuda"
    n_threads, n_iter = 4, 25
    inputs, spaces, streams, serial = [], [], [], []
    for t in range(n_threads):
        rows, cols = 96 + 8 * t, 2048
        x, bias = synth.softmax_inputs(rows, cols, F32, 10 + t, dev)
        lx, lr, lb, lg, lbe = synth.layernorm_inputs(rows, cols, BF16, 20 + t, dev)
        z, lab = synth.ce_inputs(rows, 4000, BF16, 30 + t, dev)
        gx, gg, gb = synth.groupnorm_inputs(2, 16, 28, 28, F32, 40 + t, dev)
        tg, tg2, tb, tc = synth.lstm_inputs(rows, 256, BF16, 50 + t, dev)
        inputs.append((x, bias, lx, lr, lb, lg, lbe, z, lab, gx, gg, gb, tg, tg2, tb, tc))
        spaces.append(torch.empty(max(16, kop.kop_ce_loss_rowwise_workspace_bytes(rows, 4000, kop.KOP_BF16)),
                                  dtype=torch.uint8, device=dev))
        streams.append(torch.cuda.Stream())
    torch.cuda.synchronize()
    for t in range(n_threads):                             # the reference: each mix alone
        serial.append([o.clone() for o in one_pass(kop, inputs[t], spaces[t], streams[t])])
        torch.cuda.synchronize()

    errors = []
    barrier = threading.Barrier(n_threads)

    def worker(t):
        try:
            torch.cuda.set_device(0)
            barrier.wait()
            for it in range(n_iter):
                got = one_pass(kop, inputs[t], spaces[t], streams[t])
                streams[t].synchronize()
                for k, (g, s) in enumerate(zip(got, serial[t])):
                    if not torch.equal(g, s):
                        errors.append(f"thread {t} iteration {it} output {k} differs")
                        return
        except Exception as e:                             # noqa: BLE001
            errors.append(f"thread {t}: {e!r}")

    threads = [threading.Thread(target=worker, args=(t,)) for t in range(n_threads)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=120)
    assert not any(th.is_alive() for th in threads), "a worker did not finish"
    assert not errors, errors[:3]
