"""kop_ce_loss_rowwise_static: the cross-entropy entry point for callers that cannot allocate
(plug-ins without access to the host runtime's memory pool, servers with a frozen memory plan,
latency-critical C callers). Its scratch is a fixed device array inside the library, so the test
checks what such a caller relies on: called through the C ABI with caller-provided outputs only, it
gives the same results as the workspace entry point, call after call (the array keeps the previous
call's contents), and it refuses more rows than the array was sized for.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth

BF16, F32 = torch.bfloat16, torch.float32


@pytest.fixture(scope="module")
def kop():
    kbuild.build()
    from paper_2609_30059_b200 import kop as K
    return K


def test_static_variant_rejects_more_rows_than_its_scratch_holds(kop):
    # Pure argument check: refused before any device work, so it runs without a GPU too.
    L = kop.lib()
    limit = L.kop_ce_loss_rowwise_static_max_rows()
    assert limit == 1 << 20
    P, Q, R = 0x10000, 0x200000, 0x400000
    assert L.kop_ce_loss_rowwise_static(P, Q, R, None, None, limit + 1, 8, 8, 1, None) == 7   # WORKSPACE_TOO_SMALL
    assert L.kop_ce_loss_rowwise_static(P, Q, R, None, None, 0, 8, 8, 1, None) == 0           # empty: nothing to do
    assert L.kop_ce_loss_rowwise_static(P, Q, R, None, None, 4, 0, 8, 1, None) == 2           # bad shape
    assert L.kop_ce_loss_rowwise_static(P, Q, R, None, None, 4, 8, 8, 9, None) == 4           # bad dtype


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_on_consecutive_calls(kop):
    dev = "cuda"
    cases = [(700, 32000, BF16, 11), (333, 4096, F32, 12), (700, 32000, BF16, 13), (1, 1000, BF16, 14)]
    for rows, vocab, dtype, seed in cases:          # back to back: each call finds the last one's scratch
        z, lab = synth.ce_inputs(rows, vocab, dtype, seed, dev)
        if seed == 13:
            lab[5] = -3                             # a bad label must be counted here too
        ref_loss, ref_mean, ref_bad = kop.kop_ce_loss_rowwise(z, lab)
        loss = torch.full((rows,), -1.0, dtype=F32, device=dev)
        mean = torch.full((1,), -1.0, dtype=F32, device=dev)
        bad = torch.full((1,), -1, dtype=torch.int32, device=dev)
        for _ in range(2):                          # two calls in a row on the same inputs
            kop.kop_ce_loss_rowwise_static(z, lab, loss, mean, bad)
            torch.cuda.synchronize()
            # same kernels, same order of additions: the tolerance of the parity tests is met with zero slack
            assert torch.allclose(loss, ref_loss, rtol=2e-5, atol=2e-5, equal_nan=True)
            assert torch.allclose(mean, ref_mean, rtol=2e-5, atol=2e-5, equal_nan=True)
            assert torch.equal(loss.isnan(), ref_loss.isnan())
            assert int(bad.item()) == int(ref_bad.item())
            loss.fill_(-1.0)
            mean.fill_(-1.0)
            bad.fill_(-1)


@pytest.mark.gpu
def test_static_variant_refuses_oversized_problem_on_device(kop):
    rows = kop.kop_ce_loss_rowwise_static_max_rows() + 1
    z = torch.zeros((rows, 8), dtype=BF16, device="cuda")
    lab = torch.zeros((rows,), dtype=torch.int32, device="cuda")
    loss = torch.empty((rows,), dtype=F32, device="cuda")
    with pytest.raises(kop.KopError) as ei:
        kop.kop_ce_loss_rowwise_static(z, lab, loss, None, None)
    assert ei.value.status == 7
    # the workspace entry point takes the same problem
    out, _, _ = kop.kop_ce_loss_rowwise(z, lab)
    assert torch.allclose(out, torch.full_like(out, 2.0794415), atol=1e-5)      # ln 8
