"""kop_ce_loss_rowwise_static: the cross-entropy entry point for callers that cannot allocate
(plug-ins without access to the host runtime's memory pool, servers with a frozen memory plan,
latency-critical C callers). Its scratch is a fixed device array inside the library, so the test
checks what such a caller relies on: called through the C ABI with caller-provided outputs only, it
gives the same results as the workspace entry point (bit for bit: same kernels, same order of additions)
and as the float64 oracle, call after call (the array keeps the previous call's contents), up to and
including the largest row count the array was sized for, and it refuses more rows than that, and every other
bad argument, before it touches the device.

This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import kopref
from paper_2609_30059_b200 import build as kbuild
from paper_2609_30059_b200 import synth
from tests._util import assert_close

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


def test_static_variant_validates_every_argument_before_any_device_call(kop):
    # This machine may have no GPU at all: each of these must come back with its own code, which it can only do
    # if no CUDA call precedes the check (a caller that cannot allocate can usually not afford a lost context
    # either).
    L = kop.lib()
    P, Q, R, S, T = 0x10000, 0x200000, 0x400000, 0x500000, 0x600000
    assert L.kop_ce_loss_rowwise_static(None, Q, R, S, T, 4, 8, 8, 1, None) == 1              # NULL logits
    assert L.kop_ce_loss_rowwise_static(P, None, R, S, T, 4, 8, 8, 1, None) == 1              # NULL labels
    assert L.kop_ce_loss_rowwise_static(P, Q, None, S, T, 4, 8, 8, 1, None) == 1              # NULL loss
    assert L.kop_ce_loss_rowwise_static(P, Q, R, S, T, 4, 8, 7, 1, None) == 3                 # row stride < vocab
    assert L.kop_ce_loss_rowwise_static(P + 1, Q, R, S, T, 4, 8, 8, 1, None) == 5             # logits not on an element
    assert L.kop_ce_loss_rowwise_static(P, Q + 2, R, S, T, 4, 8, 8, 1, None) == 5             # labels misaligned
    assert L.kop_ce_loss_rowwise_static(P, Q, R + 2, S, T, 4, 8, 8, 1, None) == 5             # loss misaligned
    assert L.kop_ce_loss_rowwise_static(P, Q, R, S + 1, T, 4, 8, 8, 1, None) == 5             # mean misaligned
    assert L.kop_ce_loss_rowwise_static(P, Q, R, S, T + 3, 4, 8, 8, 1, None) == 5             # count misaligned
    assert L.kop_ce_loss_rowwise_static(P, Q, R, S, T, -1, 8, 8, 1, None) == 2                # negative rows
    assert L.kop_ce_loss_rowwise_static(P, Q, R, S, T, 4, 1 << 31, 1 << 31, 1, None) == 2     # vocab beyond int32 labels


@pytest.mark.gpu
def test_static_variant_binding_refuses_outputs_it_would_overrun():
    # The Python wrapper hands the caller's own output tensors to the kernel: a short, wrongly typed or host
    # tensor must be refused on the host, not written out of bounds on the device.
    from paper_2609_30059_b200 import kop as K

    z = torch.zeros((16, 64), dtype=BF16, device="cuda")
    lab = torch.zeros((16,), dtype=torch.int32, device="cuda")
    good = torch.empty((16,), dtype=F32, device="cuda")
    for bad_loss in (torch.empty((15,), dtype=F32, device="cuda"), torch.empty((16,), dtype=torch.float64, device="cuda"),
                     torch.empty((16,), dtype=F32), torch.empty((32,), dtype=F32, device="cuda")[::2], None):
        with pytest.raises(ValueError):
            K.kop_ce_loss_rowwise_static(z, lab, bad_loss, None, None)
    with pytest.raises(ValueError):
        K.kop_ce_loss_rowwise_static(z, lab, good, torch.empty((1,), dtype=torch.float64, device="cuda"), None)
    with pytest.raises(ValueError):
        K.kop_ce_loss_rowwise_static(z, lab, good, None, torch.empty((1,), dtype=torch.int64, device="cuda"))
    with pytest.raises(ValueError):
        K.kop_ce_loss_rowwise_static(z, lab, good, torch.empty((0,), dtype=F32, device="cuda"), None)


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
            # same kernels, same order of additions: equal bit for bit (NaNs in the same places)
            assert torch.equal(loss.isnan(), ref_loss.isnan()) and torch.equal(mean.isnan(), ref_mean.isnan())
            assert torch.equal(loss.nan_to_num(nan=-5.0), ref_loss.nan_to_num(nan=-5.0))
            assert torch.equal(mean.nan_to_num(nan=-5.0), ref_mean.nan_to_num(nan=-5.0))
            assert int(bad.item()) == int(ref_bad.item())
            # and against the float64 oracle, at the parity tests' fp32-grade tolerance
            ol, omean, obad = kopref.ce_loss_rowwise(z.cpu(), lab.cpu(), threads=None)
            assert_close(loss, ol, 2e-5, "static ce loss")
            assert_close(mean, np.array([omean]), 2e-5, "static ce mean")
            assert int(bad.item()) == obad
            loss.fill_(-1.0)
            mean.fill_(-1.0)
            bad.fill_(-1)


@pytest.mark.gpu
@pytest.mark.parametrize("rows", [1 << 20, (1 << 20) - 3])
def test_static_variant_at_its_row_limit(kop, rows):
    # The largest problem the built-in scratch holds (all 4096 ticket groups, the array's last word) and one just
    # under it whose last group is ragged; vocab 8 keeps the logits at 16 MB. Twice in a row.
    z, lab = synth.ce_inputs(rows, 8, BF16, 21, "cuda")
    lab[12345] = 9                                   # one bad label among a million rows
    ref_loss, ref_mean, ref_bad = kop.kop_ce_loss_rowwise(z, lab)
    loss = torch.empty((rows,), dtype=F32, device="cuda")
    mean = torch.empty((1,), dtype=F32, device="cuda")
    bad = torch.empty((1,), dtype=torch.int32, device="cuda")
    for _ in range(2):
        loss.fill_(-1.0)
        mean.fill_(-1.0)
        bad.fill_(-1)
        kop.kop_ce_loss_rowwise_static(z, lab, loss, mean, bad)
        torch.cuda.synchronize()
        assert torch.equal(loss.nan_to_num(nan=-5.0), ref_loss.nan_to_num(nan=-5.0))
        assert bool(torch.isnan(mean[0])) and bool(torch.isnan(ref_mean[0]))
        assert int(bad.item()) == int(ref_bad.item()) == 1
    # without the bad label the mean is a number: check it against the oracle as well
    lab[12345] = 1
    kop.kop_ce_loss_rowwise_static(z, lab, loss, mean, bad)
    _, ref_mean, _ = kop.kop_ce_loss_rowwise(z, lab)
    ol, omean, _ = kopref.ce_loss_rowwise(z.cpu(), lab.cpu(), threads=None)
    assert torch.equal(mean, ref_mean) and int(bad.item()) == 0
    assert_close(loss, ol, 2e-5, "static ce loss at the limit")
    assert_close(mean, np.array([omean]), 2e-5, "static ce mean at the limit")


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
