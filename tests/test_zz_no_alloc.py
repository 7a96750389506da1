"""ak_xent_fwd_static: the cross-entropy entry point for callers that cannot allocate.

Some users of the library may not ask for device memory when they call it: a server that
gave its whole memory budget to its own arena at start-up, a job under a hard GPU quota, a
latency-critical loop that must stay out of the allocator.  For them the library carries a
fixed 1 MiB scratch array in its device image.  This test calls that entry point through the
C ABI, twice in a row (the second call finds the first call's leftovers in the shared
scratch), and checks both calls against the ordinary allocating entry point AND against the
fp64 CPU checker, with the tolerance the other cross-entropy tests use; it also checks that
the device's free memory is the same before and after the calls.  It is collected last on
purpose, and must also pass when run on its own in a fresh process (the first call then does
the one-time address look-up)."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _raw_static_call(logits, targets, loss, mean, ignore_index=-100):
    """Straight through the C ABI: output buffers exist already, the call allocates nothing."""
    rows, V = logits.shape
    return ak.lib().ak_xent_fwd_static(
        ctypes.c_void_p(logits.data_ptr()), ctypes.c_void_p(targets.data_ptr()), ignore_index,
        ctypes.c_void_p(loss.data_ptr()), ctypes.c_void_p(mean.data_ptr()), rows, V,
        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))


@pytest.mark.parametrize("rows,V", [(16, 128256), (300, 4099), (1, 50304), (700, 1000)])
def test_static_scratch_entry_matches_allocating_entry_and_checker_twice(rows, V):
    # two different inputs of the same shape: the second call inherits the first one's scratch
    for call, seed in enumerate((901, 902)):
        logits_h, targets_h = synth.xent_inputs(rows, V, seed + rows, ignore_frac=0.2)
        oracle_rows, oracle_mean, _ = oracle.xent(synth.to_bits(logits_h), targets_h.numpy())
        logits, targets = logits_h.to(DEV), targets_h.to(DEV)
        ref_rows, ref_mean = ak.ak_xent_fwd(logits, targets)
        loss = torch.full((rows,), -7.0, dtype=torch.float32, device=DEV)
        mean = torch.full((1,), -7.0, dtype=torch.float32, device=DEV)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        status = _raw_static_call(logits, targets, loss, mean)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert status == 0, ak.ak_status_string(status)
        if call > 0:   # (the very first call on a device may load the kernel's code)
            assert free_after == free_before, "the call changed the device's free memory"
        assert_loss_close(loss, oracle_rows, f"static rows vs checker, call {call} {rows}x{V}")
        assert_loss_close(mean, np.array([oracle_mean]), f"static mean vs checker, call {call} {rows}x{V}")
        assert_loss_close(loss, ref_rows.cpu().double().numpy(), f"static rows call {call} {rows}x{V}")
        assert_loss_close(mean, ref_mean.cpu().double().numpy(), f"static mean call {call} {rows}x{V}")
        ign = targets == -100
        assert bool((loss[ign] == 0).all()) and bool((loss[~ign] >= 0).all())


def test_static_scratch_entry_rejects_what_does_not_fit():
    # 200000 rows need 200000 * 8 bytes of scratch > 1 MiB (and exceed the row limit)
    rows, V = 200000, 8
    logits = torch.zeros((rows, V), dtype=torch.bfloat16, device=DEV)
    targets = torch.zeros((rows,), dtype=torch.int64, device=DEV)
    loss = torch.full((rows,), -7.0, dtype=torch.float32, device=DEV)
    mean = torch.full((1,), -7.0, dtype=torch.float32, device=DEV)
    status = _raw_static_call(logits, targets, loss, mean)
    torch.cuda.synchronize()
    assert status == 7 and "fixed scratch" in ak.ak_status_string(status)
    assert bool((loss == -7.0).all()) and mean.item() == -7.0      # nothing was launched
    # 60000 unsplit rows need 480 KB: they fit
    assert _raw_static_call(logits[:60000], targets[:60000], loss[:60000], mean) == 0
    torch.cuda.synchronize()
    assert abs(mean.item() - np.log(8.0)) < 1e-5
    with pytest.raises(ak.AkError):
        ak.ak_xent_fwd_static(logits, targets)
    # the shape limits every cross-entropy entry point applies hold here as well
    l = ak.lib()
    P = ctypes.c_void_p(logits.data_ptr())
    assert l.ak_xent_fwd_static(P, ctypes.c_void_p(targets.data_ptr()), -100, ctypes.c_void_p(loss.data_ptr()),
                                None, 1 << 40, 1 << 40, None) == 2
