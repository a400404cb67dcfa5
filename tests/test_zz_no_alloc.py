"""The allocation-free entry point, checked against the allocating one and against the oracle.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test. Users who cannot call cudaMalloc (their device memory is owned by another
allocator, or they promised a fixed footprint) call nb_gelu_dbias_noalloc; it must give what
nb_linear_backward_ex gives for the bias gradient of a GELU layer, on a first call and on a
second call that reuses the same built-in scratch array.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28568_b200 import binding as nb
from paper_2609_28568_b200 import synth
from parity import check_f32, f32


def test_no_alloc_rejects_sizes_beyond_the_builtin_scratch():
    L = nb.lib()
    P = 0x10000  # fake aligned address: a rejected call never touches it
    too_many = nb.NOALLOC_MAX_ELEMS // 8 + 1
    assert L.nb_gelu_dbias_noalloc(P, P, P, too_many, 8, 0, None) == nb.NB_ERR_UNSUPPORTED
    assert b"NB_NOALLOC_MAX_ELEMS" in L.nb_last_error()
    assert L.nb_gelu_dbias_noalloc(None, P, P, 8, 8, 0, None) == nb.NB_ERR_INVALID_ARG
    assert L.nb_gelu_dbias_noalloc(P, P, P, 8, 12, 0, None) == nb.NB_ERR_UNSUPPORTED


@pytest.mark.gpu
def test_no_alloc_matches_allocating_entry_point_twice_in_a_row():
    dev = "cuda"
    # two different problems back to back: the second reuses the scratch the first one filled,
    # with a smaller footprint, so stale contents beyond it must not leak into the result
    for call, (BT, OC) in enumerate(((1024, 3072), (392, 776))):
        dout = synth.normal(900 + call, (BT, OC), 1e-3, dev)
        pre = synth.normal(910 + call, (BT, OC), 1.0, dev)
        want = torch.full((OC,), 3.0, dtype=torch.float32, device=dev)
        got = torch.full((OC,), 3.0, dtype=torch.float32, device=dev)
        for accumulate in (0, 1):  # overwrite, then add on top
            nb.nb_linear_backward_ex(None, None, want, dout, None, None, pre, None, BT, 8, OC,
                                     nb.ACT_GELU, accumulate)
            nb.nb_gelu_dbias_noalloc(got, dout, pre, BT, OC, accumulate)
            torch.cuda.synchronize()
            check_f32(got, f32(want).astype(np.float64), f"call {call}, accumulate={accumulate}")
            assert np.abs(f32(got)).max() > 0
        # and on its own feet, against the oracle: the first call overwrote the 3.0 the buffer held
        # with the column sums of dout * gelu'(pre), the second added the same sums again
        dz = f32(dout).astype(np.float64) * oracle.gelu_grad(f32(pre).astype(np.float64))
        check_f32(got, 2.0 * oracle.reduce_dbias(dz.astype(np.float32)), f"call {call} against the oracle")
    # a call allocates nothing: free device memory is the same before and after a warmed-up call
    BT, OC = 1024, 3072
    dout = synth.normal(920, (BT, OC), 1e-3, dev)
    pre = synth.normal(921, (BT, OC), 1.0, dev)
    got = torch.zeros((OC,), dtype=torch.float32, device=dev)
    nb.nb_gelu_dbias_noalloc(got, dout, pre, BT, OC, 0)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    nb.nb_gelu_dbias_noalloc(got, dout, pre, BT, OC, 1)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the allocation-free entry point changed the free device memory"
    # empty batch: accumulate=0 zeroes, accumulate=1 leaves the gradient alone
    g = torch.full((64,), 2.0, dtype=torch.float32, device=dev)
    nb.nb_gelu_dbias_noalloc(g, 16, 16, 0, 64, 1)
    assert torch.all(g == 2.0)
    nb.nb_gelu_dbias_noalloc(g, 16, 16, 0, 64, 0)
    assert torch.all(g == 0.0)
    nb.nb_check_status()
