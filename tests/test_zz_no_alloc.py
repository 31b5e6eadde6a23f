"""cq_gemv_static, the entry point for callers that may not allocate device memory, against the
ordinary cq_gemm on the same inputs.  Collected last on purpose: it is an integration add-on, and a
run that stops at the first failure has by then exercised every parity test."""
import pytest
import torch

import datagen
import paper_2608_06763_b200 as cq
from util import logical_case, x_to_device

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_cq_gemm_twice_in_a_row():
    # a plug-in that owns nothing but its inputs and outputs calls the library back to back: the same
    # kernel on the same inputs must give the same bits as cq_gemm, and the call must not allocate
    # the set-up call of this device (done at start-up by such a caller): it resolves the built-in array, and
    # with lazy module loading this is also when the driver commits the array's memory
    c0 = logical_case(128, 256, 4, 128, seed=899)
    cq.cq_gemv_static(c0.pw, x_to_device(datagen.activations(1, 256, seed=899)))
    for B, G, seed in ((4, 128, 900), (6, 64, 910)):
        c = logical_case(640, 2048, B, G, seed=seed)
        for M in (1, 7, 16):   # one token, one token block, two token blocks; later shapes find the leftovers of earlier calls
            x = x_to_device(datagen.activations(M, 2048, seed=seed + M))
            want = cq.cq_gemm(c.pw, x, cq.CQ_MODEL_DTYPE)
            out = torch.empty_like(want)
            for call in range(2):
                torch.cuda.synchronize()
                free_before = torch.cuda.mem_get_info()[0]
                got = cq.cq_gemv_static(c.pw, x, out)
                torch.cuda.synchronize()
                free_after = torch.cuda.mem_get_info()[0]     # read before torch allocates anything for the comparison
                assert torch.equal(got.view(torch.int16), want.view(torch.int16)), (B, G, M, call)
                assert free_after == free_before, "the call changed the device's free memory"
                got.zero_()


def test_static_scratch_entry_rejects_what_does_not_fit():
    L = cq.lib()
    one = 16
    assert L.cq_gemv_static(one, 4, 128, one, one, 17, 128, 128, None) == -2          # more rows than the small-M path takes
    assert L.cq_gemv_static(one, 4, 128, one, one, 16, 1 << 29, 128, None) == -4      # its arrival counters alone exceed the built-in scratch
    assert L.cq_gemv_static(None, 4, 128, one, one, 1, 128, 128, None) == -1
