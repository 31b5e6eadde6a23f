"""cq_gemv_static, the entry point for callers that may not allocate device memory, against the
ordinary cq_gemm on the same inputs.  Collected last on purpose: it is an integration add-on, and a
run that stops at the first failure has by then exercised every parity test."""
import numpy as np
import pytest
import torch

import datagen
import paper_2608_06763_b200 as cq
from util import logical_case, x_to_device, y_to_numpy

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_cq_gemm_twice_in_a_row():
    # a plug-in that owns nothing but its inputs and outputs calls the library back to back
    c = logical_case(640, 2048, 4, 128, seed=900)
    for M, seed in ((1, 901), (7, 902)):   # the second shape finds the first call's leftovers in the array
        x = x_to_device(datagen.activations(M, 2048, seed=seed))
        want = y_to_numpy(cq.cq_gemm(c.pw, x, cq.CQ_MODEL_DTYPE))
        for call in range(2):
            got = y_to_numpy(cq.cq_gemv_static(c.pw, x))
            torch.cuda.synchronize()
            fro = np.linalg.norm(got - want) / np.linalg.norm(want)
            mx = np.abs(got - want).max() / np.abs(want).max()
            assert fro <= 5e-3 and mx <= 1e-2, (M, call, fro, mx)


def test_static_scratch_entry_rejects_what_does_not_fit():
    L = cq.lib()
    one = 16
    assert L.cq_gemv_static(one, 4, 128, one, one, 17, 128, 128, None) == -2          # more rows than the small-M path takes
    assert L.cq_gemv_static(one, 4, 128, one, one, 16, 1 << 29, 128, None) == -4      # its arrival counters alone exceed the built-in scratch
    assert L.cq_gemv_static(None, 4, 128, one, one, 1, 128, 128, None) == -1
