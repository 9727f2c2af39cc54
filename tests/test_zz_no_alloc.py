"""The allocation-free threshold entry point against the plan-based one.

dnns_magnitude_threshold_static exists for callers that may not allocate device memory (a plug-in
inside another framework's planned step, a callback under a locked allocator): its scratch is a
fixed array inside the library.  Here it is called through the C ABI twice in a row - the second
call on different data and another k, so that anything the first call left in the shared array
would show - and each record must equal, bit for bit, what dnns_magnitude_threshold gives for the
same tensor as a one-tensor model.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import REC_DTYPE, DeviceModel, Session

pytestmark = pytest.mark.gpu


def one_tensor(values, rows, cols):
    wl = W.Workload("flat", 0, W.SCOPE_GLOBAL, [W.TensorSpec("w", rows, cols, 1, 1, 1, 0)], [],
                    [W.GroupSpec(cols, W.GROUP_FROZEN), W.GroupSpec(rows, W.GROUP_FROZEN)], [], 1)
    wl.weights, wl.biases, wl.bn_params = [values.reshape(rows, cols, 1, 1)], [None], []
    return wl


def record_via_plan(values, rows, cols, dtype, k):
    wl = one_tensor(values, rows, cols)
    dm = DeviceModel(wl, dtype)
    ses = Session(dm, W.SCOPE_GLOBAL, 1, want_mask_bits=False, want_nz_map=False)
    ses.magnitude_threshold(np.array([[k]], np.uint64))
    rec = ses.records()[0, 0]
    ses.close()
    return dm, rec


@pytest.mark.parametrize("dtype", [B.DNNS_F32, B.DNNS_BF16])
def test_static_threshold_matches_plan_threshold_twice(dtype):
    rng = np.random.default_rng(5)
    thr = torch.zeros(REC_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    cases = [(1009, 991, 900_000), (509, 503, 3)]     # ragged sizes, several tiles; then a smaller tensor
    for i, (rows, cols, k) in enumerate(cases):
        n = rows * cols
        x = rng.standard_normal(n).astype(np.float32)
        x[rng.integers(0, n, n // 7)] = 0.0
        x[rng.integers(0, n, n // 9)] = np.float32(0.5)       # duplicates: ties split inside the tensor
        if i == 1:
            k = int(np.count_nonzero(x == 0)) + int(np.count_nonzero(x == 0.5)) // 2   # tau lands on the ties
        dm, want = record_via_plan(x, rows, cols, dtype, k)
        B.dnns_magnitude_threshold_static(dm.weights.data_ptr(), dtype, n, k, thr.data_ptr(), stream)
        torch.cuda.synchronize()
        got = thr.cpu().numpy().view(REC_DTYPE)[0]
        for f in ("tau_bits", "n_below", "n_tie", "n_equal"):
            assert int(got[f]) == int(want[f]), (i, f)
        assert int(got["n_below"]) + int(got["n_tie"]) == k


def test_static_threshold_rejects_what_it_cannot_hold():
    L = B.lib()
    buf = torch.zeros(64, dtype=torch.uint8, device="cuda")
    thr = torch.zeros(REC_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    p, t = buf.data_ptr(), thr.data_ptr()
    assert L.dnns_magnitude_threshold_static(p, B.DNNS_F32, B.DNNS_STATIC_MAX_NUMEL + 1, 1, t, None) == B.DNNS_ERR_STATIC_LIMIT
    assert L.dnns_magnitude_threshold_static(p, B.DNNS_F32, 16, 17, t, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_magnitude_threshold_static(p + 4, B.DNNS_F32, 8, 1, t, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_magnitude_threshold_static(None, B.DNNS_F32, 8, 1, t, None) == B.DNNS_ERR_INVALID_ARG
    assert L.dnns_magnitude_threshold_static(p, 9, 8, 1, t, None) == B.DNNS_ERR_UNSUPPORTED
    assert "DNNS_STATIC_MAX_NUMEL" in B.dnns_status_string(B.DNNS_ERR_STATIC_LIMIT)
