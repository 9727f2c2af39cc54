"""The allocation-free threshold entry point against the oracle and against the plan-based entry point.

dnns_magnitude_threshold_static exists for callers that may not allocate device memory (a plug-in
inside another framework's planned step, a callback under a locked allocator): its scratch is a
fixed array inside the library.  Here it is called through the C ABI several times in a row - later
calls on different data and other k, so that anything an earlier call left in the shared array
would show - and each record must equal, bit for bit, the oracle's record for the same tensor (a full
sort on the CPU) and what dnns_magnitude_threshold gives for it as a one-tensor model; the free device
memory must not change across a call.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
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
    # ragged sizes, several tiles; then a smaller tensor; then nothing and everything masked
    cases = [(1009, 991, 900_000), (509, 503, 3), (509, 503, 0), (64, 77, 64 * 77)]
    for i, (rows, cols, k) in enumerate(cases):
        n = rows * cols
        x = rng.standard_normal(n).astype(np.float32)
        x[rng.integers(0, n, n // 7)] = 0.0
        x[rng.integers(0, n, n // 9)] = np.float32(0.5)       # duplicates: ties split inside the tensor
        if i == 1:
            k = int(np.count_nonzero(x == 0)) + int(np.count_nonzero(x == 0.5)) // 2   # tau lands on the ties
        dm, via_plan = record_via_plan(x, rows, cols, dtype, k)
        want = O.threshold(O.OracleModel(one_tensor(x, rows, cols), dtype), W.SCOPE_GLOBAL, np.array([[k]], np.uint64))[0, 0]
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.dnns_magnitude_threshold_static(dm.weights.data_ptr(), dtype, n, k, thr.data_ptr(), stream)
        torch.cuda.synchronize()
        if i > 0:          # (the very first call on a device may load the library's device code)
            assert torch.cuda.mem_get_info()[0] == free_before
        got = thr.cpu().numpy().view(REC_DTYPE)[0]
        for f in ("tau_bits", "n_below", "n_tie", "n_equal"):
            assert int(got[f]) == int(want[f]), (i, f)               # the oracle's record
            assert int(got[f]) == int(via_plan[f]), (i, f)           # ... which the plan-based call gives too
        assert int(got["n_below"]) + int(got["n_tie"]) == k


def test_static_threshold_inside_a_stream_capture():
    """Once a device has seen a call, further calls hold nothing but kernel launches and a memset, with the
    descriptors of the call as kernel arguments: a captured call replays on the data it was captured with."""
    rng = np.random.default_rng(6)
    n, k = 300_001, 123_456
    x = rng.standard_normal(n).astype(np.float32)
    w = torch.from_numpy(x).cuda()
    thr = torch.zeros(REC_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        B.dnns_magnitude_threshold_static(w.data_ptr(), B.DNNS_F32, n, 1, thr.data_ptr(), s.cuda_stream)   # set-up done
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            B.dnns_magnitude_threshold_static(w.data_ptr(), B.DNNS_F32, n, k, thr.data_ptr(), s.cuda_stream)
        thr.zero_()
        g.replay()
        s.synchronize()
    got = thr.cpu().numpy().view(REC_DTYPE)[0]
    keys = np.sort(x.view(np.uint32) & 0x7FFFFFFF)
    assert int(got["tau_bits"]) == int(keys[k - 1]) and int(got["n_below"]) == int(np.count_nonzero(keys < keys[k - 1]))


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
