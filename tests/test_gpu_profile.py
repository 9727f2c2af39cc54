"""dnns_plan_profile / dnns_plan_profile_read: launches are counted per kernel while the profile is on,
and only then."""
import pytest
import torch

from paper_2309_06973_b200 import binding as B
from paper_2309_06973_b200 import workloads as W
from paper_2309_06973_b200.runtime import DeviceModel, Session

pytestmark = pytest.mark.gpu


def test_profile_counts_kernels_only_while_on():
    wl = W.resnet56()
    dm = DeviceModel(wl, B.DNNS_F32)
    V = len(wl.ks)
    ses = Session(dm, wl.scope, V)
    ses.magnitude_threshold(wl.ks)
    ses.variant(0, fused=True)                       # profile off: nothing recorded
    assert ses.kernel_time("k_sweep") == (0.0, 0)
    ses.profile(True)
    before = ses.launch_count()
    ses.magnitude_threshold(wl.ks)
    for v in range(3):
        ses.variant(v, fused=True)
    ses.profile(False)
    launched = ses.launch_count() - before
    ses.variant(3, fused=True)                       # off again
    per_kernel = {k: ses.kernel_time(k) for k in ["k_hist1", "k_select1", "k_hist2", "k_select2", "k_tie_find", "k_tie_pick", "k_ties", "k_tie_scan", "k_extrema_rows", "k_extrema_sweep",
                                                  "k_sweep", "k_flags", "k_propagate", "k_rebuild_layout", "k_compact"]}
    assert per_kernel["k_sweep"][1] == 3 and per_kernel["k_flags"][1] == 3 and per_kernel["k_propagate"][1] == 3
    assert per_kernel["k_hist1"][1] == 1 and per_kernel["k_compact"][1] >= 3 and per_kernel["k_rebuild_layout"][1] == 3
    assert sum(n for _, n in per_kernel.values()) == launched
    assert all(ms > 0 for ms, n in per_kernel.values() if n)
    assert ses.kernel_time("k_")[1] == launched      # prefix match
    ses.profile(True)                                # switching on drops the old records
    assert ses.kernel_time("k_sweep") == (0.0, 0)
    ses.profile(False)
    assert ses.device_status() == B.DNNS_OK
    ses.close()
