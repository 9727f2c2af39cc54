"""Run by tests/test_gpu_bounds_check.py in a process of its own, with DNNS_LIBRARY pointing at the checked
build of the library: the whole path on small models (odd shapes, ties at zero, every rebuild variant), every
output still compared with the oracle, then the number of index violations the kernels counted."""
import ctypes
import sys

import numpy as np

sys.path.insert(0, __file__.rsplit("/", 2)[0])
sys.path.insert(0, __file__.rsplit("/", 1)[0])

from gpu_compare import compare_portfolio, compare_sparse_free          # noqa: E402
from oracle import oracle as O                     # noqa: E402
from test_gpu_cascade import run_case              # noqa: E402
from paper_2309_06973_b200 import binding as B     # noqa: E402
from paper_2309_06973_b200 import workloads as W   # noqa: E402


def main():
    L = B.lib()
    L.dnns_check_bounds_violations.restype = ctypes.c_uint
    assert L.dnns_check_bounds_violations() == 0
    odd = W.chain([37, 70, 129, 33], seed=5, kernel=5, planted_frac=0.2)
    ties = W.chain([48, 64, 80], seed=7, planted_frac=0.5)
    n = ties.n_prunable
    nz0 = sum(int(np.count_nonzero(w.view(np.uint32) & 0x7FFFFFFF == 0)) for w in ties.weights)
    ties.ks = np.array([1, nz0 // 2, nz0 + 5, n * 3 // 4], np.uint64)[:, None]     # thresholds at zero that split their ties
    for dtype in (B.DNNS_F32, B.DNNS_BF16):
        for wl in (W.toy(), W.small_resnet(seed=3), odd, ties):
            compare_portfolio(wl, dtype)
            compare_portfolio(wl, dtype, multi=2, multi_plan=True)
            compare_portfolio(wl, dtype, multi=3, no_store=True)
            compare_sparse_free(wl, dtype)                          # no sparse model: flags from the maxima, masking rebuild
            compare_sparse_free(wl, dtype, one_launch=True)
            run_case(wl, dtype, len(wl.ks) - 1, O.RULE_PRODUCER | O.RULE_CONSUMER, 1, 8)   # fixed-point propagation
    print("violations", L.dnns_check_bounds_violations())


if __name__ == "__main__":
    main()
