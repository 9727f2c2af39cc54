"""Small helpers shared by CPU and GPU tests."""
import copy


def compacted_workload(wl, keep_count, weights, bn_params, biases):
    """The rebuilt variant as a workload of its own (smaller extents, same wiring)."""
    cw = copy.deepcopy(wl)
    for g, c in zip(cw.groups, keep_count):
        g.C = int(c)
    for t in cw.tensors:
        t.O = cw.groups[t.out_group].C
        t.I = cw.groups[t.in_group].C * t.in_spatial
    for b in cw.bns:
        b.C = cw.groups[cw.tensors[b.tensor].out_group].C
    cw.weights, cw.bn_params, cw.biases = weights, bn_params, biases
    return cw
