"""Test-only network executor: runs a workload's op list with torch CPU ops in float64.

A neutral library executor (conv2d / batch_norm / linear); it is never timed and
is not part of the method.  Used for the "pruned model computes what the sparse
model computes" check (Section I and Section IV-B-2: pruning is at no cost to the
accuracy of the sparse model).
"""
import numpy as np
import torch
import torch.nn.functional as F


def to_f64(w, is_bf16):
    if is_bf16:
        w = (w.astype(np.uint32) << 16).view(np.float32)
    return torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).double()


def forward(wl, weights, bn_params, biases, x, is_bf16=False):
    """weights[t]: array (O, I, KH, KW); bn_params[b]: (gamma, beta, mean, var); biases[t] or None."""
    act = {"x": x.double()}
    for op in wl.ops:
        kind = op[0]
        if kind == "conv":
            _, t, src, dst, stride, pad = op
            act[dst] = F.conv2d(act[src], to_f64(weights[t], is_bf16), None, stride, pad)
        elif kind == "bn":
            _, b, src, dst = op
            g, be, mu, va = [torch.from_numpy(np.asarray(v, np.float32)).double() for v in bn_params[b]]
            act[dst] = F.batch_norm(act[src], mu, va, g, be, False, 0.0, wl.bns[b].eps)
        elif kind == "relu":
            act[op[2]] = torch.relu(act[op[1]])
        elif kind == "add":
            act[op[3]] = act[op[1]] + act[op[2]]
        elif kind == "maxpool":
            _, src, dst, k, s, p = op
            act[dst] = F.max_pool2d(act[src], k, s, p)
        elif kind == "gap":
            act[op[2]] = act[op[1]].mean(dim=(2, 3))
        elif kind == "fc":
            _, t, src, dst = op
            w = to_f64(weights[t], is_bf16).flatten(1)
            bias = None if biases[t] is None else torch.from_numpy(biases[t]).double()
            act[dst] = F.linear(act[src], w, bias)
        else:
            raise ValueError(kind)
    return act["out"]


def silenced_reference(wl, masked_weights, bn_params, biases, keep_bits):
    """The masked model with every removed channel's producer output forced to zero.

    For a removed channel j of a group, each producer's BN gamma and beta (or its
    bias when it has no BN) are zeroed in a copy, so the channel carries exactly
    zero; the weights are left as they are.
    """
    bn = [tuple(np.array(v, np.float32) for v in p) for p in bn_params]
    bs = [None if b is None else np.array(b, np.float32) for b in biases]
    bn_of = {b.tensor: i for i, b in enumerate(wl.bns)}
    for ti, t in enumerate(wl.tensors):
        kb = keep_bits[t.out_group]
        removed = [j for j in range(t.O) if not (kb[j >> 5] >> (j & 31)) & 1]
        if not removed:
            continue
        if ti in bn_of:
            g, be, mu, va = bn[bn_of[ti]]
            g[removed] = 0.0
            be[removed] = 0.0
        elif bs[ti] is not None:
            bs[ti][removed] = 0.0
        else:
            # no BN and no bias: silence the filters themselves
            masked_weights = list(masked_weights)
            w = masked_weights[ti].copy()
            w[removed] = 0
            masked_weights[ti] = w
    return masked_weights, bn, bs
