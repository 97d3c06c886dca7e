"""The tensor-core path stores hidden activations as fp16 and saturates at 65504.  For inputs in [0, 1] the largest
activation a layer can produce is bounded by sum|w| * (bound of its input) + |b| per output unit; this pins that the
seeded weights of every configuration stay far below the saturation point, so the clamp never acts in the parity
runs (and states the condition under which it cannot act for other weights)."""
import numpy as np

import hts_workloads as wl

FP16_MAX = 65504.0


def activation_bounds(params):
    """Worst-case activation after each hidden layer for inputs in [0, 1] (interval arithmetic on |w|)."""
    bound, out = 1.0, {}
    for name in ("conv1", "conv2", "conv3", "fc"):
        w, b = np.abs(params[name + "_w"].astype(np.float64)), np.abs(params[name + "_b"].astype(np.float64))
        per_unit = w.reshape(w.shape[0], -1).sum(axis=1) * bound + b
        bound = float(per_unit.max())
        out[name] = bound
    return out


def test_seeded_weights_cannot_saturate_fp16_activations():
    for ci in (2, 3, 4, 5):
        cfg = wl.CONFIGS[ci]
        for sub in (0, 1):
            b = activation_bounds(wl.make_weights(cfg, sub=sub))
            # conv1..conv3 outputs are what the kernels store as fp16 (the FC output stays fp32)
            assert max(b["conv1"], b["conv2"], b["conv3"]) < FP16_MAX / 2, (ci, sub, b)


def test_bound_is_attained_by_a_worst_case_input():
    # one output unit of conv1 with non-negative weights, all-ones input: the activation equals the bound
    cfg = wl.CONFIGS[2]
    p = wl.make_weights(cfg)
    w = np.abs(p["conv1_w"][:1].astype(np.float64)); b = np.abs(p["conv1_b"][:1].astype(np.float64))
    q = dict(p); q["conv1_w"] = w; q["conv1_b"] = b
    assert np.isclose(activation_bounds(q)["conv1"], w.sum() + b[0])
