"""CPU oracle: whole-model chain in fp64 -- TEST INFRASTRUCTURE ONLY.

Walks the layer list in order (the layer-by-layer computation pattern the
paper's pipeline relies on, its Section 2 "Opportunities"), evaluating every
conv with the direct definition and keeping every layer's activation so a GPU
layer can be checked with oracle-fed inputs.
"""
import numpy as np

from . import conv as oconv

OP_CONV, OP_MAXPOOL, OP_GAVGPOOL = 0, 1, 2


def run_layer(L, x, w=None, bias=None, addend=None):
    """One layer on x (C,H,W); conv -> (+bias) -> (+addend) -> activation."""
    if L["op"] == OP_CONV:
        y = oconv.direct_conv(x, w, bias, L["stride"], L["pad"], L["groups"])
        if addend is not None:
            y = y + addend
        return oconv.activation(y, L["act"])
    if L["op"] == OP_MAXPOOL:
        return oconv.maxpool(np.asarray(x, dtype=np.float64), L["R"], L["stride"], L["pad"])
    if L["op"] == OP_GAVGPOOL:
        return oconv.gavgpool(np.asarray(x, dtype=np.float64))
    raise ValueError("unknown op")


def run_model(layers, weights, biases, x):
    """x: (1,C,H,W) or (C,H,W) fp32.  Returns the list of fp64 activations, one per layer."""
    x = np.asarray(x)
    if x.ndim == 4:
        x = x[0]
    acts = []
    for i, L in enumerate(layers):
        src = x if L["in0"] < 0 else acts[L["in0"]]
        add = None if L["in1"] < 0 else acts[L["in1"]]
        acts.append(run_layer(L, src, weights[i], biases[i], add))
    return acts
