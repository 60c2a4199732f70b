"""Seeded generators for weights and inputs (numpy only, no method arithmetic)."""
import numpy as np

from .configs import OP_CONV


def make_weights(layers, seed=0):
    """He-normal fp32 OIHW weights per conv layer; None for non-conv layers.

    Layer i draws from default_rng([seed, i]); std = sqrt(2 / (Cg*R*S)).
    Returns (weights, biases); biases[i] is None unless the layer has one.
    """
    ws, bs = [], []
    for i, L in enumerate(layers):
        if L["op"] != OP_CONV:
            ws.append(None)
            bs.append(None)
            continue
        cg = L["C"] // L["groups"]
        shape = (L["K"], cg, L["R"], L["S"])
        rng = np.random.default_rng([seed, i])
        w = rng.standard_normal(shape, dtype=np.float32)
        w = (w * np.float32(np.sqrt(2.0 / (cg * L["R"] * L["S"])))).astype(np.float32)
        ws.append(w)
        if L["has_bias"]:
            b = np.random.default_rng([seed, i, 1]).uniform(-0.1, 0.1, L["K"]).astype(np.float32)
        else:
            b = None
        bs.append(b)
    return ws, bs


def make_input(layers, seed=0):
    """Uniform[-1,1] fp32 NCHW input (N=1) for the model's first layer."""
    L = layers[0]
    rng = np.random.default_rng([seed, 10 ** 6])
    return rng.uniform(-1.0, 1.0, (1, L["C"], L["H"], L["W"])).astype(np.float32)


def weight_blob(layers, weights, biases, align=256):
    """Concatenate all weights/biases into one byte blob with aligned offsets.

    Returns (blob uint8 array, w_off list, b_off list); offsets are bytes,
    0 for layers without weights / bias.
    """
    w_off, b_off, chunks, pos = [], [], [], 0

    def put(a):
        nonlocal pos
        pad = (-pos) % align
        if pad:
            chunks.append(np.zeros(pad, np.uint8))
            pos += pad
        off = pos
        raw = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
        chunks.append(raw)
        pos += raw.size
        return off

    for w, b in zip(weights, biases):
        w_off.append(put(w) if w is not None else 0)
        b_off.append(put(b) if b is not None else 0)
    pad = (-pos) % align
    if pad:
        chunks.append(np.zeros(pad, np.uint8))
    blob = np.concatenate(chunks) if chunks else np.zeros(0, np.uint8)
    return blob, w_off, b_off
