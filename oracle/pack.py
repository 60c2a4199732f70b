"""CPU oracle: GEMM-ready weight repack (naive) -- TEST INFRASTRUCTURE ONLY.

The paper's sgemm/pack kernels use a "simpler weights transformation" than
Winograd (its Section 3.1.1 and the sgemm-pack4 / pack4 rows of Table 2): a
pure re-ordering of the raw weights into the layout the GEMM consumes.  The
paper does not print that layout (it is the substrate library's), so the
layout is defined here:

    raw   W[k][c][r][s]                      (OIHW, fp32)
    pack  P[k][q],  q = (r*S + s)*C + c,     row length Qp = ceil(R*S*C / 8) * 8,
          entries with q >= R*S*C are +0.0

Every element is additionally rounded, round-to-nearest-even with integer bit
operations, to the precision the tensor core multiplies in: TF32 (10 explicit
mantissa bits, kept in an fp32 word whose low 13 bits are zero) or bf16.
"""
import numpy as np


def padded_q(C, R, S):
    return -(-(R * S * C) // 8) * 8


def pack_offset(k, c, r, s, C, R, S):
    """Element offset of raw weight (k,c,r,s) inside the packed array."""
    return k * padded_q(C, R, S) + (r * S + s) * C + c


def bf16_bits_rne(a):
    """fp32 array -> uint16 bf16 bit patterns, round to nearest even (finite inputs)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bias = np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))
    return ((bits + bias) >> np.uint64(16)).astype(np.uint16)


def tf32_round_rne(a):
    """fp32 array -> fp32 array rounded to TF32 precision, round to nearest even (finite inputs)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bias = np.uint64(0xFFF) + ((bits >> np.uint64(13)) & np.uint64(1))
    out = ((bits + bias) & np.uint64(0xFFFFE000)).astype(np.uint32)
    return out.view(np.float32).reshape(np.shape(a))


def bf16_to_f32(bits16):
    return (np.asarray(bits16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def permute_weights(w):
    """The pure re-ordering (loops over c, r, s; numpy over k): (K,C,R,S) fp32 -> (K,Qp) fp32, pad +0."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    K, C, R, S = w.shape
    Qp = padded_q(C, R, S)
    flat = np.zeros(K * Qp, dtype=np.float32)
    rows = np.arange(K) * Qp                     # pack_offset is linear in k with stride Qp
    for c in range(C):
        for r in range(R):
            for s in range(S):
                flat[rows + pack_offset(0, c, r, s, C, R, S)] = w[:, c, r, s]
    return flat.reshape(K, Qp)


def pack_weights(w, bf16=False):
    """Repack then round: returns (K, Qp) fp32 words of TF32 precision, or uint16 bf16 bits."""
    P = permute_weights(w)
    if bf16:
        return bf16_bits_rne(P)
    return tf32_round_rne(P)
