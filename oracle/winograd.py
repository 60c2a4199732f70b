"""CPU oracle: Winograd F(m x m, 3 x 3) matrices, filter transform and convolution.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this file;
it exists so the CUDA kernels can be checked against a slow, plain, fp64
restatement of the mathematics.

What it follows.  The paper's "weights transformation" stage (its Section 2 and
Figure 3) converts raw 3x3 filters into the alpha x alpha Winograd domain of
Lavin & Gray's minimal filtering algorithm, which the paper cites for its
winograd kernels; the paper itself prints no matrices.  The matrices here are
therefore built from the Cook-Toom construction (polynomial evaluation at
alpha-1 finite points plus the point at infinity) in exact rational arithmetic
and rounded once to fp64:

    Y = A^T [ (G g G^T) (.) (B^T d B) ] A          (2-D nesting of F(m,3))

Functions are deliberately literal: loops over matrix indices, numpy only for
the elementwise arithmetic over the (k, c) axes.
"""
from fractions import Fraction

import numpy as np

# Interpolation points per output tile size m (alpha = m + 2 points incl. infinity).
POINTS = {
    2: [Fraction(0), Fraction(1), Fraction(-1)],
    4: [Fraction(0), Fraction(1), Fraction(-1), Fraction(2), Fraction(-2)],
    6: [Fraction(0), Fraction(1), Fraction(-1), Fraction(2), Fraction(-2),
        Fraction(1, 2), Fraction(-1, 2)],
}


def _poly_mul(a, b):
    """Product of two polynomials given as ascending coefficient lists."""
    out = [Fraction(0)] * (len(a) + len(b) - 1)
    for i, x in enumerate(a):
        for j, y in enumerate(b):
            out[i + j] += x * y
    return out


def matrices_exact(m):
    """Return (AT, G, BT) as nested lists of Fractions for F(m, 3).

    AT is m x alpha, G is alpha x 3, BT is alpha x alpha, alpha = m + 2.
    Row j < alpha-1 belongs to the finite point p_j, the last row to infinity.
    Row 0 of G and BT is negated when its Lagrange denominator is negative, so
    that G[0] is a positive multiple of [1, 0, 0].
    """
    pts = POINTS[m]
    n = m + 2
    r = 3
    # Lagrange denominators N_j = prod_{l != j} (p_j - p_l)
    N = []
    for j, pj in enumerate(pts):
        d = Fraction(1)
        for l, pl in enumerate(pts):
            if l != j:
                d *= (pj - pl)
        N.append(d)
    G = [[pts[j] ** k / N[j] for k in range(r)] for j in range(n - 1)]
    G.append([Fraction(0), Fraction(0), Fraction(1)])
    BT = []
    for j in range(n - 1):
        poly = [Fraction(1)]
        for l, pl in enumerate(pts):
            if l != j:
                poly = _poly_mul(poly, [-pl, Fraction(1)])
        BT.append(poly + [Fraction(0)])          # degree n-2, padded to n entries
    full = [Fraction(1)]
    for pl in pts:
        full = _poly_mul(full, [-pl, Fraction(1)])
    BT.append(full)                              # degree n-1
    AT = [[pts[j] ** i for j in range(n - 1)] + [Fraction(0)] for i in range(m)]
    AT[m - 1][n - 1] = Fraction(1)
    if N[0] < 0:
        G[0] = [-v for v in G[0]]
        BT[0] = [-v for v in BT[0]]
    return AT, G, BT


def matrices(m, dtype=np.float64):
    """(AT, G, BT) rounded once from exact rationals to `dtype`."""
    AT, G, BT = matrices_exact(m)

    def conv(M):
        return np.array([[float(v) for v in row] for row in M], dtype=np.float64).astype(dtype)

    return conv(AT), conv(G), conv(BT)


def filter_transform(g, m):
    """U[xi*alpha+nu, k, c] = sum_{i,j} G[xi,i] * g[k,c,i,j] * G[nu,j], fp64.

    g: (K, C, 3, 3) array (any float dtype; promoted to fp64).
    Returns U of shape (alpha*alpha, K, C), fp64.
    """
    _, G, _ = matrices(m)
    g = np.asarray(g, dtype=np.float64)
    K, C = g.shape[:2]
    a = m + 2
    U = np.zeros((a * a, K, C), dtype=np.float64)
    for xi in range(a):
        for nu in range(a):
            acc = np.zeros((K, C), dtype=np.float64)
            for i in range(3):
                for j in range(3):
                    acc += G[xi, i] * g[:, :, i, j] * G[nu, j]
            U[xi * a + nu] = acc
    return U


def pad_channels(U, Cp):
    """Zero-pad the last axis of U (.., C) to Cp entries (device layout helper)."""
    if U.shape[-1] == Cp:
        return U
    out = np.zeros(U.shape[:-1] + (Cp,), dtype=U.dtype)
    out[..., :U.shape[-1]] = U
    return out


def input_transform(x, m, pad):
    """V[xi*alpha+nu, t, c] = (B^T d B)[xi,nu] for every tile t and channel c.

    x: (C, H, W); tiles of alpha x alpha at stride m starting at -pad, zero
    outside the image; t = th * TW + tw.  Returns (V, TH, TW).
    """
    _, _, BT = matrices(m)
    x = np.asarray(x, dtype=np.float64)
    C, H, W = x.shape
    a = m + 2
    OH, OW = H + 2 * pad - 2, W + 2 * pad - 2
    TH, TW = -(-OH // m), -(-OW // m)
    V = np.zeros((a * a, TH * TW, C), dtype=np.float64)
    for th in range(TH):
        for tw in range(TW):
            d = np.zeros((C, a, a), dtype=np.float64)
            for i in range(a):
                for j in range(a):
                    h, w = th * m + i - pad, tw * m + j - pad
                    if 0 <= h < H and 0 <= w < W:
                        d[:, i, j] = x[:, h, w]
            v = np.einsum("xi,cij,yj->cxy", BT, d, BT)
            V[:, th * TW + tw, :] = v.reshape(C, a * a).T
    return V, TH, TW


def output_transform(Mt, m, K, OH, OW, TH, TW):
    """Y tile = A^T M A, written at (th*m, tw*m), clipped to OH x OW."""
    AT, _, _ = matrices(m)
    a = m + 2
    Y = np.zeros((K, OH, OW), dtype=np.float64)
    for th in range(TH):
        for tw in range(TW):
            Mx = Mt[:, th * TW + tw, :].T.reshape(K, a, a)
            y = np.einsum("ix,kxy,jy->kij", AT, Mx, AT)
            h0, w0 = th * m, tw * m
            hh, ww = min(m, OH - h0), min(m, OW - w0)
            Y[:, h0:h0 + hh, w0:w0 + ww] = y[:, :hh, :ww]
    return Y


def winograd_conv(x, w, m, pad):
    """Full fp64 Winograd convolution (3x3, stride 1, groups 1) of x (C,H,W) with w (K,C,3,3)."""
    x = np.asarray(x, dtype=np.float64)
    K = w.shape[0]
    C, H, W = x.shape
    OH, OW = H + 2 * pad - 2, W + 2 * pad - 2
    U = filter_transform(w, m)                       # (a*a, K, C)
    V, TH, TW = input_transform(x, m, pad)           # (a*a, T, C)
    a2 = (m + 2) ** 2
    Mt = np.zeros((a2, TH * TW, K), dtype=np.float64)
    for p in range(a2):
        Mt[p] = V[p] @ U[p].T                        # sum over channels
    return output_transform(Mt, m, K, OH, OW, TH, TW)
