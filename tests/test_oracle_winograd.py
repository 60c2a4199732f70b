"""Pins for oracle/winograd.py (CPU only)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import winograd as ow
from oracle import conv as oc


@pytest.mark.parametrize("m", [2, 4, 6])
def test_exact_1d_correlation_identity(m):
    """A^T[(G g) . (B^T d)] equals y_i = sum_a d[i+a] g[a] exactly on every basis pair."""
    AT, G, BT = ow.matrices_exact(m)
    n = m + 2
    for a in range(3):
        for b in range(n):
            Gg = [G[j][a] for j in range(n)]
            Bd = [BT[j][b] for j in range(n)]
            prod = [Gg[j] * Bd[j] for j in range(n)]
            y = [sum(AT[i][j] * prod[j] for j in range(n)) for i in range(m)]
            want = [Fraction(1) if i + a == b else Fraction(0) for i in range(m)]
            assert y == want, (m, a, b)


def test_f23_small_integers_exact_in_float():
    """F(2,3) reproduces direct 1-D correlation exactly on small integers in fp64."""
    AT, G, BT = ow.matrices(2)
    rng = np.random.default_rng(1)
    for _ in range(50):
        g = rng.integers(-8, 9, 3).astype(np.float64)
        d = rng.integers(-8, 9, 4).astype(np.float64)
        y = AT @ ((G @ g) * (BT @ d))
        want = np.array([d[0:3] @ g, d[1:4] @ g])
        assert np.array_equal(y, want)


@pytest.mark.parametrize("m", [2, 4, 6])
def test_matrix_shapes_and_first_rows(m):
    AT, G, BT = ow.matrices_exact(m)
    n = m + 2
    assert len(AT) == m and len(G) == n and len(BT) == n
    assert all(len(r) == n for r in AT) and all(len(r) == 3 for r in G) and all(len(r) == n for r in BT)
    assert G[0][1] == 0 and G[0][2] == 0 and G[0][0] > 0      # normalisation: point 0
    assert G[n - 1] == [0, 0, 1]                               # point at infinity


@pytest.mark.parametrize("m", [2, 4, 6])
def test_filter_transform_roundtrip(m):
    """G has full column rank, so G+ U G+^T recovers g."""
    _, G, _ = ow.matrices(m)
    rng = np.random.default_rng(2)
    g = rng.standard_normal((5, 7, 3, 3))
    U = ow.filter_transform(g, m)
    a = m + 2
    Gp = np.linalg.inv(G.T @ G) @ G.T
    Um = U.reshape(a, a, 5, 7)
    back = np.einsum("ix,xykc,jy->kcij", Gp, Um, Gp)
    assert np.max(np.abs(back - g)) < 1e-12


@pytest.mark.parametrize("m", [2, 4, 6])
def test_filter_transform_single_tap_is_outer_product(m):
    """g = unit tap at (i0,j0) gives U[xi,nu] = G[xi,i0]*G[nu,j0]; asymmetric taps catch a transpose."""
    _, G, _ = ow.matrices(m)
    a = m + 2
    for (i0, j0) in [(0, 1), (2, 0), (1, 1)]:
        g = np.zeros((1, 1, 3, 3))
        g[0, 0, i0, j0] = 1.0
        U = ow.filter_transform(g, m).reshape(a, a)
        want = np.outer(G[:, i0], G[:, j0])
        assert np.allclose(U, want, rtol=0, atol=1e-15)


def test_filter_transform_layout_plane_k_c():
    """Plane index is xi*alpha+nu, then k, then c."""
    g = np.zeros((3, 2, 3, 3))
    g[2, 1, 0, 0] = 1.0                       # only filter (k=2, c=1) is non-zero
    U = ow.filter_transform(g, 2)
    assert U.shape == (16, 3, 2)
    nz = np.argwhere(np.abs(U) > 0)
    assert set(map(tuple, nz[:, 1:])) == {(2, 1)}
    # tap (0,0): U[xi,nu] = G[xi,0]*G[nu,0]; G[:,0] = [1, 1/2, 1/2, 0]
    assert U[0 * 4 + 1, 2, 1] == 0.5 and U[1 * 4 + 0, 2, 1] == 0.5 and U[3 * 4 + 3, 2, 1] == 0.0


def test_f63_plane_count_matches_paper_figure3_and_table2_ratio():
    """F(6,3) yields 8x8 = 64 planes per filter (the paper's Figure 3 shape); the byte
    expansion 64/9 is close to Table 2's read-cache / read-raw ratio 5.23/0.70."""
    U = ow.filter_transform(np.ones((4, 4, 3, 3)), 6)
    assert U.shape[0] == 64
    ratio = 64.0 / 9.0
    assert abs(ratio - 5.23 / 0.70) / ratio < 0.06


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("shape", [(3, 5, 5, 1), (4, 7, 9, 1), (2, 14, 5, 0), (5, 9, 14, 1), (1, 3, 3, 1)])
def test_winograd_conv_equals_direct(m, shape):
    """Pins tiling, zero-padded edge tiles and clipped outputs."""
    C, H, W, pad = shape
    rng = np.random.default_rng([m, C, H, W])
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = rng.standard_normal((6, C, 3, 3)).astype(np.float32)
    y = ow.winograd_conv(x, w, m, pad)
    ref = oc.direct_conv(x, w, None, 1, pad, 1)
    assert y.shape == ref.shape
    assert np.max(np.abs(y - ref)) <= 1e-10 * max(1.0, np.max(np.abs(ref)))


def test_input_transform_constant_tile_f23():
    """A constant interior tile d = 1 gives V = (B^T 1)(B^T 1)^T; row sums of B^T for F(2,3) are [0,2,0,0]."""
    x = np.ones((1, 8, 8), dtype=np.float32)
    V, TH, TW = ow.input_transform(x, 2, 0)
    assert (TH, TW) == (3, 3)
    v = V[:, 4, 0].reshape(4, 4)
    want = np.outer([0, 2, 0, 0], [0, 2, 0, 0])
    assert np.array_equal(v, want)
