"""Pins for the float64 oracle: closed forms, brute force, invariants and library special cases.

The paper prints no worked numerical transform, so the oracle is pinned to what its equations fix:
Eq. 14 (kernel and sign), Eq. 11 (the triple sum), Eq. 12 (Kronecker form and its ordering), Eq. 5
(which side each axis multiplies), Eq. 3 (Vandermonde rows/columns), Eq. 17 (the two-stage refactoring).
Each test is chosen so that a dropped term, wrong sign, swapped axis or transposed operand fails it.
"""
import cmath
import os
from fractions import Fraction

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def rng_cube(shape, seed, dtype=np.complex128):
    r = np.random.default_rng(seed)
    return (r.standard_normal(shape) + 1j * r.standard_normal(shape)).astype(dtype)


# ---------------------------------------------------------------- 1D kernel, sign, scaling

def test_dft4_matrix_matches_golden(oracle):
    rows = [l for l in open(os.path.join(GOLDEN, "dft4_forward_matrix.txt")) if not l.startswith("#")]
    vals = np.array([[float(t) for t in l.split()] for l in rows])
    G = vals[:, 0::2] + 1j * vals[:, 1::2]
    M = oracle.axis_matrix(4, sign=-1)
    assert np.array_equal(M, G)  # exact at quarter turns
    assert np.array_equal(oracle.axis_matrix(4, sign=+1), G.conj())
    assert np.array_equal(oracle.axis_matrix(2, sign=-1), np.array([[1, 1], [1, -1]], dtype=complex))


def test_delta_gives_all_ones_and_pure_phase(oracle):
    n0, n1, n2 = 6, 5, 8
    x = np.zeros((n0, n1, n2), dtype=np.complex128)
    x[0, 0, 0] = 1.0
    X = oracle.dft3d(x)
    assert np.allclose(X, 1.0, atol=1e-15)
    # delta at (a,b,c): X[k] = exp(-2 pi i (k0 a/n0 + k1 b/n1 + k2 c/n2)); distinct a,b,c and sizes
    a, b, c = 2, 3, 5
    x[:] = 0
    x[a, b, c] = 1.0
    X = oracle.dft3d(x)
    k0, k1, k2 = np.meshgrid(np.arange(n0), np.arange(n1), np.arange(n2), indexing="ij")
    want = np.exp(-2j * np.pi * (k0 * a / n0 + k1 * b / n1 + k2 * c / n2))
    assert np.max(np.abs(X - want)) < 1e-14
    # conjugate kernel flips the sign of the phase
    Xi = oracle.dft3d(x, sign=+1)
    assert np.max(np.abs(Xi - want.conj())) < 1e-14


def test_single_exponential_gives_delta(oracle):
    n0, n1, n2 = 4, 6, 10
    f = (1, 4, 7)
    a, b, c = np.meshgrid(np.arange(n0), np.arange(n1), np.arange(n2), indexing="ij")
    x = np.exp(+2j * np.pi * (f[0] * a / n0 + f[1] * b / n1 + f[2] * c / n2))
    X = oracle.dft3d(x)
    want = np.zeros_like(X)
    want[f] = n0 * n1 * n2
    assert np.max(np.abs(X - want)) < 1e-11


def test_against_numpy_fft_noncubic(oracle):
    for shape, seed in (((2, 3, 5), 1), ((6, 4, 8), 2), ((1, 7, 3), 3), ((16, 1, 12), 4)):
        x = rng_cube(shape, seed)
        assert oracle.rel_l2(oracle.dft3d(x), np.fft.fftn(x)) < 1e-13
        # scaled inverse is numpy's ifftn
        assert oracle.rel_l2(oracle.dft3d(x, sign=+1, scaled_inverse=True), np.fft.ifftn(x)) < 1e-13
        # unscaled conjugate kernel
        assert oracle.rel_l2(oracle.dft3d(x, sign=+1), np.fft.ifftn(x) * np.prod(shape)) < 1e-13


def test_single_axis_passes_against_numpy(oracle):
    x = rng_cube((3, 4, 5), 11)
    for axis in range(3):
        assert oracle.rel_l2(oracle.dft_axis(x, axis), np.fft.fft(x, axis=axis)) < 1e-13


# ---------------------------------------------------------------- 3D composition and axis order

def test_bruteforce_triple_sum_4x4x4(oracle):
    """Eq. 11 written out in pure Python on 4x4x4 (no shared code with the oracle)."""
    n = 4
    x = rng_cube((n, n, n), 5)
    X = oracle.dft3d(x)
    for k0 in range(n):
        for k1 in range(n):
            for k2 in range(n):
                s = 0j
                for a in range(n):
                    for b in range(n):
                        for c in range(n):
                            s += x[a, b, c] * cmath.exp(-2j * cmath.pi * (k0 * a + k1 * b + k2 * c) / n)
                assert abs(X[k0, k1, k2] - s) < 1e-12


def test_kronecker_form_row_major(oracle):
    """Eq. 12: {X} = V1 (x) V2 (x) V3 {x} with {x} the row-major lumping of x."""
    shape = (2, 3, 4)
    x = rng_cube(shape, 6)
    V = [np.exp(-2j * np.pi * np.outer(np.arange(n), np.arange(n)) / n) for n in shape]
    K = np.kron(np.kron(V[0], V[1]), V[2])
    want = (K @ x.reshape(-1)).reshape(shape)
    assert oracle.rel_l2(oracle.dft3d(x), want) < 1e-13


def test_eq5_sides(oracle):
    """Eq. 5: [X] = [V1][x][V2]^T, checked on n0 = 1 with distinct nonuniform nodes per axis."""
    n1, n2 = 5, 7
    r = np.random.default_rng(7)
    t1, t2 = np.sort(r.random(n1)), np.sort(r.random(n2))
    x = rng_cube((1, n1, n2), 8)
    V1 = np.exp(-2j * np.pi * np.outer(np.arange(n1), t1))
    V2 = np.exp(-2j * np.pi * np.outer(np.arange(n2), t2))
    want = V1 @ x[0] @ V2.T
    got = oracle.dft3d(x, nodes=(None, t1, t2))
    assert oracle.rel_l2(got[0], want) < 1e-13


def test_separable_input(oracle):
    r = np.random.default_rng(9)
    a, b, c = (r.standard_normal(n) + 1j * r.standard_normal(n) for n in (4, 6, 5))
    x = np.einsum("i,j,k->ijk", a, b, c)
    want = np.einsum("i,j,k->ijk", np.fft.fft(a), np.fft.fft(b), np.fft.fft(c))
    assert oracle.rel_l2(oracle.dft3d(x), want) < 1e-13


# ---------------------------------------------------------------- invariants

def test_linearity_parseval_roundtrip(oracle):
    shape = (8, 6, 10)
    x, y = rng_cube(shape, 10), rng_cube(shape, 11)
    al, be = 0.3 - 1.1j, -2.0 + 0.5j
    lhs = oracle.dft3d(al * x + be * y)
    rhs = al * oracle.dft3d(x) + be * oracle.dft3d(y)
    assert oracle.rel_l2(lhs, rhs) < 1e-13
    X = oracle.dft3d(x)
    P = np.prod(shape)
    assert abs(np.sum(np.abs(X) ** 2) / (P * np.sum(np.abs(x) ** 2)) - 1) < 1e-12
    back = oracle.dft3d(X, sign=+1, scaled_inverse=True)
    assert oracle.rel_l2(back, x) < 1e-12


def test_uniform_matrix_rows_orthogonal(oracle):
    """The uniform Vandermonde matrix holds roots of unity and V V^H = N I."""
    n = 12
    V = oracle.axis_matrix(n)
    assert np.max(np.abs(V @ V.conj().T - n * np.eye(n))) < 1e-12
    assert np.max(np.abs(np.abs(V) - 1)) < 1e-15
    assert np.max(np.abs(V ** n - 1)) < 1e-12


# ---------------------------------------------------------------- nonuniform nodes

def _phasor_exact(k, t, sign):
    """exp(sign 2 pi i k t) with k*t reduced mod 1 in exact rational arithmetic."""
    fr = (Fraction(k) * Fraction(t)) % 1
    return cmath.exp(sign * 2j * cmath.pi * float(fr))


def test_nonuniform_matrix_entries_exact_reduction(oracle):
    r = np.random.default_rng(12)
    n = 9
    t = np.sort(r.random(n)) + np.array([0, 3, -2, 100, 0, 0, 7, -50, 1])  # any real, used mod 1
    for sign in (-1, +1):
        M = oracle.axis_matrix(n, sign=sign, nodes=t)
        for k in range(n):
            for j in range(n):
                assert abs(M[k, j] - _phasor_exact(k, t[j], sign)) < 4e-16
        Mo = oracle.axis_matrix(n, sign=sign, nodes=t, nodes_on_output=True)
        for k in range(n):
            for j in range(n):
                assert abs(Mo[k, j] - _phasor_exact(j, t[k], sign)) < 4e-16
        assert np.array_equal(Mo, M.T)
    # large k: the product k*t rounds, the fma term restores the lost bits
    n = 4096
    t = r.random(n)
    M = oracle.axis_matrix(n, nodes=t)
    for k, j in ((4095, 17), (3001, 4000), (2048, 1)):
        assert abs(M[k, j] - _phasor_exact(k, t[j], -1)) < 4e-16


def test_nonuniform_reduces_to_uniform(oracle):
    shape = (8, 4, 16)  # powers of two: j/n is exact, tables must agree to the last bit
    nodes = tuple(np.arange(n) / n for n in shape)
    for a in range(3):
        assert np.max(np.abs(oracle.axis_matrix(shape[a], nodes=nodes[a]) - oracle.axis_matrix(shape[a]))) < 2e-16
    x = rng_cube(shape, 13)
    assert oracle.rel_l2(oracle.dft3d(x, nodes=nodes), oracle.dft3d(x)) < 1e-15
    # shifting every node by an integer changes nothing
    shifted = tuple(t + 1.0 for t in nodes)
    assert oracle.rel_l2(oracle.dft3d(x, nodes=shifted), oracle.dft3d(x)) < 1e-14
    # non power of two: agreement to rounding
    shape = (3, 5, 6)
    nodes = tuple(np.arange(n) / n for n in shape)
    x = rng_cube(shape, 14)
    assert oracle.rel_l2(oracle.dft3d(x, nodes=nodes), np.fft.fftn(x)) < 1e-13


def test_nonuniform_bruteforce_3x4x5(oracle):
    shape = (3, 4, 5)
    r = np.random.default_rng(15)
    nodes = tuple(np.sort(r.random(n)) for n in shape)
    x = rng_cube(shape, 16)
    X = oracle.dft3d(x, nodes=nodes)
    Xo = oracle.dft3d(x, nodes=nodes, nodes_on_output=True)
    for k0 in range(shape[0]):
        for k1 in range(shape[1]):
            for k2 in range(shape[2]):
                s = so = 0j
                for a in range(shape[0]):
                    for b in range(shape[1]):
                        for c in range(shape[2]):
                            s += x[a, b, c] * cmath.exp(-2j * cmath.pi * (
                                k0 * nodes[0][a] + k1 * nodes[1][b] + k2 * nodes[2][c]))
                            so += x[a, b, c] * cmath.exp(-2j * cmath.pi * (
                                nodes[0][k0] * a + nodes[1][k1] * b + nodes[2][k2] * c))
                assert abs(X[k0, k1, k2] - s) < 1e-12
                assert abs(Xo[k0, k1, k2] - so) < 1e-12


def test_mixed_uniform_and_nonuniform_axes(oracle):
    shape = (4, 6, 5)
    r = np.random.default_rng(17)
    t1 = np.sort(r.random(shape[1]))
    x = rng_cube(shape, 18)
    V1 = np.exp(-2j * np.pi * np.outer(np.arange(shape[1]), t1))
    want = np.einsum("kj,ajc->akc", V1, np.fft.fft(np.fft.fft(x, axis=0), axis=2))
    assert oracle.rel_l2(oracle.dft3d(x, nodes=(None, t1, None)), want) < 1e-13


# ---------------------------------------------------------------- float32 entry, subset and single coefficients

def test_f32_entry_widens_exactly(oracle):
    x = rng_cube((4, 6, 8), 19, dtype=np.complex64)
    assert np.array_equal(oracle.dft3d(x), oracle.dft3d(x.astype(np.complex128)))


def test_subset_and_triple_loop_agree_with_full(oracle):
    shape = (12, 10, 16)
    r = np.random.default_rng(20)
    x = rng_cube(shape, 21, dtype=np.complex64)
    nodes = (None, np.sort(r.random(shape[1])), None)
    for kw in (dict(), dict(sign=+1, scaled_inverse=True), dict(nodes=nodes)):
        X = oracle.dft3d(x, **kw)
        S0, S1, S2 = np.array([0, 5, 11]), np.array([9, 2]), np.array([15, 0, 7, 8])
        sub = oracle.Subset(shape, S0, S1, S2, **kw)
        sub.feed(x[:5])       # ragged slabs
        sub.feed(x[5:6])
        sub.feed(x[6:])
        got = sub.result()
        want = X[np.ix_(S0, S1, S2)]
        assert oracle.rel_l2(got, want) < 1e-13
        for k in ((0, 0, 0), (11, 9, 15), (5, 2, 7)):
            assert abs(oracle.coeff_triple(x, k, **kw) - X[k]) < 1e-11 * max(1.0, abs(X[k]))


# ---------------------------------------------------------------- the two-stage (FFT) refactoring, Eq. 17

def two_stage_dft_1d(x, N1, N2, sign=-1):
    """Eq. 17 restated in float64 numpy: n = N2*l + beta, k = k1 + N1*k2.

    Stage 1: length-N1 DFT over l for each beta; twiddle exp(sign 2 pi i k1 beta / N);
    stage 2: length-N2 DFT over beta; output index k1 + N1*k2 (in order).
    """
    N = N1 * N2
    xm = x.reshape(N1, N2)                                    # [l, beta]
    F1 = np.exp(sign * 2j * np.pi * np.outer(np.arange(N1), np.arange(N1)) / N1)
    F2 = np.exp(sign * 2j * np.pi * np.outer(np.arange(N2), np.arange(N2)) / N2)
    T = np.exp(sign * 2j * np.pi * np.outer(np.arange(N1), np.arange(N2)) / N)
    B = F1 @ xm                                               # [k1, beta]
    C = B * T
    Y = C @ F2.T                                              # [k1, k2]
    return Y.T.reshape(N)                                     # index k2*N1 + k1


@pytest.mark.parametrize("N1,N2", [(2, 2), (4, 2), (2, 4), (8, 8), (3, 5), (16, 4), (32, 32), (64, 32)])
def test_two_stage_refactoring_equals_definition(oracle, N1, N2):
    N = N1 * N2
    x = rng_cube((1, 1, N), 100 + N1 + N2)
    for sign in (-1, +1):
        want = oracle.dft3d(x, sign=sign)[0, 0]
        assert oracle.rel_l2(two_stage_dft_1d(x[0, 0], N1, N2, sign), want) < 1e-12


# ------------------------------------------------------------------ inverse nonuniform transform (the linear solve)

def test_solve_axis_uniform_nodes_is_the_inverse_dft(oracle):
    """Nodes j/n: the system matrix is the DFT matrix, whose inverse is known in closed form; numpy's ifft is the
    independent opinion."""
    rng = np.random.default_rng(5)
    n = 24
    X = rng.standard_normal((3, n, 2)) + 1j * rng.standard_normal((3, n, 2))
    got = oracle.solve_axis(X, 1, np.arange(n) / n)
    assert np.abs(got - np.fft.ifft(X, axis=1)).max() < 1e-12


def test_solve_axis_two_points_closed_form(oracle):
    """n = 2, nodes (t0, t1): V = [[1, 1], [w0, w1]], w = exp(-2 pi i t); x = V^-1 X written out by hand."""
    t0, t1 = 0.1, 0.65
    w0, w1 = np.exp(-2j * np.pi * t0), np.exp(-2j * np.pi * t1)
    X = np.array([2.0 - 1.0j, 0.5 + 3.0j])
    det = w1 - w0
    want = np.array([(w1 * X[0] - X[1]) / det, (-w0 * X[0] + X[1]) / det])
    got = oracle.solve_axis(X.reshape(1, 1, 2), 2, np.array([t0, t1])).reshape(2)
    assert np.abs(got - want).max() < 1e-14


def test_solve_undoes_the_forward_nonuniform_transform(oracle):
    """solve3d(dft3d(x)) = x for jittered nodes on two axes and a uniform third axis; and V x = X holds with V typed
    here from Eq. 3."""
    rng = np.random.default_rng(6)
    shape = (6, 10, 8)
    nodes = [(np.arange(n) + 0.3 * rng.uniform(-1, 1, n)) / n for n in shape]
    nodes[2] = None
    x = rng.standard_normal(shape) + 1j * rng.standard_normal(shape)
    X = oracle.dft3d(x, nodes=nodes)
    assert np.abs(oracle.solve3d(X, nodes) - x).max() < 1e-11
    n = shape[1]
    V = np.exp(-2j * np.pi * np.outer(np.arange(n), nodes[1]))
    y = rng.standard_normal((1, n, 1)) + 1j * rng.standard_normal((1, n, 1))
    sol = oracle.solve_axis(y, 1, nodes[1]).reshape(n)
    assert np.abs(V @ sol - y.reshape(n)).max() < 1e-11


def test_solve_axis_nodes_on_output_solves_the_literal_system_of_eq_1(oracle):
    """nodes_on_output=True: the rows of V are the arbitrary evaluation points, V[k, n] = z_k^(-n) with
    z_k = exp(2 pi i w_k) (Eq. 1 read literally, typed here).  The solution must satisfy THAT system and not the
    transposed one (nodes on the input samples), so an orientation argument dropped on the way fails here."""
    rng = np.random.default_rng(8)
    n = 12
    w = (np.arange(n) + 0.35 * rng.uniform(-1, 1, n)) / n          # distinct, not roots of unity
    V_out = np.exp(-2j * np.pi * np.outer(w, np.arange(n)))        # V[k, n] = exp(-2 pi i w_k n)
    X = rng.standard_normal((2, n, 3)) + 1j * rng.standard_normal((2, n, 3))
    sol = oracle.solve_axis(X, 1, w, nodes_on_output=True)
    back = np.einsum("kn,anc->akc", V_out, sol)
    assert np.abs(back - X).max() < 1e-11
    back_wrong = np.einsum("kn,anc->akc", V_out.T, sol)
    assert np.abs(back_wrong - X).max() > 1e-2
    # and it undoes the forward transform of the same orientation
    x = rng.standard_normal((2, n, 3)) + 1j * rng.standard_normal((2, n, 3))
    fwd = oracle.dft_axis(x, 1, nodes=w, nodes_on_output=True)
    assert np.abs(oracle.solve_axis(fwd, 1, w, nodes_on_output=True) - x).max() < 1e-11
    # solve3d passes the orientation on to every axis that has nodes
    nodes = [None, w, None]
    X3 = oracle.dft3d(x, nodes=nodes, nodes_on_output=True)
    assert np.abs(oracle.solve3d(X3, nodes, nodes_on_output=True) - x).max() < 1e-11
