"""ctypes loader for the float64 direct-summation oracle -- TEST INFRASTRUCTURE.

Only tests, the smoke check and the bench's CPU-baseline / reference legs may
import this module.  The product package never does, and this module imports
nothing from the product package.

The functions mirror oracle_dft.c one to one; see that file for the passages
of the paper each of them follows (Eq. 11-14, Eq. 3, Eq. 5).  solve_axis /
solve3d (the inverse nonuniform transform of Section III-A as a linear solve)
are written here, with numpy.linalg.solve as the library step.  Every function
is pinned in tests/test_oracle_pins.py.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle_dft.c")
_LIB = os.path.join(_HERE, "liboracle_dft.so")

_i64 = ctypes.c_int64
_int = ctypes.c_int
_dbl = ctypes.c_double
_p = ctypes.c_void_p


def build(force=False):
    """Compile oracle_dft.c with gcc (-O3, OpenMP) into liboracle_dft.so next to it."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = _int
        _lib.oracle_axis_matrix.argtypes = [_i64, _int, _dbl, _p, _int, _p]
        _lib.oracle_axis_matrix.restype = None
        _lib.oracle_dft_axis.argtypes = [_p, _p, _i64, _i64, _i64, _int, _int, _dbl, _p, _int]
        _lib.oracle_dft_axis.restype = None
        _lib.oracle_dft3d.argtypes = [_p, _p, _i64, _i64, _i64, _int, _int, _p, _p, _p, _int]
        _lib.oracle_dft3d.restype = _int
        _lib.oracle_dft3d_f32.argtypes = [_p, _p, _i64, _i64, _i64, _int, _int, _p, _p, _p, _int]
        _lib.oracle_dft3d_f32.restype = _int
        _lib.oracle_coeff_triple_f32.argtypes = [_p, _i64, _i64, _i64, _int, _int, _p, _p, _p, _int,
                                                 _i64, _i64, _i64, _p, _p]
        _lib.oracle_coeff_triple_f32.restype = None
        _lib.oracle_subset_accumulate_f32.argtypes = [_p, _i64, _i64, _i64, _i64, _i64, _int, _int,
                                                      _p, _p, _p, _int, _p, _i64, _p, _i64, _p, _i64, _p]
        _lib.oracle_subset_accumulate_f32.restype = _int
    return _lib


def num_threads():
    return int(lib().oracle_num_threads())


def _nodes_ptr(nodes, n):
    """None or a float64 array of n nodes -> (keepalive array, pointer)."""
    if nodes is None:
        return None, None
    a = np.ascontiguousarray(nodes, dtype=np.float64)
    assert a.shape == (n,), (a.shape, n)
    return a, a.ctypes.data


def _node_triplet(nodes, shape):
    nodes = (None, None, None) if nodes is None else nodes
    keep = [_nodes_ptr(nodes[a], shape[a]) for a in range(3)]
    return keep, [k[1] for k in keep]


def axis_matrix(n, sign=-1, scale=1.0, nodes=None, nodes_on_output=False):
    """Dense n x n complex128 matrix M[k, j] of one axis."""
    M = np.empty((n, n), dtype=np.complex128)
    keep, ptr = _nodes_ptr(nodes, n)
    lib().oracle_axis_matrix(n, sign, float(scale), ptr, int(nodes_on_output), M.ctypes.data)
    return M


def dft_axis(x, axis, sign=-1, scale=1.0, nodes=None, nodes_on_output=False):
    """Direct-summation transform of one axis of a 3D complex128 array."""
    x = np.ascontiguousarray(x, dtype=np.complex128)
    assert x.ndim == 3
    out = np.empty_like(x)
    keep, ptr = _nodes_ptr(nodes, x.shape[axis])
    lib().oracle_dft_axis(x.ctypes.data, out.ctypes.data, *x.shape, axis, sign, float(scale), ptr,
                          int(nodes_on_output))
    return out


def dft3d(x, sign=-1, scaled_inverse=False, nodes=None, nodes_on_output=False):
    """3D DFT of a complex array by three direct-summation axis passes, in float64.

    complex64 input is widened exactly (the samples the GPU saw); the result is
    complex128 in the same [n0][n1][n2] layout and natural index order.
    """
    assert x.ndim == 3
    keep, ptrs = _node_triplet(nodes, x.shape)
    if x.dtype == np.complex64:
        x = np.ascontiguousarray(x)
        out = np.empty(x.shape, dtype=np.complex128)
        rc = lib().oracle_dft3d_f32(x.ctypes.data, out.ctypes.data, *x.shape, sign,
                                    int(scaled_inverse), *ptrs, int(nodes_on_output))
    else:
        x = np.ascontiguousarray(x, dtype=np.complex128)
        out = np.empty_like(x)
        rc = lib().oracle_dft3d(x.ctypes.data, out.ctypes.data, *x.shape, sign,
                                int(scaled_inverse), *ptrs, int(nodes_on_output))
    if rc != 0:
        raise MemoryError("oracle_dft3d: out of memory")
    return out


def solve_axis(X, axis, nodes, nodes_on_output=False):
    """Inverse nonuniform transform of one axis (Section III-A, below Eq. 3: for sample points that are not the roots
    of unity the inverse is the solution of the linear system of Eq. 2): x with V x = X along `axis`, V the forward
    matrix of Eq. 3 for these nodes.  numpy.linalg.solve (LAPACK, float64) is the library step."""
    X = np.ascontiguousarray(X, dtype=np.complex128)
    assert X.ndim == 3
    n = X.shape[axis]
    V = axis_matrix(n, -1, 1.0, nodes, nodes_on_output)
    moved = np.moveaxis(X, axis, 0).reshape(n, -1)
    sol = np.linalg.solve(V, moved)
    shape = (n,) + tuple(np.delete(np.array(X.shape), axis))
    return np.ascontiguousarray(np.moveaxis(sol.reshape(shape), 0, axis))


def solve3d(X, nodes, nodes_on_output=False):
    """Inverse of dft3d(., sign=-1, nodes=nodes): axes with nodes are solved, axes without use the scaled inverse
    kernel (which is the inverse of the uniform matrix)."""
    X = np.ascontiguousarray(X, dtype=np.complex128)
    for a in range(3):
        nd = None if nodes is None else nodes[a]
        if nd is None:
            X = dft_axis(X, a, sign=+1, scale=1.0 / X.shape[a])
        else:
            X = solve_axis(X, a, nd, nodes_on_output)
    return X


def coeff_triple(x, k, sign=-1, scaled_inverse=False, nodes=None, nodes_on_output=False):
    """One output coefficient X[k0,k1,k2] by the literal triple sum (complex64 input)."""
    x = np.ascontiguousarray(x, dtype=np.complex64)
    keep, ptrs = _node_triplet(nodes, x.shape)
    re, im = _dbl(), _dbl()
    lib().oracle_coeff_triple_f32(x.ctypes.data, *x.shape, sign, int(scaled_inverse), *ptrs,
                                  int(nodes_on_output), int(k[0]), int(k[1]), int(k[2]),
                                  ctypes.byref(re), ctypes.byref(im))
    return complex(re.value, im.value)


class Subset:
    """Coefficients on a product grid S0 x S1 x S2, fed one slab of n0-planes at a time."""

    def __init__(self, shape, S0, S1, S2, sign=-1, scaled_inverse=False, nodes=None,
                 nodes_on_output=False):
        self.shape = tuple(int(v) for v in shape)
        self.S = [np.ascontiguousarray(s, dtype=np.int64) for s in (S0, S1, S2)]
        for a in range(3):
            assert self.S[a].ndim == 1 and self.S[a].min() >= 0 and self.S[a].max() < self.shape[a]
        self.sign, self.scaled_inverse, self.nodes_on_output = sign, scaled_inverse, nodes_on_output
        self._keep, self._ptrs = _node_triplet(nodes, self.shape)
        self.acc = np.zeros(tuple(len(s) for s in self.S), dtype=np.complex128)
        self._next_plane = 0

    def feed(self, slab):
        """slab: complex64 [planes][n1][n2], the next planes in order of n0."""
        slab = np.ascontiguousarray(slab, dtype=np.complex64)
        planes = slab.shape[0]
        assert slab.shape[1:] == self.shape[1:]
        assert self._next_plane + planes <= self.shape[0]
        rc = lib().oracle_subset_accumulate_f32(
            slab.ctypes.data, self._next_plane, planes, *self.shape, self.sign,
            int(self.scaled_inverse), *self._ptrs, int(self.nodes_on_output),
            self.S[0].ctypes.data, len(self.S[0]), self.S[1].ctypes.data, len(self.S[1]),
            self.S[2].ctypes.data, len(self.S[2]), self.acc.ctypes.data)
        if rc != 0:
            raise MemoryError("oracle_subset_accumulate_f32: out of memory")
        self._next_plane += planes

    def result(self):
        assert self._next_plane == self.shape[0], "not all planes were fed"
        return self.acc


def rel_l2(y, ref):
    """||y - ref||_2 / ||ref||_2 over complex values, accumulated in float64."""
    y = np.asarray(y).astype(np.complex128, copy=False).ravel()
    ref = np.asarray(ref).astype(np.complex128, copy=False).ravel()
    num = np.sqrt(np.sum(np.abs(y - ref) ** 2))
    den = np.sqrt(np.sum(np.abs(ref) ** 2))
    return float(num / den) if den > 0 else float(num)
