"""CPU-only checks: the C-ABI library loads and exports what include/dft3d.h declares, argument
validation works without a GPU, and the float64 table generator agrees with the oracle's matrices
(two independent implementations of Eq. 3 / Eq. 14) and splits values into TF32 pieces correctly."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dft():
    from paper_2002_03260_b200 import build
    build.build()
    import paper_2002_03260_b200 as d
    return d


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dft3d.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dft3d_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(dft):
    names = declared_functions()
    assert len(names) >= 13
    lib = ctypes.CDLL(dft.library_path())
    for name in names:
        assert hasattr(lib, name), "libdft3d.so does not export %s" % name
    from paper_2002_03260_b200 import dft3d as binding
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    missing = [n for n in names if n not in binding.EXPORTS]
    assert not missing, "binding does not know %s" % missing


def test_status_strings(dft):
    from paper_2002_03260_b200 import dft3d as b
    seen = {b._lib.dft3d_status_string(i).decode() for i in range(6)}
    assert len(seen) == 6 and "unknown status" not in seen
    assert b._lib.dft3d_status_string(99).decode() == "unknown status"


def test_argument_validation_needs_no_gpu(dft):
    """Bad arguments are rejected before any CUDA call, with the documented status."""
    cases = [
        (dict(n=(0, 64, 64)), 1), (dict(n=(64, -64, 64)), 1), (dict(n=(64, 64, 64), mode=7), 1),
        (dict(n=(64, 64, 64), sign=0), 1), (dict(n=(64, 64, 64), flags=64), 1),
        (dict(n=(64, 64, 101)), 2), (dict(n=(16384, 64, 64)), 2), (dict(n=(256, 256, 100), mode=1), 2),
        (dict(n=(64, 64, 64), nodes=(np.array([np.nan] * 64), None, None)), 1),
        (dict(n=(64, 64, 64), mode=1, nodes=(np.arange(64) / 64.0, None, None)), 2),
        (dict(n=(64, 64, 64), mode=3), 1),           # 0, 1, 2 (KDFT, FFT, AUTO) are the modes
        (dict(n=(64, 64, 101), mode=2), 2),          # AUTO falls back to KDFT, which needs an even last axis
        (dict(n=(64, 64, 64), flags=4 | 8), 1),      # both operand splits at once
        (dict(n=(64, 64, 66), flags=4), 2),          # fp16 pieces need lengths that are multiples of 4
    ]
    for kw, status in cases:
        n = kw.pop("n")
        with pytest.raises(dft.Dft3dError) as e:
            dft.Plan(*n, **kw)
        assert e.value.status == status, (n, kw, str(e.value))
    # KDFT: axes 0 and 1 may have any length, the last axis must be even (rows of the data start on 16-byte boundaries);
    # FFT: every axis but an untransformed axis 0 needs a multiple of 64
    with pytest.raises(dft.Dft3dError) as e:
        dft.Plan(4, 6, 101, axes=(0, 1))
    assert e.value.status == 2 and "16-byte" in str(e.value)
    with pytest.raises(dft.Dft3dError) as e:
        dft.Plan(3, 100, 256, mode=1, axes=(1, 2))
    assert e.value.status == 2
    import torch
    if not torch.cuda.is_available():
        for n, axes in (((3, 128, 64), (1, 2)), ((3, 101, 64), (0, 1, 2))):
            with pytest.raises(dft.Dft3dError) as e:
                dft.Plan(*n, axes=axes)            # valid sizes: the first failure is the missing device
            assert e.value.status == 4
    from paper_2002_03260_b200 import dft3d as b
    assert b._lib.dft3d_plan_create(None, 64, 64, 64, 0, -1, None, None, None) == 1
    assert b._lib.dft3d_plan_destroy(None) == 0
    assert b._lib.dft3d_plan_workspace_bytes(None) == 0
    assert b._lib.dft3d_plan_status(None) == 1
    assert b._lib.dft3d_execute(None, None, None, None) == 1
    assert "NULL" in b._lib.dft3d_last_error().decode()


# ------------------------------------------------------------------ generator

@pytest.mark.parametrize("n", [4, 64, 96, 250, 1024])
def test_uniform_matrix_matches_oracle(dft, oracle, n):
    for sign in (-1, +1):
        M = dft.generate_axis_matrix(n, sign=sign)
        # the oracle rounds the angle 2*pi*m/n once (up to ~9e-16 absolute); the generator reduces to an octant first
        assert np.max(np.abs(M - oracle.axis_matrix(n, sign=sign))) < 1.5e-15
    # exact values on the axes of the complex plane
    M = dft.generate_axis_matrix(n)
    assert np.all(M[0] == 1) and np.all(M[:, 0] == 1)
    if n % 4 == 0:
        assert M[1, n // 4] == -1j and M[1, n // 2] == -1 and M[1, 3 * n // 4] == 1j


def test_scaled_matrix(dft, oracle):
    n = 64
    M = dft.generate_axis_matrix(n, sign=+1, scale=1.0 / n)
    assert np.max(np.abs(M - oracle.axis_matrix(n, sign=+1, scale=1.0 / n))) < 1.5e-15 / n
    assert np.max(np.abs(M @ dft.generate_axis_matrix(n, sign=-1) - np.eye(n))) < 1e-13


def test_nonuniform_matrix_matches_oracle(dft, oracle):
    r = np.random.default_rng(3)
    n = 200
    t = np.sort(r.random(n)) + r.integers(-5, 5, n)   # any finite node, used modulo 1
    for on_output in (False, True):
        M = dft.generate_axis_matrix(n, nodes=t, nodes_on_output=on_output)
        assert np.max(np.abs(M - oracle.axis_matrix(n, nodes=t, nodes_on_output=on_output))) < 1.5e-15
    # nodes j/n reproduce the uniform matrix (bit-equal for a power of two)
    n = 128
    assert np.array_equal(dft.generate_axis_matrix(n, nodes=np.arange(n) / n), dft.generate_axis_matrix(n))


def test_twiddle(dft):
    N1, N2 = 32, 16
    T = dft.generate_twiddle(N1, N2, sign=-1)
    want = np.exp(-2j * np.pi * np.outer(np.arange(N1), np.arange(N2)) / (N1 * N2))
    assert np.max(np.abs(T - want)) < 1.5e-15
    assert np.array_equal(dft.generate_twiddle(N1, N2, sign=+1), T.conj())


def test_real_table_layout_and_split(dft):
    """W[2k+p][2j+q] realises the complex product on interleaved data; hi/lo are TF32-exact and
    hi+lo reproduces the float64 entry to 2^-22 relative."""
    n = 64
    M = dft.generate_axis_matrix(n)
    hi, lo = dft.generate_real_table(n)
    W = hi.astype(np.float64) + lo.astype(np.float64)
    assert np.max(np.abs(W[0::2, 0::2] - M.real)) < 2.0 ** -21
    assert np.max(np.abs(W[1::2, 1::2] - M.real)) < 2.0 ** -21
    assert np.max(np.abs(W[0::2, 1::2] + M.imag)) < 2.0 ** -21
    assert np.max(np.abs(W[1::2, 0::2] - M.imag)) < 2.0 ** -21
    for piece in (hi, lo):
        assert not np.any(piece.view(np.uint32) & 0x1FFF), "piece has bits below the TF32 mantissa"
    assert np.max(np.abs(lo)) <= 2.0 ** -11
    # the real form equals the complex product on interleaved data
    r = np.random.default_rng(5)
    x = r.standard_normal(n) + 1j * r.standard_normal(n)
    xi = np.empty(2 * n)
    xi[0::2], xi[1::2] = x.real, x.imag
    y = W @ xi
    assert np.max(np.abs((y[0::2] + 1j * y[1::2]) - M @ x)) < 1e-4


def test_generator_rejects_bad_arguments(dft):
    from paper_2002_03260_b200 import dft3d as b
    buf = np.zeros(8)
    assert b._lib.dft3d_generate_axis_matrix(0, -1, 1.0, None, 0, buf.ctypes.data) == 1
    assert b._lib.dft3d_generate_axis_matrix(2, 3, 1.0, None, 0, buf.ctypes.data) == 1
    assert b._lib.dft3d_generate_twiddle(2, 2, -1, None) == 1
    bad = np.array([0.0, np.inf])
    assert b._lib.dft3d_generate_axis_matrix(2, -1, 1.0, bad.ctypes.data, 0, buf.ctypes.data) == 1


def test_inverse_matrix_matches_the_solve(dft, oracle):
    """The host-side inversion behind DFT3D_INVERSE_SOLVE (threaded Gauss-Jordan, no library) against the oracle's
    LAPACK solve and the defining identity; singular node sets are refused."""
    rng = np.random.default_rng(7)
    for n in (2, 16, 100, 300):
        nodes = (np.arange(n) + 0.3 * rng.uniform(-1, 1, n)) / n
        Minv, growth = dft.generate_inverse_matrix(n, nodes)
        V = oracle.axis_matrix(n, -1, 1.0, nodes)
        assert np.abs(Minv @ V - np.eye(n)).max() < 1e-11 and growth > 0
        X = rng.standard_normal((1, n, 3)) + 1j * rng.standard_normal((1, n, 3))
        want = oracle.solve_axis(X, 1, nodes)
        got = np.einsum("kj,ajc->akc", Minv, X)
        assert np.abs(got - want).max() < 1e-11 * max(1.0, growth * n)
    with pytest.raises(dft.Dft3dError) as e:
        dft.generate_inverse_matrix(4, np.array([0.25, 0.5, 0.25, 0.75]))   # two equal nodes: two equal columns
    assert e.value.status == 1
    # nodes that coincide up to rounding (1.1 is not 0.1 + 1 in binary): no zero pivot, but the growth figure says it
    _, growth = dft.generate_inverse_matrix(4, np.array([0.1, 0.3, 1.1, 0.7]))
    assert growth > 1e12


def test_static_entry_wrapper_refuses_tensors_it_cannot_vouch_for(dft):
    """The C side sees only pointers, so the binding checks what they point at before it calls the library: wrong
    device, dtype, shape or layout raise ValueError here, with no GPU involved."""
    torch = pytest.importorskip("torch")
    x = torch.zeros((64, 64, 64), dtype=torch.complex64)
    tables = [torch.zeros((2, 128, 128), dtype=torch.float32) for _ in range(3)]
    with pytest.raises(ValueError, match="CUDA"):
        dft.kdft_execute_static(x, torch.empty_like(x), tables)          # CPU tensors
    with pytest.raises(ValueError):
        dft.kdft_execute_static(x.to(torch.complex128), x, tables)       # wrong dtype
    with pytest.raises(ValueError):
        dft.kdft_execute_static(x[:, :, ::2], x, tables)                 # not contiguous
    with pytest.raises(ValueError):
        dft.kdft_execute_static(np.zeros((64, 64, 64), np.complex64), x, tables)   # not a tensor
