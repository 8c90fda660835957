"""Thin ctypes binding of the dft3d C-ABI (include/dft3d.h).

Argument marshalling only: every step of the transform runs in the library's CUDA kernels.
PyTorch supplies device memory (`tensor.data_ptr()`) and the current stream, nothing else.
There is no fallback: if libdft3d.so is missing the import fails and says how to build it.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# DFT3D_LIBRARY overrides the path of the shared library (for trying differently built variants)
_LIB_PATH = os.environ.get("DFT3D_LIBRARY") or os.path.join(_HERE, "libdft3d.so")

DFT3D_KDFT, DFT3D_FFT, DFT3D_AUTO = 0, 1, 2
DFT3D_FORWARD, DFT3D_INVERSE = -1, +1
DFT3D_NODES_ON_OUTPUT, DFT3D_UNSCALED_INVERSE, DFT3D_SPLIT_FP16, DFT3D_SPLIT_TF32, DFT3D_DESTROY_INPUT = 1, 2, 4, 8, 16
DFT3D_INVERSE_SOLVE = 32

EXPORTS = [
    "dft3d_plan_create", "dft3d_plan_create_ex", "dft3d_execute", "dft3d_execute_host", "dft3d_execute_host_batch",
    "dft3d_execute_axis",
    "dft3d_plan_status", "dft3d_plan_workspace_bytes", "dft3d_plan_launches", "dft3d_plan_split", "dft3d_plan_fft_split",
    "dft3d_plan_destroy",
    "dft3d_status_string", "dft3d_last_error", "dft3d_generate_axis_matrix", "dft3d_generate_twiddle", "dft3d_generate_inverse_matrix",
    "dft3d_generate_real_table", "dft3d_kdft_execute_static",
]


class Dft3dError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("dft3d status %d: %s" % (status, message))
        self.status = status


class _Options(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_size_t), ("flags", ctypes.c_uint),
                ("fft_split", (ctypes.c_int * 2) * 3), ("workspace_limit", ctypes.c_size_t),
                ("axes", ctypes.c_uint)]


def library_path():
    return _LIB_PATH


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            "%s is missing: build it with `python -m paper_2002_03260_b200.build` "
            "(nvcc, sm_100a); there is no CPU fallback" % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ll, ci, cd = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_double
    lib.dft3d_plan_create.argtypes = [ctypes.POINTER(vp), ll, ll, ll, ci, ci, vp, vp, vp]
    lib.dft3d_plan_create_ex.argtypes = [ctypes.POINTER(vp), ll, ll, ll, ci, ci, vp, vp, vp, ctypes.POINTER(_Options)]
    lib.dft3d_execute.argtypes = [vp, vp, vp, vp]
    lib.dft3d_execute_host.argtypes = [vp, vp, vp, vp]
    lib.dft3d_execute_host_batch.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ci, vp]
    lib.dft3d_execute_axis.argtypes = [vp, ci, vp, vp, vp]
    lib.dft3d_plan_status.argtypes = [vp]
    lib.dft3d_plan_workspace_bytes.argtypes = [vp]
    lib.dft3d_plan_workspace_bytes.restype = ctypes.c_size_t
    lib.dft3d_plan_launches.argtypes = [vp]
    lib.dft3d_plan_split.argtypes = [vp]
    lib.dft3d_plan_fft_split.argtypes = [vp, ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.dft3d_plan_destroy.argtypes = [vp]
    lib.dft3d_status_string.argtypes = [ci]
    lib.dft3d_status_string.restype = ctypes.c_char_p
    lib.dft3d_last_error.restype = ctypes.c_char_p
    lib.dft3d_generate_axis_matrix.argtypes = [ll, ci, cd, vp, ci, vp]
    lib.dft3d_generate_twiddle.argtypes = [ll, ll, ci, vp]
    lib.dft3d_generate_inverse_matrix.argtypes = [ll, vp, ci, vp, vp]
    lib.dft3d_generate_real_table.argtypes = [ll, ci, cd, vp, ci, vp, vp]
    lib.dft3d_kdft_execute_static.argtypes = [ll, ll, ll, vp, vp, vp, vp, vp, vp, ctypes.c_char_p, ctypes.c_size_t]
    return lib


_lib = _load()


def _check(status):
    if status != 0:
        raise Dft3dError(status, "%s: %s" % (_lib.dft3d_status_string(status).decode(),
                                             _lib.dft3d_last_error().decode()))


def _nodes_arg(nodes, n):
    if nodes is None:
        return None, None
    a = np.ascontiguousarray(nodes, dtype=np.float64)
    if a.shape != (n,):
        raise ValueError("node array must have shape (%d,), got %s" % (n, a.shape))
    return a, a.ctypes.data


def generate_axis_matrix(n, sign=-1, scale=1.0, nodes=None, nodes_on_output=False):
    """dft3d_generate_axis_matrix: the n x n complex128 matrix of one axis (host only)."""
    M = np.empty((n, n), dtype=np.complex128)
    keep, ptr = _nodes_arg(nodes, n)
    _check(_lib.dft3d_generate_axis_matrix(n, sign, float(scale), ptr, int(nodes_on_output), M.ctypes.data))
    return M


def generate_twiddle(N1, N2, sign=-1):
    """dft3d_generate_twiddle: T[k1, beta] = exp(sign 2 pi i k1 beta / (N1 N2)) as complex128 (host only)."""
    T = np.empty((N1, N2), dtype=np.complex128)
    _check(_lib.dft3d_generate_twiddle(N1, N2, sign, T.ctypes.data))
    return T


def generate_inverse_matrix(n, nodes, nodes_on_output=False):
    """dft3d_generate_inverse_matrix: inverse of the forward matrix of `nodes` as complex128, and the growth figure
    max|M| * max|M^-1| (host only)."""
    M = np.empty((n, n), dtype=np.complex128)
    growth = ctypes.c_double(0.0)
    keep, ptr = _nodes_arg(nodes, n)
    _check(_lib.dft3d_generate_inverse_matrix(n, ptr, int(nodes_on_output), M.ctypes.data, ctypes.byref(growth)))
    return M, growth.value


def generate_real_table(n, sign=-1, scale=1.0, nodes=None, nodes_on_output=False):
    """dft3d_generate_real_table: the (hi, lo) float32 pieces of the real 2n x 2n matrix (host only)."""
    hi = np.empty((2 * n, 2 * n), dtype=np.float32)
    lo = np.empty((2 * n, 2 * n), dtype=np.float32)
    keep, ptr = _nodes_arg(nodes, n)
    _check(_lib.dft3d_generate_real_table(n, sign, float(scale), ptr, int(nodes_on_output),
                                          hi.ctypes.data, lo.ctypes.data))
    return hi, lo


def kdft_execute_static(x, out, tables, stream=None):
    """dft3d_kdft_execute_static: KDFT of `x` into `out` without any allocation by the library.

    For callers that cannot allocate device memory where the transform is needed.  `tables` are three
    float32 CUDA tensors of shape [2, 2*n_a, 2*n_a] (the hi and lo pieces of dft3d_generate_real_table for
    each axis), owned by the caller.  Limited to n0*n1*n2 <= 2**21 points; calls on one GPU must not overlap.
    """
    import torch
    for name, t in (("x", x), ("out", out)):
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.complex64 and t.dim() == 3
                and t.is_contiguous()):
            raise ValueError("%s must be a contiguous three-dimensional complex64 CUDA tensor" % name)
    if out.shape != x.shape or out.device != x.device:
        raise ValueError("out must have the shape and device of x")
    if len(tables) != 3:
        raise ValueError("tables must hold one tensor per axis")
    for a, t in enumerate(tables):
        want = (2, 2 * x.shape[a], 2 * x.shape[a])
        if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and tuple(t.shape) == want
                and t.is_contiguous() and t.device == x.device):
            raise ValueError("tables[%d] must be a contiguous float32 CUDA tensor of shape %s on the device of x"
                             % (a, want))
    n0, n1, n2 = x.shape
    msg = ctypes.create_string_buffer(384)
    status = _lib.dft3d_kdft_execute_static(n0, n1, n2, tables[0].data_ptr(), tables[1].data_ptr(),
                                            tables[2].data_ptr(), x.data_ptr(), out.data_ptr(),
                                            _stream_ptr(stream), msg, len(msg))
    if status != 0:
        raise Dft3dError(status, "%s: %s" % (_lib.dft3d_status_string(status).decode(), msg.value.decode()))
    return out


def _stream_ptr(stream):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


class Plan:
    """dft3d_plan_create / dft3d_execute / dft3d_plan_destroy.

    plan = Plan(n0, n1, n2, mode=DFT3D_KDFT, sign=DFT3D_FORWARD, nodes=(None, None, None))
    y = plan(x)            # x: complex64 CUDA tensor [n0, n1, n2]; y: new tensor (or pass out=)
    Plan(b, n1, n2, axes=(1, 2)) is a batch of b two-dimensional transforms, axes=(2,) a batch of 1D ones.
    """

    def __init__(self, n0, n1, n2, mode=DFT3D_KDFT, sign=DFT3D_FORWARD, nodes=None, flags=0, fft_split=None,
                 workspace_limit=0, axes=None):
        self.shape = (int(n0), int(n1), int(n2))
        self.mode, self.sign = mode, sign
        self._h = ctypes.c_void_p()
        nodes = (None, None, None) if nodes is None else nodes
        keep = [_nodes_arg(nodes[a], self.shape[a]) for a in range(3)]
        opt = _Options()
        opt.struct_size = ctypes.sizeof(_Options)
        opt.flags = flags
        opt.workspace_limit = workspace_limit
        opt.axes = 0 if axes is None else sum(1 << int(a) for a in set(axes))   # e.g. axes=(1, 2): batch of 2D transforms
        if fft_split is not None:
            for a in range(3):
                if fft_split[a] is not None:
                    opt.fft_split[a][0], opt.fft_split[a][1] = fft_split[a]
        _check(_lib.dft3d_plan_create_ex(ctypes.byref(self._h), *self.shape, mode, sign,
                                         keep[0][1], keep[1][1], keep[2][1], ctypes.byref(opt)))

    def _check_tensor(self, t, name):
        import torch
        if not (t.is_cuda and t.dtype == torch.complex64 and tuple(t.shape) == self.shape and t.is_contiguous()):
            raise ValueError("%s must be a contiguous complex64 CUDA tensor of shape %s" % (name, self.shape))

    def execute(self, x, out=None, stream=None):
        import torch
        self._check_tensor(x, "x")
        if out is None:
            out = torch.empty_like(x)
        self._check_tensor(out, "out")
        _check(_lib.dft3d_execute(self._h, x.data_ptr(), out.data_ptr(), _stream_ptr(stream)))
        return out

    __call__ = execute

    def execute_axis(self, axis, x, out=None, stream=None):
        import torch
        self._check_tensor(x, "x")
        if out is None:
            out = torch.empty_like(x)
        self._check_tensor(out, "out")
        _check(_lib.dft3d_execute_axis(self._h, axis, x.data_ptr(), out.data_ptr(), _stream_ptr(stream)))
        return out

    def execute_host(self, x_host, out_host, stream=None):
        """x_host/out_host: complex64 CPU tensors or numpy arrays of the plan's shape (pinned is faster)."""
        def ptr(a):
            return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
        _check(_lib.dft3d_execute_host(self._h, ptr(x_host), ptr(out_host), _stream_ptr(stream)))
        return out_host

    def execute_host_batch(self, xs_host, outs_host, stream=None):
        """A sequence of host cubes, streamed: the download of one result overlaps the upload of the next input.
        xs_host/outs_host: equally long lists of complex64 CPU tensors or numpy arrays (pinned, or nothing overlaps)."""
        def ptr(a):
            return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
        if len(xs_host) != len(outs_host):
            raise ValueError("xs_host and outs_host must have the same length")
        n = len(xs_host)
        ins = (ctypes.c_void_p * max(n, 1))(*[ptr(a) for a in xs_host])
        outs = (ctypes.c_void_p * max(n, 1))(*[ptr(a) for a in outs_host])
        _check(_lib.dft3d_execute_host_batch(self._h, ins, outs, n, _stream_ptr(stream)))
        return outs_host

    def status(self):
        """Raises Dft3dError if a kernel of an earlier execute abandoned a wait; call after synchronising."""
        _check(_lib.dft3d_plan_status(self._h))

    @property
    def workspace_bytes(self):
        return int(_lib.dft3d_plan_workspace_bytes(self._h))

    @property
    def launches(self):
        return int(_lib.dft3d_plan_launches(self._h))

    @property
    def split(self):
        """DFT3D_SPLIT_FP16 or DFT3D_SPLIT_TF32: the operand split of the plan's tensor-core products."""
        return int(_lib.dft3d_plan_split(self._h))

    def fft_split(self, axis):
        """(N1, N2) of Eq. 17 on `axis`: the lengths of the first and the second matrix product."""
        n1, n2 = ctypes.c_int(0), ctypes.c_int(0)
        _check(_lib.dft3d_plan_fft_split(self._h, int(axis), ctypes.byref(n1), ctypes.byref(n2)))
        return n1.value, n2.value

    def destroy(self):
        if self._h:
            _lib.dft3d_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
