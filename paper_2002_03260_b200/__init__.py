"""3D complex DFT as tensor-core matrix multiplications on one B200 (KDFT and FFT formulations).

The binding (and with it libdft3d.so) is loaded on first use of any public name, so that
`paper_2002_03260_b200.build` can be imported to (re)build the library before it exists.
"""
import importlib

__all__ = ["Plan", "Dft3dError", "DFT3D_KDFT", "DFT3D_FFT", "DFT3D_AUTO", "DFT3D_FORWARD", "DFT3D_INVERSE",
           "DFT3D_NODES_ON_OUTPUT", "DFT3D_UNSCALED_INVERSE", "DFT3D_SPLIT_FP16", "DFT3D_SPLIT_TF32", "DFT3D_DESTROY_INPUT", "DFT3D_INVERSE_SOLVE", "generate_inverse_matrix", "generate_axis_matrix", "generate_real_table",
           "generate_twiddle", "kdft_execute_static", "library_path"]


def __getattr__(name):
    if name in __all__:
        binding = importlib.import_module(".dft3d", __name__)   # raises ImportError if the library is missing
        return getattr(binding, name)
    raise AttributeError("module %r has no attribute %r" % (__name__, name))
