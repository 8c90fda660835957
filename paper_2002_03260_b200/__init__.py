"""3D complex DFT as tensor-core matrix multiplications on one B200 (KDFT and FFT formulations)."""
from .dft3d import (DFT3D_FFT, DFT3D_FORWARD, DFT3D_INVERSE, DFT3D_KDFT, DFT3D_NODES_ON_OUTPUT,
                    DFT3D_UNSCALED_INVERSE, Dft3dError, Plan, generate_axis_matrix, generate_real_table,
                    generate_twiddle, library_path)

__all__ = ["Plan", "Dft3dError", "DFT3D_KDFT", "DFT3D_FFT", "DFT3D_FORWARD", "DFT3D_INVERSE",
           "DFT3D_NODES_ON_OUTPUT", "DFT3D_UNSCALED_INVERSE", "generate_axis_matrix", "generate_real_table",
           "generate_twiddle", "library_path"]
