"""libpolyspec: the chained speculative-sampling verification step of polybasic
speculative decoding as hand-written CUDA kernels for sm_100a behind a C ABI.

``binding`` holds the Python front end of the C-ABI library (argument marshalling
only), ``synth`` the seeded input generators, ``buildlib`` the nvcc build step.
Nothing is loaded at import time; the binding raises if the CUDA library is missing.
"""
__version__ = "0.3.1"      # polyspec_version() == 310
