"""B200-native hot path of ConfLayers self-speculative decoding.

``binding`` is a thin ctypes layer over the C ABI declared in ``include/conflayers.h``
(argument marshalling only; every step of the method runs in CUDA kernels inside
``libconflayers.so``).  There is no CPU fallback: if the library has not been built, or no CUDA
device is present, calls raise.
"""
from .binding import (CL_MAX_K, ConfLayersError, Context, SelectCfg, Stats, cl_layer_confidences_static,  # noqa: F401
                      exported_symbols, library_path, load_library)
