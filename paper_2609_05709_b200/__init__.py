"""B200-native SOAP descriptors and Jacobians: thin Python face of libsoap_b200.so.

Every step of the computation runs in the CUDA library behind the C ABI declared
in include/soap.h; this package only marshals arguments.  torch is used for
device memory and streams.  There is no CPU fallback: if the shared library is
missing, importing `Soap` raises.
"""
from .binding import (GTO, POLYNOMIAL, Soap, SoapError, Derivatives, CompactDerivatives, library_path, load_library,
                      neighbor_counts_static, measure_fp32_peak, EXPORTED_SYMBOLS)

__all__ = ["GTO", "POLYNOMIAL", "Soap", "SoapError", "Derivatives", "CompactDerivatives", "library_path", "load_library",
           "neighbor_counts_static", "measure_fp32_peak", "EXPORTED_SYMBOLS"]
