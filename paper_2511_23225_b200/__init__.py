"""B200 (sm_100a) kernels for the FP8 per-tensor linear path and the TWEO
activation penalty, behind a C-ABI shared library.

``paper_2511_23225_b200.binding`` is the thin ctypes layer over the library
(argument marshalling only); ``paper_2511_23225_b200.synth`` draws the seeded
synthetic inputs.  Nothing here falls back to the CPU: if the CUDA library is
missing, the first call raises.
"""

__all__ = ["binding", "synth", "build"]
