"""B200-native subspace-network (SSN) stage-boundary codec.

Two modules live here:

* ``synth``   -- seeded synthetic inputs shaped like the paper's workloads (numpy only,
                 none of the codec's arithmetic besides stating the workload itself).
* ``binding`` -- the thin ctypes layer over the C-ABI shared library built from ``csrc/``.
                 Importing it loads the library and raises if the library is missing;
                 there is no CPU fallback.

``binding`` is not imported here so that the input generator can be used on machines that
have not built the CUDA library (for example by the CPU-only oracle tests).
"""

__all__ = ["synth", "binding", "buildlib"]
