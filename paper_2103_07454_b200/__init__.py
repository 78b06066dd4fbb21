"""EventGraD event-triggered communication step for P replicas held in one B200's HBM.

``binding`` is the thin ctypes layer over the C-ABI CUDA library (``include/eventgrad.h``);
``workload`` holds the seeded synthetic input generators.  There is no CPU fallback: every
call into ``binding`` raises if the CUDA library has not been built.
"""
