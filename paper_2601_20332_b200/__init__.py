"""B200-native windowed denoising step for masked diffusion language models.

The product is the C-ABI library ``libwd.so`` (sources under ``csrc/``,
declarations in ``include/wd.h``).  ``binding`` is a thin ctypes layer with
the same names; ``synth`` holds the seeded synthetic-input generators that the
tests and the benchmark share.  Nothing is imported eagerly so that the
CPU-only test tier can use ``synth`` without loading the CUDA library.
"""

__all__ = ["binding", "synth", "build"]
