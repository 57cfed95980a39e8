"""B200-native MoE decode step with adaptive expert prefetch (APEX).

The package holds three things:

* ``csrc/``     hand-written sm_100a CUDA kernels behind a C-ABI library (``libapex.so``),
* ``binding``   a thin ctypes layer with the same names as the C entry points,
* ``synth``     seeded synthetic input generators (shapes of the paper's models; no
                method arithmetic).

Nothing here falls back to a CPU implementation: if ``libapex.so`` is missing the binding
raises at load time.
"""

__all__ = ["binding", "synth", "build"]
