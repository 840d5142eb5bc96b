"""NoLoCo outer synchronisation step and random pipeline routing on B200.

The compute lives in hand-written CUDA behind a C ABI (``include/nolo.h``,
built into ``libnolo.so`` next to this file); :mod:`.binding` marshals
arguments to it and :mod:`.synth` makes seeded synthetic inputs.  Nothing is
imported eagerly so that ``synth`` stays usable where the library is not built.
"""

__all__ = ["binding", "synth", "build"]
