"""CurDKV / AdaCurDKV prefill-time KV selection for B200 (sm_100a).

The CUDA library is loaded lazily by :mod:`paper_2509_15038_b200.binding`;
importing the package (or :mod:`.synth`) needs no GPU and no built extension.
"""

__all__ = ["binding", "synth", "build"]
