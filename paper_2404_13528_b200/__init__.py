"""B200-native layout-transformation-elimination hot path (SmartMem, ASPLOS '24).

The compute path lives in the CUDA shared library built from ``csrc/`` and is reached
through :mod:`paper_2404_13528_b200.binding`, which only marshals arguments.  Importing
the package does not load the library; the binding loads it on first use and raises if
it is missing (there is no CPU fallback).
"""
__all__ = ["binding", "synth"]
