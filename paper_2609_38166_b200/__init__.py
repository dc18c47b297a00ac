"""B200-native per-window 8-bit decode step for GDN / KDA recurrent states.

``paper_2609_38166_b200.lq`` is the thin Python binding of the C-ABI library
(built from ``csrc/`` by ``paper_2609_38166_b200.build``); ``synth`` draws the
seeded synthetic decode inputs.  Importing the package loads nothing native;
the binding loads the shared library on first use and raises if it is missing.
"""
__all__ = ["synth", "lq", "build"]
