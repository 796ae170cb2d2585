"""B200-native encode / robust-decode path of Solon (arXiv 2110.01595).

``binding`` is the ctypes layer over the C-ABI library ``libsolon.so`` (built from
``csrc/`` by ``build.py``); ``synth`` makes seeded synthetic workloads.  Importing
the package loads nothing; the first call into ``binding`` loads the library and
raises if it has not been built.
"""

__all__ = ["binding", "synth", "build"]
