"""ShadowSync hot path on one B200: CUDA kernels behind a C boundary, with a thin ctypes binding.

Submodules: ``binding`` (the ss_* calls), ``trainer`` (streams, replicas, shadow loop), ``synth`` (seeded
synthetic inputs), ``build`` (compiles libshadowsync.so in-tree).  Importing the package loads nothing;
the library is opened on the first call and its absence is an error.
"""
__all__ = ["binding", "trainer", "synth", "build"]
