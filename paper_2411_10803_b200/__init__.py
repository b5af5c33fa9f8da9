"""B200-native vision-token filter (MustDrop, arXiv 2411.10803, Sec. 3.4).

``binding`` wraps the CUDA library's C ABI; ``synth`` draws seeded synthetic inputs;
``sharding`` splits a batch of independent requests over ranks; ``build`` compiles the
library.  Importing the package does not load the shared library; the first call does, and
raises if it has not been built.
"""
__all__ = ["binding", "synth", "sharding", "build"]
