"""B200-native pattern-sparse 3x3 convolution (PatDNN's inference hot path).

``binding`` wraps the C ABI of ``libpatdnn.so`` (see ``include/patdnn.h``); ``synth`` draws the seeded synthetic
layers used by the tests and the benchmark; ``build`` compiles the library in-tree with nvcc for sm_100a.
Nothing is imported eagerly so that the generator can be used without the shared library.
"""
__all__ = ["binding", "synth", "build"]
