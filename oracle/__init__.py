"""CPU oracle package -- test infrastructure, not part of the library.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.  It holds

* ``conv_oracle.c`` / :func:`conv3x3`: the layer's plain definition (dense direct convolution over the masked
  weights, double accumulation), pinned by the CPU tests against closed forms, brute force and a library
  convolution;
* :mod:`oracle.fkw_ref`: an independent statement of the FKW storage format and the filter-kernel reorder
  (Sections 5.2 and 5.3 of the paper) used to check the library's encoder bit for bit, plus the invariant
  checkers for the paper's constraint sets.

Nothing here imports the CUDA package, and the CUDA package imports nothing from here.
"""
from .conv import build, conv3x3, conv3x3_point, maxpool2x2, num_threads, set_num_threads  # noqa: F401
