"""B200-native thresholded all-pairs similarity join (arXiv 2006.12608, Section 4).

The product is the C-ABI library built from ``csrc/`` (``libsimjoin.so``) and the
thin ctypes binding in :mod:`paper_2006_12608_b200.binding`.  Importing this
package does not load the library; the first call into the binding does, and
fails loudly if the CUDA build is missing.  There is no CPU fallback.
"""

__all__ = ["binding", "workloads", "build"]
