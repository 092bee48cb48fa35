"""B200-native 2:4-sparse INT8 linear-layer path (after GPUSQ-ViT).

The product is the C-ABI library ``libgpusq.so`` built from ``csrc/``; this
package holds its thin Python binding (``binding``) and the seeded synthetic
input generators (``inputs``).  Importing the package does not load the CUDA
library; the first call into ``binding`` does, and raises if it is missing --
there is no CPU fallback.
"""
__all__ = ["inputs", "binding"]
