"""B200-native LoMA attention hot path (arxiv 2401.09486).

The product is the C-ABI library declared in ``include/loma.h`` and built from
``csrc/``; this package is the thin Python binding around it
(:mod:`paper_2401_09486_b200.binding`) plus seeded synthetic input generators
(:mod:`paper_2401_09486_b200.synthetic`).  Importing the package does not load
the library; the first call through the binding does, and fails loudly if the
library has not been built.
"""

__all__ = ["binding", "synthetic", "build", "multi_gpu"]
