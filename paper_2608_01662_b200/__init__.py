"""B200-native LongCat-Sparse-Attention hot path: indexer + sparse attention behind a C ABI.

`binding` wraps liblsa.so (built from csrc/ by `build`); `configs` and `inputs` describe and draw the
synthetic workloads.  Importing the package loads nothing; the library is loaded at first use and
its absence is an error, not a fallback.
"""
from .configs import CONFIGS, LsaConfig  # noqa: F401
