"""B200-native ClusterAttention hot path (clustering, block selection,
block-sparse attention with striped mean-compensation).

The compute lives in the CUDA library `libclusterattn.so` built from `csrc/`;
`binding` marshals arguments for its C entry points.  Importing this package
does not load the library; the first call does, and fails loudly if the
library has not been built.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
