"""AdaDim layer quantization on B200: Python binding of the C-ABI CUDA library.

`binding` wraps libadadim.so (built by `python -m paper_2309_15531_b200.build`);
`inputs` draws the seeded synthetic layers and activations.  There is no CPU
implementation in this package.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]
