"""WaveAlign-scheduled block-sparse attention for B200: Python binding of the C-ABI library.

`binding` mirrors include/waveal.h (marshalling only); `inputs` holds the seeded synthetic
workload generators; `build` compiles the library in-tree.  Importing the package does not
load the library; the first call does, and fails loudly if it is missing.
"""
from . import binding, inputs  # noqa: F401
