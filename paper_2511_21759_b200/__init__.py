"""B200-native block-decoding hot path of ODB-dLLM: C-ABI CUDA library (csrc/, libodb.so) and its
thin Python binding.  Importing the package needs neither a GPU nor the built library."""
from . import binding  # noqa: F401
