"""B200 (sm_100a) decode path of Direct Multi-Token Decoding.

The product is the C-ABI library declared in include/dmtd.h; this package is its thin
Python binding (argument marshalling only).  Importing the package does not load the
library; creating a `Dmtd` does, and fails loudly if the library has not been built or no
CUDA device is present.  There is no CPU fallback.
"""
from .binding import Dmtd, DmtdError, load_library, library_path, declared_symbols, attention_decode, attention_decode_static  # noqa: F401
