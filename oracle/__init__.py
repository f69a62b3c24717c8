"""CPU oracle for the DMTD decode path.  TEST INFRASTRUCTURE, NOT PRODUCT.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.
"""
from .binding import (Oracle, OracleLib, lib, vanilla_generate,  # noqa: F401
                      masked_parallel_forward)
