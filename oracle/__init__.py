"""CPU oracle for one Sketched-SGD compression step -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It shares no code with the CUDA library and never imports it.
"""
from .ssgd_oracle import (FMT_BF16, FMT_F16, Oracle, build, derive_params, fill_priority, merge16,  # noqa: F401
                          quantize16, select)
