"""B200-native LBA contraction (GEMM and convolution with a low bit-width accumulator).

The compute path is the CUDA library ``liblba.so`` (C ABI in ``include/lba.h``); this package
is its thin Python binding plus seeded input generators and workload shape lists.
"""
from .formats import (LbaFormat, fixed_point_format, m4e3_input_formats, FLAG_INPUT_M4E3, FLAG_WRAP, ROUND_FLOOR, ROUND_NEAREST_EVEN, FLAG_UNDERFLOW, ORDER_SEQUENTIAL,
                      ORDER_CHUNKED, PAPER_CHUNK, code_domain_formats, M7E4_PAPER, WIDE)

__all__ = ["LbaFormat", "fixed_point_format", "m4e3_input_formats", "FLAG_INPUT_M4E3", "FLAG_WRAP", "ROUND_FLOOR", "ROUND_NEAREST_EVEN", "FLAG_UNDERFLOW", "ORDER_SEQUENTIAL",
           "ORDER_CHUNKED", "PAPER_CHUNK", "code_domain_formats", "M7E4_PAPER", "WIDE"]
