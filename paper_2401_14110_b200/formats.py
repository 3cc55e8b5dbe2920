"""Format descriptors for Q_prod and Q_acc (Eq. 2 of the paper) and the bias rules used by the harness."""
from dataclasses import dataclass

ROUND_FLOOR = 0          # floor on the magnitude: the paper's choice (Sec. 3)
ROUND_NEAREST_EVEN = 1   # a parameter of the benchmark's format sweep, not the paper's choice
FLAG_UNDERFLOW = 1       # bit0 of flags: the |x| < R_UF -> 0 branch of Eq. 2 is active
FLAG_WRAP = 2            # bit1 of flags, fixed-point formats: two's-complement wrap-around instead of saturation
FLAG_INPUT_M4E3 = 4      # bit2 of the product format's flags: operands are bytes of the paper's M4E3 W/A format (Sec. 3.1)

ORDER_SEQUENTIAL = 0     # Eq. 8-9
ORDER_CHUNKED = 1        # two hierarchies, Sec. 3 / App. D
PAPER_CHUNK = 16         # "constant chunk size of 16" (Sec. 3)


@dataclass(frozen=True)
class LbaFormat:
    """Q^FLOAT_{M,E,b}: M mantissa bits, E exponent bits, exponent bias b, rounding, flags."""
    man_bits: int
    exp_bits: int
    bias: int
    rounding: int = ROUND_FLOOR
    flags: int = FLAG_UNDERFLOW

    def as_tuple(self):
        return (self.man_bits, self.exp_bits, self.bias, self.rounding, self.flags)


def code_domain_formats(man_bits: int = 7, exp_bits: int = 4, rounding: int = ROUND_FLOOR,
                        flags: int = FLAG_UNDERFLOW, chunk: int = PAPER_CHUNK):
    """(prod_fmt, acc_fmt) for FMAq on raw E4M3 code values.

    b_prod is the largest integer bias for which the largest code product, 448^2, stays
    below R_OF (the paper's flex-bias rule of Sec. 3.1 applied to products): 2^E - 18.
    b_acc = b_prod - log2(chunk)/2 (Sec. 3, the chunk-size rule; 2 for chunk 16).
    """
    b_prod = 2 ** exp_bits - 18
    half_log = 0
    c = chunk
    while c >= 4:
        half_log += 1
        c //= 4
    prod = LbaFormat(man_bits, exp_bits, b_prod, rounding, flags)
    acc = LbaFormat(man_bits, exp_bits, b_prod - half_log, rounding, flags)
    return prod, acc


def m4e3_input_formats(man_bits: int = 7, exp_bits: int = 4, rounding: int = ROUND_FLOOR,
                       flags: int = FLAG_UNDERFLOW, chunk: int = PAPER_CHUNK):
    """(prod_fmt, acc_fmt) for FMAq on code values of the paper's own W/A format (M4E3, largest magnitude 248).

    The same two rules as ``code_domain_formats``: b_prod is the largest bias for which the largest product, 248^2,
    stays below R_OF, i.e. 2^E - 16, and b_acc = b_prod - log2(chunk)/2.  The product format carries the input flag."""
    b_prod = 2 ** exp_bits - 16
    half_log = 0
    c = chunk
    while c >= 4:
        half_log += 1
        c //= 4
    prod = LbaFormat(man_bits, exp_bits, b_prod, rounding, flags | FLAG_INPUT_M4E3)
    acc = LbaFormat(man_bits, exp_bits, b_prod - half_log, rounding, flags)
    return prod, acc


M7E4_PAPER = (LbaFormat(7, 4, 12), LbaFormat(7, 4, 10))   # real-domain biases of the ResNet runs (Sec. 3.1)
WIDE = LbaFormat(23, 8, 127)                               # binary32-like: nothing in Eq. 2 is reachable


def fixed_point_format(bits: int, bias: int = 0, wrap: bool = False) -> LbaFormat:
    """Q^FIXED_{B,b} of Eq. 1 (exp_bits = 0 selects it): B bits including the sign, integer step 2^-b, floor;
    saturation at R_min / R_max as printed, or wrap-around."""
    return LbaFormat(bits, 0, bias, ROUND_FLOOR, FLAG_WRAP if wrap else 0)
