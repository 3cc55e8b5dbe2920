"""R_OF and R_UF of Eq. 2 for a format descriptor, for the tests' non-vacuity checks (does a case really saturate,
does a product really fall under the threshold).  The library's Python package holds none of the method's arithmetic."""


def r_uf(fmt) -> float:
    return 2.0 ** (-fmt.bias)


def r_of(fmt) -> float:
    return 2.0 ** (2 ** fmt.exp_bits - fmt.bias - 1) * (2.0 - 2.0 ** (-fmt.man_bits))
