"""Error-bound coefficients of the paper, in exact rational arithmetic (test infrastructure).

  gamma(k)                 gamma_k = k u32 / (1 - k u32)                        [Table notation]
  tau()                    u16^2 (3 + 2 u16 + 2 u16^2)                          [Eq. truncation]
  ll_coeff()               u16^2 (1 + u16)^2, the dropped lo*lo term            [Eq. ll_bound]
  main_bound_coeff(k)      tau + gamma_k a^2 (1+2u16) + gamma_2 (1+gamma_k) a^2 (1+2u16)
                                                                                [Eq. main_bound]
  main_bound_first_order(k)  gamma_k + 14 u32                                   [Eq. main_bound_first_order]
"""
from fractions import Fraction

U16 = Fraction(1, 2 ** 11)
U32 = Fraction(1, 2 ** 24)


def gamma(k: int) -> Fraction:
    return (k * U32) / (1 - k * U32)


def tau() -> Fraction:
    return U16 ** 2 * (3 + 2 * U16 + 2 * U16 ** 2)


def ll_coeff() -> Fraction:
    return U16 ** 2 * (1 + U16) ** 2


def main_bound_coeff(k: int) -> Fraction:
    a = 1 + U16
    g = gamma(k)
    return tau() + g * a * a * (1 + 2 * U16) + gamma(2) * (1 + g) * a * a * (1 + 2 * U16)


def main_bound_first_order(k: int) -> Fraction:
    return gamma(k) + 14 * U32
