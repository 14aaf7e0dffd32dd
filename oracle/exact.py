"""Exact-rational statement of the W4A8 linear (Sec. 3.4): test infrastructure only.

Everything is a Python ``int`` or ``fractions.Fraction``; the two roundings the
scheme contains (token scale to binary16, quotient to the nearest integer) are
carried out on exact rationals, so this file is the arbiter when the floating
point oracles could in principle double-round.  Pure-Python loops: tiny shapes.

Scheme (the paper fixes "4-bit weights, 8-bit activations, INT8 matmul"; the
remaining choices are this build's stated readings):
  weights      q_w in 0..15, one fp16 scale s_w and one zero point z in 0..15
               per (group of `group` consecutive k, output channel n)
  activations  per token m:  s_a = fp16_rne(max_k|x| / 127)
               q_a = clamp(round_half_even(x / s_a), -127, 127); all 0 if s_a = 0
  partials     D[m,g,n] = sum_{k in g} q_w[n,k] q_a[m,k] - z[g,n] sum_{k in g} q_a[m,k]
  output       y[m,n]   = s_a[m] * sum_g s_w[g,n] * D[m,g,n]
"""
from fractions import Fraction

FP16_MAX = Fraction(65504)


def round_half_even(q: Fraction) -> int:
    """Nearest integer to the rational q, ties to the even integer."""
    fl = q.numerator // q.denominator
    rem = q - fl
    half = Fraction(1, 2)
    if rem > half:
        return fl + 1
    if rem < half:
        return fl
    return fl if fl % 2 == 0 else fl + 1


def fp16_rne(q: Fraction) -> Fraction:
    """Round a non-negative rational to binary16 (ties to even), saturating at 65504.

    Subnormals (multiples of 2^-24 below 2^-14) are kept; values that round
    below 2^-25 become 0.
    """
    assert q >= 0
    if q == 0:
        return Fraction(0)
    # exponent e with 2^e <= q < 2^(e+1)
    e = q.numerator.bit_length() - q.denominator.bit_length()
    if Fraction(2) ** e > q:
        e -= 1
    assert Fraction(2) ** e <= q < Fraction(2) ** (e + 1)
    e = max(e, -14)                      # subnormal range shares the 2^-24 spacing
    ulp = Fraction(2) ** (e - 10)
    r = round_half_even(q / ulp) * ulp
    return min(r, FP16_MAX)


def bf16_rne(q: Fraction) -> Fraction:
    """Round a rational to bfloat16 (8-bit significand, ties to even); normal range only."""
    if q == 0:
        return Fraction(0)
    s = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    ulp = Fraction(2) ** (e - 7)
    return s * round_half_even(a / ulp) * ulp


def quantize_act_row(x_row):
    """One token.  x_row: list of Fractions (exact bf16 values).  Returns (s_a, [q_a])."""
    amax = max((abs(v) for v in x_row), default=Fraction(0))
    sa = fp16_rne(amax / 127)
    if sa == 0:
        return sa, [0] * len(x_row)
    qa = [max(-127, min(127, round_half_even(v / sa))) for v in x_row]
    return sa, qa


def group_sums(qa_row, group):
    return [sum(qa_row[g0:g0 + group]) for g0 in range(0, len(qa_row), group)]


def partials(qa, qw, z, group):
    """D[m][g][n] as Python ints.  qa: [M][K]; qw: [N][K]; z: [G][N]."""
    M, N = len(qa), len(qw)
    K = len(qa[0]) if M else (len(qw[0]) if N else 0)
    G = K // group
    D = [[[0] * N for _ in range(G)] for _ in range(M)]
    for m in range(M):
        for g in range(G):
            ks = range(g * group, (g + 1) * group)
            a = sum(qa[m][k] for k in ks)
            for n in range(N):
                p = sum(qw[n][k] * qa[m][k] for k in ks)
                D[m][g][n] = p - z[g][n] * a
    return D


def linear(x, qw, sw, z, group):
    """Whole path on exact rationals.

    x: [M][K] Fractions; qw: [N][K] ints; sw: [G][N] Fractions (fp16 values);
    z: [G][N] ints.  Returns dict(sa, qa, asum, D, y) with y[m][n] exact.
    """
    sa, qa = [], []
    for row in x:
        s, q = quantize_act_row(row)
        sa.append(s)
        qa.append(q)
    D = partials(qa, qw, z, group)
    N = len(qw)
    G = len(sw)
    y = [[sa[m] * sum(sw[g][n] * D[m][g][n] for g in range(G)) for n in range(N)]
         for m in range(len(x))]
    return dict(sa=sa, qa=qa, asum=[group_sums(r, group) for r in qa], D=D, y=y)
