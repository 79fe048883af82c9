"""Float batch-norm + quantizer reference and threshold absorption (fp64).

TEST INFRASTRUCTURE ONLY.  Follows Section 2.1 of the paper:

* 2.1.1  a uniform quantizer is successive thresholding followed by an affine
         map, Q(x) = a*T(x, t) + b;
* 2.1.2  the previous layer's quantizer affine moves past the integer matrix
         product, W.(a*x + b) = a*(W.x) + W.b, and together with alpha-scaling
         and batch normalisation collapses to one per-channel a_c*x + b_c;
* 2.1.3  the affine map is absorbed into the thresholds, t <- (t - b)/a, and
         rounded up to an integer when the input is an integer.

Readings where the paper is silent:
* ties: x equal to a threshold counts as passed ("greater than or equal to");
  this is the only reading under which rounding a threshold UP keeps the
  result for integer x.
* a_c < 0 flips the inequality; the caller negates that weight row, and the
  thresholds are derived for the negated accumulator.
* a_c == 0 gives a constant code, expressed with INT32_MIN / INT32_MAX
  sentinels.
* the integer threshold is taken as the smallest integer accumulator whose
  float forward pass yields at least that code (consistent with the float
  pass by construction); the closed form ceil((t-b)/a) is tested separately
  on parameters where fp64 is exact.
"""
from dataclasses import dataclass
import math
import numpy as np

INT32_MIN = -2**31
INT32_MAX = 2**31 - 1

# 2-bit half-wave Gaussian quantizer of Section 2 (item 3) / Section 2.1.1
HWGQ_THRESHOLDS = (0.0, 0.807, 1.345)
HWGQ_STEP = 0.538


def successive_threshold(x: float, t) -> int:
    """T(x, t): number of thresholds that x is greater than or equal to."""
    return sum(1 for ti in t if x >= ti)


@dataclass
class ChannelParams:
    """Float parameters around one output channel of a quantized matrix layer."""
    a_prev: float    # previous layer's quantizer: value = a_prev*code + b_prev
    b_prev: float
    alpha: float     # alpha-scaling of this weight row
    gamma: float     # batch norm: gamma*(z - mu)/sigma + beta
    beta: float
    mu: float
    sigma: float
    row_sum: int     # sum of this row's integer weights (for the W.b term)


def float_forward(acc: int, p: ChannelParams, qthr) -> int:
    """Un-streamlined forward pass from the integer accumulator to the code."""
    z = p.a_prev * float(acc) + p.b_prev * float(p.row_sum)   # W.(a x + b)
    z = p.alpha * z                                           # alpha-scaling
    y = p.gamma * (z - p.mu) / p.sigma + p.beta               # batch norm
    return successive_threshold(y, qthr)                      # quantizer T


def collapse(p: ChannelParams):
    """Section 2.1.2: the three affine maps as one y = A*acc + B."""
    A = p.gamma * p.alpha * p.a_prev / p.sigma
    B = p.gamma * (p.alpha * p.b_prev * p.row_sum - p.mu) / p.sigma + p.beta
    return A, B


def closed_form_thresholds(p: ChannelParams, qthr):
    """Section 2.1.3 literally: ceil((t_i - B)/A), for A > 0."""
    A, B = collapse(p)
    assert A > 0
    return [int(math.ceil((t - B) / A)) for t in qthr]


def streamline(p: ChannelParams, qthr, acc_lo: int, acc_hi: int):
    """Integer thresholds for accumulators in [acc_lo, acc_hi].

    Returns (thresholds, negate): when ``negate`` is True the thresholds apply
    to the NEGATED accumulator (the caller flips the sign of the weight row)."""
    n = len(qthr)
    A, _ = collapse(p)
    if A == 0:
        c = float_forward(0, p, qthr)
        return [INT32_MIN] * c + [INT32_MAX] * (n - c), False
    negate = A < 0

    def code(x):
        return float_forward(-x if negate else x, p, qthr)

    lo, hi = (-acc_hi, -acc_lo) if negate else (acc_lo, acc_hi)
    thr = []
    for i in range(n):
        want = i + 1
        if code(hi) < want:
            thr.append(INT32_MAX)
            continue
        if code(lo) >= want:
            thr.append(INT32_MIN)
            continue
        a, b = lo, hi            # code(a) < want <= code(b)
        while b - a > 1:
            m = (a + b) // 2
            if code(m) >= want:
                b = m
            else:
                a = m
        thr.append(b)
    return thr, negate


def random_params(rng: np.random.Generator, row_sum: int, scale: float) -> ChannelParams:
    """Plausible float parameters; ``scale`` ~ std of the accumulator."""
    return ChannelParams(
        a_prev=float(rng.uniform(0.2, 1.0)),
        b_prev=float(rng.uniform(-0.5, 0.5)),
        alpha=float(rng.uniform(0.01, 0.2)),
        gamma=float(rng.uniform(0.5, 2.0) * rng.choice([-1.0, 1.0, 1.0, 1.0])),
        beta=float(rng.uniform(-0.5, 1.5)),
        mu=float(rng.normal(0.0, 0.1 * scale)),
        sigma=float(rng.uniform(0.02, 0.2) * scale),
        row_sum=int(row_sum),
    )
