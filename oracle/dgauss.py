"""Cumulative table of the truncated discrete Gaussian chi (oracle side).

TEST INFRASTRUCTURE: used only by the oracle; the CUDA library carries its own,
independently generated table.

chi (Sec. 3.2 item 2): centred discrete Gaussian with standard deviation sigma,
truncated to [-B, B].  The paper gives neither sigma nor B; the reading taken is
sigma = 3.2 cut at 6 sigma, so B = 19, Pr[x] = rho(x)/Z with
rho(x) = exp(-x^2 / (2 sigma^2)) and Z = sum_{|x| <= B} rho(x).

threshold[k] = floor(2^64 * Pr[X <= -B + k]),  k = 0 .. 2B-1, computed with
80 significant digits; a sample is -B + #{k : r >= threshold[k]} for a uniform
64-bit r.
"""
import mpmath

SIGMA = "3.2"
BOUND = 19


def pmf(bound=BOUND, sigma=SIGMA, digits=80):
    mpmath.mp.dps = digits
    s = mpmath.mpf(sigma)
    rho = [mpmath.exp(-mpmath.mpf(x * x) / (2 * s * s)) for x in range(-bound, bound + 1)]
    z = mpmath.fsum(rho)
    return [r / z for r in rho]


def thresholds(bound=BOUND, sigma=SIGMA, digits=80):
    probs = pmf(bound, sigma, digits)
    out = []
    acc = mpmath.mpf(0)
    two64 = mpmath.mpf(2) ** 64
    for k in range(2 * bound):
        acc += probs[k]
        out.append(int(mpmath.floor(acc * two64)))
    return out
