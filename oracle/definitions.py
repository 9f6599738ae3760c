"""Big-integer definitions of the D2-MHE ring operations (pure Python, tiny sizes).

TEST INFRASTRUCTURE: an oracle for the CUDA library, never imported by it.

Everything here is the definition written out with Python integers over the
full modulus q (no residue number system, no transforms):

* ring product in Z_q[X]/(X^N+1)                        (Sec. 3.2)
* BFV.SecKeyGen / PubKeyGen / Encrypt / Add / Decrypt    (Sec. 3.2 items 1-5)
* MBFV.PubKeyGen and the decryption shares of MBFV.Convert with mu_k = 0
  (Sec. 4.2 items 2-3, Eq. 2-3)
* slot packing: plaintext polynomial <-> values at psi_t^(2j+1)   (Sec. 6)

It is used to pin the C oracle (d2mhe_oracle.c) on small instances.
"""
from fractions import Fraction
from math import prod


def negacyclic_mul(a, b, q):
    """c = a*b in Z_q[X]/(X^N+1): X^N = -1 (Sec. 3.2)."""
    n = len(a)
    c = [0] * n
    for i, ai in enumerate(a):
        if ai == 0:
            continue
        for j, bj in enumerate(b):
            k = i + j
            if k < n:
                c[k] += ai * bj
            else:
                c[k - n] -= ai * bj
    return [x % q for x in c]


def poly_add(a, b, q):
    return [(x + y) % q for x, y in zip(a, b)]


def poly_neg(a, q):
    return [(-x) % q for x in a]


def centred(x, q):
    """Representative of x mod q in (-q/2, q/2] (Sec. 3.2)."""
    x %= q
    return x - q if x > q // 2 else x


def crt(residues, moduli):
    """The integer in [0, prod moduli) with the given residues."""
    q = prod(moduli)
    v = 0
    for r, m in zip(residues, moduli):
        qh = q // m
        v += r * qh * pow(qh, -1, m)
    return v % q


def round_div(num, den):
    """Nearest integer to num/den (den > 0); ties cannot occur for odd den and even num scaling."""
    return (2 * num + den) // (2 * den)


def bfv_decrypt(c0, c1, s, q, t):
    """x = [ round( t/q * [c0 + c1 s]_q ) ]_t   (Sec. 3.2 item 5)."""
    v = poly_add(c0, negacyclic_mul(c1, [x % q for x in s], q), q)
    out = []
    for vj in v:
        # exact rational rounding of t*vj/q with vj in [0, q)
        r = Fraction(t * vj, q)
        nearest = (2 * r.numerator + r.denominator) // (2 * r.denominator)
        out.append(nearest % t)
    return out


def pk_share(p1, s_k, e_k, q):
    """p_{0,k} = -(p_1 s_k + e_k)   (Sec. 4.2 item 2)."""
    return poly_neg(poly_add(negacyclic_mul(p1, [x % q for x in s_k], q), [x % q for x in e_k], q), q)


def bfv_encrypt(p0, p1, m, u, e0, e1, q, t):
    """ct = (Lambda m + u p0 + e0, u p1 + e1), Lambda = floor(q/t)   (Sec. 3.2 item 3)."""
    lam = q // t
    uq = [x % q for x in u]
    c0 = poly_add(poly_add([lam * x % q for x in m], negacyclic_mul(uq, p0, q), q), [x % q for x in e0], q)
    c1 = poly_add(negacyclic_mul(uq, p1, q), [x % q for x in e1], q)
    return c0, c1


def decryption_share(c1, s_k, e_k, q):
    """h_k = s_k c1 + e_k   (Eq. 2, first component, mu_k = 0)."""
    return poly_add(negacyclic_mul(c1, [x % q for x in s_k], q), [x % q for x in e_k], q)


def convert_share(c1, s_k, mu_k, e0_k, e1_k, p0_i, p1_i, q):
    """(h_0, h_1) = (s_k c1 + mu_k p_{0,i} + e_{0,k}, mu_k p_{1,i} + e_{1,k})   (Eq. 2)."""
    mu = [x % q for x in mu_k]
    h0 = poly_add(poly_add(negacyclic_mul(c1, [x % q for x in s_k], q), negacyclic_mul(mu, p0_i, q), q),
                  [x % q for x in e0_k], q)
    h1 = poly_add(negacyclic_mul(mu, p1_i, q), [x % q for x in e1_k], q)
    return h0, h1


def bootstrap_share(c1, alpha, s_k, m_k, e0_k, e1_k, q, t):
    """(eta_0, eta_1) = (s_k c1 - Lambda M_k + e_{0,k}, -s_k alpha + Lambda M_k + e_{1,k})   (Eq. 4)."""
    lam = q // t
    s = [x % q for x in s_k]
    lm = [lam * x % q for x in m_k]
    eta0 = poly_add(poly_add(negacyclic_mul(c1, s, q), poly_neg(lm, q), q), [x % q for x in e0_k], q)
    eta1 = poly_add(poly_add(poly_neg(negacyclic_mul(alpha, s, q), q), lm, q), [x % q for x in e1_k], q)
    return eta0, eta1


def bootstrap_combine(c0, eta0_list, eta1_list, alpha, q, t):
    """ct' = ([round(t/q [c0 + eta_0]_q)]_t Lambda + eta_1, alpha)   (Sec. 4.2 item 4)."""
    x = combine(c0, eta0_list, q, t)
    lam = q // t
    c0n = [lam * v % q for v in x]
    for e in eta1_list:
        c0n = poly_add(c0n, e, q)
    return c0n, list(alpha)


def combine(c0, shares, q, t):
    """[ round( t/q * [c0 + sum_k h_k]_q ) ]_t   (Sec. 4.2 item 3, Eq. 3; Sec. 3.2 item 5)."""
    v = list(c0)
    for h in shares:
        v = poly_add(v, h, q)
    return [round_div(t * vj, q) % t for vj in v]


def horner(poly, x, p):
    acc = 0
    for c in reversed(poly):
        acc = (acc * x + c) % p
    return acc


def decode_slots(m, psi_t, t):
    """y_j = m(psi_t^(2j+1)) mod t lifted to (-t/2, t/2)."""
    out = []
    for j in range(len(m)):
        y = horner(m, pow(psi_t, 2 * j + 1, t), t)
        out.append(y - t if y > (t - 1) // 2 else y)
    return out


def philox4x32_10(key, ctr):
    """Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11), written from the published round function."""
    m0, m1 = 0xD2511F53, 0xCD9E8D57
    w0, w1 = 0x9E3779B9, 0xBB67AE85
    c = list(ctr)
    k = list(key)
    mask = 0xFFFFFFFF
    for r in range(10):
        if r:
            k[0] = (k[0] + w0) & mask
            k[1] = (k[1] + w1) & mask
        p0 = m0 * c[0]
        p1 = m1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & mask, (p0 >> 32) ^ c[3] ^ k[1], p0 & mask]
    return c
