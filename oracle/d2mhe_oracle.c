/*
 * D2-MHE oracle: a plain, slow, CPU-only restatement of the multiparty-BFV
 * private gradient update (Sec. 3.2 items 1-5, Sec. 4.2 items 1-3, Algorithm 2).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
 * compared against something written directly from the paper's ring equations.
 * It shares no source, header, table or generator with the CUDA path and is
 * never linked into, imported by, or called from the product library.
 *
 * Style: every modular reduction is a `%` on unsigned __int128, transforms are
 * the textbook bit-reversal radix-2 FFT over Z_p, big integers are arrays of
 * 32-bit words with schoolbook routines.  Nothing is blocked, fused or lazily
 * reduced.  Polynomials are coefficient vectors a[0..N-1] of Z_p[X]/(X^N+1)
 * (Sec. 3.2: R_q = Z_q[X]/(X^n+1)); with q = prod q_l the ring element is held
 * as its L residue polynomials (Chinese remainder theorem), limb-major [L][N].
 *
 * Conventions the paper leaves open (sampler, stream map, primes, slots) are
 * documented with the functions below; they are inputs or explicit parameters
 * wherever possible so that tests can pin them independently.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

#define ORC_MAX_LIMBS 24
#define ORC_CDT_LEN 38 /* thresholds for the support [-19, 19] */

typedef struct {
  uint32_t log2_n;     /* ring degree N = 2^log2_n                      */
  uint32_t num_limbs;  /* L                                             */
  uint64_t moduli[ORC_MAX_LIMBS]; /* q_l, distinct primes = 1 mod 2N    */
  uint64_t plain_modulus;         /* t                                  */
  uint64_t psi_t;      /* primitive 2N-th root of unity mod t (slots)   */
  uint64_t seed;       /* Philox key                                    */
  uint64_t cdt[ORC_CDT_LEN]; /* cumulative Gaussian thresholds, see orc_gauss */
  int32_t gauss_bound; /* B: support of chi is [-B, B] (B = 19)         */
} orc_params;

/* ------------------------------------------------------------------ */
/* Arithmetic in Z_p, p < 2^63                                         */
/* ------------------------------------------------------------------ */

static uint64_t addm(uint64_t a, uint64_t b, uint64_t p) {
  return (uint64_t)(((u128)a + b) % p);
}
static uint64_t subm(uint64_t a, uint64_t b, uint64_t p) {
  return (uint64_t)(((u128)a + p - (b % p)) % p);
}
static uint64_t mulm(uint64_t a, uint64_t b, uint64_t p) {
  return (uint64_t)(((u128)a * b) % p);
}
static uint64_t powm(uint64_t a, uint64_t e, uint64_t p) {
  uint64_t r = 1 % p;
  a %= p;
  while (e) {
    if (e & 1) r = mulm(r, a, p);
    a = mulm(a, a, p);
    e >>= 1;
  }
  return r;
}
static uint64_t invm(uint64_t a, uint64_t p) { return powm(a, p - 2, p); }

/* residue of a small signed integer */
static uint64_t lift(int64_t v, uint64_t p) {
  int64_t r = v % (int64_t)p;
  if (r < 0) r += (int64_t)p;
  return (uint64_t)r;
}

uint64_t orc_mulmod(uint64_t a, uint64_t b, uint64_t p) { return mulm(a, b, p); }
uint64_t orc_powmod(uint64_t a, uint64_t e, uint64_t p) { return powm(a, e, p); }

/*
 * A primitive 2N-th root of unity mod p (p = 1 mod 2N): the first
 * g^((p-1)/2N), g = 2, 3, ..., whose N-th power is -1.  Which root is used
 * does not change any coefficient-domain result.
 */
uint64_t orc_find_psi(uint64_t p, uint32_t log2_n) {
  uint64_t two_n = (uint64_t)2 << log2_n;
  uint64_t n = (uint64_t)1 << log2_n;
  if ((p - 1) % two_n) return 0;
  for (uint64_t g = 2; g < 1000; ++g) {
    uint64_t c = powm(g, (p - 1) / two_n, p);
    if (powm(c, n, p) == p - 1) return c;
  }
  return 0;
}

/* ------------------------------------------------------------------ */
/* Ring product: definition and textbook transform                     */
/* ------------------------------------------------------------------ */

/*
 * Product in Z_p[X]/(X^N+1) straight from the definition (Sec. 3.2):
 * c_k = sum_{i+j=k} a_i b_j - sum_{i+j=k+N} a_i b_j  (X^N = -1).  O(N^2).
 */
void orc_negacyclic_schoolbook(const uint64_t* a, const uint64_t* b, uint64_t* c,
                               uint32_t n, uint64_t p) {
  for (uint32_t k = 0; k < n; ++k) c[k] = 0;
  for (uint32_t i = 0; i < n; ++i) {
    for (uint32_t j = 0; j < n; ++j) {
      uint64_t prod = mulm(a[i], b[j], p);
      uint32_t k = i + j;
      if (k < n)
        c[k] = addm(c[k], prod, p);
      else
        c[k - n] = subm(c[k - n], prod, p);
    }
  }
}

/* One coefficient of the same product, for spot checks at large N. */
uint64_t orc_negacyclic_coeff(const uint64_t* a, const uint64_t* b, uint32_t n,
                              uint64_t p, uint32_t k) {
  uint64_t acc = 0;
  for (uint32_t i = 0; i < n; ++i) {
    uint32_t j = (k + n - i) % n; /* i + j = k or k + N */
    uint64_t prod = mulm(a[i], b[j], p);
    if (i + j == k)
      acc = addm(acc, prod, p);
    else
      acc = subm(acc, prod, p);
  }
  return acc;
}

static uint32_t bitrev(uint32_t x, uint32_t bits) {
  uint32_t r = 0;
  for (uint32_t i = 0; i < bits; ++i) {
    r = (r << 1) | (x & 1);
    x >>= 1;
  }
  return r;
}

/*
 * Textbook cyclic DFT over Z_p: y[j] = sum_i x[i] w^(ij), w of order n.
 * Bit-reversal copy followed by log2 n passes of radix-2 butterflies.
 */
static void cyclic_dft(uint64_t* x, uint32_t log2_n, uint64_t w, uint64_t p) {
  uint32_t n = 1u << log2_n;
  for (uint32_t i = 0; i < n; ++i) {
    uint32_t r = bitrev(i, log2_n);
    if (i < r) {
      uint64_t tmp = x[i];
      x[i] = x[r];
      x[r] = tmp;
    }
  }
  for (uint32_t len = 2; len <= n; len <<= 1) {
    uint64_t wlen = powm(w, n / len, p);
    for (uint32_t start = 0; start < n; start += len) {
      uint64_t wk = 1;
      for (uint32_t k = 0; k < len / 2; ++k) {
        uint64_t u = x[start + k];
        uint64_t v = mulm(x[start + k + len / 2], wk, p);
        x[start + k] = addm(u, v, p);
        x[start + k + len / 2] = subm(u, v, p);
        wk = mulm(wk, wlen, p);
      }
    }
  }
}

/*
 * Evaluate a at the odd powers of psi, natural order: out[j] = a(psi^(2j+1)).
 * a(psi^(2j+1)) = sum_i (a_i psi^i) (psi^2)^(ij): a twist followed by the
 * cyclic DFT with w = psi^2.  These N points are the roots of X^N+1, so the
 * map is the ring isomorphism Z_p[X]/(X^N+1) -> Z_p^N.
 */
void orc_negacyclic_eval(const uint64_t* a, uint64_t* out, uint32_t log2_n,
                         uint64_t psi, uint64_t p) {
  uint32_t n = 1u << log2_n;
  uint64_t pw = 1;
  for (uint32_t i = 0; i < n; ++i) {
    out[i] = mulm(a[i] % p, pw, p);
    pw = mulm(pw, psi, p);
  }
  cyclic_dft(out, log2_n, mulm(psi, psi, p), p);
}

/* Inverse of orc_negacyclic_eval: the unique a of degree < N with the given values. */
void orc_negacyclic_interp(const uint64_t* vals, uint64_t* a, uint32_t log2_n,
                           uint64_t psi, uint64_t p) {
  uint32_t n = 1u << log2_n;
  uint64_t winv = invm(mulm(psi, psi, p), p);
  uint64_t psinv = invm(psi, p);
  uint64_t ninv = invm(n % p, p);
  for (uint32_t i = 0; i < n; ++i) a[i] = vals[i] % p;
  cyclic_dft(a, log2_n, winv, p);
  uint64_t pw = ninv;
  for (uint32_t i = 0; i < n; ++i) {
    a[i] = mulm(a[i], pw, p);
    pw = mulm(pw, psinv, p);
  }
}

/* c = a*b in Z_p[X]/(X^N+1) through evaluation, pointwise product, interpolation. */
void orc_ring_mul(const uint64_t* a, const uint64_t* b, uint64_t* c,
                  uint32_t log2_n, uint64_t p) {
  uint32_t n = 1u << log2_n;
  uint64_t psi = orc_find_psi(p, log2_n);
  uint64_t* fa = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* fb = (uint64_t*)malloc(sizeof(uint64_t) * n);
  orc_negacyclic_eval(a, fa, log2_n, psi, p);
  orc_negacyclic_eval(b, fb, log2_n, psi, p);
  for (uint32_t i = 0; i < n; ++i) fa[i] = mulm(fa[i], fb[i], p);
  orc_negacyclic_interp(fa, c, log2_n, psi, p);
  free(fa);
  free(fb);
}

/* Horner evaluation of a polynomial at one point (pin for encode/decode). */
uint64_t orc_horner(const uint64_t* a, uint32_t n, uint64_t x, uint64_t p) {
  uint64_t acc = 0;
  for (uint32_t i = n; i-- > 0;) acc = addm(mulm(acc, x, p), a[i] % p, p);
  return acc;
}

/* d = a (.) b + c, limb by limb, residue by residue (the RNS multiply-add). */
void orc_poly_muladd(const orc_params* P, const uint64_t* a, const uint64_t* b,
                     const uint64_t* c, uint64_t* d, uint32_t batch) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  for (uint32_t r = 0; r < batch; ++r)
    for (uint32_t l = 0; l < L; ++l) {
      uint64_t p = P->moduli[l];
      size_t base = ((size_t)r * L + l) * n;
      for (uint32_t j = 0; j < n; ++j)
        d[base + j] = addm(mulm(a[base + j], b[base + j], p), c[base + j], p);
    }
}

/* ------------------------------------------------------------------ */
/* Counter-based randomness: Philox4x32-10 (Salmon, Moraes, Dror, Shaw; SC'11) */
/* ------------------------------------------------------------------ */

void orc_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += W0;
      k1 += W1;
    }
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t h0 = (uint32_t)(p0 >> 32), l0 = (uint32_t)p0;
    uint32_t h1 = (uint32_t)(p1 >> 32), l1 = (uint32_t)p1;
    uint32_t n0 = h1 ^ c1 ^ k0;
    uint32_t n1 = l1;
    uint32_t n2 = h0 ^ c3 ^ k1;
    uint32_t n3 = l0;
    c0 = n0;
    c1 = n1;
    c2 = n2;
    c3 = n3;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

/* Stream tags: which random object a Philox call belongs to. */
enum {
  TAG_SECRET = 1,   /* s_k            (Sec. 4.2 item 1)                 */
  TAG_PK_ERR = 2,   /* e_k            (Sec. 4.2 item 2)                 */
  TAG_P1 = 3,       /* common p_1     (Sec. 4.2 item 2)                 */
  TAG_ENC_U = 4,    /* mu             (Sec. 3.2 item 3)                 */
  TAG_ENC_E0 = 5,   /* e_0            (Sec. 3.2 item 3)                 */
  TAG_ENC_E1 = 6,   /* e_1            (Sec. 3.2 item 3)                 */
  TAG_DEC_ERR = 7,  /* e_{0,k} in a decryption share (Eq. 2)            */
  TAG_USER_SECRET = 8,  /* sk_i of a user's own key pair (Algorithm 2, Require) */
  TAG_USER_PK_ERR = 9,  /* e_i of pk_i                                   */
  TAG_USER_P1 = 10,     /* p_{1,i} of pk_i                               */
  TAG_CONV_MU = 11,     /* mu_k of MBFV.Convert (Eq. 2)                  */
  TAG_CONV_E0 = 12,     /* e_{0,k} of MBFV.Convert                       */
  TAG_CONV_E1 = 13,     /* e_{1,k} of MBFV.Convert                       */
  TAG_BOOT_ALPHA = 14,  /* common polynomial alpha of MBFV.Bootstrap      */
  TAG_BOOT_MASK = 15,   /* M_k over R_t (Eq. 4)                          */
  TAG_BOOT_E0 = 16,     /* e_{0,k} of MBFV.Bootstrap                     */
  TAG_BOOT_E1 = 17      /* e_{1,k} of MBFV.Bootstrap                     */
};

/*
 * One Philox call per sample.  Key = (seed low word, seed high word).
 * Counter = (coefficient index j, idx, party | recipient << 16, tag | attempt << 8)
 * where idx is the ciphertext index (limb index for p_1, 0 for key material).
 */
static void draw(const orc_params* P, uint32_t tag, uint32_t attempt, uint32_t j,
                 uint32_t idx, uint32_t party, uint32_t recipient, uint32_t w[4]) {
  uint32_t key[2] = {(uint32_t)(P->seed & 0xffffffffu), (uint32_t)(P->seed >> 32)};
  uint32_t ctr[4] = {j, idx, party | (recipient << 16), tag | (attempt << 8)};
  orc_philox4x32_10(key, ctr, w);
}

/* R_3: a coefficient uniform in {-1, 0, 1} from one 32-bit word: floor(3 w / 2^32) - 1. */
static int32_t ternary_from_word(uint32_t w0) {
  return (int32_t)(((uint64_t)w0 * 3u) >> 32) - 1;
}

/*
 * chi: centred discrete Gaussian, sigma = 3.2, support [-B, B].  Inversion of the
 * cumulative table: cdt[k] = floor(2^64 * Pr[x <= -B + k]); the sample is
 * -B + #{k : r >= cdt[k]} for a uniform 64-bit r.  Integer compares only.
 */
static int32_t gauss_from_r(const orc_params* P, uint64_t r) {
  int32_t count = 0;
  for (int k = 0; k < 2 * P->gauss_bound; ++k)
    if (r >= P->cdt[k]) ++count;
  return -P->gauss_bound + count;
}

static uint32_t bit_length(uint64_t x) {
  uint32_t b = 0;
  while (x) {
    ++b;
    x >>= 1;
  }
  return b;
}

/*
 * Uniform element of Z_p by rejection: mask a 64-bit draw to bitlen(p) bits and
 * accept if below p; otherwise redraw with attempt+1.  Attempt 255 is the last:
 * its unmasked draw is reduced mod p.
 */
static uint64_t uniform_mod(const orc_params* P, uint32_t tag, uint32_t j, uint32_t idx,
                            uint32_t party, uint64_t p) {
  uint32_t bits = bit_length(p);
  uint64_t mask = bits >= 64 ? ~(uint64_t)0 : (((uint64_t)1 << bits) - 1);
  uint32_t w[4];
  for (uint32_t attempt = 0; attempt < 255; ++attempt) {
    draw(P, tag, attempt, j, idx, party, 0, w);
    uint64_t r = (((uint64_t)w[0] << 32) | w[1]) & mask;
    if (r < p) return r;
  }
  draw(P, tag, 255, j, idx, party, 0, w);
  return (((uint64_t)w[0] << 32) | w[1]) % p;
}

void orc_sample_ternary(const orc_params* P, uint32_t tag, uint32_t idx, uint32_t party,
                        uint32_t recipient, int8_t* out) {
  uint32_t n = 1u << P->log2_n, w[4];
  for (uint32_t j = 0; j < n; ++j) {
    draw(P, tag, 0, j, idx, party, recipient, w);
    out[j] = (int8_t)ternary_from_word(w[0]);
  }
}

void orc_sample_gauss(const orc_params* P, uint32_t tag, uint32_t idx, uint32_t party,
                      uint32_t recipient, int8_t* out) {
  uint32_t n = 1u << P->log2_n, w[4];
  for (uint32_t j = 0; j < n; ++j) {
    draw(P, tag, 0, j, idx, party, recipient, w);
    out[j] = (int8_t)gauss_from_r(P, ((uint64_t)w[0] << 32) | w[1]);
  }
}

/* raw access for distribution tests */
int32_t orc_gauss_from_r(const orc_params* P, uint64_t r) { return gauss_from_r(P, r); }
int32_t orc_ternary_from_word(uint32_t w) { return ternary_from_word(w); }

/* ------------------------------------------------------------------ */
/* Keys (Sec. 3.2 items 1-2, Sec. 4.2 items 1-2)                       */
/* ------------------------------------------------------------------ */

/* MBFV.SecKeyGen: party k draws s_k from R_3 by BFV.SecKeyGen. */
void orc_secret_share(const orc_params* P, uint32_t party, int8_t* s) {
  orc_sample_ternary(P, TAG_SECRET, 0, party, 0, s);
}

/* e_k from chi for the public-key share. */
void orc_pk_error(const orc_params* P, uint32_t party, int8_t* e) {
  orc_sample_gauss(P, TAG_PK_ERR, 0, party, 0, e);
}

/* The common polynomial p_1, uniform on R_q: limb l, coefficient j independent. */
void orc_common_p1(const orc_params* P, uint64_t* p1 /*[L][N]*/) {
  uint32_t n = 1u << P->log2_n;
  for (uint32_t l = 0; l < P->num_limbs; ++l)
    for (uint32_t j = 0; j < n; ++j)
      p1[(size_t)l * n + j] = uniform_mod(P, TAG_P1, j, l, 0, P->moduli[l]);
}

static void small_to_limb(const int8_t* v, uint64_t* out, uint32_t n, uint64_t p) {
  for (uint32_t j = 0; j < n; ++j) out[j] = lift(v[j], p);
}

/* p_{0,k} = -(p_1 s_k + e_k)   (MBFV.PubKeyGen) */
void orc_pk_share(const orc_params* P, uint32_t party, const uint64_t* p1, uint64_t* p0k) {
  uint32_t n = 1u << P->log2_n;
  int8_t* s = (int8_t*)malloc(n);
  int8_t* e = (int8_t*)malloc(n);
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* prod = (uint64_t*)malloc(sizeof(uint64_t) * n);
  orc_secret_share(P, party, s);
  orc_pk_error(P, party, e);
  for (uint32_t l = 0; l < P->num_limbs; ++l) {
    uint64_t p = P->moduli[l];
    small_to_limb(s, sl, n, p);
    orc_ring_mul(p1 + (size_t)l * n, sl, prod, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      p0k[(size_t)l * n + j] = subm(0, addm(prod[j], lift(e[j], p), p), p);
  }
  free(s);
  free(e);
  free(sl);
  free(prod);
}

/* pk = ([sum_k p_{0,k}]_q, p_1) over the listed parties; pk is [2][L][N]. */
void orc_collective_pk(const orc_params* P, const uint32_t* parties, uint32_t n_parties,
                       uint64_t* pk) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  uint64_t* share = (uint64_t*)malloc(sizeof(uint64_t) * poly);
  orc_common_p1(P, pk + poly);
  memset(pk, 0, sizeof(uint64_t) * poly);
  for (uint32_t i = 0; i < n_parties; ++i) {
    orc_pk_share(P, parties[i], pk + poly, share);
    for (uint32_t l = 0; l < L; ++l)
      for (uint32_t j = 0; j < n; ++j)
        pk[(size_t)l * n + j] = addm(pk[(size_t)l * n + j], share[(size_t)l * n + j], P->moduli[l]);
  }
  free(share);
}

/* ------------------------------------------------------------------ */
/* Packing (Sec. 6: SIMD packing of many values into one plaintext)    */
/* ------------------------------------------------------------------ */

/* encode: the m in R_t with m(psi_t^(2j+1)) = v_j mod t for every slot j. */
void orc_encode(const orc_params* P, const int32_t* values, uint32_t* plain) {
  uint32_t n = 1u << P->log2_n;
  uint64_t t = P->plain_modulus;
  uint64_t* v = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* m = (uint64_t*)malloc(sizeof(uint64_t) * n);
  for (uint32_t j = 0; j < n; ++j) v[j] = lift(values[j], t);
  orc_negacyclic_interp(v, m, P->log2_n, P->psi_t, t);
  for (uint32_t j = 0; j < n; ++j) plain[j] = (uint32_t)m[j];
  free(v);
  free(m);
}

/* decode: y_j = m(psi_t^(2j+1)) mod t, lifted to (-t/2, t/2). */
void orc_decode(const orc_params* P, const uint32_t* plain, int32_t* values) {
  uint32_t n = 1u << P->log2_n;
  uint64_t t = P->plain_modulus;
  uint64_t* m = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* y = (uint64_t*)malloc(sizeof(uint64_t) * n);
  for (uint32_t j = 0; j < n; ++j) m[j] = plain[j];
  orc_negacyclic_eval(m, y, P->log2_n, P->psi_t, t);
  for (uint32_t j = 0; j < n; ++j)
    values[j] = y[j] > (t - 1) / 2 ? (int32_t)((int64_t)y[j] - (int64_t)t) : (int32_t)y[j];
  free(m);
  free(y);
}

/* ------------------------------------------------------------------ */
/* Big integers (32-bit words, little endian) for CRT and the rounding */
/* ------------------------------------------------------------------ */

#define BN_WORDS 64
typedef struct {
  uint32_t w[BN_WORDS];
} bn;

static void bn_zero(bn* a) { memset(a->w, 0, sizeof(a->w)); }
static void bn_from_u64(bn* a, uint64_t v) {
  bn_zero(a);
  a->w[0] = (uint32_t)v;
  a->w[1] = (uint32_t)(v >> 32);
}
static int bn_cmp(const bn* a, const bn* b) {
  for (int i = BN_WORDS - 1; i >= 0; --i) {
    if (a->w[i] > b->w[i]) return 1;
    if (a->w[i] < b->w[i]) return -1;
  }
  return 0;
}
static void bn_add(bn* a, const bn* b) {
  uint64_t carry = 0;
  for (int i = 0; i < BN_WORDS; ++i) {
    uint64_t s = (uint64_t)a->w[i] + b->w[i] + carry;
    a->w[i] = (uint32_t)s;
    carry = s >> 32;
  }
}
static void bn_sub(bn* a, const bn* b) { /* a >= b */
  int64_t borrow = 0;
  for (int i = 0; i < BN_WORDS; ++i) {
    int64_t d = (int64_t)a->w[i] - b->w[i] - borrow;
    borrow = d < 0;
    a->w[i] = (uint32_t)(d + (borrow ? ((int64_t)1 << 32) : 0));
  }
}
static void bn_mul_u64(bn* a, uint64_t m) {
  uint32_t mw[2] = {(uint32_t)m, (uint32_t)(m >> 32)};
  bn r;
  bn_zero(&r);
  for (int k = 0; k < 2; ++k) {
    uint64_t carry = 0;
    for (int i = 0; i + k < BN_WORDS; ++i) {
      uint64_t cur = (uint64_t)a->w[i] * mw[k] + r.w[i + k] + carry;
      r.w[i + k] = (uint32_t)cur;
      carry = cur >> 32;
    }
  }
  *a = r;
}
static void bn_shl1(bn* a) {
  uint32_t carry = 0;
  for (int i = 0; i < BN_WORDS; ++i) {
    uint32_t nc = a->w[i] >> 31;
    a->w[i] = (a->w[i] << 1) | carry;
    carry = nc;
  }
}
static uint64_t bn_mod_u64(const bn* a, uint64_t m) {
  u128 r = 0;
  for (int i = BN_WORDS - 1; i >= 0; --i) r = ((r << 32) | a->w[i]) % m;
  return (uint64_t)r;
}

typedef struct {
  bn q;                      /* prod q_l                             */
  bn qhat[ORC_MAX_LIMBS];    /* q / q_l                              */
  uint64_t qhat_inv[ORC_MAX_LIMBS]; /* (q/q_l)^-1 mod q_l            */
  bn two_q_shift[33];        /* 2q << b, b = 0..32                   */
} crt_ctx;

static void crt_init(const orc_params* P, crt_ctx* C) {
  uint32_t L = P->num_limbs;
  bn_from_u64(&C->q, 1);
  for (uint32_t l = 0; l < L; ++l) bn_mul_u64(&C->q, P->moduli[l]);
  for (uint32_t l = 0; l < L; ++l) {
    bn_from_u64(&C->qhat[l], 1);
    for (uint32_t m = 0; m < L; ++m)
      if (m != l) bn_mul_u64(&C->qhat[l], P->moduli[m]);
    C->qhat_inv[l] = invm(bn_mod_u64(&C->qhat[l], P->moduli[l]), P->moduli[l]);
  }
  C->two_q_shift[0] = C->q;
  bn_shl1(&C->two_q_shift[0]);
  for (int b = 1; b <= 32; ++b) {
    C->two_q_shift[b] = C->two_q_shift[b - 1];
    bn_shl1(&C->two_q_shift[b]);
  }
}

/* The integer v in [0, q) with v = r_l mod q_l for all l (Chinese remainder theorem). */
static void crt_compose(const orc_params* P, const crt_ctx* C, const uint64_t* r, bn* v) {
  bn_zero(v);
  for (uint32_t l = 0; l < P->num_limbs; ++l) {
    bn term = C->qhat[l];
    bn_mul_u64(&term, mulm(r[l] % P->moduli[l], C->qhat_inv[l], P->moduli[l]));
    bn_add(v, &term);
  }
  while (bn_cmp(v, &C->q) >= 0) bn_sub(v, &C->q);
}

/*
 * BFV.Decrypt's rounding (Sec. 3.2 item 5): x = [ round(t v / q) ]_t for
 * v = [c_0 + c_1 s]_q taken in [0, q).  round(t v / q) = floor((2 t v + q) / (2 q));
 * the quotient is at most t < 2^32, found by restoring division on 33 bits.
 * (Taking the representative in (-q/2, q/2] instead changes the result by a
 * multiple of t only.)
 */
static uint32_t scale_round(const orc_params* P, const crt_ctx* C, const bn* v) {
  bn num = *v;
  bn_mul_u64(&num, 2 * P->plain_modulus);
  bn_add(&num, &C->q);
  uint64_t quot = 0;
  for (int b = 32; b >= 0; --b) {
    if (bn_cmp(&num, &C->two_q_shift[b]) >= 0) {
      bn_sub(&num, &C->two_q_shift[b]);
      quot |= (uint64_t)1 << b;
    }
  }
  return (uint32_t)(quot % P->plain_modulus);
}

/* floor(q / t) mod q_l for every limb: the Lambda of Sec. 3.2. */
static void delta_residues(const orc_params* P, const crt_ctx* C, uint64_t* delta) {
  /* q = Lambda t + (q mod t)  =>  Lambda = (q - (q mod t)) / t exactly. */
  uint64_t t = P->plain_modulus;
  uint64_t q_mod_t = bn_mod_u64(&C->q, t);
  for (uint32_t l = 0; l < P->num_limbs; ++l) {
    uint64_t p = P->moduli[l];
    /* (q - q mod t) = -(q mod t) mod q_l since q = 0 mod q_l */
    delta[l] = mulm(subm(0, q_mod_t % p, p), invm(t % p, p), p);
  }
}

void orc_delta(const orc_params* P, uint64_t* delta) {
  crt_ctx* C = (crt_ctx*)malloc(sizeof(crt_ctx));
  crt_init(P, C);
  delta_residues(P, C, delta);
  free(C);
}

/* Expose composition + rounding for the big-integer pins. */
uint32_t orc_scale_round_residues(const orc_params* P, const uint64_t* residues) {
  crt_ctx* C = (crt_ctx*)malloc(sizeof(crt_ctx));
  crt_init(P, C);
  bn v;
  crt_compose(P, C, residues, &v);
  uint32_t x = scale_round(P, C, &v);
  free(C);
  return x;
}

/* v as 32-bit words (little endian), for comparison with Python integers. */
void orc_crt_words(const orc_params* P, const uint64_t* residues, uint32_t* words64) {
  crt_ctx* C = (crt_ctx*)malloc(sizeof(crt_ctx));
  crt_init(P, C);
  bn v;
  crt_compose(P, C, residues, &v);
  memcpy(words64, v.w, sizeof(v.w));
  free(C);
}

/* ------------------------------------------------------------------ */
/* Encrypt, add, decryption shares, combine                            */
/* ------------------------------------------------------------------ */

/*
 * BFV.Encrypt (Sec. 3.2 item 3): ct = (Lambda m + u p_0 + e_0, u p_1 + e_1),
 * u from R_3, e_0, e_1 from chi, drawn on the stream (party, ct_index).
 * plain is m in [0,t)^N; ct is [2][L][N].
 */
void orc_encrypt(const orc_params* P, const uint64_t* pk, uint32_t party, uint32_t ct_index,
                 const uint32_t* plain, uint64_t* ct) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int8_t* u = (int8_t*)malloc(n);
  int8_t* e0 = (int8_t*)malloc(n);
  int8_t* e1 = (int8_t*)malloc(n);
  uint64_t* ul = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* prod = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t delta[ORC_MAX_LIMBS];
  orc_delta(P, delta);
  orc_sample_ternary(P, TAG_ENC_U, ct_index, party, 0, u);
  orc_sample_gauss(P, TAG_ENC_E0, ct_index, party, 0, e0);
  orc_sample_gauss(P, TAG_ENC_E1, ct_index, party, 0, e1);
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    small_to_limb(u, ul, n, p);
    orc_ring_mul(ul, pk + (size_t)l * n, prod, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j) {
      uint64_t dm = mulm(delta[l], plain[j] % p, p);
      ct[(size_t)l * n + j] = addm(addm(dm, prod[j], p), lift(e0[j], p), p);
    }
    orc_ring_mul(ul, pk + poly + (size_t)l * n, prod, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      ct[poly + (size_t)l * n + j] = addm(prod[j], lift(e1[j], p), p);
  }
  free(u);
  free(e0);
  free(e1);
  free(ul);
  free(prod);
}

/*
 * BFV.Add over a list (the neighbour-sum step of Algorithm 2, with unit weights): out = sum of the
 * listed ciphertexts, component by component, mod q.  cts is [n_rows][2][L][N].
 */
void orc_aggregate(const orc_params* P, const uint64_t* cts, const uint32_t* rows,
                   uint32_t n_list, uint64_t* out) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t ct_words = (size_t)2 * L * n;
  memset(out, 0, sizeof(uint64_t) * ct_words);
  for (uint32_t a = 0; a < n_list; ++a) {
    const uint64_t* src = cts + (size_t)rows[a] * ct_words;
    for (uint32_t comp = 0; comp < 2; ++comp)
      for (uint32_t l = 0; l < L; ++l)
        for (uint32_t j = 0; j < n; ++j) {
          size_t o = ((size_t)comp * L + l) * n + j;
          out[o] = addm(out[o], src[o], P->moduli[l]);
        }
  }
}

/*
 * Decryption share of party k for recipient i (Eq. 2 with mu_k = 0, i.e. the
 * first component with no re-encryption term): h = s_k c_1 + e, e from chi on
 * the stream (party, recipient, ct_index).  c1 and h are [L][N].
 */
void orc_partial_decrypt(const orc_params* P, uint32_t party, uint32_t recipient,
                         uint32_t ct_index, const uint64_t* c1, uint64_t* h) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  int8_t* s = (int8_t*)malloc(n);
  int8_t* e = (int8_t*)malloc(n);
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  orc_secret_share(P, party, s);
  orc_sample_gauss(P, TAG_DEC_ERR, ct_index, party, recipient, e);
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    small_to_limb(s, sl, n, p);
    orc_ring_mul(sl, c1 + (size_t)l * n, h + (size_t)l * n, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      h[(size_t)l * n + j] = addm(h[(size_t)l * n + j], lift(e[j], p), p);
  }
  free(s);
  free(e);
  free(sl);
}

/*
 * Combine (Sec. 4.2 item 3 then Sec. 3.2 item 5): v = [c_0 + sum_k h_k]_q,
 * x = [round(t v / q)]_t.  c0 is [L][N]; shares is [n_shares][L][N].
 */
void orc_combine(const orc_params* P, const uint64_t* c0, const uint64_t* shares,
                 uint32_t n_shares, uint32_t* plain) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  crt_ctx* C = (crt_ctx*)malloc(sizeof(crt_ctx));
  crt_init(P, C);
  for (uint32_t j = 0; j < n; ++j) {
    uint64_t r[ORC_MAX_LIMBS];
    for (uint32_t l = 0; l < L; ++l) {
      uint64_t p = P->moduli[l];
      uint64_t acc = c0[(size_t)l * n + j] % p;
      for (uint32_t k = 0; k < n_shares; ++k)
        acc = addm(acc, shares[(size_t)k * poly + (size_t)l * n + j], p);
      r[l] = acc;
    }
    bn v;
    crt_compose(P, C, r, &v);
    plain[j] = scale_round(P, C, &v);
  }
  free(C);
}

/*
 * BFV.Decrypt with an explicit (small integer) secret: x = [round(t/q [c_0 + c_1 s]_q)]_t.
 * Used to check that collective decryption equals decryption under s = sum_k s_k.
 * Also returns, when noise != NULL, the centred value of c_0 + c_1 s - Lambda m
 * (m = the decrypted plaintext) per coefficient; it must fit in 63 bits.
 */
int orc_decrypt_single(const orc_params* P, const uint64_t* ct, const int32_t* s,
                       uint32_t* plain, int64_t* noise) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* v = (uint64_t*)malloc(sizeof(uint64_t) * poly);
  uint64_t delta[ORC_MAX_LIMBS];
  crt_ctx* C = (crt_ctx*)malloc(sizeof(crt_ctx));
  crt_init(P, C);
  delta_residues(P, C, delta);
  int status = 0;
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    for (uint32_t j = 0; j < n; ++j) sl[j] = lift(s[j], p);
    orc_ring_mul(sl, ct + poly + (size_t)l * n, v + (size_t)l * n, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      v[(size_t)l * n + j] = addm(v[(size_t)l * n + j], ct[(size_t)l * n + j], p);
  }
  bn half_q = C->q; /* floor(q/2) */
  for (int i = 0; i < BN_WORDS; ++i) {
    uint32_t lo = half_q.w[i] >> 1;
    uint32_t hi = i + 1 < BN_WORDS ? (half_q.w[i + 1] & 1u) << 31 : 0;
    half_q.w[i] = lo | hi;
  }
  for (uint32_t j = 0; j < n; ++j) {
    uint64_t r[ORC_MAX_LIMBS];
    for (uint32_t l = 0; l < L; ++l) r[l] = v[(size_t)l * n + j];
    bn big;
    crt_compose(P, C, r, &big);
    plain[j] = scale_round(P, C, &big);
    if (noise) {
      for (uint32_t l = 0; l < L; ++l)
        r[l] = subm(r[l], mulm(delta[l], plain[j] % P->moduli[l], P->moduli[l]), P->moduli[l]);
      crt_compose(P, C, r, &big);
      int negative = bn_cmp(&big, &half_q) > 0;
      if (negative) {
        bn tmp = C->q;
        bn_sub(&tmp, &big);
        big = tmp;
      }
      for (int i = 2; i < BN_WORDS; ++i)
        if (big.w[i]) status = -1;
      if (big.w[1] >> 31) status = -1;
      int64_t mag = (int64_t)(((uint64_t)big.w[1] << 32) | big.w[0]);
      noise[j] = negative ? -mag : mag;
    }
  }
  free(sl);
  free(v);
  free(C);
  return status;
}

/* ------------------------------------------------------------------ */
/* MBFV.Convert to a recipient's own key (Sec. 4.2 item 3, Eq. 2-3)    */
/* ------------------------------------------------------------------ */

/* sk_i of user i's own BFV key pair (Algorithm 2, Require): BFV.SecKeyGen. */
void orc_user_secret(const orc_params* P, uint32_t user, int8_t* s) {
  orc_sample_ternary(P, TAG_USER_SECRET, 0, user, 0, s);
}

/* pk_i = (-(sk_i p_{1,i} + e_i), p_{1,i}) (BFV.PubKeyGen, Sec. 3.2 item 2); pk is [2][L][N]. */
void orc_user_pk(const orc_params* P, uint32_t user, uint64_t* pk) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int8_t* s = (int8_t*)malloc(n);
  int8_t* e = (int8_t*)malloc(n);
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* prod = (uint64_t*)malloc(sizeof(uint64_t) * n);
  orc_user_secret(P, user, s);
  orc_sample_gauss(P, TAG_USER_PK_ERR, 0, user, 0, e);
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    uint64_t* p1 = pk + poly + (size_t)l * n;
    for (uint32_t j = 0; j < n; ++j) p1[j] = uniform_mod(P, TAG_USER_P1, j, l, user, p);
    small_to_limb(s, sl, n, p);
    orc_ring_mul(p1, sl, prod, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      pk[(size_t)l * n + j] = subm(0, addm(prod[j], lift(e[j], p), p), p);
  }
  free(s);
  free(e);
  free(sl);
  free(prod);
}

/*
 * Conversion share of party k for recipient i (Eq. 2):
 *   (h_0, h_1) = (s_k c_1 + mu_k p_{0,i} + e_{0,k},  mu_k p_{1,i} + e_{1,k}),
 * mu_k, e_{0,k}, e_{1,k} from chi on the stream (party, recipient, ct_index).
 * pk_i is [2][L][N], c1 is [L][N], h is [2][L][N].
 */
void orc_convert_share(const orc_params* P, const uint64_t* pk_i, uint32_t party, uint32_t recipient,
                       uint32_t ct_index, const uint64_t* c1, uint64_t* h) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int8_t* s = (int8_t*)malloc(n);
  int8_t* mu = (int8_t*)malloc(n);
  int8_t* e0 = (int8_t*)malloc(n);
  int8_t* e1 = (int8_t*)malloc(n);
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* ml = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* a = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* b = (uint64_t*)malloc(sizeof(uint64_t) * n);
  orc_secret_share(P, party, s);
  orc_sample_gauss(P, TAG_CONV_MU, ct_index, party, recipient, mu);
  orc_sample_gauss(P, TAG_CONV_E0, ct_index, party, recipient, e0);
  orc_sample_gauss(P, TAG_CONV_E1, ct_index, party, recipient, e1);
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    small_to_limb(s, sl, n, p);
    small_to_limb(mu, ml, n, p);
    orc_ring_mul(sl, c1 + (size_t)l * n, a, P->log2_n, p);
    orc_ring_mul(ml, pk_i + (size_t)l * n, b, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j)
      h[(size_t)l * n + j] = addm(addm(a[j], b[j], p), lift(e0[j], p), p);
    orc_ring_mul(ml, pk_i + poly + (size_t)l * n, b, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j) h[poly + (size_t)l * n + j] = addm(b[j], lift(e1[j], p), p);
  }
  free(s);
  free(mu);
  free(e0);
  free(e1);
  free(sl);
  free(ml);
  free(a);
  free(b);
}

/* agg [n_rec][n_cts][2][L][N], pk_users [n_rec][2][L][N] -> shares [n_rec][n_parties][n_cts][2][L][N]. */
void orc_convert_share_batch(const orc_params* P, const uint64_t* agg, const uint64_t* pk_users,
                             const uint32_t* recipients, uint32_t n_rec, const uint32_t* parties,
                             uint32_t n_parties, uint32_t ct_first, uint32_t n_cts, uint64_t* shares) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int64_t total = (int64_t)n_rec * n_parties * n_cts;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < total; ++u) {
    uint32_t c = (uint32_t)(u % n_cts);
    uint32_t k = (uint32_t)((u / n_cts) % n_parties);
    uint32_t i = (uint32_t)(u / ((int64_t)n_cts * n_parties));
    const uint64_t* c1 = agg + (((size_t)i * n_cts + c) * 2 + 1) * poly;
    orc_convert_share(P, pk_users + (size_t)i * 2 * poly, parties[k], recipients[i], ct_first + c, c1,
                      shares + (size_t)u * 2 * poly);
  }
}

/* ct' = (c_0 + sum_k h_{0,k}, sum_k h_{1,k}); out [n_rec][n_cts][2][L][N]. */
void orc_convert_combine_batch(const orc_params* P, const uint64_t* agg, const uint64_t* shares,
                               uint32_t n_rec, uint32_t n_shares, uint32_t n_cts, uint64_t* out) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_rec * n_cts; ++u) {
    uint32_t i = (uint32_t)(u / n_cts), c = (uint32_t)(u % n_cts);
    for (uint32_t comp = 0; comp < 2; ++comp)
      for (uint32_t l = 0; l < L; ++l)
        for (uint32_t j = 0; j < n; ++j) {
          size_t o = ((size_t)comp * L + l) * n + j;
          uint64_t acc = comp == 0 ? agg[(size_t)u * 2 * poly + o] % P->moduli[l] : 0;
          for (uint32_t k = 0; k < n_shares; ++k)
            acc = addm(acc, shares[(((size_t)i * n_shares + k) * n_cts + c) * 2 * poly + o], P->moduli[l]);
          out[(size_t)u * 2 * poly + o] = acc;
        }
  }
}

/* BFV.Decrypt of ct [n][n_cts][2][L][N] with explicit small secrets [n][N] -> plain [n][n_cts][N]. */
void orc_decrypt_batch(const orc_params* P, const uint64_t* ct, const int32_t* secrets, uint32_t n_users,
                       uint32_t n_cts, uint32_t* plain) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_users * n_cts; ++u) {
    uint32_t i = (uint32_t)(u / n_cts);
    orc_decrypt_single(P, ct + (size_t)u * 2 * poly, secrets + (size_t)i * n, plain + (size_t)u * n, NULL);
  }
}

/* ------------------------------------------------------------------ */
/* MBFV.Bootstrap (Sec. 4.2 item 4, Eq. 4)                             */
/* ------------------------------------------------------------------ */

/* The common random polynomial alpha for (recipient, ct_index): uniform on R_q, limb by limb.
 * Counter: (j, ct_index, limb | recipient << 16, tag | attempt << 8). */
void orc_boot_alpha(const orc_params* P, uint32_t recipient, uint32_t ct_index, uint64_t* alpha) {
  uint32_t n = 1u << P->log2_n;
  for (uint32_t l = 0; l < P->num_limbs; ++l) {
    uint64_t p = P->moduli[l];
    uint32_t bits = bit_length(p);
    uint64_t mask = (((uint64_t)1 << bits) - 1);
    for (uint32_t j = 0; j < n; ++j) {
      uint32_t w[4];
      uint64_t val = 0;
      int done = 0;
      for (uint32_t attempt = 0; attempt < 255 && !done; ++attempt) {
        draw(P, TAG_BOOT_ALPHA, attempt, j, ct_index, l, recipient, w);
        uint64_t r = (((uint64_t)w[0] << 32) | w[1]) & mask;
        if (r < p) {
          val = r;
          done = 1;
        }
      }
      if (!done) {
        draw(P, TAG_BOOT_ALPHA, 255, j, ct_index, l, recipient, w);
        val = (((uint64_t)w[0] << 32) | w[1]) % p;
      }
      alpha[(size_t)l * n + j] = val;
    }
  }
}

/* M_k uniform over R_t: rejection on bitlen(t)-bit draws, stream (party, recipient, ct_index). */
void orc_boot_mask(const orc_params* P, uint32_t party, uint32_t recipient, uint32_t ct_index,
                   uint32_t* mask_out) {
  uint32_t n = 1u << P->log2_n;
  uint64_t t = P->plain_modulus;
  uint64_t m = (((uint64_t)1 << bit_length(t)) - 1);
  for (uint32_t j = 0; j < n; ++j) {
    uint32_t w[4];
    uint64_t val = 0;
    int done = 0;
    for (uint32_t attempt = 0; attempt < 255 && !done; ++attempt) {
      draw(P, TAG_BOOT_MASK, attempt, j, ct_index, party, recipient, w);
      uint64_t r = (((uint64_t)w[0] << 32) | w[1]) & m;
      if (r < t) {
        val = r;
        done = 1;
      }
    }
    if (!done) {
      draw(P, TAG_BOOT_MASK, 255, j, ct_index, party, recipient, w);
      val = (((uint64_t)w[0] << 32) | w[1]) % t;
    }
    mask_out[j] = (uint32_t)val;
  }
}

/*
 * Bootstrap share of party k (Eq. 4):
 *   (eta_0, eta_1) = (s_k c_1 - Lambda M_k + e_{0,k},  -s_k alpha + Lambda M_k + e_{1,k}).
 * c1, alpha are [L][N]; eta is [2][L][N].
 */
void orc_boot_share(const orc_params* P, uint32_t party, uint32_t recipient, uint32_t ct_index,
                    const uint64_t* c1, const uint64_t* alpha, uint64_t* eta) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int8_t* s = (int8_t*)malloc(n);
  int8_t* e0 = (int8_t*)malloc(n);
  int8_t* e1 = (int8_t*)malloc(n);
  uint32_t* mk = (uint32_t*)malloc(sizeof(uint32_t) * n);
  uint64_t* sl = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t* a = (uint64_t*)malloc(sizeof(uint64_t) * n);
  uint64_t delta[ORC_MAX_LIMBS];
  orc_delta(P, delta);
  orc_secret_share(P, party, s);
  orc_boot_mask(P, party, recipient, ct_index, mk);
  orc_sample_gauss(P, TAG_BOOT_E0, ct_index, party, recipient, e0);
  orc_sample_gauss(P, TAG_BOOT_E1, ct_index, party, recipient, e1);
  for (uint32_t l = 0; l < L; ++l) {
    uint64_t p = P->moduli[l];
    small_to_limb(s, sl, n, p);
    orc_ring_mul(sl, c1 + (size_t)l * n, a, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j) {
      uint64_t dm = mulm(delta[l], mk[j] % p, p);
      eta[(size_t)l * n + j] = addm(subm(a[j], dm, p), lift(e0[j], p), p);
    }
    orc_ring_mul(sl, alpha + (size_t)l * n, a, P->log2_n, p);
    for (uint32_t j = 0; j < n; ++j) {
      uint64_t dm = mulm(delta[l], mk[j] % p, p);
      eta[poly + (size_t)l * n + j] = addm(addm(subm(0, a[j], p), dm, p), lift(e1[j], p), p);
    }
  }
  free(s);
  free(e0);
  free(e1);
  free(mk);
  free(sl);
  free(a);
}

/* agg [n_rec][n_cts][2][L][N] -> shares [n_rec][n_parties][n_cts][2][L][N]. */
void orc_boot_share_batch(const orc_params* P, const uint64_t* agg, const uint32_t* recipients,
                          uint32_t n_rec, const uint32_t* parties, uint32_t n_parties,
                          uint32_t ct_first, uint32_t n_cts, uint64_t* shares) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int64_t total = (int64_t)n_rec * n_parties * n_cts;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < total; ++u) {
    uint32_t c = (uint32_t)(u % n_cts);
    uint32_t k = (uint32_t)((u / n_cts) % n_parties);
    uint32_t i = (uint32_t)(u / ((int64_t)n_cts * n_parties));
    uint64_t* alpha = (uint64_t*)malloc(sizeof(uint64_t) * poly);
    orc_boot_alpha(P, recipients[i], ct_first + c, alpha);
    const uint64_t* c1 = agg + (((size_t)i * n_cts + c) * 2 + 1) * poly;
    orc_boot_share(P, parties[k], recipients[i], ct_first + c, c1, alpha, shares + (size_t)u * 2 * poly);
    free(alpha);
  }
}

/*
 * ct' = ( [round(t/q [c_0 + eta_0]_q)]_t Lambda + eta_1,  alpha ),  eta_d = sum_k eta_{d,k}.
 * agg [n_rec][n_cts][2][L][N], shares [n_rec][n_shares][n_cts][2][L][N] -> out [n_rec][n_cts][2][L][N].
 */
void orc_boot_combine_batch(const orc_params* P, const uint64_t* agg, const uint64_t* shares,
                            const uint32_t* recipients, uint32_t n_rec, uint32_t n_shares,
                            uint32_t ct_first, uint32_t n_cts, uint64_t* out) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  uint64_t delta[ORC_MAX_LIMBS];
  orc_delta(P, delta);
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_rec * n_cts; ++u) {
    uint32_t i = (uint32_t)(u / n_cts), c = (uint32_t)(u % n_cts);
    uint64_t* eta0 = (uint64_t*)malloc(sizeof(uint64_t) * poly * n_shares);
    uint32_t* x = (uint32_t*)malloc(sizeof(uint32_t) * n);
    for (uint32_t k = 0; k < n_shares; ++k)
      memcpy(eta0 + (size_t)k * poly, shares + ((((size_t)i * n_shares + k) * n_cts + c) * 2) * poly,
             sizeof(uint64_t) * poly);
    orc_combine(P, agg + (size_t)u * 2 * poly, eta0, n_shares, x);
    uint64_t* o = out + (size_t)u * 2 * poly;
    for (uint32_t l = 0; l < L; ++l) {
      uint64_t p = P->moduli[l];
      for (uint32_t j = 0; j < n; ++j) {
        uint64_t acc = mulm(delta[l], x[j] % p, p);
        for (uint32_t k = 0; k < n_shares; ++k)
          acc = addm(acc, shares[((((size_t)i * n_shares + k) * n_cts + c) * 2 + 1) * poly + (size_t)l * n + j], p);
        o[(size_t)l * n + j] = acc;
      }
    }
    orc_boot_alpha(P, recipients[i], ct_first + c, o + poly);
    free(eta0);
    free(x);
  }
}

/* ------------------------------------------------------------------ */
/* Whole round over a batch, for parity at full configuration sizes    */
/* and for timing.  Units (user, ciphertext) are independent; they are */
/* spread over OpenMP threads when compiled with -fopenmp.             */
/* ------------------------------------------------------------------ */

#ifdef _OPENMP
#include <omp.h>
int orc_threads(void) { return omp_get_max_threads(); }
#else
int orc_threads(void) { return 1; }
#endif

void orc_encode_batch(const orc_params* P, const int32_t* values, uint32_t n_cts, uint32_t* plain) {
  uint32_t n = 1u << P->log2_n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t c = 0; c < (int64_t)n_cts; ++c) orc_encode(P, values + c * n, plain + c * n);
}

void orc_decode_batch(const orc_params* P, const uint32_t* plain, uint32_t n_cts, int32_t* values) {
  uint32_t n = 1u << P->log2_n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t c = 0; c < (int64_t)n_cts; ++c) orc_decode(P, plain + c * n, values + c * n);
}

/* plain [n_parties][n_cts][N] -> ct [n_parties][n_cts][2][L][N]; stream index = ct_first + c. */
void orc_encrypt_batch(const orc_params* P, const uint64_t* pk, const uint32_t* parties,
                       uint32_t n_parties, uint32_t ct_first, uint32_t n_cts,
                       const uint32_t* plain, uint64_t* ct) {
  uint32_t n = 1u << P->log2_n;
  size_t ct_words = (size_t)2 * P->num_limbs * n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_parties * n_cts; ++u) {
    uint32_t k = (uint32_t)(u / n_cts), c = (uint32_t)(u % n_cts);
    orc_encrypt(P, pk, parties[k], ct_first + c, plain + (size_t)u * n, ct + (size_t)u * ct_words);
  }
}

/* ct [n_rows][n_cts][2][L][N], CSR lists -> agg [n_out][n_cts][2][L][N]. */
void orc_aggregate_batch(const orc_params* P, const uint64_t* ct, uint32_t n_rows, uint32_t n_cts,
                         const uint32_t* offsets, const uint32_t* rows, uint32_t n_out,
                         uint64_t* agg) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t ct_words = (size_t)2 * L * n;
  (void)n_rows;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_out * n_cts; ++u) {
    uint32_t i = (uint32_t)(u / n_cts), c = (uint32_t)(u % n_cts);
    uint64_t* out = agg + (size_t)u * ct_words;
    memset(out, 0, sizeof(uint64_t) * ct_words);
    for (uint32_t a = offsets[i]; a < offsets[i + 1]; ++a) {
      const uint64_t* src = ct + ((size_t)rows[a] * n_cts + c) * ct_words;
      for (uint32_t comp = 0; comp < 2; ++comp)
        for (uint32_t l = 0; l < L; ++l)
          for (uint32_t j = 0; j < n; ++j) {
            size_t o = ((size_t)comp * L + l) * n + j;
            out[o] = addm(out[o], src[o], P->moduli[l]);
          }
    }
  }
}

/* agg [n_rec][n_cts][2][L][N] -> shares [n_rec][n_parties][n_cts][L][N]. */
void orc_partial_decrypt_batch(const orc_params* P, const uint64_t* agg, const uint32_t* recipients,
                               uint32_t n_rec, const uint32_t* parties, uint32_t n_parties,
                               uint32_t ct_first, uint32_t n_cts, uint64_t* shares) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
  int64_t total = (int64_t)n_rec * n_parties * n_cts;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < total; ++u) {
    uint32_t c = (uint32_t)(u % n_cts);
    uint32_t k = (uint32_t)((u / n_cts) % n_parties);
    uint32_t i = (uint32_t)(u / ((int64_t)n_cts * n_parties));
    const uint64_t* c1 = agg + (((size_t)i * n_cts + c) * 2 + 1) * poly;
    orc_partial_decrypt(P, parties[k], recipients[i], ct_first + c, c1, shares + (size_t)u * poly);
  }
}

/* agg [n_rec][n_cts][2][L][N], shares [n_rec][n_shares][n_cts][L][N] -> plain [n_rec][n_cts][N]. */
void orc_combine_batch(const orc_params* P, const uint64_t* agg, const uint64_t* shares,
                       uint32_t n_rec, uint32_t n_shares, uint32_t n_cts, uint32_t* plain) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
  size_t poly = (size_t)L * n;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)n_rec * n_cts; ++u) {
    uint32_t i = (uint32_t)(u / n_cts), c = (uint32_t)(u % n_cts);
    /* gather this (recipient, ciphertext)'s shares into [n_shares][L][N] */
    uint64_t* tmp = (uint64_t*)malloc(sizeof(uint64_t) * poly * n_shares);
    for (uint32_t k = 0; k < n_shares; ++k)
      memcpy(tmp + (size_t)k * poly, shares + (((size_t)i * n_shares + k) * n_cts + c) * poly,
             sizeof(uint64_t) * poly);
    orc_combine(P, agg + ((size_t)u * 2) * poly, tmp, n_shares, plain + (size_t)u * n);
    free(tmp);
  }
}

/* Forward / inverse transform of a batch [batch][L][N] at caller-given roots psi[l]. */
void orc_ntt_batch(const orc_params* P, const uint64_t* psi, const uint64_t* in, uint64_t* out,
                   uint32_t batch, int inverse) {
  uint32_t n = 1u << P->log2_n, L = P->num_limbs;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < (int64_t)batch * L; ++u) {
    uint32_t l = (uint32_t)(u % L);
    if (inverse)
      orc_negacyclic_interp(in + (size_t)u * n, out + (size_t)u * n, P->log2_n, psi[l], P->moduli[l]);
    else
      orc_negacyclic_eval(in + (size_t)u * n, out + (size_t)u * n, P->log2_n, psi[l], P->moduli[l]);
  }
}
