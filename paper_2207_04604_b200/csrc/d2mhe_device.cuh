// Device-side building blocks: 64-bit modular arithmetic, the Philox4x32-10 sampler,
// and the shared-memory negacyclic NTT engine used by every kernel.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

typedef unsigned long long u64;
typedef unsigned int u32;

// ---------------------------------------------------------------------------
// Per-limb constants (one entry per RNS prime q_l), resident in global memory.
// ---------------------------------------------------------------------------
struct LimbTab {
  u64 p;             // q_l
  u64 twop;          // 2 q_l
  u64 np;            // -q_l mod 2^64
  u64 pinv;          // q_l^-1 mod 2^64 (Montgomery)
  u64 one_sh;        // floor(2^64 / q_l): Shoup companion of 1, reduces any 64-bit value
  u64 ninv, ninv_sh; // N^-1 mod q_l with Shoup companion
  u64 mont_ninv, mont_ninv_sh;  // N^-1 * 2^64 mod q_l: x -> x * N^-1 in Montgomery form
  u64 delta, delta_sh;          // floor(q/t) mod q_l
  u64 tmod, tmod_sh;            // t mod q_l
  u64 half;                     // (q-1)/2 mod q_l
  u64 cq;                       // ceil(2^61 / q_l) * q_l: keeps Garner differences non-negative
  u64 mask;                     // 2^bitlen(q_l) - 1, for the rejection sampler
  u64 rmod, rmod_sh;            // 2^64 mod q_l: leaves Montgomery form; builds Shoup companions
  u32 red_shift, red_mul;       // bitlen(q_l) - 1 and floor(2^(bitlen + 15) / q_l): small-quotient reduction
  u32 sf_d, sf_shift;           // q_l = 2^b - sf_d with b = 32 + sf_shift (set when b >= 32 and sf_d < 2^32)
  const ulonglong2* W;          // [N] forward twiddles psi^brv(i) as {w, floor(w 2^64 / q_l)}
  const ulonglong2* IW;         // [N] their inverses
  // The seven twiddles of octet i in the stride-1 round (last forward, first inverse), regrouped
  // as seven arrays over i so that the threads of a warp load consecutive entries:
  // [0][i] = W[N/8 + i], [1 + b][i] = W[N/4 + 2i + b], [3 + r][i] = W[N/2 + 4i + r].
  const ulonglong2* WL;         // [7][N/8]
  const ulonglong2* IWL;        // [7][N/8]
  u32* chk;                     // device check words (read by the checked kernel build only)
};

// ---------------------------------------------------------------------------
// Checked build.  Compiled with D2MHE_CHECKED every kernel tests the indices it is about to use
// (coefficient and octet numbers, shared-memory byte offsets, twiddle indices, party numbers read
// from index lists) against their limits.  A violation is recorded once in four device words
// {site, index, limit, block} and the access is skipped: no trap, no assert, the context stays
// usable, and the host reads the words at the next synchronisation.  Without the macro the checks
// compile to nothing.
// ---------------------------------------------------------------------------
enum : u32 {
  SITE_LOAD = 1,       // coefficient index handed to a load functor
  SITE_STORE = 2,      // coefficient index handed to a store functor
  SITE_OCTET = 3,      // octet index handed to a fetch / emit functor
  SITE_SMEM = 4,       // byte offset into the shared-memory polynomial
  SITE_TWIDDLE = 5,    // twiddle-table index
  SITE_PARTY = 6,      // party / user / recipient number read from an index list
  SITE_LIMB = 7,       // limb number
  SITE_ELEMENT = 8,    // element index of a streaming kernel
  SITE_STAGED = 9,     // offset into staged bytes in shared memory
  SITE_SELFTEST = 15   // raised on purpose by the self-test hook
};
#ifdef D2MHE_CHECKED
__device__ __forceinline__ bool d2mhe_chk(u32* w, unsigned long long idx, unsigned long long limit, u32 site) {
  if (idx < limit) return true;
  if (w && atomicCAS(w, 0u, site) == 0u) {
    w[1] = (u32)idx;
    w[2] = (u32)limit;
    w[3] = blockIdx.x;
  }
  return false;
}
#define D2MHE_CHK(w, idx, limit, site) d2mhe_chk((w), (unsigned long long)(idx), (unsigned long long)(limit), (site))
#else
#define D2MHE_CHK(w, idx, limit, site) true
#endif

// ---------------------------------------------------------------------------
// Modular arithmetic on [0, 2^64)
// ---------------------------------------------------------------------------

// x*w mod p in [0, 2p) for any 64-bit x, given ws = floor(w 2^64 / p), w < p.
__host__ __device__ __forceinline__ u64 mulhi_u64(u64 a, u64 b) {
#ifdef __CUDA_ARCH__
  return __umul64hi(a, b);
#else
  return (u64)(((unsigned __int128)a * b) >> 64);
#endif
}
__host__ __device__ __forceinline__ u64 shoup_lazy(u64 x, u64 w, u64 ws, u64 p) {
  return x * w - mulhi_u64(x, ws) * p;
}
__host__ __device__ __forceinline__ u64 csub(u64 x, u64 p) { return x >= p ? x - p : x; }
__host__ __device__ __forceinline__ u64 shoup_full(u64 x, u64 w, u64 ws, u64 p) {
  return csub(shoup_lazy(x, w, ws, p), p);
}
// a * b * 2^-64 mod p in (0, 2p); needs b < p (a arbitrary 64-bit), pinv = p^-1 mod 2^64.
__host__ __device__ __forceinline__ u64 mont_lazy(u64 a, u64 b, u64 p, u64 pinv) {
  u64 lo = a * b, hi = mulhi_u64(a, b);
  u64 h2 = mulhi_u64(lo * pinv, p);
  return hi - h2 + p;
}
__host__ __device__ __forceinline__ u64 addmod(u64 a, u64 b, u64 p) { return csub(a + b, p); }
// residue of a small signed integer
__host__ __device__ __forceinline__ u64 lift_small(int v, u64 p) {
  return v < 0 ? p - (u64)(-v) : (u64)v;
}

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) and the samplers
// ---------------------------------------------------------------------------
__host__ __device__ __forceinline__ void philox4x32_10(u32 k0, u32 k1, u32 c0, u32 c1, u32 c2,
                                                        u32 c3, u32& o0, u32& o1, u32& o2,
                                                        u32& o3) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    u64 p0 = (u64)0xD2511F53u * c0;
    u64 p1 = (u64)0xCD9E8D57u * c2;
    u32 n0 = (u32)(p1 >> 32) ^ c1 ^ k0;
    u32 n2 = (u32)(p0 >> 32) ^ c3 ^ k1;
    c1 = (u32)p1;
    c3 = (u32)p0;
    c0 = n0;
    c2 = n2;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  o0 = c0;
  o1 = c1;
  o2 = c2;
  o3 = c3;
}

// Stream tags (fourth counter word, low byte)
enum : u32 {
  TAG_SECRET = 1,
  TAG_PK_ERR = 2,
  TAG_P1 = 3,
  TAG_ENC_U = 4,
  TAG_ENC_E0 = 5,
  TAG_ENC_E1 = 6,
  TAG_DEC_ERR = 7,
  TAG_USER_SECRET = 8,
  TAG_USER_PK_ERR = 9,
  TAG_USER_P1 = 10,
  TAG_CONV_MU = 11,
  TAG_CONV_E0 = 12,
  TAG_CONV_E1 = 13,
  TAG_BOOT_ALPHA = 14,
  TAG_BOOT_MASK = 15,
  TAG_BOOT_E0 = 16,
  TAG_BOOT_E1 = 17
};

// One stream: counter = (j, idx, party | recipient << 16, tag | attempt << 8).
struct Stream {
  u32 k0, k1;  // seed words
  u32 c1, c2, tag;
  __host__ __device__ __forceinline__ Stream(u64 seed, u32 tag_, u32 idx, u32 party, u32 recipient)
      : k0((u32)seed), k1((u32)(seed >> 32)), c1(idx), c2(party | (recipient << 16)), tag(tag_) {}
  __host__ __device__ __forceinline__ u64 draw64(u32 j, u32 attempt = 0) const {
    u32 o0, o1, o2, o3;
    philox4x32_10(k0, k1, j, c1, c2, tag | (attempt << 8), o0, o1, o2, o3);
    return ((u64)o0 << 32) | o1;
  }
  // uniform in {-1, 0, 1}: floor(3 w0 / 2^32) - 1
  __host__ __device__ __forceinline__ int ternary(u32 j) const {
    u32 o0, o1, o2, o3;
    philox4x32_10(k0, k1, j, c1, c2, tag, o0, o1, o2, o3);
    return (int)(((u64)o0 * 3u) >> 32) - 1;
  }
};

// Discrete Gaussian by inversion of the cumulative table: -B + #{k : r >= cdt[k]}.
// lut[r >> 56] = (#thresholds <= bucket start) | (#thresholds inside the bucket) << 8.
#define D2MHE_GAUSS_B 19
#define D2MHE_CDT_LEN 38
struct GaussTab {
  u64 cdt[D2MHE_CDT_LEN];
  unsigned short lut[256];
};
__device__ __forceinline__ int gauss_from_r(const GaussTab& g, u64 r) {
  u32 e = g.lut[r >> 56];
  u32 base = e & 0xffu, inside = e >> 8;
  u32 cnt = base;
  for (u32 i = 0; i < inside; ++i) cnt += (r >= g.cdt[base + i]) ? 1u : 0u;
  return (int)cnt - D2MHE_GAUSS_B;
}
// uniform on Z_p by rejection on bitlen(p)-bit draws (attempt index in the counter)
__host__ __device__ __forceinline__ u64 uniform_mod(const Stream& s, u32 j, u64 p, u64 mask) {
  for (u32 attempt = 0; attempt < 255; ++attempt) {
    u64 r = s.draw64(j, attempt) & mask;
    if (r < p) return r;
  }
  return s.draw64(j, 255) % p;
}

// ---------------------------------------------------------------------------
// Shared-memory NTT engine
//
// One CTA transforms one residue polynomial of N = 2^logn coefficients held in shared
// memory.  Work is organised in radix-8 rounds: in the round that starts at stage s
// (m = 2^s butterfly groups) a thread owns the "octet" of coefficients
//     i * (N/m) + o + k * st,  k = 0..7,  st = N / (8m),
// applies three butterfly stages to it in registers and writes it back; rounds are
// separated by one barrier.  When log2 N is not a multiple of 3 the first forward
// (last inverse) round applies only 1 or 2 stages.  The forward transform is
// Cooley-Tukey with twiddles psi^brv(m+i) (natural order in, bit-reversed out), the
// inverse is Gentleman-Sande; values stay in [0,4p) / [0,2p) between butterflies
// (Harvey's lazy reduction with Shoup multiplication).
//
// The last forward round has st = 1: the thread ends with positions 8q..8q+7 in
// registers, exactly the operands of the first inverse round, so pointwise products
// are fused between the two without touching memory.
// ---------------------------------------------------------------------------

// Shared-memory index swizzle: XOR the low four index bits with bits 4..6 so that the
// 16 threads of a half warp hit 16 distinct 8-byte banks for every stride (.., 64, 8, 1).
__device__ __forceinline__ u32 swz(u32 a) { return a ^ ((a >> 4) & 7u) ^ (((a >> 6) & 1u) << 3); }

// --- multiplication by a constant with an approximate quotient -------------------------
// Returns y*w - q*p (mod 2^64) with q = ah*bh + hi32(ah*bl) + hi32(al*bh) for a = y,
// b = ws = floor(w 2^64 / p): q is the true floor(y ws / 2^64) or up to 2 below it, so the
// result is congruent to y*w and lies in [0, 4p) for ANY 64-bit y.  Five widening / high and
// four 32-bit multiply-adds, written with explicit 32-bit halves so that no 64-bit multiply
// is synthesised (the integer multiplier is the scarce pipe on B200).
__device__ __forceinline__ u64 madwide(u32 a, u32 b, u64 c) {
  u64 r;
  asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(r) : "r"(a), "r"(b), "l"(c));
  return r;
}
__device__ __forceinline__ u32 madlo(u32 a, u32 b, u32 c) {
  u32 r;
  asm("mad.lo.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
__device__ __forceinline__ u64 mulwide(u32 a, u32 b) {
  u64 r;
  asm("mul.wide.u32 %0, %1, %2;" : "=l"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ u32 mulhi32(u32 a, u32 b) {
  u32 r;
  asm("mul.hi.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ u32 madhi32(u32 a, u32 b, u32 c) {  // hi32(a b) + c, wrapping
  u32 r;
  asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
__device__ __forceinline__ void split64(u64 x, u32& lo, u32& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(x));
}
__device__ __forceinline__ u64 join64(u32 lo, u32 hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ u64 shoup_approx(u64 y, u64 w, u64 ws, u64 np) {
  u32 yl, yh, sl, sh, wl, wh, nl, nh;
  split64(y, yl, yh);
  split64(ws, sl, sh);
  split64(w, wl, wh);
  split64(np, nl, nh);
  const u64 q = madwide(yh, sh, (u64)mulhi32(yh, sl) + (u64)mulhi32(yl, sh));
  u32 ql, qh, rl, rh;
  split64(q, ql, qh);
  split64(madwide(ql, nl, mulwide(yl, wl)), rl, rh);
  rh = madlo(yl, wh, rh);
  rh = madlo(yh, wl, rh);
  rh = madlo(ql, nh, rh);
  rh = madlo(qh, nl, rh);
  return join64(rl, rh);
}

// The same for a prime of the form p = 2^b - d, b >= 32, d < 2^32 (every "largest prime below 2^b"
// is): -q p = q d - q 2^b, and q 2^b only reaches the high word as ql << (b - 32), so one of the low
// multiplies becomes a shift.
// D2MHE_SHIFT_AS_MULTIPLY (set by a translation unit before it includes this header): the term
// -(ql << shift) as a fourth low multiply-add instead of a shift and a subtraction, i.e. one
// instruction less per butterfly on one more multiply slot.  Measured at N = 16384: the share kernel
// gains 1.8 %, the encryption kernel nothing, the stand-alone inverse transform loses 3.7 %; so only
// the share kernel sets it.  (Summing the two high halves with mad.hi was slower everywhere.)
#ifndef D2MHE_SHIFT_AS_MULTIPLY
#define D2MHE_SHIFT_AS_MULTIPLY 0
#endif
__device__ __forceinline__ u64 shoup_approx_sf(u64 y, u64 w, u64 ws, u32 d, u32 shift) {
  u32 yl, yh, sl, sh, wl, wh;
  split64(y, yl, yh);
  split64(ws, sl, sh);
  split64(w, wl, wh);
  // the two high halves are summed first: the 64-bit sum is a register pair that the widening
  // multiply-add takes as it is (a zero-extended single word would need a move).  Measured on this
  // GPU, in units of one mad.lo.u32: mul.hi 2.0, mul.wide 2.2, mad.hi 2.2, mad.wide with its 64-bit
  // addend 2.8.  Splitting either widening multiply-add into mul.wide plus a 64-bit addition on the
  // other integer pipe, or taking the high halves from mul.wide, made the butterfly 2-10 % slower.
  const u64 q = madwide(yh, sh, (u64)mulhi32(yh, sl) + (u64)mulhi32(yl, sh));
  u32 ql, qh, rl, rh;
  split64(q, ql, qh);
  split64(madwide(ql, d, mulwide(yl, wl)), rl, rh);
  rh = madlo(yl, wh, rh);
  rh = madlo(yh, wl, rh);
  rh = madlo(qh, d, rh);
#if D2MHE_SHIFT_AS_MULTIPLY
  rh = madlo(ql, 0u - (1u << shift), rh);  // -(ql << shift) as one multiply-add instead of a shift and a subtraction
#else
  rh -= ql << shift;
#endif
  return join64(rl, rh);
}

// Lazy-reduction policy.  WIDE (every prime below 2^56 and of the form above): values may grow across stages, so
// the forward transform needs no conditional subtraction at all and the inverse reduces only
// the one element per octet that accumulates the sums.  Otherwise (primes up to 2^61) values
// are kept below 8p with one conditional subtraction per butterfly.
struct Mod {
  u64 p, np, twop, fourp;
  u32 red_shift, red_mul, sf_d, sf_shift;
  u32* chk;       // check words and limits of the checked build (unused otherwise)
  u32 tw_limit;   // entries of the twiddle tables W / IW
  u32 twl_limit;  // entries of the regrouped tables WL / IWL
  __device__ __forceinline__ explicit Mod(const LimbTab& lt)
      : p(lt.p), np(lt.np), twop(lt.twop), fourp(2 * lt.twop), red_shift(lt.red_shift), red_mul(lt.red_mul),
        sf_d(lt.sf_d), sf_shift(lt.sf_shift), chk(lt.chk), tw_limit(0xffffffffu), twl_limit(0xffffffffu) {}
};
__device__ __forceinline__ ulonglong2 tw_ld(const ulonglong2* __restrict__ T, u32 idx, u32 limit, const Mod& m) {
  if (!D2MHE_CHK(m.chk, idx, limit, SITE_TWIDDLE)) return make_ulonglong2(0, 0);
  return __ldg(T + idx);
}

// x - q p with q = floor(floor(x / 2^(b-1)) * floor(2^(b+15) / p) / 2^16), b = bitlen(p): q is
// floor(x/p) or up to 2 below it, so the result is below 3p.  Needs x < 2^(b+8) (true for every
// lazily grown value here: at most 128p).  One 32-bit, one widening and one low multiply.
__device__ __forceinline__ u64 reduce_small(u64 x, const Mod& m) {
  const u32 q = ((u32)(x >> m.red_shift) * m.red_mul) >> 16;
  u32 nl, nh, rl, rh;
  split64(m.np, nl, nh);
  split64(madwide(q, nl, x), rl, rh);
  return join64(rl, madlo(q, nh, rh));
}

// Arithmetic mode of the engine: 0 = one residue per word, primes up to 2^61; 1 = the same with
// the WIDE policy above (primes below 2^56); 2 = "pair": every 64-bit word carries two 32-bit
// residues of the same prime below 2^30 (two polynomials transformed side by side with the
// same twiddles), each half with Harvey's lazy butterflies in 32-bit arithmetic: one high and
// two low multiplies per butterfly instead of five and four.
enum : int { MODE_STRICT = 0, MODE_WIDE = 1, MODE_PAIR = 2 };

__device__ __forceinline__ u32 csub32(u32 x, u32 p) { return min(x, x - p); }  // x - p wraps above x when x < p
// y*w mod p in [0, 2p) for any 32-bit y, given ws = floor(w 2^32 / p), p < 2^31
__device__ __forceinline__ u32 shoup32(u32 y, u32 w, u32 ws, u32 p) { return y * w - mulhi32(y, ws) * p; }
// The 32-bit companion is the high half of the 64-bit one: floor(floor(w 2^64 / p) / 2^32).
__device__ __forceinline__ void ct_bfly_pair(u64& X, u64& Y, const ulonglong2 w, const Mod& m) {
  const u32 p = (u32)m.p, twop = (u32)m.twop, wl = (u32)w.x, ws = (u32)(w.y >> 32);
  u32 xa, xb, ya, yb;
  split64(X, xa, xb);
  split64(Y, ya, yb);
  xa = csub32(xa, twop);  // inputs below 4p, kept below 4p
  xb = csub32(xb, twop);
  const u32 ta = shoup32(ya, wl, ws, p), tb = shoup32(yb, wl, ws, p);
  X = join64(xa + ta, xb + tb);
  Y = join64(xa - ta + twop, xb - tb + twop);
}
__device__ __forceinline__ void gs_bfly_pair(u64& X, u64& Y, const ulonglong2 w, const Mod& m) {
  const u32 p = (u32)m.p, twop = (u32)m.twop, wl = (u32)w.x, ws = (u32)(w.y >> 32);
  u32 xa, xb, ya, yb;
  split64(X, xa, xb);
  split64(Y, ya, yb);
  X = join64(csub32(xa + ya, twop), csub32(xb + yb, twop));  // inputs below 2p, kept below 2p
  Y = join64(shoup32(xa - ya + twop, wl, ws, p), shoup32(xb - yb + twop, wl, ws, p));
}

// forward (Cooley-Tukey): (X, Y) -> (X + wY, X - wY)
template <int MODE>
__device__ __forceinline__ void ct_bfly(u64& X, u64& Y, const ulonglong2 w, const Mod& m) {
  if (MODE == MODE_PAIR) {
    ct_bfly_pair(X, Y, w, m);
    return;
  }
  constexpr bool WIDE = MODE == MODE_WIDE;
  const u64 x = WIDE ? X : csub(X, m.fourp);
  const u64 t = WIDE ? shoup_approx_sf(Y, w.x, w.y, m.sf_d, m.sf_shift) : shoup_approx(Y, w.x, w.y, m.np);  // [0,4p)
  X = x + t;
  Y = x - t + m.fourp;
}
// inverse (Gentleman-Sande): (X, Y) -> (X + Y, w(X - Y)); c >= bound of Y, a multiple of p
template <int MODE>
__device__ __forceinline__ void gs_bfly(u64& X, u64& Y, const ulonglong2 w, const Mod& m, u64 c) {
  if (MODE == MODE_PAIR) {
    gs_bfly_pair(X, Y, w, m);
    return;
  }
  constexpr bool WIDE = MODE == MODE_WIDE;
  const u64 s = X + Y;
  const u64 d = X - Y + (WIDE ? c : m.fourp);
  X = WIDE ? s : csub(s, m.fourp);
  Y = WIDE ? shoup_approx_sf(d, w.x, w.y, m.sf_d, m.sf_shift) : shoup_approx(d, w.x, w.y, m.np);
}

// three (or fewer) forward stages on an octet; m = groups at the first stage, i = group index
template <int WIDE>
__device__ __forceinline__ void fwd_octet(u64 (&x)[8], const ulonglong2* __restrict__ W, u32 m,
                                          u32 i, int nst, const Mod& md) {
  {
    const ulonglong2 w = tw_ld(W, m + i, md.tw_limit, md);
#pragma unroll
    for (int k = 0; k < 4; ++k) ct_bfly<WIDE>(x[k], x[k + 4], w, md);
  }
  if (nst >= 2) {
    const ulonglong2 w0 = tw_ld(W, 2 * m + 2 * i, md.tw_limit, md), w1 = tw_ld(W, 2 * m + 2 * i + 1, md.tw_limit, md);
    ct_bfly<WIDE>(x[0], x[2], w0, md);
    ct_bfly<WIDE>(x[1], x[3], w0, md);
    ct_bfly<WIDE>(x[4], x[6], w1, md);
    ct_bfly<WIDE>(x[5], x[7], w1, md);
  }
  if (nst >= 3) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const ulonglong2 w = tw_ld(W, 4 * m + 4 * i + r, md.tw_limit, md);
      ct_bfly<WIDE>(x[2 * r], x[2 * r + 1], w, md);
    }
  }
}
// The three stages of the stride-1 round on octet i, twiddles from the regrouped table.
template <int MODE>
__device__ __forceinline__ void fwd_octet_last(u64 (&x)[8], const ulonglong2* __restrict__ WL, u32 oc,
                                               u32 i, const Mod& md) {
  {
    const ulonglong2 w = tw_ld(WL, i, md.twl_limit, md);
#pragma unroll
    for (int k = 0; k < 4; ++k) ct_bfly<MODE>(x[k], x[k + 4], w, md);
  }
  {
    const ulonglong2 w0 = tw_ld(WL, oc + i, md.twl_limit, md), w1 = tw_ld(WL, 2 * oc + i, md.twl_limit, md);
    ct_bfly<MODE>(x[0], x[2], w0, md);
    ct_bfly<MODE>(x[1], x[3], w0, md);
    ct_bfly<MODE>(x[4], x[6], w1, md);
    ct_bfly<MODE>(x[5], x[7], w1, md);
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const ulonglong2 w = tw_ld(WL, (3 + r) * oc + i, md.twl_limit, md);
    ct_bfly<MODE>(x[2 * r], x[2 * r + 1], w, md);
  }
}
template <int MODE>
__device__ __forceinline__ void inv_octet_first(u64 (&x)[8], const ulonglong2* __restrict__ IWL, u32 oc,
                                                u32 i, const Mod& md, bool reduce0 = true) {
  const u64 c16 = md.fourp << 2, c32 = md.fourp << 3, c64 = md.fourp << 4;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const ulonglong2 w = tw_ld(IWL, (3 + r) * oc + i, md.twl_limit, md);
    gs_bfly<MODE>(x[2 * r], x[2 * r + 1], w, md, c16);
  }
  {
    const ulonglong2 w0 = tw_ld(IWL, oc + i, md.twl_limit, md), w1 = tw_ld(IWL, 2 * oc + i, md.twl_limit, md);
    gs_bfly<MODE>(x[0], x[2], w0, md, c32);
    gs_bfly<MODE>(x[1], x[3], w0, md, c32);
    gs_bfly<MODE>(x[4], x[6], w1, md, c32);
    gs_bfly<MODE>(x[5], x[7], w1, md, c32);
  }
  {
    const ulonglong2 w = tw_ld(IWL, i, md.twl_limit, md);
#pragma unroll
    for (int k = 0; k < 4; ++k) gs_bfly<MODE>(x[k], x[k + 4], w, md, c64);
  }
  if (MODE == MODE_WIDE && reduce0) x[0] = reduce_small(x[0], md);
}

// Inverse stages on an octet whose inputs are all below 16p (WIDE) / 4p (otherwise).
// WIDE bounds after the round: x0 < 128p, x1 < 16p, x2, x3 < 8p, x4..x7 < 4p; x0 is brought
// back below 4p here, so every output is again below 16p.
template <int MODE>
__device__ __forceinline__ void inv_octet(u64 (&x)[8], const ulonglong2* __restrict__ IW, u32 m,
                                          u32 i, int nst, const Mod& md, bool reduce0 = true) {
  const u64 c16 = md.fourp << 2, c32 = md.fourp << 3, c64 = md.fourp << 4;
  if (nst >= 3) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const ulonglong2 w = tw_ld(IW, 4 * m + 4 * i + r, md.tw_limit, md);
      gs_bfly<MODE>(x[2 * r], x[2 * r + 1], w, md, c16);
    }
  }
  if (nst >= 2) {
    const ulonglong2 w0 = tw_ld(IW, 2 * m + 2 * i, md.tw_limit, md), w1 = tw_ld(IW, 2 * m + 2 * i + 1, md.tw_limit, md);
    gs_bfly<MODE>(x[0], x[2], w0, md, c32);
    gs_bfly<MODE>(x[1], x[3], w0, md, c32);
    gs_bfly<MODE>(x[4], x[6], w1, md, c32);
    gs_bfly<MODE>(x[5], x[7], w1, md, c32);
  }
  {
    const ulonglong2 w = tw_ld(IW, m + i, md.tw_limit, md);
#pragma unroll
    for (int k = 0; k < 4; ++k) gs_bfly<MODE>(x[k], x[k + 4], w, md, c64);
  }
  if (MODE == MODE_WIDE && reduce0) x[0] = reduce_small(x[0], md);
}

// Brings the outputs of the last inverse round below 4p.  After a full round the bounds are
// those listed at inv_octet; a 2-stage round leaves x1 < 64p, x2, x3 < 8p and a 1-stage round
// x1..x3 < 32p (x0 has already been reduced, x4..x7 are products).
template <int MODE>
__device__ __forceinline__ void finish_octet(u64 (&x)[8], int nst, const Mod& md) {
  if (MODE == MODE_WIDE) {
    if (nst >= 3) {
      x[1] = csub(csub(x[1], md.fourp << 1), md.fourp);
    } else {
      x[1] = reduce_small(x[1], md);
    }
    if (nst >= 2) {
      x[2] = csub(x[2], md.fourp);
      x[3] = csub(x[3], md.fourp);
    } else {
      x[2] = reduce_small(x[2], md);
      x[3] = reduce_small(x[3], md);
    }
  }
}
// canonical representative of a value below 4p
__device__ __forceinline__ u64 canon4(u64 v, const LimbTab& lt) { return csub(csub(v, lt.twop), lt.p); }

// Geometry shared by all kernels: LOGN > 0 fixes the size at compile time (strides, loop
// counts and shared-memory offsets fold to constants); LOGN == 0 takes it from the run-time
// argument.  T = threads per CTA = N / (8 G) (at least one warp).
template <int LOGN, int G>
struct NttGeom {
  u32 logn, n, octets, r0, T;
  __device__ __forceinline__ explicit NttGeom(u32 logn_rt) {
    logn = LOGN ? (u32)LOGN : logn_rt;
    n = 1u << logn;
    octets = n >> 3;
    r0 = logn % 3u;
    T = LOGN ? ((octets / G) < 32u ? 32u : (octets / G)) : blockDim.x;
  }
};

// Thread groups (N = 16384 only: one 1024-thread CTA per SM, where a CTA-wide barrier idles the
// whole SM).  After its first two stages a forward transform is four independent quarter-size
// transforms, and an inverse transform is so until its last two stages.  The threads of group h own
// the octets of the h-th quarter in every round that stays inside the quarters (first stage
// s >= GB), so those rounds are separated by a named barrier of the group only and the groups drift
// apart: one group's shared-memory phase overlaps another's arithmetic.  Rounds that span the
// quarters keep the CTA-wide barrier.  GB = 0 turns this off.
#ifndef D2MHE_LATE_BARRIER
#define D2MHE_LATE_BARRIER 0
#endif
#ifndef D2MHE_GB14
#define D2MHE_GB14 2
#endif
#ifndef D2MHE_GB13
#define D2MHE_GB13 0
#endif
__host__ __device__ constexpr int ntt_group_bits(int logn, int mode) {
  return mode == MODE_PAIR ? 0 : logn == 14 ? D2MHE_GB14 : logn == 13 ? D2MHE_GB13 : 0;
}
template <int GB>
__device__ __forceinline__ u32 group_octet(u32 tid, int g, u32 T, u32 octets) {
  if (GB == 0) return tid + (u32)g * T;
  const u32 Tg = T >> GB;
  return (tid / Tg) * (octets >> GB) + (tid % Tg) + (u32)g * Tg;
}
// inside: this round and the next one both stay inside the groups' parts
template <int GB>
__device__ __forceinline__ void group_barrier(u32 tid, u32 T, bool inside) {
  if (GB == 0 || !inside) {
    __syncthreads();
  } else {
    const u32 Tg = T >> GB;  // a multiple of the warp size
    asm volatile("bar.sync %0, %1;" ::"r"(1u + tid / Tg), "r"(Tg) : "memory");
  }
}

// Byte offsets into the swizzled shared-memory polynomial for the eight elements
// base + (k << sh) of an octet.  The swizzle XORs the low four index bits with bits 4..6;
// for the strides that occur (sh = 0, 3, 6 and >= 7) most of it is per-octet work, so an
// element costs at most one XOR:
//   sh >= 7: swz(base) + k*st            sh == 6: (swz(base) ^ 12*(k&1)) + 64k
//   sh == 3: base - o + 16(k>>1) + ((o ^ 12*bit6(base)) ^ (8(k&1) ^ (k>>1)))
//   sh == 0: swz(base) ^ k
struct OctAddr {
  u32 a, b;
  __device__ __forceinline__ OctAddr(u32 base, u32 sh) {
    if (sh >= 6 || sh == 0) {
      a = swz(base) << 3;
      b = a ^ (12u << 3);
    } else if (sh == 3) {
      const u32 o = base & 7u;
      a = (base - o) << 3;
      b = (o ^ (((base >> 6) & 1u) * 12u)) << 3;
    } else {
      a = base;
      b = 0;
    }
  }
  __device__ __forceinline__ u32 at(int k, u32 sh) const {
    if (sh >= 7) return a + ((u32)k << (sh + 3));
    if (sh == 6) return ((k & 1) ? b : a) + ((u32)k << 9);
    if (sh == 3) return a + 128u * (u32)(k >> 1) + (b ^ ((u32)((8 * (k & 1)) ^ (k >> 1)) << 3));
    if (sh == 0) return a ^ ((u32)k << 3);
    return swz(a + ((u32)k << sh)) << 3;
  }
};
__device__ __forceinline__ u64& sm_at(u64* sm, u32 byte_off) {
  return *reinterpret_cast<u64*>(reinterpret_cast<unsigned char*>(sm) + byte_off);
}
// the same through the checked build's test: byte_off must lie inside the polynomial and be a multiple of 8
__device__ __forceinline__ u64 sm_get(u64* sm, u32 byte_off, u32 bytes, const Mod& m) {
  if (!D2MHE_CHK(m.chk, byte_off | ((byte_off & 7u) ? 0x80000000u : 0u), bytes, SITE_SMEM)) return 0;
  return sm_at(sm, byte_off);
}
__device__ __forceinline__ void sm_put(u64* sm, u32 byte_off, u64 v, u32 bytes, const Mod& m) {
  if (D2MHE_CHK(m.chk, byte_off | ((byte_off & 7u) ? 0x80000000u : 0u), bytes, SITE_SMEM)) sm_at(sm, byte_off) = v;
}

// A transform of size N' = 2^logn can also be block `blk` of a larger transform whose first
// `soff` stages were applied elsewhere (two-pass transforms for N > 16384): the block then
// uses the twiddles of the sub-tree below node (soff, blk), i.e. index (m << soff) + (blk << s) + i.
//
// Forward transform.  load(j) returns coefficient j (any lazily reduced value below 8p);
// emit(g, q, x) receives the octet of positions 8q..8q+7 (lazily reduced values: below 66p when
// WIDE, below 8p otherwise), q = tid + g*T.  The third template argument is the arithmetic mode
// (0 / 1 = not WIDE / WIDE; MODE_PAIR: words are pairs of 32-bit residues below 4p, both ways).
template <int LOGN, int G, int WIDE, class Load, class Emit>
__device__ __forceinline__ void ntt_forward(u64* __restrict__ sm, const LimbTab& lt, u32 logn_rt,
                                            Load load, Emit emit, u32 soff = 0, u32 blk = 0) {
  const NttGeom<LOGN, G> ge(logn_rt);
  const u32 T = ge.T, tid = threadIdx.x;
  constexpr int GB = ntt_group_bits(LOGN, WIDE);
  Mod md(lt);
  md.tw_limit = ge.n << soff;
  md.twl_limit = 7u * ge.octets;
  const u32 smb = ge.n << 3;  // bytes of the shared-memory polynomial
  const ulonglong2* __restrict__ W = lt.W;
  u64 x[8];
  __syncthreads();  // previous users of sm are done
  u32 s = 0;
  bool from_load = true;
  if (ge.r0) {
    const u32 sh = ge.logn - 3;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const u32 q = group_octet<GB>(tid, g, T, ge.octets);
      if (LOGN || q < ge.octets) {
        const OctAddr ad(q, sh);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const u32 j = q + ((u32)k << sh);
          x[k] = D2MHE_CHK(md.chk, j, ge.n, SITE_LOAD) ? load(j) : 0;
        }
        fwd_octet<WIDE>(x, W, 1u << soff, blk, (int)ge.r0, md);
#pragma unroll
        for (int k = 0; k < 8; ++k) sm_put(sm, ad.at(k, sh), x[k], smb, md);
      }
    }
    s = ge.r0;
    from_load = false;
    __syncthreads();
  }
#pragma unroll
  for (; s < ge.logn; s += 3) {
    const u32 sh = ge.logn - s - 3;  // log2 of the stride
    const u32 m = 1u << s;
    const bool last = (s + 3 == ge.logn);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const u32 q = group_octet<GB>(tid, g, T, ge.octets);
      if (LOGN || q < ge.octets) {
        const u32 i = q >> sh, o = q & ((1u << sh) - 1);
        const u32 base = ((i << 3) << sh) + o;
        const OctAddr ad(base, sh);
        if (from_load) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const u32 j = base + ((u32)k << sh);
            x[k] = D2MHE_CHK(md.chk, j, ge.n, SITE_LOAD) ? load(j) : 0;
          }
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = sm_get(sm, ad.at(k, sh), smb, md);
        }
        if (last && soff == 0)  // every thread has seven twiddles of its own here: consecutive entries of the regrouped copy
          fwd_octet_last<WIDE>(x, lt.WL, ge.octets, i, md);
        else
          fwd_octet<WIDE>(x, W, m << soff, (blk << s) + i, 3, md);
        if (last) {
          if (D2MHE_CHK(md.chk, q, ge.octets, SITE_OCTET)) emit(g, q, x);
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) sm_put(sm, ad.at(k, sh), x[k], smb, md);
        }
      }
    }
    from_load = false;
    if (!last) group_barrier<GB>(tid, T, (int)s >= GB);  // the next round starts at stage s + 3
  }
}

// Inverse transform (without the N^-1 scaling: fold it into an operand).
// fetch(g, q, x) fills the octet of positions 8q..8q+7 with values below 4p (below 16p when WIDE);
// store(j, v) receives coefficient j, v in [0,4p).  MODE_PAIR: halves below 2p in and out.
struct NoHook {
  __device__ __forceinline__ void operator()() const {}
};
// before_final() is called by every thread just before the round that calls store().
// LAZY_OUT (WIDE only): the last round skips its reductions and store() receives values below 129p
// (the bounds listed at inv_octet, without bringing x0 back); for a caller whose store() reduces by the
// 2^b - d fold (canon8<true>), which takes any such value in one step.
template <int LOGN, int G, int WIDE, bool LAZY_OUT = false, class Fetch, class Store, class Hook = NoHook>
__device__ __forceinline__ void ntt_inverse(u64* __restrict__ sm, const LimbTab& lt, u32 logn_rt,
                                            Fetch fetch, Store store, u32 soff = 0, u32 blk = 0,
                                            Hook before_final = Hook()) {
  const NttGeom<LOGN, G> ge(logn_rt);
  const u32 T = ge.T, tid = threadIdx.x;
  constexpr int GB = ntt_group_bits(LOGN, WIDE);
  Mod md(lt);
  md.tw_limit = ge.n << soff;
  md.twl_limit = 7u * ge.octets;
  const u32 smb = ge.n << 3;  // bytes of the shared-memory polynomial
  const ulonglong2* __restrict__ IW = lt.IW;
  u64 x[8];
#if !D2MHE_LATE_BARRIER
  __syncthreads();  // previous users of sm are done
#endif
  bool from_fetch = true;
#pragma unroll
  for (int s = (int)ge.logn - 3; s >= (int)ge.r0; s -= 3) {
    const u32 sh = ge.logn - (u32)s - 3;
    const u32 m = 1u << s;
    const bool final_round = (s == 0);
    if (final_round) before_final();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const u32 q = group_octet<GB>(tid, g, T, ge.octets);
      if (LOGN || q < ge.octets) {
        const u32 i = q >> sh, o = q & ((1u << sh) - 1);
        const u32 base = ((i << 3) << sh) + o;
        const OctAddr ad(base, sh);
        if (from_fetch) {
          if (D2MHE_CHK(md.chk, q, ge.octets, SITE_OCTET)) {
            fetch(g, q, x);
          } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) x[k] = 0;
          }
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = sm_get(sm, ad.at(k, sh), smb, md);
        }
        if (from_fetch && soff == 0)
          inv_octet_first<WIDE>(x, lt.IWL, ge.octets, i, md, !(LAZY_OUT && final_round));
        else
          inv_octet<WIDE>(x, IW, m << soff, (blk << s) + i, 3, md, !(LAZY_OUT && final_round));
#if D2MHE_LATE_BARRIER
      }
      // Previous users of sm are done.  The first octet of a transform is fetched and taken through its
      // first round before this barrier, which only the shared-memory stores have to wait for: the skew
      // between the threads of the block is spent on loads and arithmetic instead of idling.
      if (from_fetch && g == 0) __syncthreads();
      if (LOGN || q < ge.octets) {
        const u32 i = q >> sh, o = q & ((1u << sh) - 1);
        const u32 base = ((i << 3) << sh) + o;
        const OctAddr ad(base, sh);
#endif
        if (final_round) {
          if (!LAZY_OUT) finish_octet<WIDE>(x, 3, md);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const u32 j = base + ((u32)k << sh);
            if (D2MHE_CHK(md.chk, j, ge.n, SITE_STORE)) store(j, x[k]);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 8; ++k) sm_put(sm, ad.at(k, sh), x[k], smb, md);
        }
      }
    }
    from_fetch = false;
    // the next round starts at stage s - 3, or is the short round that starts at stage 0
    if (!final_round) group_barrier<GB>(tid, T, s - 3 >= (int)ge.r0 && s - 3 >= GB);
  }
  if (ge.r0) {
    const u32 sh = ge.logn - 3;
    before_final();
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const u32 q = group_octet<GB>(tid, g, T, ge.octets);
      if (LOGN || q < ge.octets) {
        const OctAddr ad(q, sh);
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = sm_get(sm, ad.at(k, sh), smb, md);
        inv_octet<WIDE>(x, IW, 1u << soff, blk, (int)ge.r0, md, !LAZY_OUT);
        if (!LAZY_OUT) finish_octet<WIDE>(x, (int)ge.r0, md);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const u32 j = q + ((u32)k << sh);
          if (D2MHE_CHK(md.chk, j, ge.n, SITE_STORE)) store(j, x[k]);
        }
      }
    }
  }
}
