// CUDA kernels of the D2-MHE hot path (sm_100a) and their launchers.
//
// Work decomposition: one CTA owns one residue polynomial (one RNS limb of one ring
// element) in shared memory and runs the register/shared-memory NTT engine on it; the
// samplers, the pointwise products and the additive terms are fused into the first and
// last rounds of the transforms, so a protocol message is written to HBM exactly once
// and intermediate polynomials never leave the SM.
#include "d2mhe_internal.h"

namespace {

// Shared-memory layout: [GaussTab][polynomial].
__device__ __forceinline__ void load_gauss(GaussTab* dst, const GaussTab* __restrict__ src) {
  const u32* s = reinterpret_cast<const u32*>(src);
  u32* d = reinterpret_cast<u32*>(dst);
  for (u32 i = threadIdx.x; i < sizeof(GaussTab) / 4; i += blockDim.x) d[i] = s[i];
  __syncthreads();
}

extern __shared__ __align__(16) unsigned char smem_raw[];

__device__ __forceinline__ u64* poly_smem() {
  return reinterpret_cast<u64*>(smem_raw + ((sizeof(GaussTab) + 15) / 16) * 16);
}
__device__ __forceinline__ GaussTab* gauss_smem() { return reinterpret_cast<GaussTab*>(smem_raw); }

__device__ __forceinline__ void store_octet(u64* __restrict__ dst, const u64 (&x)[8]) {
  ulonglong2* d = reinterpret_cast<ulonglong2*>(dst);
#pragma unroll
  for (int k = 0; k < 4; ++k) d[k] = make_ulonglong2(x[2 * k], x[2 * k + 1]);
}
__device__ __forceinline__ void load_octet(const u64* __restrict__ src, u64 (&x)[8]) {
  const ulonglong2* s = reinterpret_cast<const ulonglong2*>(src);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    ulonglong2 v = __ldg(s + k);
    x[2 * k] = v.x;
    x[2 * k + 1] = v.y;
  }
}

// ---------------------------------------------------------------------------
// MBFV.SecKeyGen: s_k from R_3, kept as NTT(s_k) * N^-1 in Montgomery form.
// grid = n_parties * L
// ---------------------------------------------------------------------------
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1) k_keygen(DevView v, const u32* __restrict__ parties) {
  const u32 l = blockIdx.x % v.L, party = parties[blockIdx.x / v.L];
  const LimbTab lt = v.limbs[l];
  const Stream st(v.seed, TAG_SECRET, 0, party, 0);
  u64* out = v.s_mont + ((size_t)party * v.L + l) * v.n;
  ntt_forward<LOGN, G>(
      poly_smem(), lt, v.logn, [&](u32 j) { return lift_small(st.ternary(j), lt.p); },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
        store_octet(out + 8 * (size_t)q, x);
      });
}

// ---------------------------------------------------------------------------
// MBFV.PubKeyGen: p_1 uniform; p_{0,k} = -(p_1 s_k + e_k); p_0 = sum_k p_{0,k}.
// grid = L (one CTA per limb walks over the parties; executed once per training).
// ---------------------------------------------------------------------------
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1)
    k_collective_pk(DevView v, const u32* __restrict__ parties, u32 n_parties,
                    u64* __restrict__ shares_out) {
  const u32 l = blockIdx.x;
  const LimbTab lt = v.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  u64* p0c = v.pk_coef + row;
  u64* p1c = v.pk_coef + poly + row;
  u64 p1h[G][8];
  {
    const Stream st(v.seed, TAG_P1, l, 0, 0);
    ntt_forward<LOGN, G>(
        sm, lt, v.logn,
        [&](u32 j) {
          u64 r = uniform_mod(st, j, lt.p, lt.mask);
          p1c[j] = r;
          p0c[j] = 0;
          return r;
        },
        [&](int g, u32 q, u64(&x)[8]) {
          u64 y[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            p1h[g][k] = x[k];
            y[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
          }
          store_octet(v.pk_mont + poly + row + 8 * (size_t)q, y);
        });
  }
  for (u32 a = 0; a < n_parties; ++a) {
    const u32 party = parties[a];
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
    const Stream se(v.seed, TAG_PK_ERR, 0, party, 0);
    u64* share = shares_out ? shares_out + ((size_t)a * v.L + l) * v.n : nullptr;
    ntt_inverse<LOGN, G>(
        sm, lt, v.logn,
        [&](int g, u32 q, u64(&x)[8]) {
          load_octet(sk + 8 * (size_t)q, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(p1h[g][k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          val = csub(val, lt.p);
          val = addmod(val, lift_small(gauss_from_r(*gt, se.draw64(j)), lt.p), lt.p);
          val = val ? lt.p - val : 0;
          if (share) share[j] = val;
          p0c[j] = addmod(p0c[j], val, lt.p);  // same thread owns j for every party
        });
  }
  __syncthreads();  // p0c complete and visible to the whole CTA
  ntt_forward<LOGN, G>(
      sm, lt, v.logn, [&](u32 j) { return p0c[j]; },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
        store_octet(v.pk_mont + row + 8 * (size_t)q, x);
      });
}

// ---------------------------------------------------------------------------
// BFV.Encrypt: ct = (Lambda m + u p_0 + e_0, u p_1 + e_1).   grid = n_units * L
// ---------------------------------------------------------------------------
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1)
    k_encrypt(DevView v, const u32* __restrict__ parties, u32 ct_first, u32 n_cts,
              const u32* __restrict__ plain, u64* __restrict__ ct) {
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 party = parties[unit / n_cts], c = ct_first + unit % n_cts;
  const LimbTab lt = v.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u32* m = plain + (size_t)unit * v.n;
  u64 uh[G][8];
  {
    const Stream su(v.seed, TAG_ENC_U, c, party, 0);
    ntt_forward<LOGN, G>(
        sm, lt, v.logn, [&](u32 j) { return lift_small(su.ternary(j), lt.p); },
        [&](int g, u32, u64(&x)[8]) {
#pragma unroll
          for (int k = 0; k < 8; ++k) uh[g][k] = x[k];
        });
  }
#pragma unroll 1
  for (u32 comp = 0; comp < 2; ++comp) {
    const u64* pkh = v.pk_mont + comp * poly + row;
    u64* out = ct + ((size_t)unit * 2 + comp) * poly + row;
    const Stream se(v.seed, comp ? TAG_ENC_E1 : TAG_ENC_E0, c, party, 0);
    ntt_inverse<LOGN, G>(
        sm, lt, v.logn,
        [&](int g, u32 q, u64(&x)[8]) {
          load_octet(pkh + 8 * (size_t)q, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(uh[g][k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          val = csub(val, lt.p);
          val = addmod(val, lift_small(gauss_from_r(*gt, se.draw64(j)), lt.p), lt.p);
          if (comp == 0)
            val = addmod(val, shoup_full((u64)m[j], lt.delta, lt.delta_sh, lt.p), lt.p);
          out[j] = val;
        });
  }
}

// ---------------------------------------------------------------------------
// Decryption shares: h = s_k c_1 + e for every listed party.   grid = n_rec * n_cts * L
// NTT(c_1) is computed once and kept in registers across the party loop.
// ---------------------------------------------------------------------------
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1)
    k_partial_decrypt(DevView v, const u64* __restrict__ agg, const u32* __restrict__ recipients,
                      const u32* __restrict__ parties, u32 n_parties, u32 ct_first, u32 n_cts,
                      u64* __restrict__ shares) {
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 irec = unit / n_cts, cl = unit % n_cts, c = ct_first + cl;
  const u32 recipient = recipients[irec];
  const LimbTab lt = v.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = agg + ((size_t)unit * 2 + 1) * poly + row;
  u64 ch[G][8];
  ntt_forward<LOGN, G>(
      sm, lt, v.logn, [&](u32 j) { return __ldg(c1 + j); },
      [&](int g, u32, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) ch[g][k] = x[k];
      });
#pragma unroll 1
  for (u32 a = 0; a < n_parties; ++a) {
    const u32 party = parties[a];
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
    u64* out = shares + (((size_t)irec * n_parties + a) * n_cts + cl) * poly + row;
    const Stream se(v.seed, TAG_DEC_ERR, c, party, recipient);
    ntt_inverse<LOGN, G>(
        sm, lt, v.logn,
        [&](int g, u32 q, u64(&x)[8]) {
          load_octet(sk + 8 * (size_t)q, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(ch[g][k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          val = csub(val, lt.p);
          out[j] = addmod(val, lift_small(gauss_from_r(*gt, se.draw64(j)), lt.p), lt.p);
        });
  }
}

// ---------------------------------------------------------------------------
// Stand-alone transforms (in place) for the kernel sweep.   grid = batch * L
// ---------------------------------------------------------------------------
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1) k_ntt_fwd(DevView v, u64* __restrict__ polys) {
  const u32 l = blockIdx.x % v.L;
  const LimbTab lt = v.limbs[l];
  u64* row = polys + (size_t)blockIdx.x * v.n;
  ntt_forward<LOGN, G>(
      poly_smem(), lt, v.logn, [&](u32 j) { return row[j]; },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = csub(csub(x[k], lt.twop), lt.p);
        store_octet(row + 8 * (size_t)q, x);
      });
}
template <int LOGN, int G>
__global__ void __launch_bounds__(1024, 1) k_ntt_inv(DevView v, u64* __restrict__ polys) {
  const u32 l = blockIdx.x % v.L;
  const LimbTab lt = v.limbs[l];
  u64* row = polys + (size_t)blockIdx.x * v.n;
  ntt_inverse<LOGN, G>(
      poly_smem(), lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) {
        const ulonglong2* s = reinterpret_cast<const ulonglong2*>(row + 8 * (size_t)q);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          ulonglong2 t = s[k];
          x[2 * k] = t.x;
          x[2 * k + 1] = t.y;
        }
      },
      [&](u32 j, u64 val) { row[j] = shoup_full(val, lt.ninv, lt.ninv_sh, lt.p); });
}

// d = a (.) b + c per residue; two residues per thread (16-byte accesses).
__global__ void __launch_bounds__(256) k_muladd(DevView v, const u64* __restrict__ a,
                                                const u64* __restrict__ b,
                                                const u64* __restrict__ c, u64* __restrict__ d,
                                                size_t n_pairs) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_pairs; e += stride) {
    const u32 l = (u32)(((e * 2) >> v.logn) % v.L);
    const LimbTab* lt = v.limbs + l;
    const u64 p = lt->p, pinv = lt->pinv, r = lt->rmod, rs = lt->rmod_sh;
    const ulonglong2 av = reinterpret_cast<const ulonglong2*>(a)[e];
    const ulonglong2 bv = reinterpret_cast<const ulonglong2*>(b)[e];
    const ulonglong2 cv = reinterpret_cast<const ulonglong2*>(c)[e];
    ulonglong2 o;
    o.x = addmod(shoup_full(mont_lazy(av.x, bv.x, p, pinv), r, rs, p), cv.x, p);
    o.y = addmod(shoup_full(mont_lazy(av.y, bv.y, p, pinv), r, rs, p), cv.y, p);
    reinterpret_cast<ulonglong2*>(d)[e] = o;
  }
}

// ---------------------------------------------------------------------------
// BFV.Add over neighbour lists.  grid = (n_out * n_cts, chunks); two residues per thread.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    k_aggregate(DevView v, const u64* __restrict__ ct, u32 n_cts, const u32* __restrict__ offsets,
                const u32* __restrict__ rows, u64* __restrict__ agg) {
  const u32 unit = blockIdx.x, i = unit / n_cts, c = unit % n_cts;
  const size_t ct_pairs = (size_t)v.L * v.n;  // 2*L*N residues = L*N pairs
  const u32 beg = offsets[i], end = offsets[i + 1];
  ulonglong2* out = reinterpret_cast<ulonglong2*>(agg) + (size_t)unit * ct_pairs;
  for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < ct_pairs;
       e += (size_t)gridDim.y * blockDim.x) {
    const u32 l = (u32)(((e * 2) >> v.logn) % v.L);
    const u64 p = v.limbs[l].p;
    ulonglong2 acc = make_ulonglong2(0, 0);
    for (u32 a = beg; a < end; ++a) {
      const ulonglong2 x =
          __ldg(reinterpret_cast<const ulonglong2*>(ct) + ((size_t)rows[a] * n_cts + c) * ct_pairs + e);
      acc.x = addmod(acc.x, x.x, p);
      acc.y = addmod(acc.y, x.y, p);
    }
    out[e] = acc;
  }
}

// ---------------------------------------------------------------------------
// Combine + exact scale-and-round.  One thread per coefficient.
//   v_l = c_0 + sum_k h_k mod q_l;  w'_l = t v_l + (q-1)/2 mod q_l;
//   mixed-radix digits d_i of w' in [0,q);  w' mod t = sum d_i prod_{j<i} q_j mod t;
//   x = ((q-1)/2 - w') q^-1 mod t  =  round(t v / q) mod t.
// grid = (n_rec * n_cts, N / 256)
// ---------------------------------------------------------------------------
template <int LMAX>
__global__ void __launch_bounds__(256)
    k_combine(DevView v, const u64* __restrict__ agg, const u64* __restrict__ shares, u32 n_shares,
              u32 n_cts, u32* __restrict__ plain) {
  const u32 unit = blockIdx.x, irec = unit / n_cts, cl = unit % n_cts;
  const u32 j = blockIdx.y * blockDim.x + threadIdx.x;
  if (j >= v.n) return;
  const u32 L = v.L;
  const size_t poly = (size_t)L * v.n;
  const u64* c0 = agg + (size_t)unit * 2 * poly;
  u64 d[LMAX];
#pragma unroll
  for (int l = 0; l < LMAX; ++l) {
    if (l < (int)L) {
      const LimbTab* lt = v.limbs + l;
      const u64 p = lt->p;
      u64 acc = __ldg(c0 + (size_t)l * v.n + j);
      for (u32 k = 0; k < n_shares; ++k)
        acc = addmod(acc, __ldg(shares + (((size_t)irec * n_shares + k) * n_cts + cl) * poly +
                                (size_t)l * v.n + j), p);
      d[l] = addmod(shoup_full(acc, lt->tmod, lt->tmod_sh, p), lt->half, p);
    }
  }
  // mixed-radix (Garner) digits in place: d_i <- ((w'_i - d_0) q_0^-1 - d_1) q_1^-1 ... mod q_i
#pragma unroll
  for (int i = 1; i < LMAX; ++i) {
    if (i < (int)L) {
      const LimbTab* lt = v.limbs + i;
      const u64 p = lt->p, cq = lt->cq;
      u64 tmp = d[i];
#pragma unroll
      for (int jj = 0; jj < i; ++jj) {
        const ulonglong2 gi = __ldg(v.round.ginv + i * L + jj);
        tmp = shoup_full(tmp + cq - d[jj], gi.x, gi.y, p);
      }
      d[i] = tmp;
    }
  }
  const u64 t = v.round.t, tsh = v.round.t_sh;
  u64 acc = 0;
#pragma unroll
  for (int i = 0; i < LMAX; ++i) {
    if (i < (int)L) {
      const u64 di = shoup_full(d[i], 1, tsh, t);  // d_i mod t
      acc = shoup_full(acc + di * v.round.prefix_mod_t[i], 1, tsh, t);
    }
  }
  const u64 diff = v.round.half_mod_t + t - acc;  // in (0, 2t)
  plain[(size_t)unit * v.n + j] = (u32)shoup_full(diff * v.round.qinv_mod_t, 1, tsh, t);
}

// ---------------------------------------------------------------------------
// Packing: negacyclic transforms mod t in shared memory (32-bit arithmetic).
// Slot j sits at transform position brv(j).  grid = n_cts
// ---------------------------------------------------------------------------
__device__ __forceinline__ u32 shoup32_lazy(u32 x, uint2 w, u32 t) {
  return x * w.x - __umulhi(x, w.y) * t;
}
__device__ __forceinline__ u32 csub32(u32 x, u32 t) { return x >= t ? x - t : x; }

__global__ void __launch_bounds__(1024)
    k_encode(DevView v, const int32_t* __restrict__ values, u32* __restrict__ plain) {
  u32* sm = reinterpret_cast<u32*>(smem_raw);
  const PlainTab pt = v.plain;
  const u32 n = v.n, logn = v.logn, t = pt.t, twot = pt.twot;
  const int32_t* in = values + (size_t)blockIdx.x * n;
  u32* out = plain + (size_t)blockIdx.x * n;
  bool bad = false;
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) {
    const int32_t val = in[j];
    bad |= (val > (int32_t)pt.half) || (val < -(int32_t)pt.half);
    int32_t r = val % (int32_t)t;
    if (r < 0) r += (int32_t)t;
    sm[__brev(j) >> (32 - logn)] = (u32)r;
  }
  if (bad) atomicOr(v.range_flag, 1u);
  __syncthreads();
  u32 lt = 0;  // log2 of the butterfly span
  for (u32 m = n >> 1; m >= 1; m >>= 1, ++lt) {
    for (u32 b = threadIdx.x; b < (n >> 1); b += blockDim.x) {
      const u32 i = b >> lt, jj = b & ((1u << lt) - 1);
      const u32 idx = (i << (lt + 1)) + jj;
      const u32 X = sm[idx], Y = sm[idx + (1u << lt)];
      const uint2 w = __ldg(pt.IW + m + i);
      sm[idx] = csub32(X + Y, twot);
      sm[idx + (1u << lt)] = shoup32_lazy(X - Y + twot, w, t);
    }
    __syncthreads();
  }
  const uint2 ninv = make_uint2(pt.ninv, pt.ninv_sh);
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) out[j] = csub32(shoup32_lazy(sm[j], ninv, t), t);
}

__global__ void __launch_bounds__(1024)
    k_decode(DevView v, const u32* __restrict__ plain, int32_t* __restrict__ values) {
  u32* sm = reinterpret_cast<u32*>(smem_raw);
  const PlainTab pt = v.plain;
  const u32 n = v.n, logn = v.logn, t = pt.t, twot = pt.twot;
  const u32* in = plain + (size_t)blockIdx.x * n;
  int32_t* out = values + (size_t)blockIdx.x * n;
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) sm[j] = in[j];
  __syncthreads();
  u32 lt = logn - 1;
  for (u32 m = 1; m < n; m <<= 1, --lt) {
    for (u32 b = threadIdx.x; b < (n >> 1); b += blockDim.x) {
      const u32 i = b >> lt, jj = b & ((1u << lt) - 1);
      const u32 idx = (i << (lt + 1)) + jj;
      const u32 X = csub32(sm[idx], twot);
      const uint2 w = __ldg(pt.W + m + i);
      const u32 T = shoup32_lazy(sm[idx + (1u << lt)], w, t);
      sm[idx] = X + T;
      sm[idx + (1u << lt)] = X - T + twot;
    }
    __syncthreads();
  }
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) {
    const u32 y = csub32(csub32(sm[__brev(j) >> (32 - logn)], twot), t);
    out[j] = y > pt.half ? (int32_t)y - (int32_t)t : (int32_t)y;
  }
}

// ---------------------------------------------------------------------------
// Launch plumbing
// ---------------------------------------------------------------------------
size_t ntt_smem_bytes(u32 n) {
  return ((sizeof(GaussTab) + 15) / 16) * 16 + (size_t)n * sizeof(u64);
}
u32 ntt_threads(u32 n, int g) {
  u32 t = n / 8 / g;
  return t < 32 ? 32 : t;
}

template <class K>
cudaError_t set_smem(K kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Picks the instantiation for the ring degree: compile-time sizes for the production
// degrees, the run-time-size build for everything else.
#define D2MHE_DISPATCH(KERNEL, logn, grid, stream, ...)                              \
  do {                                                                                         \
    cudaError_t e_;                                                                            \
    const u32 n_ = 1u << (logn);                                                               \
    const size_t smem_ = poly_bytes(n_);                                           \
    switch (logn) {                                                                            \
      case 12:                                                                                 \
        if ((e_ = set_smem(KERNEL<12, 1>, smem_)) != cudaSuccess) return e_;                   \
        KERNEL<12, 1><<<grid, ntt_threads(n_, 1), smem_, stream>>>(__VA_ARGS__);               \
        break;                                                                                 \
      case 13:                                                                                 \
        if ((e_ = set_smem(KERNEL<13, 1>, smem_)) != cudaSuccess) return e_;                   \
        KERNEL<13, 1><<<grid, ntt_threads(n_, 1), smem_, stream>>>(__VA_ARGS__);               \
        break;                                                                                 \
      case 14:                                                                                 \
        if ((e_ = set_smem(KERNEL<14, 2>, smem_)) != cudaSuccess) return e_;                   \
        KERNEL<14, 2><<<grid, ntt_threads(n_, 2), smem_, stream>>>(__VA_ARGS__);               \
        break;                                                                                 \
      default:                                                                                 \
        if ((logn) > 13) return cudaErrorInvalidValue;                                         \
        if ((e_ = set_smem(KERNEL<0, 1>, smem_)) != cudaSuccess) return e_;                    \
        KERNEL<0, 1><<<grid, ntt_threads(n_, 1), smem_, stream>>>(__VA_ARGS__);                \
        break;                                                                                 \
    }                                                                                          \
    return cudaGetLastError();                                                                 \
  } while (0)

size_t poly_bytes(u32 n) { return ntt_smem_bytes(n); }

}  // namespace

namespace d2mhe_launch {

cudaError_t keygen(const DevView& v, cudaStream_t s, const u32* parties_dev, u32 n_parties) {
  D2MHE_DISPATCH(k_keygen, v.logn, n_parties * v.L, s, v, parties_dev);
}

cudaError_t collective_pk(const DevView& v, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                          u64* shares_out) {
  D2MHE_DISPATCH(k_collective_pk, v.logn, v.L, s, v, parties_dev, n_parties, shares_out);
}

cudaError_t encrypt(const DevView& v, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                    u32 ct_first, u32 n_cts, const u32* plain, u64* ct) {
  D2MHE_DISPATCH(k_encrypt, v.logn, n_parties * n_cts * v.L, s, v, parties_dev, ct_first,
                 n_cts, plain, ct);
}

cudaError_t partial_decrypt(const DevView& v, cudaStream_t s, const u64* agg,
                            const u32* recipients_dev, u32 n_rec, const u32* parties_dev,
                            u32 n_parties, u32 ct_first, u32 n_cts, u64* shares) {
  D2MHE_DISPATCH(k_partial_decrypt, v.logn, n_rec * n_cts * v.L, s, v, agg, recipients_dev,
                 parties_dev, n_parties, ct_first, n_cts, shares);
}

cudaError_t ntt(const DevView& v, cudaStream_t s, u64* polys, u32 batch, bool inverse) {
  if (inverse) {
    D2MHE_DISPATCH(k_ntt_inv, v.logn, batch * v.L, s, v, polys);
  } else {
    D2MHE_DISPATCH(k_ntt_fwd, v.logn, batch * v.L, s, v, polys);
  }
}

cudaError_t muladd(const DevView& v, cudaStream_t s, const u64* a, const u64* b, const u64* c,
                   u64* d, u32 batch) {
  const size_t n_pairs = (size_t)batch * v.L * v.n / 2;
  size_t blocks = (n_pairs + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  k_muladd<<<(u32)blocks, 256, 0, s>>>(v, a, b, c, d, n_pairs);
  return cudaGetLastError();
}

cudaError_t aggregate(const DevView& v, cudaStream_t s, const u64* ct, u32 n_cts,
                      const u32* offsets_dev, const u32* rows_dev, u32 n_out, u64* agg) {
  const size_t ct_pairs = (size_t)v.L * v.n;
  u32 by = (u32)((ct_pairs + 255) / 256);
  if (by > 32768) by = 32768;
  dim3 grid(n_out * n_cts, by);
  k_aggregate<<<grid, 256, 0, s>>>(v, ct, n_cts, offsets_dev, rows_dev, agg);
  return cudaGetLastError();
}

cudaError_t combine(const DevView& v, cudaStream_t s, const u64* agg, const u64* shares, u32 n_rec,
                    u32 n_shares, u32 n_cts, u32* plain) {
  dim3 grid(n_rec * n_cts, (v.n + 255) / 256);
  if (v.L <= 4)
    k_combine<4><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, n_cts, plain);
  else if (v.L <= 8)
    k_combine<8><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, n_cts, plain);
  else
    k_combine<D2MHE_MAX_LIMBS><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, n_cts, plain);
  return cudaGetLastError();
}

cudaError_t encode(const DevView& v, cudaStream_t s, const int32_t* values, u32 n_cts, u32* plain) {
  const size_t smem = (size_t)v.n * 4;
  cudaError_t e = set_smem(k_encode, smem);
  if (e != cudaSuccess) return e;
  u32 threads = v.n / 2 < 1024 ? (v.n / 2 < 32 ? 32 : v.n / 2) : 1024;
  k_encode<<<n_cts, threads, smem, s>>>(v, values, plain);
  return cudaGetLastError();
}

cudaError_t decode(const DevView& v, cudaStream_t s, const u32* plain, u32 n_cts, int32_t* values) {
  const size_t smem = (size_t)v.n * 4;
  cudaError_t e = set_smem(k_decode, smem);
  if (e != cudaSuccess) return e;
  u32 threads = v.n / 2 < 1024 ? (v.n / 2 < 32 ? 32 : v.n / 2) : 1024;
  k_decode<<<n_cts, threads, smem, s>>>(v, plain, values);
  return cudaGetLastError();
}

}  // namespace d2mhe_launch
