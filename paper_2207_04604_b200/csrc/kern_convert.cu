// MBFV.Convert to a recipient's own key pair (Sec. 4.2 item 3, Eq. 2-3) and BFV.Decrypt under it.
#include <algorithm>

#define D2MHE_SHIFT_AS_MULTIPLY 1  // as in the decryption-share kernel: measured 0.7-1 % faster here with both
#define D2MHE_LATE_BARRIER 1
#include "d2mhe_kernels_common.cuh"

namespace {

// Montgomery form (times N^-1) of the eight transform values x[k]
__device__ __forceinline__ void store_octet_mont_il(u64* row, u32 q, u32 octets, u64 (&x)[8], const LimbTab& lt) {
#pragma unroll
  for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
  store_octet_il(row, q, octets, x);
}

// Own key pair of user i (Algorithm 2, Require): sk_i from R_3 (BFV.SecKeyGen),
// pk_i = (-(sk_i p_{1,i} + e_i), p_{1,i}) with p_{1,i} uniform (BFV.PubKeyGen).  grid = n_users * L.
// NTT(p_{1,i}) is parked in the row that finally receives p_{0,i}.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_user_keygen(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ users) {
  const u32 l = blockIdx.x % v.L, user = users[blockIdx.x / v.L];
  if (!D2MHE_CHK(v.chk, user, v.K, SITE_PARTY)) return;
  const LimbTab& lt = lp.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  u64* skm = v.usk_mont + (size_t)user * poly + row;
  u64* pkm0 = v.upk_mont + (size_t)user * 2 * poly + row;
  u64* pkm1 = pkm0 + poly;
  u64* pkc0 = v.upk_coef + (size_t)user * 2 * poly + row;
  u64* pkc1 = pkc0 + poly;
  {
    const Stream st(v.seed, TAG_USER_SECRET, 0, user, 0);
    ntt_forward<LOGN, G, WIDE>(
        sm, lt, v.logn, [&](u32 j) { return lift_small(st.ternary(j), lt.p); },
        [&](int, u32 q, u64(&x)[8]) { store_octet_mont_il(skm, q, v.n >> 3, x, lt); });
  }
  {
    const Stream st(v.seed, TAG_USER_P1, l, user, 0);
    ntt_forward<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](u32 j) {
          const u64 r = uniform_mod(st, j, lt.p, lt.mask);
          pkc1[j] = r;
          return r;
        },
        [&](int, u32 q, u64(&x)[8]) {
          store_octet_il(pkc0, q, v.n >> 3, x);  // parked, lazily reduced
          store_octet_mont_il(pkm1, q, v.n >> 3, x, lt);
        });
  }
  {
    const Stream se(v.seed, TAG_USER_PK_ERR, 0, user, 0);
    ntt_inverse<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 a[8];
          load_octet_rw_il(pkc0, q, v.n >> 3, a);
          load_octet_rw_il(skm, q, v.n >> 3, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a[k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          val = add_small_canon(val, gauss_from_r(*gt, se.draw64(j)), lt);
          pkc0[j] = val ? lt.p - val : 0;
        });
  }
  __syncthreads();
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return pkc0[j]; },
      [&](int, u32 q, u64(&x)[8]) { store_octet_mont_il(pkm0, q, v.n >> 3, x, lt); });
}

// mu_k, e_{0,k}, e_{1,k} of a conversion share do not depend on the limb: like the noise of the
// decryption shares they are sampled once per share by a kernel of its own, one byte per
// coefficient, into scratch memory that the caller of the launcher lends ([mu | e_0 | e_1], N bytes
// each, per (recipient, ciphertext) unit and party), so the share kernel needs no clusters.
// grid = ceil(n_units * n_parties * 3 * N / 4 / 256); one thread = four samples = one packed word.
__global__ void __launch_bounds__(256)
    k_sample_convert_noise(DevView v, const u32* __restrict__ recipients, const u32* __restrict__ parties,
                           u32 n_parties, u32 ct_first, u32 n_cts, u32 unit_first, u32 n_units,
                           u32* __restrict__ out) {
  __shared__ GaussTab gt;
  load_gauss(&gt, v.gauss);
  const u32 words = v.n >> 2;
  const size_t total = (size_t)n_units * n_parties * 3 * words;
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;  // the last block is ragged
  const u32 w = (u32)(e % words), which = (u32)((e / words) % 3);
  const size_t share = e / (3 * (size_t)words);
  const u32 a = (u32)(share % n_parties), unit = unit_first + (u32)(share / n_parties);
  const u32 party = parties[a], recipient = recipients[unit / n_cts];
  if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY) || !D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) return;
  const Stream st(v.seed, which == 0 ? TAG_CONV_MU : which == 1 ? TAG_CONV_E0 : TAG_CONV_E1, ct_first + unit % n_cts,
                  party, recipient);
  u32 pack = 0;
#pragma unroll
  for (u32 b = 0; b < 4; ++b) pack |= ((u32)gauss_from_r(gt, st.draw64(4 * w + b)) & 0xffu) << (8 * b);
  out[e] = pack;
}

// Conversion shares (Eq. 2): (h_0, h_1) = (s_k c_1 + mu_k p_{0,i} + e_{0,k}, mu_k p_{1,i} + e_{1,k}).
// grid = n_units * L; units unit_first .. unit_first + n_units - 1 of the (recipient, ciphertext) grid.
// NTT(c_1) is parked in the h_0 row of the last share, NTT(mu_k) in the h_1 row of its own share.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_convert_share(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ agg,
                    const u32* __restrict__ recipients, const u32* __restrict__ parties, u32 n_parties,
                    u32 n_cts, u32 unit_first, const u32* __restrict__ sampled, u64* shares) {
  const u32 l = blockIdx.x % v.L, ulocal = blockIdx.x / v.L, unit = unit_first + ulocal;
  const u32 irec = unit / n_cts, cl = unit % n_cts;
  const u32 recipient = recipients[irec];
  if (!D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) return;
  const LimbTab& lt = lp.limbs[l];
  signed char* small = bytes_smem();  // mu, e_0, e_1: N bytes each
  u64* sm = poly_smem(3 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = agg + ((size_t)unit * 2 + 1) * poly + row;
  const u64* pk0 = v.upk_mont + (size_t)recipient * 2 * poly + row;
  const u64* pk1 = pk0 + poly;
  u64* park = shares + ((((size_t)irec * n_parties + (n_parties - 1)) * n_cts + cl) * 2) * poly + row;
  // Iteration -1 transforms c_1 (parked for all shares); iteration a >= 0 produces share a.
  // One forward and one inverse call site serve all transforms of the kernel.
#pragma unroll 1
  for (int a = -1; a < (int)n_parties; ++a) {
    const u32 party = a < 0 ? 0u : parties[a];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) continue;
    if (a >= 0) {
      __syncthreads();  // every thread is done with the previous share's samples
      const u32* src = sampled + ((size_t)ulocal * n_parties + a) * 3 * (v.n >> 2);
      for (u32 w = threadIdx.x; w < 3 * (v.n >> 2); w += blockDim.x) reinterpret_cast<u32*>(small)[w] = __ldg(src + w);
      // the barrier that opens the forward transform publishes the copy
    }
    u64* h0 = a < 0 ? park : shares + ((((size_t)irec * n_parties + a) * n_cts + cl) * 2) * poly + row;
    u64* h1 = h0 + poly;
    u64* fwd_dst = a < 0 ? park : h1;  // NTT(c_1) -> park, NTT(mu_k) -> the share's own h_1 row
    ntt_forward<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](u32 j) { return a < 0 ? __ldg(c1 + j) : lift_small((int)small[j], lt.p); },
        [&](int, u32 q, u64(&x)[8]) { store_octet_il(fwd_dst, q, v.n >> 3, x); });
    if (a < 0) continue;
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
#pragma unroll 1
    for (u32 comp = 0; comp < 2; ++comp) {
      const u64* pkc = comp ? pk1 : pk0;
      u64* out = comp ? h1 : h0;
      const signed char* e = small + (comp + 1) * v.n;
      ntt_inverse<LOGN, G, WIDE, true>(
          sm, lt, v.logn,
          [&](int, u32 q, u64(&x)[8]) {
            u64 a8[8];
            load_octet_rw_il(h1, q, v.n >> 3, a8);
            load_octet_il(pkc, q, v.n >> 3, x);
#pragma unroll
            for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a8[k], x[k], lt.p, lt.pinv);
            if (comp == 0) {
              u64 b8[8];
              load_octet_rw_il(park, q, v.n >> 3, a8);
              load_octet_il(sk, q, v.n >> 3, b8);
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] += mont_lazy(a8[k], b8[k], lt.p, lt.pinv);  // below 4p
            }
          },
          [&](u32 j, u64 val) { out[j] = add_small_canon<WIDE>(val, (int)e[j], lt); });
    }
  }
}

// ct' = (c_0 + sum_k h_{0,k}, sum_k h_{1,k}).  grid = (n_rec * n_cts, chunks); two residues per thread.
__global__ void __launch_bounds__(256)
    k_convert_combine(DevView v, const u64* __restrict__ agg, const u64* __restrict__ shares,
                      u32 n_shares, u32 n_cts, u64* __restrict__ out) {
  const u32 unit = blockIdx.x, irec = unit / n_cts, cl = unit % n_cts;
  const size_t ct_pairs = (size_t)v.L * v.n;  // pairs of residues in one ciphertext
  const ulonglong2* in0 = reinterpret_cast<const ulonglong2*>(agg) + (size_t)unit * ct_pairs;
  ulonglong2* o = reinterpret_cast<ulonglong2*>(out) + (size_t)unit * ct_pairs;
  for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < ct_pairs;
       e += (size_t)gridDim.y * blockDim.x) {
    const u32 l = (u32)(((e * 2) >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, ct_pairs, SITE_ELEMENT)) continue;
    const u64 p = v.limbs[l].p;
    ulonglong2 acc = (e < ct_pairs / 2) ? __ldg(in0 + e) : make_ulonglong2(0, 0);  // c_0 only
    for (u32 k = 0; k < n_shares; ++k) {
      const ulonglong2 x = __ldg(reinterpret_cast<const ulonglong2*>(shares) +
                                 (((size_t)irec * n_shares + k) * n_cts + cl) * ct_pairs + e);
      acc.x = addmod(acc.x, x.x, p);
      acc.y = addmod(acc.y, x.y, p);
    }
    o[e] = acc;
  }
}

// c_1 sk_i for BFV.Decrypt under the user's own key.  grid = n_users * n_cts * L.
// NTT(c_1) is parked in the output row.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_secret_product(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ ct,
                     const u32* __restrict__ users, u32 n_cts, u64* prod) {
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 user = users[unit / n_cts];
  if (!D2MHE_CHK(v.chk, user, v.K, SITE_PARTY)) return;
  const LimbTab& lt = lp.limbs[l];
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = ct + ((size_t)unit * 2 + 1) * poly + row;
  const u64* sk = v.usk_mont + (size_t)user * poly + row;
  u64* out = prod + (size_t)unit * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return __ldg(c1 + j); },
      [&](int, u32 q, u64(&x)[8]) { store_octet_il(out, q, v.n >> 3, x); });
  ntt_inverse<LOGN, G, WIDE>(
      sm, lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) {
        u64 a8[8];
        load_octet_rw_il(out, q, v.n >> 3, a8);
        load_octet_il(sk, q, v.n >> 3, x);
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a8[k], x[k], lt.p, lt.pinv);
      },
      [&](u32 j, u64 val) { out[j] = canon4(val, lt); });
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

cudaError_t user_keygen(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* users_dev,
                        u32 n_users) {
  D2MHE_DISPATCH(k_user_keygen, v, n_users * v.L, s, v, lp, users_dev);
}

static cudaError_t convert_share_units(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                       const u32* recipients_dev, const u32* parties_dev, u32 n_parties, u32 n_cts,
                                       u32 unit_first, u32 n_units, const u32* sampled, u64* shares) {
  D2MHE_DISPATCH_EX(k_convert_share, v, n_units * v.L, s, 3 * (size_t)v.n, 1, v, lp, agg, recipients_dev, parties_dev,
                    n_parties, n_cts, unit_first, sampled, shares);
}

// scratch: at least n_parties * 3 N bytes; (recipient, ciphertext) units are processed in batches of as
// many as it holds.
cudaError_t convert_share(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                          const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties,
                          u32 ct_first, u32 n_cts, u64* shares, void* scratch, size_t scratch_bytes, u32* launches) {
  const size_t per_unit = (size_t)n_parties * 3 * v.n;
  const u32 n_units = n_rec * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  per_batch = whole_wave_batch(v, per_batch, n_units, v.L);
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    const size_t words = (size_t)nu * per_unit / 4;
    k_sample_convert_noise<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(
        v, recipients_dev, parties_dev, n_parties, ct_first, n_cts, first, nu, reinterpret_cast<u32*>(scratch));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = convert_share_units(v, lp, s, agg, recipients_dev, parties_dev, n_parties, n_cts, first, nu,
                            reinterpret_cast<const u32*>(scratch), shares);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

cudaError_t convert_combine(const DevView& v, cudaStream_t s, const u64* agg, const u64* shares, u32 n_rec,
                            u32 n_shares, u32 n_cts, u64* out) {
  const size_t ct_pairs = (size_t)v.L * v.n;
  u32 by = (u32)((ct_pairs + 255) / 256);
  if (by > 32768) by = 32768;
  dim3 grid(n_rec * n_cts, by);
  k_convert_combine<<<grid, 256, 0, s>>>(v, agg, shares, n_shares, n_cts, out);
  return cudaGetLastError();
}

cudaError_t secret_product(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* ct,
                           const u32* users_dev, u32 n_users, u32 n_cts, u64* prod) {
  D2MHE_DISPATCH(k_secret_product, v, n_users * n_cts * v.L, s, v, lp, ct, users_dev, n_cts, prod);
}

}  // namespace D2MHE_LAUNCH_NS
