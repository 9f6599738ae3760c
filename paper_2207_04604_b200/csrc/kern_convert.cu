// MBFV.Convert to a recipient's own key pair (Sec. 4.2 item 3, Eq. 2-3) and BFV.Decrypt under it.
#include "d2mhe_kernels_common.cuh"

namespace cg = cooperative_groups;

namespace {

// Montgomery form (times N^-1) of the eight transform values x[k]
__device__ __forceinline__ void store_octet_mont(u64* __restrict__ dst, u64 (&x)[8], const LimbTab& lt) {
#pragma unroll
  for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
  store_octet(dst, x);
}

// Own key pair of user i (Algorithm 2, Require): sk_i from R_3 (BFV.SecKeyGen),
// pk_i = (-(sk_i p_{1,i} + e_i), p_{1,i}) with p_{1,i} uniform (BFV.PubKeyGen).  grid = n_users * L.
// NTT(p_{1,i}) is parked in the row that finally receives p_{0,i}.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
    k_user_keygen(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ users) {
  const u32 l = blockIdx.x % v.L, user = users[blockIdx.x / v.L];
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
        [&](int, u32 q, u64(&x)[8]) { store_octet_mont(skm + 8 * (size_t)q, x, lt); });
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
          store_octet(pkc0 + 8 * (size_t)q, x);  // parked, lazily reduced
          store_octet_mont(pkm1 + 8 * (size_t)q, x, lt);
        });
  }
  {
    const Stream se(v.seed, TAG_USER_PK_ERR, 0, user, 0);
    ntt_inverse<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 a[8];
          load_octet_rw(pkc0 + 8 * (size_t)q, a);
          load_octet_rw(skm + 8 * (size_t)q, x);
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
      [&](int, u32 q, u64(&x)[8]) { store_octet_mont(pkm0 + 8 * (size_t)q, x, lt); });
}

// Conversion shares (Eq. 2): (h_0, h_1) = (s_k c_1 + mu_k p_{0,i} + e_{0,k}, mu_k p_{1,i} + e_{1,k}).
// grid = n_rec * n_cts * L in clusters over limbs (mu, e_0, e_1 are sampled once per cluster).
// NTT(c_1) is parked in the h_0 row of the last share, NTT(mu_k) in the h_1 row of its own share.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
    k_convert_share(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ agg,
                    const u32* __restrict__ recipients, const u32* __restrict__ parties, u32 n_parties,
                    u32 ct_first, u32 n_cts, u64* shares) {
  cg::cluster_group cluster = cg::this_cluster();
  const u32 cs = cluster.num_blocks(), rank = cluster.block_rank();
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 irec = unit / n_cts, cl = unit % n_cts, c = ct_first + cl;
  const u32 recipient = recipients[irec];
  const LimbTab& lt = lp.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
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
    if (a >= 0) {
      cluster.sync();  // every CTA is done with the previous share's samples
      const Stream sm_(v.seed, TAG_CONV_MU, c, party, recipient);
      const Stream s0(v.seed, TAG_CONV_E0, c, party, recipient);
      const Stream s1(v.seed, TAG_CONV_E1, c, party, recipient);
      const u32 quarter = v.n >> 2;
      // words 0..N/4-1: mu, N/4..N/2-1: e_0, N/2..3N/4-1: e_1 (four samples per word)
#pragma unroll 1
      for (u32 w = rank + cs * threadIdx.x; w < 3 * quarter; w += cs * blockDim.x) {
        const u32 which = w / quarter, j0 = 4 * (w - which * quarter);
        const Stream& st = which == 0 ? sm_ : which == 1 ? s0 : s1;
        u32 pack = 0;
#pragma unroll
        for (u32 b = 0; b < 4; ++b) pack |= ((u32)gauss_from_r(*gt, st.draw64(j0 + b)) & 0xffu) << (8 * b);
        for (u32 r = 0; r < cs; ++r) cluster.map_shared_rank(reinterpret_cast<u32*>(small), r)[w] = pack;
      }
      cluster.sync();  // all samples of this share have landed everywhere
    }
    u64* h0 = a < 0 ? park : shares + ((((size_t)irec * n_parties + a) * n_cts + cl) * 2) * poly + row;
    u64* h1 = h0 + poly;
    u64* fwd_dst = a < 0 ? park : h1;  // NTT(c_1) -> park, NTT(mu_k) -> the share's own h_1 row
    ntt_forward<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](u32 j) { return a < 0 ? __ldg(c1 + j) : lift_small((int)small[j], lt.p); },
        [&](int, u32 q, u64(&x)[8]) { store_octet(fwd_dst + 8 * (size_t)q, x); });
    if (a < 0) continue;
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
#pragma unroll 1
    for (u32 comp = 0; comp < 2; ++comp) {
      const u64* pkc = comp ? pk1 : pk0;
      u64* out = comp ? h1 : h0;
      const signed char* e = small + (comp + 1) * v.n;
      ntt_inverse<LOGN, G, WIDE>(
          sm, lt, v.logn,
          [&](int, u32 q, u64(&x)[8]) {
            u64 a8[8];
            load_octet_rw(h1 + 8 * (size_t)q, a8);
            load_octet(pkc + 8 * (size_t)q, x);
#pragma unroll
            for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a8[k], x[k], lt.p, lt.pinv);
            if (comp == 0) {
              u64 b8[8];
              load_octet_rw(park + 8 * (size_t)q, a8);
              load_octet(sk + 8 * (size_t)q, b8);
#pragma unroll
              for (int k = 0; k < 8; ++k) x[k] += mont_lazy(a8[k], b8[k], lt.p, lt.pinv);  // below 4p
            }
          },
          [&](u32 j, u64 val) { out[j] = add_small_canon<WIDE>(val, (int)e[j], lt); });
    }
  }
  cluster.sync();
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
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
    k_secret_product(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ ct,
                     const u32* __restrict__ users, u32 n_cts, u64* prod) {
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 user = users[unit / n_cts];
  const LimbTab& lt = lp.limbs[l];
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = ct + ((size_t)unit * 2 + 1) * poly + row;
  const u64* sk = v.usk_mont + (size_t)user * poly + row;
  u64* out = prod + (size_t)unit * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return __ldg(c1 + j); },
      [&](int, u32 q, u64(&x)[8]) { store_octet(out + 8 * (size_t)q, x); });
  ntt_inverse<LOGN, G, WIDE>(
      sm, lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) {
        u64 a8[8];
        load_octet_rw(out + 8 * (size_t)q, a8);
        load_octet(sk + 8 * (size_t)q, x);
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a8[k], x[k], lt.p, lt.pinv);
      },
      [&](u32 j, u64 val) { out[j] = canon4(val, lt); });
}

}  // namespace

namespace d2mhe_launch {

cudaError_t user_keygen(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* users_dev,
                        u32 n_users) {
  D2MHE_DISPATCH(k_user_keygen, v, n_users * v.L, s, v, lp, users_dev);
}

cudaError_t convert_share(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                          const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties,
                          u32 ct_first, u32 n_cts, u64* shares) {
  D2MHE_DISPATCH_EX(k_convert_share, v, n_rec * n_cts * v.L, s, 3 * (size_t)v.n, cluster_size_for(v.L, v.logn), v,
                    lp, agg, recipients_dev, parties_dev, n_parties, ct_first, n_cts, shares);
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

}  // namespace d2mhe_launch
