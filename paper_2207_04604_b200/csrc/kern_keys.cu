// Key material: MBFV.SecKeyGen and MBFV.PubKeyGen (executed once per training).
#include "d2mhe_kernels_common.cuh"

namespace {

// s_k from R_3, kept as NTT(s_k) * N^-1 in Montgomery form.   grid = n_parties * L
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_keygen(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ parties) {
  const u32 l = blockIdx.x % v.L, party = parties[blockIdx.x / v.L];
  if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) return;
  const LimbTab& lt = lp.limbs[l];
  const Stream st(v.seed, TAG_SECRET, 0, party, 0);
  u64* out = v.s_mont + ((size_t)party * v.L + l) * v.n;
  ntt_forward<LOGN, G, WIDE>(
      poly_smem(), lt, v.logn, [&](u32 j) { return lift_small(st.ternary(j), lt.p); },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
        store_octet_il(out, q, v.n >> 3, x);
      });
}

// p_1 uniform; p_{0,k} = -(p_1 s_k + e_k); p_0 = sum_k p_{0,k}.
// grid = L: one CTA per limb walks over the parties.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_collective_pk(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ parties, u32 n_parties,
                    u64* __restrict__ shares_out) {
  const u32 l = blockIdx.x;
  const LimbTab& lt = lp.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  u64* sm = poly_smem();
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  u64* p0c = v.pk_coef + row;
  u64* p1c = v.pk_coef + poly + row;
  u64 p1h[G][8];
  {
    const Stream st(v.seed, TAG_P1, l, 0, 0);
    ntt_forward<LOGN, G, WIDE>(
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
          store_octet_il(v.pk_mont + poly + row, q, v.n >> 3, y);
        });
  }
  for (u32 a = 0; a < n_parties; ++a) {
    const u32 party = parties[a];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) continue;
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
    const Stream se(v.seed, TAG_PK_ERR, 0, party, 0);
    u64* share = shares_out ? shares_out + ((size_t)a * v.L + l) * v.n : nullptr;
    ntt_inverse<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](int g, u32 q, u64(&x)[8]) {
          load_octet_il(sk, q, v.n >> 3, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(p1h[g][k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          val = add_small_canon(val, gauss_from_r(*gt, se.draw64(j)), lt);
          val = val ? lt.p - val : 0;
          if (share) share[j] = val;
          p0c[j] = addmod(p0c[j], val, lt.p);  // the same thread owns j for every party
        });
  }
  __syncthreads();  // p0c complete and visible to the whole CTA
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return p0c[j]; },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], lt.mont_ninv, lt.mont_ninv_sh, lt.p);
        store_octet_il(v.pk_mont + row, q, v.n >> 3, x);
      });
}

// Test hook: a stored key (rows of NTT(s) * N^-1 in Montgomery form, one per limb) brought back to
// the coefficient domain; out[l][j] = the coefficient as -1, 0 or 1, or 127 if the residue of limb l
// is none of these.   grid = L
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_export_secret(DevView v, const __grid_constant__ LimbParams lp, const u64* key, signed char* __restrict__ out) {
  const u32 l = blockIdx.x;
  const LimbTab& lt = lp.limbs[l];
  const u64* row = key + (size_t)l * v.n;
  signed char* o = out + (size_t)l * v.n;
  ntt_inverse<LOGN, G, WIDE>(
      poly_smem(), lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) {
        load_octet_rw_il(row, q, v.n >> 3, x);
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = mont_lazy(x[k], 1, lt.p, lt.pinv);  // leaves Montgomery form; below 2p
      },
      [&](u32 j, u64 val) {
        const u64 c = canon4(val, lt);
        o[j] = c == 0 ? 0 : c == 1 ? 1 : c == lt.p - 1 ? -1 : 127;
      });
}

// Test hook of the checked build: the index test on an index equal to its limit.  Touches no memory
// beyond the check words; compiles to an empty kernel without D2MHE_CHECKED.
__global__ void k_check_selftest(DevView v) { (void)D2MHE_CHK(v.chk, 1, 1, SITE_SELFTEST); }

}  // namespace

namespace D2MHE_LAUNCH_NS {

cudaError_t check_selftest(const DevView& v, cudaStream_t s) {
  k_check_selftest<<<1, 1, 0, s>>>(v);
  return cudaGetLastError();
}

cudaError_t export_secret(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* key, signed char* out) {
  D2MHE_DISPATCH(k_export_secret, v, v.L, s, v, lp, key, out);
}

cudaError_t keygen(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties) {
  D2MHE_DISPATCH(k_keygen, v, n_parties * v.L, s, v, lp, parties_dev);
}

cudaError_t collective_pk(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                          u64* shares_out) {
  D2MHE_DISPATCH(k_collective_pk, v, v.L, s, v, lp, parties_dev, n_parties, shares_out);
}

}  // namespace D2MHE_LAUNCH_NS
