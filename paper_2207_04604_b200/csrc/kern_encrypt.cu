// BFV.Encrypt under the collective key: ct = (Lambda m + u p_0 + e_0, u p_1 + e_1).
#include "d2mhe_kernels_common.cuh"

namespace cg = cooperative_groups;

namespace {

// grid = n_units * L, launched in thread-block clusters of cs CTAs = cs limbs of the same
// (party, ciphertext).  u, e_0 and e_1 do not depend on the limb: each CTA samples 1/cs of
// their coefficients and pushes them (four to a word) into the shared memory of all cs CTAs.
// NTT(u) is parked in the output row of c_1 (re-read for both components, overwritten by
// c_1 at the very end), so no registers are held across the two inverse transforms.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
    k_encrypt(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ parties, u32 ct_first, u32 n_cts,
              const u32* __restrict__ plain, u64* ct) {
  cg::cluster_group cluster = cg::this_cluster();
  const u32 cs = cluster.num_blocks(), rank = cluster.block_rank();
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 party = parties[unit / n_cts], c = ct_first + unit % n_cts;
  const LimbTab& lt = lp.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  signed char* small = bytes_smem();  // u, e_0, e_1: N bytes each
  u64* sm = poly_smem(3 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u32* m = plain + (size_t)unit * v.n;
  {
    const Stream su(v.seed, TAG_ENC_U, c, party, 0);
    const Stream s0(v.seed, TAG_ENC_E0, c, party, 0);
    const Stream s1(v.seed, TAG_ENC_E1, c, party, 0);
    for (u32 w = rank + cs * threadIdx.x; w < (v.n >> 2); w += cs * blockDim.x) {
      u32 pu = 0, p0 = 0, p1 = 0;
#pragma unroll
      for (u32 b = 0; b < 4; ++b) {
        pu |= ((u32)su.ternary(4 * w + b) & 0xffu) << (8 * b);
        p0 |= ((u32)gauss_from_r(*gt, s0.draw64(4 * w + b)) & 0xffu) << (8 * b);
        p1 |= ((u32)gauss_from_r(*gt, s1.draw64(4 * w + b)) & 0xffu) << (8 * b);
      }
      for (u32 r = 0; r < cs; ++r) {
        u32* dst = cluster.map_shared_rank(reinterpret_cast<u32*>(small), r);
        dst[w] = pu;
        dst[(v.n >> 2) + w] = p0;
        dst[(v.n >> 1) + w] = p1;
      }
    }
  }
  cluster.sync();  // all samples have landed everywhere; nothing is pushed after this point
  u64* park = ct + ((size_t)unit * 2 + 1) * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return lift_small((int)small[j], lt.p); },
      [&](int, u32 q, u64(&x)[8]) { store_octet(park + 8 * (size_t)q, x); });
#pragma unroll 1
  for (u32 comp = 0; comp < 2; ++comp) {
    const u64* pkh = v.pk_mont + comp * poly + row;
    u64* out = ct + ((size_t)unit * 2 + comp) * poly + row;
    const signed char* e = small + (comp + 1) * v.n;
    ntt_inverse<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 uh[8];
          load_octet_rw(park + 8 * (size_t)q, uh);  // written by this same thread
          load_octet(pkh + 8 * (size_t)q, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(uh[k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          if (comp == 0) {
            // below 4p + (p + 19) + 2p
            u64 t = val + lt.p + (u64)(long long)e[j] + shoup_u32(m[j], lt.delta, lt.delta_sh, lt.np);
            out[j] = canon8<WIDE>(t, lt);  // t below 7p + 19
          } else {
            out[j] = add_small_canon<WIDE>(val, (int)e[j], lt);
          }
        });
  }
}

}  // namespace

namespace d2mhe_launch {

cudaError_t encrypt(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                    u32 ct_first, u32 n_cts, const u32* plain, u64* ct) {
  D2MHE_DISPATCH_EX(k_encrypt, v, n_parties * n_cts * v.L, s, 3 * (size_t)v.n, cluster_size_for(v.L, v.logn), v, lp,
                    parties_dev, ct_first, n_cts, plain, ct);
}

}  // namespace d2mhe_launch
