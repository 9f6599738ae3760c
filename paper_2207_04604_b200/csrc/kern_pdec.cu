// Decryption shares: h = s_k c_1 + e for every listed share holder.
#include "d2mhe_kernels_common.cuh"

namespace cg = cooperative_groups;

namespace {

// grid = n_rec * n_cts * L, launched in thread-block clusters of cs CTAs = cs limbs of the same
// (recipient, ciphertext).  The noise polynomial e of a share is the same for every limb, so
// each CTA of the cluster samples 1/cs of its coefficients (Philox + table inversion) and
// pushes them, four to a word, into the shared memory of all cs CTAs (distributed shared
// memory); two noise buffers alternate so that one cluster barrier per share suffices, and
// that barrier is split: arrive after the push, wait just before the last inverse round.
// NTT(c_1) is computed once per CTA and parked in the output row of the LAST share
// (L2-resident, re-read for every share, overwritten by that share at the very end), so no
// registers are held across the party loop.  Each share costs one pointwise product, one
// inverse transform and one store.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
    k_partial_decrypt(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ agg, const u32* __restrict__ recipients,
                      const u32* __restrict__ parties, u32 n_parties, u32 ct_first, u32 n_cts,
                      u64* shares) {
  cg::cluster_group cluster = cg::this_cluster();
  const u32 cs = cluster.num_blocks(), rank = cluster.block_rank();
  const u32 l = blockIdx.x % v.L, unit = blockIdx.x / v.L;
  const u32 irec = unit / n_cts, cl = unit % n_cts, c = ct_first + cl;
  const u32 recipient = recipients[irec];
  const LimbTab& lt = lp.limbs[l];
  GaussTab* gt = gauss_smem();
  load_gauss(gt, v.gauss);
  signed char* noise = bytes_smem();  // two buffers of N bytes
  u64* sm = poly_smem(2 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = agg + ((size_t)unit * 2 + 1) * poly + row;
  u64* park = shares + (((size_t)irec * n_parties + (n_parties - 1)) * n_cts + cl) * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return __ldg(c1 + j); },
      [&](int, u32 q, u64(&x)[8]) { store_octet(park + 8 * (size_t)q, x); });
#pragma unroll 1
  for (u32 a = 0; a < n_parties; ++a) {
    const u32 party = parties[a];
    signed char* buf = noise + (a & 1u) * v.n;
    {
      const Stream se(v.seed, TAG_DEC_ERR, c, party, recipient);
      for (u32 w = rank + cs * threadIdx.x; w < (v.n >> 2); w += cs * blockDim.x) {
        u32 pack = 0;
#pragma unroll
        for (u32 b = 0; b < 4; ++b)
          pack |= ((u32)gauss_from_r(*gt, se.draw64(4 * w + b)) & 0xffu) << (8 * b);
        for (u32 r = 0; r < cs; ++r) cluster.map_shared_rank(reinterpret_cast<u32*>(buf), r)[w] = pack;
      }
    }
    cluster.barrier_arrive();  // waited for just before the last round, the only reader of the noise
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
    u64* out = shares + (((size_t)irec * n_parties + a) * n_cts + cl) * poly + row;
    ntt_inverse<LOGN, G, WIDE>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 ch[8];
          load_octet_rw(park + 8 * (size_t)q, ch);  // written by this same thread
          load_octet(sk + 8 * (size_t)q, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(ch[k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) { out[j] = add_small_canon<WIDE>(val, (int)buf[j], lt); }, 0, 0,
        [&]() { cluster.barrier_wait(); });  // every CTA's part of e has landed in every CTA's buffer
  }
  cluster.sync();  // no CTA leaves while a peer may still write into its buffers
}

}  // namespace

namespace d2mhe_launch {

cudaError_t partial_decrypt(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                            const u32* recipients_dev, u32 n_rec, const u32* parties_dev,
                            u32 n_parties, u32 ct_first, u32 n_cts, u64* shares) {
  D2MHE_DISPATCH_EX(k_partial_decrypt, v, n_rec * n_cts * v.L, s, 2 * (size_t)v.n,
                    cluster_size_for(v.L, v.logn), v, lp, agg, recipients_dev, parties_dev, n_parties, ct_first,
                    n_cts, shares);
}

}  // namespace d2mhe_launch
