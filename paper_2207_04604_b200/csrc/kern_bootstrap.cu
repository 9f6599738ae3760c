// MBFV.Bootstrap (Sec. 4.2 item 4, Eq. 4): collective noise refresh.
#include <algorithm>

#define D2MHE_SHIFT_AS_MULTIPLY 1  // as in the decryption-share kernel: measured 0.7-1 % faster here with both
#define D2MHE_LATE_BARRIER 1
#include "d2mhe_kernels_common.cuh"

namespace {

// e_{0,k}, e_{1,k} (one byte per coefficient) and the mask M_k (one 32-bit word per coefficient,
// uniform mod t) of a share do not depend on the limb: a kernel of its own samples them once per
// share into scratch memory that the caller of the launcher lends ([e_0 | e_1 | M_k] = 6 N bytes per
// (recipient, ciphertext) unit and party), so the share kernel needs no clusters.
// grid = ceil(n_units * n_parties * (3 N / 2) / 256); one thread = one word.
__global__ void __launch_bounds__(256)
    k_sample_boot_noise(DevView v, const u32* __restrict__ recipients, const u32* __restrict__ parties,
                        u32 n_parties, u32 ct_first, u32 n_cts, u32 unit_first, u32 n_units,
                        u32* __restrict__ out) {
  __shared__ GaussTab gt;
  load_gauss(&gt, v.gauss);
  const u32 quarter = v.n >> 2, words = 2 * quarter + v.n;
  const size_t total = (size_t)n_units * n_parties * words;
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;  // the last block is ragged
  const u32 w = (u32)(e % words);
  const size_t share = e / words;
  const u32 a = (u32)(share % n_parties), unit = unit_first + (u32)(share / n_parties);
  const u32 party = parties[a], recipient = recipients[unit / n_cts], c = ct_first + unit % n_cts;
  if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY) || !D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) return;
  u32 word;
  if (w < 2 * quarter) {
    const Stream st(v.seed, w < quarter ? TAG_BOOT_E0 : TAG_BOOT_E1, c, party, recipient);
    const u32 j0 = 4 * (w < quarter ? w : w - quarter);
    word = 0;
#pragma unroll
    for (u32 b = 0; b < 4; ++b) word |= ((u32)gauss_from_r(gt, st.draw64(j0 + b)) & 0xffu) << (8 * b);
  } else {
    const Stream sk_(v.seed, TAG_BOOT_MASK, c, party, recipient);
    const u64 t = v.round.t;
    u64 tmask = 1;
    while (tmask <= t) tmask <<= 1;
    tmask -= 1;
    word = (u32)uniform_mod(sk_, w - 2 * quarter, t, tmask);
  }
  out[e] = word;
}

// Shares (eta_0, eta_1) = (s_k c_1 - Lambda M_k + e_{0,k}, -s_k alpha + Lambda M_k + e_{1,k}).
// grid = n_units * L; units unit_first .. unit_first + n_units - 1 of the (recipient, ciphertext) grid.
// NTT(c_1) is parked in the eta_0 row and NTT(alpha) in the eta_1 row of the last share.
// Iterations -2 and -1 run the two forward transforms, iteration a >= 0 produces share a, so that
// one forward and one inverse call site serve the whole kernel.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_boot_share(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ agg,
                 const u32* __restrict__ recipients, const u32* __restrict__ parties, u32 n_parties,
                 u32 ct_first, u32 n_cts, u32 unit_first, const u32* __restrict__ sampled, u64* shares) {
  const u32 l = blockIdx.x % v.L, ulocal = blockIdx.x / v.L, unit = unit_first + ulocal;
  const u32 irec = unit / n_cts, cl = unit % n_cts, c = ct_first + cl;
  const u32 recipient = recipients[irec];
  if (!D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) return;
  const LimbTab& lt = lp.limbs[l];
  signed char* small = bytes_smem();                        // e_0, e_1: N bytes each
  u32* mask = reinterpret_cast<u32*>(small + 2 * v.n);      // M_k: N words
  u64* sm = poly_smem(6 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = agg + ((size_t)unit * 2 + 1) * poly + row;
  u64* park = shares + ((((size_t)irec * n_parties + (n_parties - 1)) * n_cts + cl) * 2) * poly + row;
  const Stream sa(v.seed, TAG_BOOT_ALPHA, c, l, recipient);
  const u32 words = 2 * (v.n >> 2) + v.n;
#pragma unroll 1
  for (int a = -2; a < (int)n_parties; ++a) {
    const u32 party = a < 0 ? 0u : parties[a];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) continue;
    if (a >= 0) {
      __syncthreads();  // every thread is done with the previous share's samples
      const u32* src = sampled + ((size_t)ulocal * n_parties + a) * words;
      for (u32 w = threadIdx.x; w < words; w += blockDim.x) reinterpret_cast<u32*>(small)[w] = __ldg(src + w);
      // the barrier that opens the first inverse transform publishes the copy
    }
    u64* h0 = a < 0 ? park : shares + ((((size_t)irec * n_parties + a) * n_cts + cl) * 2) * poly + row;
    u64* h1 = h0 + poly;
    if (a < 0) {
      u64* dst = a == -2 ? park : park + poly;
      ntt_forward<LOGN, G, WIDE>(
          sm, lt, v.logn,
          [&](u32 j) { return a == -2 ? __ldg(c1 + j) : uniform_mod(sa, j, lt.p, lt.mask); },
          [&](int, u32 q, u64(&x)[8]) { store_octet_il(dst, q, v.n >> 3, x); });
      continue;
    }
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
#pragma unroll 1
    for (u32 comp = 0; comp < 2; ++comp) {
      const u64* src = comp ? park + poly : park;
      u64* out = comp ? h1 : h0;
      const signed char* e = small + comp * v.n;
      ntt_inverse<LOGN, G, WIDE>(
          sm, lt, v.logn,
          [&](int, u32 q, u64(&x)[8]) {
            u64 a8[8];
            load_octet_rw_il(src, q, v.n >> 3, a8);
            load_octet_il(sk, q, v.n >> 3, x);
#pragma unroll
            for (int k = 0; k < 8; ++k) x[k] = mont_lazy(a8[k], x[k], lt.p, lt.pinv);
          },
          [&](u32 j, u64 val) {
            const u64 dm = shoup_u32(mask[j], lt.delta, lt.delta_sh, lt.np);  // Lambda M_k, below 2p
            // eta_0 = val - dm + e,  eta_1 = -val + dm + e; both sums below 8p
            const u64 s = (comp ? (2 * lt.twop - val) + dm : val + (lt.twop - dm)) + lt.p + (u64)(long long)e[j];
            out[j] = canon8<WIDE>(s, lt);
          });
    }
  }
}

// ct' = (Lambda x + sum_k eta_{1,k}, alpha) with x the rounded plaintext of c_0 + eta_0.
// grid = (n_rec * n_cts, chunks); one residue per thread and iteration.
__global__ void __launch_bounds__(256)
    k_boot_finish(DevView v, const u32* __restrict__ x, const u64* __restrict__ shares,
                  const u32* __restrict__ recipients, u32 n_shares, u32 ct_first, u32 n_cts,
                  u64* __restrict__ out) {
  const u32 unit = blockIdx.x, irec = unit / n_cts, cl = unit % n_cts;
  const u32 recipient = recipients[irec];
  if (!D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) return;
  const size_t poly = (size_t)v.L * v.n;
  for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < poly; e += (size_t)gridDim.y * blockDim.x) {
    const u32 l = (u32)(e >> v.logn), j = (u32)(e & (v.n - 1));
    const LimbTab* lt = v.limbs + l;
    const u64 p = lt->p;
    u64 acc = csub(shoup_u32(x[(size_t)unit * v.n + j], lt->delta, lt->delta_sh, lt->np), p);
    for (u32 k = 0; k < n_shares; ++k)
      acc = addmod(acc, __ldg(shares + ((((size_t)irec * n_shares + k) * n_cts + cl) * 2 + 1) * poly + e), p);
    out[(size_t)unit * 2 * poly + e] = acc;
    const Stream sa(v.seed, TAG_BOOT_ALPHA, ct_first + cl, l, recipient);
    out[(size_t)unit * 2 * poly + poly + e] = uniform_mod(sa, j, p, lt->mask);
  }
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

static cudaError_t boot_share_units(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                    const u32* recipients_dev, const u32* parties_dev, u32 n_parties, u32 ct_first,
                                    u32 n_cts, u32 unit_first, u32 n_units, const u32* sampled, u64* shares) {
  D2MHE_DISPATCH_EX(k_boot_share, v, n_units * v.L, s, 6 * (size_t)v.n, 1, v, lp, agg, recipients_dev, parties_dev,
                    n_parties, ct_first, n_cts, unit_first, sampled, shares);
}

// scratch: at least n_parties * 6 N bytes; (recipient, ciphertext) units are processed in batches of as
// many as it holds.
cudaError_t boot_share(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                       const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties,
                       u32 ct_first, u32 n_cts, u64* shares, void* scratch, size_t scratch_bytes, u32* launches) {
  const size_t per_unit = (size_t)n_parties * 6 * v.n;
  const u32 n_units = n_rec * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  per_batch = whole_wave_batch(v, per_batch, n_units, v.L);
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    const size_t words = (size_t)nu * per_unit / 4;
    k_sample_boot_noise<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(
        v, recipients_dev, parties_dev, n_parties, ct_first, n_cts, first, nu, reinterpret_cast<u32*>(scratch));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = boot_share_units(v, lp, s, agg, recipients_dev, parties_dev, n_parties, ct_first, n_cts, first, nu,
                         reinterpret_cast<const u32*>(scratch), shares);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

cudaError_t boot_finish(const DevView& v, cudaStream_t s, const u32* x, const u64* shares,
                        const u32* recipients_dev, u32 n_rec, u32 n_shares, u32 ct_first, u32 n_cts, u64* out) {
  const size_t poly = (size_t)v.L * v.n;
  u32 by = (u32)((poly + 255) / 256);
  if (by > 32768) by = 32768;
  dim3 grid(n_rec * n_cts, by);
  k_boot_finish<<<grid, 256, 0, s>>>(v, x, shares, recipients_dev, n_shares, ct_first, n_cts, out);
  return cudaGetLastError();
}

}  // namespace D2MHE_LAUNCH_NS
