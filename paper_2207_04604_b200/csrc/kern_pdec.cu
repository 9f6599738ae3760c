// Decryption shares: h = s_k c_1 + e for every listed share holder.
#include <algorithm>

#ifndef D2MHE_SHIFT_AS_MULTIPLY
#define D2MHE_SHIFT_AS_MULTIPLY 1  // see shoup_approx_sf: measured faster in this kernel only
#endif
#define D2MHE_LATE_BARRIER 1       // see ntt_inverse: 0.3-0.7 % here, slower in the stand-alone inverse transform
#include "d2mhe_kernels_common.cuh"

namespace {

// mont_lazy for p = 2^b - d (b = 32 + shift, d < 2^32): with m = lo(a b) p^-1 mod 2^64 the high half of
// m p = m 2^b - m d is (m >> (64 - b)) - hi64-part of m d - borrow, and the borrow of the low halves is
// known without computing them, because lo(m p) = lo(a b): it is set exactly when lo(a b) > lo(m 2^b).
// One high and one widening multiply instead of the four of a full 64 x 64 high half.  Measured on the
// share kernel: 1.3 % faster at N = 8192, 0.8 % slower at N = 16384 (one 1024-thread block per SM, where
// the extra shifts and the comparison cost more than the multiplies they replace), so N = 16384 keeps
// the general form.
__device__ __forceinline__ u64 mont_lazy_sf(u64 a, u64 b, u64 p, u64 pinv, u32 d, u32 shift) {
  const u64 lo = a * b, hi = __umul64hi(a, b);
  const u64 m = lo * pinv;
  u32 ml, mh;
  split64(m, ml, mh);
  const u64 t1 = madwide(mh, d, (u64)mulhi32(ml, d));  // floor(m d / 2^32)
  const u32 bb = 32u + shift;
  const u64 h2 = (m >> (64u - bb)) - (t1 >> 32) - (u64)(lo > (m << bb));
  return hi - h2 + p;
}

// The noise polynomial e of a share does not depend on the limb.  It is sampled once per share by a
// kernel of its own (Philox + table inversion, one byte per coefficient, into scratch memory that
// the caller of the launcher lends), so the share kernel needs no thread-block clusters: every CTA
// is placed freely and spends its time on the transforms.  (A variant that sampled inside the share
// kernel and spread the samples over a cluster of the limbs' CTAs was 3 % slower at N = 8192 and
// 8 % at N = 16384, where clusters of one-CTA-per-SM blocks also leave SMs idle.)
//
// grid = ceil(n_units * n_parties * N / 4 / (256 * wpt)); one packed word = four samples, wpt words per thread.
// noise[(u * n_parties + a) * N + j], u = unit - unit_first, unit = irec * n_cts + cl.
__global__ void __launch_bounds__(256)
    k_sample_share_noise(DevView v, const u32* __restrict__ recipients, const u32* __restrict__ parties,
                         u32 n_parties, u32 ct_first, u32 n_cts, u32 unit_first, u32 n_units,
                         u32* __restrict__ noise, u32 wpt) {
  __shared__ GaussTab gt;
  load_gauss(&gt, v.gauss);
  const u32 words = v.n >> 2;
  const size_t total = (size_t)n_units * n_parties * words;
#pragma unroll 1
  for (u32 it = 0; it < wpt; ++it) {  // several words per thread: the table load above is paid once
    const size_t e = ((size_t)blockIdx.x * wpt + it) * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const u32 w = (u32)(e % words);
    const size_t share = e / words;
    const u32 a = (u32)(share % n_parties), unit = unit_first + (u32)(share / n_parties);
    const u32 party = parties[a], recipient = recipients[unit / n_cts];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY) || !D2MHE_CHK(v.chk, recipient, v.K, SITE_PARTY)) continue;
    const Stream se(v.seed, TAG_DEC_ERR, ct_first + unit % n_cts, party, recipient);
    u32 pack = 0;
#pragma unroll
    for (u32 b = 0; b < 4; ++b) pack |= ((u32)gauss_from_r(gt, se.draw64(4 * w + b)) & 0xffu) << (8 * b);
    noise[e] = pack;
  }
}

// grid = n_units * L * split; units unit_first .. unit_first + n_units - 1 of the (recipient, ciphertext)
// grid.  split > 1 (chosen by the launcher when the grid would otherwise leave most SMs idle) gives the
// parties of a unit's list to `split` thread blocks, party a to block a mod split; each of them
// transforms c_1 for itself and parks it in the row of the last share that it writes.
// (The split is a template switch: as a run-time argument it cost the common, unsplit case registers.)
template <int LOGN, int G, bool WIDE, bool SPLIT>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_partial_decrypt_pre(DevView v, const __grid_constant__ LimbParams lp, const u64* __restrict__ agg,
                          const u32* __restrict__ parties, u32 n_parties, u32 n_cts, u32 unit_first,
                          const signed char* __restrict__ noise, u64* shares, u32 split_arg) {
  const u32 split = SPLIT ? split_arg : 1u;
  const u32 part = SPLIT ? blockIdx.x % split : 0u, rest = SPLIT ? blockIdx.x / split : blockIdx.x;
  const u32 l = rest % v.L, ulocal = rest / v.L, unit = unit_first + ulocal;
  if (SPLIT && part >= n_parties) return;
  const u32 a_last = SPLIT ? part + split * ((n_parties - 1 - part) / split) : n_parties - 1;  // the last party of this block
  const u32 irec = unit / n_cts, cl = unit % n_cts;
  const LimbTab& lt = lp.limbs[l];
  signed char* staged = bytes_smem();  // two buffers of N bytes: the noise of this share and of the next
  u64* sm = poly_smem(2 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u64* c1 = agg + ((size_t)unit * 2 + 1) * poly + row;
  u64* park = shares + (((size_t)irec * n_parties + a_last) * n_cts + cl) * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return __ldg(c1 + j); },
      [&](int, u32 q, u64(&x)[8]) { store_octet_il(park, q, v.n >> 3, x); });
#pragma unroll 1
  for (u32 a = part; a < n_parties; a += split) {
    const u32 it = SPLIT ? (a - part) / split : a;  // iteration number of this block
    const u32 party = parties[a];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) continue;
    const u64* sk = v.s_mont + ((size_t)party * v.L + l) * v.n;
    // The buffer of iteration it was last read in the final round of iteration it - 2, which every
    // thread left before it passed the barrier that opens the transform of iteration it - 1; the copy
    // is published by the barriers between this share's rounds (see below).
    signed char* e = staged + (it & 1u) * v.n;
    {
      const signed char* src = noise + ((size_t)ulocal * n_parties + a) * v.n;
      if ((v.n & 15u) == 0) {
        // 16 bytes per thread, global -> shared without passing through registers; every thread waits
        // for its own copies at the end of the fetch phase and the barriers between the rounds publish
        // them long before the final round reads them.  (Rows of N < 16 bytes are not 16-byte aligned.)
        for (u32 w = threadIdx.x * 16u; w < v.n; w += blockDim.x * 16u) {
          const u32 dst = (u32)__cvta_generic_to_shared(e + w);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src + w) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      } else {
        for (u32 w = threadIdx.x; w < (v.n >> 2); w += blockDim.x)
          reinterpret_cast<u32*>(e)[w] = __ldg(reinterpret_cast<const u32*>(src) + w);
      }
    }
    u64* out = shares + (((size_t)irec * n_parties + a) * n_cts + cl) * poly + row;
    ntt_inverse<LOGN, G, WIDE, true>(  // the store below folds any value the lazy last round leaves
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 ch[8];
          load_octet_rw_il(park, q, v.n >> 3, ch);  // written by this same thread
          load_octet_il(sk, q, v.n >> 3, x);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            x[k] = (WIDE && LOGN != 14) ? mont_lazy_sf(ch[k], x[k], lt.p, lt.pinv, lt.sf_d, lt.sf_shift)
                                        : mont_lazy(ch[k], x[k], lt.p, lt.pinv);
          asm volatile("cp.async.wait_all;" ::: "memory");  // this thread's part of the noise bytes has landed
        },
        [&](u32 j, u64 val) { out[j] = add_small_canon<WIDE>(val, (int)e[j], lt); });
  }
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

// the noise of the shares of units unit_first .. unit_first + n_units - 1: N bytes per (unit, party)
cudaError_t sample_share_noise(const DevView& v, cudaStream_t s, const u32* recipients_dev, const u32* parties_dev,
                               u32 n_parties, u32 ct_first, u32 n_cts, u32 unit_first, u32 n_units, u32* out) {
  const size_t words = (size_t)n_units * n_parties * v.n / 4;
  // four words per thread once the grid is several waves deep (the table load and its barrier are then paid
  // once per 4096 samples); small calls keep one word per thread: their latency is what counts
  const u32 wpt = words >= (size_t)256 * 4 * 8 * v.sms * 2 ? 4u : 1u;
  k_sample_share_noise<<<(unsigned)((words + 256 * (size_t)wpt - 1) / (256 * (size_t)wpt)), 256, 0, s>>>(
      v, recipients_dev, parties_dev, n_parties, ct_first, n_cts, unit_first, n_units, out, wpt);
  return cudaGetLastError();
}

#undef D2MHE_EXTRA_TARGS
#define D2MHE_EXTRA_TARGS , false
static cudaError_t pdec_units_plain(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                    const u32* parties_dev, u32 n_parties, u32 n_cts, u32 unit_first, u32 n_units,
                                    const signed char* noise, u64* shares) {
  D2MHE_DISPATCH_EX(k_partial_decrypt_pre, v, n_units * v.L, s, 2 * (size_t)v.n, 1, v, lp, agg, parties_dev, n_parties,
                    n_cts, unit_first, noise, shares, 1u);
}
// The split variant serves calls of a few thread blocks, where the latency of one block's transforms is
// what counts: at N = 4096 it runs with one octet per thread and round (512 threads per polynomial
// instead of 128; measured 3 x faster per block there).
#undef D2MHE_EXTRA_TARGS
#define D2MHE_EXTRA_TARGS , true
#undef D2MHE_DISPATCH_G12
#define D2MHE_DISPATCH_G12 1
static cudaError_t pdec_units_split(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                    const u32* parties_dev, u32 n_parties, u32 n_cts, u32 unit_first, u32 n_units,
                                    const signed char* noise, u64* shares, u32 split) {
  D2MHE_DISPATCH_EX(k_partial_decrypt_pre, v, n_units * v.L * split, s, 2 * (size_t)v.n, 1, v, lp, agg, parties_dev,
                    n_parties, n_cts, unit_first, noise, shares, split);
}
#undef D2MHE_EXTRA_TARGS
#define D2MHE_EXTRA_TARGS
#undef D2MHE_DISPATCH_G12
#define D2MHE_DISPATCH_G12 D2MHE_G12

static cudaError_t pdec_pre_units(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                  const u32* parties_dev, u32 n_parties, u32 n_cts, u32 unit_first,
                                  u32 n_units, const signed char* noise, u64* shares) {
  // A small call (fewer thread blocks than the GPU holds at once) spreads each unit's parties over
  // several blocks: the latency of the call is then that of a few transforms, not of the whole list.
  const u32 resident = resident_ctas(v);
  u32 split = 1;
  if (n_units * v.L * 2 <= resident) split = std::min(n_parties, resident / (n_units * v.L));
  if (split > 1) return pdec_units_split(v, lp, s, agg, parties_dev, n_parties, n_cts, unit_first, n_units, noise, shares, split);
  return pdec_units_plain(v, lp, s, agg, parties_dev, n_parties, n_cts, unit_first, n_units, noise, shares);
}

// Shares with the noise sampled ahead into `scratch` (scratch_bytes >= n_parties * N), in batches of
// as many (recipient, ciphertext) units as the scratch holds.  *launches receives the number of
// kernel launches.
cudaError_t partial_decrypt_scratch(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg,
                                    const u32* recipients_dev, u32 n_rec, const u32* parties_dev,
                                    u32 n_parties, u32 ct_first, u32 n_cts, u64* shares, void* scratch,
                                    size_t scratch_bytes, u32* launches) {
  const size_t per_unit = (size_t)n_parties * v.n;
  const u32 n_units = n_rec * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  per_batch = whole_wave_batch(v, per_batch, n_units, v.L);
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    cudaError_t e = sample_share_noise(v, s, recipients_dev, parties_dev, n_parties, ct_first, n_cts, first, nu,
                                       reinterpret_cast<u32*>(scratch));
    if (e != cudaSuccess) return e;
    e = pdec_pre_units(v, lp, s, agg, parties_dev, n_parties, n_cts, first, nu,
                       reinterpret_cast<const signed char*>(scratch), shares);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

}  // namespace D2MHE_LAUNCH_NS
