// The protocol calls on 32-bit words, for parameter sets whose primes are all below 2^30:
// ciphertexts, neighbour sums and decryption shares are uint32 [.., L, N] (half the bytes of the
// 64-bit calls) and every transform runs in the engine's pair mode: one CTA transforms the same
// limb of TWO polynomials side by side (element j of both travels as one 64-bit word), a butterfly
// is two independent 32-bit Harvey butterflies.  Encryption pairs the ciphertexts of two
// (party, ciphertext) units, the share kernel the shares of two (recipient, ciphertext) units under
// the same party's key.  Samples, streams and results are those of the 64-bit calls.
#include <algorithm>

#include "d2mhe_kernels_common.cuh"

namespace {

// Key rows for the 32-bit kernels: every residue k' (transform domain, times N^-1, out of Montgomery
// form, canonical) with its 32-bit Shoup companion floor(k' 2^32 / p) as one 64-bit word {k', companion}.
// src: rows of N residues in Montgomery form, limb of row r = r mod L.   grid-stride over rows * N.
__global__ void __launch_bounds__(256)
    k_make_tab32(DevView v, const u64* __restrict__ src, u64* __restrict__ dst, size_t count) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += stride) {
    const u32 l = (u32)((e >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, count, SITE_ELEMENT) || !D2MHE_CHK(v.chk, l, v.L, SITE_LIMB)) continue;
    const LimbTab* lt = v.limbs + l;
    const u64 k = csub(csub(mont_lazy(src[e], 1, lt->p, lt->pinv), lt->p), lt->p);  // leaves Montgomery form
    dst[e] = join64((u32)k, (u32)((k << 32) / lt->p));
  }
}

// the two units of a CTA: local indices 2 pr and 2 pr + 1 of this launch (the last pair of an odd
// count has one unit: b aliases a and its stores are skipped)
struct UnitPair {
  u32 la, lb;  // local unit indices
  bool has_b;
};
__device__ __forceinline__ UnitPair unit_pair(u32 pr, u32 n_units) {
  UnitPair u;
  u.la = 2 * pr;
  u.has_b = 2 * pr + 1 < n_units;
  u.lb = u.has_b ? u.la + 1 : u.la;
  return u;
}

// Parked 32-bit rows are in interleaved octet order like the key rows: the two 16-byte halves of octet q
// in slots q and octets + q, so that a warp's access covers 512 consecutive bytes.
__device__ __forceinline__ void load_octet32_il(const u32* row, u32 q, u32 octets, u32 (&x)[8]) {  // coherent: this kernel's own data
  const uint4* s = reinterpret_cast<const uint4*>(row) + q;
  const uint4 a = s[0], b = s[octets];
  x[0] = a.x, x[1] = a.y, x[2] = a.z, x[3] = a.w, x[4] = b.x, x[5] = b.y, x[6] = b.z, x[7] = b.w;
}
__device__ __forceinline__ void store_octet32_il(u32* row, u32 q, u32 octets, const u32 (&x)[8]) {
  uint4* d = reinterpret_cast<uint4*>(row) + q;
  d[0] = make_uint4(x[0], x[1], x[2], x[3]);
  d[octets] = make_uint4(x[4], x[5], x[6], x[7]);
}
// halves of the eight pair words -> the two polynomials' parked rows
__device__ __forceinline__ void store_octet_halves(u32* ra, u32* rb, u32 q, u32 octets, bool has_b, const u64 (&x)[8]) {
  u32 lo[8], hi[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) split64(x[k], lo[k], hi[k]);
  store_octet32_il(ra, q, octets, lo);
  if (has_b) store_octet32_il(rb, q, octets, hi);
}
// pointwise products of both parked transforms with one key row: halves below 2p
// (the parked rows and the key row are in interleaved order: octet q of `octets`)
__device__ __forceinline__ void product_octet_pair(const u32* pa, const u32* pb, const u64* __restrict__ key, u32 q,
                                                   u32 octets, u32 p, u64 (&x)[8]) {
  u32 a[8], b[8];
  u64 k[8];
  load_octet32_il(pa, q, octets, a);
  load_octet32_il(pb, q, octets, b);
  load_octet_il(key, q, octets, k);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    u32 kl, kh;
    split64(k[i], kl, kh);
    x[i] = join64(shoup32(a[i], kl, kh, p), shoup32(b[i], kl, kh, p));
  }
}
// v (below 2p) + small signed e, canonical
__device__ __forceinline__ u32 add_small_canon32(u32 v, int e, u32 p) {
  return csub32(csub32(v + p + (u32)e, 2 * p), p);  // below 3p + 19 < 2^32
}

// BFV.Encrypt, two (party, ciphertext) units per CTA.   grid = ceil(n_units / 2) * L
// sampled: [u | e_0 | e_1] bytes per unit of this launch (as for the 64-bit kernel).
// NTT(u) of both units is parked in their c_1 rows.
template <int LOGN, int G>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_encrypt32(DevView v, const __grid_constant__ LimbParams lp, u32 unit_first, u32 n_units,
                const u32* __restrict__ sampled, const u32* __restrict__ plain, u32* ct) {
  const u32 l = blockIdx.x % v.L;
  const UnitPair up = unit_pair(blockIdx.x / v.L, n_units);
  const u32 ua = unit_first + up.la, ub = unit_first + up.lb;
  const LimbTab& lt = lp.limbs[l];
  const u32 p = (u32)lt.p;
  signed char* small = bytes_smem();  // [u | e_0 | e_1] of unit a, then of unit b: 6 N bytes
  u64* sm = poly_smem(6 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u32 words = 3 * (v.n >> 2);
  for (u32 w = threadIdx.x; w < words; w += blockDim.x) {
    reinterpret_cast<u32*>(small)[w] = __ldg(sampled + (size_t)up.la * words + w);
    reinterpret_cast<u32*>(small)[words + w] = __ldg(sampled + (size_t)up.lb * words + w);
  }
  const signed char* sa = small;
  const signed char* sb = small + 3 * v.n;
  u32* park_a = ct + ((size_t)ua * 2 + 1) * poly + row;
  u32* park_b = ct + ((size_t)ub * 2 + 1) * poly + row;
  // the barrier that opens the forward transform publishes the copy
  ntt_forward<LOGN, G, MODE_PAIR>(
      sm, lt, v.logn,
      [&](u32 j) {
        const int a = sa[j], b = sb[j];
        return join64(a < 0 ? p + (u32)a : (u32)a, b < 0 ? p + (u32)b : (u32)b);
      },
      [&](int, u32 q, u64(&x)[8]) { store_octet_halves(park_a, park_b, q, v.n >> 3, up.has_b, x); });
  const u32* ma = plain + (size_t)ua * v.n;
  const u32* mb = plain + (size_t)ub * v.n;
  const u32 delta = (u32)lt.delta, delta_sh = (u32)(lt.delta_sh >> 32);
#pragma unroll 1
  for (u32 comp = 0; comp < 2; ++comp) {
    const u64* key = v.pk32 + comp * poly + row;
    u32* out_a = ct + ((size_t)ua * 2 + comp) * poly + row;
    u32* out_b = ct + ((size_t)ub * 2 + comp) * poly + row;
    const signed char* ea = sa + (comp + 1) * v.n;
    const signed char* eb = sb + (comp + 1) * v.n;
    ntt_inverse<LOGN, G, MODE_PAIR>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          product_octet_pair(park_a, park_b, key, q, v.n >> 3, p, x);
        },
        [&](u32 j, u64 val) {
          u32 lo, hi;
          split64(val, lo, hi);
          if (comp == 0) {  // + Lambda m: both terms brought below p first so that the sum stays below 2^32
            lo = csub32(lo, p) + csub32(shoup32(ma[j], delta, delta_sh, p), p);
            hi = csub32(hi, p) + csub32(shoup32(mb[j], delta, delta_sh, p), p);
          }
          out_a[j] = add_small_canon32(lo, (int)ea[j], p);
          if (up.has_b) out_b[j] = add_small_canon32(hi, (int)eb[j], p);
        });
  }
}

// Decryption shares h = s_k c_1 + e, two (recipient, ciphertext) units per CTA, every listed party
// in turn.   grid = ceil(n_units / 2) * L
// noise[(u * n_parties + a) * N + j] for local unit u, as for the 64-bit kernel.
// NTT(c_1) of both units is parked in the rows of their last shares.
template <int LOGN, int G>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_partial_decrypt32(DevView v, const __grid_constant__ LimbParams lp, const u32* __restrict__ agg,
                        const u32* __restrict__ parties, u32 n_parties, u32 n_cts, u32 unit_first, u32 n_units,
                        const signed char* __restrict__ noise, u32* shares) {
  const u32 l = blockIdx.x % v.L;
  const UnitPair up = unit_pair(blockIdx.x / v.L, n_units);
  const u32 ua = unit_first + up.la, ub = unit_first + up.lb;
  const u32 ira = ua / n_cts, cla = ua % n_cts, irb = ub / n_cts, clb = ub % n_cts;
  const LimbTab& lt = lp.limbs[l];
  const u32 p = (u32)lt.p;
  signed char* staged = bytes_smem();  // two buffers of 2 N bytes: the noise of this pair of shares and of the next
  u64* sm = poly_smem(4 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u32* c1a = agg + ((size_t)ua * 2 + 1) * poly + row;
  const u32* c1b = agg + ((size_t)ub * 2 + 1) * poly + row;
  u32* park_a = shares + (((size_t)ira * n_parties + (n_parties - 1)) * n_cts + cla) * poly + row;
  u32* park_b = shares + (((size_t)irb * n_parties + (n_parties - 1)) * n_cts + clb) * poly + row;
  ntt_forward<LOGN, G, MODE_PAIR>(
      sm, lt, v.logn, [&](u32 j) { return join64(__ldg(c1a + j), __ldg(c1b + j)); },
      [&](int, u32 q, u64(&x)[8]) { store_octet_halves(park_a, park_b, q, v.n >> 3, up.has_b, x); });
#pragma unroll 1
  for (u32 a = 0; a < n_parties; ++a) {
    const u32 party = parties[a];
    if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) continue;
    const u64* key = v.s32 + ((size_t)party * v.L + l) * v.n;
    // Buffer a & 1 was last read in the final round of share a - 2, which every thread left before it
    // passed the barrier that opens the transform of share a - 1; the barrier that opens this
    // share's transform publishes the copy.
    signed char* ea = staged + (a & 1u) * 2 * v.n;
    signed char* eb = ea + v.n;
    {
      const u32* src_a = reinterpret_cast<const u32*>(noise + ((size_t)up.la * n_parties + a) * v.n);
      const u32* src_b = reinterpret_cast<const u32*>(noise + ((size_t)up.lb * n_parties + a) * v.n);
      for (u32 w = threadIdx.x; w < (v.n >> 2); w += blockDim.x) {
        reinterpret_cast<u32*>(ea)[w] = __ldg(src_a + w);
        reinterpret_cast<u32*>(eb)[w] = __ldg(src_b + w);
      }
    }
    u32* out_a = shares + (((size_t)ira * n_parties + a) * n_cts + cla) * poly + row;
    u32* out_b = shares + (((size_t)irb * n_parties + a) * n_cts + clb) * poly + row;
    ntt_inverse<LOGN, G, MODE_PAIR>(
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          product_octet_pair(park_a, park_b, key, q, v.n >> 3, p, x);
        },
        [&](u32 j, u64 val) {
          u32 lo, hi;
          split64(val, lo, hi);
          out_a[j] = add_small_canon32(lo, (int)ea[j], p);
          if (up.has_b) out_b[j] = add_small_canon32(hi, (int)eb[j], p);
        });
  }
}

// BFV.Add over neighbour lists on 32-bit words.  grid = (n_out * n_cts, chunks); four residues per thread.
__global__ void __launch_bounds__(256)
    k_aggregate32(DevView v, const u32* __restrict__ ct, u32 n_cts, const u32* __restrict__ offsets,
                  const u32* __restrict__ rows, u32* __restrict__ agg) {
  const u32 unit = blockIdx.x, i = unit / n_cts, c = unit % n_cts;
  const size_t ct_quads = (size_t)v.L * v.n / 2;  // 2 L N residues = L N / 2 quads
  const u32 beg = offsets[i], end = offsets[i + 1];
  uint4* out = reinterpret_cast<uint4*>(agg) + (size_t)unit * ct_quads;
  for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < ct_quads; e += (size_t)gridDim.y * blockDim.x) {
    const u32 l = (u32)(((e * 4) >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, ct_quads, SITE_ELEMENT) || !D2MHE_CHK(v.chk, l, v.L, SITE_LIMB)) continue;
    const u32 p = (u32)v.limbs[l].p;
    uint4 acc = make_uint4(0, 0, 0, 0);
    for (u32 a = beg; a < end; ++a) {
      const uint4 x = __ldg(reinterpret_cast<const uint4*>(ct) + ((size_t)rows[a] * n_cts + c) * ct_quads + e);
      acc.x = csub32(acc.x + x.x, p);
      acc.y = csub32(acc.y + x.y, p);
      acc.z = csub32(acc.z + x.z, p);
      acc.w = csub32(acc.w + x.w, p);
    }
    out[e] = acc;
  }
}

template <int LOGN, int G>
cudaError_t launch_encrypt32(const DevView& v, const LimbParams& lp, cudaStream_t s, u32 unit_first, u32 n_units,
                             const u32* sampled, const u32* plain, u32* ct) {
  const u32 n = 1u << v.logn;
  return launch_clustered(k_encrypt32<LOGN, G>, ((n_units + 1) / 2) * v.L, ntt_threads(n, G), poly_bytes(n, 6 * (size_t)n),
                          s, 1, v, lp, unit_first, n_units, sampled, plain, ct);
}
template <int LOGN, int G>
cudaError_t launch_pdec32(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* agg, const u32* parties_dev,
                          u32 n_parties, u32 n_cts, u32 unit_first, u32 n_units, const signed char* noise, u32* shares) {
  const u32 n = 1u << v.logn;
  return launch_clustered(k_partial_decrypt32<LOGN, G>, ((n_units + 1) / 2) * v.L, ntt_threads(n, G),
                          poly_bytes(n, 4 * (size_t)n), s, 1, v, lp, agg, parties_dev, n_parties, n_cts, unit_first,
                          n_units, noise, shares);
}

#define D2MHE_DISPATCH32(FN, ...)                                        \
  switch (v.logn) {                                                      \
    case 12: return FN<12, D2MHE_G12>(__VA_ARGS__);                      \
    case 13: return FN<13, D2MHE_G13>(__VA_ARGS__);                      \
    case 14: return FN<14, D2MHE_G14>(__VA_ARGS__);                      \
    default:                                                             \
      if (v.logn > 13) return cudaErrorInvalidValue;                     \
      return FN<0, 1>(__VA_ARGS__);                                      \
  }

cudaError_t encrypt32_units(const DevView& v, const LimbParams& lp, cudaStream_t s, u32 unit_first, u32 n_units,
                            const u32* sampled, const u32* plain, u32* ct) {
  D2MHE_DISPATCH32(launch_encrypt32, v, lp, s, unit_first, n_units, sampled, plain, ct)
}
cudaError_t pdec32_units(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* agg, const u32* parties_dev,
                         u32 n_parties, u32 n_cts, u32 unit_first, u32 n_units, const signed char* noise, u32* shares) {
  D2MHE_DISPATCH32(launch_pdec32, v, lp, s, agg, parties_dev, n_parties, n_cts, unit_first, n_units, noise, shares)
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

// rows of N Montgomery-form residues (limb of row r = r mod L) -> {residue, 32-bit Shoup companion} words
cudaError_t make_tab32(const DevView& v, cudaStream_t s, const u64* src, u64* dst, size_t rows) {
  const size_t count = rows * v.n;
  size_t blocks = (count + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  k_make_tab32<<<(u32)blocks, 256, 0, s>>>(v, src, dst, count);
  return cudaGetLastError();
}

// (the samples come from the sampling kernels of the 64-bit calls: the same bytes)
cudaError_t encrypt32(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                      u32 ct_first, u32 n_cts, const u32* plain, u32* ct, void* scratch, size_t scratch_bytes,
                      u32* launches) {
  const size_t per_unit = 3 * (size_t)v.n;
  const u32 n_units = n_parties * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (per_batch > 1) per_batch &= ~1u;  // whole pairs per batch
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    cudaError_t e = sample_encrypt_noise(v, s, parties_dev, ct_first, n_cts, first, nu, reinterpret_cast<u32*>(scratch));
    if (e != cudaSuccess) return e;
    e = encrypt32_units(v, lp, s, first, nu, reinterpret_cast<const u32*>(scratch), plain, ct);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

cudaError_t aggregate32(const DevView& v, cudaStream_t s, const u32* ct, u32 n_cts, const u32* offsets_dev,
                        const u32* rows_dev, u32 n_out, u32* agg) {
  const size_t ct_quads = (size_t)v.L * v.n / 2;
  u32 by = (u32)((ct_quads + 255) / 256);
  if (by > 32768) by = 32768;
  if (by == 0) by = 1;
  dim3 grid(n_out * n_cts, by);
  k_aggregate32<<<grid, 256, 0, s>>>(v, ct, n_cts, offsets_dev, rows_dev, agg);
  return cudaGetLastError();
}

cudaError_t partial_decrypt32(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* agg,
                              const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties,
                              u32 ct_first, u32 n_cts, u32* shares, void* scratch, size_t scratch_bytes,
                              u32* launches) {
  const size_t per_unit = (size_t)n_parties * v.n;
  const u32 n_units = n_rec * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  if (per_batch < n_units && per_batch > 1) {
    per_batch = 2 * whole_wave_batch(v, per_batch / 2, (n_units + 1) / 2, v.L);  // whole pairs, whole waves
  }
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    cudaError_t e = sample_share_noise(v, s, recipients_dev, parties_dev, n_parties, ct_first, n_cts, first, nu,
                                       reinterpret_cast<u32*>(scratch));
    if (e != cudaSuccess) return e;
    e = pdec32_units(v, lp, s, agg, parties_dev, n_parties, n_cts, first, nu,
                     reinterpret_cast<const signed char*>(scratch), shares);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

}  // namespace D2MHE_LAUNCH_NS
