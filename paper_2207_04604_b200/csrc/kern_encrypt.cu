// BFV.Encrypt under the collective key: ct = (Lambda m + u p_0 + e_0, u p_1 + e_1).
#include <algorithm>

#include "d2mhe_kernels_common.cuh"

namespace {

// u, e_0 and e_1 do not depend on the limb: a kernel of its own samples them once per (party,
// ciphertext), one byte per coefficient, into scratch memory that the caller of the launcher lends
// ([u | e_0 | e_1], N bytes each), and the encryption kernel stages them in shared memory.  No
// thread-block clusters: every CTA is placed freely.
// grid = ceil(n_units * 3 * N / 4 / 256); one thread = four samples = one packed word.
__global__ void __launch_bounds__(256)
    k_sample_encrypt_noise(DevView v, const u32* __restrict__ parties, u32 ct_first, u32 n_cts, u32 unit_first,
                           u32 n_units, u32* __restrict__ small) {
  __shared__ GaussTab gt;
  load_gauss(&gt, v.gauss);
  const u32 words = v.n >> 2;
  const size_t total = (size_t)n_units * 3 * words;
  const size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const u32 w = (u32)(e % words), which = (u32)((e / words) % 3), unit = unit_first + (u32)(e / (3 * (size_t)words));
  const u32 party = parties[unit / n_cts], c = ct_first + unit % n_cts;
  if (!D2MHE_CHK(v.chk, party, v.K, SITE_PARTY)) return;
  const Stream st(v.seed, which == 0 ? TAG_ENC_U : which == 1 ? TAG_ENC_E0 : TAG_ENC_E1, c, party, 0);
  u32 pack = 0;
  if (which == 0) {
#pragma unroll
    for (u32 b = 0; b < 4; ++b) pack |= ((u32)st.ternary(4 * w + b) & 0xffu) << (8 * b);
  } else {
#pragma unroll
    for (u32 b = 0; b < 4; ++b) pack |= ((u32)gauss_from_r(gt, st.draw64(4 * w + b)) & 0xffu) << (8 * b);
  }
  small[e] = pack;
}

// grid = n_units * L * split; units unit_first .. unit_first + n_units - 1 of the (party, ciphertext) grid.
// NTT(u) is parked in the output row of c_1 (re-read for both components, overwritten by
// c_1 at the very end), so no registers are held across the two inverse transforms.
// split = 2 (chosen by the launcher when the grid would otherwise leave most SMs idle) gives the two
// components to two thread blocks; each transforms u for itself and parks it in its own output row.
// (The split is a template switch: as a run-time argument it cost the common, unsplit case registers.)
template <int LOGN, int G, bool WIDE, bool SPLIT>
__device__ __forceinline__ void encrypt_body(const DevView& v, const LimbParams& lp, u32 unit_first,
                                             const u32* __restrict__ sampled, const u32* __restrict__ plain, u64* ct) {
  const u32 split = SPLIT ? 2u : 1u;
  const u32 part = SPLIT ? blockIdx.x % 2u : 0u, rest = SPLIT ? blockIdx.x / 2u : blockIdx.x;
  const u32 l = rest % v.L, ulocal = rest / v.L, unit = unit_first + ulocal;
  const LimbTab& lt = lp.limbs[l];
  signed char* small = bytes_smem();  // u, e_0, e_1: N bytes each
  u64* sm = poly_smem(3 * v.n);
  const size_t row = (size_t)l * v.n, poly = (size_t)v.L * v.n;
  const u32* m = plain + (size_t)unit * v.n;
  {
    const u32* src = sampled + (size_t)ulocal * 3 * (v.n >> 2);
    for (u32 w = threadIdx.x; w < 3 * (v.n >> 2); w += blockDim.x) reinterpret_cast<u32*>(small)[w] = __ldg(src + w);
  }
  // the barrier that opens the forward transform publishes the copy
  u64* park = ct + ((size_t)unit * 2 + (split > 1 ? part : 1u)) * poly + row;
  ntt_forward<LOGN, G, WIDE>(
      sm, lt, v.logn, [&](u32 j) { return lift_small((int)small[j], lt.p); },
      [&](int, u32 q, u64(&x)[8]) { store_octet_il(park, q, v.n >> 3, x); });
#pragma unroll 1
  for (u32 comp = split > 1 ? part : 0u; comp < (split > 1 ? part + 1u : 2u); ++comp) {
    const u64* pkh = v.pk_mont + comp * poly + row;
    u64* out = ct + ((size_t)unit * 2 + comp) * poly + row;
    const signed char* e = small + (comp + 1) * v.n;
    ntt_inverse<LOGN, G, WIDE, true>(  // lazy last round: both stores below reduce by the 2^b - d fold
        sm, lt, v.logn,
        [&](int, u32 q, u64(&x)[8]) {
          u64 uh[8];
          load_octet_rw_il(park, q, v.n >> 3, uh);  // written by this same thread
          load_octet_il(pkh, q, v.n >> 3, x);
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = mont_lazy(uh[k], x[k], lt.p, lt.pinv);
        },
        [&](u32 j, u64 val) {
          if (comp == 0) {
            // below 4p + (p + 19) + 2p (WIDE: val below 129p, the fold takes it)
            u64 t = val + lt.p + (u64)(long long)e[j] + shoup_u32(m[j], lt.delta, lt.delta_sh, lt.np);
            out[j] = canon8<WIDE>(t, lt);  // t below 7p + 19 (WIDE: below 132p + 19)
          } else {
            out[j] = add_small_canon<WIDE>(val, (int)e[j], lt);
          }
        });
  }
}

template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_encrypt(DevView v, const __grid_constant__ LimbParams lp, u32 unit_first, const u32* __restrict__ sampled,
              const u32* __restrict__ plain, u64* ct) {
  encrypt_body<LOGN, G, WIDE, false>(v, lp, unit_first, sampled, plain, ct);
}
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_encrypt_split(DevView v, const __grid_constant__ LimbParams lp, u32 unit_first, const u32* __restrict__ sampled,
                    const u32* __restrict__ plain, u64* ct) {
  encrypt_body<LOGN, G, WIDE, true>(v, lp, unit_first, sampled, plain, ct);
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

// u, e_0, e_1 of units unit_first .. unit_first + n_units - 1 into out ([u | e_0 | e_1], N bytes each, per unit)
cudaError_t sample_encrypt_noise(const DevView& v, cudaStream_t s, const u32* parties_dev, u32 ct_first, u32 n_cts,
                                 u32 unit_first, u32 n_units, u32* out) {
  const size_t words = (size_t)n_units * 3 * v.n / 4;
  k_sample_encrypt_noise<<<(unsigned)((words + 255) / 256), 256, 0, s>>>(v, parties_dev, ct_first, n_cts, unit_first,
                                                                        n_units, out);
  return cudaGetLastError();
}

// The split variant serves calls of a few thread blocks, where the latency of one block's transforms is
// what counts: at N = 4096 it runs with one octet per thread and round (512 threads per polynomial).
#undef D2MHE_DISPATCH_G12
#define D2MHE_DISPATCH_G12 1
static cudaError_t encrypt_units_split(const DevView& v, const LimbParams& lp, cudaStream_t s, u32 unit_first,
                                       u32 n_units, const u32* sampled, const u32* plain, u64* ct) {
  D2MHE_DISPATCH_EX(k_encrypt_split, v, n_units * v.L * 2, s, 3 * (size_t)v.n, 1, v, lp, unit_first, sampled, plain,
                    ct);
}
#undef D2MHE_DISPATCH_G12
#define D2MHE_DISPATCH_G12 D2MHE_G12

static cudaError_t encrypt_units(const DevView& v, const LimbParams& lp, cudaStream_t s, u32 unit_first, u32 n_units,
                                 const u32* sampled, const u32* plain, u64* ct) {
  // a small call (at most half of the thread blocks that the GPU holds at once) uses one block per component
  if (n_units * v.L * 2 <= resident_ctas(v)) return encrypt_units_split(v, lp, s, unit_first, n_units, sampled, plain, ct);
  D2MHE_DISPATCH_EX(k_encrypt, v, n_units * v.L, s, 3 * (size_t)v.n, 1, v, lp, unit_first, sampled, plain, ct);
}

// scratch: at least 3 N bytes; (party, ciphertext) units are processed in batches of as many as it holds.
cudaError_t encrypt(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties,
                    u32 ct_first, u32 n_cts, const u32* plain, u64* ct, void* scratch, size_t scratch_bytes,
                    u32* launches) {
  const size_t per_unit = 3 * (size_t)v.n;
  const u32 n_units = n_parties * n_cts;
  u32 per_batch = (u32)std::min<size_t>(scratch_bytes / per_unit, n_units);
  if (launches) *launches = 0;
  if (per_batch == 0) return cudaErrorInvalidValue;
  per_batch = whole_wave_batch(v, per_batch, n_units, v.L);
  for (u32 first = 0; first < n_units; first += per_batch) {
    const u32 nu = std::min(per_batch, n_units - first);
    cudaError_t e = sample_encrypt_noise(v, s, parties_dev, ct_first, n_cts, first, nu, reinterpret_cast<u32*>(scratch));
    if (e != cudaSuccess) return e;
    e = encrypt_units(v, lp, s, first, nu, reinterpret_cast<const u32*>(scratch), plain, ct);
    if (e != cudaSuccess) return e;
    if (launches) *launches += 2;
  }
  return cudaSuccess;
}

}  // namespace D2MHE_LAUNCH_NS
