// 32-bit-word transforms for parameter sets whose primes are all below 2^30: residues are
// u32, polynomials u32[L][N].  One CTA transforms the same limb of TWO polynomials of the batch
// side by side: element j of both travels as one 64-bit word (low half / high half), so the
// shared-memory layout, the swizzle and the round structure are those of the 64-bit engine,
// the twiddle is loaded once for both, and every butterfly is two independent 32-bit Harvey
// butterflies (one high and two low multiplies each).  grid = ceil(batch / 2) * L.
#include "d2mhe_kernels_common.cuh"

namespace {

struct Rows32 {
  u32* a;
  u32* b;
  bool has_b;  // false for the odd polynomial at the end of the batch (b aliases a, stores skipped)
};
__device__ __forceinline__ Rows32 rows_of(const DevView& v, u32* polys, u32 batch) {
  const u32 l = blockIdx.x % v.L, pair = blockIdx.x / v.L;
  Rows32 r;
  r.a = polys + ((size_t)(2 * pair) * v.L + l) * v.n;
  r.has_b = 2 * pair + 1 < batch;
  r.b = r.has_b ? r.a + (size_t)v.L * v.n : r.a;
  return r;
}
__device__ __forceinline__ void load_octet_pair(const u32* a, const u32* b, u64 (&x)[8]) {
  const uint4 a0 = reinterpret_cast<const uint4*>(a)[0], a1 = reinterpret_cast<const uint4*>(a)[1];
  const uint4 b0 = reinterpret_cast<const uint4*>(b)[0], b1 = reinterpret_cast<const uint4*>(b)[1];
  x[0] = join64(a0.x, b0.x);
  x[1] = join64(a0.y, b0.y);
  x[2] = join64(a0.z, b0.z);
  x[3] = join64(a0.w, b0.w);
  x[4] = join64(a1.x, b1.x);
  x[5] = join64(a1.y, b1.y);
  x[6] = join64(a1.z, b1.z);
  x[7] = join64(a1.w, b1.w);
}

template <int LOGN, int G>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt32_fwd(DevView v, const __grid_constant__ LimbParams lp, u32* __restrict__ polys, u32 batch) {
  const LimbTab& lt = lp.limbs[blockIdx.x % v.L];
  const Rows32 r = rows_of(v, polys, batch);
  const u32 p = (u32)lt.p, twop = (u32)lt.twop;
  ntt_forward<LOGN, G, MODE_PAIR>(
      poly_smem(), lt, v.logn, [&](u32 j) { return join64(r.a[j], r.b[j]); },
      [&](int, u32 q, u64(&x)[8]) {
        u32 lo[8], hi[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          split64(x[k], lo[k], hi[k]);
          lo[k] = csub32(csub32(lo[k], twop), p);
          hi[k] = csub32(csub32(hi[k], twop), p);
        }
        uint4* da = reinterpret_cast<uint4*>(r.a + 8 * (size_t)q);
        da[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        da[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
        if (r.has_b) {
          uint4* db = reinterpret_cast<uint4*>(r.b + 8 * (size_t)q);
          db[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          db[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
        }
      });
}

template <int LOGN, int G>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt32_inv(DevView v, const __grid_constant__ LimbParams lp, u32* __restrict__ polys, u32 batch) {
  const LimbTab& lt = lp.limbs[blockIdx.x % v.L];
  const Rows32 r = rows_of(v, polys, batch);
  const u32 p = (u32)lt.p, ninv = (u32)lt.ninv, ninv_sh = (u32)(lt.ninv_sh >> 32);
  ntt_inverse<LOGN, G, MODE_PAIR>(
      poly_smem(), lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) { load_octet_pair(r.a + 8 * (size_t)q, r.b + 8 * (size_t)q, x); },
      [&](u32 j, u64 val) {
        u32 lo, hi;
        split64(val, lo, hi);
        r.a[j] = csub32(shoup32(lo, ninv, ninv_sh, p), p);
        if (r.has_b) r.b[j] = csub32(shoup32(hi, ninv, ninv_sh, p), p);
      });
}

// d = a (.) b + c per residue, four residues per thread (16-byte accesses).
__global__ void __launch_bounds__(256) k_muladd32(DevView v, const u32* __restrict__ a, const u32* __restrict__ b,
                                                  const u32* __restrict__ c, u32* __restrict__ d, size_t n_quads) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_quads; e += stride) {
    const u32 l = (u32)(((e * 4) >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, n_quads, SITE_ELEMENT) || !D2MHE_CHK(v.chk, l, v.L, SITE_LIMB)) continue;
    const LimbTab* lt = v.limbs + l;
    const u64 p = lt->p, one_sh = lt->one_sh;
    const uint4 av = reinterpret_cast<const uint4*>(a)[e];
    const uint4 bv = reinterpret_cast<const uint4*>(b)[e];
    const uint4 cv = reinterpret_cast<const uint4*>(c)[e];
    uint4 o;  // a b + c < 2^60 + 2^30: one reduction by floor(2^64 / p)
    o.x = (u32)shoup_full(mulwide(av.x, bv.x) + cv.x, 1, one_sh, p);
    o.y = (u32)shoup_full(mulwide(av.y, bv.y) + cv.y, 1, one_sh, p);
    o.z = (u32)shoup_full(mulwide(av.z, bv.z) + cv.z, 1, one_sh, p);
    o.w = (u32)shoup_full(mulwide(av.w, bv.w) + cv.w, 1, one_sh, p);
    reinterpret_cast<uint4*>(d)[e] = o;
  }
}

template <int LOGN, int G>
cudaError_t launch_ntt32(const DevView& v, const LimbParams& lp, cudaStream_t s, u32* polys, u32 batch,
                         bool inverse) {
  const u32 n = 1u << v.logn, grid = ((batch + 1) / 2) * v.L;
  const size_t smem = poly_bytes(n);
  if (inverse)
    return launch_clustered(k_ntt32_inv<LOGN, G>, grid, ntt_threads(n, G), smem, s, 1, v, lp, polys, batch);
  return launch_clustered(k_ntt32_fwd<LOGN, G>, grid, ntt_threads(n, G), smem, s, 1, v, lp, polys, batch);
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

cudaError_t ntt32(const DevView& v, const LimbParams& lp, cudaStream_t s, u32* polys, u32 batch, bool inverse) {
  switch (v.logn) {
    case 12: return launch_ntt32<12, D2MHE_G12>(v, lp, s, polys, batch, inverse);
    case 13: return launch_ntt32<13, D2MHE_G13>(v, lp, s, polys, batch, inverse);
    case 14: return launch_ntt32<14, D2MHE_G14>(v, lp, s, polys, batch, inverse);
    default:
      if (v.logn > 13) return cudaErrorInvalidValue;
      return launch_ntt32<0, 1>(v, lp, s, polys, batch, inverse);
  }
}

cudaError_t muladd32(const DevView& v, cudaStream_t s, const u32* a, const u32* b, const u32* c, u32* d,
                     u32 batch) {
  const size_t n_quads = (size_t)batch * v.L * v.n / 4;
  size_t blocks = (n_quads + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  k_muladd32<<<(u32)blocks, 256, 0, s>>>(v, a, b, c, d, n_quads);
  return cudaGetLastError();
}

}  // namespace D2MHE_LAUNCH_NS
