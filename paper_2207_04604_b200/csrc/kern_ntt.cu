// Stand-alone batched transforms (in place) for the kernel sweep.   grid = batch * L
#include "d2mhe_kernels_common.cuh"

namespace {

template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt_fwd(DevView v, const __grid_constant__ LimbParams lp, u64* __restrict__ polys) {
  const u32 l = blockIdx.x % v.L;
  const LimbTab& lt = lp.limbs[l];
  u64* row = polys + (size_t)blockIdx.x * v.n;
  ntt_forward<LOGN, G, WIDE>(
      poly_smem(), lt, v.logn, [&](u32 j) { return row[j]; },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], 1, lt.one_sh, lt.p);
        store_octet(row + 8 * (size_t)q, x);
      });
}

template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt_inv(DevView v, const __grid_constant__ LimbParams lp, u64* __restrict__ polys) {
  const u32 l = blockIdx.x % v.L;
  const LimbTab& lt = lp.limbs[l];
  u64* row = polys + (size_t)blockIdx.x * v.n;
  ntt_inverse<LOGN, G, WIDE>(
      poly_smem(), lt, v.logn,
      [&](int, u32 q, u64(&x)[8]) {
        const ulonglong2* s = reinterpret_cast<const ulonglong2*>(row + 8 * (size_t)q);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          ulonglong2 t = s[k];
          x[2 * k] = t.x;
          x[2 * k + 1] = t.y;
        }
      },
      [&](u32 j, u64 val) { row[j] = shoup_full(val, lt.ninv, lt.ninv_sh, lt.p); });
}


// ---- two-pass transforms for N = 2^15, 2^16 (one polynomial does not fit one CTA) ----------
// Pass A applies the first SA = log2 N - 12 stages in registers: thread o owns the 2^SA
// coefficients o + k * 4096 (coalesced across threads; every thread uses the same 2^SA - 1
// twiddles).  After it the array is 2^SA independent blocks of 4096, each finished by the
// shared-memory engine with the twiddles of its sub-tree (pass B).  The inverse runs B then A.
// Between the passes values are lazily reduced (below 8p); pass A always uses the
// one-conditional-subtraction butterflies, which are valid for every prime below 2^61.
template <int SA, bool INV>
__global__ void __launch_bounds__(256)
    k_ntt_strided(DevView v, const __grid_constant__ LimbParams lp, u64* __restrict__ polys) {
  constexpr int R = 1 << SA;
  const u32 r = blockIdx.x >> 4;  // polynomial-limb; 16 CTAs of 256 columns each
  const LimbTab& lt = lp.limbs[r % v.L];
  const Mod md(lt);
  const u32 o = (blockIdx.x & 15u) * blockDim.x + threadIdx.x;  // < 4096
  u64* row = polys + (size_t)r * v.n + o;
  if (!D2MHE_CHK(v.chk, (size_t)o + ((size_t)(R - 1) << 12), v.n, SITE_LOAD)) return;
  u64 x[R];
#pragma unroll
  for (int k = 0; k < R; ++k) x[k] = row[(size_t)k << 12];
  if (!INV) {
#pragma unroll
    for (int s = 0; s < SA; ++s) {
      const int m = 1 << s, half = R >> (s + 1);
#pragma unroll
      for (int i = 0; i < m; ++i) {
        const ulonglong2 w = __ldg(lt.W + m + i);
#pragma unroll
        for (int j = 0; j < half; ++j) ct_bfly<false>(x[i * 2 * half + j], x[i * 2 * half + j + half], w, md);
      }
    }
#pragma unroll
    for (int k = 0; k < R; ++k) row[(size_t)k << 12] = x[k];
  } else {
#pragma unroll
    for (int s = SA - 1; s >= 0; --s) {
      const int m = 1 << s, half = R >> (s + 1);
#pragma unroll
      for (int i = 0; i < m; ++i) {
        const ulonglong2 w = __ldg(lt.IW + m + i);
#pragma unroll
        for (int j = 0; j < half; ++j)
          gs_bfly<false>(x[i * 2 * half + j], x[i * 2 * half + j + half], w, md, 0);
      }
    }
#pragma unroll
    for (int k = 0; k < R; ++k) row[(size_t)k << 12] = shoup_full(x[k], lt.ninv, lt.ninv_sh, lt.p);
  }
}

// Pass B: block b of polynomial-limb r; grid = batch * L * 2^soff.
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt_fwd_blk(DevView v, const __grid_constant__ LimbParams lp, u64* __restrict__ polys, u32 soff) {
  const u32 b = blockIdx.x & ((1u << soff) - 1), r = blockIdx.x >> soff;
  const LimbTab& lt = lp.limbs[r % v.L];
  u64* row = polys + (size_t)r * v.n + ((size_t)b << LOGN);
  ntt_forward<LOGN, G, WIDE>(
      poly_smem(), lt, LOGN, [&](u32 j) { return row[j]; },
      [&](int, u32 q, u64(&x)[8]) {
#pragma unroll
        for (int k = 0; k < 8; ++k) x[k] = shoup_full(x[k], 1, lt.one_sh, lt.p);
        store_octet(row + 8 * (size_t)q, x);
      },
      soff, b);
}
template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN, G))
    k_ntt_inv_blk(DevView v, const __grid_constant__ LimbParams lp, u64* __restrict__ polys, u32 soff) {
  const u32 b = blockIdx.x & ((1u << soff) - 1), r = blockIdx.x >> soff;
  const LimbTab& lt = lp.limbs[r % v.L];
  u64* row = polys + (size_t)r * v.n + ((size_t)b << LOGN);
  ntt_inverse<LOGN, G, WIDE>(
      poly_smem(), lt, LOGN,
      [&](int, u32 q, u64(&x)[8]) {
        const ulonglong2* s = reinterpret_cast<const ulonglong2*>(row + 8 * (size_t)q);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          ulonglong2 t = s[k];
          x[2 * k] = t.x;
          x[2 * k + 1] = t.y;
        }
      },
      [&](u32 j, u64 val) { row[j] = val; },  // below 4p; pass A scales and reduces
      soff, b);
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

static cudaError_t ntt_two_pass(const DevView& v, const LimbParams& lp, cudaStream_t s, u64* polys,
                                u32 batch, bool inverse) {
  const u32 soff = v.logn - 12, rows = batch * v.L;
  const size_t smem = poly_bytes(4096);
  const u32 grid_a = rows * 16;
  const u32 grid_b = rows << soff, threads = ntt_threads(4096, D2MHE_G12);
  cudaError_t e;
#define D2MHE_STRIDED(SA_, INV_) k_ntt_strided<SA_, INV_><<<grid_a, 256, 0, s>>>(v, lp, polys)
  if (!inverse) {
    if (soff == 3) D2MHE_STRIDED(3, false); else D2MHE_STRIDED(4, false);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (v.wide)
      e = launch_clustered(k_ntt_fwd_blk<12, D2MHE_G12, true>, grid_b, threads, smem, s, 1, v, lp, polys, soff);
    else
      e = launch_clustered(k_ntt_fwd_blk<12, D2MHE_G12, false>, grid_b, threads, smem, s, 1, v, lp, polys, soff);
    return e;
  }
  if (v.wide)
    e = launch_clustered(k_ntt_inv_blk<12, D2MHE_G12, true>, grid_b, threads, smem, s, 1, v, lp, polys, soff);
  else
    e = launch_clustered(k_ntt_inv_blk<12, D2MHE_G12, false>, grid_b, threads, smem, s, 1, v, lp, polys, soff);
  if (e != cudaSuccess) return e;
  if (soff == 3) D2MHE_STRIDED(3, true); else D2MHE_STRIDED(4, true);
#undef D2MHE_STRIDED
  return cudaGetLastError();
}

cudaError_t ntt(const DevView& v, const LimbParams& lp, cudaStream_t s, u64* polys, u32 batch, bool inverse) {
  if (v.logn > 14) return ntt_two_pass(v, lp, s, polys, batch, inverse);
  if (inverse) {
    D2MHE_DISPATCH(k_ntt_inv, v, batch * v.L, s, v, lp, polys);
  } else {
    D2MHE_DISPATCH(k_ntt_fwd, v, batch * v.L, s, v, lp, polys);
  }
}

}  // namespace D2MHE_LAUNCH_NS
