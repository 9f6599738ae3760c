// Stand-alone batched transforms (in place) for the kernel sweep.   grid = batch * L
#include "d2mhe_kernels_common.cuh"

namespace {

template <int LOGN, int G, bool WIDE>
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
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
__global__ void __launch_bounds__(ntt_threads_ct(LOGN, G), ntt_minb_ct(LOGN))
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

}  // namespace

namespace d2mhe_launch {

cudaError_t ntt(const DevView& v, const LimbParams& lp, cudaStream_t s, u64* polys, u32 batch, bool inverse) {
  if (inverse) {
    D2MHE_DISPATCH(k_ntt_inv, v, batch * v.L, s, v, lp, polys);
  } else {
    D2MHE_DISPATCH(k_ntt_fwd, v, batch * v.L, s, v, lp, polys);
  }
}

}  // namespace d2mhe_launch
