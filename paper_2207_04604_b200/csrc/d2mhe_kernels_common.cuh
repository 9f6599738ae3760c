// Shared pieces of the kernel translation units: shared-memory layout, octet I/O, dispatch.
#pragma once
#include <cstdlib>

#include "d2mhe_internal.h"

// Octets per thread and round (G) and resident CTAs per SM aimed at, per ring degree.
// Threads per CTA = N / (8 G).
#ifndef D2MHE_G12
#define D2MHE_G12 2
#endif
#ifndef D2MHE_G13
#define D2MHE_G13 2
#endif
#ifndef D2MHE_G14
#define D2MHE_G14 2
#endif
#ifndef D2MHE_MINB12
#define D2MHE_MINB12 4
#endif
#ifndef D2MHE_MINB13
#define D2MHE_MINB13 2
#endif
#ifndef D2MHE_MINB14
#define D2MHE_MINB14 1
#endif

namespace {

// Resident thread blocks per SM that the kernels of ring degree 2^logn are compiled for.  A build
// with fewer octets per thread than the default (more threads per polynomial: the low-latency
// variants of small calls) is compiled for two blocks per SM (64 registers at 512 threads).
constexpr int ntt_default_g(int logn) { return logn == 12 ? D2MHE_G12 : logn == 13 ? D2MHE_G13 : logn == 14 ? D2MHE_G14 : 1; }
constexpr int ntt_minb_ct(int logn, int g) {
  return g != ntt_default_g(logn) ? 2
                                  : logn == 12 ? D2MHE_MINB12 : logn == 13 ? D2MHE_MINB13 : logn == 14 ? D2MHE_MINB14 : 1;
}

// Shared-memory layout of the transform kernels: [GaussTab][polynomial].
__device__ __forceinline__ void load_gauss(GaussTab* dst, const GaussTab* __restrict__ src) {
  const u32* s = reinterpret_cast<const u32*>(src);
  u32* d = reinterpret_cast<u32*>(dst);
  for (u32 i = threadIdx.x; i < sizeof(GaussTab) / 4; i += blockDim.x) d[i] = s[i];
  __syncthreads();
}

extern __shared__ __align__(16) unsigned char smem_raw[];

// [GaussTab][small-sample bytes: extra_bytes][polynomial]
#define D2MHE_GAUSS_BYTES (((sizeof(GaussTab) + 15) / 16) * 16)
__device__ __forceinline__ GaussTab* gauss_smem() { return reinterpret_cast<GaussTab*>(smem_raw); }
__device__ __forceinline__ signed char* bytes_smem() {
  return reinterpret_cast<signed char*>(smem_raw + D2MHE_GAUSS_BYTES);
}
__device__ __forceinline__ u64* poly_smem(u32 extra_bytes = 0) {
  return reinterpret_cast<u64*>(smem_raw + D2MHE_GAUSS_BYTES + extra_bytes);
}

__device__ __forceinline__ void store_octet(u64* __restrict__ dst, const u64 (&x)[8]) {
  ulonglong2* d = reinterpret_cast<ulonglong2*>(dst);
#pragma unroll
  for (int k = 0; k < 4; ++k) d[k] = make_ulonglong2(x[2 * k], x[2 * k + 1]);
}
__device__ __forceinline__ void load_octet(const u64* __restrict__ src, u64 (&x)[8]) {
  const ulonglong2* s = reinterpret_cast<const ulonglong2*>(src);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    ulonglong2 v = __ldg(s + k);
    x[2 * k] = v.x;
    x[2 * k + 1] = v.y;
  }
}

// plain (coherent) load of an octet that this kernel wrote earlier
__device__ __forceinline__ void load_octet_rw(const u64* src, u64 (&x)[8]) {
  const ulonglong2* s = reinterpret_cast<const ulonglong2*>(src);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    ulonglong2 v = s[k];
    x[2 * k] = v.x;
    x[2 * k + 1] = v.y;
  }
}

// Rows in the transform domain that only this library reads (key tables, parked transforms) are kept
// in interleaved order: the k-th pair of values of octet q (positions 8q + 2k, 8q + 2k + 1) sits in
// 16-byte slot k * octets + q, octets = N / 8.  The threads of a warp own consecutive octets, so each of
// the four 16-byte accesses of an octet covers 512 consecutive bytes (four 128-byte wavefronts of the
// load/store pipe) instead of one slot in each of sixteen lines: measured 5-6 % on the share kernel,
// whose other limit beside the integer multiplier is that pipe.  Pointwise work is indifferent to the
// order; rows that cross the C ABI in the transform domain keep the plain order.
__device__ __forceinline__ void store_octet_il(u64* row, u32 q, u32 octets, const u64 (&x)[8]) {
  ulonglong2* d = reinterpret_cast<ulonglong2*>(row) + q;
#pragma unroll
  for (int k = 0; k < 4; ++k) d[(size_t)k * octets] = make_ulonglong2(x[2 * k], x[2 * k + 1]);
}
__device__ __forceinline__ void load_octet_il(const u64* __restrict__ row, u32 q, u32 octets, u64 (&x)[8]) {
  const ulonglong2* s = reinterpret_cast<const ulonglong2*>(row) + q;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const ulonglong2 t = __ldg(s + (size_t)k * octets);
    x[2 * k] = t.x;
    x[2 * k + 1] = t.y;
  }
}
// plain (coherent) load of an octet that this kernel wrote earlier
__device__ __forceinline__ void load_octet_rw_il(const u64* row, u32 q, u32 octets, u64 (&x)[8]) {
  const ulonglong2* s = reinterpret_cast<const ulonglong2*>(row) + q;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const ulonglong2 t = s[(size_t)k * octets];
    x[2 * k] = t.x;
    x[2 * k + 1] = t.y;
  }
}

// Lambda * m for a plaintext coefficient m < 2^32: exact quotient from two widening
// products, result in [0, 2p).
__device__ __forceinline__ u64 shoup_u32(u32 m, u64 w, u64 ws, u64 np) {
  u32 sl, sh, wl, wh, nl, nh, ql, q, rl, rh;
  split64(ws, sl, sh);
  split64(w, wl, wh);
  split64(np, nl, nh);
  split64(madwide(m, sh, join64(mulhi32(m, sl), 0u)), ql, q);  // q = floor(m ws / 2^64) exactly
  split64(madwide(q, nl, mulwide(m, wl)), rl, rh);
  rh = madlo(m, wh, rh);
  rh = madlo(q, nh, rh);
  return join64(rl, rh);
}

// Canonical representative of s < 8p.  SF: the prime is 2^b - d with 256 d < 2^b (every context that
// runs the WIDE policy); then s = k 2^b + rem is congruent to rem + k d, which is below
// 2^b + 7d < 2p: one widening multiply-add and one conditional subtraction instead of three.
// With SF the same holds for any s below 2^(b+7) + 2^b (k <= 129: rem + k d < p + 130 d < 2p), which is
// what an inverse transform with LAZY_OUT hands over.
template <bool SF = false>
__device__ __forceinline__ u64 canon8(u64 s, const LimbTab& lt) {
  if (SF) {
    u32 s0, s1;
    split64(s, s0, s1);
    const u32 k = s1 >> lt.sf_shift;  // s / 2^b
    return csub(madwide(k, lt.sf_d, join64(s0, s1 & ((1u << lt.sf_shift) - 1u))), lt.p);
  }
  return csub(csub(csub(s, 2 * lt.twop), lt.twop), lt.p);
}

// v (below 4p; with SF below 129p) + small signed e, canonical in [0, p)
template <bool SF = false>
__device__ __forceinline__ u64 add_small_canon(u64 v, int e, const LimbTab& lt) {
  return canon8<SF>(v + lt.p + (u64)(long long)e, lt);  // below 5p + 19 (SF: below 130p + 19)
}

constexpr u32 ntt_threads_ct(int logn, int g) {
  return logn == 0 ? 1024u : (((1u << logn) / 8u / (u32)g) < 32u ? 32u : ((1u << logn) / 8u / (u32)g));
}

// Thread blocks of a transform kernel that the device holds at once.
inline u32 resident_ctas(const DevView& v) { return v.sms * (u32)ntt_minb_ct((int)v.logn, ntt_default_g((int)v.logn)); }
// A call that must be cut into batches (its scratch holds `cap` of its `n_units` units, each unit
// ctas_per_unit thread blocks) takes batches of whole waves of thread blocks when a batch is at least
// one wave: a batch that ends part-way through a wave leaves SMs idle until its last blocks finish.
inline u32 whole_wave_batch(const DevView& v, u32 cap, u32 n_units, u32 ctas_per_unit) {
  if (cap >= n_units) return n_units;
  const u32 res = resident_ctas(v), ctas = cap * ctas_per_unit;
  if (ctas < res) return cap;
  const u32 whole = (ctas / res) * res / ctas_per_unit;
  return whole ? whole : cap;
}

inline size_t poly_bytes(u32 n, size_t extra_bytes = 0) {
  return D2MHE_GAUSS_BYTES + extra_bytes + (size_t)n * sizeof(u64);
}
inline u32 ntt_threads(u32 n, int g) {
  u32 t = n / 8 / g;
  return t < 32 ? 32 : t;
}

// Launch with a thread-block cluster of `cs` CTAs along x (cs = 1: plain launch, which is what every
// kernel of the library uses: kernels that sampled inside clusters were measured slower than
// sampling ahead of the kernel).  Falls back to cs = 1 when the device cannot co-schedule such a
// cluster for this kernel.
template <class... KArgs, class... Args>
cudaError_t launch_clustered(void (*kernel)(KArgs...), u32 grid, u32 threads, size_t smem,
                             cudaStream_t stream, u32 cs, Args... args) {
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(threads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cs > 1) {
    int max_clusters = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg);
    if (e != cudaSuccess || max_clusters < 1) {
      (void)cudaGetLastError();
      attr[0].val.clusterDim.x = 1;
    }
  }
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// D2MHE_EXTRA_TARGS: further template arguments of the kernel (", true"), empty by default; a
// translation unit redefines it around the launcher that needs them.  D2MHE_DISPATCH_G12: octets per
// thread that the dispatch below uses for N = 4096 (the default, or 1 around the launchers of the
// low-latency variants).
#define D2MHE_EXTRA_TARGS
#define D2MHE_DISPATCH_G12 D2MHE_G12
#define D2MHE_LAUNCH_ONE(KERNEL, LOGN_, G_, WIDE_, grid, stream, cs, ...)                      \
  do {                                                                                         \
    cudaError_t e_ = launch_clustered(KERNEL<LOGN_, G_, WIDE_ D2MHE_EXTRA_TARGS>, grid, ntt_threads(n_, G_), \
                                      smem_, stream, cs, __VA_ARGS__);                         \
    if (e_ != cudaSuccess) return e_;                                                          \
  } while (0)

#define D2MHE_LAUNCH_W(KERNEL, LOGN_, G_, wide, grid, stream, cs, ...)                         \
  do {                                                                                         \
    if (wide)                                                                                  \
      D2MHE_LAUNCH_ONE(KERNEL, LOGN_, G_, true, grid, stream, cs, __VA_ARGS__);                \
    else                                                                                       \
      D2MHE_LAUNCH_ONE(KERNEL, LOGN_, G_, false, grid, stream, cs, __VA_ARGS__);               \
  } while (0)

// Picks the instantiation for the ring degree: compile-time sizes for the production
// degrees (with the octets-per-thread count G chosen per degree), the run-time-size build
// for everything else; `wide` selects the lazy-reduction policy (all primes below 2^56).
// extra = bytes of small-sample storage in front of the polynomial; cs = cluster size.
#define D2MHE_DISPATCH_EX(KERNEL, view, grid, stream, extra, cs, ...)                          \
  do {                                                                                         \
    const u32 logn_ = (view).logn, n_ = 1u << logn_;                                           \
    const size_t smem_ = poly_bytes(n_, extra);                                                \
    const bool wide_ = (view).wide != 0;                                                       \
    switch (logn_) {                                                                           \
      case 12:                                                                                 \
        D2MHE_LAUNCH_W(KERNEL, 12, D2MHE_DISPATCH_G12, wide_, grid, stream, cs, __VA_ARGS__);  \
        break;                                                                                 \
      case 13:                                                                                 \
        D2MHE_LAUNCH_W(KERNEL, 13, D2MHE_G13, wide_, grid, stream, cs, __VA_ARGS__);           \
        break;                                                                                 \
      case 14:                                                                                 \
        D2MHE_LAUNCH_W(KERNEL, 14, D2MHE_G14, wide_, grid, stream, cs, __VA_ARGS__);           \
        break;                                                                                 \
      default:                                                                                 \
        if (logn_ > 13) return cudaErrorInvalidValue;                                          \
        D2MHE_LAUNCH_W(KERNEL, 0, 1, wide_, grid, stream, cs, __VA_ARGS__);                    \
        break;                                                                                 \
    }                                                                                          \
    return cudaGetLastError();                                                                 \
  } while (0)

#define D2MHE_DISPATCH(KERNEL, view, grid, stream, ...) \
  D2MHE_DISPATCH_EX(KERNEL, view, grid, stream, 0, 1, __VA_ARGS__)

template <class K>
cudaError_t set_smem(K kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace
