// Streaming kernels: RNS multiply-add, neighbour sums, combine + exact scale-and-round, packing.
#include "d2mhe_kernels_common.cuh"

namespace {

// d = a (.) b + c per residue; two residues per thread (16-byte accesses).
__global__ void __launch_bounds__(256) k_muladd(DevView v, const u64* __restrict__ a,
                                                const u64* __restrict__ b,
                                                const u64* __restrict__ c, u64* __restrict__ d,
                                                size_t n_pairs) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_pairs; e += stride) {
    const u32 l = (u32)(((e * 2) >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, n_pairs, SITE_ELEMENT) || !D2MHE_CHK(v.chk, l, v.L, SITE_LIMB)) continue;
    const LimbTab* lt = v.limbs + l;
    const u64 p = lt->p, pinv = lt->pinv, r = lt->rmod, rs = lt->rmod_sh;
    const ulonglong2 av = reinterpret_cast<const ulonglong2*>(a)[e];
    const ulonglong2 bv = reinterpret_cast<const ulonglong2*>(b)[e];
    const ulonglong2 cv = reinterpret_cast<const ulonglong2*>(c)[e];
    ulonglong2 o;
    o.x = addmod(shoup_full(mont_lazy(av.x, bv.x, p, pinv), r, rs, p), cv.x, p);
    o.y = addmod(shoup_full(mont_lazy(av.y, bv.y, p, pinv), r, rs, p), cv.y, p);
    reinterpret_cast<ulonglong2*>(d)[e] = o;
  }
}

// ---------------------------------------------------------------------------
// BFV.Add over neighbour lists.  grid = (n_out * n_cts, chunks); two residues per thread.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    k_aggregate(DevView v, const u64* __restrict__ ct, u32 n_cts, const u32* __restrict__ offsets,
                const u32* __restrict__ rows, u64* __restrict__ agg) {
  const u32 unit = blockIdx.x, i = unit / n_cts, c = unit % n_cts;
  const size_t ct_pairs = (size_t)v.L * v.n;  // 2*L*N residues = L*N pairs
  const u32 beg = offsets[i], end = offsets[i + 1];
  const bool lazy = v.wide != 0 && end - beg < 64;
  ulonglong2* out = reinterpret_cast<ulonglong2*>(agg) + (size_t)unit * ct_pairs;
  for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < ct_pairs;
       e += (size_t)gridDim.y * blockDim.x) {
    // a block of 256 pairs lies inside one limb row whenever N >= 512: take the row from a
    // block-uniform index so that the division runs on the uniform datapath
    const size_t e_row = v.n >= 512 ? e - threadIdx.x : e;
    const u32 l = (u32)(((e_row * 2) >> v.logn) % v.L);
    if (!D2MHE_CHK(v.chk, e, ct_pairs, SITE_ELEMENT) || !D2MHE_CHK(v.chk, l, v.L, SITE_LIMB)) continue;
    const u64 p = v.limbs[l].p;
    ulonglong2 acc = make_ulonglong2(0, 0);
    if (lazy) {
      // primes below 2^57 and fewer than 64 addends: the plain 64-bit sums cannot overflow, so the
      // loads are independent (several in flight per thread) and one reduction at the end replaces
      // one per addend
#pragma unroll 4
      for (u32 a = beg; a < end; ++a) {
        const ulonglong2 x =
            __ldg(reinterpret_cast<const ulonglong2*>(ct) + ((size_t)rows[a] * n_cts + c) * ct_pairs + e);
        acc.x += x.x;
        acc.y += x.y;
      }
      const u64 one_sh = v.limbs[l].one_sh;
      acc.x = shoup_full(acc.x, 1, one_sh, p);
      acc.y = shoup_full(acc.y, 1, one_sh, p);
    } else {
      for (u32 a = beg; a < end; ++a) {
        const ulonglong2 x =
            __ldg(reinterpret_cast<const ulonglong2*>(ct) + ((size_t)rows[a] * n_cts + c) * ct_pairs + e);
        acc.x = addmod(acc.x, x.x, p);
        acc.y = addmod(acc.y, x.y, p);
      }
    }
    out[e] = acc;
  }
}

// ---------------------------------------------------------------------------
// Combine + exact scale-and-round.  One thread per coefficient.
//   v_l = c_0 + sum_k h_k mod q_l;  w'_l = t v_l + (q-1)/2 mod q_l;
//   mixed-radix digits d_i of w' in [0,q);  w' mod t = sum d_i prod_{j<i} q_j mod t;
//   x = ((q-1)/2 - w') q^-1 mod t  =  round(t v / q) mod t.
// grid = (n_rec * n_cts, N / 256)
// ---------------------------------------------------------------------------
// Up to 8 limbs the kernel is held to 32 registers (a few spilled words) so that 8 CTAs = 2048 threads
// are resident per SM: the share streams need the loads in flight more than the registers
// (measured: -13 % at N = 16384, L = 8, 20 shares; -2 % at N = 8192, L = 4, 10 shares).
// W = u64, or u32 for the 32-bit-word messages (same arithmetic on the loaded residues).
template <int LMAX, class W>
__global__ void __launch_bounds__(256, LMAX <= 8 ? 8 : 3)
    k_combine(DevView v, const W* __restrict__ agg, const W* __restrict__ shares, u32 n_shares,
              u32 share_comps, u32 n_cts, u32* __restrict__ plain) {
  const u32 unit = blockIdx.x, irec = unit / n_cts, cl = unit % n_cts;
  const u32 j = blockIdx.y * blockDim.x + threadIdx.x;
  if (j >= v.n) return;
  const u32 L = v.L;
  if (!D2MHE_CHK(v.chk, L, (u32)LMAX + 1u, SITE_LIMB)) return;
  const size_t poly = (size_t)L * v.n;
  const W* c0 = agg + (size_t)unit * 2 * poly;
  const bool lazy = (v.wide != 0 || sizeof(W) == 4) && n_shares < 120;
  u64 d[LMAX];
#pragma unroll
  for (int l = 0; l < LMAX; ++l) {
    if (l < (int)L) {
      const LimbTab* lt = v.limbs + l;
      const u64 p = lt->p;
      u64 acc = __ldg(c0 + (size_t)l * v.n + j);
      const W* sh = shares + ((size_t)irec * n_shares * n_cts + cl) * share_comps * poly + (size_t)l * v.n + j;
      const size_t kstride = (size_t)n_cts * share_comps * poly;
      if (lazy) {
        // primes below 2^57 and fewer than 120 shares: the plain 64-bit sum cannot overflow and the
        // multiplication by t below reduces any 64-bit value, so the loads are all independent
#pragma unroll 8
        for (u32 k = 0; k < n_shares; ++k) acc += __ldg(sh + k * kstride);
      } else {
        for (u32 k = 0; k < n_shares; ++k) acc = addmod(acc, __ldg(sh + k * kstride), p);
      }
      d[l] = addmod(shoup_full(acc, lt->tmod, lt->tmod_sh, p), lt->half, p);
    }
  }
  // mixed-radix (Garner) digits in place: d_i <- ((w'_i - d_0) q_0^-1 - d_1) q_1^-1 ... mod q_i
#pragma unroll
  for (int i = 1; i < LMAX; ++i) {
    if (i < (int)L) {
      const LimbTab* lt = v.limbs + i;
      const u64 p = lt->p, cq = lt->cq;
      u64 tmp = d[i];
#pragma unroll
      for (int jj = 0; jj < i; ++jj) {
        const ulonglong2 gi = __ldg(v.round.ginv + i * L + jj);
        tmp = shoup_full(tmp + cq - d[jj], gi.x, gi.y, p);
      }
      d[i] = tmp;
    }
  }
  const u64 t = v.round.t, tsh = v.round.t_sh;
  u64 acc = 0;
#pragma unroll
  for (int i = 0; i < LMAX; ++i) {
    if (i < (int)L) {
      const u64 di = shoup_full(d[i], 1, tsh, t);  // d_i mod t
      acc = shoup_full(acc + di * v.round.prefix_mod_t[i], 1, tsh, t);
    }
  }
  const u64 diff = v.round.half_mod_t + t - acc;  // in (0, 2t)
  plain[(size_t)unit * v.n + j] = (u32)shoup_full(diff * v.round.qinv_mod_t, 1, tsh, t);
}

// ---------------------------------------------------------------------------
// Packing: negacyclic transforms mod t in shared memory (32-bit arithmetic).
// Slot j sits at transform position brv(j).  grid = n_cts
// ---------------------------------------------------------------------------
__device__ __forceinline__ u32 shoup32_lazy(u32 x, uint2 w, u32 t) {
  return x * w.x - __umulhi(x, w.y) * t;
}
__device__ __forceinline__ u32 csub32(u32 x, u32 t) { return x >= t ? x - t : x; }

// Gentleman-Sande / Cooley-Tukey butterflies mod t on lazily reduced 32-bit values (below 2t)
__device__ __forceinline__ void gs32(u32& X, u32& Y, uint2 w, u32 t, u32 twot) {
  const u32 s = X + Y, d = X - Y + twot;
  X = csub32(s, twot);
  Y = shoup32_lazy(d, w, t);
}
__device__ __forceinline__ void ct32(u32& X, u32& Y, uint2 w, u32 t, u32 twot) {
  const u32 x = csub32(X, twot), T = shoup32_lazy(Y, w, t);
  X = x + T;
  Y = x - T + twot;
}

// encode: values -> slots at bit-reversed positions -> inverse transform, two stages per barrier
// values and plain may be the same storage (every CTA reads its whole row into shared memory before
// it writes the row back), so neither pointer is declared __restrict__
__global__ void __launch_bounds__(1024)
    k_encode(DevView v, const int32_t* values, u32* plain, u32 group, size_t group_stride) {
  u32* sm = reinterpret_cast<u32*>(smem_raw);
  const PlainTab pt = v.plain;
  const u32 n = v.n, logn = v.logn, t = pt.t, twot = pt.twot;
  // the values of block b = (g, c), c < group, start at g * group_stride + c * N: contiguous rows when
  // group_stride = group * N, a slice of a larger [.., n_cts, N] array otherwise
  const int32_t* in = values + (size_t)(blockIdx.x / group) * group_stride + (size_t)(blockIdx.x % group) * n;
  u32* out = plain + (size_t)blockIdx.x * n;
  bool bad = false;
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) {
    const int32_t val = in[j];
    bad |= (val > (int32_t)pt.half) || (val < -(int32_t)pt.half);
    int32_t r = val % (int32_t)t;
    if (r < 0) r += (int32_t)t;
    const u32 pos = __brev(j) >> (32 - logn);
    if (D2MHE_CHK(v.chk, pos, n, SITE_STAGED)) sm[pos] = (u32)r;
  }
  if (bad) atomicOr(v.range_flag, 1u);
  __syncthreads();
  u32 lt = 0;  // log2 of the butterfly span of the next stage
  for (; lt + 1 < logn; lt += 2) {
    const u32 span = 1u << lt, m = n >> (lt + 1);
    for (u32 b = threadIdx.x; b < (n >> 2); b += blockDim.x) {
      const u32 i2 = b >> lt, jj = b & (span - 1);
      const u32 base = (i2 << (lt + 2)) + jj;
      if (!D2MHE_CHK(v.chk, base + 3 * span, n, SITE_STAGED) || !D2MHE_CHK(v.chk, m + 2 * i2 + 1, n, SITE_TWIDDLE)) continue;
      u32 x0 = sm[base], x1 = sm[base + span], x2 = sm[base + 2 * span], x3 = sm[base + 3 * span];
      gs32(x0, x1, __ldg(pt.IW + m + 2 * i2), t, twot);
      gs32(x2, x3, __ldg(pt.IW + m + 2 * i2 + 1), t, twot);
      const uint2 w = __ldg(pt.IW + (m >> 1) + i2);
      gs32(x0, x2, w, t, twot);
      gs32(x1, x3, w, t, twot);
      sm[base] = x0;
      sm[base + span] = x1;
      sm[base + 2 * span] = x2;
      sm[base + 3 * span] = x3;
    }
    __syncthreads();
  }
  if (lt < logn) {  // odd number of stages: the last one (m = 1)
    const u32 span = 1u << lt;
    const uint2 w = __ldg(pt.IW + 1);
    for (u32 b = threadIdx.x; b < (n >> 1); b += blockDim.x) {
      u32 x0 = sm[b], x1 = sm[b + span];
      gs32(x0, x1, w, t, twot);
      sm[b] = x0;
      sm[b + span] = x1;
    }
    __syncthreads();
  }
  const uint2 ninv = make_uint2(pt.ninv, pt.ninv_sh);
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) out[j] = csub32(shoup32_lazy(sm[j], ninv, t), t);
}

// decode: forward transform (two stages per barrier), slots read back from bit-reversed positions
// plain and values may be the same storage (see k_encode)
__global__ void __launch_bounds__(1024)
    k_decode(DevView v, const u32* plain, int32_t* values, u32 group, size_t group_stride) {
  u32* sm = reinterpret_cast<u32*>(smem_raw);
  const PlainTab pt = v.plain;
  const u32 n = v.n, logn = v.logn, t = pt.t, twot = pt.twot;
  const u32* in = plain + (size_t)blockIdx.x * n;
  int32_t* out = values + (size_t)(blockIdx.x / group) * group_stride + (size_t)(blockIdx.x % group) * n;  // as in k_encode
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) sm[j] = in[j];
  __syncthreads();
  int lt = (int)logn - 1;  // log2 span of the next stage (m = n >> (lt + 1) groups)
  if (logn & 1u) {  // odd number of stages: do the first one (m = 1) alone
    const u32 span = 1u << lt;
    const uint2 w = __ldg(pt.W + 1);
    for (u32 b = threadIdx.x; b < (n >> 1); b += blockDim.x) {
      u32 x0 = sm[b], x1 = sm[b + span];
      ct32(x0, x1, w, t, twot);
      sm[b] = x0;
      sm[b + span] = x1;
    }
    __syncthreads();
    --lt;
  }
  for (; lt >= 1; lt -= 2) {
    // stages with spans 2^lt (m2 groups) then 2^(lt-1) (2 m2 groups)
    const u32 span = 1u << (lt - 1), m2 = n >> (lt + 1);
    for (u32 b = threadIdx.x; b < (n >> 2); b += blockDim.x) {
      const u32 i2 = b >> (lt - 1), jj = b & (span - 1);
      const u32 base = (i2 << (lt + 1)) + jj;
      if (!D2MHE_CHK(v.chk, base + 3 * span, n, SITE_STAGED) || !D2MHE_CHK(v.chk, 2 * m2 + 2 * i2 + 1, n, SITE_TWIDDLE)) continue;
      u32 x0 = sm[base], x1 = sm[base + span], x2 = sm[base + 2 * span], x3 = sm[base + 3 * span];
      const uint2 w = __ldg(pt.W + m2 + i2);
      ct32(x0, x2, w, t, twot);
      ct32(x1, x3, w, t, twot);
      ct32(x0, x1, __ldg(pt.W + 2 * m2 + 2 * i2), t, twot);
      ct32(x2, x3, __ldg(pt.W + 2 * m2 + 2 * i2 + 1), t, twot);
      sm[base] = x0;
      sm[base + span] = x1;
      sm[base + 2 * span] = x2;
      sm[base + 3 * span] = x3;
    }
    __syncthreads();
  }
  for (u32 j = threadIdx.x; j < n; j += blockDim.x) {
    const u32 pos = __brev(j) >> (32 - logn);
    if (!D2MHE_CHK(v.chk, pos, n, SITE_STAGED)) continue;
    const u32 y = csub32(csub32(sm[pos], twot), t);
    out[j] = y > pt.half ? (int32_t)y - (int32_t)t : (int32_t)y;
  }
}

}  // namespace

namespace D2MHE_LAUNCH_NS {

cudaError_t muladd(const DevView& v, cudaStream_t s, const u64* a, const u64* b, const u64* c,
                   u64* d, u32 batch) {
  const size_t n_pairs = (size_t)batch * v.L * v.n / 2;
  size_t blocks = (n_pairs + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  k_muladd<<<(u32)blocks, 256, 0, s>>>(v, a, b, c, d, n_pairs);
  return cudaGetLastError();
}

cudaError_t aggregate(const DevView& v, cudaStream_t s, const u64* ct, u32 n_cts,
                      const u32* offsets_dev, const u32* rows_dev, u32 n_out, u64* agg) {
  const size_t ct_pairs = (size_t)v.L * v.n;
  u32 by = (u32)((ct_pairs + 255) / 256);
  if (by > 32768) by = 32768;
  dim3 grid(n_out * n_cts, by);
  k_aggregate<<<grid, 256, 0, s>>>(v, ct, n_cts, offsets_dev, rows_dev, agg);
  return cudaGetLastError();
}

template <class W>
static cudaError_t combine_words(const DevView& v, cudaStream_t s, const W* agg, const W* shares, u32 n_rec,
                                 u32 n_shares, u32 share_comps, u32 n_cts, u32* plain) {
  dim3 grid(n_rec * n_cts, (v.n + 255) / 256);
  if (v.L <= 4)
    k_combine<4, W><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, share_comps, n_cts, plain);
  else if (v.L <= 8)
    k_combine<8, W><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, share_comps, n_cts, plain);
  else
    k_combine<D2MHE_MAX_LIMBS, W><<<grid, 256, 0, s>>>(v, agg, shares, n_shares, share_comps, n_cts, plain);
  return cudaGetLastError();
}
cudaError_t combine(const DevView& v, cudaStream_t s, const u64* agg, const u64* shares, u32 n_rec,
                    u32 n_shares, u32 share_comps, u32 n_cts, u32* plain) {
  return combine_words<u64>(v, s, agg, shares, n_rec, n_shares, share_comps, n_cts, plain);
}
cudaError_t combine32(const DevView& v, cudaStream_t s, const u32* agg, const u32* shares, u32 n_rec, u32 n_shares,
                      u32 n_cts, u32* plain) {
  return combine_words<u32>(v, s, agg, shares, n_rec, n_shares, 1, n_cts, plain);
}

// values: n_groups groups of `group` rows of N values, group g starting at values + g * group_stride
// (elements); plain: [n_groups * group, N] contiguous
cudaError_t encode_strided(const DevView& v, cudaStream_t s, const int32_t* values, u32 n_groups, u32 group,
                           size_t group_stride, u32* plain) {
  const size_t smem = (size_t)v.n * 4;
  cudaError_t e = set_smem(k_encode, smem);
  if (e != cudaSuccess) return e;
  u32 threads = v.n / 4 < 1024 ? (v.n / 4 < 32 ? 32 : v.n / 4) : 1024;
  k_encode<<<n_groups * group, threads, smem, s>>>(v, values, plain, group, group_stride);
  return cudaGetLastError();
}
cudaError_t encode(const DevView& v, cudaStream_t s, const int32_t* values, u32 n_cts, u32* plain) {
  return encode_strided(v, s, values, 1, n_cts, (size_t)n_cts * v.n, plain);
}

cudaError_t decode_strided(const DevView& v, cudaStream_t s, const u32* plain, u32 n_groups, u32 group,
                           size_t group_stride, int32_t* values) {
  const size_t smem = (size_t)v.n * 4;
  cudaError_t e = set_smem(k_decode, smem);
  if (e != cudaSuccess) return e;
  u32 threads = v.n / 4 < 1024 ? (v.n / 4 < 32 ? 32 : v.n / 4) : 1024;
  k_decode<<<n_groups * group, threads, smem, s>>>(v, plain, values, group, group_stride);
  return cudaGetLastError();
}
cudaError_t decode(const DevView& v, cudaStream_t s, const u32* plain, u32 n_cts, int32_t* values) {
  return decode_strided(v, s, plain, 1, n_cts, (size_t)n_cts * v.n, values);
}

}  // namespace D2MHE_LAUNCH_NS
