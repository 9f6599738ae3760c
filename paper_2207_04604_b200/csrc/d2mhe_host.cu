// Host side of the C ABI: parameter validation, table construction, argument checks,
// index staging and the chunked whole-round driver.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/d2mhe.h"
#include "d2mhe_internal.h"

typedef unsigned __int128 u128;

// launcher of the context's kernel build (plain, or with index checks in every kernel)
#define L_(fn) (c->checked ? d2mhe_launch_chk::fn : d2mhe_launch::fn)

namespace {

const u64 kGaussCdt[D2MHE_CDT_LEN] = {
#include "dgauss_cdt.inc"
};

// ---- host arithmetic (table construction only) ------------------------------------
u64 h_mul(u64 a, u64 b, u64 p) { return (u64)((u128)a * b % p); }
u64 h_pow(u64 a, u64 e, u64 p) {
  u64 r = 1 % p;
  a %= p;
  for (; e; e >>= 1) {
    if (e & 1) r = h_mul(r, a, p);
    a = h_mul(a, a, p);
  }
  return r;
}
u64 h_inv(u64 a, u64 p) { return h_pow(a, p - 2, p); }
u64 h_shoup(u64 w, u64 p) { return (u64)(((u128)w << 64) / p); }

bool h_is_prime(u64 n) {
  if (n < 2) return false;
  static const u64 bases[] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
  for (u64 b : bases) {
    if (n % b == 0) return n == b;
  }
  u64 d = n - 1;
  int r = 0;
  while ((d & 1) == 0) {
    d >>= 1;
    ++r;
  }
  for (u64 a : bases) {
    u64 x = h_pow(a, d, n);
    if (x == 1 || x == n - 1) continue;
    bool composite = true;
    for (int i = 1; i < r; ++i) {
      x = h_mul(x, x, n);
      if (x == n - 1) {
        composite = false;
        break;
      }
    }
    if (composite) return false;
  }
  return true;
}

// first g^((p-1)/2N), g = 2, 3, ..., of multiplicative order exactly 2N
u64 h_find_root(u64 p, u32 logn) {
  const u64 two_n = (u64)2 << logn, n = (u64)1 << logn;
  for (u64 g = 2; g < 4096; ++g) {
    u64 c = h_pow(g, (p - 1) / two_n, p);
    if (h_pow(c, n, p) == p - 1) return c;
  }
  return 0;
}

// smallest primitive root of the prime t
u64 h_primitive_root(u64 t) {
  std::vector<u64> factors;
  u64 m = t - 1;
  for (u64 f = 2; f * f <= m; ++f) {
    if (m % f == 0) {
      factors.push_back(f);
      while (m % f == 0) m /= f;
    }
  }
  if (m > 1) factors.push_back(m);
  for (u64 g = 2; g < t; ++g) {
    bool ok = true;
    for (u64 f : factors) {
      if (h_pow(g, (t - 1) / f, t) == 1) {
        ok = false;
        break;
      }
    }
    if (ok) return g;
  }
  return 0;
}

u32 h_brv(u32 x, u32 bits) {
  u32 r = 0;
  for (u32 i = 0; i < bits; ++i) {
    r = (r << 1) | (x & 1);
    x >>= 1;
  }
  return r;
}

}  // namespace

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

template <class T>
T* dev_upload(d2mhe_ctx* c, const std::vector<T>& h, cudaError_t* err) {
  void* d = nullptr;
  size_t bytes = std::max<size_t>(h.size() * sizeof(T), 16);
  *err = cudaMalloc(&d, bytes);
  if (*err != cudaSuccess) return nullptr;
  c->allocs.push_back(d);
  if (!h.empty()) *err = cudaMemcpy(d, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice);
  return reinterpret_cast<T*>(d);
}
template <class T>
T* dev_alloc(d2mhe_ctx* c, size_t count, cudaError_t* err) {
  void* d = nullptr;
  *err = cudaMalloc(&d, std::max<size_t>(count * sizeof(T), 16));
  if (*err != cudaSuccess) return nullptr;
  c->allocs.push_back(d);
  return reinterpret_cast<T*>(d);
}

d2mhe_status fail_cuda(d2mhe_ctx* c, cudaError_t e) {
  if (c) c->last_cuda = e;
  return D2MHE_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Stage host index arrays into the next ring slot; returns device pointers for each.
// The slot is reused only after the work that read it has finished (event per slot).
struct Staged {
  const u32* dev[4] = {nullptr, nullptr, nullptr, nullptr};
  int slot = -1;
};
d2mhe_status stage_indices(d2mhe_ctx* c, const u32* const* arrays, const size_t* counts, int n_arrays,
                           Staged* out) {
  size_t total = 0;
  for (int i = 0; i < n_arrays; ++i) total += (counts[i] + 3) & ~(size_t)3;
  if (total > kIdxSlotWords) return D2MHE_ERR_RANGE;
  const int slot = c->idx_next;
  c->idx_next = (c->idx_next + 1) % kIdxSlots;
  if (c->idx_event_valid[slot]) {
    cudaError_t e = cudaEventSynchronize(c->idx_event[slot]);
    if (e != cudaSuccess) return fail_cuda(c, e);
  }
  u32* h = c->idx_host + (size_t)slot * kIdxSlotWords;
  u32* d = c->idx_dev + (size_t)slot * kIdxSlotWords;
  size_t off = 0;
  for (int i = 0; i < n_arrays; ++i) {
    std::memcpy(h + off, arrays[i], counts[i] * sizeof(u32));
    out->dev[i] = d + off;
    off += (counts[i] + 3) & ~(size_t)3;
  }
  cudaError_t e = cudaMemcpyAsync(d, h, off * sizeof(u32), cudaMemcpyHostToDevice, c->stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  out->slot = slot;
  return D2MHE_OK;
}
d2mhe_status release_slot(d2mhe_ctx* c, const Staged& s) {
  cudaError_t e = cudaEventRecord(c->idx_event[s.slot], c->stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->idx_event_valid[s.slot] = true;
  return D2MHE_OK;
}
// Exit of a call that staged indices and then failed with CUDA error `e`: the slot still gets its
// event (whatever was queued before the failure reads it), and the failure is what is reported.
d2mhe_status fail_staged(d2mhe_ctx* c, const Staged& s, cudaError_t e) {
  (void)release_slot(c, s);
  return fail_cuda(c, e);
}

d2mhe_status check_party_list(const d2mhe_ctx* c, const u32* parties, u32 n, bool need_share,
                              bool distinct) {
  if (!parties || n == 0) return D2MHE_ERR_INVALID_ARG;
  std::vector<bool> seen(distinct ? c->params.num_parties : 0, false);
  for (u32 i = 0; i < n; ++i) {
    if (parties[i] >= c->params.num_parties) return D2MHE_ERR_RANGE;
    if (need_share && !c->has_share[parties[i]]) return D2MHE_ERR_STATE;
    if (distinct) {
      if (seen[parties[i]]) return D2MHE_ERR_INVALID_ARG;
      seen[parties[i]] = true;
    }
  }
  return D2MHE_OK;
}

d2mhe_status build_tables(d2mhe_ctx* c) {
  const d2mhe_params& P = c->params;
  const u32 logn = P.log2_n, n = 1u << logn, L = P.num_limbs;
  const u64 t = P.plain_modulus;
  cudaError_t err = cudaSuccess;

  // q as a little-endian multi-word integer is never needed: everything about q that the
  // kernels use is a residue, computed limb by limb.
  // check words of the checked kernel build: {site, index, limit, block}
  c->view.chk = dev_alloc<u32>(c, 4, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  err = cudaMemset(c->view.chk, 0, 16);
  if (err != cudaSuccess) return fail_cuda(c, err);

  std::vector<LimbTab> limbs(L);
  // (q-1)/2 mod m and q mod m for a word-size m: q = prod q_l, so q mod m by repeated products;
  // (q-1)/2 mod m = (q-1) * 2^-1 mod m for odd m.
  auto q_mod = [&](u64 m) {
    u64 r = 1 % m;
    for (u32 l = 0; l < L; ++l) r = h_mul(r, c->moduli[l] % m, m);
    return r;
  };
  // floor(q/t) mod q_l: q = Delta t + (q mod t)  =>  Delta = -(q mod t) t^-1 (mod q_l)
  const u64 q_mod_t = q_mod(t);

  bool all_special = true;  // every prime is 2^b - d with b >= 32, d < 2^32 and 256 d < 2^b
  for (u32 l = 0; l < L; ++l) {
    const u64 p = c->moduli[l];
    LimbTab& T = limbs[l];
    T.chk = c->view.chk;
    T.p = p;
    T.twop = 2 * p;
    T.np = 0 - p;
    u64 inv = 1;  // Newton iteration for p^-1 mod 2^64
    for (int i = 0; i < 6; ++i) inv *= 2 - p * inv;
    T.pinv = inv;
    T.one_sh = h_shoup(1, p);
    T.ninv = h_inv(n % p, p);
    T.ninv_sh = h_shoup(T.ninv, p);
    const u64 r64 = (u64)(((u128)1 << 64) % p);
    T.mont_ninv = h_mul(T.ninv, r64, p);
    T.mont_ninv_sh = h_shoup(T.mont_ninv, p);
    T.rmod = r64;
    T.rmod_sh = h_shoup(r64, p);
    T.delta = h_mul((p - q_mod_t % p) % p, h_inv(t % p, p), p);
    T.delta_sh = h_shoup(T.delta, p);
    T.tmod = t % p;
    T.tmod_sh = h_shoup(T.tmod, p);
    // (q-1)/2 mod q_l: q = 0 mod q_l, so (q-1)/2 = -(2^-1) mod q_l = (q_l - 1)/2
    T.half = (p - 1) / 2;
    const u64 two61 = (u64)1 << 61;
    T.cq = ((two61 + p - 1) / p) * p;
    u32 bits = 0;
    for (u64 x = p; x; x >>= 1) ++bits;
    T.mask = bits >= 64 ? ~(u64)0 : (((u64)1 << bits) - 1);
    T.red_shift = bits - 1;
    T.red_mul = (u32)(((u128)1 << (bits + 15)) / p);
    const u64 gap = bits >= 64 ? 0 : (((u64)1 << bits) - p);  // p = 2^bits - gap
    const bool special = bits >= 32 && gap < ((u64)1 << 32) && (u128)256 * gap < ((u128)1 << bits);
    T.sf_d = special ? (u32)gap : 0;
    T.sf_shift = special ? bits - 32 : 0;
    if (!special) all_special = false;

    const u64 psi = c->roots[l], psi_inv = h_inv(psi, p);
    std::vector<u64> pw(n), ipw(n);
    pw[0] = ipw[0] = 1;
    for (u32 i = 1; i < n; ++i) {
      pw[i] = h_mul(pw[i - 1], psi, p);
      ipw[i] = h_mul(ipw[i - 1], psi_inv, p);
    }
    std::vector<ulonglong2> W(n), IW(n);
    for (u32 i = 0; i < n; ++i) {
      const u32 r = h_brv(i, logn);
      W[i] = make_ulonglong2(pw[r], h_shoup(pw[r], p));
      IW[i] = make_ulonglong2(ipw[r], h_shoup(ipw[r], p));
    }
    T.W = dev_upload(c, W, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    T.IW = dev_upload(c, IW, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    // stride-1 round: the seven twiddles of every octet, one array per twiddle
    const u32 oc = n / 8;
    std::vector<ulonglong2> WL(7 * (size_t)oc), IWL(7 * (size_t)oc);
    for (u32 i = 0; i < oc; ++i) {
      const u32 src[7] = {oc + i, 2 * oc + 2 * i, 2 * oc + 2 * i + 1, 4 * oc + 4 * i, 4 * oc + 4 * i + 1,
                          4 * oc + 4 * i + 2, 4 * oc + 4 * i + 3};
      for (u32 k = 0; k < 7; ++k) {
        WL[(size_t)k * oc + i] = W[src[k]];
        IWL[(size_t)k * oc + i] = IW[src[k]];
      }
    }
    T.WL = dev_upload(c, WL, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    T.IWL = dev_upload(c, IWL, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
  }
  for (u32 l = 0; l < L; ++l) c->limb_params.limbs[l] = limbs[l];
  c->view.limbs = dev_upload(c, limbs, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);

  // Gaussian table and its first-level lookup on the top byte
  {
    std::vector<GaussTab> g(1);
    for (int k = 0; k < D2MHE_CDT_LEN; ++k) g[0].cdt[k] = kGaussCdt[k];
    for (u32 b = 0; b < 256; ++b) {
      const u64 lo = (u64)b << 56;
      const u64 hi = b == 255 ? ~(u64)0 : (((u64)(b + 1) << 56) - 1);
      u32 base = 0, inside = 0;
      for (int k = 0; k < D2MHE_CDT_LEN; ++k) {
        if (kGaussCdt[k] <= lo)
          ++base;
        else if (kGaussCdt[k] <= hi)
          ++inside;
      }
      g[0].lut[b] = (unsigned short)(base | (inside << 8));
    }
    c->view.gauss = dev_upload(c, g, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
  }

  // plaintext-modulus transforms
  PlainTab& pt = c->view.plain;
  std::memset(&pt, 0, sizeof(pt));
  pt.t = (u32)t;
  pt.twot = (u32)(2 * t);
  pt.half = (u32)((t - 1) / 2);
  if (c->can_pack) {
    const u64 g = h_primitive_root(t);
    c->psi_t = h_pow(g, (t - 1) / ((u64)2 << logn), t);
    const u64 psi = c->psi_t, psi_inv = h_inv(psi, t);
    auto sh32 = [&](u64 w) { return (u32)((w << 32) / t); };
    std::vector<u64> pw(n), ipw(n);
    pw[0] = ipw[0] = 1;
    for (u32 i = 1; i < n; ++i) {
      pw[i] = h_mul(pw[i - 1], psi, t);
      ipw[i] = h_mul(ipw[i - 1], psi_inv, t);
    }
    std::vector<uint2> W(n), IW(n);
    for (u32 i = 0; i < n; ++i) {
      const u32 r = h_brv(i, logn);
      W[i] = make_uint2((u32)pw[r], sh32(pw[r]));
      IW[i] = make_uint2((u32)ipw[r], sh32(ipw[r]));
    }
    pt.W = dev_upload(c, W, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    pt.IW = dev_upload(c, IW, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    pt.ninv = (u32)h_inv(n % t, t);
    pt.ninv_sh = sh32(pt.ninv);
  }

  // exact scale-and-round constants
  RoundTab& rt = c->view.round;
  {
    std::vector<ulonglong2> ginv((size_t)L * L, make_ulonglong2(0, 0));
    std::vector<u64> prefix(L);
    u64 acc = 1 % t;
    for (u32 i = 0; i < L; ++i) {
      prefix[i] = acc;
      acc = h_mul(acc, c->moduli[i] % t, t);
      for (u32 j = 0; j < i; ++j) {
        const u64 pi = c->moduli[i];
        const u64 w = h_inv(c->moduli[j] % pi, pi);
        ginv[(size_t)i * L + j] = make_ulonglong2(w, h_shoup(w, pi));
      }
    }
    rt.ginv = dev_upload(c, ginv, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    rt.prefix_mod_t = dev_upload(c, prefix, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    rt.t = t;
    rt.t_sh = h_shoup(1, t);
    // (q-1)/2 mod t = (q mod t - 1) * 2^-1 mod t   (t odd)
    rt.half_mod_t = h_mul((q_mod_t + t - 1) % t, h_inv(2, t), t);
    rt.qinv_mod_t = h_inv(q_mod_t, t);
  }

  // key storage
  const size_t poly = (size_t)L * n;
  c->view.s_mont = dev_alloc<u64>(c, (size_t)P.num_parties * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.pk_mont = dev_alloc<u64>(c, 2 * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.pk_coef = dev_alloc<u64>(c, 2 * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.usk_mont = dev_alloc<u64>(c, (size_t)P.num_parties * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.upk_mont = dev_alloc<u64>(c, (size_t)P.num_parties * 2 * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.upk_coef = dev_alloc<u64>(c, (size_t)P.num_parties * 2 * poly, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  if (c->narrow && P.log2_n <= D2MHE_MAX_SMEM_LOGN) {
    c->view.s32 = dev_alloc<u64>(c, (size_t)P.num_parties * poly, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
    c->view.pk32 = dev_alloc<u64>(c, 2 * poly, &err);
    if (err != cudaSuccess) return fail_cuda(c, err);
  }
  {
    // two waves of thread blocks = 2 * resident / L (recipient, ciphertext) units of K shares each
    int sms = 0;
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    if (err != cudaSuccess) return fail_cuda(c, err);
    const size_t per_sm = logn == 12 ? 4 : logn == 13 ? 2 : 1;  // resident blocks of the transform kernels
    const size_t units = (2 * (size_t)sms * per_sm + L - 1) / L;
    const size_t want = units * P.num_parties * 6 * n;
    c->noise_scratch_bytes = std::min(kNoiseScratchMaxBytes, std::max(kNoiseScratchBytes, (want + 255) / 256 * 256));
  }
  c->noise_scratch = dev_alloc<unsigned char>(c, c->noise_scratch_bytes, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->view.range_flag = dev_alloc<u32>(c, 4, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  err = cudaMemset(c->view.range_flag, 0, 16);
  if (err != cudaSuccess) return fail_cuda(c, err);

  {
    int sms = 0;
    err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device);
    if (err != cudaSuccess) return fail_cuda(c, err);
    c->view.sms = sms > 0 ? (u32)sms : 1u;
  }
  c->view.seed = P.seed;
  c->view.logn = logn;
  c->view.n = n;
  c->view.L = L;
  c->view.K = P.num_parties;
  c->view.wide = all_special ? 1 : 0;
  for (u32 l = 0; l < L; ++l)
    if (c->moduli[l] >= ((u64)1 << 56)) c->view.wide = 0;  // 130 p (a lazily grown value plus its additive terms) must fit 64 bits

  // index staging ring
  err = cudaMallocHost(reinterpret_cast<void**>(&c->idx_host), kIdxSlots * kIdxSlotWords * sizeof(u32));
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->idx_dev = dev_alloc<u32>(c, kIdxSlots * kIdxSlotWords, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  for (int i = 0; i < kIdxSlots; ++i) {
    err = cudaEventCreateWithFlags(&c->idx_event[i], cudaEventDisableTiming);
    if (err != cudaSuccess) return fail_cuda(c, err);
    c->idx_event_valid[i] = false;
  }
  err = cudaMallocHost(reinterpret_cast<void**>(&c->round_lists_host), kIdxSlotWords * sizeof(u32));
  if (err != cudaSuccess) return fail_cuda(c, err);
  c->round_lists_dev = dev_alloc<u32>(c, kIdxSlotWords, &err);
  if (err != cudaSuccess) return fail_cuda(c, err);
  err = cudaEventCreateWithFlags(&c->round_lists_event, cudaEventDisableTiming);
  if (err != cudaSuccess) return fail_cuda(c, err);
  // lanes of the whole-round entry points
  for (int i = 0; i < kRoundLanes; ++i) {
    err = cudaStreamCreateWithFlags(&c->lane_stream[i], cudaStreamNonBlocking);
    if (err != cudaSuccess) return fail_cuda(c, err);
    err = cudaEventCreateWithFlags(&c->lane_event[i], cudaEventDisableTiming);
    if (err != cudaSuccess) return fail_cuda(c, err);
  }
  err = cudaEventCreateWithFlags(&c->fork_event, cudaEventDisableTiming);
  if (err != cudaSuccess) return fail_cuda(c, err);
  return D2MHE_OK;
}

bool protocol_ok(const d2mhe_ctx* c) { return c->params.log2_n <= D2MHE_MAX_SMEM_LOGN; }

}  // namespace

extern "C" {

const char* d2mhe_strerror(d2mhe_status s) {
  switch (s) {
    case D2MHE_OK: return "success";
    case D2MHE_ERR_INVALID_ARG: return "invalid argument";
    case D2MHE_ERR_BAD_PARAMS: return "bad scheme parameters";
    case D2MHE_ERR_STATE: return "call out of order";
    case D2MHE_ERR_WORKSPACE: return "workspace too small";
    case D2MHE_ERR_CUDA: return "CUDA error";
    case D2MHE_ERR_RANGE: return "index or value out of range";
    case D2MHE_ERR_UNSUPPORTED: return "unsupported for these parameters";
    case D2MHE_ERR_DEVICE_CHECK: return "a device-side check failed";
    default: return "unknown status";
  }
}

d2mhe_status d2mhe_create(const d2mhe_params* P, d2mhe_ctx** out) {
  if (out) *out = nullptr;
  if (!P || !out) return D2MHE_ERR_INVALID_ARG;
  if (P->struct_size != sizeof(d2mhe_params)) return D2MHE_ERR_INVALID_ARG;
  if (!P->moduli) return D2MHE_ERR_INVALID_ARG;
  if (P->log2_n < 3 || P->log2_n > 16) return D2MHE_ERR_BAD_PARAMS;
  if (P->num_limbs < 1 || P->num_limbs > D2MHE_MAX_LIMBS) return D2MHE_ERR_BAD_PARAMS;
  if (P->num_parties < 1 || P->num_parties > 65535) return D2MHE_ERR_BAD_PARAMS;
  if (P->gauss_bound != D2MHE_GAUSS_B || (P->flags & ~(u32)D2MHE_FLAG_DEVICE_CHECKS) != 0) return D2MHE_ERR_BAD_PARAMS;
  const u64 t = P->plain_modulus, two_n = (u64)2 << P->log2_n;
  if (t < 3 || t >= ((u64)1 << 30) || !h_is_prime(t)) return D2MHE_ERR_BAD_PARAMS;
  for (u32 l = 0; l < P->num_limbs; ++l) {
    const u64 p = P->moduli[l];
    if (p >= ((u64)1 << 61) || p <= two_n || p % two_n != 1 || p == t || !h_is_prime(p))
      return D2MHE_ERR_BAD_PARAMS;
    for (u32 m = 0; m < l; ++m)
      if (P->moduli[m] == p) return D2MHE_ERR_BAD_PARAMS;
  }
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || P->device < 0 || P->device >= n_dev)
    return D2MHE_ERR_CUDA;

  d2mhe_ctx* c = new (std::nothrow) d2mhe_ctx();
  if (!c) return D2MHE_ERR_CUDA;
  c->params = *P;
  c->moduli.assign(P->moduli, P->moduli + P->num_limbs);
  c->params.moduli = reinterpret_cast<const uint64_t*>(c->moduli.data());
  c->device = P->device;
  c->checked = (P->flags & D2MHE_FLAG_DEVICE_CHECKS) != 0;
  c->can_pack = (t - 1) % two_n == 0;
  c->narrow = true;
  for (u32 l = 0; l < P->num_limbs; ++l)
    if (P->moduli[l] >= ((u64)1 << 30)) c->narrow = false;
  c->all_parties.resize(P->num_parties);
  for (u32 i = 0; i < P->num_parties; ++i) c->all_parties[i] = i;
  c->has_share.assign(P->num_parties, false);
  c->has_user_key.assign(P->num_parties, false);
  std::memset(&c->view, 0, sizeof(c->view));
  std::memset(&c->limb_params, 0, sizeof(c->limb_params));
  for (u32 l = 0; l < P->num_limbs; ++l) {
    u64 r = h_find_root(c->moduli[l], P->log2_n);
    if (!r) {
      delete c;
      return D2MHE_ERR_BAD_PARAMS;
    }
    c->roots.push_back(r);
  }
  DeviceGuard guard(c->device);
  if (!guard.ok) {
    delete c;
    return D2MHE_ERR_CUDA;
  }
  d2mhe_status st = build_tables(c);
  if (st != D2MHE_OK) {
    d2mhe_destroy(c);
    return st;
  }
  *out = c;
  return D2MHE_OK;
}

void d2mhe_destroy(d2mhe_ctx* c) {
  if (!c) return;
  DeviceGuard guard(c->device);
  cudaDeviceSynchronize();
  for (void* p : c->allocs) cudaFree(p);
  if (c->idx_host) cudaFreeHost(c->idx_host);
  if (c->round_lists_host) cudaFreeHost(c->round_lists_host);
  if (c->round_lists_event) cudaEventDestroy(c->round_lists_event);
  for (int i = 0; i < kIdxSlots; ++i)
    if (c->idx_event[i]) cudaEventDestroy(c->idx_event[i]);
  for (int i = 0; i < kRoundLanes; ++i) {
    if (c->lane_event[i]) cudaEventDestroy(c->lane_event[i]);
    if (c->lane_stream[i]) cudaStreamDestroy(c->lane_stream[i]);
  }
  if (c->fork_event) cudaEventDestroy(c->fork_event);
  delete c;
}

d2mhe_status d2mhe_set_stream(d2mhe_ctx* c, void* stream) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  c->stream = reinterpret_cast<cudaStream_t>(stream);
  return D2MHE_OK;
}

d2mhe_status d2mhe_sync(d2mhe_ctx* c) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  u32 flag = 0;
  e = cudaMemcpy(&flag, c->view.range_flag, sizeof(u32), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail_cuda(c, e);
  if (c->checked) {
    u32 words[4] = {0, 0, 0, 0};
    e = cudaMemcpy(words, c->view.chk, sizeof(words), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(c, e);
    if (words[0]) {
      std::memcpy(c->last_check, words, sizeof(words));
      e = cudaMemset(c->view.chk, 0, sizeof(words));
      if (e != cudaSuccess) return fail_cuda(c, e);
      if (flag) (void)cudaMemset(c->view.range_flag, 0, sizeof(u32));
      return D2MHE_ERR_DEVICE_CHECK;
    }
  }
  if (flag) {
    e = cudaMemset(c->view.range_flag, 0, sizeof(u32));
    if (e != cudaSuccess) return fail_cuda(c, e);
    return D2MHE_ERR_RANGE;
  }
  return D2MHE_OK;
}

d2mhe_status d2mhe_debug_last_device_check(const d2mhe_ctx* c, uint32_t info[4]) {
  if (!c || !info) return D2MHE_ERR_INVALID_ARG;
  std::memcpy(info, c->last_check, sizeof(c->last_check));
  return D2MHE_OK;
}

d2mhe_status d2mhe_debug_check_selftest(d2mhe_ctx* c) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(check_selftest)(c->view, c->stream);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

d2mhe_status d2mhe_keygen_share(d2mhe_ctx* c, const u32* parties, u32 n_parties) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, parties, n_parties, false, true);
  if (st != D2MHE_OK) return st;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {parties};
  const size_t counts[1] = {n_parties};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  cudaError_t e = L_(keygen)(c->view, c->limb_params, c->stream, sg.dev[0], n_parties);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 1;
  if (c->view.s32) {  // the same key shares in the form the 32-bit-word calls read
    const size_t poly = (size_t)c->view.L * c->view.n;
    for (u32 i = 0; i < n_parties; ++i) {
      e = L_(make_tab32)(c->view, c->stream, c->view.s_mont + parties[i] * poly, c->view.s32 + parties[i] * poly,
                         c->view.L);
      if (e != cudaSuccess) return fail_staged(c, sg, e);
      c->launches += 1;
    }
  }
  for (u32 i = 0; i < n_parties; ++i) c->has_share[parties[i]] = true;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_collective_pk(d2mhe_ctx* c, const u32* parties, u32 n_parties,
                                 uint64_t* pk_shares_dev, uint64_t* pk_dev) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, parties, n_parties, true, true);
  if (st != D2MHE_OK) return st;
  if (!aligned16(pk_shares_dev) || !aligned16(pk_dev)) return D2MHE_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {parties};
  const size_t counts[1] = {n_parties};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  cudaError_t e = L_(collective_pk)(c->view, c->limb_params, c->stream, sg.dev[0], n_parties,
                                              reinterpret_cast<u64*>(pk_shares_dev));
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 1;
  if (c->view.pk32) {
    e = L_(make_tab32)(c->view, c->stream, c->view.pk_mont, c->view.pk32, 2 * (size_t)c->view.L);
    if (e != cudaSuccess) return fail_staged(c, sg, e);
    c->launches += 1;
  }
  if (pk_dev) {
    e = cudaMemcpyAsync(pk_dev, c->view.pk_coef, 2 * (size_t)c->view.L * c->view.n * sizeof(u64),
                        cudaMemcpyDeviceToDevice, c->stream);
    if (e != cudaSuccess) return fail_staged(c, sg, e);
  }
  c->pk_parties.assign(parties, parties + n_parties);
  c->has_pk = true;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_encode(d2mhe_ctx* c, const int32_t* values_dev, u32 n_cts, u32* plain_dev) {
  if (!c || !values_dev || !plain_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(values_dev) || !aligned16(plain_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->can_pack || c->params.log2_n > 15) return D2MHE_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(encode)(c->view, c->stream, values_dev, n_cts, plain_dev);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

d2mhe_status d2mhe_decode(d2mhe_ctx* c, const u32* plain_dev, u32 n_cts, int32_t* values_dev) {
  if (!c || !values_dev || !plain_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(values_dev) || !aligned16(plain_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->can_pack || c->params.log2_n > 15) return D2MHE_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(decode)(c->view, c->stream, plain_dev, n_cts, values_dev);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

d2mhe_status d2mhe_encrypt(d2mhe_ctx* c, const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                           const u32* plain_dev, uint64_t* ct_dev) {
  if (!c || !plain_dev || !ct_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(plain_dev) || !aligned16(ct_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  d2mhe_status st = check_party_list(c, parties, n_parties, false, false);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_parties * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {parties};
  const size_t counts[1] = {n_parties};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  // u, e_0, e_1 are sampled ahead into the context's scratch, batch by batch
  u32 launched = 0;
  cudaError_t e = L_(encrypt)(c->view, c->limb_params, c->stream, sg.dev[0], n_parties, ct_first, n_cts,
                                        plain_dev, reinterpret_cast<u64*>(ct_dev), c->noise_scratch,
                                        c->noise_scratch_bytes, &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_aggregate(d2mhe_ctx* c, const uint64_t* ct_dev, u32 n_rows, u32 n_cts,
                             const u32* nbr_offsets, const u32* nbr_rows, u32 n_out,
                             uint64_t* agg_dev) {
  if (!c || !ct_dev || !agg_dev || !nbr_offsets || n_rows == 0 || n_cts == 0 || n_out == 0)
    return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(ct_dev) || !aligned16(agg_dev)) return D2MHE_ERR_INVALID_ARG;
  if (n_out > 65536) return D2MHE_ERR_RANGE;
  if (nbr_offsets[0] != 0) return D2MHE_ERR_INVALID_ARG;
  for (u32 i = 0; i < n_out; ++i)
    if (nbr_offsets[i + 1] < nbr_offsets[i]) return D2MHE_ERR_INVALID_ARG;
  const u32 nnz = nbr_offsets[n_out];
  if (nnz > 1048576) return D2MHE_ERR_RANGE;
  if (nnz && !nbr_rows) return D2MHE_ERR_INVALID_ARG;
  for (u32 a = 0; a < nnz; ++a)
    if (nbr_rows[a] >= n_rows) return D2MHE_ERR_RANGE;
  if ((u64)n_out * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32 dummy = 0;
  const u32* arrays[2] = {nbr_offsets, nnz ? nbr_rows : &dummy};
  const size_t counts[2] = {(size_t)n_out + 1, nnz ? (size_t)nnz : 1};
  d2mhe_status st = stage_indices(c, arrays, counts, 2, &sg);
  if (st != D2MHE_OK) return st;
  cudaError_t e = L_(aggregate)(c->view, c->stream, reinterpret_cast<const u64*>(ct_dev), n_cts,
                                          sg.dev[0], sg.dev[1], n_out, reinterpret_cast<u64*>(agg_dev));
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 1;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_partial_decrypt(d2mhe_ctx* c, const uint64_t* agg_dev, const u32* recipients, u32 n_rec,
                                   const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                                   uint64_t* shares_dev) {
  if (!c || !agg_dev || !shares_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, recipients, n_rec, false, false);
  if (st != D2MHE_OK) return st;
  st = check_party_list(c, parties, n_parties, true, true);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_rec * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[2] = {recipients, parties};
  const size_t counts[2] = {n_rec, n_parties};
  // the noise of the shares is sampled ahead into the context's scratch, batch by batch
  if ((size_t)n_parties * c->view.n > c->noise_scratch_bytes) return D2MHE_ERR_UNSUPPORTED;
  if ((st = stage_indices(c, arrays, counts, 2, &sg)) != D2MHE_OK) return st;
  u32 launched = 0;
  cudaError_t e = L_(partial_decrypt_scratch)(
      c->view, c->limb_params, c->stream, reinterpret_cast<const u64*>(agg_dev), sg.dev[0], n_rec, sg.dev[1], n_parties,
      ct_first, n_cts, reinterpret_cast<u64*>(shares_dev), c->noise_scratch, c->noise_scratch_bytes, &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_combine_decrypt(d2mhe_ctx* c, const uint64_t* agg_dev,
                                   const uint64_t* shares_dev, u32 n_rec,
                                   u32 n_shares, u32 n_cts, u32* plain_dev) {
  if (!c || !agg_dev || !shares_dev || !plain_dev || n_rec == 0 || n_cts == 0)
    return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev) || !aligned16(plain_dev))
    return D2MHE_ERR_INVALID_ARG;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  if (n_shares != c->pk_parties.size()) return D2MHE_ERR_INVALID_ARG;
  if ((u64)n_rec * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(combine)(c->view, c->stream, reinterpret_cast<const u64*>(agg_dev),
                                        reinterpret_cast<const u64*>(shares_dev), n_rec, n_shares, 1, n_cts,
                                        plain_dev);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

static d2mhe_status ntt_common(d2mhe_ctx* c, u64* polys_dev, u32 batch, bool inverse) {
  if (!c || !polys_dev || batch == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(polys_dev)) return D2MHE_ERR_INVALID_ARG;
  if ((u64)batch * c->view.L * (c->params.log2_n > D2MHE_MAX_SMEM_LOGN ? 16u : 1u) > 0x7fffffffull)
    return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(ntt)(c->view, c->limb_params, c->stream, polys_dev, batch, inverse);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += c->params.log2_n > D2MHE_MAX_SMEM_LOGN ? 2 : 1;
  return D2MHE_OK;
}
d2mhe_status d2mhe_ntt_forward(d2mhe_ctx* c, uint64_t* polys_dev, u32 batch) {
  return ntt_common(c, reinterpret_cast<u64*>(polys_dev), batch, false);
}
d2mhe_status d2mhe_ntt_inverse(d2mhe_ctx* c, uint64_t* polys_dev, u32 batch) {
  return ntt_common(c, reinterpret_cast<u64*>(polys_dev), batch, true);
}

static d2mhe_status ntt32_common(d2mhe_ctx* c, u32* polys_dev, u32 batch, bool inverse) {
  if (!c || !polys_dev || batch == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(polys_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->narrow || !protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  if ((u64)batch * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(ntt32)(c->view, c->limb_params, c->stream, polys_dev, batch, inverse);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}
d2mhe_status d2mhe_ntt32_forward(d2mhe_ctx* c, uint32_t* polys_dev, u32 batch) {
  return ntt32_common(c, polys_dev, batch, false);
}
d2mhe_status d2mhe_ntt32_inverse(d2mhe_ctx* c, uint32_t* polys_dev, u32 batch) {
  return ntt32_common(c, polys_dev, batch, true);
}
d2mhe_status d2mhe_poly_muladd32(d2mhe_ctx* c, const uint32_t* a, const uint32_t* b, const uint32_t* cc,
                                 uint32_t* d, u32 batch) {
  if (!c || !a || !b || !cc || !d || batch == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(a) || !aligned16(b) || !aligned16(cc) || !aligned16(d)) return D2MHE_ERR_INVALID_ARG;
  if (!c->narrow) return D2MHE_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(muladd32)(c->view, c->stream, a, b, cc, d, batch);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

// ---- the protocol calls on 32-bit words (every prime below 2^30) ------------------------

static bool proto32_ok(const d2mhe_ctx* c) { return c->narrow && protocol_ok(c) && c->view.s32 && c->view.pk32; }

d2mhe_status d2mhe_encrypt32(d2mhe_ctx* c, const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                             const u32* plain_dev, uint32_t* ct_dev) {
  if (!c || !plain_dev || !ct_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(plain_dev) || !aligned16(ct_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!proto32_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  d2mhe_status st = check_party_list(c, parties, n_parties, false, false);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_parties * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {parties};
  const size_t counts[1] = {n_parties};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  u32 launched = 0;
  cudaError_t e = L_(encrypt32)(c->view, c->limb_params, c->stream, sg.dev[0], n_parties, ct_first, n_cts, plain_dev,
                                ct_dev, c->noise_scratch, c->noise_scratch_bytes, &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_aggregate32(d2mhe_ctx* c, const uint32_t* ct_dev, u32 n_rows, u32 n_cts, const u32* nbr_offsets,
                               const u32* nbr_rows, u32 n_out, uint32_t* agg_dev) {
  if (!c || !ct_dev || !agg_dev || !nbr_offsets || n_rows == 0 || n_cts == 0 || n_out == 0)
    return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(ct_dev) || !aligned16(agg_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->narrow || c->params.log2_n < 1) return D2MHE_ERR_UNSUPPORTED;
  if (n_out > 65536) return D2MHE_ERR_RANGE;
  if (nbr_offsets[0] != 0) return D2MHE_ERR_INVALID_ARG;
  for (u32 i = 0; i < n_out; ++i)
    if (nbr_offsets[i + 1] < nbr_offsets[i]) return D2MHE_ERR_INVALID_ARG;
  const u32 nnz = nbr_offsets[n_out];
  if (nnz > 1048576) return D2MHE_ERR_RANGE;
  if (nnz && !nbr_rows) return D2MHE_ERR_INVALID_ARG;
  for (u32 a = 0; a < nnz; ++a)
    if (nbr_rows[a] >= n_rows) return D2MHE_ERR_RANGE;
  if ((u64)n_out * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32 dummy = 0;
  const u32* arrays[2] = {nbr_offsets, nnz ? nbr_rows : &dummy};
  const size_t counts[2] = {(size_t)n_out + 1, nnz ? (size_t)nnz : 1};
  d2mhe_status st = stage_indices(c, arrays, counts, 2, &sg);
  if (st != D2MHE_OK) return st;
  cudaError_t e = L_(aggregate32)(c->view, c->stream, ct_dev, n_cts, sg.dev[0], sg.dev[1], n_out, agg_dev);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 1;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_partial_decrypt32(d2mhe_ctx* c, const uint32_t* agg_dev, const u32* recipients, u32 n_rec,
                                     const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                                     uint32_t* shares_dev) {
  if (!c || !agg_dev || !shares_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!proto32_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, recipients, n_rec, false, false);
  if (st != D2MHE_OK) return st;
  st = check_party_list(c, parties, n_parties, true, true);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_rec * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  if ((size_t)n_parties * c->view.n > c->noise_scratch_bytes) return D2MHE_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[2] = {recipients, parties};
  const size_t counts[2] = {n_rec, n_parties};
  if ((st = stage_indices(c, arrays, counts, 2, &sg)) != D2MHE_OK) return st;
  u32 launched = 0;
  cudaError_t e = L_(partial_decrypt32)(c->view, c->limb_params, c->stream, agg_dev, sg.dev[0], n_rec, sg.dev[1],
                                        n_parties, ct_first, n_cts, shares_dev, c->noise_scratch,
                                        c->noise_scratch_bytes, &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_combine_decrypt32(d2mhe_ctx* c, const uint32_t* agg_dev, const uint32_t* shares_dev, u32 n_rec,
                                     u32 n_shares, u32 n_cts, u32* plain_dev) {
  if (!c || !agg_dev || !shares_dev || !plain_dev || n_rec == 0 || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev) || !aligned16(plain_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->narrow) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  if (n_shares != c->pk_parties.size()) return D2MHE_ERR_INVALID_ARG;
  if ((u64)n_rec * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(combine32)(c->view, c->stream, agg_dev, shares_dev, n_rec, n_shares, n_cts, plain_dev);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

d2mhe_status d2mhe_poly_muladd(d2mhe_ctx* c, const uint64_t* a, const uint64_t* b,
                               const uint64_t* cc, uint64_t* d, u32 batch) {
  if (!c || !a || !b || !cc || !d || batch == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(a) || !aligned16(b) || !aligned16(cc) || !aligned16(d)) return D2MHE_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(muladd)(c->view, c->stream, reinterpret_cast<const u64*>(a),
                                       reinterpret_cast<const u64*>(b), reinterpret_cast<const u64*>(cc),
                                       reinterpret_cast<u64*>(d), batch);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

// ---- MBFV.Convert to a recipient's own key ---------------------------------------------

d2mhe_status d2mhe_user_keygen(d2mhe_ctx* c, const u32* users, u32 n_users, uint64_t* pk_out_dev) {
  if (!c) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, users, n_users, false, true);
  if (st != D2MHE_OK) return st;
  if (!aligned16(pk_out_dev)) return D2MHE_ERR_INVALID_ARG;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {users};
  const size_t counts[1] = {n_users};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  cudaError_t e = L_(user_keygen)(c->view, c->limb_params, c->stream, sg.dev[0], n_users);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 1;
  const size_t pk_words = 2 * (size_t)c->view.L * c->view.n;
  if (pk_out_dev) {
    for (u32 i = 0; i < n_users; ++i) {
      e = cudaMemcpyAsync(pk_out_dev + (size_t)i * pk_words, c->view.upk_coef + (size_t)users[i] * pk_words,
                          pk_words * sizeof(u64), cudaMemcpyDeviceToDevice, c->stream);
      if (e != cudaSuccess) return fail_staged(c, sg, e);
    }
  }
  for (u32 i = 0; i < n_users; ++i) c->has_user_key[users[i]] = true;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_convert_share(d2mhe_ctx* c, const uint64_t* agg_dev, const u32* recipients, u32 n_rec,
                                 const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                                 uint64_t* shares_dev) {
  if (!c || !agg_dev || !shares_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, recipients, n_rec, false, false);
  if (st != D2MHE_OK) return st;
  for (u32 i = 0; i < n_rec; ++i)
    if (!c->has_user_key[recipients[i]]) return D2MHE_ERR_STATE;
  st = check_party_list(c, parties, n_parties, true, true);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_rec * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[2] = {recipients, parties};
  const size_t counts[2] = {n_rec, n_parties};
  // mu_k, e_{0,k}, e_{1,k} are sampled ahead into the context's scratch, batch by batch
  if ((size_t)n_parties * 3 * c->view.n > c->noise_scratch_bytes) return D2MHE_ERR_UNSUPPORTED;
  if ((st = stage_indices(c, arrays, counts, 2, &sg)) != D2MHE_OK) return st;
  u32 launched = 0;
  cudaError_t e = L_(convert_share)(c->view, c->limb_params, c->stream, reinterpret_cast<const u64*>(agg_dev),
                                    sg.dev[0], n_rec, sg.dev[1], n_parties, ct_first, n_cts,
                                    reinterpret_cast<u64*>(shares_dev), c->noise_scratch, c->noise_scratch_bytes,
                                    &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_convert_combine(d2mhe_ctx* c, const uint64_t* agg_dev, const uint64_t* shares_dev,
                                   u32 n_rec, u32 n_shares, u32 n_cts, uint64_t* ct_out_dev) {
  if (!c || !agg_dev || !shares_dev || !ct_out_dev || n_rec == 0 || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev) || !aligned16(ct_out_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  if (n_shares != c->pk_parties.size()) return D2MHE_ERR_INVALID_ARG;
  if ((u64)n_rec * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  cudaError_t e = L_(convert_combine)(c->view, c->stream, reinterpret_cast<const u64*>(agg_dev),
                                                reinterpret_cast<const u64*>(shares_dev), n_rec, n_shares, n_cts,
                                                reinterpret_cast<u64*>(ct_out_dev));
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 1;
  return D2MHE_OK;
}

d2mhe_status d2mhe_decrypt(d2mhe_ctx* c, const u32* users, u32 n_users, const uint64_t* ct_dev, u32 n_cts,
                           uint64_t* scratch_dev, u32* plain_dev) {
  if (!c || !ct_dev || !scratch_dev || !plain_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(ct_dev) || !aligned16(scratch_dev) || !aligned16(plain_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, users, n_users, false, false);
  if (st != D2MHE_OK) return st;
  for (u32 i = 0; i < n_users; ++i)
    if (!c->has_user_key[users[i]]) return D2MHE_ERR_STATE;
  if ((u64)n_users * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {users};
  const size_t counts[1] = {n_users};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  cudaError_t e = L_(secret_product)(c->view, c->limb_params, c->stream,
                                               reinterpret_cast<const u64*>(ct_dev), sg.dev[0], n_users, n_cts,
                                               reinterpret_cast<u64*>(scratch_dev));
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  // [c_0 + c_1 sk_i]_q then the exact scale-and-round: the product plays the role of one share
  e = L_(combine)(c->view, c->stream, reinterpret_cast<const u64*>(ct_dev),
                            reinterpret_cast<const u64*>(scratch_dev), n_users, 1, 1, n_cts, plain_dev);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 2;
  return release_slot(c, sg);
}

// ---- MBFV.Bootstrap ---------------------------------------------------------------------

d2mhe_status d2mhe_bootstrap_share(d2mhe_ctx* c, const uint64_t* agg_dev, const u32* recipients, u32 n_rec,
                                   const u32* parties, u32 n_parties, u32 ct_first, u32 n_cts,
                                   uint64_t* shares_dev) {
  if (!c || !agg_dev || !shares_dev || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev)) return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  d2mhe_status st = check_party_list(c, recipients, n_rec, false, false);
  if (st != D2MHE_OK) return st;
  st = check_party_list(c, parties, n_parties, true, true);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if ((u64)n_rec * n_cts * c->view.L > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[2] = {recipients, parties};
  const size_t counts[2] = {n_rec, n_parties};
  // e_{0,k}, e_{1,k} and the masks M_k are sampled ahead into the context's scratch, batch by batch
  if ((size_t)n_parties * 6 * c->view.n > c->noise_scratch_bytes) return D2MHE_ERR_UNSUPPORTED;
  if ((st = stage_indices(c, arrays, counts, 2, &sg)) != D2MHE_OK) return st;
  u32 launched = 0;
  cudaError_t e = L_(boot_share)(c->view, c->limb_params, c->stream, reinterpret_cast<const u64*>(agg_dev),
                                 sg.dev[0], n_rec, sg.dev[1], n_parties, ct_first, n_cts,
                                 reinterpret_cast<u64*>(shares_dev), c->noise_scratch, c->noise_scratch_bytes,
                                 &launched);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += launched;
  return release_slot(c, sg);
}

d2mhe_status d2mhe_bootstrap_combine(d2mhe_ctx* c, const uint64_t* agg_dev, const uint64_t* shares_dev,
                                     const u32* recipients, u32 n_rec, u32 n_shares, u32 ct_first,
                                     u32 n_cts, u32* plain_scratch_dev, uint64_t* ct_out_dev) {
  if (!c || !agg_dev || !shares_dev || !plain_scratch_dev || !ct_out_dev || n_cts == 0)
    return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(agg_dev) || !aligned16(shares_dev) || !aligned16(plain_scratch_dev) || !aligned16(ct_out_dev))
    return D2MHE_ERR_INVALID_ARG;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  if (n_shares != c->pk_parties.size()) return D2MHE_ERR_INVALID_ARG;
  d2mhe_status st = check_party_list(c, recipients, n_rec, false, false);
  if (st != D2MHE_OK) return st;
  if ((u64)ct_first + n_cts > 0x100000000ull || (u64)n_rec * n_cts > 0x7fffffffull) return D2MHE_ERR_RANGE;
  DeviceGuard guard(c->device);
  Staged sg;
  const u32* arrays[1] = {recipients};
  const size_t counts[1] = {n_rec};
  if ((st = stage_indices(c, arrays, counts, 1, &sg)) != D2MHE_OK) return st;
  cudaError_t e = L_(combine)(c->view, c->stream, reinterpret_cast<const u64*>(agg_dev),
                                        reinterpret_cast<const u64*>(shares_dev), n_rec, n_shares, 2, n_cts,
                                        plain_scratch_dev);
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  e = L_(boot_finish)(c->view, c->stream, plain_scratch_dev, reinterpret_cast<const u64*>(shares_dev),
                                sg.dev[0], n_rec, n_shares, ct_first, n_cts, reinterpret_cast<u64*>(ct_out_dev));
  if (e != cudaSuccess) return fail_staged(c, sg, e);
  c->launches += 2;
  return release_slot(c, sg);
}

// ---- whole round ---------------------------------------------------------------------

// Per ciphertext index of a chunk: plain K*N u32, ct and agg K*2*L*N u64 each,
// shares K*K*L*N u64 (S = K share holders), and one byte per sample for what is sampled ahead of the
// encryption and share kernels (3 K N for the ciphertexts, then K S N for the shares, in the same place).
static size_t round_noise_bytes_per_ct(const d2mhe_ctx* c) {
  const size_t K = c->params.num_parties, S = c->pk_parties.empty() ? K : c->pk_parties.size();
  return (std::max(K * S, 3 * K) * c->view.n + 15) / 16 * 16;  // shares' noise, or [u | e_0 | e_1] per ciphertext
}
static size_t round_bytes_per_ct(const d2mhe_ctx* c) {
  const size_t K = c->params.num_parties, S = c->pk_parties.empty() ? K : c->pk_parties.size();
  const size_t n = c->view.n, poly = (size_t)c->view.L * n * sizeof(u64);
  return K * n * sizeof(u32) + 2 * (K * 2 * poly) + K * S * poly + round_noise_bytes_per_ct(c);
}

size_t d2mhe_round_workspace_bytes(const d2mhe_ctx* c, u32 chunk_cts) {
  if (!c || chunk_cts == 0) return 0;
  return round_bytes_per_ct(c) * chunk_cts + 256;
}

// Fewest sub-chunks (a whole number of passes over the lanes, sizes differing by at most one,
// larger ones first) such that the first pass, which holds the largest ones, fits a workspace
// for `cap` ciphertext indices and no sub-chunk exceeds `max_sub`.
struct RoundPlan {
  u32 lanes, n_sub, sub_small, n_large;  // the first n_large sub-chunks hold sub_small + 1 indices
};
static RoundPlan plan_round(u32 n_cts, size_t cap, size_t max_sub, int max_lanes) {
  RoundPlan pl;
  // fewer than four indices: one stream (the fork and join of a second one cost more than they hide)
  if (n_cts < 4) max_lanes = 1;
  pl.lanes = (u32)std::min<size_t>(std::min<size_t>(max_lanes, cap), n_cts);
  u32 n_sub = pl.lanes;
  for (;; n_sub += pl.lanes) {
    if (n_sub >= n_cts) {
      n_sub = n_cts;
      break;
    }
    const u32 small = n_cts / n_sub, n_big = n_cts % n_sub;
    size_t first_pass = 0;
    for (u32 l = 0; l < pl.lanes; ++l) first_pass += small + (l < n_big ? 1u : 0u);
    if (first_pass <= cap && small + (n_big ? 1u : 0u) <= max_sub) break;
  }
  pl.n_sub = n_sub;
  pl.sub_small = n_cts / n_sub;
  pl.n_large = n_cts % n_sub;
  return pl;
}

uint32_t d2mhe_round_plan(u32 n_cts, uint64_t cap_cts, u32* sizes, u32 max_out, u32* lanes_out) {
  if (n_cts == 0 || cap_cts == 0) return 0;
  const RoundPlan pl = plan_round(n_cts, (size_t)cap_cts, 0x7fffffffu, kRoundLanesDevice);
  if (lanes_out) *lanes_out = pl.lanes;
  for (u32 i = 0; sizes && i < pl.n_sub && i < max_out; ++i) sizes[i] = pl.sub_small + (i < pl.n_large ? 1u : 0u);
  return pl.n_sub;
}

// The ciphertext-index range is cut into sub-chunks that are issued in turn on a few
// internal streams ("lanes"), each with its own part of the workspace: one lane's copies,
// memory-bound kernels and partial last waves overlap the other lane's arithmetic.  The
// lanes start after everything queued on the context's stream so far and the context's
// stream continues after all of them have finished.
static d2mhe_status round_impl(d2mhe_ctx* c, const int32_t* values, bool host_io, u32 ct_first,
                               u32 n_cts, const u32* nbr_offsets, const u32* nbr_rows,
                               int32_t* sums, void* ws, size_t ws_bytes) {
  if (!c || !values || !sums || !nbr_offsets || !ws || n_cts == 0) return D2MHE_ERR_INVALID_ARG;
  if (!aligned16(ws) || (!host_io && (!aligned16(values) || !aligned16(sums))))
    return D2MHE_ERR_INVALID_ARG;
  if (!protocol_ok(c) || !c->can_pack) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_pk) return D2MHE_ERR_STATE;
  const u32 K = c->params.num_parties, S = (u32)c->pk_parties.size(), L = c->view.L;
  if ((u64)ct_first + n_cts > 0x100000000ull) return D2MHE_ERR_RANGE;
  if (nbr_offsets[0] != 0) return D2MHE_ERR_INVALID_ARG;
  for (u32 i = 0; i < K; ++i)
    if (nbr_offsets[i + 1] < nbr_offsets[i]) return D2MHE_ERR_INVALID_ARG;
  const u32 nnz = nbr_offsets[K];
  if (nnz > 1048576) return D2MHE_ERR_RANGE;
  if (nnz && !nbr_rows) return D2MHE_ERR_INVALID_ARG;
  for (u32 a = 0; a < nnz; ++a)
    if (nbr_rows[a] >= K) return D2MHE_ERR_RANGE;
  const size_t n = c->view.n, polyw = (size_t)L * n;
  const size_t per_ct = round_bytes_per_ct(c);
  if (ws_bytes < per_ct + 256) return D2MHE_ERR_WORKSPACE;
  const size_t cap = (ws_bytes - 256) / per_ct;  // ciphertext indices the workspace holds
  const size_t grid_cap = 0x7fffffffull / ((u64)K * std::max(L, 2u));  // launch-grid limit of the kernels
  const RoundPlan plan = plan_round(n_cts, cap, grid_cap, host_io ? kRoundLanesHost : kRoundLanesDevice);
  const u32 lanes = plan.lanes, n_sub = plan.n_sub, sub_small = plan.sub_small, n_large = plan.n_large;
  size_t lane_first[kRoundLanes + 1] = {};                       // lane l starts this many indices into the workspace
  for (u32 l = 0; l < lanes; ++l) lane_first[l + 1] = lane_first[l] + sub_small + (l < n_large ? 1u : 0u);

  DeviceGuard guard(c->device);
  const u32 dummy = 0;
  // The four index lists of every sub-chunk.  They rarely change from one round to the next, so they
  // stay on the device and are uploaded (stream-ordered after the earlier rounds that read them) only
  // when they differ from what is there.
  Staged sg;
  const u32* arrays[4] = {c->all_parties.data(), c->pk_parties.data(), nbr_offsets, nnz ? nbr_rows : &dummy};
  const size_t counts[4] = {K, S, (size_t)K + 1, nnz ? (size_t)nnz : 1};
  d2mhe_status st = D2MHE_OK;
  {
    size_t off[5] = {0, 0, 0, 0, 0};
    for (int i = 0; i < 4; ++i) off[i + 1] = off[i] + ((counts[i] + 3) & ~(size_t)3);
    if (off[4] > kIdxSlotWords) return D2MHE_ERR_RANGE;
    bool same = c->round_lists_valid && c->round_lists_cache.size() == off[4];
    for (int i = 0; same && i < 4; ++i)
      same = std::memcmp(c->round_lists_cache.data() + off[i], arrays[i], counts[i] * sizeof(u32)) == 0;
    if (!same) {
      cudaError_t e2 = c->round_lists_valid ? cudaEventSynchronize(c->round_lists_event) : cudaSuccess;  // the pinned source is free again
      if (e2 != cudaSuccess) return fail_cuda(c, e2);
      c->round_lists_valid = false;
      c->round_lists_cache.assign(off[4], 0u);
      for (int i = 0; i < 4; ++i)
        std::memcpy(c->round_lists_cache.data() + off[i], arrays[i], counts[i] * sizeof(u32));
      std::memcpy(c->round_lists_host, c->round_lists_cache.data(), off[4] * sizeof(u32));
      e2 = cudaMemcpyAsync(c->round_lists_dev, c->round_lists_host, off[4] * sizeof(u32), cudaMemcpyHostToDevice,
                           c->stream);
      if (e2 == cudaSuccess) e2 = cudaEventRecord(c->round_lists_event, c->stream);
      if (e2 != cudaSuccess) return fail_cuda(c, e2);
      c->round_lists_valid = true;
    }
    for (int i = 0; i < 4; ++i) sg.dev[i] = c->round_lists_dev + off[i];
  }
  unsigned char* base = reinterpret_cast<unsigned char*>(ws);
  // Everything between the fork and the join; a failure stops issuing, and the join below still runs,
  // so that the context's stream stays ordered after whatever the lanes were given.
  auto issue = [&]() -> cudaError_t {
    cudaError_t e;
    if (lanes > 1) {
      if ((e = cudaEventRecord(c->fork_event, c->stream)) != cudaSuccess) return e;
      for (u32 l = 0; l < lanes; ++l)
        if ((e = cudaStreamWaitEvent(c->lane_stream[l], c->fork_event, 0)) != cudaSuccess) return e;
    }
    u32 done = 0;
    for (u32 i = 0; i < n_sub; ++i) {
      const u32 cc = sub_small + (i < n_large ? 1u : 0u), lane = i % lanes;
      cudaStream_t s = lanes > 1 ? c->lane_stream[lane] : c->stream;
      // layout of the lane's part (all 16-byte aligned: every block is a multiple of 16 bytes)
      unsigned char* lane_base = base + lane_first[lane] * per_ct;
      u32* plain = reinterpret_cast<u32*>(lane_base);
      u64* ct = reinterpret_cast<u64*>(lane_base + (size_t)K * cc * n * sizeof(u32));
      u64* agg = ct + (size_t)K * cc * 2 * polyw;
      u64* shares = agg + (size_t)K * cc * 2 * polyw;
      int32_t* vals_dev = reinterpret_cast<int32_t*>(plain);  // with host buffers encode and decode run in place
      // values are [K, n_cts, N]: the sub-chunk is K groups of cc rows, groups n_cts*N apart.  Device
      // buffers are read and written in place by the packing kernels; host buffers go through one
      // strided copy each way.
      if (host_io) {
        e = cudaMemcpy2DAsync(vals_dev, (size_t)cc * n * sizeof(int32_t), values + (size_t)done * n,
                              (size_t)n_cts * n * sizeof(int32_t), (size_t)cc * n * sizeof(int32_t), K,
                              cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return e;
        if ((e = L_(encode)(c->view, s, vals_dev, K * cc, plain)) != cudaSuccess) return e;
      } else {
        if ((e = L_(encode_strided)(c->view, s, values + (size_t)done * n, K, cc, (size_t)n_cts * n, plain)) !=
            cudaSuccess)
          return e;
      }
      unsigned char* noise = reinterpret_cast<unsigned char*>(shares + (size_t)K * S * cc * polyw);
      const size_t noise_bytes = round_noise_bytes_per_ct(c) * cc;  // first u, e_0, e_1, later the shares' noise
      u32 enc_launches = 0;
      if ((e = L_(encrypt)(c->view, c->limb_params, s, sg.dev[0], K, ct_first + done, cc, plain, ct, noise,
                           noise_bytes, &enc_launches)) != cudaSuccess)
        return e;
      if ((e = L_(aggregate)(c->view, s, ct, cc, sg.dev[2], sg.dev[3], K, agg)) != cudaSuccess) return e;
      u32 pdec_launches = 0;
      if ((e = L_(partial_decrypt_scratch)(c->view, c->limb_params, s, agg, sg.dev[0], K, sg.dev[1], S,
                                           ct_first + done, cc, shares, noise, noise_bytes, &pdec_launches)) !=
          cudaSuccess)
        return e;
      if ((e = L_(combine)(c->view, s, agg, shares, K, S, 1, cc, plain)) != cudaSuccess) return e;
      c->launches += 4 + enc_launches + pdec_launches;
      if (host_io) {
        if ((e = L_(decode)(c->view, s, plain, K * cc, vals_dev)) != cudaSuccess) return e;
        e = cudaMemcpy2DAsync(sums + (size_t)done * n, (size_t)n_cts * n * sizeof(int32_t), vals_dev,
                              (size_t)cc * n * sizeof(int32_t), (size_t)cc * n * sizeof(int32_t), K,
                              cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return e;
      } else {
        if ((e = L_(decode_strided)(c->view, s, plain, K, cc, (size_t)n_cts * n, sums + (size_t)done * n)) !=
            cudaSuccess)
          return e;
      }
      done += cc;
    }
    return cudaSuccess;
  };
  cudaError_t e = issue();
  if (lanes > 1) {
    for (u32 l = 0; l < lanes; ++l) {
      cudaError_t j = cudaEventRecord(c->lane_event[l], c->lane_stream[l]);
      if (j == cudaSuccess) j = cudaStreamWaitEvent(c->stream, c->lane_event[l], 0);
      if (e == cudaSuccess) e = j;
    }
  }
  if (e != cudaSuccess) return fail_cuda(c, e);
  if (host_io) {
    // the call returns when the sums are in host memory, so it can also report values that
    // d2mhe_encode found out of range (the flag is cleared, as d2mhe_sync does)
    if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) return fail_cuda(c, e);
    u32 flag = 0;
    if ((e = cudaMemcpy(&flag, c->view.range_flag, sizeof(u32), cudaMemcpyDeviceToHost)) != cudaSuccess)
      return fail_cuda(c, e);
    if (flag) {
      if ((e = cudaMemset(c->view.range_flag, 0, sizeof(u32))) != cudaSuccess) return fail_cuda(c, e);
      return D2MHE_ERR_RANGE;
    }
  }
  return D2MHE_OK;
}

d2mhe_status d2mhe_round_device(d2mhe_ctx* c, const int32_t* values_dev, u32 ct_first, u32 n_cts,
                                const u32* nbr_offsets, const u32* nbr_rows, int32_t* sums_dev,
                                void* workspace_dev, size_t workspace_bytes) {
  return round_impl(c, values_dev, false, ct_first, n_cts, nbr_offsets, nbr_rows, sums_dev,
                    workspace_dev, workspace_bytes);
}
d2mhe_status d2mhe_round_host(d2mhe_ctx* c, const int32_t* values_host, u32 ct_first, u32 n_cts,
                              const u32* nbr_offsets, const u32* nbr_rows, int32_t* sums_host,
                              void* workspace_dev, size_t workspace_bytes) {
  return round_impl(c, values_host, true, ct_first, n_cts, nbr_offsets, nbr_rows, sums_host,
                    workspace_dev, workspace_bytes);
}

// ---- test hooks ----------------------------------------------------------------------

// What the device holds for a key, read back: the stored rows go through an inverse transform on the
// GPU (one CTA per limb) and every limb must give the same polynomial with coefficients in {-1, 0, 1}.
// Allocates a temporary device buffer and synchronises: a test hook, not a hot call.
static d2mhe_status export_key(d2mhe_ctx* c, const u64* key_dev, int8_t* s_host) {
  DeviceGuard guard(c->device);
  const size_t n = c->view.n, L = c->view.L;
  signed char* tmp = nullptr;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&tmp), L * n);
  if (e != cudaSuccess) return fail_cuda(c, e);
  std::vector<signed char> host(L * n);
  e = L_(export_secret)(c->view, c->limb_params, c->stream, key_dev, tmp);
  if (e == cudaSuccess) {
    c->launches += 1;
    e = cudaMemcpyAsync(host.data(), tmp, L * n, cudaMemcpyDeviceToHost, c->stream);
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  cudaFree(tmp);
  if (e != cudaSuccess) return fail_cuda(c, e);
  for (size_t j = 0; j < n; ++j) {
    const signed char v0 = host[j];
    if (v0 == 127) return D2MHE_ERR_DEVICE_CHECK;
    for (size_t l = 1; l < L; ++l)
      if (host[l * n + j] != v0) return D2MHE_ERR_DEVICE_CHECK;
    s_host[j] = (int8_t)v0;
  }
  return D2MHE_OK;
}

d2mhe_status d2mhe_debug_export_secret(d2mhe_ctx* c, u32 party, int8_t* s_host) {
  if (!c || !s_host) return D2MHE_ERR_INVALID_ARG;
  if (party >= c->params.num_parties) return D2MHE_ERR_RANGE;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_share[party]) return D2MHE_ERR_STATE;
  return export_key(c, c->view.s_mont + (size_t)party * c->view.L * c->view.n, s_host);
}

d2mhe_status d2mhe_debug_export_user_secret(d2mhe_ctx* c, u32 user, int8_t* s_host) {
  if (!c || !s_host) return D2MHE_ERR_INVALID_ARG;
  if (user >= c->params.num_parties) return D2MHE_ERR_RANGE;
  if (!protocol_ok(c)) return D2MHE_ERR_UNSUPPORTED;
  if (!c->has_user_key[user]) return D2MHE_ERR_STATE;
  return export_key(c, c->view.usk_mont + (size_t)user * c->view.L * c->view.n, s_host);
}

d2mhe_status d2mhe_debug_int_throughput(d2mhe_ctx* c, u32 kind, u32 iters, double* ops_per_second) {
  if (!c || !ops_per_second || kind > 6 || iters == 0 || iters > (1u << 24)) return D2MHE_ERR_INVALID_ARG;
  if (kind == 3 && !c->view.wide) return D2MHE_ERR_UNSUPPORTED;
  DeviceGuard guard(c->device);
  float ms = 0.f;
  double ops = 0.0;
  // the loops never store (their store is guarded by a condition that does not occur); the sink is
  // the context's scratch all the same
  cudaError_t e = L_(int_probe)(c->view, c->limb_params, c->stream, kind, iters,
                                reinterpret_cast<u32*>(c->noise_scratch), &ms, &ops);
  if (e != cudaSuccess) return fail_cuda(c, e);
  c->launches += 2;
  *ops_per_second = ms > 0.f ? ops / (ms * 1e-3) : 0.0;
  return D2MHE_OK;
}

d2mhe_status d2mhe_get_root(const d2mhe_ctx* c, u32 limb, uint64_t* psi) {
  if (!c || !psi) return D2MHE_ERR_INVALID_ARG;
  if (limb >= c->params.num_limbs) return D2MHE_ERR_RANGE;
  *psi = c->roots[limb];
  return D2MHE_OK;
}

d2mhe_status d2mhe_get_plain_root(const d2mhe_ctx* c, uint64_t* psi_t) {
  if (!c || !psi_t) return D2MHE_ERR_INVALID_ARG;
  if (!c->can_pack) return D2MHE_ERR_UNSUPPORTED;
  *psi_t = c->psi_t;
  return D2MHE_OK;
}

uint64_t d2mhe_launch_count(const d2mhe_ctx* c) { return c ? c->launches : 0; }

size_t d2mhe_sample_scratch_bytes(const d2mhe_ctx* c) { return c ? c->noise_scratch_bytes : 0; }

}  // extern "C"
