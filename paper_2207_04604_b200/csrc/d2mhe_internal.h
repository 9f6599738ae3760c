// Host-side view of the context and the kernel launch entry points.
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

#include "d2mhe_device.cuh"

#define D2MHE_MAX_LIMBS 24
#define D2MHE_MAX_SMEM_LOGN 14  // largest polynomial that fits one CTA's shared memory

// Constants for the plaintext-modulus transforms (32-bit arithmetic).
struct PlainTab {
  u32 t, twot;
  u32 ninv, ninv_sh;   // N^-1 mod t with 32-bit Shoup companion
  u32 half;            // (t-1)/2
  const uint2* W;      // [N] psi_t^brv(i) as {w, floor(w 2^32 / t)}
  const uint2* IW;     // [N] inverses
};

// Constants of the exact scale-and-round (mixed-radix conversion).
struct RoundTab {
  const ulonglong2* ginv;  // [L*L]: entry i*L+j (j < i) = q_j^-1 mod q_i with Shoup companion
  const u64* prefix_mod_t; // [L]: prod_{j<i} q_j mod t
  u64 t, t_sh;             // t and floor(2^64 / t)
  u64 half_mod_t;          // (q-1)/2 mod t
  u64 qinv_mod_t;          // q^-1 mod t
};

// The per-limb constants travel as a kernel parameter (constant bank): indexed by the
// CTA-uniform limb number they are read through the uniform datapath instead of occupying
// vector registers in every thread.
struct LimbParams {
  LimbTab limbs[D2MHE_MAX_LIMBS];
};

// Everything a kernel needs, passed by value.
struct DevView {
  const LimbTab* limbs;
  const GaussTab* gauss;
  PlainTab plain;
  RoundTab round;
  u64 seed;
  u32 logn, n, L, K;
  u32 sms;       // multiprocessors of the device (launch shaping only)
  u32 wide;      // 1 if every q_l < 2^56: lazy-reduction policy with no conditional subtractions
  u64* s_mont;   // [K][L][N]  NTT(s_k) * N^-1 in Montgomery form
  u64* pk_mont;  // [2][L][N]  NTT(p_0), NTT(p_1) * N^-1 in Montgomery form
  u64* pk_coef;  // [2][L][N]  (p_0, p_1), coefficient domain
  u64* usk_mont;  // [K][L][N]     NTT(sk_i) * N^-1 (Montgomery form) of the users' own keys
  u64* upk_mont;  // [K][2][L][N]  NTT(p_{0,i}), NTT(p_{1,i}) * N^-1 (Montgomery form)
  u64* upk_coef;  // [K][2][L][N]  pk_i, coefficient domain
  // only when every prime is below 2^30 (the 32-bit-word protocol calls): the same keys as words
  // {residue out of Montgomery form, its 32-bit Shoup companion}
  u64* s32;       // [K][L][N]
  u64* pk32;      // [2][L][N]
  u32* range_flag;
  u32* chk;       // four check words {site, index, limit, block} of the checked build
};

// ---- host-side context (shared by the translation units that implement the C ABI) ----
#include <vector>

#include "../../include/d2mhe.h"

static const size_t kIdxSlotWords = (size_t)1 << 21;  // u32 words per staging slot (8 MiB)
static const int kIdxSlots = 4;
// Sample scratch of a context (for the single calls): 64 MiB, or what two waves of thread blocks of
// the share kernel with the largest samples (MBFV.Bootstrap: 6 N bytes per share) need, up to 512 MiB.
static const size_t kNoiseScratchBytes = (size_t)64 << 20;
static const size_t kNoiseScratchMaxBytes = (size_t)512 << 20;
#ifndef D2MHE_ROUND_LANES
#define D2MHE_ROUND_LANES 2
#endif
#ifndef D2MHE_ROUND_LANES_HOST
#define D2MHE_ROUND_LANES_HOST 3
#endif
// Internal streams of the whole-round entry points: two for device buffers (measured best at
// configuration 2: 0.89 ms against 0.91 ms with three), three when the call also copies from and to
// host buffers (1.02 ms against 1.04 ms with two: one more stream hides the copies better).
static const int kRoundLanesDevice = D2MHE_ROUND_LANES;
static const int kRoundLanesHost = D2MHE_ROUND_LANES_HOST;
static const int kRoundLanes = kRoundLanesDevice > kRoundLanesHost ? kRoundLanesDevice : kRoundLanesHost;

struct d2mhe_ctx {
  d2mhe_params params;
  std::vector<u64> moduli;
  std::vector<u64> roots;
  u64 psi_t = 0;
  bool can_pack = false;
  bool narrow = false;  // every prime below 2^30: the 32-bit-word calls are available
  int device = 0;
  cudaStream_t stream = nullptr;
  DevView view;
  LimbParams limb_params;
  std::vector<void*> allocs;        // device allocations to free
  std::vector<bool> has_share;
  std::vector<bool> has_user_key;
  std::vector<u32> pk_parties;      // party set of the last collective_pk
  std::vector<u32> all_parties;     // 0 .. K-1 (the users of a whole-round call)
  bool has_pk = false;
  u64 launches = 0;
  // index staging: pinned host ring + device ring, one event per slot
  u32* idx_host = nullptr;
  u32* idx_dev = nullptr;
  cudaEvent_t idx_event[kIdxSlots] = {};
  bool idx_event_valid[kIdxSlots] = {};
  int idx_next = 0;
  // the four index lists of the whole-round calls: kept on the device from one call to the next and
  // uploaded again only when they change
  u32* round_lists_host = nullptr;        // pinned
  u32* round_lists_dev = nullptr;
  std::vector<u32> round_lists_cache;     // what round_lists_dev holds
  cudaEvent_t round_lists_event = nullptr;  // after the last upload
  bool round_lists_valid = false;
  cudaStream_t lane_stream[kRoundLanes] = {};
  cudaEvent_t lane_event[kRoundLanes] = {};
  cudaEvent_t fork_event = nullptr;
  unsigned char* noise_scratch = nullptr;  // device: noise bytes of the shares of one d2mhe_partial_decrypt batch
  size_t noise_scratch_bytes = 0;
  cudaError_t last_cuda = cudaSuccess;
  bool checked = false;             // launches the checked kernel build
  u32 last_check[4] = {};           // the last violation that d2mhe_sync reported
};

// The kernel translation units are compiled twice: as they are into namespace d2mhe_launch, and
// with D2MHE_CHECKED (index checks in every kernel, see d2mhe_device.cuh) into d2mhe_launch_chk.
// A context created with D2MHE_FLAG_DEVICE_CHECKS launches the second set.
#ifdef D2MHE_CHECKED
#define D2MHE_LAUNCH_NS d2mhe_launch_chk
#else
#define D2MHE_LAUNCH_NS d2mhe_launch
#endif

// Launchers (one per kernel or kernel sequence).  Notes: encrypt and partial_decrypt_scratch sample
// u, e_0, e_1 / the shares' noise ahead into caller-lent scratch (at least 3 N / n_parties N bytes)
// and report their number of launches, and so do convert_share (n_parties 3 N bytes) and boot_share
// (n_parties 6 N bytes); combine sums the first of share_comps polynomials per
// (recipient, party, ciphertext); int_probe synchronises the stream; export_secret turns key rows
// [L][N] (transform domain, Montgomery form) into int8 coefficients [L][N] (127 = not ternary);
// check_selftest makes one thread of the checked build raise SITE_SELFTEST (no memory access).
#define D2MHE_LAUNCHER_DECLS \
cudaError_t keygen(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties); \
cudaError_t collective_pk(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties, \
                          u64* shares_out); \
cudaError_t int_probe(const DevView& v, const LimbParams& lp, cudaStream_t s, u32 kind, u32 iters, u32* sink, \
                      float* ms, double* lane_ops); \
cudaError_t export_secret(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* key, signed char* out); \
cudaError_t encode(const DevView& v, cudaStream_t s, const int32_t* values, u32 n_cts, u32* plain); \
cudaError_t decode(const DevView& v, cudaStream_t s, const u32* plain, u32 n_cts, int32_t* values); \
cudaError_t encode_strided(const DevView& v, cudaStream_t s, const int32_t* values, u32 n_groups, u32 group, \
                           size_t group_stride, u32* plain); \
cudaError_t decode_strided(const DevView& v, cudaStream_t s, const u32* plain, u32 n_groups, u32 group, \
                           size_t group_stride, int32_t* values); \
cudaError_t encrypt(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties, \
                    u32 ct_first, u32 n_cts, const u32* plain, u64* ct, void* scratch, size_t scratch_bytes, \
                    u32* launches); \
cudaError_t aggregate(const DevView& v, cudaStream_t s, const u64* ct, u32 n_cts, \
                      const u32* offsets_dev, const u32* rows_dev, u32 n_out, u64* agg); \
cudaError_t partial_decrypt_scratch(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg, \
                                    const u32* recipients_dev, u32 n_rec, const u32* parties_dev, \
                                    u32 n_parties, u32 ct_first, u32 n_cts, u64* shares, void* scratch, \
                                    size_t scratch_bytes, u32* launches); \
cudaError_t combine(const DevView& v, cudaStream_t s, const u64* agg, const u64* shares, u32 n_rec, \
                    u32 n_shares, u32 share_comps, u32 n_cts, u32* plain); \
cudaError_t boot_share(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg, \
                       const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties, \
                       u32 ct_first, u32 n_cts, u64* shares, void* scratch, size_t scratch_bytes, u32* launches); \
cudaError_t boot_finish(const DevView& v, cudaStream_t s, const u32* x, const u64* shares, \
                        const u32* recipients_dev, u32 n_rec, u32 n_shares, u32 ct_first, u32 n_cts, u64* out); \
cudaError_t ntt(const DevView& v, const LimbParams& lp, cudaStream_t s, u64* polys, u32 batch, bool inverse); \
cudaError_t ntt32(const DevView& v, const LimbParams& lp, cudaStream_t s, u32* polys, u32 batch, bool inverse); \
cudaError_t muladd32(const DevView& v, cudaStream_t s, const u32* a, const u32* b, const u32* c, u32* d, \
                     u32 batch); \
cudaError_t user_keygen(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* users_dev, \
                        u32 n_users); \
cudaError_t convert_share(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* agg, \
                          const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties, \
                          u32 ct_first, u32 n_cts, u64* shares, void* scratch, size_t scratch_bytes, u32* launches); \
cudaError_t convert_combine(const DevView& v, cudaStream_t s, const u64* agg, const u64* shares, u32 n_rec, \
                            u32 n_shares, u32 n_cts, u64* out); \
cudaError_t secret_product(const DevView& v, const LimbParams& lp, cudaStream_t s, const u64* ct, \
                           const u32* users_dev, u32 n_users, u32 n_cts, u64* prod); \
cudaError_t muladd(const DevView& v, cudaStream_t s, const u64* a, const u64* b, const u64* c, \
                   u64* d, u32 batch); \
cudaError_t check_selftest(const DevView& v, cudaStream_t s); \
cudaError_t sample_encrypt_noise(const DevView& v, cudaStream_t s, const u32* parties_dev, u32 ct_first, u32 n_cts, \
                                 u32 unit_first, u32 n_units, u32* out); \
cudaError_t sample_share_noise(const DevView& v, cudaStream_t s, const u32* recipients_dev, const u32* parties_dev, \
                               u32 n_parties, u32 ct_first, u32 n_cts, u32 unit_first, u32 n_units, u32* out); \
cudaError_t make_tab32(const DevView& v, cudaStream_t s, const u64* src, u64* dst, size_t rows); \
cudaError_t encrypt32(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* parties_dev, u32 n_parties, \
                      u32 ct_first, u32 n_cts, const u32* plain, u32* ct, void* scratch, size_t scratch_bytes, \
                      u32* launches); \
cudaError_t aggregate32(const DevView& v, cudaStream_t s, const u32* ct, u32 n_cts, const u32* offsets_dev, \
                        const u32* rows_dev, u32 n_out, u32* agg); \
cudaError_t partial_decrypt32(const DevView& v, const LimbParams& lp, cudaStream_t s, const u32* agg, \
                              const u32* recipients_dev, u32 n_rec, const u32* parties_dev, u32 n_parties, \
                              u32 ct_first, u32 n_cts, u32* shares, void* scratch, size_t scratch_bytes, \
                              u32* launches); \
cudaError_t combine32(const DevView& v, cudaStream_t s, const u32* agg, const u32* shares, u32 n_rec, u32 n_shares, \
                      u32 n_cts, u32* plain);

namespace d2mhe_launch {
D2MHE_LAUNCHER_DECLS
}
namespace d2mhe_launch_chk {
D2MHE_LAUNCHER_DECLS
}

