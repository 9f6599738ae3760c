/*
 * d2mhe.h - C ABI of the B200 (sm_100a) library for the private gradient update
 * of D2-MHE: multiparty BFV over R_q = Z_q[X]/(X^N+1) in residue-number-system
 * form, every party simulated as a batch dimension on one GPU.
 *
 * Citations name the passage of the paper (arXiv 2207.04604) that defines the
 * operation: "Sec. 3.2 item k" is the k-th algorithm of the BFV summary,
 * "Sec. 4.2 item k" the k-th multiparty function, "Algorithm 2" the
 * privacy-preserving D-PSGD loop.
 *
 * Conventions
 *  - Polynomials are row-major uint64 arrays [..., L, N] (N contiguous), limb l
 *    holding the residues mod q_l in [0, q_l), in the COEFFICIENT domain.
 *  - Unless a parameter says "host", every data pointer is a DEVICE pointer,
 *    16-byte aligned, sized exactly as annotated, owned by the caller.
 *  - Hot calls are asynchronous on the context's stream and allocate nothing.  Calls that take
 *    HOST index lists (parties, recipients, neighbour lists) copy them through a ring of four
 *    pinned staging slots; a call waits on the host only when all four slots belong to calls whose
 *    work on the GPU has not finished yet, i.e. from the fifth such call in flight.  The library
 *    allocates only in d2mhe_create (and in the test hooks).
 *  - Every function returns a d2mhe_status (0 = success, < 0 = error) and
 *    never aborts.  Arguments visible on the host are validated before any
 *    launch; a failed validation launches nothing.  Asynchronous CUDA errors
 *    and the device range flag are reported by d2mhe_sync.
 *  - One context per host thread.  Randomness is counter based
 *    (Philox4x32-10 keyed by `seed`), so every output is a deterministic
 *    function of (params, seed, inputs, stream indices).
 */
#ifndef D2MHE_H
#define D2MHE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct d2mhe_ctx d2mhe_ctx; /* opaque: tables, secret shares, collective key */
typedef int32_t d2mhe_status;

enum {
  D2MHE_OK = 0,
  D2MHE_ERR_INVALID_ARG = -1, /* NULL / misaligned pointer, zero count, bad struct_size */
  D2MHE_ERR_BAD_PARAMS = -2,  /* moduli not prime / not 1 mod 2N / repeated / too wide  */
  D2MHE_ERR_STATE = -3,       /* call order: keygen -> collective_pk -> encrypt ...      */
  D2MHE_ERR_WORKSPACE = -4,   /* caller-provided workspace too small                     */
  D2MHE_ERR_CUDA = -5,        /* a CUDA runtime call failed                              */
  D2MHE_ERR_RANGE = -6,       /* index out of range, or a value outside (-t/2, t/2)      */
  D2MHE_ERR_UNSUPPORTED = -7, /* operation not available for these parameters            */
  D2MHE_ERR_DEVICE_CHECK = -8 /* a check that runs on the device failed (see `flags`)    */
};

/* d2mhe_params.flags: run this context on the checked build of every kernel.  Each kernel then
 * tests the indices it is about to use (coefficient and octet numbers, shared-memory offsets,
 * twiddle indices, party numbers read from the index lists) against their limits; the first
 * violation is recorded in a device word and the access is skipped (no trap: the context stays
 * usable).  d2mhe_sync returns D2MHE_ERR_DEVICE_CHECK once for it.  Results are the same as
 * without the flag; the kernels are a few per cent slower. */
#define D2MHE_FLAG_DEVICE_CHECKS 1u

typedef struct {
  uint32_t struct_size;   /* = sizeof(d2mhe_params)                                      */
  uint32_t log2_n;        /* ring degree N = 2^log2_n, 3 <= log2_n <= 16.  The protocol
                             calls need log2_n <= 14; 15 and 16 serve the transform and
                             multiply-add entry points only.                            */
  uint32_t num_limbs;     /* L, 1..24                                                    */
  uint32_t num_parties;   /* K, 1..65535                                                 */
  const uint64_t* moduli; /* HOST array of L distinct primes, q_l = 1 mod 2N, q_l < 2^61 */
  uint64_t plain_modulus; /* t: prime < 2^30, coprime to every q_l.  Packing
                             (encode/decode) additionally needs t = 1 mod 2N.            */
  uint64_t seed;          /* Philox key                                                  */
  uint32_t gauss_bound;   /* B of the error distribution; must be 19 (sigma = 3.2)       */
  uint32_t flags;         /* 0, or D2MHE_FLAG_DEVICE_CHECKS; other bits must be 0        */
  int32_t device;         /* CUDA device ordinal                                         */
} d2mhe_params;

/* Validates params, builds all tables on `device` and allocates the context's device memory (tables,
 * key storage, index staging, and the scratch for the samples that d2mhe_encrypt,
 * d2mhe_partial_decrypt, d2mhe_convert_share and d2mhe_bootstrap_share draw ahead of their kernels:
 * 64 MiB, or what two waves of thread blocks of the share kernels need for this parameter set, at
 * most 512 MiB; d2mhe_sample_scratch_bytes reports it).  *out is NULL on failure. */
d2mhe_status d2mhe_create(const d2mhe_params* params, d2mhe_ctx** out);
void d2mhe_destroy(d2mhe_ctx* ctx);
/* Stream (a cudaStream_t passed as void*) on which later calls are enqueued; NULL = default. */
d2mhe_status d2mhe_set_stream(d2mhe_ctx* ctx, void* cuda_stream);
/* Waits for the stream; returns the first asynchronous error, D2MHE_ERR_DEVICE_CHECK if a kernel of
 * a context created with D2MHE_FLAG_DEVICE_CHECKS recorded an index violation since the last sync,
 * or D2MHE_ERR_RANGE if d2mhe_encode saw a value outside [-(t-1)/2, (t-1)/2] since the last sync
 * (either record is cleared by the call that reports it). */
d2mhe_status d2mhe_sync(d2mhe_ctx* ctx);
const char* d2mhe_strerror(d2mhe_status status);

/*
 * MBFV.SecKeyGen (Sec. 4.2 item 1; BFV.SecKeyGen, Sec. 3.2 item 1): each listed
 * party k draws s_k uniformly from R_3 (coefficients in {-1,0,1}).  The shares stay
 * inside the context (transform domain); s = sum s_k is never formed.
 * parties: HOST array of n_parties distinct indices < K.
 */
d2mhe_status d2mhe_keygen_share(d2mhe_ctx* ctx, const uint32_t* parties, uint32_t n_parties);

/*
 * MBFV.PubKeyGen (Sec. 4.2 item 2): common p_1 uniform on R_q; each listed party
 * samples e_k from chi and forms p_{0,k} = -(p_1 s_k + e_k); pk = ([sum_k p_{0,k}]_q, p_1).
 * All listed parties must have key shares.  The party set of the last call is the set
 * of share holders that d2mhe_combine_decrypt expects.
 * pk_shares_dev: optional out [n_parties, L, N] (may be NULL).
 * pk_dev:        optional out [2, L, N] = (p_0, p_1) (may be NULL).
 */
d2mhe_status d2mhe_collective_pk(d2mhe_ctx* ctx, const uint32_t* parties, uint32_t n_parties,
                                 uint64_t* pk_shares_dev, uint64_t* pk_dev);

/*
 * Packing (Sec. 6, SIMD slots): values int32 [n_cts, N] (caller zero-pads), each in
 * [-(t-1)/2, (t-1)/2] -> plaintext polynomials uint32 [n_cts, N] in [0,t) with
 * m(psi_t^(2j+1)) = value_j mod t, psi_t = g^((t-1)/2N) for the smallest primitive
 * root g of t.  d2mhe_decode is the inverse, returning centred values.
 * In-place use (values == plain storage) is allowed.
 */
d2mhe_status d2mhe_encode(d2mhe_ctx* ctx, const int32_t* values_dev, uint32_t n_cts,
                          uint32_t* plain_dev);
d2mhe_status d2mhe_decode(d2mhe_ctx* ctx, const uint32_t* plain_dev, uint32_t n_cts,
                          int32_t* values_dev);

/*
 * BFV.Encrypt under the collective key (Sec. 3.2 item 3; the encryption steps of Algorithm 2):
 * ct = (Lambda m + u p_0 + e_0, u p_1 + e_1), Lambda = floor(q/t), u from R_3,
 * e_0, e_1 from chi.  The randomness of unit (parties[a], c) is the stream
 * (party = parties[a], ciphertext index = ct_first + c).
 * plain_dev: [n_parties, n_cts, N] uint32 in [0,t);  ct_dev: out [n_parties, n_cts, 2, L, N].
 */
d2mhe_status d2mhe_encrypt(d2mhe_ctx* ctx, const uint32_t* parties, uint32_t n_parties,
                           uint32_t ct_first, uint32_t n_cts, const uint32_t* plain_dev,
                           uint64_t* ct_dev);

/*
 * BFV.Add over neighbour lists (Sec. 3.2 item 4; the neighbour-sum step of Algorithm 2, with unit weights):
 * agg[i, c] = sum_{r in list(i)} ct[r, c] mod q, both components.
 * ct_dev: [n_rows, n_cts, 2, L, N].  nbr_offsets (HOST, n_out+1 entries, non-decreasing,
 * nbr_offsets[0] = 0) and nbr_rows (HOST, nbr_offsets[n_out] entries, each < n_rows) are
 * the lists in CSR form; they are validated on the host.  An empty list gives zero.
 * agg_dev: out [n_out, n_cts, 2, L, N]; must not overlap ct_dev.
 * Limits: n_out <= 65536 and nbr_offsets[n_out] <= 1048576.
 */
d2mhe_status d2mhe_aggregate(d2mhe_ctx* ctx, const uint64_t* ct_dev, uint32_t n_rows,
                             uint32_t n_cts, const uint32_t* nbr_offsets,
                             const uint32_t* nbr_rows, uint32_t n_out, uint64_t* agg_dev);

/*
 * Decryption shares (Sec. 4.2 item 3, Eq. 2 with mu_k = 0; equally Eq. 4 with M_k = 0):
 * shares[i, a, c] = s_k c_1 + e, k = parties[a], c_1 the second component of agg[i, c],
 * e from chi on the stream (party k, recipient recipients[i], ciphertext index ct_first + c).
 * agg_dev: [n_rec, n_cts, 2, L, N];  shares_dev: out [n_rec, n_parties, n_cts, L, N].
 * recipients, parties: HOST arrays of indices < K.
 * The noise of the shares is sampled by a kernel of its own into the scratch buffer that the
 * context owns (one byte per share coefficient; as many (recipient, ciphertext) pairs per launch as
 * fit, rounded down to whole waves of thread blocks), so the call is one or more pairs of launches
 * on the context's stream.
 * D2MHE_ERR_UNSUPPORTED if n_parties * N exceeds that buffer (d2mhe_convert_share and
 * d2mhe_bootstrap_share work the same way with 3 and 6 bytes per share coefficient).
 */
d2mhe_status d2mhe_partial_decrypt(d2mhe_ctx* ctx, const uint64_t* agg_dev,
                                   const uint32_t* recipients, uint32_t n_rec,
                                   const uint32_t* parties, uint32_t n_parties,
                                   uint32_t ct_first, uint32_t n_cts, uint64_t* shares_dev);

/*
 * Combine and decrypt (Sec. 4.2 item 3: c_0 + sum_k h_k; Sec. 3.2 item 5:
 * x = [ round(t/q [.]_q) ]_t, computed exactly in RNS by a mixed-radix conversion).
 * n_shares must equal the size of the party set of the last d2mhe_collective_pk.
 * agg_dev: [n_rec, n_cts, 2, L, N] (only c_0 is read);
 * shares_dev: [n_rec, n_shares, n_cts, L, N];  plain_dev: out [n_rec, n_cts, N] in [0,t).
 */
d2mhe_status d2mhe_combine_decrypt(d2mhe_ctx* ctx, const uint64_t* agg_dev,
                                   const uint64_t* shares_dev, uint32_t n_rec,
                                   uint32_t n_shares, uint32_t n_cts, uint32_t* plain_dev);

/*
 * MBFV.Convert (Sec. 4.2 item 3, Eq. 2-3; the decryption steps of Algorithm 2): re-encryption of an aggregate
 * from the collective key to the recipient's OWN key pair, followed by BFV.Decrypt under it.
 *
 * d2mhe_user_keygen: every listed user i generates sk_i <- R_3 and
 *   pk_i = (-(sk_i p_{1,i} + e_i), p_{1,i}), p_{1,i} uniform, e_i from chi (Algorithm 2, Require;
 *   Sec. 3.2 items 1-2).  pk_out_dev: optional out [n_users, 2, L, N].
 * d2mhe_convert_share: shares[i, a, c] = (h_0, h_1) =
 *   (s_k c_1 + mu_k p_{0,i} + e_{0,k},  mu_k p_{1,i} + e_{1,k}),  k = parties[a], i = recipients[i],
 *   mu_k, e_{0,k}, e_{1,k} from chi (the paper draws mu_k from chi) on the stream
 *   (party k, recipient i, ciphertext index ct_first + c).  Recipients need own keys, parties key shares.
 *   agg_dev: [n_rec, n_cts, 2, L, N];  shares_dev: out [n_rec, n_parties, n_cts, 2, L, N].
 * d2mhe_convert_combine: ct'[i, c] = (c_0 + sum_k h_{0,k}, sum_k h_{1,k}); n_shares must equal the
 *   size of the collective key's party set.  ct_out_dev: out [n_rec, n_cts, 2, L, N].
 * d2mhe_decrypt: BFV.Decrypt(sk_i, ct) (Sec. 3.2 item 5) for users[i] on ct_dev [n_users, n_cts, 2, L, N];
 *   scratch_dev: caller-provided [n_users, n_cts, L, N] uint64 (receives c_1 sk_i);
 *   plain_dev: out [n_users, n_cts, N] in [0,t).
 * users, recipients, parties: HOST arrays.
 */
d2mhe_status d2mhe_user_keygen(d2mhe_ctx* ctx, const uint32_t* users, uint32_t n_users,
                               uint64_t* pk_out_dev);
d2mhe_status d2mhe_convert_share(d2mhe_ctx* ctx, const uint64_t* agg_dev, const uint32_t* recipients,
                                 uint32_t n_rec, const uint32_t* parties, uint32_t n_parties,
                                 uint32_t ct_first, uint32_t n_cts, uint64_t* shares_dev);
d2mhe_status d2mhe_convert_combine(d2mhe_ctx* ctx, const uint64_t* agg_dev, const uint64_t* shares_dev,
                                   uint32_t n_rec, uint32_t n_shares, uint32_t n_cts,
                                   uint64_t* ct_out_dev);
d2mhe_status d2mhe_decrypt(d2mhe_ctx* ctx, const uint32_t* users, uint32_t n_users,
                           const uint64_t* ct_dev, uint32_t n_cts, uint64_t* scratch_dev,
                           uint32_t* plain_dev);

/*
 * MBFV.Bootstrap (Sec. 4.2 item 4, Eq. 4): collective noise refresh of agg[i, c].
 * d2mhe_bootstrap_share: shares[i, a, c] = (eta_0, eta_1) =
 *   (s_k c_1 - Lambda M_k + e_{0,k},  -s_k alpha + Lambda M_k + e_{1,k}),  k = parties[a],
 *   M_k uniform over R_t, e_{0,k}, e_{1,k} from chi on the stream (party k, recipient, ciphertext
 *   index ct_first + c); alpha is the common polynomial, uniform on R_q, derived from
 *   (recipient, ciphertext index).  shares_dev: out [n_rec, n_parties, n_cts, 2, L, N].
 * d2mhe_bootstrap_combine: ct'[i, c] = ([round(t/q [c_0 + sum_k eta_{0,k}]_q)]_t Lambda + sum_k eta_{1,k}, alpha).
 *   n_shares must equal the size of the collective key's party set; recipients and ct_first as in
 *   the share call (they select alpha).  plain_scratch_dev: caller-provided uint32 [n_rec, n_cts, N]
 *   (receives the masked plaintext); ct_out_dev: out [n_rec, n_cts, 2, L, N].
 */
d2mhe_status d2mhe_bootstrap_share(d2mhe_ctx* ctx, const uint64_t* agg_dev, const uint32_t* recipients,
                                   uint32_t n_rec, const uint32_t* parties, uint32_t n_parties,
                                   uint32_t ct_first, uint32_t n_cts, uint64_t* shares_dev);
d2mhe_status d2mhe_bootstrap_combine(d2mhe_ctx* ctx, const uint64_t* agg_dev, const uint64_t* shares_dev,
                                     const uint32_t* recipients, uint32_t n_rec, uint32_t n_shares,
                                     uint32_t ct_first, uint32_t n_cts, uint32_t* plain_scratch_dev,
                                     uint64_t* ct_out_dev);

/*
 * Batched negacyclic number-theoretic transform of [batch, L, N], in place.
 * Forward: position p of limb l receives a(psi_l^(2 brv(p) + 1)), brv = reversal of
 * the log2_n-bit index, psi_l the root reported by d2mhe_get_root.  Inverse undoes it.
 * N <= 16384 runs as one kernel with the polynomial in shared memory; N = 32768, 65536 run
 * as two passes (the first 3 or 4 stages in registers, then 4096-point blocks).
 * These are the ring isomorphism behind every product of Sec. 3.2 / 4.2.
 */
d2mhe_status d2mhe_ntt_forward(d2mhe_ctx* ctx, uint64_t* polys_dev, uint32_t batch);
d2mhe_status d2mhe_ntt_inverse(d2mhe_ctx* ctx, uint64_t* polys_dev, uint32_t batch);
/* d = a (.) b + c residue by residue on [batch, L, N] (the RNS multiply-add inside
 * u p_0 + e_0 and s_k c_1 + e_k).  d may alias a, b or c. */
d2mhe_status d2mhe_poly_muladd(d2mhe_ctx* ctx, const uint64_t* a_dev, const uint64_t* b_dev,
                               const uint64_t* c_dev, uint64_t* d_dev, uint32_t batch);

/*
 * The same three operations on 32-bit words, for parameter sets whose primes are all below
 * 2^30 (D2MHE_ERR_UNSUPPORTED otherwise): polynomials are uint32 [batch, L, N], residues in
 * [0, q_l).  Half the bytes and less than a third of the multiplier work of the 64-bit calls per
 * coefficient; a ciphertext modulus of the same size needs about twice the limbs.  The
 * transforms need log2_n <= 14 (two polynomials of the batch share one thread block and
 * shared memory); results are defined exactly as for the 64-bit calls.
 */
d2mhe_status d2mhe_ntt32_forward(d2mhe_ctx* ctx, uint32_t* polys_dev, uint32_t batch);
d2mhe_status d2mhe_ntt32_inverse(d2mhe_ctx* ctx, uint32_t* polys_dev, uint32_t batch);
d2mhe_status d2mhe_poly_muladd32(d2mhe_ctx* ctx, const uint32_t* a_dev, const uint32_t* b_dev,
                                 const uint32_t* c_dev, uint32_t* d_dev, uint32_t batch);

/*
 * The protocol calls on 32-bit words, for the same parameter sets (every prime below 2^30,
 * log2_n <= 14; D2MHE_ERR_UNSUPPORTED otherwise): ciphertexts, neighbour sums and decryption shares
 * are uint32 arrays of the shapes given above, residues in [0, q_l).  Keys come from
 * d2mhe_keygen_share and d2mhe_collective_pk as before; plaintexts from d2mhe_encode and to
 * d2mhe_decode.  Streams, samples and every result equal those of the 64-bit calls on the same
 * context (BFV.Encrypt, Sec. 3.2 item 3; BFV.Add, item 4; decryption shares and their combination,
 * Sec. 4.2 item 3 and Sec. 3.2 item 5).  Two units share a thread block, so even counts of
 * (party, ciphertext) and (recipient, ciphertext) pairs use the GPU best.
 */
d2mhe_status d2mhe_encrypt32(d2mhe_ctx* ctx, const uint32_t* parties, uint32_t n_parties,
                             uint32_t ct_first, uint32_t n_cts, const uint32_t* plain_dev,
                             uint32_t* ct_dev);
d2mhe_status d2mhe_aggregate32(d2mhe_ctx* ctx, const uint32_t* ct_dev, uint32_t n_rows, uint32_t n_cts,
                               const uint32_t* nbr_offsets, const uint32_t* nbr_rows, uint32_t n_out,
                               uint32_t* agg_dev);
d2mhe_status d2mhe_partial_decrypt32(d2mhe_ctx* ctx, const uint32_t* agg_dev, const uint32_t* recipients,
                                     uint32_t n_rec, const uint32_t* parties, uint32_t n_parties,
                                     uint32_t ct_first, uint32_t n_cts, uint32_t* shares_dev);
d2mhe_status d2mhe_combine_decrypt32(d2mhe_ctx* ctx, const uint32_t* agg_dev, const uint32_t* shares_dev,
                                     uint32_t n_rec, uint32_t n_shares, uint32_t n_cts,
                                     uint32_t* plain_dev);

/*
 * One whole private gradient update for ciphertext indices ct_first .. ct_first+n_cts-1
 * of all K parties (Algorithm 2 from encryption to decryption, without the model update): encode,
 * encrypt, neighbour sums, shares from every share holder, combine, decode.  Ciphertext
 * indices are processed in sub-chunks so that all protocol messages of the sub-chunks in
 * flight (ciphertexts, aggregates, shares, and one noise byte per share coefficient) live in
 * the caller's workspace.  Up to two sub-chunks (three for d2mhe_round_host) are in flight
 * at a time on internal streams, so that one sub-chunk's copies
 * and memory-bound kernels overlap another's arithmetic; the internal streams start after
 * the work already queued on the context's stream, and the context's stream continues
 * after they have finished (so the call behaves like one operation on that stream).
 *   values:  int32 [K, n_cts, N]   in (d2mhe_round_device reads it in place, sub-chunk by sub-chunk)
 *   sums:    int32 [K, n_cts, N]   out: sums[i] = sum over list(i) of the values (written in place)
 *   nbr_offsets / nbr_rows: HOST CSR lists over parties, K lists.
 *   workspace_dev / workspace_bytes: device scratch, at least
 *   d2mhe_round_workspace_bytes(ctx, 1); d2mhe_round_workspace_bytes(ctx, n_cts) holds
 *   the whole range at once (the fastest choice when it fits); anything in between makes
 *   more, smaller sub-chunks.  The contents left in the workspace are unspecified.
 * d2mhe_round_device takes device values/sums.  d2mhe_round_host takes HOST values/sums
 * (pinned memory recommended), copies each sub-chunk in and out on the stream that
 * computes it and returns after all of it has finished; it returns D2MHE_ERR_RANGE (sums then
 * unspecified) if a value was outside [-(t-1)/2, (t-1)/2].  If a launch or copy fails part-way,
 * the internal streams are still joined back into the context's stream before the call returns.
 */
size_t d2mhe_round_workspace_bytes(const d2mhe_ctx* ctx, uint32_t chunk_cts);
/*
 * Host-only (touches no device): how d2mhe_round_device cuts n_cts ciphertext indices when its
 * workspace holds cap_cts of them.  Writes the sizes of the first max_out sub-chunks to sizes
 * (may be NULL) and the number of internal streams used to *lanes_out (may be NULL); returns the
 * number of sub-chunks, 0 for n_cts == 0 or cap_cts == 0.  Sub-chunk i runs on stream i mod
 * lanes; sizes differ by at most one, larger ones first; the sizes of the first `lanes`
 * sub-chunks add up to at most cap_cts.  Fewer than four indices run on one stream.
 * (d2mhe_round_host cuts by the same rule over three streams.)
 */
uint32_t d2mhe_round_plan(uint32_t n_cts, uint64_t cap_cts, uint32_t* sizes, uint32_t max_out,
                          uint32_t* lanes_out);
d2mhe_status d2mhe_round_device(d2mhe_ctx* ctx, const int32_t* values_dev, uint32_t ct_first,
                                uint32_t n_cts, const uint32_t* nbr_offsets,
                                const uint32_t* nbr_rows, int32_t* sums_dev,
                                void* workspace_dev, size_t workspace_bytes);
d2mhe_status d2mhe_round_host(d2mhe_ctx* ctx, const int32_t* values_host, uint32_t ct_first,
                              uint32_t n_cts, const uint32_t* nbr_offsets,
                              const uint32_t* nbr_rows, int32_t* sums_host,
                              void* workspace_dev, size_t workspace_bytes);

/*
 * The same round as d2mhe_round_device for callers that cannot allocate device memory
 * (the paper has no counterpart: this is a packaging variant, not a protocol step).
 * Think of a service that gave all device memory to a fixed pool at start-up, a plug-in
 * that receives only its input and output buffers, or a latency-critical loop in which
 * cudaMalloc is banned because it synchronises the device.  The chunk's protocol messages
 * live in a 64 MiB array that is part of the library image (a GPU reserves those 64 MiB when the
 * first call of this function on it loads that part of the image, and holds them until the process
 * exits); the caller passes only values and sums.
 *  - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - Returns D2MHE_ERR_WORKSPACE when one ciphertext index of this parameter set needs more
 *    than 64 MiB, i.e. when d2mhe_round_workspace_bytes(ctx, 1) > 67108864 (configuration 2,
 *    K = 10, N = 8192, L = 4, needs 36.3 MB and fits; K = 20, N = 16384, L = 8 does not).
 *  - The first call on a device loads the array's image and looks up its device address (a
 *    synchronous runtime query that makes the device set the 64 MiB aside): make that first call
 *    at start-up, before the rest of the device memory is handed to a pool and before starting any
 *    stream capture.  If the device has no room left, that call returns D2MHE_ERR_CUDA and a later
 *    call tries again.  Later calls only read the cached address; first calls from several host
 *    threads are serialised by a lock.
 *  - All contexts and all calls on one GPU share the array, which keeps the last call's
 *    contents.  Nothing has to be cleared (every buffer is written before it is read), but
 *    two calls whose work overlaps on the GPU (different streams, threads or contexts) race.
 * Arguments as for d2mhe_round_device.
 */
d2mhe_status d2mhe_round_device_static(d2mhe_ctx* ctx, const int32_t* values_dev, uint32_t ct_first,
                                       uint32_t n_cts, const uint32_t* nbr_offsets,
                                       const uint32_t* nbr_rows, int32_t* sums_dev);

/* Test hooks. */
/* The violation that d2mhe_sync last reported as D2MHE_ERR_DEVICE_CHECK:
 * info = {site (1 load, 2 store, 3 octet, 4 shared-memory offset, 5 twiddle index, 6 party number,
 * 7 limb, 8 streaming element, 9 staged bytes, 15 self-test), index, limit, thread block}. */
d2mhe_status d2mhe_debug_last_device_check(const d2mhe_ctx* ctx, uint32_t info[4]);
/* Launches one thread that runs the checked build's index test on the index 1 with limit 1 (it
 * touches no memory): with D2MHE_FLAG_DEVICE_CHECKS the next d2mhe_sync returns
 * D2MHE_ERR_DEVICE_CHECK with site 15, without the flag nothing happens. */
d2mhe_status d2mhe_debug_check_selftest(d2mhe_ctx* ctx);
/* s_k as int8 [N] on the HOST (needs a key share for `party`): the key that the device stores (in
 * the transform domain) is inverse-transformed on the GPU, limb by limb, and copied back;
 * D2MHE_ERR_DEVICE_CHECK if the limbs disagree or a coefficient is not in {-1, 0, 1}.  Allocates a
 * temporary device buffer and synchronises the stream. */
d2mhe_status d2mhe_debug_export_secret(d2mhe_ctx* ctx, uint32_t party, int8_t* s_host);
/* The same for sk_i of a user's own key pair (needs d2mhe_user_keygen for `user`). */
d2mhe_status d2mhe_debug_export_user_secret(d2mhe_ctx* ctx, uint32_t user, int8_t* s_host);
/* Measurement hook for the integer roofline of the transform kernels (Sec. 3.2 / 4.2: the ring
 * products are where the time goes): runs a loop on registers only that fills every SM (2048
 * resident threads, eight independent chains per thread, no memory traffic) for `iters`
 * iterations and reports lane operations per second, timed with CUDA events on the context's
 * stream (the call synchronises).  kind 0: mad.lo.u32, 1: mad.wide.u32 with a 64-bit addend,
 * 2: mad.hi.u32 (32 lane operations per warp instruction), 3: the engine's forward butterfly on
 * eight coefficients per thread (operations = butterflies; needs a parameter set whose primes
 * are all below 2^56 and of the form 2^b - d, else D2MHE_ERR_UNSUPPORTED), 4: mul.wide.u32,
 * 5: mul.hi.u32 (both without an addend), 6: mad.wide.u32 with a loop-invariant addend.
 * 1 <= iters <= 2^24. */
d2mhe_status d2mhe_debug_int_throughput(d2mhe_ctx* ctx, uint32_t kind, uint32_t iters,
                                        double* ops_per_second);
/* The primitive 2N-th root of unity used for limb `limb`. */
d2mhe_status d2mhe_get_root(const d2mhe_ctx* ctx, uint32_t limb, uint64_t* psi);
/* psi_t, the slot root (D2MHE_ERR_UNSUPPORTED if t != 1 mod 2N). */
d2mhe_status d2mhe_get_plain_root(const d2mhe_ctx* ctx, uint64_t* psi_t);
/* Number of kernels this context has launched since creation. */
uint64_t d2mhe_launch_count(const d2mhe_ctx* ctx);
/* Bytes of the context's sample scratch (see d2mhe_create): a single call whose samples need more
 * runs as several batches. */
size_t d2mhe_sample_scratch_bytes(const d2mhe_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* D2MHE_H */
