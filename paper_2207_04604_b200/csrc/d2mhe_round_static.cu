// d2mhe_round_device_static: the whole-round driver for callers that must not allocate.
//
// d2mhe_round_device keeps a chunk's protocol messages (ciphertexts, neighbour sums,
// decryption shares) in a workspace the caller allocates.  Some callers cannot provide
// one: a service that has handed all device memory to a fixed pool at start-up, a plug-in
// that is only given its input and output buffers, code running where cudaMalloc is
// forbidden because its implicit device synchronisation would stall other streams.  For
// them the same round runs here with the messages in a fixed array that is part of the
// library image.
#include "d2mhe_internal.h"

#define D2MHE_STATIC_SCRATCH_BYTES ((size_t)64 << 20)
#define D2MHE_STATIC_MAX_DEVICES 64

// Part of this translation unit's device image: a GPU reserves the 64 MiB when the runtime loads
// that image there, which (with the runtime's lazy module loading) happens at the address lookup
// below, i.e. in the first d2mhe_round_device_static call on that GPU, and keeps them until the
// process exits.  Shared by all contexts and all calls on that GPU.
static __device__ __align__(256) unsigned char g_round_scratch[D2MHE_STATIC_SCRATCH_BYTES];

// In host code `g_round_scratch` is only a handle for the runtime, not an address a kernel
// can use: the device address is looked up once per device, with that device current.
// Guarded by a mutex so that contexts on different host threads may make their first call at
// the same time.
#include <mutex>
static void* g_scratch_addr[D2MHE_STATIC_MAX_DEVICES] = {};
static std::mutex g_scratch_mutex;

extern "C" d2mhe_status d2mhe_round_device_static(d2mhe_ctx* ctx, const int32_t* values_dev,
                                                  uint32_t ct_first, uint32_t n_cts,
                                                  const uint32_t* nbr_offsets,
                                                  const uint32_t* nbr_rows, int32_t* sums_dev) {
  if (!ctx) return D2MHE_ERR_INVALID_ARG;
  const int dev = ctx->device;
  if (dev < 0 || dev >= D2MHE_STATIC_MAX_DEVICES) return D2MHE_ERR_UNSUPPORTED;
  // One ciphertext index of this parameter set must fit the fixed array.
  const size_t need = d2mhe_round_workspace_bytes(ctx, 1);
  if (need == 0 || need > D2MHE_STATIC_SCRATCH_BYTES) return D2MHE_ERR_WORKSPACE;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
      // First call on this device: loads the image that holds the array (the device reserves its
      // 64 MiB now; cudaErrorMemoryAllocation here means the device had no room left for it) and
      // asks for the array's address.  A synchronous runtime query: not for use during capture.
      int prev = -1;
      cudaError_t e = cudaGetDevice(&prev);
      if (e == cudaSuccess && prev != dev) e = cudaSetDevice(dev);
      void* ptr = nullptr;
      if (e == cudaSuccess) {
        e = cudaGetSymbolAddress(&ptr, g_round_scratch);
        if (prev != dev) cudaSetDevice(prev);
      }
      if (e == cudaSuccess && !ptr) e = cudaErrorInvalidSymbol;  // success without an address: treat as a failed lookup
      if (e != cudaSuccess) {
        ctx->last_cuda = e;
        (void)cudaGetLastError();
        return D2MHE_ERR_CUDA;
      }
      g_scratch_addr[dev] = ptr;
    }
    scratch = g_scratch_addr[dev];
  }
  // Every buffer of a chunk is written in full before it is read (encode -> encrypt ->
  // sums -> shares -> combine -> decode), so what an earlier call left in the array is
  // never observed and nothing needs clearing.
  return d2mhe_round_device(ctx, values_dev, ct_first, n_cts, nbr_offsets, nbr_rows, sums_dev,
                            scratch, D2MHE_STATIC_SCRATCH_BYTES);
}
