// buzz_prefill_static: the prefill of one layer with its scratch in a library-owned device array.
//
// Who this is for: code that runs where device memory cannot be allocated -- a plugin called from
// inside another framework's memory pool, a
// real-time loop that must not touch the allocator, a process whose memory was carved up once at
// start-up. Such a caller can still hand over its inputs and outputs, but it has nowhere to get
// the prefill's temporary buffers from (the per-row softmax statistics and the per-key column
// sums, normally part of the scratch allocation given to buzz_create). Here they live in one
// fixed array that the library image itself carries.
//
// Which kernels: always the CUDA-core (fp32-pipe) prefill kernels, whatever the dtype and head
// dimension, because their two temporaries are plain [heads][total_tokens] arrays that fit the
// built-in array exactly (the tensor-core kernels want padded, aligned row statistics). The results
// agree with buzz_prefill's within the library's tolerances, scores to rel 1e-3, not bit for bit.
//
// Cost and limits: the array takes BUZZ_STATIC_SCRATCH_FLOATS * 4 bytes (4 MiB) on every GPU that
// loads the library, until the process exits. A call needs (q_heads + kv_heads) * total_tokens
// floats and is refused with BUZZ_ERR_TOO_LARGE if that exceeds the array. All calls on a device
// share the array: its contents are whatever the previous call left (every entry a call reads is
// written by that same call first, so nothing has to be cleared), and two calls whose kernels
// overlap on the GPU (different streams, no dependency) would corrupt each other.
//
// The array's name means a device address only inside device code. On the host it is just a
// handle, so the address the kernels are given is looked up with cudaGetSymbolAddress, once per
// device, the first time this entry point is called with that device current. That first call
// should therefore be made outside any stream capture.
#include "buzz_internal.cuh"

cudaError_t buzz_launch_prefill_simt(buzz_ctx* c, const void* q, const void* k, const void* v,
                                     const int32_t* cu, int batch, int max_seqlen, void* out,
                                     cudaStream_t stream, int* launches);

static __device__ __align__(256) float buzz_static_scratch[BUZZ_STATIC_SCRATCH_FLOATS];

namespace {

constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices];   // device address of buzz_static_scratch, per device ordinal

// Resolves (once per device) the device address behind the symbol for the current device.
cudaError_t static_scratch(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_scratch_addr[dev]) {
    float* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), buzz_static_scratch);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int buzz_prefill_static(buzz_t c, int layer, const void* q, const void* k, const void* v,
                                   const int32_t* cu_seqlens_dev, int batch, int total_tokens,
                                   int max_seqlen, void* out, void* stream) {
  if (!c || layer < 0 || layer >= c->sh.layers || batch < 1 || batch > c->sh.max_batch) return BUZZ_ERR_INVALID;
  if (total_tokens < 1 || max_seqlen < 1 || max_seqlen > total_tokens) return BUZZ_ERR_INVALID;
  if (!q || !k || !v || !out || !cu_seqlens_dev) return BUZZ_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
       reinterpret_cast<uintptr_t>(out)) & 15u)
    return BUZZ_ERR_INVALID;
  const size_t need = (size_t)(c->sh.q_heads + c->sh.kv_heads) * (size_t)total_tokens;
  if (need > BUZZ_STATIC_SCRATCH_FLOATS) return BUZZ_ERR_TOO_LARGE;   // beyond the built-in array
  float* base = nullptr;
  if (static_scratch(&base) != cudaSuccess) return BUZZ_ERR_CUDA;
  // A private view of the object whose prefill temporaries point into the built-in array, packed
  // with a row stride of exactly total_tokens. The persistent state is shared with `c`.
  buzz_ctx view = *c;
  view.sh.max_prompt_tokens = total_tokens;
  view.lse = base;
  view.lse_stride = total_tokens;   // unused by the CUDA-core kernels (their row stride is max_prompt_tokens)
  view.pscore = base + (size_t)c->sh.q_heads * total_tokens;
  view.launches = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int launches = 0;
  cudaError_t e = buzz_launch_prefill_simt(&view, q, k, v, cu_seqlens_dev, batch, max_seqlen, out, s, &launches);
  if (e != cudaSuccess) return BUZZ_ERR_CUDA;
  c->batch[layer] = batch;          // the host array is shared between `c` and the view
  e = buzz_launch_prefill_fill(&view, layer, k, v, cu_seqlens_dev, batch, max_seqlen, s);
  c->maybe_full[layer] = 0;
  c->launches += launches + view.launches;
  c->last_kind = view.last_kind;     // bookkeeping the launches made on the view
  return e == cudaSuccess ? BUZZ_OK : BUZZ_ERR_CUDA;
}
