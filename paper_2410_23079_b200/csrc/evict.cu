// BUZZ eviction as a call of its own: segmented select-and-compact, one CTA per (layer, sequence,
// KV head) instance (Algorithm 1's sampling line and final concatenation; Algorithm 2). The trigger
// is a device predicate, so the call needs no host decision; an instance below its budget costs one
// counter read. The work itself is buzz_dev::evict_instance (cache_ops.cuh), which the decode
// kernels can also run in their tail.
#include "cache_ops.cuh"

namespace {

constexpr int kThreads = 256;

template <int ROW_BYTES>
__global__ void __launch_bounds__(kThreads)
evict_kernel(BuzzState st, BuzzPolicy pol, int layer_begin, int max_batch, int kv_heads, int batch) {
  extern __shared__ int32_t src[];   // work area: source slot of every surviving middle slot, staged scores and positions
  const int head = blockIdx.x, seq = blockIdx.y, layer = layer_begin + blockIdx.z;
  if (seq >= batch) return;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int n = st.n[inst];
  if (n < pol.budget) return;                       // threshold buffering: evict only when full
  if (n <= pol.sink + pol.window) return;           // Remark 1
  buzz_dev::evict_instance<ROW_BYTES, kThreads>(st, pol, inst, n, st.n_old[inst], src);
}

}  // namespace

cudaError_t buzz_launch_evict(buzz_ctx* c, int layer_begin, int layer_count, cudaStream_t stream) {
  int batch = 0;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) batch = max(batch, c->batch[l]);
  if (batch == 0) return cudaSuccess;
  dim3 grid(c->sh.kv_heads, batch, layer_count);
  (void)cudaGetLastError();   // drop a stale non-sticky error left by an earlier runtime call of the process
  const size_t smem = buzz_dev::evict_smem_bytes(c->pol);
  const int row_bytes = c->sh.head_dim * (int)c->esize;
#define BUZZ_EVICT_CASE(RB)                                                                        \
  case RB: {                                                                                       \
    static BuzzSmemOptIn opt_in;                                                                   \
    if (cudaError_t e = opt_in.ensure(evict_kernel<RB>, smem); e != cudaSuccess) return e;         \
    evict_kernel<RB><<<grid, kThreads, smem, stream>>>(c->st, c->pol, layer_begin, c->sh.max_batch, \
                                                       c->sh.kv_heads, batch);                     \
    break;                                                                                         \
  }
  switch (row_bytes) {
    BUZZ_EVICT_CASE(128)
    BUZZ_EVICT_CASE(256)
    BUZZ_EVICT_CASE(512)
    default: return cudaErrorInvalidValue;
  }
#undef BUZZ_EVICT_CASE
  c->launches += 1;
  c->last_kind = 2;
  return cudaGetLastError();
}
