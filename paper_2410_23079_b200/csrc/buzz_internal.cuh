// Internal definitions shared by the libbuzz translation units (host object, device views,
// launch wrappers). Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "buzz.h"

// BUZZ policy constants as the kernels see them (Table 1 of the paper).
struct BuzzPolicy {
  int sink;      // k
  int window;    // w
  int segment;   // s
  int hitters;   // winners per segment
  int budget;    // T + k + w
  int s_hat;     // stride for old tokens: floor((s+1)/2) unless overridden
  int interval_new;  // 1: interval sampling for new tokens too (ablation), 0: local max (Algorithm 2)
  int policy;        // BUZZ_POLICY_BEEHIVE (sampling module) or BUZZ_POLICY_GLOBAL_TOPK
};

// Device view of the persistent state. Instance index = ((layer * max_batch) + seq) * kv_heads + head.
// Slot layout of an instance: [sink | window ring | middle (old, then new)], see cache_ops.cuh.
struct BuzzState {
  char* K;            // [inst][budget][d] elements
  char* V;            // [inst][budget][d] elements
  float* score;       // [inst][budget]
  int32_t* pos;       // [inst][budget]
  int32_t* n;         // [inst] retained slots
  int32_t* n_old;     // [inst] middle slots that survived an eviction
  int32_t* total;     // [inst] tokens seen so far (next position)
  int32_t* ring;      // [inst] ring index of the oldest window token (0 while the ring is filling)
  int32_t* status;    // [4]: first error code, instance, detail, spare
};

struct buzz_ctx {
  BuzzPolicy pol;
  buzz_shape sh;
  int group;          // q_heads / kv_heads
  size_t esize;       // bytes per K/V element
  BuzzState st;
  // scratch partition
  float* lse;         // [q_heads][lse_stride] row log-sum-exp (log2 domain) of one prefill; the tensor-core path
                      // starts each sequence's rows at a multiple of four floats (16-byte-aligned bulk copies)
  int lse_stride;     // floats per head: max_prompt_tokens + 4 per sequence + one tile of slack, a multiple of 4
  float* pscore;      // [kv_heads][max_prompt_tokens] pre-eviction prompt scores
  char* stage;        // staging for the host-buffer entries: per layer q | k | v, then per layer out
  size_t stage_q, stage_kv;  // byte sizes of one q-shaped and one kv-shaped staging tensor
  int* batch;         // active sequences per layer (host array)
  int decode_cluster; // 0 = choose automatically
  int sm_count;       // multiprocessors of the device that was current at buzz_create
  int fused_evict;    // 1: a decode step runs the eviction of an instance that it fills, in its own tail
  char* maybe_full;   // per layer (host): 1 if some cache of the layer may hold >= budget slots
  long long launches;
  // what the library launched last through this object (0 nothing, 1 a bf16 decode step, 2 anything else)
  int last_kind, last_layer;
  void* last_stream;
};

__host__ __device__ inline size_t buzz_inst(const buzz_shape& sh, int layer, int seq, int head) {
  return ((size_t)layer * sh.max_batch + seq) * sh.kv_heads + head;
}

// Records the first error seen on the device; later ones are dropped.
__device__ inline void buzz_set_status(int32_t* status, int code, int inst, int detail) {
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = inst;
    status[2] = detail;
  }
}

// The opt-in to more than 48 KB of dynamic shared memory is a per-DEVICE property of a kernel. One of
// these per kernel (a function-local static) remembers, per device ordinal, the largest size already
// applied, so that a process driving several GPUs sets it on each of them.
constexpr int kBuzzMaxDevices = 64;
struct BuzzSmemOptIn {
  size_t applied[kBuzzMaxDevices] = {};
  template <typename Kernel>
  cudaError_t ensure(Kernel kernel, size_t bytes) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kBuzzMaxDevices) return cudaErrorInvalidDevice;
    if (bytes <= applied[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) applied[dev] = bytes;
    return e;
  }
};

// ---- launch wrappers (each returns a cudaError_t from the launch) ---------------------------
// chain_pos: -1 for a single-layer call, else the index of this launch within one multi-layer call
// (whose inputs are all complete before the call and whose layers are distinct); next_layer: the
// layer the following launch will read (-1 unknown), used only as a prefetch hint.
cudaError_t buzz_launch_decode(buzz_ctx* c, int layer, const void* q, const void* k_new,
                               const void* v_new, void* out, cudaStream_t stream, int chain_pos = -1,
                               int next_layer = -1);
cudaError_t buzz_launch_evict(buzz_ctx* c, int layer_begin, int layer_count, cudaStream_t stream);
cudaError_t buzz_launch_prefill_attention(buzz_ctx* c, const void* q, const void* k, const void* v,
                                          const int32_t* cu, int batch, int total_tokens,
                                          int max_seqlen, void* out, cudaStream_t stream,
                                          int* launches);
cudaError_t buzz_launch_prefill_fill(buzz_ctx* c, int layer, const void* k, const void* v,
                                     const int32_t* cu, int batch, int max_seqlen,
                                     cudaStream_t stream);
