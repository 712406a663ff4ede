/* libbuzz -- C ABI of the BUZZ sparse KV-cache hot path on one NVIDIA B200 (sm_100a).
 *
 * BUZZ (arXiv 2410.23079) keeps, per attention head, a bounded KV cache made of four parts, in
 * position order  [ sink | old | new | window ]  (Algorithm 1): the first `sink` tokens, survivors of
 * earlier evictions ("old"), tokens that left the sliding window since the last eviction ("new"),
 * and the last `window` tokens. (In device memory the window is a ring that sits right behind the
 * sink, so that neither a decode step nor an eviction ever moves it; every call that hands cache
 * contents to the host returns them in position order.) Each retained token carries an accumulated attention score
 * (Algorithm 2's input A). When the cache is full, the new tokens are cut into segments of
 * `segment` tokens and the top-scoring `hitters` of each segment survive, while the old tokens are
 * thinned to every s_hat-th, s_hat = floor((segment+1)/2) (Section 3.3).
 *
 * Conventions for every call:
 *   - All tensor pointers are DEVICE pointers unless the name says `_host`. The caller allocates
 *     and owns all device memory and the stream; the library allocates no device memory, creates
 *     no stream, and (except where stated) does not synchronise.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Return value: BUZZ_OK or a negative BUZZ_ERR_* code. Nothing throws, traps or aborts.
 *     Conditions found on the device (slot overflow, an eviction that cannot shrink the cache)
 *     are recorded in a device status word, the affected sequence is left untouched, and the
 *     code surfaces at buzz_status().
 *   - Element type `dtype`: BUZZ_F32 (4-byte IEEE) or BUZZ_BF16 (2-byte bfloat16) for Q/K/V/O and
 *     the caches; scores are always fp32, positions int32. All pointers must be 16-byte aligned.
 *   - One instance = (layer, sequence, KV head). With grouped-query attention the q_heads/kv_heads
 *     query heads of a group share the instance and their probabilities are summed into one score.
 */
#ifndef BUZZ_H_
#define BUZZ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { BUZZ_F32 = 0, BUZZ_BF16 = 1 };

enum {
  BUZZ_OK = 0,
  BUZZ_ERR_INVALID = -1,     /* bad argument (synchronous, nothing was launched)            */
  BUZZ_ERR_OVERFLOW = -2,    /* decode step on a full cache (evict was not called in time)   */
  BUZZ_ERR_NO_PROGRESS = -3, /* an eviction left the cache full (degenerate parameters)      */
  BUZZ_ERR_TIMEOUT = -4,     /* a bounded on-device wait expired                             */
  BUZZ_ERR_CUDA = -5,        /* a CUDA runtime call failed                                   */
  BUZZ_ERR_TOO_LARGE = -6    /* request exceeds a built-in fixed-size buffer or shared memory  */
};

typedef struct buzz_ctx* buzz_t;

typedef struct buzz_shape {
  int32_t layers;            /* L                                                            */
  int32_t max_batch;         /* sequences per layer the caches are sized for                 */
  int32_t q_heads;           /* Hq                                                           */
  int32_t kv_heads;          /* Hkv, must divide Hq                                          */
  int32_t head_dim;          /* d: 64 or 128                                                 */
  int32_t dtype;             /* BUZZ_F32 or BUZZ_BF16                                        */
  int32_t max_prompt_tokens; /* upper bound on the packed token count of one buzz_prefill    */
  int32_t flags;             /* BUZZ_FLAG_*                                                  */
} buzz_shape;

enum {
  BUZZ_FLAG_LOGN = 1         /* scale logits by log_512(tokens seen)/sqrt(d) (Section 3.5)   */
};

enum {
  BUZZ_POLICY_BEEHIVE = 0,     /* BUZZ's sampling module: Algorithms 1 and 2 (the default)        */
  BUZZ_POLICY_GLOBAL_TOPK = 1  /* global top-k of the accumulated scores (Sections 3.2 and 4.3)   */
};

/* Sizes of the two device allocations buzz_create needs (Section 3.3 fixes the cache at
 * budget = T + sink + window slots per instance).
 *   state   : K and V caches [L][max_batch][Hkv][budget][d], score and pos [L][max_batch][Hkv][budget],
 *             counters n / n_old / total_len [L][max_batch][Hkv], and the status words.
 *   scratch : per-row softmax statistics and per-key column sums of one prefill, plus staging
 *             buffers (one set per layer) for the host-buffer decode entries. Contents are not carried between calls.
 * Returns BUZZ_ERR_INVALID for a shape or budget the library does not support: any of layers,
 * max_batch, q_heads, kv_heads, max_prompt_tokens < 1; kv_heads not dividing q_heads; a group size
 * q_heads / kv_heads other than 1, 2, 4 or 8; head_dim other than 64 or 128; an unknown dtype;
 * budget < 1 or budget > 32768; a null pointer. */
int buzz_workspace_bytes(const buzz_shape* shape, int budget, size_t* state_bytes, size_t* scratch_bytes);

/* Creates a cache policy object (Table 1: k = sink, w = window, s = segment; budget = T + k + w,
 * Remark 2). `hitters` is the number of winners kept per segment. Both allocations must be at
 * least as large as buzz_workspace_bytes reports and 256-byte aligned; `state_dev` is zeroed here
 * (one synchronous memset on the default stream). The device that is current at this call is the
 * one the object's kernels are sized for.
 * Rejects (BUZZ_ERR_INVALID, nothing allocated): everything buzz_workspace_bytes rejects; sink < 0;
 * window < 1; segment < 2 or segment > 1024; hitters < 1 or hitters >= segment;
 * budget < sink + window + segment; null, undersized or misaligned buffers. */
int buzz_create(buzz_t* out, int sink, int window, int segment, int hitters, int budget,
                const buzz_shape* shape, void* state_dev, size_t state_bytes,
                void* scratch_dev, size_t scratch_bytes);

/* Frees the host object only. */
void buzz_destroy(buzz_t ctx);

/* Prefill of one layer (Eqs. 1 and 3; Remark 2).
 *   q  [total_tokens][Hq][d], k, v [total_tokens][Hkv][d], out [total_tokens][Hq][d], all packed
 *   over `batch` sequences by cu_seqlens_dev [batch+1] (int32, device; cu[0] = 0, non-decreasing,
 *   cu[batch] = total_tokens -- the library never reads the array on the host and does not verify it).
 * Computes causal attention out = Softmax(q k^T / sqrt(d)) v per sequence and head, the initial
 * score of every key = the sum of the probabilities it received (column sums, summed over the
 * query heads of its group, in a fixed order), then, while a sequence holds >= budget tokens,
 * eviction rounds (first round: segment-wise top-`hitters` over everything between sink and
 * window; later rounds: every s_hat-th survivor), and writes the survivors' K, V, score and
 * position into the layer's cache. Resets that layer's sequences 0..batch-1.
 * `max_seqlen` is an upper bound on any sequence's length (host value, used for grid sizing).
 * Rejects: layer outside [0, layers); batch < 1 or > max_batch; total_tokens < 1 or
 * > max_prompt_tokens; max_seqlen < 1 or > total_tokens; null or misaligned pointers. */
int buzz_prefill(buzz_t ctx, int layer, const void* q, const void* k, const void* v,
                 const int32_t* cu_seqlens_dev, int batch, int total_tokens, int max_seqlen,
                 void* out, void* stream);

/* buzz_prefill for callers that cannot allocate device memory. (The paper has no counterpart;
 * this is a property of the library, not of the method.)
 * Some code runs where cudaMalloc is off limits: inside another framework's memory pool, in a
 * real-time loop, in a process whose device memory was handed out once at start-up. Such a caller
 * passes its inputs and outputs exactly as for buzz_prefill, and the prefill's temporaries (row
 * softmax statistics and per-key column sums) are placed in a fixed 4 MiB array built into the
 * library instead of in the scratch buffer given to buzz_create. Every GPU that loads the library
 * holds that array until the process exits.
 *   - Limit: (q_heads + kv_heads) * total_tokens <= BUZZ_STATIC_SCRATCH_FLOATS (1,048,576 floats);
 *     larger calls return BUZZ_ERR_TOO_LARGE and launch nothing. total_tokens need not respect
 *     max_prompt_tokens. cu_seqlens_dev[batch] must equal total_tokens as for buzz_prefill: an
 *     array that runs past it would make the kernels write beyond the built-in array.
 *   - Kernels: this entry always runs the library's CUDA-core (fp32-pipe) prefill kernels, also for
 *     bf16 with head_dim 128 where buzz_prefill uses the tensor-core kernels; it is meant for
 *     modest prompts. Outputs agree with buzz_prefill's within the library's tolerances and the
 *     scores to rel 1e-3, not bit for bit, so where two candidates of a segment are tied to that
 *     precision the two entries may retain different tokens.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) with
 *     that device current; make that first call outside any stream capture. If the process has not
 *     yet run any of the library's kernels on that device, that first call is also when the driver
 *     loads the library's device code and places the array, which is a driver-side allocation; from
 *     the second call on a device on, nothing is allocated or freed.
 *   - All calls on a device share the array, which keeps the previous call's contents (each call
 *     overwrites every entry before reading it, so no clearing is needed); calls whose kernels
 *     overlap on the GPU race on it, so order them on one stream or with events.
 *   - buzz_export_prefill_scores does not see this call's scores (they are in the built-in array).
 * Arguments, cache update and error behaviour are otherwise those of buzz_prefill. */
#define BUZZ_STATIC_SCRATCH_FLOATS (1u << 20)
int buzz_prefill_static(buzz_t ctx, int layer, const void* q, const void* k, const void* v,
                        const int32_t* cu_seqlens_dev, int batch, int total_tokens, int max_seqlen,
                        void* out, void* stream);

/* One decode step of one layer (Eqs. 2 and 3) for the `batch` sequences of the last prefill:
 *   q [batch][Hq][d], k_new, v_new [batch][Hkv][d], out [batch][Hq][d].
 * Appends (k_new, v_new) at slot n with score 0 and position total_len, attends over all n+1
 * retained slots, and adds each slot's probability (summed over the group's query heads) to its
 * score. A sequence whose cache is already full is skipped and BUZZ_ERR_OVERFLOW is recorded. */
int buzz_decode_step(buzz_t ctx, int layer, const void* q, const void* k_new, const void* v_new,
                     void* out, void* stream);

/* The same step with HOST buffers (pinned memory recommended): copies q/k_new/v_new to the
 * library's staging area in scratch, runs the step, copies `out` back, all on `stream`, without
 * synchronising. Layouts as in buzz_decode_step. If the three inputs are contiguous in host memory in
 * the order q, k_new, v_new (one allocation holding the packed record) they are sent in a single
 * copy; buffers that merely happen to be adjacent but were pinned separately are copied one by one.
 * If all four buffers are pinned and mapped, the kernel reads and writes them in place and nothing
 * is copied (see buzz_decode_layers_host). */
int buzz_decode_step_host(buzz_t ctx, int layer, const void* q_host, const void* k_new_host,
                          const void* v_new_host, void* out_host, void* stream);

/* One decode step (Eqs. 2 and 3) of SEVERAL layers in one call: the attention-only step of a layer
 * stack whose per-layer inputs already exist, e.g. a benchmark of the cache policy or a caller
 * that batches independent attention calls. `layers` (host array of `count` pairwise distinct
 * layer indices) is walked in order; q, k_new, v_new and out are host arrays of `count` device
 * pointers with the layouts of buzz_decode_step for each layer's own batch. Results are those of
 * `count` buzz_decode_step calls: bit for bit when the cluster size is fixed with
 * buzz_set_decode_cluster; with the built-in choice the two entry points may split an instance's
 * slots over a different number of CTAs, which changes the fp32 summation order and nothing else.
 * Contract: every input buffer must be complete (in stream order) before this call, and no `out`
 * buffer may alias another member's buffers. Within the call the launches are NOT serialised:
 * CTAs of consecutive layers occupy the SMs back to back and each member finishes only after the
 * members before it, so work enqueued after the call sees all of them complete. The first member
 * waits for all earlier work in the stream.
 * Returns BUZZ_ERR_INVALID for a repeated or out-of-range layer or a null / misaligned pointer. */
int buzz_decode_layers(buzz_t ctx, int count, const int* layers, const void* const* q,
                       const void* const* k_new, const void* const* v_new, void* const* out,
                       void* stream);

/* buzz_decode_layers with HOST buffers (pinned memory recommended). `in_host` is one packed buffer,
 * for each listed layer in order its q | k_new | v_new tensors (layouts of buzz_decode_step, sized by
 * that layer's batch); `out_host` receives the outputs packed the same way. Nothing synchronises.
 * Buffers the GPU can address in place (pinned and mapped: cudaHostAlloc, cudaHostRegister, a
 * framework's pinned tensors) are read and written by the kernels directly, so the transfers overlap
 * the step; otherwise: one host-to-device copy into the library's staging area, the launches, one
 * device-to-host copy, all on `stream`. Either way `out_host` is valid once `stream` has reached the
 * end of the call, and `in_host` must stay unchanged until then. */
int buzz_decode_layers_host(buzz_t ctx, int count, const int* layers, const void* in_host,
                            void* out_host, void* stream);

/* BUZZ eviction (Algorithm 1's sampling line and final concatenation; Algorithm 2) for one layer,
 * or for all layers when layer = -1. Per instance, entirely on the device: nothing happens unless
 * n >= budget (threshold buffering, Section 3.3) and n > sink + window (Remark 1). Otherwise the
 * old tokens keep offsets 0, s_hat, 2 s_hat, ...; the new tokens (everything that left the window
 * since the last eviction) are cut into segments of `segment` tokens (a short last one allowed) and
 * each keeps its top min(hitters, length) tokens by (score descending, position ascending), in
 * position order; K, V, score and pos of the survivors are compacted in place (sink and window are
 * not moved); n_old becomes |old'| + |new'|. Calling it after every decode step is the intended use;
 * when the library knows that no cache of the requested layers can be full (their last operation
 * was a prefill, an eviction, or a decode step in fused mode) the call returns without launching. */
int buzz_evict(buzz_t ctx, int layer, void* stream);

/* Fused mode (Section 3.3's buffering without a second launch). With on != 0 every decode step
 * (buzz_decode_step, buzz_decode_layers and their host-buffer forms) checks, in the kernel's own
 * tail, whether the step has filled an instance's cache (n >= budget) and if so runs that instance's
 * eviction right there, exactly as buzz_evict would have on the next call. The caches are then never
 * full between calls, buzz_evict has nothing to do (and launches nothing), and the state after each
 * step is bit-identical to decode step + buzz_evict in the default mode. Default: off.
 * Returns BUZZ_ERR_TOO_LARGE (and leaves the mode off) when the eviction's work area would not fit
 * beside a decode CTA's buffers in shared memory, which only very large budgets with large groups
 * reach (e.g. budget 32768 with 8 query heads per KV head); buzz_evict as a call of its own has no such limit. */
int buzz_set_fused_evict(buzz_t ctx, int on);

/* Test/checkpoint getter for one instance. Synchronises `stream`-independent: it waits for the
 * device. Any output pointer may be NULL. pos_host/score_host receive n entries, k_host/v_host
 * n*d elements of the cache dtype, in position order (sink, old, new, window; the window ring is
 * un-rotated). Buffers must hold `budget` entries. */
int buzz_export_state(buzz_t ctx, int layer, int seq, int kv_head, int32_t* n, int32_t* n_old,
                      int32_t* total_len, int32_t* pos_host, float* score_host, void* k_host,
                      void* v_host);

/* The inverse of buzz_export_state (checkpoint restore, and how tests plant a cache state): loads
 * n tokens (n <= budget, n_old <= max(n - sink - window, 0), total_len >= n) of one instance from
 * host buffers in position order, as buzz_export_state writes them, and marks sequences 0..seq of
 * the layer active. Waits for the device before and after copying. */
int buzz_import_state(buzz_t ctx, int layer, int seq, int kv_head, int32_t n, int32_t n_old,
                      int32_t total_len, const int32_t* pos_host, const float* score_host,
                      const void* k_host, const void* v_host);

/* Copies the pre-eviction prompt scores of the last buzz_prefill (one fp32 per prompt token of
 * KV head `kv_head`, packed like the prompt) to score_host [total_tokens]. Waits for the device. */
int buzz_export_prefill_scores(buzz_t ctx, int kv_head, int total_tokens, float* score_host);

/* Waits for `stream`, then returns the first error recorded on the device since the last call
 * (BUZZ_OK if none) and clears it. */
int buzz_status(buzz_t ctx, void* stream);

/* Self-test of the failure-detection path (not part of the method). Every wait inside the library's
 * kernels is bounded: after a fixed number of polls it gives up, records BUZZ_ERR_TIMEOUT in the
 * device status word and the kernel runs to its end. This call makes that happen on purpose and
 * harmlessly: one small CTA waits, through the same bounded wait, on a barrier at which nobody ever
 * arrives, with a limit of `polls` polls (1..65536; each poll may itself block for a few
 * microseconds). The kernel ends by itself; afterwards buzz_status() returns BUZZ_ERR_TIMEOUT once
 * and the object stays fully usable. No cache contents are touched. */
int buzz_selftest_wait_expiry(buzz_t ctx, int polls, void* stream);

/* Number of kernels the library has launched through this object (for launch accounting). */
int64_t buzz_launch_count(buzz_t ctx);

/* Sampling variants of the paper's ablation study (Section 4.3). By default new tokens are sampled
 * by local maximum with stride `segment` (Algorithm 2) and old tokens at intervals of
 * s_hat = floor((segment+1)/2). This call replaces the two strides (e.g. swapped, the "small stride
 * for old tokens" ablation) and, with interval_new != 0, samples new tokens at intervals as well
 * (the "no local max" ablation: the first min(hitters, length) slots of every segment are kept and
 * scores are ignored). Takes effect from the next prefill / eviction; counts stay score-independent.
 * Rejects new_stride < 2, hitters >= new_stride, old_stride < 1, budget < sink + window + new_stride. */
int buzz_set_sampling(buzz_t ctx, int interval_new, int new_stride, int old_stride);

/* Eviction policy. BUZZ_POLICY_BEEHIVE is the paper's method. BUZZ_POLICY_GLOBAL_TOPK is the
 * heavy-hitter selection the paper compares against (Section 3.2, "top-k tokens based on attention
 * scores A outside the sliding window"; Section 4.3, a top-k module on accumulated scores "instead of
 * the sampling module"): sink and window are kept as always, and of ALL tokens in between, old and
 * new alike, the M with the largest accumulated score survive (ties to the lowest position, emitted
 * in position order), where M is the number of tokens the sampling module would have kept at that
 * eviction, so that both policies follow the same cache-length schedule. Applies to prefill-time
 * rounds and decode-time evictions from the next call on. Rejects an unknown policy. */
int buzz_set_policy(buzz_t ctx, int policy);

/* Tuning knob: number of CTAs (1, 2, 4 or 8) of the thread-block cluster that shares one instance's
 * slots in buzz_decode_step; 0 restores the built-in choice. Results do not depend on it beyond
 * fp32 summation order. */
int buzz_set_decode_cluster(buzz_t ctx, int cluster_size);

/* Static description of an error code. */
const char* buzz_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* BUZZ_H_ */
