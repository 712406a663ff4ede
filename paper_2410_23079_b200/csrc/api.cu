// libbuzz C ABI: argument checking, workspace partitioning and kernel dispatch.
#include <stdlib.h>
#include <string.h>

#include <new>

#include "buzz_internal.cuh"
#include "cache_ops.cuh"

cudaError_t buzz_launch_prefill_simt(buzz_ctx* c, const void* q, const void* k, const void* v,
                                     const int32_t* cu, int batch, int max_seqlen, void* out,
                                     cudaStream_t stream, int* launches);

cudaError_t buzz_launch_prefill_tc(buzz_ctx* c, const void* q, const void* k, const void* v,
                                   const int32_t* cu, int batch, int total_tokens, int max_seqlen,
                                   void* out, cudaStream_t stream, int* launches);

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t k, v, score, pos, n, n_old, total, ring, status, state_bytes;
  size_t lse, pscore, stage, scratch_bytes, stage_q, stage_kv;
};

bool shape_ok(const buzz_shape* s, int budget) {
  if (!s) return false;
  if (s->layers < 1 || s->max_batch < 1 || s->q_heads < 1 || s->kv_heads < 1) return false;
  if (s->q_heads % s->kv_heads) return false;
  const int g = s->q_heads / s->kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8) return false;
  if (s->head_dim != 64 && s->head_dim != 128) return false;
  if (s->dtype != BUZZ_F32 && s->dtype != BUZZ_BF16) return false;
  if (s->max_prompt_tokens < 1) return false;
  if (budget < 1 || budget > 32768) return false;
  return true;
}

// floats per head of the row-statistics scratch: every sequence may start up to 4 floats later than
// its token offset (alignment), and a tile read may run 127 rows past a sequence's end
inline int lse_stride_of(const buzz_shape& s) { return ((s.max_prompt_tokens + 4 * s.max_batch + 128 + 3) & ~3) + 4; }

Layout make_layout(const buzz_shape& s, int budget) {
  Layout L{};
  const size_t e = s.dtype == BUZZ_BF16 ? 2 : 4;
  const size_t inst = (size_t)s.layers * s.max_batch * s.kv_heads;
  size_t off = 0;
  L.k = off; off = align_up(off + inst * budget * s.head_dim * e);
  L.v = off; off = align_up(off + inst * budget * s.head_dim * e);
  L.score = off; off = align_up(off + inst * budget * sizeof(float));
  L.pos = off; off = align_up(off + inst * budget * sizeof(int32_t));
  L.n = off; off = align_up(off + inst * sizeof(int32_t));
  L.n_old = off; off = align_up(off + inst * sizeof(int32_t));
  L.total = off; off = align_up(off + inst * sizeof(int32_t));
  L.ring = off; off = align_up(off + inst * sizeof(int32_t));
  L.status = off; off = align_up(off + 4 * sizeof(int32_t));
  L.state_bytes = off;
  off = 0;
  L.lse = off; off = align_up(off + (size_t)s.q_heads * lse_stride_of(s) * sizeof(float));
  L.pscore = off; off = align_up(off + (size_t)s.kv_heads * s.max_prompt_tokens * sizeof(float));
  L.stage_q = align_up((size_t)s.max_batch * s.q_heads * s.head_dim * e);
  L.stage_kv = align_up((size_t)s.max_batch * s.kv_heads * s.head_dim * e);
  L.stage = off; off += (size_t)s.layers * (2 * L.stage_q + 2 * L.stage_kv);
  L.scratch_bytes = off;
  return L;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The device-side address of a HOST buffer the GPU can read and write in place (pinned and mapped,
// which is what cudaHostAlloc / cudaHostRegister give under unified addressing), or null if the
// buffer is pageable, partly outside one such allocation, or misaligned for the kernels.
void* mapped_device_ptr(const void* host, size_t bytes) {
  if (!host || bytes == 0) return nullptr;
  cudaPointerAttributes first, last;
  if (cudaPointerGetAttributes(&first, host) != cudaSuccess ||
      cudaPointerGetAttributes(&last, static_cast<const char*>(host) + bytes - 1) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  if (first.type != cudaMemoryTypeHost || last.type != cudaMemoryTypeHost || !first.devicePointer || !last.devicePointer)
    return nullptr;
  if (static_cast<char*>(last.devicePointer) - static_cast<char*>(first.devicePointer) != (ptrdiff_t)(bytes - 1)) return nullptr;
  return aligned16(first.devicePointer) ? first.devicePointer : nullptr;
}

}  // namespace

extern "C" {

int buzz_workspace_bytes(const buzz_shape* shape, int budget, size_t* state_bytes, size_t* scratch_bytes) {
  if (!shape_ok(shape, budget) || !state_bytes || !scratch_bytes) return BUZZ_ERR_INVALID;
  const Layout L = make_layout(*shape, budget);
  *state_bytes = L.state_bytes;
  *scratch_bytes = L.scratch_bytes;
  return BUZZ_OK;
}

int buzz_create(buzz_t* out, int sink, int window, int segment, int hitters, int budget,
                const buzz_shape* shape, void* state_dev, size_t state_bytes, void* scratch_dev,
                size_t scratch_bytes) {
  if (!out) return BUZZ_ERR_INVALID;
  *out = nullptr;
  if (!shape_ok(shape, budget)) return BUZZ_ERR_INVALID;
  if (sink < 0 || window < 1 || segment < 2 || segment > 1024 || hitters < 1 || hitters >= segment)
    return BUZZ_ERR_INVALID;
  if (budget < sink + window + segment) return BUZZ_ERR_INVALID;
  const Layout L = make_layout(*shape, budget);
  if (!state_dev || !scratch_dev || state_bytes < L.state_bytes || scratch_bytes < L.scratch_bytes)
    return BUZZ_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(state_dev) | reinterpret_cast<uintptr_t>(scratch_dev)) & (kAlign - 1))
    return BUZZ_ERR_INVALID;
  buzz_ctx* c = new (std::nothrow) buzz_ctx();
  if (!c) return BUZZ_ERR_INVALID;
  c->pol = BuzzPolicy{sink, window, segment, hitters, budget, (segment + 1) / 2, 0, BUZZ_POLICY_BEEHIVE};
  c->sh = *shape;
  c->group = shape->q_heads / shape->kv_heads;
  c->esize = shape->dtype == BUZZ_BF16 ? 2 : 4;
  char* sb = static_cast<char*>(state_dev);
  c->st.K = sb + L.k;
  c->st.V = sb + L.v;
  c->st.score = reinterpret_cast<float*>(sb + L.score);
  c->st.pos = reinterpret_cast<int32_t*>(sb + L.pos);
  c->st.n = reinterpret_cast<int32_t*>(sb + L.n);
  c->st.n_old = reinterpret_cast<int32_t*>(sb + L.n_old);
  c->st.total = reinterpret_cast<int32_t*>(sb + L.total);
  c->st.ring = reinterpret_cast<int32_t*>(sb + L.ring);
  c->st.status = reinterpret_cast<int32_t*>(sb + L.status);
  char* sc = static_cast<char*>(scratch_dev);
  c->lse = reinterpret_cast<float*>(sc + L.lse);
  c->lse_stride = lse_stride_of(*shape);
  c->pscore = reinterpret_cast<float*>(sc + L.pscore);
  c->stage = sc + L.stage;
  c->stage_q = L.stage_q;
  c->stage_kv = L.stage_kv;
  c->batch = static_cast<int*>(calloc(shape->layers, sizeof(int)));
  c->maybe_full = static_cast<char*>(calloc(shape->layers, 1));
  c->fused_evict = 0;
  c->decode_cluster = 0;
  c->sm_count = 148;
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      c->sm_count = sms;
    else
      (void)cudaGetLastError();
  }
  c->launches = 0;
  c->last_kind = 0; c->last_layer = -1; c->last_stream = nullptr;
  if (!c->batch || !c->maybe_full) { free(c->batch); free(c->maybe_full); delete c; return BUZZ_ERR_INVALID; }
  if (cudaMemset(state_dev, 0, L.state_bytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    free(c->batch);
    free(c->maybe_full);
    delete c;
    return BUZZ_ERR_CUDA;
  }
  *out = c;
  return BUZZ_OK;
}

void buzz_destroy(buzz_t c) {
  if (!c) return;
  free(c->batch);
  free(c->maybe_full);
  delete c;
}

int buzz_prefill(buzz_t c, int layer, const void* q, const void* k, const void* v,
                 const int32_t* cu_seqlens_dev, int batch, int total_tokens, int max_seqlen,
                 void* out, void* stream) {
  if (!c || layer < 0 || layer >= c->sh.layers || batch < 1 || batch > c->sh.max_batch) return BUZZ_ERR_INVALID;
  if (total_tokens < 1 || total_tokens > c->sh.max_prompt_tokens || max_seqlen < 1 || max_seqlen > total_tokens)
    return BUZZ_ERR_INVALID;
  if (!q || !k || !v || !out || !cu_seqlens_dev) return BUZZ_ERR_INVALID;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return BUZZ_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int launches = 0;
  cudaError_t e;
  if (c->sh.dtype == BUZZ_BF16 && c->sh.head_dim == 128)   // tensor-core path (TMA + tcgen05 + TMEM)
    e = buzz_launch_prefill_tc(c, q, k, v, cu_seqlens_dev, batch, total_tokens, max_seqlen, out, s, &launches);
  else
    e = buzz_launch_prefill_simt(c, q, k, v, cu_seqlens_dev, batch, max_seqlen, out, s, &launches);
  c->launches += launches;
  if (e != cudaSuccess) return BUZZ_ERR_CUDA;
  c->batch[layer] = batch;
  e = buzz_launch_prefill_fill(c, layer, k, v, cu_seqlens_dev, batch, max_seqlen, s);
  c->maybe_full[layer] = 0;   // the sampling rounds leave every sequence below its budget
  return e == cudaSuccess ? BUZZ_OK : BUZZ_ERR_CUDA;
}

int buzz_decode_step(buzz_t c, int layer, const void* q, const void* k_new, const void* v_new,
                     void* out, void* stream) {
  if (!c || layer < 0 || layer >= c->sh.layers || !q || !k_new || !v_new || !out) return BUZZ_ERR_INVALID;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return BUZZ_ERR_INVALID;
  cudaError_t e = buzz_launch_decode(c, layer, q, k_new, v_new, out, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? BUZZ_OK : BUZZ_ERR_CUDA;
}

int buzz_decode_step_host(buzz_t c, int layer, const void* q_host, const void* k_new_host,
                          const void* v_new_host, void* out_host, void* stream) {
  if (!c || layer < 0 || layer >= c->sh.layers || !q_host || !k_new_host || !v_new_host || !out_host)
    return BUZZ_ERR_INVALID;
  const int batch = c->batch[layer];
  if (batch == 0) return BUZZ_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t qb = (size_t)batch * c->sh.q_heads * c->sh.head_dim * c->esize;
  const size_t kb = (size_t)batch * c->sh.kv_heads * c->sh.head_dim * c->esize;
  // staging is packed q | k | v (row sizes are multiples of 16 bytes), so host buffers laid out the
  // same way go down in ONE copy; `out` has its own region behind them
  {   // buffers the GPU can address in place need no staging copies: the kernel reads and writes them over the bus
    void* mq = mapped_device_ptr(q_host, qb);
    void* mk = mapped_device_ptr(k_new_host, kb);
    void* mv = mapped_device_ptr(v_new_host, kb);
    void* mo = mapped_device_ptr(out_host, qb);
    if (mq && mk && mv && mo)
      return buzz_launch_decode(c, layer, mq, mk, mv, mo, s) == cudaSuccess ? BUZZ_OK : BUZZ_ERR_CUDA;
  }
  char* dq = c->stage;
  char* dk = dq + qb;
  char* dv = dk + kb;
  char* dout = c->stage + (size_t)c->sh.layers * (c->stage_q + 2 * c->stage_kv);
  const char* qh = static_cast<const char*>(q_host);
  bool sent = false;
  if (static_cast<const char*>(k_new_host) == qh + qb && static_cast<const char*>(v_new_host) == qh + qb + kb) {
    // Adjacent addresses do not prove one allocation: a copy that spans separately pinned buffers is
    // refused at the call ("invalid argument", nothing queued). Then clear that error and copy by parts.
    sent = cudaMemcpyAsync(dq, q_host, qb + 2 * kb, cudaMemcpyHostToDevice, s) == cudaSuccess;
    if (!sent) (void)cudaGetLastError();
  }
  if (!sent) {
    if (cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (cudaMemcpyAsync(dk, k_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (cudaMemcpyAsync(dv, v_new_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return BUZZ_ERR_CUDA;
  }
  if (buzz_launch_decode(c, layer, dq, dk, dv, dout, s) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpyAsync(out_host, dout, qb, cudaMemcpyDeviceToHost, s) != cudaSuccess) return BUZZ_ERR_CUDA;
  return BUZZ_OK;
}

namespace {
// Position order <-> slot order of one instance ([sink | window ring | middle], cache_ops.cuh): the
// retained tokens in position order are at most four contiguous runs of slots.
struct Run { int first_out, first_slot, count; };
int position_runs(const BuzzPolicy& pol, int n, int head, Run (&runs)[4]) {
  const int k = pol.sink, w = pol.window;
  int r = 0;
  if (n <= k + w) {                       // ring still filling: slots are in position order
    if (n > 0) runs[r++] = Run{0, 0, n};
    return r;
  }
  const int m = n - k - w;
  if (k > 0) runs[r++] = Run{0, 0, k};
  runs[r++] = Run{k, k + w, m};
  runs[r++] = Run{k + m, k + head, w - head};
  if (head > 0) runs[r++] = Run{k + m + w - head, k, head};
  return r;
}

// layers of one multi-layer call: in range, prefilled or empty, and pairwise distinct
bool layers_ok(buzz_t c, int count, const int* layers) {
  if (!c || !layers || count < 1 || count > c->sh.layers) return false;
  for (int i = 0; i < count; ++i) {
    if (layers[i] < 0 || layers[i] >= c->sh.layers) return false;
    for (int j = 0; j < i; ++j)
      if (layers[j] == layers[i]) return false;
  }
  return true;
}
}  // namespace

int buzz_decode_layers(buzz_t c, int count, const int* layers, const void* const* q,
                       const void* const* k_new, const void* const* v_new, void* const* out,
                       void* stream) {
  if (!layers_ok(c, count, layers) || !q || !k_new || !v_new || !out) return BUZZ_ERR_INVALID;
  for (int i = 0; i < count; ++i) {
    if (!q[i] || !k_new[i] || !v_new[i] || !out[i]) return BUZZ_ERR_INVALID;
    if (!aligned16(q[i]) || !aligned16(k_new[i]) || !aligned16(v_new[i]) || !aligned16(out[i])) return BUZZ_ERR_INVALID;
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int pos = 0;                 // launches made so far in this call (empty layers launch nothing)
  for (int i = 0; i < count; ++i) {
    if (c->batch[layers[i]] == 0) continue;
    int next = -1;
    for (int j = i + 1; j < count && next < 0; ++j)
      if (c->batch[layers[j]] != 0) next = layers[j];
    if (buzz_launch_decode(c, layers[i], q[i], k_new[i], v_new[i], out[i], s, pos, next) != cudaSuccess)
      return BUZZ_ERR_CUDA;
    ++pos;
  }
  return BUZZ_OK;
}

int buzz_decode_layers_host(buzz_t c, int count, const int* layers, const void* in_host, void* out_host,
                            void* stream) {
  if (!layers_ok(c, count, layers) || !in_host || !out_host) return BUZZ_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t row_q = (size_t)c->sh.q_heads * c->sh.head_dim * c->esize;
  const size_t row_kv = (size_t)c->sh.kv_heads * c->sh.head_dim * c->esize;
  size_t in_bytes = 0, out_bytes = 0;
  for (int i = 0; i < count; ++i) {
    in_bytes += c->batch[layers[i]] * (row_q + 2 * row_kv);
    out_bytes += c->batch[layers[i]] * row_q;
  }
  if (in_bytes == 0) return BUZZ_OK;
  char* din = c->stage;
  char* dout = c->stage + (size_t)c->sh.layers * (c->stage_q + 2 * c->stage_kv);
  // Pinned, mapped host buffers are used in place: each kernel fetches its few input rows and writes
  // its output rows over the bus while the cache streams from HBM, so the transfers overlap the
  // step instead of bracketing it. Pageable buffers go through the staging area with one copy each way.
  void* min = mapped_device_ptr(in_host, in_bytes);
  void* mout = mapped_device_ptr(out_host, out_bytes);
  const bool in_place = min && mout;
  if (in_place) {
    din = static_cast<char*>(min);
    dout = static_cast<char*>(mout);
  } else if (cudaMemcpyAsync(din, in_host, in_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
    return BUZZ_ERR_CUDA;
  }
  size_t io = 0, oo = 0;
  int pos = 0;
  for (int i = 0; i < count; ++i) {
    const size_t b = c->batch[layers[i]];
    if (b == 0) continue;
    int next = -1;
    for (int j = i + 1; j < count && next < 0; ++j)
      if (c->batch[layers[j]] != 0) next = layers[j];
    const char* dq = din + io;
    if (buzz_launch_decode(c, layers[i], dq, dq + b * row_q, dq + b * (row_q + row_kv), dout + oo, s, pos, next) != cudaSuccess)
      return BUZZ_ERR_CUDA;
    io += b * (row_q + 2 * row_kv);
    oo += b * row_q;
    ++pos;
  }
  if (!in_place && cudaMemcpyAsync(out_host, dout, out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return BUZZ_ERR_CUDA;
  return BUZZ_OK;
}

int buzz_evict(buzz_t c, int layer, void* stream) {
  if (!c || layer < -1 || layer >= c->sh.layers) return BUZZ_ERR_INVALID;
  // Layers whose caches are all known to be below their budget (a prefill, a fused decode step or an
  // eviction was the last thing done to them) need no launch: the device predicate would find nothing.
  const int begin = layer < 0 ? 0 : layer, count = layer < 0 ? c->sh.layers : 1;
  bool due = false;
  for (int l = begin; l < begin + count; ++l) due = due || c->maybe_full[l];
  if (!due) return BUZZ_OK;
  cudaError_t e = buzz_launch_evict(c, begin, count, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return BUZZ_ERR_CUDA;
  for (int l = begin; l < begin + count; ++l) c->maybe_full[l] = 0;
  return BUZZ_OK;
}

int buzz_set_fused_evict(buzz_t c, int on) {
  if (!c) return BUZZ_ERR_INVALID;
  if (on) {
    // A decode CTA then holds the eviction's work area beside its own buffers in shared memory; with the
    // instance split over the largest cluster (8 CTAs) that must stay within what a CTA may use.
    const size_t G = c->group, D = c->sh.head_dim;
    const size_t decode = 2048 + 4 * (2 * G + G * D) + 4 * (80 + 10 * G + 8 * G * D) + 4 * G * ((size_t)c->pol.budget / 8 + 4);
    if (decode + buzz_dev::evict_smem_bytes(c->pol) > 200 * 1024) return BUZZ_ERR_TOO_LARGE;
  }
  c->fused_evict = on ? 1 : 0;
  return BUZZ_OK;
}

int buzz_export_state(buzz_t c, int layer, int seq, int kv_head, int32_t* n, int32_t* n_old,
                      int32_t* total_len, int32_t* pos_host, float* score_host, void* k_host,
                      void* v_host) {
  if (!c || layer < 0 || layer >= c->sh.layers || seq < 0 || seq >= c->sh.max_batch || kv_head < 0 ||
      kv_head >= c->sh.kv_heads)
    return BUZZ_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) return BUZZ_ERR_CUDA;
  const size_t inst = buzz_inst(c->sh, layer, seq, kv_head);
  int32_t cnt[4];
  if (cudaMemcpy(&cnt[0], c->st.n + inst, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(&cnt[1], c->st.n_old + inst, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(&cnt[2], c->st.total + inst, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(&cnt[3], c->st.ring + inst, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (n) *n = cnt[0];
  if (n_old) *n_old = cnt[1];
  if (total_len) *total_len = cnt[2];
  const int m = cnt[0];
  if (m < 0 || m > c->pol.budget || cnt[3] < 0 || cnt[3] >= c->pol.window) return BUZZ_ERR_INVALID;
  const size_t row = (size_t)c->sh.head_dim * c->esize;
  const size_t slot0 = inst * c->pol.budget;
  Run runs[4];
  const int nr = position_runs(c->pol, m, cnt[3], runs);
  for (int r = 0; r < nr; ++r) {           // the window ring is un-rotated: the output is in position order
    const size_t o = runs[r].first_out, sl = slot0 + runs[r].first_slot, len = runs[r].count;
    if (pos_host && cudaMemcpy(pos_host + o, c->st.pos + sl, len * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (score_host && cudaMemcpy(score_host + o, c->st.score + sl, len * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (k_host && cudaMemcpy(static_cast<char*>(k_host) + o * row, c->st.K + sl * row, len * row, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (v_host && cudaMemcpy(static_cast<char*>(v_host) + o * row, c->st.V + sl * row, len * row, cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  }
  return BUZZ_OK;
}

int buzz_import_state(buzz_t c, int layer, int seq, int kv_head, int32_t n, int32_t n_old,
                      int32_t total_len, const int32_t* pos_host, const float* score_host,
                      const void* k_host, const void* v_host) {
  if (!c || layer < 0 || layer >= c->sh.layers || seq < 0 || seq >= c->sh.max_batch || kv_head < 0 ||
      kv_head >= c->sh.kv_heads)
    return BUZZ_ERR_INVALID;
  if (n < 0 || n > c->pol.budget || n_old < 0 || total_len < n) return BUZZ_ERR_INVALID;
  if (n_old > (n > c->pol.sink + c->pol.window ? n - c->pol.sink - c->pol.window : 0)) return BUZZ_ERR_INVALID;
  if (n > 0 && (!pos_host || !score_host || !k_host || !v_host)) return BUZZ_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) return BUZZ_ERR_CUDA;
  const size_t inst = buzz_inst(c->sh, layer, seq, kv_head);
  const size_t row = (size_t)c->sh.head_dim * c->esize;
  const size_t slot0 = inst * c->pol.budget;
  Run runs[4];
  const int nr = position_runs(c->pol, n, 0, runs);      // the window goes into the ring in order, head 0
  for (int r = 0; r < nr; ++r) {
    const size_t o = runs[r].first_out, sl = slot0 + runs[r].first_slot, len = runs[r].count;
    if (cudaMemcpy(c->st.pos + sl, pos_host + o, len * 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (cudaMemcpy(c->st.score + sl, score_host + o, len * 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (cudaMemcpy(c->st.K + sl * row, static_cast<const char*>(k_host) + o * row, len * row, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
    if (cudaMemcpy(c->st.V + sl * row, static_cast<const char*>(v_host) + o * row, len * row, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
  }
  const int32_t cnt[4] = {n, n_old, total_len, 0};
  if (cudaMemcpy(c->st.n + inst, &cnt[0], 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(c->st.n_old + inst, &cnt[1], 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(c->st.total + inst, &cnt[2], 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(c->st.ring + inst, &cnt[3], 4, cudaMemcpyHostToDevice) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (c->batch[layer] < seq + 1) c->batch[layer] = seq + 1;
  c->maybe_full[layer] = 1;
  c->last_kind = 2;
  return BUZZ_OK;
}

int buzz_export_prefill_scores(buzz_t c, int kv_head, int total_tokens, float* score_host) {
  if (!c || kv_head < 0 || kv_head >= c->sh.kv_heads || total_tokens < 1 ||
      total_tokens > c->sh.max_prompt_tokens || !score_host)
    return BUZZ_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) return BUZZ_ERR_CUDA;
  if (cudaMemcpy(score_host, c->pscore + (size_t)kv_head * c->sh.max_prompt_tokens,
                 (size_t)total_tokens * 4, cudaMemcpyDeviceToHost) != cudaSuccess)
    return BUZZ_ERR_CUDA;
  return BUZZ_OK;
}

int buzz_status(buzz_t c, void* stream) {
  if (!c) return BUZZ_ERR_INVALID;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return BUZZ_ERR_CUDA;
  int32_t word[4];
  if (cudaMemcpy(word, c->st.status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return BUZZ_ERR_CUDA;
  if (word[0] != 0 && cudaMemset(c->st.status, 0, sizeof(word)) != cudaSuccess) return BUZZ_ERR_CUDA;
  return word[0];
}

int64_t buzz_launch_count(buzz_t c) { return c ? c->launches : 0; }

int buzz_set_sampling(buzz_t c, int interval_new, int new_stride, int old_stride) {
  if (!c) return BUZZ_ERR_INVALID;
  if (new_stride < 2 || new_stride > 1024 || c->pol.hitters >= new_stride || old_stride < 1 ||
      c->pol.budget < c->pol.sink + c->pol.window + new_stride)
    return BUZZ_ERR_INVALID;
  c->pol.segment = new_stride;
  c->pol.s_hat = old_stride;
  c->pol.interval_new = interval_new ? 1 : 0;
  return BUZZ_OK;
}

int buzz_set_policy(buzz_t c, int policy) {
  if (!c || (policy != BUZZ_POLICY_BEEHIVE && policy != BUZZ_POLICY_GLOBAL_TOPK)) return BUZZ_ERR_INVALID;
  c->pol.policy = policy;
  return BUZZ_OK;
}

int buzz_set_decode_cluster(buzz_t c, int cluster_size) {
  if (!c) return BUZZ_ERR_INVALID;
  if (cluster_size != 0 && cluster_size != 1 && cluster_size != 2 && cluster_size != 4 && cluster_size != 8)
    return BUZZ_ERR_INVALID;
  c->decode_cluster = cluster_size;
  return BUZZ_OK;
}

const char* buzz_error_string(int code) {
  switch (code) {
    case BUZZ_OK: return "ok";
    case BUZZ_ERR_INVALID: return "invalid argument";
    case BUZZ_ERR_OVERFLOW: return "decode step on a full cache (call buzz_evict after every step)";
    case BUZZ_ERR_NO_PROGRESS: return "eviction cannot shrink the cache (segment too small for this budget)";
    case BUZZ_ERR_TIMEOUT: return "a bounded on-device wait expired";
    case BUZZ_ERR_CUDA: return "a CUDA runtime call failed";
    case BUZZ_ERR_TOO_LARGE: return "request exceeds the library's built-in fixed-size scratch array";
    default: return "unknown error";
  }
}

}  // extern "C"
