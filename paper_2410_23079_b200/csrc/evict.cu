// BUZZ eviction: segmented select-and-compact, one CTA per (layer, sequence, KV head) instance.
//
// Algorithm 1 (sampling line + final concatenation) and Algorithm 2 of the paper:
//   old region  [sink, sink + n_old)          keep offsets 0, s_hat, 2 s_hat, ...   (interval sampling)
//   new region  [sink + n_old, n - window)    per segment of s slots keep the top-h by
//                                             (score desc, position asc), in position order
//   sink [0, sink) and window [n - window, n) always kept.
// The counts depend only on n and n_old, so every destination offset is closed-form; only the
// winners inside each segment depend on the scores. A warp owns a segment: each lane holds the
// candidates lane, lane+32, ...; h rounds of a shuffle arg-max (ties -> lowest slot) flag the
// winners, and ballots + popcounts give their rank in position order.
//
// Compaction is an in-place stable left shift (destination <= source for every survivor): the
// CTA walks the destination rows in ascending chunks, reads a whole chunk's sources into
// registers, synchronises, then writes. A later chunk's sources lie at or beyond that chunk's
// first destination, so earlier writes never clobber them.
#include "buzz_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerPass = 4;   // rows of K and of V each 16-byte lane moves per pass

struct Cand {
  float v;
  int idx;   // slot index, -1 = none
};

__device__ inline Cand better(Cand a, Cand b) {
  // The winner is the larger score; equal scores go to the lower slot (= lower position).
  if (a.idx < 0) return b;
  if (b.idx < 0) return a;
  if (b.v > a.v || (b.v == a.v && b.idx < a.idx)) return b;
  return a;
}

template <int ROW_BYTES>
__global__ void __launch_bounds__(kThreads)
evict_kernel(BuzzState st, BuzzPolicy pol, int layer_begin, int max_batch, int kv_heads, int batch) {
  extern __shared__ int32_t src[];   // [budget] source slot of every destination slot
  const int head = blockIdx.x, seq = blockIdx.y, layer = layer_begin + blockIdx.z;
  if (seq >= batch) return;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int n = st.n[inst];
  const int n_old = st.n_old[inst];
  if (n < pol.budget) return;                       // threshold buffering: evict only when full
  if (n <= pol.sink + pol.window) return;           // Remark 1
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int s = pol.segment, h = pol.hitters, s_hat = pol.s_hat;
  const int new_begin = pol.sink + n_old;
  const int new_end = n - pol.window;
  const int n_new = new_end - new_begin;
  const int kept_old = (n_old + s_hat - 1) / s_hat;
  const int nseg = (n_new + s - 1) / s;
  const int last_len = n_new - (nseg - 1) * s;
  const int kept_new = nseg > 0 ? (nseg - 1) * h + min(h, last_len) : 0;
  const int kept_mid = kept_old + kept_new;
  const int n2 = pol.sink + kept_mid + pol.window;

  float* score = st.score + inst * pol.budget;
  int32_t* pos = st.pos + inst * pol.budget;

  // ---- selection: fill src[] ------------------------------------------------------------
  for (int t = tid; t < pol.sink; t += kThreads) src[t] = t;
  for (int t = tid; t < kept_old; t += kThreads) src[pol.sink + t] = pol.sink + t * s_hat;
  for (int t = tid; t < pol.window; t += kThreads) src[pol.sink + kept_mid + t] = new_end + t;
  for (int seg = warp; seg < nseg; seg += kThreads / 32) {
    const int lo = new_begin + seg * s;
    const int len = min(s, new_end - lo);
    const int want = min(h, len);
    const int out0 = pol.sink + kept_old + seg * h;
    if (pol.interval_new) {                         // ablation: the first `want` slots of the segment
      for (int r = lane; r < want; r += 32) src[out0 + r] = lo + r;
      continue;
    }
    unsigned chosen = 0;                            // bit i: candidate lo + i*32 + lane is a winner
    for (int r = 0; r < want; ++r) {
      Cand best{0.f, -1};
      for (int i = 0, j = lane; j < len; ++i, j += 32) {
        if (chosen >> i & 1u) continue;
        best = better(best, Cand{score[lo + j], lo + j});
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        Cand o;
        o.v = __shfl_xor_sync(0xffffffffu, best.v, off);
        o.idx = __shfl_xor_sync(0xffffffffu, best.idx, off);
        best = better(best, o);
      }
      const int w = best.idx - lo;
      if ((w & 31) == lane) chosen |= 1u << (w >> 5);
    }
    int before = 0;                                 // winners at lower positions
    for (int i = 0; i * 32 < len; ++i) {
      const bool mine = chosen >> i & 1u;
      const unsigned b = __ballot_sync(0xffffffffu, mine);
      if (mine) src[out0 + before + __popc(b & ((1u << lane) - 1u))] = lo + i * 32 + lane;
      before += __popc(b);
    }
  }
  __syncthreads();

  // ---- compaction of score and pos ------------------------------------------------------
  for (int base = 0; base < n2; base += kThreads) {
    const int t = base + tid;
    float sc = 0.f;
    int32_t ps = 0;
    if (t < n2) { sc = score[src[t]]; ps = pos[src[t]]; }
    __syncthreads();
    if (t < n2) { score[t] = sc; pos[t] = ps; }
  }

  // ---- compaction of the K and V rows ---------------------------------------------------
  constexpr int LPR = ROW_BYTES / 16;               // 16-byte lanes per row
  constexpr int ROWS = kThreads / LPR * kRowsPerPass;
  uint4* Kc = reinterpret_cast<uint4*>(st.K + inst * (size_t)pol.budget * ROW_BYTES);
  uint4* Vc = reinterpret_cast<uint4*>(st.V + inst * (size_t)pol.budget * ROW_BYTES);
  const int sub = tid % LPR, rgrp = tid / LPR;
  // Rows below `first` stay where they are (sink, and the first old survivor).
  const int first = pol.sink + (kept_old > 0 ? 1 : 0);
  for (int base = first; base < n2; base += ROWS) {
    uint4 kr[kRowsPerPass], vr[kRowsPerPass];
#pragma unroll
    for (int u = 0; u < kRowsPerPass; ++u) {
      const int t = base + u * (kThreads / LPR) + rgrp;
      if (t < n2) {
        const int sj = src[t];
        kr[u] = Kc[(size_t)sj * LPR + sub];
        vr[u] = Vc[(size_t)sj * LPR + sub];
      }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kRowsPerPass; ++u) {
      const int t = base + u * (kThreads / LPR) + rgrp;
      if (t < n2) {
        Kc[(size_t)t * LPR + sub] = kr[u];
        Vc[(size_t)t * LPR + sub] = vr[u];
      }
    }
  }

  if (tid == 0) {
    st.n[inst] = n2;
    st.n_old[inst] = kept_mid;
    if (n2 >= pol.budget) buzz_set_status(st.status, BUZZ_ERR_NO_PROGRESS, (int)inst, n2);
  }
}

}  // namespace

cudaError_t buzz_launch_evict(buzz_ctx* c, int layer_begin, int layer_count, cudaStream_t stream) {
  int batch = 0;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) batch = max(batch, c->batch[l]);
  if (batch == 0) return cudaSuccess;
  dim3 grid(c->sh.kv_heads, batch, layer_count);
  (void)cudaGetLastError();   // drop a stale non-sticky error left by an earlier runtime call of the process
  const size_t smem = (size_t)c->pol.budget * sizeof(int32_t);
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
