// Prefill-time eviction and cache fill (Remark 2 of the paper): "sample repeatedly until the
// selected tokens fit within a container of length T + k + w", then gather the survivors' K, V,
// score and position from the packed prompt tensors into the layer's cache.
//
// The first round is Algorithm 2 (segment-wise top-h over everything between sink and window);
// every later round sees only "old" tokens and keeps offsets 0, s_hat, 2 s_hat, ... of the
// survivors. Counts never depend on the scores, so after R rounds the f-th middle survivor is
// the (f * s_hat^(R-1))-th winner of round one: destination slots are closed-form and the gather
// is embarrassingly parallel -- each 16-lane group resolves its own slot's source token (rescanning
// one segment of <= s scores) and copies that row. The cache is laid out [sink | window ring |
// middle] (cache_ops.cuh): the prompt's last `window` tokens fill the ring in order (head 0) and
// the survivors between sink and window follow it.
// Under the global top-k policy the rounds are nested (the heaviest M2 of the heaviest M1 are the
// heaviest M2), so the middle survivors are simply the n_mid heaviest prompt tokens between sink
// and window: one CTA per instance selects them first and leaves their token indices in the cache's
// position array, where the gather then finds its sources.
#include "cache_ops.cuh"

namespace {

constexpr int kThreads = 256;

struct FillPlan {
  int rounds;      // eviction rounds (0 = prompt shorter than the budget: keep everything)
  int n_mid;       // survivors between sink and window after the last round
  long stride;     // s_hat^(rounds-1): distance, in round-one winners, between final survivors
  int n_final;     // retained slots
  int error;       // nonzero: the rounds cannot shrink the cache (s_hat == 1)
};

__device__ inline FillPlan make_plan(int N, const BuzzPolicy& pol) {
  FillPlan p{0, 0, 1, N, 0};
  if (N < pol.budget || N <= pol.sink + pol.window) { p.n_mid = max(N - pol.sink - pol.window, 0); return p; }
  const int n_new = N - pol.sink - pol.window;
  const int nseg = (n_new + pol.segment - 1) / pol.segment;
  const int last_len = n_new - (nseg - 1) * pol.segment;
  int mid = (nseg - 1) * pol.hitters + min(pol.hitters, last_len);
  p.rounds = 1;
  while (pol.sink + mid + pol.window >= pol.budget) {
    if (pol.s_hat <= 1 || p.rounds > 40) { p.error = 1; break; }
    mid = (mid + pol.s_hat - 1) / pol.s_hat;
    p.stride *= pol.s_hat;
    p.rounds += 1;
  }
  p.n_mid = mid;
  p.n_final = pol.sink + mid + pol.window;
  return p;
}

// Source token (relative to the sequence start) of round-one winner m1: the (m1 % h)-th, in
// position order, of the top-h of segment m1 / h. Ties go to the lower position.
__device__ inline int round_one_winner(const float* __restrict__ sc, int N, const BuzzPolicy& pol, int m1) {
  const int seg = m1 / pol.hitters, rank = m1 % pol.hitters;
  const int lo = pol.sink + seg * pol.segment;
  const int hi = min(lo + pol.segment, N - pol.window);
  const int want = min(pol.hitters, hi - lo);
  if (pol.interval_new) return lo + rank;           // ablation: interval sampling, scores ignored
  if (want == 1) {
    int best = lo;
    float bv = sc[lo];
    for (int j = lo + 1; j < hi; ++j) {
      const float v = sc[j];
      if (v > bv) { bv = v; best = j; }
    }
    return best;
  }
  // general case: j is among the top `want` iff fewer than `want` candidates beat it
  int seen = 0;
  for (int j = lo; j < hi; ++j) {
    const float vj = sc[j];
    int beat = 0;
    for (int i = lo; i < hi; ++i) {
      const float vi = sc[i];
      beat += (vi > vj || (vi == vj && i < j)) ? 1 : 0;
    }
    if (beat < want) {
      if (seen == rank) return j;
      ++seen;
    }
  }
  return lo;   // unreachable for NaN-free scores
}

// Global top-k policy: the middle survivors of one instance, in position order, into pos[middle slots].
__global__ void __launch_bounds__(kThreads)
prefill_topk_kernel(BuzzState st, BuzzPolicy pol, const int32_t* __restrict__ cu, const float* __restrict__ pscore,
                    int stride, int layer, int max_batch, int kv_heads) {
  const int head = blockIdx.x, seq = blockIdx.y;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int tok0 = cu[seq], N = cu[seq + 1] - tok0;
  const FillPlan plan = make_plan(N, pol);
  if (plan.error || plan.rounds == 0) return;
  int32_t* mid_pos = st.pos + inst * (size_t)pol.budget + buzz_dev::middle_begin(pol);
  buzz_dev::topk_select<kThreads>(pscore + (size_t)head * stride + tok0 + pol.sink, N - pol.sink - pol.window,
                                  plan.n_mid, [&](int t, int j) { mid_pos[t] = pol.sink + j; });
}

template <int ROW_BYTES>
__global__ void __launch_bounds__(kThreads)
prefill_fill_kernel(BuzzState st, BuzzPolicy pol, const char* __restrict__ k, const char* __restrict__ v,
                    const int32_t* __restrict__ cu, const float* __restrict__ pscore, int stride,
                    int layer, int max_batch, int kv_heads) {
  constexpr int LPR = ROW_BYTES / 16;
  constexpr int SLOTS = kThreads / LPR;              // slots per CTA pass
  const int head = blockIdx.y, seq = blockIdx.z;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int tok0 = cu[seq], N = cu[seq + 1] - tok0;
  const FillPlan plan = make_plan(N, pol);
  const int tid = threadIdx.x, sub = tid % LPR, grp = tid / LPR;
  if (blockIdx.x == 0 && tid == 0) {
    if (plan.error) {
      buzz_set_status(st.status, BUZZ_ERR_NO_PROGRESS, (int)inst, N);
      st.n[inst] = 0; st.n_old[inst] = 0; st.total[inst] = N; st.ring[inst] = 0;
    } else {
      st.ring[inst] = 0;
      st.n[inst] = plan.n_final;
      st.n_old[inst] = plan.rounds > 0 ? plan.n_mid : 0;
      st.total[inst] = N;
    }
  }
  if (plan.error) return;
  const float* sc = pscore + (size_t)head * stride + tok0;
  const size_t cache_row0 = inst * (size_t)pol.budget;
  for (int t = blockIdx.x * SLOTS + grp; t < plan.n_final; t += gridDim.x * SLOTS) {
    int src;
    if (plan.rounds == 0 || t < pol.sink) src = t;
    else if (t < pol.sink + plan.n_mid)
      src = pol.policy == BUZZ_POLICY_GLOBAL_TOPK ? st.pos[cache_row0 + t + pol.window]   // left there by prefill_topk_kernel
                                                  : round_one_winner(sc, N, pol, (int)((t - pol.sink) * plan.stride));
    else src = N - pol.window + (t - pol.sink - plan.n_mid);
    // t counts the survivors in position order; their slots: sink, then (behind the ring) the middle,
    // and the last `window` tokens in the ring right after the sink
    const int slot = t < pol.sink ? t : (t < pol.sink + plan.n_mid ? t + pol.window : t - plan.n_mid);
    const size_t g = ((size_t)(tok0 + src) * kv_heads + head) * LPR + sub;
    const size_t d = (cache_row0 + slot) * LPR + sub;
    reinterpret_cast<uint4*>(st.K)[d] = __ldg(reinterpret_cast<const uint4*>(k) + g);
    reinterpret_cast<uint4*>(st.V)[d] = __ldg(reinterpret_cast<const uint4*>(v) + g);
    if (sub == 0) {
      st.score[cache_row0 + slot] = sc[src];
      st.pos[cache_row0 + slot] = src;
    }
  }
}

}  // namespace

cudaError_t buzz_launch_prefill_fill(buzz_ctx* c, int layer, const void* k, const void* v,
                                     const int32_t* cu, int batch, int max_seqlen,
                                     cudaStream_t stream) {
  const int row_bytes = c->sh.head_dim * (int)c->esize;
  const int lpr = row_bytes / 16;
  const int slots = kThreads / lpr;
  const int n_max = max_seqlen < c->pol.budget ? max_seqlen : c->pol.budget;
  int bx = (n_max + slots - 1) / slots;
  if (bx < 1) bx = 1;
  dim3 grid(bx, c->sh.kv_heads, batch);
  (void)cudaGetLastError();   // drop a stale non-sticky error left by an earlier runtime call of the process
  if (c->pol.policy == BUZZ_POLICY_GLOBAL_TOPK) {
    prefill_topk_kernel<<<dim3(c->sh.kv_heads, batch), kThreads, 0, stream>>>(
        c->st, c->pol, cu, c->pscore, c->sh.max_prompt_tokens, layer, c->sh.max_batch, c->sh.kv_heads);
    c->launches += 1;
    if (cudaError_t e = cudaGetLastError(); e != cudaSuccess) return e;
  }
#define BUZZ_FILL_CASE(RB)                                                                      \
  case RB:                                                                                      \
    prefill_fill_kernel<RB><<<grid, kThreads, 0, stream>>>(                                     \
        c->st, c->pol, (const char*)k, (const char*)v, cu, c->pscore, c->sh.max_prompt_tokens,  \
        layer, c->sh.max_batch, c->sh.kv_heads);                                                \
    break;
  switch (row_bytes) {
    BUZZ_FILL_CASE(128)
    BUZZ_FILL_CASE(256)
    BUZZ_FILL_CASE(512)
    default: return cudaErrorInvalidValue;
  }
#undef BUZZ_FILL_CASE
  c->launches += 1;
  c->last_kind = 2;
  return cudaGetLastError();
}
