// BUZZ CPU oracle -- TEST INFRASTRUCTURE, not the product.
//
// A plain, slow, double-precision restatement of what the BUZZ hot path computes for ONE
// (layer, sequence, KV-head) instance: g query heads share one K/V cache of head dimension d.
// It exists so that the CUDA library can be checked against something written straight from
// the paper; nothing in the product path may call it, and it shares no code with the kernels.
//
// What follows the paper, and where:
//   * attention                : Eq. 3  (A = Softmax(Q K^T / sqrt(d)), O = A V); the token being
//                                decoded is appended first (Eq. 2), so it attends to itself.
//   * prefill cache            : Eq. 1  (the cache starts as the prompt's K, V).
//   * accumulated scores A     : input of Algorithm 2; read as the running sum of the softmax
//                                probabilities a key has received (column sums of the causal
//                                prefill probabilities, then += p at every decode step), summed
//                                over the g query heads of the group.
//   * eviction                 : Algorithm 1 (sink | old | new | window) with Algorithm 2
//                                (local-max sampling, stride s) on the new tokens and interval
//                                sampling with stride s_hat = floor((s+1)/2) on the old ones
//                                (Section 3.3, "BeeHive" and the sentence introducing Alg. 1/2).
//   * short sequences          : Remark 1 (nothing is evicted while n <= k + w).
//   * over-long prompts        : Remark 2 (sample repeatedly until the cache fits T + k + w).
//   * global top-k policy      : the heavy-hitter selection the paper compares against (Section 3.2:
//                                "top-k tokens based on attention scores A outside the sliding window";
//                                Section 4.3: a top-k module on accumulated scores "instead of the
//                                sampling module"). Read here as: at an eviction, sink and window
//                                stay, and of ALL middle tokens (old and new alike) the M with the
//                                largest accumulated score survive, M being the number the sampling
//                                module would have kept, so that both policies run on the same cache
//                                schedule. Ties go to the lowest position.
//   * log-n scaled attention   : Section 3.5 (logits scaled by log_512(n)/sqrt(d), n = tokens seen so
//                                far: row index + 1 at prefill, total length incl. the new token at
//                                decode -- not the number of retained slots).
//
// Readings taken where the paper is silent or inconsistent:
//   T is the capacity of the middle region, budget = T + k + w (Remark 2, Fig. 3 caption);
//   eviction fires when n >= budget; argmax ties go to the lowest position; a partial last
//   segment is a short segment; interval sampling keeps offsets 0, s_hat, 2 s_hat, ...;
//   `hitters` winners per segment are the top-h by (score desc, position asc), emitted in
//   position order; at prefill the first round treats everything between sink and window as new,
//   later rounds treat the survivors as old.
//
// Parity unpinned: the choice among those readings has no external pin (the authors' code is
// deliberately not consulted). Everything else is pinned by tests/test_oracle_*.py.
//
// Build: g++ -O2 -std=c++17 -shared -fPIC -o libbuzz_oracle.so buzz_oracle.cpp

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace {

struct Head {
  int g, d;
  int sink, window, segment, hitters, budget;
  int logn;            // 0: scale 1/sqrt(d) (Eq. 3); 1: scale log_512(n)/sqrt(d) (Section 3.5)
  int old_stride = 0;  // stride for old tokens; 0 = the paper's s_hat = floor((s+1)/2)
  int interval_new = 0;  // 1: interval sampling for new tokens too (the "no local max" ablation, Section 4.3)
  int global_topk = 0;   // 1: global top-k of the accumulated scores instead of the sampling module (Sections 3.2, 4.3)
  int n = 0, n_old = 0, total_len = 0;
  std::vector<double> K, V;   // [n][d], position order
  std::vector<double> score;  // [n]
  std::vector<int32_t> pos;   // [n] original token position
};

enum { BO_OK = 0, BO_BAD_ARG = -1, BO_OVERFLOW = -2, BO_NO_PROGRESS = -3 };

double logit_scale(const Head& h, int n_true) {
  double sc = 1.0 / std::sqrt((double)h.d);
  if (h.logn) sc *= std::log((double)n_true) / std::log(512.0);
  return sc;
}

// Softmax of `len` logits in place (Eq. 3), the textbook max-subtracted form.
void softmax_inplace(double* x, int len) {
  double mx = x[0];
  for (int j = 1; j < len; ++j) mx = std::max(mx, x[j]);
  double sum = 0.0;
  for (int j = 0; j < len; ++j) { x[j] = std::exp(x[j] - mx); sum += x[j]; }
  for (int j = 0; j < len; ++j) x[j] /= sum;
}

// The sampling module (Algorithm 1's sampling line; Algorithm 2): appends to `keep` the surviving
// middle slots, old region [k, k + n_old) first, then the new region [k + n_old, new_end).
void sample_middle(const Head& h, int s_hat, int new_end, std::vector<int>& keep) {
  const int k = h.sink, s = h.segment;
  for (int off = 0; off < h.n_old; off += s_hat) keep.push_back(k + off);  // interval_sample(s_hat, old)
  // local_max_sample(s, new): one hive per s consecutive new tokens
  for (int idx = k + h.n_old; idx < new_end; idx += s) {
    const int hi = std::min(idx + s, new_end);
    const int want = std::min(h.hitters, hi - idx);
    if (h.interval_new) {                 // ablation: the first `want` slots of the hive, scores ignored
      for (int r = 0; r < want; ++r) keep.push_back(idx + r);
      continue;
    }
    std::vector<int> chosen;
    for (int r = 0; r < want; ++r) {
      int best = -1;
      for (int j = idx; j < hi; ++j) {
        if (std::find(chosen.begin(), chosen.end(), j) != chosen.end()) continue;
        if (best < 0 || h.score[j] > h.score[best]) best = j;  // strict '>' => first occurrence wins ties
      }
      chosen.push_back(best);
    }
    std::sort(chosen.begin(), chosen.end());
    for (int j : chosen) keep.push_back(j);
  }
}

// The global top-k module (Sections 3.2 and 4.3): of all middle slots [k, new_end) the M with the
// largest accumulated score survive, M = the number sample_middle would keep.
void topk_middle(const Head& h, int s_hat, int new_end, std::vector<int>& keep) {
  const int k = h.sink, s = h.segment;
  int M = 0;
  for (int off = 0; off < h.n_old; off += s_hat) ++M;
  for (int idx = k + h.n_old; idx < new_end; idx += s) M += std::min(h.hitters, std::min(idx + s, new_end) - idx);
  // greedy heavy hitters: M times, take the best remaining middle token (first occurrence wins ties)
  std::vector<int> chosen;
  for (int r = 0; r < M; ++r) {
    int best = -1;
    for (int j = k; j < new_end; ++j) {
      if (std::find(chosen.begin(), chosen.end(), j) != chosen.end()) continue;
      if (best < 0 || h.score[j] > h.score[best]) best = j;
    }
    chosen.push_back(best);
  }
  std::sort(chosen.begin(), chosen.end());
  for (int j : chosen) keep.push_back(j);
}

// One eviction (Algorithm 1, the sampling line and the final concatenation; Algorithm 2).
// Returns 1 if the cache was rewritten, 0 if the trigger did not fire, <0 on error.
int evict_once(Head& h) {
  const int k = h.sink, w = h.window, s = h.segment;
  if (h.n < h.budget) return 0;          // threshold buffering: evict only when full
  if (h.n <= k + w) return 0;            // Remark 1: sink and window are filled first
  const int s_hat = h.old_stride > 0 ? h.old_stride : (s + 1) / 2;   // floor((s+1)/2) unless overridden (Section 4.3)
  const int new_end = h.n - w;

  std::vector<int> keep;
  for (int j = 0; j < k; ++j) keep.push_back(j);                       // K[:k]
  if (h.global_topk) topk_middle(h, s_hat, new_end, keep);
  else sample_middle(h, s_hat, new_end, keep);
  int kept_mid = (int)keep.size() - k;
  for (int j = new_end; j < h.n; ++j) keep.push_back(j);                // K[-w:]

  const int n2 = (int)keep.size();
  const bool progress = n2 < h.n;
  std::vector<double> K2((size_t)n2 * h.d), V2((size_t)n2 * h.d), sc2(n2);
  std::vector<int32_t> pos2(n2);
  for (int t = 0; t < n2; ++t) {
    const int j = keep[t];
    std::memcpy(&K2[(size_t)t * h.d], &h.K[(size_t)j * h.d], sizeof(double) * h.d);
    std::memcpy(&V2[(size_t)t * h.d], &h.V[(size_t)j * h.d], sizeof(double) * h.d);
    sc2[t] = h.score[j];
    pos2[t] = h.pos[j];
  }
  h.K.swap(K2); h.V.swap(V2); h.score.swap(sc2); h.pos.swap(pos2);
  h.n = n2;
  h.n_old = kept_mid;   // "all current tokens become the old tokens" (Fig. 3 caption)
  if (!progress) return BO_NO_PROGRESS;
  return 1;
}

}  // namespace

extern "C" {

void* bo_create(int g, int d, int sink, int window, int segment, int hitters, int budget, int logn) {
  if (g < 1 || d < 1 || sink < 0 || window < 1 || segment < 2 || hitters < 1 || hitters >= segment ||
      budget < sink + window + segment)
    return nullptr;
  Head* h = new Head();
  h->g = g; h->d = d; h->sink = sink; h->window = window; h->segment = segment;
  h->hitters = hitters; h->budget = budget; h->logn = logn;
  return h;
}

void bo_destroy(void* p) { delete (Head*)p; }

// Sampling variants of the ablation study (Section 4.3): interval sampling for new tokens as well,
// and free choice of the two strides (e.g. swapped). new_stride replaces s, old_stride replaces s_hat.
int bo_set_sampling(void* p, int interval_new, int new_stride, int old_stride) {
  Head& h = *(Head*)p;
  if (new_stride < 2 || h.hitters >= new_stride || old_stride < 1 || h.budget < h.sink + h.window + new_stride)
    return BO_BAD_ARG;
  h.segment = new_stride;
  h.old_stride = old_stride;
  h.interval_new = interval_new ? 1 : 0;
  return BO_OK;
}

// Selects the eviction policy: 0 = BUZZ's sampling module (Algorithms 1 and 2), 1 = global top-k of
// the accumulated scores over the whole middle region (the heavy-hitter baseline, Sections 3.2, 4.3).
int bo_set_policy(void* p, int policy) {
  if (policy != 0 && policy != 1) return BO_BAD_ARG;
  ((Head*)p)->global_topk = policy;
  return BO_OK;
}

// Causal prefill (Eqs. 1 and 3) + initial scores + Remark 2's repeated sampling.
//   Q [g][N][d], K [N][d], V [N][d] -> O [g][N][d]; full_score [N] (may be null) receives the
//   column sums before any eviction. Returns the number of eviction rounds, or <0.
int bo_prefill(void* p, int N, const double* Q, const double* K, const double* V, double* O,
               double* full_score) {
  Head& h = *(Head*)p;
  if (N < 1) return BO_BAD_ARG;
  const int d = h.d, g = h.g;
  std::vector<double> colsum(N, 0.0), row(N);
  for (int q = 0; q < g; ++q) {
    for (int i = 0; i < N; ++i) {
      const double sc = logit_scale(h, i + 1);
      const double* qi = Q + ((size_t)q * N + i) * d;
      for (int j = 0; j <= i; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += qi[c] * K[(size_t)j * d + c];
        row[j] = dot * sc;
      }
      softmax_inplace(row.data(), i + 1);
      double* oi = O + ((size_t)q * N + i) * d;
      for (int c = 0; c < d; ++c) oi[c] = 0.0;
      for (int j = 0; j <= i; ++j) {
        colsum[j] += row[j];
        for (int c = 0; c < d; ++c) oi[c] += row[j] * V[(size_t)j * d + c];
      }
    }
  }
  if (full_score) std::memcpy(full_score, colsum.data(), sizeof(double) * N);
  h.K.assign(K, K + (size_t)N * d);
  h.V.assign(V, V + (size_t)N * d);
  h.score = colsum;
  h.pos.resize(N);
  for (int j = 0; j < N; ++j) h.pos[j] = j;
  h.n = N; h.n_old = 0; h.total_len = N;
  int rounds = 0;
  while (h.n >= h.budget) {
    int r = evict_once(h);
    if (r < 0) return r;
    ++rounds;
  }
  return rounds;
}

// One decode step (Eqs. 2 and 3): append, attend over all retained slots, add p to the scores.
//   q [g][d], k [d], v [d] -> o [g][d].
int bo_decode(void* p, const double* q, const double* k, const double* v, double* o) {
  Head& h = *(Head*)p;
  if (h.n >= h.budget) return BO_OVERFLOW;
  const int d = h.d;
  h.K.insert(h.K.end(), k, k + d);
  h.V.insert(h.V.end(), v, v + d);
  h.score.push_back(0.0);
  h.pos.push_back(h.total_len);
  h.n += 1; h.total_len += 1;
  const double sc = logit_scale(h, h.total_len);
  std::vector<double> pr(h.n);
  for (int qh = 0; qh < h.g; ++qh) {
    for (int j = 0; j < h.n; ++j) {
      double dot = 0.0;
      for (int c = 0; c < d; ++c) dot += q[(size_t)qh * d + c] * h.K[(size_t)j * d + c];
      pr[j] = dot * sc;
    }
    softmax_inplace(pr.data(), h.n);
    for (int c = 0; c < d; ++c) o[(size_t)qh * d + c] = 0.0;
    for (int j = 0; j < h.n; ++j) {
      h.score[j] += pr[j];
      for (int c = 0; c < d; ++c) o[(size_t)qh * d + c] += pr[j] * h.V[(size_t)j * d + c];
    }
  }
  return BO_OK;
}

int bo_evict(void* p) { return evict_once(*(Head*)p); }

void bo_get_counts(void* p, int* n, int* n_old, int* total_len) {
  Head& h = *(Head*)p;
  *n = h.n; *n_old = h.n_old; *total_len = h.total_len;
}

// Copies out whatever pointers are non-null: pos [n], score [n], K [n][d], V [n][d].
void bo_get_state(void* p, int32_t* pos, double* score, double* K, double* V) {
  Head& h = *(Head*)p;
  if (pos) std::memcpy(pos, h.pos.data(), sizeof(int32_t) * h.n);
  if (score) std::memcpy(score, h.score.data(), sizeof(double) * h.n);
  if (K) std::memcpy(K, h.K.data(), sizeof(double) * (size_t)h.n * h.d);
  if (V) std::memcpy(V, h.V.data(), sizeof(double) * (size_t)h.n * h.d);
}

// Overwrites the n running scores (used by the lock-step protocol: the decision of an argmax is
// then taken on exactly the values the other side holds).
void bo_set_scores(void* p, const double* score) {
  Head& h = *(Head*)p;
  std::memcpy(h.score.data(), score, sizeof(double) * h.n);
}

// Loads a cache state directly (no prefill): pos/score/K/V of n slots, of which n_old are "old".
int bo_set_state(void* p, int n, int n_old, int total_len, const int32_t* pos, const double* score,
                 const double* K, const double* V) {
  Head& h = *(Head*)p;
  if (n < 0 || n_old < 0 || n_old > n) return BO_BAD_ARG;   // n may exceed the budget (a prompt)
  h.n = n; h.n_old = n_old; h.total_len = total_len;
  h.pos.assign(pos, pos + n);
  h.score.assign(score, score + n);
  h.K.assign(K, K + (size_t)n * h.d);
  h.V.assign(V, V + (size_t)n * h.d);
  return BO_OK;
}

}  // extern "C"
