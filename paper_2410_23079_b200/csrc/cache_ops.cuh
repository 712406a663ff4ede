// Device-side operations on one instance's cache that more than one kernel needs: where an appended
// token goes (Eq. 2 of the paper), and the BUZZ eviction of one instance (Algorithm 1's sampling
// line and concatenation, Algorithm 2). Not part of the public ABI.
//
// Slot layout of an instance (budget slots, of which [0, n) are occupied):
//   [0, sink)                    the first `sink` tokens                        (attention sink)
//   [sink, sink + window)        the last `window` tokens, kept as a RING: ring index `head` holds the
//                                oldest of them once the ring is full; while it is filling, tokens sit
//                                at ring indices 0, 1, ... in order and head is 0
//   [sink + window, n)           the middle region in position order: n_old survivors of earlier
//                                evictions ("old"), then the tokens that have left the window since
//                                the last eviction ("new")
// Appending a token to a full ring replaces the oldest window token, which moves to slot n (the end
// of the new tokens); an eviction therefore rewrites the middle region only and never moves the
// window or the sink. Position order of the retained tokens is sink, middle, ring from `head` on.
#pragma once

#include "buzz_internal.cuh"

namespace buzz_dev {

__host__ __device__ inline int middle_begin(const BuzzPolicy& p) { return p.sink + p.window; }

// Where the token appended at this step goes. slot_moved >= 0: the ring is full, the oldest window
// token leaves slot_new for slot_moved (= n0) first.
struct AppendPlan {
  int slot_new;
  int slot_moved;
  int head_next;
};
__device__ inline AppendPlan plan_append(const BuzzPolicy& pol, int n0, int head) {
  AppendPlan a;
  if (n0 < pol.sink + pol.window) {
    a.slot_new = n0; a.slot_moved = -1; a.head_next = head;
  } else {
    a.slot_new = pol.sink + head; a.slot_moved = n0; a.head_next = (head + 1 == pol.window) ? 0 : head + 1;
  }
  return a;
}

// Writes the appended token's K and V rows and position (and moves the token that leaves the window,
// if any: its K, V and position; its score travels with the score update of the step). Called by
// threads 0 .. 2*LPR of ONE CTA after every reader of the old rows is done. LPR = 16-byte lanes per row.
template <int LPR>
__device__ inline void append_rows(const BuzzState& st, const BuzzPolicy& pol, size_t inst, const AppendPlan& a,
                                   int tot, const uint4* __restrict__ knew, const uint4* __restrict__ vnew, int tid) {
  uint4* Kc = reinterpret_cast<uint4*>(st.K) + inst * (size_t)pol.budget * LPR;
  uint4* Vc = reinterpret_cast<uint4*>(st.V) + inst * (size_t)pol.budget * LPR;
  int32_t* pos = st.pos + inst * pol.budget;
  if (tid < LPR) {
    if (a.slot_moved >= 0) Kc[(size_t)a.slot_moved * LPR + tid] = Kc[(size_t)a.slot_new * LPR + tid];
    Kc[(size_t)a.slot_new * LPR + tid] = knew[tid];
  } else if (tid < 2 * LPR) {
    const int t = tid - LPR;
    if (a.slot_moved >= 0) Vc[(size_t)a.slot_moved * LPR + t] = Vc[(size_t)a.slot_new * LPR + t];
    Vc[(size_t)a.slot_new * LPR + t] = vnew[t];
  } else if (tid == 2 * LPR) {
    if (a.slot_moved >= 0) pos[a.slot_moved] = pos[a.slot_new];
    pos[a.slot_new] = tot;
  }
}

// The same stores from rows staged in shared memory by the calling threads themselves: stage[0, LPR)
// and [LPR, 2 LPR) hold the K and V rows of the token that leaves the window (if any), the next 2 LPR
// entries the appended token's K and V rows, *stage_pos the leaving token's position. Thread t reads
// only what thread t staged, so no barrier is needed between staging and this call.
template <int LPR>
__device__ inline void append_staged(const BuzzState& st, const BuzzPolicy& pol, size_t inst, const AppendPlan& a,
                                     int tot, const uint4* stage, const int32_t* stage_pos, int tid) {
  int32_t* pos = st.pos + inst * pol.budget;
  if (tid < 2 * LPR) {
    uint4* cache = reinterpret_cast<uint4*>(tid < LPR ? st.K : st.V) + inst * (size_t)pol.budget * LPR;
    const int t = tid < LPR ? tid : tid - LPR;
    if (a.slot_moved >= 0) cache[(size_t)a.slot_moved * LPR + t] = stage[tid];
    cache[(size_t)a.slot_new * LPR + t] = stage[2 * LPR + tid];
  } else if (tid == 2 * LPR) {
    if (a.slot_moved >= 0) pos[a.slot_moved] = *stage_pos;
    pos[a.slot_new] = tot;
  }
}

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

// Order-preserving key of a score: a larger float gives a larger unsigned integer (-0 counts as +0).
__device__ inline uint32_t order_key(float v) {
  const uint32_t b = __float_as_uint(v + 0.0f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Global top-M selection by one whole CTA (the heavy-hitter policy the paper compares against,
// Sections 3.2 and 4.3): of cand[0 .. count) the M largest survive, equal scores going to the lowest
// index; emit(t, j) is called once per survivor, t = its rank in index order, j = its index.
// Exact and deterministic: a four-pass radix select (8 bits per pass, shared-memory histogram with
// warp-aggregated increments) finds the M-th largest key and how many keys equal to it survive; one
// ordered pass over the candidates then hands out the ranks with ballots and popcounts.
template <int THREADS, typename Emit>
__device__ void topk_select(const float* __restrict__ cand, int count, int M, Emit emit) {
  __shared__ int hist[256];
  __shared__ int warp_cnt[2][THREADS / 32];
  __shared__ uint32_t found_prefix;
  __shared__ int found_remaining;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (M <= 0) return;
  if (M >= count) {
    for (int j = tid; j < count; j += THREADS) emit(j, j);
    return;
  }
  uint32_t prefix = 0, mask = 0;
  int remaining = M;                       // survivors still to be found among the keys matching `prefix`
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += THREADS) hist[i] = 0;
    __syncthreads();
    for (int base = 0; base < count; base += THREADS) {
      const int j = base + tid;
      int bin = -1;
      if (j < count) {
        const uint32_t key = order_key(cand[j]);
        if ((key & mask) == prefix) bin = (int)((key >> shift) & 255u);
      }
      const unsigned peers = __match_any_sync(0xffffffffu, bin);
      if (bin >= 0 && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
    }
    __syncthreads();
    if (warp == 0) {                       // lane l owns bins 8l .. 8l+7; walk from the top bin down
      int c[8], mine = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { c[i] = hist[8 * lane + i]; mine += c[i]; }
      int incl = mine;                     // keys in this lane's bins and all higher lanes' bins
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
      }
      int cum = incl - mine;               // keys in strictly higher bins than this lane's
#pragma unroll
      for (int i = 7; i >= 0; --i) {
        if (cum < remaining && cum + c[i] >= remaining) {
          found_prefix = prefix | ((uint32_t)(8 * lane + i) << shift);
          found_remaining = remaining - cum;
        }
        cum += c[i];
      }
    }
    __syncthreads();
    prefix = found_prefix;
    remaining = found_remaining;
    mask |= 255u << shift;
  }
  // prefix is now the M-th largest key; `remaining` of the keys equal to it survive, lowest index first
  int eq_base = 0, out_base = 0;
  for (int base = 0; base < count; base += THREADS) {
    const int j = base + tid;
    bool gt = false, eq = false;
    if (j < count) {
      const uint32_t key = order_key(cand[j]);
      gt = key > prefix;
      eq = key == prefix;
    }
    const unsigned lower = (1u << lane) - 1u;
    const unsigned be = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) warp_cnt[0][warp] = __popc(be);
    __syncthreads();
    int eq_before = eq_base + __popc(be & lower), eq_total = 0;
#pragma unroll
    for (int w = 0; w < THREADS / 32; ++w) {
      if (w < warp) eq_before += warp_cnt[0][w];
      eq_total += warp_cnt[0][w];
    }
    const bool take = gt || (eq && eq_before < remaining);
    const unsigned bt = __ballot_sync(0xffffffffu, take);
    if (lane == 0) warp_cnt[1][warp] = __popc(bt);
    __syncthreads();
    int out = out_base + __popc(bt & lower), take_total = 0;
#pragma unroll
    for (int w = 0; w < THREADS / 32; ++w) {
      if (w < warp) out += warp_cnt[1][w];
      take_total += warp_cnt[1][w];
    }
    if (take) emit(out, j);
    eq_base += eq_total;
    out_base += take_total;
  }
}

// Shared memory one eviction needs: the source-slot list, and (when it fits) a staged copy of the
// middle region's scores and positions, so that the selection reads no global memory at all.
constexpr int kEvictStageLimit = 5440;        // middle-region capacity up to which scores and positions are staged
__host__ __device__ inline bool evict_staged(const BuzzPolicy& p) { return p.budget - middle_begin(p) <= kEvictStageLimit; }
__host__ __device__ inline size_t evict_smem_bytes(const BuzzPolicy& p) {
  return (size_t)(p.budget - middle_begin(p)) * 4u * (evict_staged(p) ? 3u : 1u);
}

// One eviction of one instance by one whole CTA of THREADS threads (all of them must call it; the
// trigger n >= budget and Remark 1's n > sink + window are the caller's to check).
//   old region  [mb, mb + n_old)   keep offsets 0, s_hat, 2 s_hat, ...          (interval sampling)
//   new region  [mb + n_old, n)    per segment of s slots keep the top-h by (score desc, position asc),
//                                  in position order                            (Algorithm 2)
// with mb = sink + window. The counts depend only on n and n_old, so every destination is closed-form;
// only the winners inside a segment depend on the scores. The middle region's scores and positions
// are first copied to shared memory with coalesced loads (one memory latency instead of one per
// segment). A warp owns a segment: each lane holds the candidates lane, lane+32, ...; h rounds of a
// shuffle arg-max flag the winners, ballots + popcounts give their rank in position order. Under the
// global top-k policy the same number of survivors is taken from the whole middle region by score
// alone (topk_select). Compaction is an in-place stable left shift (destination <= source):
// ascending chunks, a chunk's sources read into registers, a barrier, then the writes.
// `work` is shared memory of evict_smem_bytes(pol) bytes.
template <int ROW_BYTES, int THREADS>
__device__ void evict_instance(const BuzzState& st, const BuzzPolicy& pol, size_t inst, int n, int n_old,
                               int32_t* work) {
  constexpr int kRowsPerPass = 2;   // rows of K and of V each 16-byte lane holds per register set (two sets in flight)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int s = pol.segment, h = pol.hitters, s_hat = pol.s_hat;
  const int mb = middle_begin(pol);
  const int cap = pol.budget - mb;                   // capacity of the middle region
  const int m = n - mb;                              // its occupancy
  const int new_begin = mb + n_old;
  const int n_new = n - new_begin;
  const int kept_old = (n_old + s_hat - 1) / s_hat;
  const int nseg = (n_new + s - 1) / s;
  const int last_len = n_new - (nseg - 1) * s;
  const int kept_new = nseg > 0 ? (nseg - 1) * h + min(h, last_len) : 0;
  const int kept_mid = kept_old + kept_new;
  const bool staged = evict_staged(pol);

  float* score = st.score + inst * pol.budget;
  int32_t* pos = st.pos + inst * pol.budget;
  int32_t* src = work;
  float* sc_s = reinterpret_cast<float*>(work + cap);
  int32_t* pos_s = work + 2 * cap;
  if (staged) {
    for (int j = tid; j < m; j += THREADS) { sc_s[j] = score[mb + j]; pos_s[j] = pos[mb + j]; }
    __syncthreads();
  }
  const float* sc = staged ? sc_s - mb : score;      // sc[slot] for slots of the middle region

  // ---- selection: src[t] = source slot of middle destination mb + t ---------------------------
  if (pol.policy == BUZZ_POLICY_GLOBAL_TOPK) {
    topk_select<THREADS>(sc + mb, m, kept_mid, [&](int t, int j) { src[t] = mb + j; });
  } else {
    for (int t = tid; t < kept_old; t += THREADS) src[t] = mb + t * s_hat;
    for (int seg = warp; seg < nseg; seg += THREADS / 32) {
      const int lo = new_begin + seg * s;
      const int len = min(s, n - lo);
      const int want = min(h, len);
      const int out0 = kept_old + seg * h;
      if (pol.interval_new) {                         // ablation: the first `want` slots of the segment
        for (int r = lane; r < want; r += 32) src[out0 + r] = lo + r;
        continue;
      }
      unsigned chosen = 0;                            // bit i: candidate lo + i*32 + lane is a winner
      for (int r = 0; r < want; ++r) {
        Cand best{0.f, -1};
        for (int i = 0, j = lane; j < len; ++i, j += 32) {
          if (chosen >> i & 1u) continue;
          best = better(best, Cand{sc[lo + j], lo + j});
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
  }
  __syncthreads();

  // ---- compaction of score and pos ------------------------------------------------------------
  if (staged) {                                      // sources are the shared-memory copies: no hazard
    for (int t = tid; t < kept_mid; t += THREADS) {
      const int j = src[t] - mb;
      score[mb + t] = sc_s[j];
      pos[mb + t] = pos_s[j];
    }
  } else {
    for (int base = 0; base < kept_mid; base += THREADS) {
      const int t = base + tid;
      float v = 0.f;
      int32_t ps = 0;
      if (t < kept_mid) { v = score[src[t]]; ps = pos[src[t]]; }
      __syncthreads();
      if (t < kept_mid) { score[mb + t] = v; pos[mb + t] = ps; }
    }
  }

  // ---- compaction of the K and V rows ---------------------------------------------------------
  constexpr int LPR = ROW_BYTES / 16;               // 16-byte lanes per row
  constexpr int ROWS = THREADS / LPR * kRowsPerPass;
  uint4* Kc = reinterpret_cast<uint4*>(st.K + inst * (size_t)pol.budget * ROW_BYTES);
  uint4* Vc = reinterpret_cast<uint4*>(st.V + inst * (size_t)pol.budget * ROW_BYTES);
  const int sub = tid % LPR, rgrp = tid / LPR;
  // Under the sampling policy the first old survivor stays where it is. The loop is software-pipelined
  // over two register sets: a chunk's destinations lie in front of every later chunk's sources
  // (destination mb + t <= mb + t' <= src[t'] for t < t'), so the NEXT chunk's loads may be issued before
  // this chunk is written; only a chunk's own loads have to be done (the barrier) before its stores.
  auto load_rows = [&](int base, uint4 (&kr)[kRowsPerPass], uint4 (&vr)[kRowsPerPass]) {
#pragma unroll
    for (int u = 0; u < kRowsPerPass; ++u) {
      const int t = base + u * (THREADS / LPR) + rgrp;
      if (t < kept_mid) {
        const int sj = src[t];
        kr[u] = Kc[(size_t)sj * LPR + sub];
        vr[u] = Vc[(size_t)sj * LPR + sub];
      }
    }
  };
  auto store_rows = [&](int base, const uint4 (&kr)[kRowsPerPass], const uint4 (&vr)[kRowsPerPass]) {
#pragma unroll
    for (int u = 0; u < kRowsPerPass; ++u) {
      const int t = base + u * (THREADS / LPR) + rgrp;
      if (t < kept_mid) {
        Kc[(size_t)(mb + t) * LPR + sub] = kr[u];
        Vc[(size_t)(mb + t) * LPR + sub] = vr[u];
      }
    }
  };
  uint4 ka[kRowsPerPass], va[kRowsPerPass], kb[kRowsPerPass], vb[kRowsPerPass];
  int base = (kept_old > 0 && pol.policy != BUZZ_POLICY_GLOBAL_TOPK) ? 1 : 0;
  load_rows(base, ka, va);
  while (base < kept_mid) {                          // uniform over the CTA
    load_rows(base + ROWS, kb, vb);
    __syncthreads();
    store_rows(base, ka, va);
    base += ROWS;
    if (base >= kept_mid) break;
    load_rows(base + ROWS, ka, va);
    __syncthreads();
    store_rows(base, kb, vb);
    base += ROWS;
  }

  if (tid == 0) {
    const int n2 = mb + kept_mid;
    st.n[inst] = n2;
    st.n_old[inst] = kept_mid;
    if (n2 >= pol.budget) buzz_set_status(st.status, BUZZ_ERR_NO_PROGRESS, (int)inst, n2);
  }
}

}  // namespace buzz_dev
