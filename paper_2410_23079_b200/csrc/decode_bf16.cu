// BUZZ decode step for bf16 caches: the same cluster-per-instance, two-phase structure as the
// fp32 kernel (decode.cu), with both contractions on the tensor cores so that the instruction
// stream stays far below the issue limit while K and V stream from HBM at full width.
//
// Per step and instance the work is Eq. 3 of the paper for up to 8 query heads that share one KV
// head: logits q.K^T/sqrt(d), softmax, output p.V, and score += sum over heads of p (Algorithm 2's
// accumulated attention). Both products are written "transposed" so that the long index (keys,
// then output dims) sits on the 16-row side of the m16n8k16 MMA and the heads on the 8-column
// side; every fragment is then built from plain 16-byte global loads, with no shared-memory
// staging and no cross-lane shuffles:
//   phase 1  S^T[16 keys x 8 heads] = K[16 keys x d] . Q^T[d x 8 heads]
//            lane (r = lane/4, c = lane%4) loads 16-byte chunk c+4i of key rows r and r+8; the four
//            32-bit words of a chunk feed two MMAs (the contraction order over d is a fixed
//            permutation applied to K and Q alike). Logits go to shared memory; per-head maxima.
//   phase 2  O^T[16 dims x 8 heads] += V^T[16 dims x 16 keys] . P^T[16 keys x 8 heads]
//            lane loads chunk r+8j of key rows 2c, 2c+1, 2c+8, 2c+9 and interleaves two rows' words
//            with one byte-permute per operand register; P = 2^(S - max) rounded to bf16 for the
//            product, summed in fp32 for the normaliser.
//   combine  as in decode.cu: partial (max, sum, output) per CTA in shared memory, one cluster
//            barrier, exact probabilities of the CTA's own chunk added to the scores, CTA 0 writes
//            the output. No global scratch, no atomics, fixed-order reductions.
//   append   after the barrier (every reader of the old rows is done) CTA 0 stores the new token: into
//            the window ring, whose oldest token first moves to the end of the middle region (see
//            cache_ops.cuh); that token's score moves with the score update.
//   evict    (fused mode) if the step filled the cache, CTA 0 runs the instance's eviction in the
//            kernel's tail, so no separate eviction launch is needed.
#include <cooperative_groups.h>

#include "cache_ops.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxCluster = 8;
constexpr int kHeads = 8;       // MMA column count: query heads of one group, zero-padded
constexpr int kTile = 16;       // keys per warp tile
constexpr int kPrefetchLines = 256;   // 128-byte lines of K a CTA may pull towards L2 before its wait (measured best)
enum { kWaitFirst = 0, kHintFirst = 1, kOverlap = 2 };
constexpr int kAhead = 2;   // rolling L2 prefetch runs this many loop iterations (kWarps * kTile rows each) ahead of the register loads (measured best of 0..5)

__device__ inline uint4 ld_stream(const uint4* p) { return __ldcs(p); }

// Asynchronous global -> shared copies (no register, no stall at issue); a thread that later reads
// what it copied itself only needs its own cp_async_wait().
__device__ inline void cp_async16(void* dst_smem, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ inline void cp_async4(void* dst_smem, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src) : "memory");
}
__device__ inline void cp_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ inline void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ inline uint32_t word(const uint4& v, int i) {
  return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

__device__ inline uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&p);
}

template <int D>
constexpr int kStageBytes = 4 * (D / 8) * 16 + 16;

template <int G, int D>
struct Partial {       // what a CTA publishes to its cluster
  float m[G];          // chunk-local max of the log2-domain logits
  float l[G];          // sum of 2^(logit - m) over the chunk
  float o[G][D];       // sum of 2^(logit - m) * V over the chunk
};

template <int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_bf16_kernel(BuzzState st, BuzzPolicy pol, const __nv_bfloat16* __restrict__ q,
                   const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                   __nv_bfloat16* __restrict__ out, int layer, int max_batch, int kv_heads,
                   int chunk_cap, float scale_log2, int logn, int mode, int next_layer, int fused_evict) {
  constexpr int NCH = D / 8;          // 16-byte chunks per row
  constexpr int KL = NCH / 4;         // K chunks per lane and row
  constexpr int VJ = NCH / 8;         // V chunks per lane and row
  static_assert(G >= 1 && G <= kHeads, "at most 8 query heads per KV head");

  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.y, seq = blockIdx.z;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r8 = lane >> 2, c4 = lane & 3;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  // rows the append will store after the cluster barrier, fetched asynchronously at the start (CTA 0):
  // [0, NCH) the window token that moves to the middle (K), [NCH, 2 NCH) its V, then the new K and V rows
  uint4* stage = reinterpret_cast<uint4*>(smem_raw);
  int32_t* stage_pos = reinterpret_cast<int32_t*>(stage + 4 * NCH);     // position of the moving token
  Partial<G, D>* part = reinterpret_cast<Partial<G, D>*>(smem_raw + kStageBytes<D>);
  float* red = reinterpret_cast<float*>(part + 1);           // [kWarps][kHeads]
  float* mloc = red + kWarps * kHeads;                       // [kHeads] chunk-local max
  float* fr = mloc + kHeads;                                 // [kMaxCluster][G] merge factors
  float* Mg = fr + kMaxCluster * G;                          // [G] global max
  float* invL = Mg + G;                                      // [G]
  float* owarp = invL + G;                                   // [kWarps][G][D]
  float* sl = owarp + kWarps * G * D;                        // [G][chunk_cap] logits (log2 domain)
  int32_t* evict_src = reinterpret_cast<int32_t*>(sl + (size_t)G * chunk_cap);   // fused mode: work area of the eviction

  // Programmatic dependent launch; the host picks one of three modes.
  //   kWaitFirst  wait for everything earlier in the stream, then let the next launch begin.
  //   kHintFirst  the launch just before this one (same object, same stream) was a decode step of
  //               another layer: let the next launch begin, pull the head of this chunk's K rows
  //               towards L2 using a possibly stale length, then wait, then read everything for real.
  //   kOverlap    this launch is a later member of one buzz_decode_layers call: all inputs of the
  //               call were complete before its first kernel (a kWaitFirst one) passed its wait, and
  //               no other member touches this layer, so the whole step runs without waiting and
  //               CTAs of consecutive layers fill the SMs back to back. The wait moves to the end
  //               (before `out` is written), which keeps completion in stream order.
  if (mode == kWaitFirst) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (mode == kHintFirst) {
    const int nh = min(st.n[inst], pol.budget - 1) + 1;
    const int ch = ((nh + C - 1) / C + 1) & ~1;
    const int lh = min(rank * ch, nh), cnth = min(lh + ch, nh) - lh;
    const char* kb = reinterpret_cast<const char*>(st.K) + (inst * (size_t)pol.budget + lh) * (D * 2);
    // only the head of the chunk: enough to cover the start-up latency without flooding L2
    const int lines = min((cnth * D * 2) >> 7, kPrefetchLines);
    for (int i = tid; i < lines; i += kThreads) {
      asm volatile("prefetch.global.L2 [%0];" ::"l"(kb + (size_t)i * 128));
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");         // counters, q, k_new, v_new are read after this
  }
  if (mode == kWaitFirst && rank == 0) {
    // CTA 0's chunk starts at slot 0 whatever the length: pull its first rows towards L2 while the
    // counters are on their way (a line of an unoccupied slot is fetched for nothing, never used)
    const char* kb = reinterpret_cast<const char*>(st.K) + inst * (size_t)pol.budget * (D * 2);
    if (tid * 128 < min(pol.budget, 64) * D * 2) asm volatile("prefetch.global.L2 [%0];" ::"l"(kb + (size_t)tid * 128));
  }
  const int n0 = st.n[inst];
  const int tot = st.total[inst];
  const int ring_head = st.ring[inst];
  if (n0 >= pol.budget) {          // uniform over the cluster: every CTA read the same n0
    if (rank == 0 && tid == 0) buzz_set_status(st.status, BUZZ_ERR_OVERFLOW, (int)inst, n0);
    if (mode == kOverlap) asm volatile("griddepcontrol.wait;" ::: "memory");   // still finish after the member before
    return;
  }
  const int n1 = n0 + 1;
  const int chunk = ((n1 + C - 1) / C + 1) & ~1;             // even, so float2 accesses stay aligned
  const int lo = min(rank * chunk, n1);
  const int hi = min(lo + chunk, n1);
  const int cnt = hi - lo;
  float scale = scale_log2;
  if (logn) scale *= __logf((float)(tot + 1)) * (1.0f / 6.2383246250395077f);   // log_512(tokens seen)

  const size_t cache_off = inst * (size_t)pol.budget * NCH;      // in uint4 units
  const uint4* Kc = reinterpret_cast<const uint4*>(st.K) + cache_off;
  const uint4* Vc = reinterpret_cast<const uint4*>(st.V) + cache_off;
  const uint4* knew = reinterpret_cast<const uint4*>(k_new) + ((size_t)seq * kv_heads + head) * NCH;
  const uint4* vnew = reinterpret_cast<const uint4*>(v_new) + ((size_t)seq * kv_heads + head) * NCH;

  // Logical slot n0 is the token being appended (Eq. 2): it is read from k_new / v_new throughout and
  // stored only after the cluster barrier below, because with a full window ring it replaces the
  // oldest window token, whose row other CTAs are still reading until then.
  const buzz_dev::AppendPlan app = buzz_dev::plan_append(pol, n0, ring_head);
  if (rank == 0) {   // nobody writes these rows before the barrier, so they can be fetched now and only stored in the tail
    if (tid < 2 * NCH) {
      const uint4* cache = tid < NCH ? Kc : Vc;
      const int t = tid < NCH ? tid : tid - NCH;
      if (app.slot_moved >= 0) cp_async16(stage + tid, cache + (size_t)app.slot_new * NCH + t);
      cp_async16(stage + 2 * NCH + tid, (tid < NCH ? knew : vnew) + t);
    } else if (tid == 2 * NCH && app.slot_moved >= 0) {
      cp_async4(stage_pos, st.pos + inst * pol.budget + app.slot_new);
    }
  }

  // Rolling L2 prefetch. The CTA's traffic is one stream: its K rows, then its V rows, then (as a
  // hint only) the head of the same chunk in the NEXT layer's K cache, which the next decode launch
  // of a layer stack reads first; pulling that towards L2 while this kernel reduces and updates its
  // scores keeps HBM busy across the launch boundary. Row index `vr` runs over that stream with each
  // part padded to a multiple of the rows one loop iteration covers. One line per lane and tile.
  constexpr int kIterRows = kWarps * kTile;
  constexpr int kLinesPerRow = (D * 2) / 128;                  // 1 (d = 64) or 2 (d = 128)
  const int cntR = (cnt + kIterRows - 1) / kIterRows * kIterRows;
  const char* pfK = reinterpret_cast<const char*>(Kc + (size_t)lo * NCH);
  const char* pfV = reinterpret_cast<const char*>(Vc + (size_t)lo * NCH);
  const size_t inst_next = ((size_t)max(next_layer, 0) * max_batch + seq) * kv_heads + head;
  const char* pfN = reinterpret_cast<const char*>(reinterpret_cast<const uint4*>(st.K) +
                                                  (inst_next * (size_t)pol.budget + lo) * NCH);
  auto prefetch_tile = [&](int vr) {
    int row = vr + lane / kLinesPerRow;
    if (lane >= kTile * kLinesPerRow) return;
    const char* b = pfK;
    if (vr >= 2 * cntR) { if (next_layer < 0) return; row -= 2 * cntR; b = pfN; }
    else if (vr >= cntR) { row -= cntR; b = pfV; }
    if (row < cnt) asm volatile("prefetch.global.L2 [%0];" ::"l"(b + (size_t)row * (D * 2) + (lane % kLinesPerRow) * 128));
  };
  {   // this chunk's score words are read at the very end: start them towards L2 now
    const char* sb = reinterpret_cast<const char*>(st.score + inst * pol.budget + lo);
    if (tid * 128 < cnt * 4) asm volatile("prefetch.global.L2 [%0];" ::"l"(sb + (size_t)tid * 128));
  }

  // ---- phase 1: logits, S^T = K Q^T ------------------------------------------------------
  float mx[2] = {-INFINITY, -INFINITY};          // heads 2*c4 and 2*c4+1
  {
    uint4 qv[KL];                                // Q^T fragment: head r8, chunk c4 + 4i
#pragma unroll
    for (int i = 0; i < KL; ++i) {
      qv[i] = make_uint4(0, 0, 0, 0);
      if (r8 < G) qv[i] = reinterpret_cast<const uint4*>(q)[(((size_t)seq * kv_heads + head) * G + r8) * NCH + c4 + 4 * i];
    }
    auto load_k = [&](int base, uint4 (&ka)[KL], uint4 (&kb)[KL]) {
      const int ra = base + r8, rb = base + r8 + 8;
      const uint4* pa = (lo + ra == n0) ? knew : Kc + (size_t)(lo + ra) * NCH;
      const uint4* pb = (lo + rb == n0) ? knew : Kc + (size_t)(lo + rb) * NCH;
#pragma unroll
      for (int i = 0; i < KL; ++i) {
        ka[i] = (ra < cnt) ? ld_stream(pa + c4 + 4 * i) : make_uint4(0, 0, 0, 0);
        kb[i] = (rb < cnt) ? ld_stream(pb + c4 + 4 * i) : make_uint4(0, 0, 0, 0);
      }
    };
    uint4 ka[KL], kb[KL], ka2[KL], kb2[KL];
    load_k(warp * kTile, ka, kb);                 // rows beyond cnt load nothing
    for (int base = warp * kTile; base < cnt; base += kWarps * kTile) {
      const int ra = base + r8, rb = base + r8 + 8;
      load_k(base + kWarps * kTile, ka2, kb2);    // next tile's loads are in flight during the MMAs
      if (kAhead > 0) prefetch_tile(base + (kAhead + 1) * kIterRows);
      float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < KL; ++i)
#pragma unroll
        for (int h = 0; h < 2; ++h)
          mma_bf16(s, word(ka[i], 2 * h), word(kb[i], 2 * h), word(ka[i], 2 * h + 1), word(kb[i], 2 * h + 1),
                   word(qv[i], 2 * h), word(qv[i], 2 * h + 1));
      // s[0], s[1]: key ra, heads 2*c4, 2*c4+1;  s[2], s[3]: key rb
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int hd = 2 * c4 + e;
        if (hd < G) {
          if (ra < cnt) { const float v = s[e] * scale; sl[hd * chunk_cap + ra] = v; mx[e] = fmaxf(mx[e], v); }
          if (rb < cnt) { const float v = s[2 + e] * scale; sl[hd * chunk_cap + rb] = v; mx[e] = fmaxf(mx[e], v); }
        }
      }
#pragma unroll
      for (int i = 0; i < KL; ++i) { ka[i] = ka2[i]; kb[i] = kb2[i]; }
    }
  }
  auto load_v = [&](int base, uint4 (&vv)[4][VJ]) {
    const int row[4] = {base + 2 * c4, base + 2 * c4 + 1, base + 2 * c4 + 8, base + 2 * c4 + 9};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      const uint4* p = (lo + row[x] == n0) ? vnew : Vc + (size_t)(lo + row[x]) * NCH;
#pragma unroll
      for (int j = 0; j < VJ; ++j)
        vv[x][j] = (row[x] < cnt) ? ld_stream(p + r8 + 8 * j) : make_uint4(0, 0, 0, 0);
    }
  };
  uint4 vv[4][VJ], vn[4][VJ];
  load_v(warp * kTile, vv);                      // in flight across the reduction of the maxima
#pragma unroll
  for (int e = 0; e < 2; ++e) {
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], off));
    if (r8 == 0) red[warp * kHeads + 2 * c4 + e] = mx[e];
  }
  __syncthreads();
  if (tid < kHeads) {
    float m = red[tid];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) m = fmaxf(m, red[w * kHeads + tid]);
    mloc[tid] = m;
  }
  __syncthreads();

  // ---- phase 2: O^T += V^T P^T -------------------------------------------------------------
  float ls = 0.f;                                // sum of p for head r8 over this lane's keys
  {
    float oc[VJ][4][4];
#pragma unroll
    for (int j = 0; j < VJ; ++j)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
#pragma unroll
        for (int e = 0; e < 4; ++e) oc[j][jj][e] = 0.f;
    const float mh = (r8 < G) ? mloc[r8] : 0.f;
    for (int base = warp * kTile; base < cnt; base += kWarps * kTile) {
      const int row[4] = {base + 2 * c4, base + 2 * c4 + 1, base + 2 * c4 + 8, base + 2 * c4 + 9};
      load_v(base + kWarps * kTile, vn);
      if (kAhead > 0) prefetch_tile(cntR + base + (kAhead + 1) * kIterRows);
      // P^T fragment: head r8, keys base + 2*c4 + {0,1} and + 8
      float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
      if (r8 < G) {
        const float* srow = sl + r8 * chunk_cap;
        if (row[1] < cnt) {
          const float2 t = *reinterpret_cast<const float2*>(srow + row[0]);
          p0 = exp2f(t.x - mh); p1 = exp2f(t.y - mh);
        } else if (row[0] < cnt) {
          p0 = exp2f(srow[row[0]] - mh);
        }
        if (row[3] < cnt) {
          const float2 t = *reinterpret_cast<const float2*>(srow + row[2]);
          p2 = exp2f(t.x - mh); p3 = exp2f(t.y - mh);
        } else if (row[2] < cnt) {
          p2 = exp2f(srow[row[2]] - mh);
        }
      }
      ls += (p0 + p1) + (p2 + p3);
      const uint32_t b0 = pack_bf16(p0, p1), b1 = pack_bf16(p2, p3);
#pragma unroll
      for (int j = 0; j < VJ; ++j)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const uint32_t wa = word(vv[0][j], jj), wb = word(vv[1][j], jj);
          const uint32_t wc = word(vv[2][j], jj), wd = word(vv[3][j], jj);
          mma_bf16(oc[j][jj], __byte_perm(wa, wb, 0x5410), __byte_perm(wa, wb, 0x7632),
                   __byte_perm(wc, wd, 0x5410), __byte_perm(wc, wd, 0x7632), b0, b1);
        }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int j = 0; j < VJ; ++j) vv[x][j] = vn[x][j];
    }
    // oc[j][jj]: [0],[1] -> dim (r8 + 8j)*8 + 2jj, heads 2*c4, 2*c4+1;  [2],[3] -> that dim + 1
#pragma unroll
    for (int j = 0; j < VJ; ++j)
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int hd = 2 * c4 + e;
          if (hd < G) {
            const int dim = (r8 + 8 * j) * 8 + 2 * jj;
            owarp[(warp * G + hd) * D + dim] = oc[j][jj][e];
            owarp[(warp * G + hd) * D + dim + 1] = oc[j][jj][2 + e];
          }
        }
  }
  ls += __shfl_xor_sync(0xffffffffu, ls, 1);
  ls += __shfl_xor_sync(0xffffffffu, ls, 2);
  if (c4 == 0) red[warp * kHeads + r8] = ls;
  __syncthreads();
  if (tid < G) {
    float l = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) l += red[w * kHeads + tid];
    part->l[tid] = l;
    part->m[tid] = mloc[tid];
  }
  for (int idx = tid; idx < G * D; idx += kThreads) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += owarp[w * G * D + idx];
    part->o[idx / D][idx % D] = v;
  }

  // ---- combine across the cluster -------------------------------------------------------
  // (a cluster of one CTA needs only the CTA barrier: a cluster barrier with release/acquire
  // semantics also waits for the CTA's outstanding stores, about a microsecond each time)
  if (C == 1) __syncthreads(); else cluster.sync();
  if (mode == kOverlap) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (rank == 0) {                   // every CTA has read n0/tot/ring and all old rows before the barrier
    if (tid <= 2 * NCH) cp_async_wait();
    buzz_dev::append_staged<NCH>(st, pol, inst, app, tot, stage, stage_pos, tid);
    if (tid == kThreads - 1) {
      st.n[inst] = n1;
      st.total[inst] = tot + 1;
      st.ring[inst] = app.head_next;
    }
  }
  if (tid < G) {
    float M = -INFINITY;
    for (int r = 0; r < C; ++r) M = fmaxf(M, cluster.map_shared_rank(part, r)->m[tid]);
    float L = 0.f;
    for (int r = 0; r < C; ++r) {
      const Partial<G, D>* pr = cluster.map_shared_rank(part, r);
      const float f = (pr->m[tid] == -INFINITY) ? 0.f : exp2f(pr->m[tid] - M);   // empty chunk
      fr[r * G + tid] = f;
      L += pr->l[tid] * f;
    }
    Mg[tid] = M;
    invL[tid] = 1.0f / L;
  }
  __syncthreads();
  // scores of this CTA's chunk: += sum over the group's heads of the exact fp32 probabilities. With a
  // full ring the token leaving the window (still at slot app.slot_new) takes its score along to slot
  // n0, and the appended token's first score lands in app.slot_new -- stored only after the last
  // barrier, once the thread that reads the old value there is done.
  float pending_score = 0.f;
  bool has_pending = false;
  {
    float* score = st.score + inst * pol.budget;
    constexpr int U = 4;                             // slots per thread and pass: their old scores are fetched together
    for (int j0 = tid; j0 < cnt; j0 += U * kThreads) {
      float old[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int j = j0 + u * kThreads;
        old[u] = (j < cnt && lo + j != n0) ? score[lo + j] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int j = j0 + u * kThreads;
        if (j >= cnt) break;
        float add = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) add += exp2f(sl[g * chunk_cap + j] - Mg[g]) * invL[g];
        const int slot = lo + j;
        if (slot == n0) {
          if (app.slot_moved >= 0) { pending_score = add; has_pending = true; }
          else score[n0] = add;
        } else if (slot == app.slot_new) {           // only with a full ring: slot_new < n0
          score[n0] = old[u] + add;
        } else {
          score[slot] = old[u] + add;
        }
      }
    }
  }
  if (rank == 0) {
    __nv_bfloat16* o = out + ((size_t)seq * kv_heads + head) * G * D;
    for (int idx = tid; idx < G * D; idx += kThreads) {
      const int g = idx / D;
      float acc = 0.f;
      for (int r = 0; r < C; ++r) acc += cluster.map_shared_rank(part, r)->o[g][idx % D] * fr[r * G + g];
      o[idx] = __float2bfloat16_rn(acc * invL[g]);
    }
  }
  // Peers may still be reading this CTA's shared memory, and the thread that moves the leaving
  // token's score must have read it before the pending store below. Only the fused eviction reads
  // what OTHER CTAs of the cluster wrote to global memory, so only it needs release/acquire.
  if (C == 1) __syncthreads();
  else if (fused_evict) cluster.sync();
  else asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
  if (has_pending) st.score[inst * pol.budget + app.slot_new] = pending_score;
  // Fused eviction (Algorithm 1's trigger: the cache is full after this step). Every score, row and
  // counter of the instance was written before the barrier above, by this cluster.
  if (fused_evict && rank == 0 && n1 >= pol.budget && n1 > pol.sink + pol.window)
    buzz_dev::evict_instance<D * 2, kThreads>(st, pol, inst, n1, st.n_old[inst], evict_src);
}

template <int D, int G>
cudaError_t launch(buzz_ctx* c, int layer, const void* q, const void* k_new, const void* v_new,
                   void* out, int cluster_size, int mode, int next_layer, cudaStream_t stream) {
  const int batch = c->batch[layer];
  // A CTA keeps the logits of its chunk (and, in fused mode, the eviction's work area) in shared
  // memory: if that does not fit, split the instance over more CTAs.
  int chunk_cap;
  size_t smem;
  for (;; cluster_size *= 2) {
    chunk_cap = (((c->pol.budget + cluster_size - 1) / cluster_size + 1) & ~1) + 2;
    smem = kStageBytes<D> + sizeof(Partial<G, D>) +
           sizeof(float) * (kWarps * kHeads + kHeads + kMaxCluster * G + 2 * G + kWarps * G * D + (size_t)G * chunk_cap) +
           (c->fused_evict ? buzz_dev::evict_smem_bytes(c->pol) : 0);
    if (smem <= 200 * 1024 || cluster_size >= kMaxCluster) break;
  }
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  static BuzzSmemOptIn opt_in;
  if (cudaError_t e = opt_in.ensure(decode_bf16_kernel<D, G>, smem); e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cluster_size, c->sh.kv_heads, batch);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_size;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // the kernel waits on its own
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  return cudaLaunchKernelEx(&cfg, decode_bf16_kernel<D, G>, c->st, c->pol, (const __nv_bfloat16*)q,
                            (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, (__nv_bfloat16*)out,
                            layer, c->sh.max_batch, c->sh.kv_heads, chunk_cap, scale_log2,
                            (c->sh.flags & BUZZ_FLAG_LOGN) ? 1 : 0, mode, next_layer, c->fused_evict);
}

template <int D>
cudaError_t launch_g(buzz_ctx* c, int layer, const void* q, const void* k_new, const void* v_new,
                     void* out, int cs, int mode, int next_layer, cudaStream_t stream) {
  switch (c->group) {
    case 1: return launch<D, 1>(c, layer, q, k_new, v_new, out, cs, mode, next_layer, stream);
    case 2: return launch<D, 2>(c, layer, q, k_new, v_new, out, cs, mode, next_layer, stream);
    case 4: return launch<D, 4>(c, layer, q, k_new, v_new, out, cs, mode, next_layer, stream);
    case 8: return launch<D, 8>(c, layer, q, k_new, v_new, out, cs, mode, next_layer, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t buzz_launch_decode_bf16(buzz_ctx* c, int layer, const void* q, const void* k_new,
                                    const void* v_new, void* out, int cluster_size, int mode, int next_layer,
                                    cudaStream_t stream) {
  return c->sh.head_dim == 128 ? launch_g<128>(c, layer, q, k_new, v_new, out, cluster_size, mode, next_layer, stream)
                               : launch_g<64>(c, layer, q, k_new, v_new, out, cluster_size, mode, next_layer, stream);
}
