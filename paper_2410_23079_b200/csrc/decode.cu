// BUZZ decode step: append + attention over the compacted cache + score accumulation, one thread-
// block CLUSTER per (sequence, KV head) instance of a layer (Eqs. 2 and 3 of the paper; the score
// is Algorithm 2's accumulated attention A, += p per step, summed over the group's query heads).
//
// The step is HBM-bound: every retained K row and V row is read exactly once per step, whatever
// the number of query heads in the group, and the only other traffic is 8 bytes per slot for the
// score read-modify-write. The cluster's CTAs split the n+1 slots into contiguous chunks:
//   phase 1  stream the chunk's K rows (16-byte loads, a warp covers whole consecutive rows),
//            logits for the G query heads -> shared memory, chunk-local max;
//   phase 2  p~ = 2^(logit - local max), local sum, stream the chunk's V rows into a partial output;
//   combine  the CTAs publish (max, sum, partial output) in their own shared memory; after one
//            cluster barrier each CTA reads the others' (max, sum) through distributed shared
//            memory, derives the global normaliser, adds the now-exact probabilities of ITS chunk
//            to the scores, and CTA 0 merges the partial outputs.
// Nothing is staged in global memory and every reduction has a fixed order, so the result is
// deterministic. The appended token's row is read from k_new/v_new throughout and stored after the
// cluster barrier: into the window ring, whose oldest token first moves to the end of the middle
// region (cache_ops.cuh). In fused mode CTA 0 then runs the instance's eviction if the step filled
// the cache.
#include <cooperative_groups.h>

#include "cache_ops.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kUnroll = 8;      // 16-byte loads in flight per thread
constexpr int kMaxCluster = 8;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  __device__ static void unpack(const uint4& u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y);
    f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void unpack(const uint4& u, float (&f)[8]) {
    // a bf16 is the upper half of an fp32
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
    f[4] = __uint_as_float(u.z << 16); f[5] = __uint_as_float(u.z & 0xffff0000u);
    f[6] = __uint_as_float(u.w << 16); f[7] = __uint_as_float(u.w & 0xffff0000u);
  }
};

__device__ inline uint4 ld_stream(const uint4* p) { return __ldcs(p); }

__device__ inline void store_out(float* p, float v) { *p = v; }
__device__ inline void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <int G, int D>
struct Partial {       // what a CTA publishes to its cluster
  float m[G];          // chunk-local max of the log2-domain logits
  float l[G];          // sum of 2^(logit - m) over the chunk
  float o[G][D];       // sum of 2^(logit - m) * V over the chunk
};

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_kernel(BuzzState st, BuzzPolicy pol, const T* __restrict__ q, const T* __restrict__ k_new,
              const T* __restrict__ v_new, T* __restrict__ out, int layer, int max_batch,
              int kv_heads, int chunk_cap, float scale_log2, int logn, int fused_evict) {
  constexpr int EPL = Vec16<T>::N;              // elements per 16-byte lane
  constexpr int LPR = D / EPL;                  // lanes per row
  constexpr int RPW = 32 / LPR;                 // rows per warp-wide load
  constexpr int ROWS_PER_ITER = kWarps * RPW * kUnroll;
  static_assert(LPR >= 1 && LPR <= 32 && (32 % LPR) == 0, "row must tile a warp");

  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int head = blockIdx.y, seq = blockIdx.z;
  const size_t inst = ((size_t)layer * max_batch + seq) * kv_heads + head;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, col = lane % LPR;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  Partial<G, D>* part = reinterpret_cast<Partial<G, D>*>(smem_raw);
  float* red = reinterpret_cast<float*>(part + 1);           // [kWarps][G]
  float* fr = red + kWarps * G;                              // [kMaxCluster][G] merge factors
  float* invL = fr + kMaxCluster * G;                        // [G]
  float* owarp = invL + G;                                   // [kWarps][G][D]
  float* sl = owarp + kWarps * G * D;                        // [G][chunk_cap]
  int32_t* evict_src = reinterpret_cast<int32_t*>(sl + (size_t)G * chunk_cap);   // fused mode: work area of the eviction

  const int n0 = st.n[inst];
  const int tot = st.total[inst];
  const int ring_head = st.ring[inst];
  if (n0 >= pol.budget) {          // uniform over the cluster: every CTA read the same n0
    if (rank == 0 && tid == 0) buzz_set_status(st.status, BUZZ_ERR_OVERFLOW, (int)inst, n0);
    return;
  }
  const int n1 = n0 + 1;
  const int chunk = (n1 + C - 1) / C;
  const int lo = min(rank * chunk, n1);
  const int hi = min(lo + chunk, n1);
  const int cnt = hi - lo;
  float scale = scale_log2;
  if (logn) scale *= __logf((float)(tot + 1)) * (1.0f / 6.2383246250395077f);   // log_512(tokens seen)

  const size_t cache_off = inst * (size_t)pol.budget * LPR;      // in uint4 units
  const uint4* Kc = reinterpret_cast<const uint4*>(st.K) + cache_off;
  const uint4* Vc = reinterpret_cast<const uint4*>(st.V) + cache_off;
  const uint4* knew = reinterpret_cast<const uint4*>(k_new) + ((size_t)seq * kv_heads + head) * LPR;
  const uint4* vnew = reinterpret_cast<const uint4*>(v_new) + ((size_t)seq * kv_heads + head) * LPR;

  // Logical slot n0 is the token being appended (Eq. 2): read from k_new / v_new throughout, stored
  // after the cluster barrier (with a full window ring it replaces the oldest window token, whose
  // row other CTAs are still reading until then).
  const buzz_dev::AppendPlan app = buzz_dev::plan_append(pol, n0, ring_head);

  // ---- phase 1: logits ------------------------------------------------------------------
  float mx[G];
  {
    float qf[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 u = reinterpret_cast<const uint4*>(q)[(((size_t)seq * kv_heads + head) * G + g) * LPR + col];
      Vec16<T>::unpack(u, qf[g]);
      mx[g] = -INFINITY;
    }
    for (int base = 0; base < cnt; base += ROWS_PER_ITER) {
      uint4 buf[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int r = base + (u * kWarps + warp) * RPW + sub;
        const int slot = lo + r;
        const uint4* p = (slot == n0) ? knew + col : Kc + (size_t)slot * LPR + col;
        buf[u] = (r < cnt) ? ld_stream(p) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int r = base + (u * kWarps + warp) * RPW + sub;
        float kf[EPL];
        Vec16<T>::unpack(buf[u], kf);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < EPL; ++e) dot = fmaf(qf[g][e], kf[e], dot);
#pragma unroll
          for (int off = LPR / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
          dot *= scale;
          if (r < cnt) {
            mx[g] = fmaxf(mx[g], dot);
            if (col == 0) sl[g * chunk_cap + r] = dot;
          }
        }
      }
    }
  }
  // chunk-local max per query head
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], off));
    if (lane == 0) red[warp * G + g] = mx[g];
  }
  __syncthreads();
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float m = red[g];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) m = fmaxf(m, red[w * G + g]);
    mx[g] = m;
  }
  __syncthreads();

  // ---- phase 2a: p~ and its sum ---------------------------------------------------------
  float ls[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    ls[g] = 0.f;
    for (int j = tid; j < cnt; j += kThreads) {
      const float p = exp2f(sl[g * chunk_cap + j] - mx[g]);
      sl[g * chunk_cap + j] = p;
      ls[g] += p;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ls[g] += __shfl_xor_sync(0xffffffffu, ls[g], off);
    if (lane == 0) red[warp * G + g] = ls[g];
  }
  __syncthreads();
  if (tid < G) {
    float l = 0.f;
    for (int w = 0; w < kWarps; ++w) l += red[w * G + tid];
    part->l[tid] = l;
#pragma unroll
    for (int g = 0; g < G; ++g)
      if (tid == g) part->m[g] = mx[g];
  }

  // ---- phase 2b: partial output ---------------------------------------------------------
  {
    float of[G][EPL];
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPL; ++e) of[g][e] = 0.f;
    for (int base = 0; base < cnt; base += ROWS_PER_ITER) {
      uint4 buf[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int r = base + (u * kWarps + warp) * RPW + sub;
        const int slot = lo + r;
        const uint4* p = (slot == n0) ? vnew + col : Vc + (size_t)slot * LPR + col;
        buf[u] = (r < cnt) ? ld_stream(p) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int r = base + (u * kWarps + warp) * RPW + sub;
        if (r < cnt) {
          float vf[EPL];
          Vec16<T>::unpack(buf[u], vf);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float p = sl[g * chunk_cap + r];
#pragma unroll
            for (int e = 0; e < EPL; ++e) of[g][e] = fmaf(p, vf[e], of[g][e]);
          }
        }
      }
    }
    // rows of one warp-wide load -> one row's worth, then across warps through shared memory
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        float v = of[g][e];
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if (sub == 0) owarp[(warp * G + g) * D + col * EPL + e] = v;
      }
  }
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += kThreads) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += owarp[w * G * D + idx];
    part->o[idx / D][idx % D] = v;
  }

  // ---- combine across the cluster -------------------------------------------------------
  cluster.sync();
  if (rank == 0) {                   // every CTA has read n0/tot/ring and all old rows before the barrier
    buzz_dev::append_rows<LPR>(st, pol, inst, app, tot, knew, vnew, tid);
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
      const float f = exp2f(pr->m[tid] - M);      // 0 for an empty chunk (m = -inf)
      fr[r * G + tid] = f;
      L += pr->l[tid] * f;
    }
    invL[tid] = 1.0f / L;
  }
  __syncthreads();
  // scores of this CTA's chunk: += sum over the group's heads of the exact probabilities. With a full
  // ring the token leaving the window (still at slot app.slot_new) takes its score along to slot n0,
  // and the appended token's first score lands in app.slot_new after the last barrier.
  float pending_score = 0.f;
  bool has_pending = false;
  {
    float* score = st.score + inst * pol.budget;
    for (int j = tid; j < cnt; j += kThreads) {
      float add = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) add += sl[g * chunk_cap + j] * (fr[rank * G + g] * invL[g]);
      const int slot = lo + j;
      if (slot == n0) {
        if (app.slot_moved >= 0) { pending_score = add; has_pending = true; }
        else score[n0] = add;
      } else if (slot == app.slot_new) {             // only with a full ring: slot_new < n0
        score[n0] = score[slot] + add;
      } else {
        score[slot] += add;
      }
    }
  }
  if (rank == 0) {
    T* o = out + ((size_t)seq * kv_heads + head) * G * D;
    for (int idx = tid; idx < G * D; idx += kThreads) {
      const int g = idx / D;
      float acc = 0.f;
      for (int r = 0; r < C; ++r) acc += cluster.map_shared_rank(part, r)->o[g][idx % D] * fr[r * G + g];
      store_out(o + idx, acc * invL[g]);
    }
  }
  cluster.sync();                    // peers may still be reading this CTA's shared memory
  if (has_pending) st.score[inst * pol.budget + app.slot_new] = pending_score;
  if (fused_evict && rank == 0 && n1 >= pol.budget && n1 > pol.sink + pol.window)
    buzz_dev::evict_instance<D * (int)sizeof(T), kThreads>(st, pol, inst, n1, st.n_old[inst], evict_src);
}

template <typename T, int D, int G>
cudaError_t launch(buzz_ctx* c, int layer, const void* q, const void* k_new, const void* v_new,
                   void* out, int cluster_size, cudaStream_t stream) {
  const int batch = c->batch[layer];
  const int chunk_cap = (c->pol.budget + cluster_size - 1) / cluster_size;
  const size_t smem = sizeof(Partial<G, D>) +
                      sizeof(float) * (kWarps * G + kMaxCluster * G + G + kWarps * G * D + (size_t)G * chunk_cap) +
                      (c->fused_evict ? buzz_dev::evict_smem_bytes(c->pol) : 0);
  static BuzzSmemOptIn opt_in;
  if (cudaError_t e = opt_in.ensure(decode_kernel<T, D, G>, smem); e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cluster_size, c->sh.kv_heads, batch);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_size;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  return cudaLaunchKernelEx(&cfg, decode_kernel<T, D, G>, c->st, c->pol, (const T*)q, (const T*)k_new,
                            (const T*)v_new, (T*)out, layer, c->sh.max_batch, c->sh.kv_heads,
                            chunk_cap, scale_log2, (c->sh.flags & BUZZ_FLAG_LOGN) ? 1 : 0, c->fused_evict);
}

template <typename T, int D>
cudaError_t launch_g(buzz_ctx* c, int layer, const void* q, const void* k_new, const void* v_new,
                     void* out, int cs, cudaStream_t stream) {
  switch (c->group) {
    case 1: return launch<T, D, 1>(c, layer, q, k_new, v_new, out, cs, stream);
    case 2: return launch<T, D, 2>(c, layer, q, k_new, v_new, out, cs, stream);
    case 4: return launch<T, D, 4>(c, layer, q, k_new, v_new, out, cs, stream);
    case 8: return launch<T, D, 8>(c, layer, q, k_new, v_new, out, cs, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t buzz_launch_decode_bf16(buzz_ctx* c, int layer, const void* q, const void* k_new,
                                    const void* v_new, void* out, int cluster_size, int mode, int next_layer,
                                    cudaStream_t stream);

cudaError_t buzz_launch_decode(buzz_ctx* c, int layer, const void* q, const void* k_new,
                               const void* v_new, void* out, cudaStream_t stream, int chain_pos,
                               int next_layer) {
  if (c->batch[layer] == 0) return cudaSuccess;
  int cs = c->decode_cluster;
  if (cs == 0) {
    // The whole grid should be one resident wave of long-lived CTAs: the smallest power-of-two
    // split that gives every SM (148 on a B200) at least one or two CTAs (measured best on C2 and
    // C4 shapes), while every CTA still streams at least ~64 rows.
    // A member of a multi-layer call shares the SMs with its neighbours in the call, so it need not
    // fill the GPU by itself and does better with fewer, longer-lived CTAs (a CTA's fixed cost is
    // several microseconds): three quarters of the SMs are enough there (measured on 128 instances
    // of ~1500 slots: 18 us per launch with one CTA per instance against 20 us with two).
    const long inst = (long)c->batch[layer] * c->sh.kv_heads;
    const long want = chain_pos >= 0 ? (long)c->sm_count * 3 / 4 : (long)c->sm_count * 3 / 2;
    cs = 1;
    while (cs < kMaxCluster && inst * cs < want && (c->pol.budget / (cs * 2)) >= 64) cs *= 2;
  }
  // the logits of a chunk must fit in shared memory
  while (cs < kMaxCluster && (size_t)c->group * ((c->pol.budget + cs - 1) / cs) * sizeof(float) > 96 * 1024) cs *= 2;
  cudaError_t e;
  if (c->sh.dtype == BUZZ_BF16) {
    // Dependency mode of the kernel (see decode_bf16.cu). A later member of one multi-layer call
    // overlaps with the members before it; a single call may only warm L2 ahead of its wait, and
    // only if the launch before it was a decode step of another layer through this object and stream.
    int mode = 0;
    if (chain_pos > 0) mode = 2;
    else if (chain_pos < 0 && c->last_kind == 1 && c->last_layer != layer && c->last_stream == (void*)stream) mode = 1;
    if (chain_pos < 0) next_layer = layer + 1 == c->sh.layers ? 0 : layer + 1;   // a layer stack is walked in order
    e = buzz_launch_decode_bf16(c, layer, q, k_new, v_new, out, cs, mode, next_layer, stream);   // tensor-core kernel
    if (e == cudaSuccess) { c->last_kind = 1; c->last_layer = layer; c->last_stream = (void*)stream; }
  } else {
    e = c->sh.head_dim == 128 ? launch_g<float, 128>(c, layer, q, k_new, v_new, out, cs, stream)
                              : launch_g<float, 64>(c, layer, q, k_new, v_new, out, cs, stream);
    c->last_kind = 2;
  }
  if (e == cudaSuccess) {
    c->launches += 1;
    c->maybe_full[layer] = c->fused_evict ? 0 : 1;   // a fused step leaves every cache below its budget
  }
  return e;
}
