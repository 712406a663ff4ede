// Prefill attention with per-key column sums on the ordinary fp32 pipes. This is the path for
// fp32 caches (any head_dim the library supports) -- a tiled two-pass kernel pair:
//
//   pass A (query-tile stationary)  O = Softmax(Q K^T / sqrt(d)) V with an online softmax over the
//                                   key tiles up to the diagonal (Eq. 3), and per row the
//                                   log2-sum-exp  lse_i = m_i + log2(l_i);
//   pass B (key-tile stationary)    recomputes S for the tiles at and below the diagonal, forms the
//                                   exact probabilities 2^(S_ij - lse_i) and sums them down the
//                                   columns: score_j = sum over the group's query heads and rows
//                                   i >= j of P_ij (Algorithm 2's accumulated attention A at the
//                                   end of the prompt). Each thread adds its rows in a fixed
//                                   order and the 16 row groups are merged in a fixed order, so
//                                   the sums are reproducible bit for bit.
//
// The column sums need every row's final normaliser, which is why S is computed twice.
#include "buzz_internal.cuh"

namespace {

constexpr int BM = 64;          // query rows per tile
constexpr int BN = 64;          // keys per tile
constexpr int kThreads = 256;   // 16 x 16: ty owns 4 rows, tx owns 4 columns (tx, tx+16, ...)
constexpr float kInvLn512 = 1.0f / 6.2383246250395077f;

__device__ inline float to_f(float x) { return x; }
__device__ inline float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ inline void from_f(float* p, float v) { *p = v; }
__device__ inline void from_f(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Loads rows [row0, row0+64) x D of a [tokens][heads][D] tensor into smem as fp32, zero beyond `rows`.
template <typename T, int D>
__device__ inline void load_tile(float* dst, const T* src, size_t tok0, int rows, int heads, int head) {
  constexpr int LD = D + 4;
  for (int idx = threadIdx.x; idx < 64 * (D / 4); idx += kThreads) {
    const int r = idx / (D / 4), c4 = idx % (D / 4);
    float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < rows) {
      const T* p = src + ((tok0 + r) * heads + head) * D + c4 * 4;
      val = make_float4(to_f(p[0]), to_f(p[1]), to_f(p[2]), to_f(p[3]));
    }
    *reinterpret_cast<float4*>(dst + r * LD + c4 * 4) = val;
  }
}

// acc[i][u] = sum_c A[ty*4+i][c] * B[tx+16u][c]
template <int D>
__device__ inline void tile_dot(const float* A, const float* B, int ty, int tx, float (&acc)[4][4]) {
  constexpr int LD = D + 4;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[i][u] = 0.f;
  for (int c = 0; c < D; c += 4) {
    float4 a[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(A + (ty * 4 + i) * LD + c);
#pragma unroll
    for (int u = 0; u < 4; ++u) b[u] = *reinterpret_cast<const float4*>(B + (tx + 16 * u) * LD + c);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        acc[i][u] = fmaf(a[i].x, b[u].x, acc[i][u]);
        acc[i][u] = fmaf(a[i].y, b[u].y, acc[i][u]);
        acc[i][u] = fmaf(a[i].z, b[u].z, acc[i][u]);
        acc[i][u] = fmaf(a[i].w, b[u].w, acc[i][u]);
      }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
prefill_attn_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                    const int32_t* __restrict__ cu, T* __restrict__ out, float* __restrict__ lse,
                    int Hq, int Hkv, int lse_stride, float scale_log2, int logn) {
  constexpr int LD = D + 4, LP = BN + 4, DPT = D / 16;
  extern __shared__ __align__(16) float sm[];
  float* Qs = sm;
  float* Ks = Qs + BM * LD;
  float* Vs = Ks + BN * LD;
  float* Ps = Vs + BN * LD;
  const int b = blockIdx.z, h = blockIdx.y, kvh = h / (Hq / Hkv);
  const int tok0 = cu[b], N = cu[b + 1] - tok0;
  const int qt = gridDim.x - 1 - blockIdx.x;       // heaviest (last) query tiles first
  const int row0 = qt * BM;
  if (row0 >= N) return;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;

  load_tile<T, D>(Qs, q, (size_t)tok0 + row0, min(BM, N - row0), Hq, h);
  float m[4], l[4], o[4][DPT], rs[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = -INFINITY; l[i] = 0.f;
    rs[i] = scale_log2 * (logn ? __logf((float)(row0 + ty * 4 + i + 1)) * kInvLn512 : 1.0f);
#pragma unroll
    for (int c = 0; c < DPT; ++c) o[i][c] = 0.f;
  }
  for (int kt = 0; kt <= qt; ++kt) {
    const int key0 = kt * BN;
    __syncthreads();                               // previous tile's Ks/Vs/Ps are no longer read
    load_tile<T, D>(Ks, k, (size_t)tok0 + key0, min(BN, N - key0), Hkv, kvh);
    load_tile<T, D>(Vs, v, (size_t)tok0 + key0, min(BN, N - key0), Hkv, kvh);
    __syncthreads();
    float acc[4][4];
    tile_dot<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int qi = row0 + ty * 4 + i;
      float tmax = -INFINITY;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int kj = key0 + tx + 16 * u;
        acc[i][u] = (kj <= qi && kj < N) ? acc[i][u] * rs[i] : -INFINITY;
        tmax = fmaxf(tmax, acc[i][u]);
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
      const float m_new = fmaxf(m[i], tmax);
      const float alpha = (m[i] == -INFINITY) ? 0.f : exp2f(m[i] - m_new);
      float psum = 0.f;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float p = (acc[i][u] == -INFINITY) ? 0.f : exp2f(acc[i][u] - m_new);
        Ps[(ty * 4 + i) * LP + tx + 16 * u] = p;
        psum += p;
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
      l[i] = l[i] * alpha + psum;
      m[i] = m_new;
#pragma unroll
      for (int c = 0; c < DPT; ++c) o[i][c] *= alpha;
    }
    __syncthreads();
    for (int kk = 0; kk < BN; ++kk) {
      float vv[DPT];
#pragma unroll
      for (int c = 0; c < DPT; c += 4)
        *reinterpret_cast<float4*>(vv + c) = *reinterpret_cast<const float4*>(Vs + kk * LD + tx * DPT + c);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float p = Ps[(ty * 4 + i) * LP + kk];
#pragma unroll
        for (int c = 0; c < DPT; ++c) o[i][c] = fmaf(p, vv[c], o[i][c]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int qi = row0 + ty * 4 + i;
    if (qi < N) {
      const float inv = 1.0f / l[i];
      T* op = out + (((size_t)tok0 + qi) * Hq + h) * D + tx * DPT;
#pragma unroll
      for (int c = 0; c < DPT; ++c) from_f(op + c, o[i][c] * inv);
      if (tx == 0) lse[(size_t)h * lse_stride + tok0 + qi] = m[i] + log2f(l[i]);
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
prefill_colsum_kernel(const T* __restrict__ q, const T* __restrict__ k, const int32_t* __restrict__ cu,
                      const float* __restrict__ lse, float* __restrict__ pscore, int Hq, int Hkv,
                      int stride, float scale_log2, int logn) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float sm[];
  float* Qs = sm;
  float* Ks = Qs + BM * LD;
  float* Ls = Ks + BN * LD;        // [BM] row lse
  float* Cp = Ls + BM;             // [16][BN] per-row-group column partials
  const int b = blockIdx.z, kvh = blockIdx.y, G = Hq / Hkv;
  const int tok0 = cu[b], N = cu[b + 1] - tok0;
  const int kt = blockIdx.x, key0 = kt * BN;
  if (key0 >= N) return;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const int q_tiles = (N + BM - 1) / BM;

  load_tile<T, D>(Ks, k, (size_t)tok0 + key0, min(BN, N - key0), Hkv, kvh);
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  for (int g = 0; g < G; ++g) {
    const int h = kvh * G + g;
    for (int qt = kt; qt < q_tiles; ++qt) {
      const int row0 = qt * BM;
      __syncthreads();
      load_tile<T, D>(Qs, q, (size_t)tok0 + row0, min(BM, N - row0), Hq, h);
      if (tid < BM) Ls[tid] = (row0 + tid < N) ? lse[(size_t)h * stride + tok0 + row0 + tid] : 0.f;
      __syncthreads();
      float acc[4][4];
      tile_dot<D>(Qs, Ks, ty, tx, acc);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int qi = row0 + ty * 4 + i;
        const float rs = scale_log2 * (logn ? __logf((float)(qi + 1)) * kInvLn512 : 1.0f);
        const float li = Ls[ty * 4 + i];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int kj = key0 + tx + 16 * u;
          if (kj <= qi && qi < N) col[u] += exp2f(acc[i][u] * rs - li);
        }
      }
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) Cp[ty * BN + tx + 16 * u] = col[u];
  __syncthreads();
  if (tid < BN && key0 + tid < N) {
    float s = 0.f;
    for (int r = 0; r < 16; ++r) s += Cp[r * BN + tid];
    pscore[(size_t)kvh * stride + tok0 + key0 + tid] = s;
  }
}

template <typename T, int D>
cudaError_t launch_simt(buzz_ctx* c, const void* q, const void* k, const void* v, const int32_t* cu,
                        int batch, int max_seqlen, void* out, cudaStream_t stream, int* launches) {
  constexpr int LD = D + 4;
  const size_t smemA = sizeof(float) * (BM * LD + 2 * BN * LD + BM * (BN + 4));
  const size_t smemB = sizeof(float) * (BM * LD + BN * LD + BM + 16 * BN);
  static BuzzSmemOptIn opt_in_a, opt_in_b;
  if (cudaError_t e = opt_in_a.ensure(prefill_attn_kernel<T, D>, smemA); e != cudaSuccess) return e;
  if (cudaError_t e = opt_in_b.ensure(prefill_colsum_kernel<T, D>, smemB); e != cudaSuccess) return e;
  const int tiles = (max_seqlen + BM - 1) / BM;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  const int logn = (c->sh.flags & BUZZ_FLAG_LOGN) ? 1 : 0;
  (void)cudaGetLastError();   // drop a stale non-sticky error left by an earlier runtime call of the process
  prefill_attn_kernel<T, D><<<dim3(tiles, c->sh.q_heads, batch), kThreads, smemA, stream>>>(
      (const T*)q, (const T*)k, (const T*)v, cu, (T*)out, c->lse, c->sh.q_heads, c->sh.kv_heads,
      c->sh.max_prompt_tokens, scale_log2, logn);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  prefill_colsum_kernel<T, D><<<dim3(tiles, c->sh.kv_heads, batch), kThreads, smemB, stream>>>(
      (const T*)q, (const T*)k, cu, c->lse, c->pscore, c->sh.q_heads, c->sh.kv_heads,
      c->sh.max_prompt_tokens, scale_log2, logn);
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace

cudaError_t buzz_launch_prefill_simt(buzz_ctx* c, const void* q, const void* k, const void* v,
                                     const int32_t* cu, int batch, int max_seqlen, void* out,
                                     cudaStream_t stream, int* launches) {
  if (c->sh.dtype == BUZZ_BF16) {
    return c->sh.head_dim == 128
               ? launch_simt<__nv_bfloat16, 128>(c, q, k, v, cu, batch, max_seqlen, out, stream, launches)
               : launch_simt<__nv_bfloat16, 64>(c, q, k, v, cu, batch, max_seqlen, out, stream, launches);
  }
  return c->sh.head_dim == 128
             ? launch_simt<float, 128>(c, q, k, v, cu, batch, max_seqlen, out, stream, launches)
             : launch_simt<float, 64>(c, q, k, v, cu, batch, max_seqlen, out, stream, launches);
}
