// Prefill attention with per-key column sums for bf16, head_dim 128, on the Blackwell tensor
// cores: TMA-fed tcgen05 MMAs with accumulators in tensor memory (TMEM).
//
// What is computed (Eqs. 1 and 3 of the paper, and Algorithm 2's accumulated attention A):
//   O = Softmax(Q K^T / sqrt(d)) V, causal, per sequence and query head, and for every key j
//   score_j = sum over the group's query heads and rows i >= j of P_ij.
// The column sums need each row's FINAL normaliser, so S = Q K^T is formed twice:
//   pass A  (attn_tc_kernel, query-tile stationary) flash-style attention over key tiles of 64: S
//           in TMEM, one thread per row does the online softmax, P goes back to TMEM as bf16 and is
//           the A operand of the P V MMA; the output accumulator lives in TMEM and is rescaled
//           lazily (P is formed with the maximum in use; only a tile whose probabilities add up
//           to more than 2^20 makes the warp take maxima and rescale). Two CTAs share an SM.
//           Writes O and the row log2-sum-exp.
//   pass B  (colsum_tc_kernel, key-tile stationary) S^T = K Q^T in TMEM with KEYS on the TMEM
//           lanes, so one thread owns one key: it forms the exact probabilities 2^(S - lse) in
//           fp32 and adds them up over the query rows in a fixed order (heads, then tiles, then
//           rows ascending) -- no cross-thread reduction, no atomics, bit-reproducible.
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM owner; in pass A a further warp
// issues the second product), the remaining warps = one thread per TMEM lane. All mbarrier waits
// are bounded; a wait that gives up sets BUZZ_ERR_TIMEOUT and the CTA runs to its end without
// touching more data.
#include <math.h>

#include "buzz_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int D = 128;                    // head dim
constexpr int BT = 128;                   // tile edge: query rows and keys per tile
constexpr uint32_t kBlockBytes = BT * 128;          // one [128 rows x 64 bf16] swizzled block
constexpr uint32_t kTileBytes = 2 * kBlockBytes;    // a [128 x 128] bf16 tile = two blocks
constexpr float kInvLn512 = 1.0f / 6.2383246250395077f;
constexpr uint32_t kIdescKK = idesc_bf16(BT, BT, false, false);   // both operands K-major
constexpr uint32_t kIdescKM = idesc_bf16(BT, BT, false, true);    // B operand MN-major (V)

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

struct TimeoutFlag {
  int32_t* status;
  int inst;
  __device__ void raise(int where) const { buzz_set_status(status, BUZZ_ERR_TIMEOUT, inst, where); }
};

// K-major operand tile ([rows][128 dims] as two swizzled blocks): descriptor of k-step ks (16 dims).
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile_saddr, int ks) {
  return smem_desc_sw128(tile_saddr + (ks >> 2) * kBlockBytes + (ks & 3) * 32, 16, 1024);
}
// MN-major operand tile (V: [keys][128 dims]): descriptor of k-step ks (16 keys), N = 128 dims.
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t tile_saddr, int ks) {
  return smem_desc_sw128(tile_saddr + ks * 16 * 128, kBlockBytes, 1024);
}

// One [128 x 128] bf16 tile = two TMA boxes of 64 columns.
__device__ __forceinline__ void load_tile(void* dst, const CUtensorMap* map, int col0, int row0, uint64_t* bar) {
  tma_load_2d(dst, map, col0, row0, bar);
  tma_load_2d(static_cast<char*>(dst) + kBlockBytes, map, col0 + 64, row0, bar);
}

// One key's 128 logits against one query tile -> exact probabilities added into four interleaved
// accumulators (column c -> acc[c % 4]), so the summation order is fixed and the adds pipeline.
template <bool LOGN, int NC>
__device__ __forceinline__ void colsum_tile(const uint32_t (&r)[NC], const float* __restrict__ rs,
                                            const float (&lse)[NC], float scale_log2, bool diag,
                                            bool tail, int q0, int kpos, int N, float (&acc)[4]) {
  if (!diag && !tail) {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const float sc = LOGN ? rs[c] : scale_log2;
      acc[c & 3] += exp2f(fmaf(__uint_as_float(r[c]), sc, -lse[c]));
    }
  } else {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const float sc = LOGN ? rs[c] : scale_log2;
      const float p = exp2f(fmaf(__uint_as_float(r[c]), sc, -lse[c]));
      const int qpos = q0 + c;
      acc[c & 3] += (qpos >= kpos && qpos < N) ? p : 0.f;
    }
  }
}

// =================================================================================================
// Pass B: column sums. grid (key tiles, kv heads, sequences), 2 CTAs per SM. A key (TMEM lane) is
// shared by two threads, one per compute warpgroup: warpgroup g sums query columns [64g, 64g+64)
// of every tile, and the two partial sums are added in a fixed order at the end.
// =================================================================================================
// A slot of row statistics is rewritten kLseSlots iterations after it was filled. The producer fills
// the slot of iteration `it` once the MMA of it-2 has completed, which was issued only after every
// compute thread had taken the logits of it-4 out of TMEM, i.e. had finished iteration it-5.
constexpr int kLseSlots = 8;
// Row statistics are stored with each sequence's rows starting at a multiple of four floats, so
// that a tile's 128 values can be fetched with one 16-byte-aligned bulk copy.
__device__ __forceinline__ int lse_offset(int tok0, int b) { return (tok0 & ~3) + 4 * b; }
struct SmemB {
  alignas(1024) unsigned char k[kTileBytes];
  alignas(1024) unsigned char q[2][kTileBytes];
  alignas(16) float lse[kLseSlots][BT];    // row log-sum-exp of the query tile of iteration it, slot it % kLseSlots (bulk-copied)
  float rs[2][8][64];                      // log-n row scales, [tile parity][compute warp][column of its half]: per-warp copies
  float part[BT];                          // warpgroup 1's partial column sums
  uint64_t k_full, q_full[2], q_empty[2], s_full[2], s_empty[2], lse_full[kLseSlots];
  uint32_t tmem_base;
};

constexpr int kThreadsB = 320;            // TMA warp, MMA warp, 2 x 4 compute warps
__global__ void __launch_bounds__(kThreadsB, 2)
colsum_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const int32_t* __restrict__ cu, const float* __restrict__ lse, float* __restrict__ pscore,
                 int32_t* status, int Hq, int Hkv, int stride, int lse_stride, float scale_log2, int logn) {
  extern __shared__ unsigned char smem_raw[];
  SmemB& sm = *reinterpret_cast<SmemB*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int b = blockIdx.z, kvh = blockIdx.y, G = Hq / Hkv;
  const int tok0 = cu[b], N = cu[b + 1] - tok0;
  const int kt = blockIdx.x, key0 = kt * BT;
  if (key0 >= N) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q_tiles = (N + BT - 1) / BT;
  const int nq = q_tiles - kt;
  const int iters = G * nq;
  const TimeoutFlag tf{status, (b * Hkv + kvh) * 4096 + kt};

  if (threadIdx.x == 0) {
    mbar_init(&sm.k_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.q_full[s], 1);
      mbar_init(&sm.q_empty[s], 1);
      mbar_init(&sm.s_full[s], 1);
      mbar_init(&sm.s_empty[s], 256);
    }
    for (int s = 0; s < kLseSlots; ++s) mbar_init(&sm.lse_full[s], 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0) {
    // ---- TMA producer ----
    if (elect_one()) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      mbar_expect_tx(&sm.k_full, kTileBytes);
      load_tile(sm.k, &map_k, kvh * D, tok0 + key0, &sm.k_full);
      int pg = 0, pqt = kt;
      for (int it = 0; it < iters; ++it) {
        const int st = it & 1, use = it >> 1;
        if (use > 0 && !mbar_wait(&sm.q_empty[st], (use - 1) & 1)) { tf.raise(1); break; }
        mbar_expect_tx(&sm.q_full[st], kTileBytes);
        load_tile(sm.q[st], &map_q, (kvh * G + pg) * D, tok0 + pqt * BT, &sm.q_full[st]);
        // the tile's row statistics: a barrier of their own, because the threads that read them must
        // observe the copy's completion themselves (q_full may be two phases ahead by then)
        mbar_expect_tx(&sm.lse_full[it % kLseSlots], BT * 4);
        bulk_load_1d(sm.lse[it % kLseSlots], lse + (size_t)(kvh * G + pg) * lse_stride + lse_offset(tok0, b) + pqt * BT,
                     BT * 4, &sm.lse_full[it % kLseSlots]);
        if (++pqt == q_tiles) { pqt = kt; ++pg; }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: S^T[keys x rows] = K Q^T ----
    if (elect_one()) {
      bool ok = mbar_wait(&sm.k_full, 0);
      if (!ok) tf.raise(2);
      for (int it = 0; ok && it < iters; ++it) {
        const int st = it & 1, use = it >> 1;
        if (!mbar_wait(&sm.q_full[st], use & 1)) { tf.raise(3); break; }
        if (use > 0 && !mbar_wait(&sm.s_empty[st], (use - 1) & 1)) { tf.raise(4); break; }
        tc_fence_after();
        const uint32_t ka = smem_u32(sm.k), qa = smem_u32(sm.q[st]);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          mma_ss(tmem + st * BT, kmajor_desc(ka, ks), kmajor_desc(qa, ks), kIdescKK, ks > 0);
        mma_commit(&sm.s_full[st]);
        mma_commit(&sm.q_empty[st]);
      }
    }
  } else {
    // ---- thread (g, key): exact probabilities of query columns [64g, 64g+64), summed down the column ----
    const int g = (warp - 2) >> 2;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;              // TMEM lane = key within the tile
    const int kpos = key0 + row;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};           // column c adds into acc[c % 4]: a fixed order
    bool ok = true;
    const int cw = warp - 2;                          // compute warp 0..7
    int qt = kt, ntile = kt;                          // this iteration's query tile; the next one's
    for (int it = 0; it < iters; ++it) {
      const int st = it & 1, use = it >> 1;
      qt = ntile;
      if (++ntile == q_tiles) ntile = kt;
      const int q0 = qt * BT;
      if (logn) {                                     // this warp's private copy of its columns' row scales
        sm.rs[st][cw][lane] = scale_log2 * __logf((float)(q0 + g * 64 + lane + 1)) * kInvLn512;
        sm.rs[st][cw][lane + 32] = scale_log2 * __logf((float)(q0 + g * 64 + lane + 33)) * kInvLn512;
        __syncwarp();
      }
      if (!mbar_wait(&sm.lse_full[it % kLseSlots], (it / kLseSlots) & 1)) { tf.raise(6); ok = false; break; }
      if (!mbar_wait(&sm.s_full[st], use & 1)) { tf.raise(5); ok = false; break; }
      tc_fence_after();
      const bool diag = (qt == kt), tail = (q0 + BT > N);
      // this thread's 64 logits in two halves of 32: the logits from TMEM and the columns' row statistics
      // from shared memory (16-byte loads: memory instructions queue behind the exponentials), then 32
      // independent exponentials
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t r[32];
        float ls[32];
        tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + st * BT + g * 64 + h * 32, r);
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          const float4 t = *reinterpret_cast<const float4*>(&sm.lse[it % kLseSlots][g * 64 + h * 32 + c]);
          ls[c] = t.x; ls[c + 1] = t.y; ls[c + 2] = t.z; ls[c + 3] = t.w;
        }
        tmem_wait_ld();
        tmem_pin32(r);
        if (h == 1) {
          tc_fence_before();
          mbar_arrive(&sm.s_empty[st]);                // S^T[st] may be overwritten once all 256 have arrived
        }
        if (logn) colsum_tile<true, 32>(r, sm.rs[st][cw] + h * 32, ls, scale_log2, diag, tail, q0 + g * 64 + h * 32, kpos, N, acc);
        else colsum_tile<false, 32>(r, sm.rs[st][cw] + h * 32, ls, scale_log2, diag, tail, q0 + g * 64 + h * 32, kpos, N, acc);
      }
      if (logn) __syncwarp();                         // the row-scale copy is rewritten two iterations from now
    }
    const float mine = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    if (g == 1) sm.part[row] = mine;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (g == 0 && ok && kpos < N) pscore[(size_t)kvh * stride + tok0 + kpos] = mine + sm.part[row];
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// =================================================================================================
// Pass A: attention output and row log-sum-exp. grid (query tiles, query heads, sequences), TWO
// CTAs per SM. A CTA owns 128 query rows and walks the keys in tiles of 64, one thread per row:
//   TMEM columns (256 per CTA): S0 [0,64)  S1 [64,128)  O [128,256).
// P (bf16 pairs, 32 columns) overwrites the start of the S buffer it was computed from. The
// tensor core may still be reading P as the A operand long after the MMA was issued, so the
// logits that reuse an S buffer are only issued once the P V product on it has been seen to
// complete (pv_done). Inside one CTA the chain logits -> softmax -> P V -> next-but-one logits is
// latency-bound (every barrier hand-over costs a few hundred cycles, more when the memory
// instruction queue is full of exponentials); the second CTA on the SM fills those gaps, and
// CTAs starting and finishing overlap with one in full flight.
// Three warps do the asynchronous work: TMA producer, Q K^T issuer, P V issuer (one issuing
// thread for both products was the longest serial chain in the loop).
// =================================================================================================
constexpr int KT = 64;                    // keys per tile in pass A
constexpr uint32_t kKvBlockBytes = KT * 128;        // one [64 keys x 64 bf16] swizzled block
constexpr uint32_t kKvTileBytes = 2 * kKvBlockBytes;
constexpr int kThreadsA = 224;            // TMA warp, Q K^T issuer, 4 softmax warps, P V issuer
constexpr int kStagesA = 2;
constexpr uint32_t kIdescQK = idesc_bf16(BT, KT, false, false);
struct SmemA {
  alignas(1024) unsigned char q[kTileBytes];
  alignas(1024) unsigned char k[kStagesA][kKvTileBytes];
  alignas(1024) unsigned char v[kStagesA][kKvTileBytes];
  float xch[BT];
  uint64_t q_full, k_full[kStagesA], k_empty[kStagesA], v_full[kStagesA], v_empty[kStagesA];
  uint64_t s_full[2], p_full[2], pv_done[2];
  uint32_t tmem_base;
};
constexpr uint32_t kColO = 128;
// A speculative tile stands while its probabilities add up to at most 2^20 (P, the row sums and O stay
// far inside the fp32/bf16 exponent range). When one does not, every row of the warp whose maximum
// has grown by more than 2^8 since it was last set is brought up to date, so that a row is not
// caught again at the next tile.
constexpr float kRescaleThreshold = 8.0f;
constexpr float kSpeculationLimit = 1048576.0f;

// K-major [64 keys][128 dims] tile as two swizzled blocks: descriptor of k-step ks (16 dims).
__device__ __forceinline__ uint64_t kmajor_desc_kv(uint32_t tile_saddr, int ks) {
  return smem_desc_sw128(tile_saddr + (ks >> 2) * kKvBlockBytes + (ks & 3) * 32, 16, 1024);
}
// MN-major V tile [64 keys][128 dims]: descriptor of k-step ks (16 keys), N = 128 dims.
__device__ __forceinline__ uint64_t mnmajor_desc_kv(uint32_t tile_saddr, int ks) {
  return smem_desc_sw128(tile_saddr + ks * 16 * 128, kKvBlockBytes, 1024);
}
__device__ __forceinline__ void load_kv_tile(void* dst, const CUtensorMap* map, int col0, int row0, uint64_t* bar) {
  tma_load_2d(dst, map, col0, row0, bar);
  tma_load_2d(static_cast<char*>(dst) + kKvBlockBytes, map, col0 + 64, row0, bar);
}

__global__ void __launch_bounds__(kThreadsA, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const int32_t* __restrict__ cu,
               __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int32_t* status, int Hq, int Hkv,
               int stride, float scale_log2, int logn) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  SmemA& sm = *reinterpret_cast<SmemA*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int b = blockIdx.z, h = blockIdx.y, kvh = h / (Hq / Hkv);
  const int tok0 = cu[b], N = cu[b + 1] - tok0;
  const int qt = gridDim.x - 1 - blockIdx.x;          // heaviest (last) query tiles first
  const int row0 = qt * BT;
  if (row0 >= N) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nt = min(2 * qt + 2, (N + KT - 1) / KT);  // key tiles 0 .. (causal, clipped to the sequence)
  const TimeoutFlag tf{status, (b * Hq + h) * 4096 + qt};

  if (threadIdx.x == 0) {
    mbar_init(&sm.q_full, 1);
    for (int s = 0; s < kStagesA; ++s) {
      mbar_init(&sm.k_full[s], 1); mbar_init(&sm.k_empty[s], 1);
      mbar_init(&sm.v_full[s], 1); mbar_init(&sm.v_empty[s], 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&sm.s_full[s], 1); mbar_init(&sm.pv_done[s], 1); mbar_init(&sm.p_full[s], 128);
    }
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_base, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;

  if (warp == 0) {
    // ---- TMA producer ----
    if (elect_one()) {
      prefetch_tensormap(&map_q); prefetch_tensormap(&map_k); prefetch_tensormap(&map_v);
      mbar_expect_tx(&sm.q_full, kTileBytes);
      load_tile(sm.q, &map_q, h * D, tok0 + row0, &sm.q_full);
      for (int j = 0; j < nt; ++j) {
        const int st = j % kStagesA, use = j / kStagesA;
        if (use > 0 && !mbar_wait(&sm.k_empty[st], (use - 1) & 1)) { tf.raise(11); break; }
        mbar_expect_tx(&sm.k_full[st], kKvTileBytes);
        load_kv_tile(sm.k[st], &map_k, kvh * D, tok0 + j * KT, &sm.k_full[st]);
        if (use > 0 && !mbar_wait(&sm.v_empty[st], (use - 1) & 1)) { tf.raise(12); break; }
        mbar_expect_tx(&sm.v_full[st], kKvTileBytes);
        load_kv_tile(sm.v[st], &map_v, kvh * D, tok0 + j * KT, &sm.v_full[st]);
      }
    }
  } else if (warp == 1) {
    // ---- Q K^T issuer: S[j%2] = Q K_j^T, up to two tiles ahead of the softmax ----
    if (elect_one()) {
      const uint32_t qa = smem_u32(sm.q);
      bool ok = mbar_wait(&sm.q_full, 0);
      if (!ok) tf.raise(14);
      for (int j = 0; ok && j < nt; ++j) {
        const int st = j % kStagesA;
        if (!mbar_wait(&sm.k_full[st], (j / kStagesA) & 1)) { tf.raise(13); break; }
        // S[j%2] still holds P of tile j-2: its P V product must have completed
        if (j >= 2 && !mbar_wait(&sm.pv_done[j & 1], ((j - 2) >> 1) & 1)) { tf.raise(21); break; }
        tc_fence_after();
        const uint32_t ka = smem_u32(sm.k[st]);
#pragma unroll
        for (int s = 0; s < D / 16; ++s)
          mma_ss(tmem + (j & 1) * KT, kmajor_desc(qa, s), kmajor_desc_kv(ka, s), kIdescQK, s > 0);
        mma_commit(&sm.s_full[j & 1]);
        mma_commit(&sm.k_empty[st]);
      }
    }
  } else if (warp == 6) {
    // ---- P V issuer: O += P V_j, 16 keys per step ----
    if (elect_one()) {
      for (int j = 0; j < nt; ++j) {
        const int sb = j & 1, st = j % kStagesA;
        if (!mbar_wait(&sm.v_full[st], (j / kStagesA) & 1)) { tf.raise(16); break; }
        if (!mbar_wait(&sm.p_full[sb], (j >> 1) & 1)) { tf.raise(15); break; }
        tc_fence_after();
        const uint32_t va = smem_u32(sm.v[st]);
#pragma unroll
        for (int s = 0; s < KT / 16; ++s)
          mma_ts(tmem + kColO, tmem + sb * KT + s * 8, mnmajor_desc_kv(va, s), kIdescKM, (j > 0 || s > 0) ? 1u : 0u);
        mma_commit(&sm.v_empty[st]);
        mma_commit(&sm.pv_done[sb]);
      }
    }
  } else {
    // ---- softmax: one thread per query row, 64 logits per tile ----
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int qpos = row0 + row;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    // Row scale. With log-n scaling the first row of a sequence has log_512(1) = 0: its only unmasked
    // logit is scaled to 0 and its probability is 1. The scale is kept a hair above zero there so that
    // a masked logit (-inf) times the scale stays -inf instead of becoming NaN; a finite logit times
    // 1e-30 is 0 to far below fp32 resolution, so row 0 still gets exactly P = 1.
    const float rs = logn ? fmaxf(scale_log2 * __logf((float)(qpos + 1)) * kInvLn512, 1e-30f) : scale_log2;
    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < nt; ++j) {
      const int sb = j & 1;
      const uint32_t colS = sb * KT;
      if (!mbar_wait(&sm.s_full[sb], (j >> 1) & 1)) { tf.raise(17); ok = false; break; }
      tc_fence_after();
      // the raw logits of this row (rs > 0 always, see above, so the maximum can be taken before scaling)
      uint32_t sa[32], sb2[32];
      tmem_ld32(tmem + lane_base + colS, sa);
      tmem_ld32(tmem + lane_base + colS + 32, sb2);
      tmem_wait_ld();
      tmem_pin32(sa);
      tmem_pin32(sb2);
      float s[64];
#pragma unroll
      for (int c = 0; c < 32; ++c) { s[c] = __uint_as_float(sa[c]); s[32 + c] = __uint_as_float(sb2[c]); }
      if (j * KT + KT - 1 > row0) {                    // a tile that crosses the diagonal: causal mask
#pragma unroll
        for (int c = 0; c < 64; ++c)
          if (j * KT + c > qpos) s[c] = -INFINITY;
      }
      // P = 2^(S rs - m) as bf16 pairs (they will overwrite the first 32 columns of this S buffer) and their sum
      uint32_t pk[32];
      float tile_sum = 0.f;
      auto exp_pass = [&]() {
        const float neg_m = -m_used;
        float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float p0 = exp2f(fmaf(s[2 * c], rs, neg_m));
          const float p1 = exp2f(fmaf(s[2 * c + 1], rs, neg_m));
          l4[c & 3] += p0 + p1;
          const __nv_bfloat162 pp = __floats2bfloat162_rn(p0, p1);
          pk[c] = *reinterpret_cast<const uint32_t*>(&pp);
        }
        tile_sum = (l4[0] + l4[1]) + (l4[2] + l4[3]);
      };
      // After the first tile the maximum in use is almost always good enough (a stale maximum only
      // makes P, the row sum and O larger by the same factor), so P is formed SPECULATIVELY with it and
      // the pass over the logits that takes their maximum is skipped: if the tile's probabilities add
      // up to no more than kSpeculationLimit, none of them exceeds it and the tile stands. Otherwise
      // (some row of the warp says so, or an overflow made the sum infinite) the maximum is taken
      // properly, O is rescaled where needed and P is formed again.
      bool settled = false;
      if (j > 0) {
        exp_pass();
        settled = !__any_sync(0xffffffffu, !(tile_sum <= kSpeculationLimit));
      }
      if (!settled) {
        float mx4[4] = {s[0], s[1], s[2], s[3]};       // four chains of three-input maxima over s[4..63]
#pragma unroll
        for (int c = 4; c + 8 <= 64; c += 8) {         // s[4..59]
#pragma unroll
          for (int e = 0; e < 4; ++e) mx4[e] = max3(mx4[e], s[c + 2 * e], s[c + 2 * e + 1]);
        }
        mx4[0] = max3(mx4[0], s[60], s[61]);
        mx4[1] = max3(mx4[1], s[62], s[63]);
        const float mx = fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]) * rs;   // -inf if the whole tile is masked for this row
        const float m_new = fmaxf(m_used, mx);
        if (j == 0) {
          m_used = m_new;                              // finite: key 0 is never masked
        } else {
          const bool need = m_new > m_used + kRescaleThreshold;
          if (__any_sync(0xffffffffu, need)) {
            const float alpha = need ? exp2f(m_used - m_new) : 1.0f;
            if (need) m_used = m_new;
            l *= alpha;
            if (!mbar_wait(&sm.pv_done[(j - 1) & 1], ((j - 1) >> 1) & 1)) { tf.raise(18); ok = false; break; }   // P V of tile j-1 landed
            tc_fence_after();
#pragma unroll 1
            for (int c0 = 0; c0 < D; c0 += 32) {
              uint32_t r[32];
              tmem_ld32(tmem + lane_base + kColO + c0, r);
              tmem_wait_ld();
              tmem_pin32(r);
#pragma unroll
              for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
              tmem_st32(tmem + lane_base + kColO + c0, r);
            }
            tmem_wait_st();
          }
        }
        exp_pass();
      }
      tmem_st32(tmem + lane_base + colS, pk);
      l += tile_sum;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&sm.p_full[sb]);
    }
    // ---- epilogue: O / l -> bf16, row log2-sum-exp ----
    if (ok && !mbar_wait(&sm.pv_done[(nt - 1) & 1], ((nt - 1) >> 1) & 1)) { tf.raise(19); ok = false; }
    tc_fence_after();
    if (ok) {
      const float inv = 1.0f / l;
      __nv_bfloat16* orow = out + ((size_t)(tok0 + qpos) * Hq + h) * D;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t r0[32];
        tmem_ld32(tmem + lane_base + kColO + c0, r0);
        tmem_wait_ld();
        tmem_pin32(r0);
        if (qpos < N) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            float o[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = __uint_as_float(r0[c + e]) * inv;
            uint4 w;
            __nv_bfloat162 t0 = __floats2bfloat162_rn(o[0], o[1]), t1 = __floats2bfloat162_rn(o[2], o[3]);
            __nv_bfloat162 t2 = __floats2bfloat162_rn(o[4], o[5]), t3 = __floats2bfloat162_rn(o[6], o[7]);
            w.x = *reinterpret_cast<uint32_t*>(&t0); w.y = *reinterpret_cast<uint32_t*>(&t1);
            w.z = *reinterpret_cast<uint32_t*>(&t2); w.w = *reinterpret_cast<uint32_t*>(&t3);
            *reinterpret_cast<uint4*>(orow + c0 + c) = w;
          }
        }
      }
      if (qpos < N) lse[(size_t)h * stride + lse_offset(tok0, b) + qpos] = m_used + log2f(l);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// ---- host side --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [tokens][heads * 128] bf16, boxes of 64 columns x 128 rows, 128-byte swizzle, zero fill out of range.
bool make_map(CUtensorMap* map, const void* base, int tokens, int heads, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)heads * D, (cuuint64_t)tokens};
  const cuuint64_t strides[1] = {(cuuint64_t)heads * D * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t buzz_launch_prefill_tc(buzz_ctx* c, const void* q, const void* k, const void* v,
                                   const int32_t* cu, int batch, int total_tokens, int max_seqlen,
                                   void* out, cudaStream_t stream, int* launches) {
  CUtensorMap mq, mk, mk64, mv64;                      // 128-row boxes for Q and pass B's keys, 64-row boxes for pass A's K and V
  if (!make_map(&mq, q, total_tokens, c->sh.q_heads, BT) || !make_map(&mk, k, total_tokens, c->sh.kv_heads, BT) ||
      !make_map(&mk64, k, total_tokens, c->sh.kv_heads, KT) || !make_map(&mv64, v, total_tokens, c->sh.kv_heads, KT))
    return cudaErrorInvalidValue;
  const size_t smemA = sizeof(SmemA) + 1024, smemB = sizeof(SmemB) + 1024;
  static BuzzSmemOptIn opt_in_a, opt_in_b;
  if (cudaError_t e = opt_in_a.ensure(attn_tc_kernel, smemA); e != cudaSuccess) return e;
  if (cudaError_t e = opt_in_b.ensure(colsum_tc_kernel, smemB); e != cudaSuccess) return e;
  const int tiles = (max_seqlen + BT - 1) / BT;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)D);
  const int logn = (c->sh.flags & BUZZ_FLAG_LOGN) ? 1 : 0;
  (void)cudaGetLastError();   // drop a stale non-sticky error left by an earlier runtime call of the process
  attn_tc_kernel<<<dim3(tiles, c->sh.q_heads, batch), kThreadsA, smemA, stream>>>(
      mq, mk64, mv64, cu, (__nv_bfloat16*)out, c->lse, c->st.status, c->sh.q_heads, c->sh.kv_heads,
      c->lse_stride, scale_log2, logn);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  colsum_tc_kernel<<<dim3(tiles, c->sh.kv_heads, batch), kThreadsB, smemB, stream>>>(
      mq, mk, cu, c->lse, c->pscore, c->st.status, c->sh.q_heads, c->sh.kv_heads, c->sh.max_prompt_tokens, c->lse_stride,
      scale_log2, logn);
  *launches += 2;
  return cudaGetLastError();
}
