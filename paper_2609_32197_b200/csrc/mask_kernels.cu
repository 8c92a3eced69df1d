// Step 1: mean-pool Q and K per block, score pooled-Q x pooled-K^T per head (fp32 SIMT GEMM with a
// fixed accumulation order), warp-level top-k per row.
//
// Arithmetic contract (the result decides which blocks are kept, so it is fixed to the operation):
//   pool : fp32 sum of the block's valid tokens in ascending token order starting from 0, then one
//          IEEE division by the valid count;
//   score: acc = fmaf(q_c, k_c, acc) from acc = 0, channel c ascending;
//   top-k: score descending, index ascending on equal scores, -0 == +0.
#include "common.cuh"

namespace sparsp {

// ------------------------------------------------------------------------------------------------
// pool: a group of d/8 lanes owns one (tensor, batch*head, block) tile; lane l owns channels
// 8l..8l+7 and walks the tile's rows with 16-byte loads, so every channel is one sequential chain.
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) pool_kernel(const __nv_bfloat16* __restrict__ Q,
                                                   const __nv_bfloat16* __restrict__ K,
                                                   float* __restrict__ pq, float* __restrict__ pk,
                                                   int H, int NB, int b, int64_t N, int64_t sB,
                                                   int64_t sH, int64_t sT, int64_t n_tiles) {
  constexpr int G = D / 8;  // lanes per tile
  constexpr int U = 8;      // rows in flight per lane
  const int64_t tile = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int lane = threadIdx.x % G;
  if (tile >= 2 * n_tiles) return;
  const bool is_k = tile >= n_tiles;
  const int64_t t = is_k ? tile - n_tiles : tile;  // (batch*H + head) * NB + block
  const int blk = (int)(t % NB);
  const int64_t bh = t / NB;
  const int64_t batch = bh / H, head = bh % H;
  const int64_t tok0 = (int64_t)blk * b;
  const int n = (int)min((int64_t)b, N - tok0);
  const __nv_bfloat16* src = (is_k ? K : Q) + batch * sB + head * sH + tok0 * sT + lane * 8;

  float acc[8];
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] = 0.0f;

  int r = 0;
  for (; r + U <= n; r += U) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) v[u] = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)(r + u) * sT));
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        acc[2 * p] = __fadd_rn(acc[2 * p], __uint_as_float(w[p] << 16));
        acc[2 * p + 1] = __fadd_rn(acc[2 * p + 1], __uint_as_float(w[p] & 0xffff0000u));
      }
    }
  }
  for (; r < n; ++r) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)r * sT));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      acc[2 * p] = __fadd_rn(acc[2 * p], __uint_as_float(w[p] << 16));
      acc[2 * p + 1] = __fadd_rn(acc[2 * p + 1], __uint_as_float(w[p] & 0xffff0000u));
    }
  }
  const float cntf = (float)n;
  float* dst = (is_k ? pk : pq) + t * D + lane * 8;
  float4 o0, o1;
  o0.x = __fdiv_rn(acc[0], cntf);
  o0.y = __fdiv_rn(acc[1], cntf);
  o0.z = __fdiv_rn(acc[2], cntf);
  o0.w = __fdiv_rn(acc[3], cntf);
  o1.x = __fdiv_rn(acc[4], cntf);
  o1.y = __fdiv_rn(acc[5], cntf);
  o1.z = __fdiv_rn(acc[6], cntf);
  o1.w = __fdiv_rn(acc[7], cntf);
  reinterpret_cast<float4*>(dst)[0] = o0;
  reinterpret_cast<float4*>(dst)[1] = o1;
}

int launch_pool(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, float* pq,
                float* pk, cudaStream_t st) {
  const int64_t n_tiles = (int64_t)g.B * g.H * g.NB;
  const int G = g.d / 8;
  const int64_t threads = 2 * n_tiles * G;
  const int grid = (int)((threads + 255) / 256);
  auto q = (const __nv_bfloat16*)Q;
  auto k = (const __nv_bfloat16*)K;
  if (g.d == 64)
    pool_kernel<64><<<grid, 256, 0, st>>>(q, k, pq, pk, g.H, g.NB, g.b, g.N, s.stride_batch,
                                          s.stride_head, s.stride_token, n_tiles);
  else
    pool_kernel<128><<<grid, 256, 0, st>>>(q, k, pq, pk, g.H, g.NB, g.b, g.N, s.stride_batch,
                                           s.stride_head, s.stride_token, n_tiles);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

// ------------------------------------------------------------------------------------------------
// score: S[bh][i][j] = sum_c pQ[i][c] * pK[j][c] as one fused-multiply-add chain per output, c
// ascending (a no-split-K SIMT GEMM).  A CTA computes a 64 x 64 tile; a thread owns 4 rows x 4
// columns (columns tx, tx+16, tx+32, tx+48 so that its 16-byte shared-memory reads of pooled K never
// conflict), i.e. 16 independent chains fed by 8 vector loads per 4 channels.  Scores go to a
// workspace buffer: at most 83 MB, written and read once, ~25 us of HBM time on the largest workload.
// ------------------------------------------------------------------------------------------------
constexpr int kScoreTile = 64;
constexpr int kScoreThreads = 256;

template <int D>
__global__ void __launch_bounds__(kScoreThreads) score_kernel(const float* __restrict__ pq,
                                                              const float* __restrict__ pk, int NB,
                                                              float* __restrict__ scores) {
  constexpr int LD = D + 4;  // row pitch in floats: 16 bytes of skew per row
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* sQ = reinterpret_cast<float*>(smem_raw);  // [64][LD]
  float* sK = sQ + kScoreTile * LD;                // [64][LD]
  const int64_t bh = blockIdx.z;
  const int row0 = blockIdx.y * kScoreTile, col0 = blockIdx.x * kScoreTile;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;

  for (int idx = threadIdx.x; idx < kScoreTile * (D / 4); idx += kScoreThreads) {
    const int r = idx / (D / 4), c4 = idx % (D / 4);
    float4 q = make_float4(0.f, 0.f, 0.f, 0.f), k = q;
    if (row0 + r < NB) q = __ldg(reinterpret_cast<const float4*>(pq + (bh * NB + row0 + r) * D) + c4);
    if (col0 + r < NB) k = __ldg(reinterpret_cast<const float4*>(pk + (bh * NB + col0 + r) * D) + c4);
    *reinterpret_cast<float4*>(sQ + r * LD + c4 * 4) = q;
    *reinterpret_cast<float4*>(sK + r * LD + c4 * 4) = k;
  }
  __syncthreads();

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

#pragma unroll 4
  for (int c = 0; c < D; c += 4) {
    float4 q[4], k[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) q[i] = *reinterpret_cast<const float4*>(sQ + (ty * 4 + i) * LD + c);
#pragma unroll
    for (int j = 0; j < 4; ++j) k[j] = *reinterpret_cast<const float4*>(sK + (tx + 16 * j) * LD + c);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float a = acc[i][j];
        a = __fmaf_rn(q[i].x, k[j].x, a);
        a = __fmaf_rn(q[i].y, k[j].y, a);
        a = __fmaf_rn(q[i].z, k[j].z, a);
        a = __fmaf_rn(q[i].w, k[j].w, a);
        acc[i][j] = a;
      }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = row0 + ty * 4 + i;
    if (r >= NB) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int cidx = col0 + tx + 16 * j;
      if (cidx < NB) scores[(bh * NB + r) * NB + cidx] = acc[i][j];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// top-k: one warp per (batch, head, query block) row.  The row's scores become order-preserving
// uint32 keys in registers (lane l holds blocks l, l + 32, ...); the warp finds the k-th largest key by a 32-step radix search with
// ballots/popcounts, breaks ties towards the lower index, forces the text blocks on, and emits the
// mask words and the ascending kept list by ballot-prefix compaction.
// ------------------------------------------------------------------------------------------------
constexpr int kTopkWarps = 8;

__device__ __forceinline__ uint32_t score_key(float s) {
  if (s == 0.0f) s = 0.0f;  // -0 -> +0 so that they compare equal
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int WMAX>  // mask words per row this instance can hold (keys live in registers: WMAX per lane)
__global__ void __launch_bounds__(kTopkWarps * 32) topk_kernel(const float* __restrict__ scores, int64_t n_rows,
                                                               int NB, int Wd, int nb_cand, int topk,
                                                               int kept_cap, uint32_t* __restrict__ mask,
                                                               int32_t* __restrict__ kv_list,
                                                               int32_t* __restrict__ kv_count) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kTopkWarps + warp;  // (batch*H + head) * NB + i
  if (row >= n_rows) return;
  const float* srow = scores + row * NB;
  // lane l holds the keys of blocks l, l + 32, ...; a block that is not a candidate (text, padding) holds 0,
  // which no trial threshold (>= 1) counts
  uint32_t key[WMAX];
#pragma unroll
  for (int t = 0; t < WMAX; ++t) {
    const int j = t * 32 + lane;
    key[t] = (t < Wd && j < nb_cand) ? score_key(__ldcs(srow + j)) : 0u;
  }

  const uint32_t lt_mask = (1u << lane) - 1u;
  // largest T with |{ candidates : key >= T }| >= topk  ==> T is the topk-th largest key
  uint32_t T = 0;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t trial = T | (1u << bit);
    int c = 0;
#pragma unroll
    for (int t = 0; t < WMAX; ++t) c += key[t] >= trial ? 1 : 0;
    c = __reduce_add_sync(0xffffffffu, c);
    if (c >= topk) T = trial;
  }
  int gt = 0;
#pragma unroll
  for (int t = 0; t < WMAX; ++t) gt += key[t] > T ? 1 : 0;
  gt = __reduce_add_sync(0xffffffffu, gt);
  const int need_eq = topk - gt;  // ties at T taken in ascending index order
  int eq_seen = 0, out_pos = 0;
#pragma unroll
  for (int t = 0; t < WMAX; ++t) {
    if (t < Wd) {
      const int j = t * 32 + lane;
      const bool cand = j < nb_cand;
      const bool is_eq = cand && key[t] == T;
      const uint32_t eq_ballot = __ballot_sync(0xffffffffu, is_eq);
      const bool take_eq = is_eq && (eq_seen + __popc(eq_ballot & lt_mask) < need_eq);
      eq_seen += __popc(eq_ballot);
      const bool keep = (cand && key[t] > T) || take_eq || (j >= nb_cand && j < NB);
      const uint32_t word = __ballot_sync(0xffffffffu, keep);
      if (lane == 0) mask[row * Wd + t] = word;
      if (kv_list && keep) {
        const int pos = out_pos + __popc(word & lt_mask);
        if (pos < kept_cap) kv_list[row * kept_cap + pos] = j;
      }
      out_pos += __popc(word);
    }
  }
  if (kv_count && lane == 0) kv_count[row] = out_pos;
}

// ------------------------------------------------------------------------------------------------
// CDF-threshold selection (Section 8.1): per row, softmax over the candidate scores, keep the smallest
// top set by score (whole groups of equal scores) whose mass reaches tau.  The mass is counted in integers, so
// that the kept set does not depend on the order of the additions:
//   x_j = (S_j - max S) * (scale * log2 e)  (fp32);  p_j = exp2c(x_j)  (fp32: clamp at -125, nearest-integer
//   split, degree-5 Horner polynomial with fused multiply-adds, integer part added into the exponent field);
//   w_j = floor(p_j * 2^26);  Z = sum w_j;  kept = { key >= T } for the largest T with
//   mass{ key >= T } >= ceil(tau * Z), the product taken once in fp64.
// One warp per row; T is found by a 32-step search over the order-preserving key space, which is valid
// because the mass of { key >= t } never grows with t.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float exp2c(float x) {
  x = fmaxf(x, -125.0f);
  const float fi = rintf(x);
  const float f = x - fi;
  float p = 0.0013400432653725147f;
  p = fmaf(p, f, 0.009676037356257439f);
  p = fmaf(p, f, 0.05550327152013779f);
  p = fmaf(p, f, 0.2402210682630539f);
  p = fmaf(p, f, 0.6931471824645996f);
  p = fmaf(p, f, 1.0000001192092896f);
  return __int_as_float(__float_as_int(p) + (int)fi * (1 << 23));
}

// Sum over the warp of one 32-bit partial sum per lane (each < 2^32, the total needs up to 37 bits): the halves of
// the partial sums are added by the warp-reduction instruction and put together again.
__device__ __forceinline__ unsigned long long warp_sum(uint32_t v) {
  const uint32_t lo = __reduce_add_sync(0xffffffffu, v & 0xffffu), hi = __reduce_add_sync(0xffffffffu, v >> 16);
  return ((unsigned long long)hi << 16) + lo;
}

template <int WMAX>  // mask words per row this instance can hold (keys and terms live in registers)
__global__ void __launch_bounds__(kTopkWarps * 32) cdf_kernel(const float* __restrict__ scores, int64_t n_rows, int NB,
                                                              int Wd, int nb_cand, float tau, float c,
                                                              uint32_t* __restrict__ mask,
                                                              int32_t* __restrict__ kv_count) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * kTopkWarps + warp;  // (batch*H + head) * NB + i
  if (row >= n_rows) return;
  const float* srow = scores + row * NB;
  // lane l holds blocks l, l + 32, ...  A block that is not a candidate holds key 0 (no trial threshold, all
  // >= 1, selects it) and the weight 0.
  uint32_t key[WMAX];
  uint32_t w[WMAX];
  float mx = -INFINITY;
#pragma unroll
  for (int t = 0; t < WMAX; ++t) {
    const int j = t * 32 + lane;
    const bool cand = t < Wd && j < nb_cand;
    const float s = cand ? __ldcs(srow + j) : -INFINITY;
    w[t] = __float_as_uint(s);
    key[t] = cand ? score_key(s) : 0u;
    mx = fmaxf(mx, s);
  }
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
  uint32_t acc = 0;  // at most 32 terms of at most 2^26 + 8 each
#pragma unroll
  for (int t = 0; t < WMAX; ++t) {
    const int j = t * 32 + lane;
    uint32_t wj = 0u;
    if (t < Wd && j < nb_cand) {
      // the scaling is exact, the conversion truncates
      wj = __float2uint_rz(__fmul_rn(exp2c(__fmul_rn(__fsub_rn(__uint_as_float(w[t]), mx), c)), 67108864.0f));
      acc += wj;
    }
    w[t] = wj;
  }
  const unsigned long long theta = (unsigned long long)ceil(__dmul_rn((double)tau, (double)warp_sum(acc)));
  // largest T with mass{ key >= T } >= theta
  uint32_t T = 0;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t trial = T | (1u << bit);
    uint32_t m = 0;
#pragma unroll
    for (int t = 0; t < WMAX; ++t) m += key[t] >= trial ? w[t] : 0u;
    if (warp_sum(m) >= theta) T = trial;
  }
  int cnt = 0;
#pragma unroll
  for (int t = 0; t < WMAX; ++t) {
    if (t < Wd) {
      const int j = t * 32 + lane;
      const bool keep = (j < nb_cand && key[t] >= T) || (j >= nb_cand && j < NB);
      const uint32_t word = __ballot_sync(0xffffffffu, keep);
      if (lane == 0) mask[row * Wd + t] = word;
      cnt += __popc(word);
    }
  }
  if (kv_count && lane == 0) kv_count[row] = cnt;
}

int launch_score_cdf(const Geometry& g, const float* pq, const float* pk, float* scores, float tau, float scale,
                     uint32_t* mask, int32_t* kv_count, cudaStream_t st) {
  {
    const size_t smem = (size_t)2 * kScoreTile * (g.d + 4) * 4;
    const int nt = (g.NB + kScoreTile - 1) / kScoreTile;
    dim3 grid(nt, nt, g.B * g.H);
    auto kern = g.d == 64 ? score_kernel<64> : score_kernel<128>;
    SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)kern, (int)smem));
    kern<<<grid, kScoreThreads, smem, st>>>(pq, pk, g.NB, scores);
  }
  {
    const int64_t n_rows = (int64_t)g.B * g.H * g.NB;
    const float c = scale * 1.4426950408889634f;  // fp32 product, as in the definition above
    const unsigned grid = (unsigned)((n_rows + kTopkWarps - 1) / kTopkWarps);
    auto kern = g.Wd <= 4 ? cdf_kernel<4> : g.Wd <= 8 ? cdf_kernel<8> : g.Wd <= 16 ? cdf_kernel<16> : cdf_kernel<32>;
    kern<<<grid, kTopkWarps * 32, 0, st>>>(scores, n_rows, g.NB, g.Wd, g.nb_cand, tau, c, mask, kv_count);
  }
  count_launch(2);
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

int launch_score_topk(const Geometry& g, const float* pq, const float* pk, float* scores, int topk,
                      uint32_t* mask, int32_t* kv_list, int32_t* kv_count, cudaStream_t st) {
  const int kept_cap = topk + (g.NB - g.nb_cand);
  {
    const size_t smem = (size_t)2 * kScoreTile * (g.d + 4) * 4;
    const int nt = (g.NB + kScoreTile - 1) / kScoreTile;
    dim3 grid(nt, nt, g.B * g.H);
    auto kern = g.d == 64 ? score_kernel<64> : score_kernel<128>;
    SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)kern, (int)smem));
    kern<<<grid, kScoreThreads, smem, st>>>(pq, pk, g.NB, scores);
  }
  {
    const int64_t n_rows = (int64_t)g.B * g.H * g.NB;
    const unsigned grid = (unsigned)((n_rows + kTopkWarps - 1) / kTopkWarps);
    auto kern = g.Wd <= 4 ? topk_kernel<4> : g.Wd <= 8 ? topk_kernel<8> : g.Wd <= 16 ? topk_kernel<16> : topk_kernel<32>;
    kern<<<grid, kTopkWarps * 32, 0, st>>>(scores, n_rows, g.NB, g.Wd, g.nb_cand, topk, kept_cap, mask, kv_list, kv_count);
  }
  count_launch(2);
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

}  // namespace sparsp
