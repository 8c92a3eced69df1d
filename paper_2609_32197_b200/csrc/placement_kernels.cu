// Placement tools (Section 4.3: the layout is applied as a deterministic permutation of whole KV blocks,
// undone by the inverse permutation; Section 3.2: how widely a received K block is shared by the
// receiving rank's query blocks).  permute_tokens_kernel is an HBM-bound copy of block-sized runs of
// token rows; sharing_kernel counts bits of mask columns.
#include "common.cuh"

namespace sparsp {

// One CTA per (slot, head, batch): copies the tokens of one block between logical and permuted order.
// A token row is d bf16 = d/8 16-byte vectors; consecutive threads take consecutive vectors of a row.
template <int D>
__global__ void __launch_bounds__(256) permute_tokens_kernel(const __nv_bfloat16* __restrict__ X,
                                                             __nv_bfloat16* __restrict__ Y,
                                                             const int32_t* __restrict__ block_of_slot,
                                                             const int64_t* __restrict__ token_offset_of_slot, int b,
                                                             int64_t N, int64_t sB, int64_t sH, int64_t sT,
                                                             int inverse) {
  constexpr int VPR = D / 8;
  const int s = blockIdx.x;
  const int64_t lo_new = token_offset_of_slot[s];
  const int n_j = (int)(token_offset_of_slot[s + 1] - lo_new);
  const int64_t lo_old = (int64_t)block_of_slot[s] * b;
  const int64_t base = (int64_t)blockIdx.z * sB + (int64_t)blockIdx.y * sH;
  const int64_t src0 = base + (inverse ? lo_new : lo_old) * sT;
  const int64_t dst0 = base + (inverse ? lo_old : lo_new) * sT;
  for (int idx = threadIdx.x; idx < n_j * VPR; idx += blockDim.x) {
    const int t = idx / VPR, v = idx % VPR;
    const uint4 val = __ldcs(reinterpret_cast<const uint4*>(X + src0 + (int64_t)t * sT + v * 8));
    __stcs(reinterpret_cast<uint4*>(Y + dst0 + (int64_t)t * sT + v * 8), val);
  }
}

int launch_permute_tokens(const sparsp_shape& s, const Geometry& g, const void* X, void* Y,
                          const int32_t* block_of_slot, const int64_t* token_offset_of_slot, int inverse,
                          cudaStream_t st) {
  dim3 grid((unsigned)g.NB, (unsigned)g.H, (unsigned)g.B);
  if (g.d == 64)
    permute_tokens_kernel<64><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X, (__nv_bfloat16*)Y, block_of_slot,
                                                    token_offset_of_slot, g.b, g.N, s.stride_batch, s.stride_head,
                                                    s.stride_token, inverse);
  else
    permute_tokens_kernel<128><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X, (__nv_bfloat16*)Y, block_of_slot,
                                                     token_offset_of_slot, g.b, g.N, s.stride_batch, s.stride_head,
                                                     s.stride_token, inverse);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

// hist[b][r][q], q = 0..100: number of (head, remote block j) pairs of consumer r for which
// floor(100 * |{ i in Q_r : M[b,h,i,j] }| / |Q_r|) == q and the count is positive.
// One warp per (batch, consumer, head, 32-block word of j): lane t owns block j = 32 w + t.
__global__ void __launch_bounds__(256) sharing_kernel(const uint32_t* __restrict__ mask,
                                                      const int32_t* __restrict__ rank, int B, int H, int NB, int Wd,
                                                      int P, unsigned long long* __restrict__ hist) {
  const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t total = (int64_t)B * P * H * Wd;
  if (wid >= total) return;
  const int w = (int)(wid % Wd);
  const int h = (int)((wid / Wd) % H);
  const int r = (int)((wid / ((int64_t)Wd * H)) % P);
  const int bb = (int)(wid / ((int64_t)Wd * H * P));
  const uint32_t* m = mask + ((int64_t)(bb * H + h) * NB) * Wd + w;
  int count = 0, n_local = 0;
  for (int i = 0; i < NB; ++i) {
    if (rank[i] == r) {  // warp-uniform
      ++n_local;
      count += (m[(int64_t)i * Wd] >> lane) & 1u;
    }
  }
  const int j = w * 32 + lane;
  if (j < NB && rank[j] != r && count > 0)
    atomicAdd(hist + ((int64_t)(bb * P + r) * 101 + (100 * count) / n_local), 1ULL);
}

int launch_sharing(const Geometry& g, const uint32_t* mask, const int32_t* rank, int P, int64_t* hist,
                   cudaStream_t st) {
  SPARSP_CUDA_OK(cudaMemsetAsync(hist, 0, (size_t)g.B * P * 101 * 8, st));
  const int64_t warps = (int64_t)g.B * P * g.H * g.Wd;
  sharing_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(mask, rank, g.B, g.H, g.NB, g.Wd, P,
                                                                    (unsigned long long*)hist);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

}  // namespace sparsp
