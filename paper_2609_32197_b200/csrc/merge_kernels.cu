// Consumer-side helpers of the demand-routed exchange: the mask of one hop (consumer rank's query
// blocks x producer rank's KV blocks) and the log-sum-exp merge of per-hop partial attention results.
// Both are small element-wise kernels; the merge is HBM-bound (reads two outputs, writes one).
#include "common.cuh"

namespace sparsp {

// hop[b][h][i][w] = (rank[i] == consumer and head_begin <= h < head_end) ? mask[b][h][i][w] & own_producer[w] : 0.
// Thread per word.
__global__ void hop_mask_kernel(const uint32_t* __restrict__ mask, const int32_t* __restrict__ rank, int H, int NB,
                                int Wd, int64_t n_words, int consumer, int producer, int head_begin, int head_end,
                                uint32_t* __restrict__ hop) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_words) return;
  const int w = (int)(idx % Wd);
  const int i = (int)((idx / Wd) % NB);
  const int h = (int)((idx / ((int64_t)Wd * NB)) % H);
  uint32_t out = 0;
  if (rank[i] == consumer && h >= head_begin && h < head_end) {
    uint32_t own = 0;
    for (int t = 0; t < 32; ++t) {
      const int j = w * 32 + t;
      if (j < NB && rank[j] == producer) own |= 1u << t;
    }
    out = mask[idx] & own;
  }
  hop[idx] = out;
}

// One CTA per (token block, head, batch); a thread handles (row, 8 columns) units of the block.  O_a, O_b, O: bf16
// with the shape's strides; lse: fp32 [B][H][N].  O may be O_a or O_b and lse may be lse_a or lse_b (no pointer is
// declared restrict): a thread reads the 16 bytes it later writes, and only the row's first thread touches the
// log-sum-exp values -- it reads both inputs, computes the weights and hands them to the row's other threads by
// shuffle (the D/8 threads of a row are consecutive lanes of one warp) before it writes the merged value.
// With `rank` given, only the blocks of `consumer` in heads [head_begin, head_begin + gridDim.y) are merged (one
// chunk of one hop of one rank): a CTA of another rank's block returns at once, every other row stays untouched.
template <int D>
__global__ void __launch_bounds__(256) attn_merge_kernel(const __nv_bfloat16* Oa, const float* la,
                                                         const __nv_bfloat16* Ob, const float* lb, __nv_bfloat16* O,
                                                         float* lse, int H, int64_t N, int b, int64_t sB, int64_t sH,
                                                         int64_t sT, const int32_t* __restrict__ rank, int consumer,
                                                         int head_begin) {
  constexpr int VPR = D / 8;
  const int blk = blockIdx.x, head = head_begin + blockIdx.y, batch = blockIdx.z;
  if (rank != nullptr && rank[blk] != consumer) return;
  const int64_t tok0 = (int64_t)blk * b;
  const int n_rows = (int)min((int64_t)b, N - tok0);
  const int leader = (threadIdx.x & 31) & ~(VPR - 1);  // lane of the row's first thread
  for (int u0 = 0; u0 < n_rows * VPR; u0 += blockDim.x) {  // blockDim.x is a multiple of VPR: a row never splits
    const int u = u0 + threadIdx.x;
    const int r = u / VPR, col = u % VPR;
    const bool live = r < n_rows;
    const int64_t row = ((int64_t)batch * H + head) * N + tok0 + r;
    float wa = 0.0f, wb = 0.0f, out_lse = -INFINITY;
    if (live && col == 0) {
      const float a = la[row], c = lb[row];
      const float m = fmaxf(a, c);
      if (m > -INFINITY) {
        const float ea = __expf(a - m), eb = __expf(c - m);
        const float tot = ea + eb;
        wa = ea / tot;
        wb = eb / tot;
        out_lse = m + __logf(tot);
      }
    }
    wa = __shfl_sync(0xffffffffu, wa, leader);
    wb = __shfl_sync(0xffffffffu, wb, leader);
    if (!live) continue;
    const int64_t off = (int64_t)batch * sB + (int64_t)head * sH + (tok0 + r) * sT + col * 8;
    const uint4 va = *reinterpret_cast<const uint4*>(Oa + off);
    const uint4 vb = *reinterpret_cast<const uint4*>(Ob + off);
    const uint32_t xa[4] = {va.x, va.y, va.z, va.w}, xb[4] = {vb.x, vb.y, vb.z, vb.w};
    uint32_t w[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a0 = __uint_as_float(xa[e] << 16), a1 = __uint_as_float(xa[e] & 0xffff0000u);
      const float b0 = __uint_as_float(xb[e] << 16), b1 = __uint_as_float(xb[e] & 0xffff0000u);
      const __nv_bfloat162 h2 = __floats2bfloat162_rn(a0 * wa + b0 * wb, a1 * wa + b1 * wb);
      w[e] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    *reinterpret_cast<uint4*>(O + off) = make_uint4(w[0], w[1], w[2], w[3]);
    if (col == 0) lse[row] = out_lse;
  }
}

int launch_hop_mask(const Geometry& g, const uint32_t* mask, const int32_t* rank, int consumer, int producer,
                    int head_begin, int head_end, uint32_t* hop, cudaStream_t st) {
  const int64_t n_words = (int64_t)g.B * g.H * g.NB * g.Wd;
  hop_mask_kernel<<<(unsigned)((n_words + 255) / 256), 256, 0, st>>>(mask, rank, g.H, g.NB, g.Wd, n_words, consumer,
                                                                     producer, head_begin, head_end, hop);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

int launch_attn_merge(const sparsp_shape& s, const Geometry& g, const void* Oa, const float* la, const void* Ob,
                      const float* lb, void* O, float* lse, const int32_t* rank, int consumer, int head_begin,
                      int head_end, cudaStream_t st) {
  if (head_end <= head_begin) return SPARSP_OK;
  dim3 grid((unsigned)g.NB, (unsigned)(head_end - head_begin), (unsigned)g.B);
  auto a = (const __nv_bfloat16*)Oa;
  auto b = (const __nv_bfloat16*)Ob;
  auto o = (__nv_bfloat16*)O;
  if (g.d == 64)
    attn_merge_kernel<64><<<grid, 256, 0, st>>>(a, la, b, lb, o, lse, g.H, g.N, g.b, s.stride_batch, s.stride_head,
                                                s.stride_token, rank, consumer, head_begin);
  else
    attn_merge_kernel<128><<<grid, 256, 0, st>>>(a, la, b, lb, o, lse, g.H, g.N, g.b, s.stride_batch, s.stride_head,
                                                 s.stride_token, rank, consumer, head_begin);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

}  // namespace sparsp
