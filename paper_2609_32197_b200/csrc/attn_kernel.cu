// Step 3: block-sparse FlashAttention forward on tcgen05 tensor cores (sm_100a).
//
// A CTA owns two adjacent query blocks of one (batch, head) and runs two independent softmax
// "streams" so that one stream's exponentials overlap the other stream's MMAs:
//   block = 128: the two query blocks are two 128-row Q tiles; stream s = Q tile s.  The CTA walks
//                the UNION of the two rows' kept KV blocks; a stream skips the blocks its own row
//                does not keep, K/V tiles that both keep are loaded once.
//   block = 64 : the two query blocks are stacked into ONE 128-row Q tile (full-rate M = 128 MMAs);
//                a KV tile is two entries of the union list (128 keys, full-rate N = 128); each
//                64x64 quadrant the mask does not keep is zeroed in P.  Stream s takes the KV tiles
//                of parity s into its own accumulator; the two partial results are merged at the end.
// Warp roles (384 threads): warp 0 = TMA producer (K ring and V ring, polled independently),
// warp 1 = MMA issuer (one thread), warps 2-3 idle, warps 4-7 / 8-11 = softmax warpgroups of stream
// 0 / 1, one query row per thread; the first warpgroup gives registers up to the softmax ones.  Tensor memory: S_s (128 fp32 columns, overwritten in place by bf16 P_s, which
// the P.V MMA reads straight from tensor memory) and O_s (d fp32 columns) per stream.
// Online softmax is base-2 in fp32; O is rescaled lazily, only when a row's maximum has grown by
// more than 2^8 since the reference last moved.
// Every mbarrier wait is bounded; a wait that runs out sets SPARSP_ERR_TIMEOUT in the status word
// and raises a CTA-wide flag that makes all later waits fall through, so the CTA still drains.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace sparsp {

using namespace ptx;

struct AttnParams {
  const uint32_t* mask;
  __nv_bfloat16* O;
  float* lse;
  int32_t* status;
  int64_t N;
  int64_t sB, sH, sT;
  int H, NB, Wd;
  float scale_log2;  // softmax scale * log2(e)
  long long wait_limit;
};

constexpr int kAttnThreads = 384;
constexpr int kTmemCols = 512;
constexpr float kGrowThreshold = 8.0f;

template <int D, int BLK>
struct AttnCfg {
  static constexpr bool kSplitKV = (BLK == 64);   // one Q tile, streams split the KV tiles
  static constexpr int kQTiles = kSplitKV ? 1 : 2;
  static constexpr int kEPT = 128 / BLK;          // union-list entries per 128-key KV tile
  static constexpr int kStages = (D == 64) ? 4 : 2;
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kTileBytes = 128 * D * 2;  // one K or V tile
  static constexpr int kOffQ = 0;
  static constexpr int kOffK = kOffQ + kQTiles * kQBytes;
  static constexpr int kOffV = kOffK + kStages * kTileBytes;
  static constexpr int kOffEntJ = kOffV + kStages * kTileBytes;  // uint16 [1024] union list
  static constexpr int kOffEntF = kOffEntJ + 2 * kMaxBlocks;     // uint8 [1024] bit q: kept by query block q
  static constexpr int kOffStat = kOffEntF + kMaxBlocks;         // float2 [2][128] stream statistics
  static constexpr int kOffBars = kOffStat + 2 * 128 * 8;
  static constexpr int kNumBars = 1 + 4 * kStages + 6;
  static constexpr int kOffMisc = kOffBars + 8 * kNumBars;
  static constexpr int kTotal = kOffMisc + 32;
  static constexpr int kDynamic = kTotal + 1024;  // slack for the 1024-byte alignment of the base
  static constexpr int kMergeStride = D / 2 + 4;  // floats per row of the merge buffer
  static_assert(2 * 128 * kMergeStride * 4 <= 2 * kStages * kTileBytes, "merge buffer must fit the K/V rings");
  static_assert(kDynamic <= 232448, "shared memory budget");
};

__device__ __forceinline__ void named_bar_sync(int id, int n) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}

template <int D, int BLK>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using C = AttnCfg<D, BLK>;
  constexpr int S = C::kStages;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem + C::kOffQ;
  unsigned char* sK = smem + C::kOffK;
  unsigned char* sV = smem + C::kOffV;
  uint16_t* sEntJ = reinterpret_cast<uint16_t*>(smem + C::kOffEntJ);
  uint8_t* sEntF = smem + C::kOffEntF;
  float2* sStat = reinterpret_cast<float2*>(smem + C::kOffStat);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
  uint64_t* bar_q = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + S;
  uint64_t* v_full = k_empty + S;
  uint64_t* v_empty = v_full + S;
  uint64_t* s_full = v_empty + S;  // [2] S_s written by Q K^T
  uint64_t* p_full = s_full + 2;   // [2] P_s written by the softmax warpgroup (128 arrivals)
  uint64_t* o_full = p_full + 2;   // [2] a P V of stream s has completed
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  int* s_nent = reinterpret_cast<int*>(smem + C::kOffMisc + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  const int batch = bh / p.H, head = bh % p.H;
  const int i0 = blockIdx.x * 2;  // first of the CTA's two query blocks
  const int64_t q0 = (int64_t)i0 * BLK;

  // ---- setup ------------------------------------------------------------------------------
  if (tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(bar_q, 1);
    for (int s = 0; s < S; ++s) {
      mbar_init(k_full + s, 1);
      mbar_init(k_empty + s, 1);
      mbar_init(v_full + s, 1);
      mbar_init(v_empty + s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(s_full + s, 1);
      mbar_init(p_full + s, 128);
      mbar_init(o_full + s, 1);
    }
    mbar_init_fence();
    *s_abort = 0;
  }
  if (warp == 1) {
    tmem_alloc(s_tmem, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0) {
    // union of the two mask rows -> ascending entry list; flag bit q = kept by query block i0 + q
    const uint32_t* mrow = p.mask + ((int64_t)bh * p.NB + i0) * p.Wd;
    int running = 0;
    for (int w0 = 0; w0 < p.Wd; w0 += 32) {
      const int w = w0 + lane;
      uint32_t rb[2];
      rb[0] = (w < p.Wd) ? mrow[w] : 0u;
      rb[1] = (w < p.Wd && i0 + 1 < p.NB) ? mrow[p.Wd + w] : 0u;
      uint32_t u = rb[0] | rb[1];
      const int mine = __popc(u);
      int incl = mine;
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, s);
        if (lane >= s) incl += v;
      }
      int pos = running + incl - mine;
      while (u) {
        const int t = __ffs(u) - 1;
        u &= u - 1;
        sEntJ[pos] = (uint16_t)(w * 32 + t);
        sEntF[pos] = (uint8_t)(((rb[0] >> t) & 1u) | (((rb[1] >> t) & 1u) << 1));
        ++pos;
      }
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) *s_nent = running;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int n_ent = *s_nent;
  const int n_tiles = (n_ent + C::kEPT - 1) / C::kEPT;

  // which streams work on KV tile n
  auto stream_mask = [&](int n) -> int { return C::kSplitKV ? (1 << (n & 1)) : (int)sEntF[n]; };

  if (warp == 0) {
    // ================================ TMA producer ========================================
    if (lane == 0 && n_tiles > 0) {
      mbar_expect_tx(bar_q, C::kQTiles * C::kQBytes);
#pragma unroll
      for (int t = 0; t < C::kQTiles; ++t)
#pragma unroll
        for (int c = 0; c < D / 64; ++c)
          tma_load_4d(sQ + t * C::kQBytes + c * 16384, &tmQ, bar_q, c * 64, (int)q0 + t * 128, head, batch);
      auto load_tile = [&](unsigned char* dst, const CUtensorMap* tm, uint64_t* bar, int n) {
        mbar_expect_tx(bar, C::kTileBytes);
#pragma unroll
        for (int e = 0; e < C::kEPT; ++e) {
          const int ent = min(n * C::kEPT + e, n_ent - 1);  // an absent second half re-reads the last entry
          const int j = sEntJ[ent];
#pragma unroll
          for (int c = 0; c < D / 64; ++c)
            tma_load_4d(dst + c * 16384 + e * (BLK * 128), tm, bar, c * 64, j * BLK, head, batch);
        }
      };
      int kn = 0, vn = 0;
      const long long t0 = clock64();
      while ((kn < n_tiles || vn < n_tiles) && !*s_abort) {
        bool progressed = false;
        if (kn < n_tiles && mbar_try_wait(k_empty + kn % S, ((kn / S) & 1) ^ 1)) {
          load_tile(sK + (kn % S) * C::kTileBytes, &tmK, k_full + kn % S, kn);
          ++kn;
          progressed = true;
        }
        if (vn < n_tiles && mbar_try_wait(v_empty + vn % S, ((vn / S) & 1) ^ 1)) {
          load_tile(sV + (vn % S) * C::kTileBytes, &tmV, v_full + vn % S, vn);
          ++vn;
          progressed = true;
        }
        if (!progressed && clock64() - t0 > p.wait_limit * 8) {
          *s_abort = 1;
          if (atomicCAS(p.status, 0, SPARSP_ERR_TIMEOUT) == 0) p.status[1] = 10;
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ==========================================
    if (lane == 0 && n_tiles > 0) {
      constexpr uint32_t kIdescQK = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t kIdescPV = make_idesc_bf16(128, D, 0, 1);
      int pending[2] = {-1, -1};  // KV tile whose S_s is with the softmax warpgroup
      int pcnt[2] = {0, 0};       // P tiles consumed per stream
      bool started[2] = {false, false};
      int v_users[S];             // P V MMAs still to be issued per V stage
#pragma unroll
      for (int s = 0; s < S; ++s) v_users[s] = 0;

      auto flush = [&](int s) {  // issue O_s += P_s V for the stream's pending tile
        const int m = pending[s];
        mbar_wait_bounded(p_full + s, pcnt[s] & 1, s_abort, p.status, 20 + s, p.wait_limit);
        ++pcnt[s];
        mbar_wait_bounded(v_full + m % S, (m / S) & 1, s_abort, p.status, 22, p.wait_limit);
        tc_fence_after();
        const uint32_t b0 = smem_u32(sV + (m % S) * C::kTileBytes);
        const uint32_t tP = tmem_base + s * 128;
        const uint32_t tO = tmem_base + 256 + s * D;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t db = make_smem_desc(b0 + kk * 2048, 16384, 1024);
          mma_ts(tO, tP + kk * 8, db, kIdescPV, (started[s] || kk > 0) ? 1u : 0u);
        }
        started[s] = true;
        mma_commit(o_full + s);
        pending[s] = -1;
#pragma unroll
        for (int st = 0; st < S; ++st)
          if (st == m % S && --v_users[st] == 0) mma_commit(v_empty + st);
      };

      mbar_wait_bounded(bar_q, 0, s_abort, p.status, 11, p.wait_limit);
      for (int n = 0; n < n_tiles; ++n) {
        const int sm = stream_mask(n);
        // a stream that skipped tile n-1 may still owe the P V of an older tile: issue it first, so
        // that its V stage is released no later than two steps after it was filled
#pragma unroll
        for (int s = 0; s < 2; ++s)
          if (pending[s] >= 0 && pending[s] < n - 1) flush(s);
        mbar_wait_bounded(k_full + n % S, (n / S) & 1, s_abort, p.status, 12, p.wait_limit);
        tc_fence_after();
#pragma unroll
        for (int st = 0; st < S; ++st)
          if (st == n % S) v_users[st] = (sm & 1) + ((sm >> 1) & 1);
#pragma unroll
        for (int s = 0; s < 2; ++s) {
          if (!((sm >> s) & 1)) continue;
          if (pending[s] >= 0) flush(s);  // tile n-1: frees S_s for the next Q K^T
          const uint32_t a0 = smem_u32(sQ + (C::kSplitKV ? 0 : s) * C::kQBytes);
          const uint32_t b0 = smem_u32(sK + (n % S) * C::kTileBytes);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint64_t da = make_smem_desc(a0 + (kk / 4) * 16384 + (kk % 4) * 32, 16, 1024);
            const uint64_t db = make_smem_desc(b0 + (kk / 4) * 16384 + (kk % 4) * 32, 16, 1024);
            mma_ss(tmem_base + s * 128, da, db, kIdescQK, kk > 0 ? 1u : 0u);
          }
          mma_commit(s_full + s);
          pending[s] = n;
        }
        mma_commit(k_empty + n % S);
      }
#pragma unroll
      for (int s = 0; s < 2; ++s)
        if (pending[s] >= 0) flush(s);
    }
  } else if (warp >= 4) {
    // ================================ softmax warpgroups ==================================
    const int wg = (warp - 4) >> 2;  // stream
    const int rgrp = warp & 3;       // tensor-memory lane group this warp may access
    const int row = rgrp * 32 + lane;
    const int rh = row >> 6;         // which query block of a stacked Q tile the row belongs to
    const uint32_t lane_off = (uint32_t)(rgrp * 32) << 16;
    const uint32_t tS = tmem_base + wg * 128 + lane_off;
    const uint32_t tO = tmem_base + 256 + wg * D + lane_off;
    float m_used = -INFINITY;  // reference maximum (log2 domain) of the row's exponentials
    float l_run = 0.0f;
    int cnt = 0;

    for (int n = 0; n < n_tiles; ++n) {
      if (!((stream_mask(n) >> wg) & 1)) continue;
      // valid / kept columns of each 32-column chunk (warp-uniform)
      int valid[4];
      if (C::kSplitKV) {
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          const int ent = n * 2 + ch;
          int nv = 0;
          if (ent < n_ent && ((sEntF[ent] >> rh) & 1))
            nv = (int)min((int64_t)64, p.N - (int64_t)sEntJ[ent] * 64);
          valid[2 * ch] = min(nv, 32);
          valid[2 * ch + 1] = max(nv - 32, 0);
        }
      } else {
        const int nv = (int)min((int64_t)128, p.N - (int64_t)sEntJ[n] * 128);
#pragma unroll
        for (int c = 0; c < 4; ++c) valid[c] = max(0, min(32, nv - 32 * c));
      }

      mbar_wait_bounded(s_full + wg, cnt & 1, s_abort, p.status, 30 + wg, p.wait_limit);
      tc_fence_after();
      // pass 1: row maximum over the kept, valid columns (two 64-column halves)
      float mx = -INFINITY;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float sv[64];
        tmem_ld32(tS + h * 64, reinterpret_cast<uint32_t*>(sv));
        tmem_ld32(tS + h * 64 + 32, reinterpret_cast<uint32_t*>(sv) + 32);
        tmem_ld_wait();
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int vc = valid[2 * h + cc];
          if (vc == 32) {
#pragma unroll
            for (int e = 0; e < 32; e += 2) mx = fmaxf(mx, fmaxf(sv[cc * 32 + e], sv[cc * 32 + e + 1]));
          } else if (vc > 0) {
#pragma unroll
            for (int e = 0; e < 32; ++e) mx = fmaxf(mx, e < vc ? sv[cc * 32 + e] : -INFINITY);
          }
        }
      }
      mx *= p.scale_log2;
      const float m_new = fmaxf(m_used, mx);
      const bool grow = m_new > m_used + kGrowThreshold || (m_used == -INFINITY && m_new > -INFINITY);
      if (__any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? ex2(m_used - m_new) : 1.0f;  // m_used = -inf -> 0
        if (cnt > 0) {  // S_s of this tile is complete, hence so is every earlier P V of the stream
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tO + c * 32, o);
          }
        }
        l_run *= alpha;
        if (grow) m_used = m_new;
      }

      // pass 2: exponentials chunk by chunk; bf16 P overwrites S in place (P chunk c occupies
      // columns [16c, 16c+16), which lie inside the S columns already consumed)
      float lsum = 0.0f;
      const float neg_m = -m_used;
      float buf[2][32];
      tmem_ld32(tS, reinterpret_cast<uint32_t*>(buf[0]));
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        tmem_ld_wait();
        if (c < 3) tmem_ld32(tS + (c + 1) * 32, reinterpret_cast<uint32_t*>(buf[(c + 1) & 1]));
        const float* sv = buf[c & 1];
        uint32_t pk[16];
        if (valid[c] == 32) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = ex2(fmaf(sv[2 * e], p.scale_log2, neg_m));
            const float p1 = ex2(fmaf(sv[2 * e + 1], p.scale_log2, neg_m));
            lsum += p0 + p1;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        } else if (valid[c] > 0) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = 2 * e < valid[c] ? ex2(fmaf(sv[2 * e], p.scale_log2, neg_m)) : 0.0f;
            const float p1 = 2 * e + 1 < valid[c] ? ex2(fmaf(sv[2 * e + 1], p.scale_log2, neg_m)) : 0.0f;
            lsum += p0 + p1;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) pk[e] = 0u;
        }
        tmem_st16(tS + c * 16, pk);
      }
      l_run += lsum;
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(p_full + wg);
      ++cnt;
    }

    // ---- epilogue -------------------------------------------------------------------------
    if (cnt > 0) {
      mbar_wait_bounded(o_full + wg, (cnt - 1) & 1, s_abort, p.status, 40 + wg, p.wait_limit);
      tc_fence_after();
    }
    if (!C::kSplitKV) {
      const int64_t tok = q0 + wg * 128 + row;
      const float inv_l = l_run > 0.0f ? 1.0f / l_run : 0.0f;
      __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        if (cnt > 0) {  // warp-uniform: tensor-memory loads are warp-collective
          tmem_ld32(tO + c * 32, o);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = 0u;
        }
        if (tok < p.N) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * e]) * inv_l,
                                                              __uint_as_float(o[v * 8 + 2 * e + 1]) * inv_l);
              w[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (p.lse && tok < p.N)
        p.lse[(int64_t)bh * p.N + tok] = l_run > 0.0f ? (m_used + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
    } else {
      // merge the two streams' partial results: stream s finalises columns [s*D/2, (s+1)*D/2)
      constexpr int HALF = D / 2;
      float* mbuf = reinterpret_cast<float*>(sK);  // K/V rings are idle once both streams are done
      sStat[wg * 128 + row] = make_float2(m_used, l_run);
      named_bar_sync(1, 256);
      const float2 other = sStat[(1 - wg) * 128 + row];
      const float m = fmaxf(m_used, other.x);
      const float a_me = m_used > -INFINITY ? ex2(m_used - m) : 0.0f;
      const float a_ot = other.x > -INFINITY ? ex2(other.x - m) : 0.0f;
      const float l = l_run * a_me + other.y * a_ot;
      const float inv_l = l > 0.0f ? 1.0f / l : 0.0f;
      // hand the partner its half of my accumulator, scaled to the common reference
      float* give = mbuf + ((size_t)wg * 128 + row) * C::kMergeStride;
#pragma unroll
      for (int c = 0; c < HALF / 32; ++c) {
        uint32_t o[32];
        if (cnt > 0) {
          tmem_ld32(tO + (1 - wg) * HALF + c * 32, o);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = 0u;
        }
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<float4*>(give + c * 32 + v * 4) =
              make_float4(__uint_as_float(o[v * 4]) * a_me, __uint_as_float(o[v * 4 + 1]) * a_me,
                          __uint_as_float(o[v * 4 + 2]) * a_me, __uint_as_float(o[v * 4 + 3]) * a_me);
      }
      named_bar_sync(1, 256);
      const int64_t tok = q0 + row;
      const float* take = mbuf + ((size_t)(1 - wg) * 128 + row) * C::kMergeStride;
      __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT + wg * HALF;
#pragma unroll
      for (int c = 0; c < HALF / 32; ++c) {
        uint32_t o[32];
        if (cnt > 0) {
          tmem_ld32(tO + wg * HALF + c * 32, o);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = 0u;
        }
        if (tok < p.N) {
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            const float4 t0 = *reinterpret_cast<const float4*>(take + c * 32 + v * 8);
            const float4 t1 = *reinterpret_cast<const float4*>(take + c * 32 + v * 8 + 4);
            const float tt[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float x0 = (__uint_as_float(o[v * 8 + 2 * e]) * a_me + tt[2 * e]) * inv_l;
              const float x1 = (__uint_as_float(o[v * 8 + 2 * e + 1]) * a_me + tt[2 * e + 1]) * inv_l;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
              w[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(orow + c * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (p.lse && wg == 0 && tok < p.N)
        p.lse[(int64_t)bh * p.N + tok] = l > 0.0f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor viewed as (d, N, H, B) with a box of (64, rows, 1, 1) and 128-byte swizzle.
static int make_tmap(CUtensorMap* out, const void* base, const sparsp_shape& s, const Geometry& g, int rows) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) {
    set_error("cuTensorMapEncodeTiled is not available from the driver");
    return SPARSP_ERR_CUDA;
  }
  cuuint64_t dims[4] = {(cuuint64_t)g.d, (cuuint64_t)g.N, (cuuint64_t)g.H, (cuuint64_t)g.B};
  const int64_t batch_stride = s.stride_batch > 0 ? s.stride_batch : g.N * s.stride_token;
  cuuint64_t strides[3] = {(cuuint64_t)s.stride_token * 2, (cuuint64_t)s.stride_head * 2,
                           (cuuint64_t)batch_stride * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled failed with %d", (int)r);
    return SPARSP_ERR_CUDA;
  }
  return SPARSP_OK;
}

template <int D, int BLK>
static int launch_attn_t(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                         const AttnParams& p, cudaStream_t st) {
  CUtensorMap tq, tk, tv;
  int rc;
  if ((rc = make_tmap(&tq, Q, s, g, 128)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tk, K, s, g, BLK)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tv, V, s, g, BLK)) != SPARSP_OK) return rc;
  auto kern = attn_fwd_kernel<D, BLK>;
  const int smem = AttnCfg<D, BLK>::kDynamic;
  SPARSP_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  dim3 grid((unsigned)((g.NB + 1) / 2), (unsigned)(g.B * g.H));
  kern<<<grid, kAttnThreads, smem, st>>>(tq, tk, tv, p);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

int launch_attn(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                const uint32_t* mask, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                cudaStream_t st) {
  AttnParams p;
  p.mask = mask;
  p.O = (__nv_bfloat16*)O;
  p.lse = lse;
  p.status = (int32_t*)(ws + L.status);
  p.N = g.N;
  p.sB = s.stride_batch;
  p.sH = s.stride_head;
  p.sT = s.stride_token;
  p.H = g.H;
  p.NB = g.NB;
  p.Wd = g.Wd;
  const float sc = scale > 0.0f ? scale : 1.0f / sqrtf((float)g.d);
  p.scale_log2 = sc * 1.4426950408889634f;
  p.wait_limit = 200000000LL;  // about 0.1 s of SM clocks
  if (g.d == 64 && g.b == 64) return launch_attn_t<64, 64>(s, g, Q, K, V, p, st);
  if (g.d == 64 && g.b == 128) return launch_attn_t<64, 128>(s, g, Q, K, V, p, st);
  if (g.d == 128 && g.b == 64) return launch_attn_t<128, 64>(s, g, Q, K, V, p, st);
  return launch_attn_t<128, 128>(s, g, Q, K, V, p, st);
}

}  // namespace sparsp
