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
// Warp roles (608 threads): warp 0 = TMA producer (K ring and V ring, polled independently),
// warps 1 and 18 = MMA issuers of stream 0 / 1 (one thread each, so the streams never serialise on
// one instruction stream), warps 2-9 / 10-17 = softmax warps of stream 0 / 1.  A query row
// is shared by TWO threads of different warps, each owning 64 of the tile's 128 key columns: a row
// of S is read from tensor memory once, in 64 registers, and the pair exchanges its two partial row
// maxima through shared memory behind a 64-thread named barrier.  Tensor memory: S_s (128 fp32 columns, overwritten in place by bf16 P_s, which
// the P.V MMA reads straight from tensor memory) and O_s (d fp32 columns) per stream.
// Online softmax is base-2 in fp32; O is rescaled lazily, only when a row's maximum has grown by
// more than 2^8 since the reference last moved.
// Every mbarrier wait is bounded; a wait that runs out sets SPARSP_ERR_TIMEOUT in the status word
// and raises a CTA-wide flag that makes all later waits fall through, so the CTA still drains.
#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace sparsp {

using namespace ptx;

struct AttnParams {
  const uint32_t* mask;
  const int32_t* pairs;  // [B*H][ceil(NB/2)][2] query blocks of each CTA (second may be -1)
  // packed-source mode (NULL = every tile comes from K / V): slot[bh][j] = entry index of KV block j in
  // the consumer's packed buffer, or -1 if the consumer owns the block; tile_base = index of the
  // consumer's first tile in the packed tensor map (a device scalar)
  const int32_t* slot;
  const int64_t* tile_base;
  __nv_bfloat16* O;
  float* lse;
  int32_t* status;
  int64_t N;
  int64_t sB, sH, sT;
  int H, NB, Wd;
  float scale_log2;  // softmax scale * log2(e)
  long long wait_limit;
};

constexpr int kAttnThreads = 608;
constexpr int kIssuer1Warp = 18;  // warp 1 issues the MMAs of stream 0, warp 18 those of stream 1
constexpr int kTmemCols = 512;
constexpr float kGrowThreshold = 8.0f;
// Tuning switches (compile-time): packed fp32x2 arithmetic in the exponential loop, and how many of
// the exponentials go to the FMA pipe instead of the special-function unit (every n-th pair; 0 = none).
#ifndef SPARSP_TUNE_F32X2
#define SPARSP_TUNE_F32X2 1
#endif
#ifndef SPARSP_TUNE_POLY
#define SPARSP_TUNE_POLY 3
#endif

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
  static constexpr int kOffStat = kOffEntF + kMaxBlocks;         // float2 [2 streams][2 halves][128]
  static constexpr int kOffMax = kOffStat + 2 * 2 * 128 * 8;     // float [2 parities][2][2][128]
  static constexpr int kOffSlot = kOffMax + 2 * 2 * 2 * 128 * 4;  // int32 [1024] packed-buffer slot per list entry
  static constexpr int kOffBars = kOffSlot + 4 * kMaxBlocks;
  static constexpr int kNumBars = 1 + 4 * kStages + 8;
  // head_dim 64 leaves tensor-memory room for P next to S (S 2x128 + P 2x64 + O 2x64 = 512 columns):
  // Q K^T of the next tile can then start as soon as the softmax warps have READ S, instead of
  // waiting for P V to finish reading P out of the same columns.
  static constexpr bool kDecoupledP = (D == 64);
  static constexpr int kColP = 256;                       // first P column (decoupled layout)
  static constexpr int kColO = kDecoupledP ? 384 : 256;   // first O column
  static constexpr int kOffMisc = kOffBars + 8 * kNumBars;
  static constexpr int kTotal = kOffMisc + 32;
  static constexpr int kDynamic = kTotal + 1024;  // slack for the 1024-byte alignment of the base
  static constexpr int kMergeStride = D / 4 + 4;  // floats per row of the merge buffer
  static_assert(4 * 128 * kMergeStride * 4 <= 2 * kStages * kTileBytes, "merge buffer must fit the K/V rings");
  static_assert(kDynamic <= 232448, "shared memory budget");
};

#ifdef SPARSP_ATTN_PROFILE
// Optional cycle accounting for tuning builds: per-phase SM-clock totals of one softmax lane and of
// the MMA thread of every CTA.  Off in normal builds.
__device__ unsigned long long g_attn_prof[16];
#define PROF_T(var) const long long var = clock64()
#define PROF_ADD(slot, a, b) \
  if (lane == 0 && (warp == 2 || warp == 1)) atomicAdd(&g_attn_prof[slot], (unsigned long long)((b) - (a)))
#else
#define PROF_T(var)
#define PROF_ADD(slot, a, b)
#endif

// Packed fp32 pairs (one instruction for two lanes' worth of fused multiply-add / add).
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  unsigned long long ra, rb, rc, rd;
  float2 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rc) : "f"(c.x), "f"(c.y));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
  return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  unsigned long long ra, rb, rd;
  float2 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(ra) : "f"(a.x), "f"(a.y));
  asm("mov.b64 %0, {%1, %2};" : "=l"(rb) : "f"(b.x), "f"(b.y));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
  asm("mov.b64 {%0, %1}, %2;" : "=f"(d.x), "=f"(d.y) : "l"(rd));
  return d;
}

// 2^x for a pair of fp32 values on the FMA/ALU pipes (no special-function unit): round-to-nearest
// split x = i + f, f in [-0.5, 0.5], cubic minimax polynomial for 2^f (relative error 7.5e-5, far
// below bf16 rounding), exponent added into the bit pattern.  x is clamped at -126 (result >= 2^-126).
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  const float kMagic = 12582912.0f;  // 1.5 * 2^23: adding it rounds to an integer in the low mantissa bits
  x.x = fmaxf(x.x, -126.0f);
  x.y = fmaxf(x.y, -126.0f);
  const float2 t = fadd2(x, make_float2(kMagic, kMagic));
  const float2 fi = fadd2(t, make_float2(-kMagic, -kMagic));
  const float2 f = fadd2(x, make_float2(-fi.x, -fi.y));
  float2 q = ffma2(f, make_float2(0.0551716685f, 0.0551716685f), make_float2(0.2426111251f, 0.2426111251f));
  q = ffma2(q, f, make_float2(0.6932609677f, 0.6932609677f));
  q = ffma2(q, f, make_float2(0.9999280572f, 0.9999280572f));
  q.x = __int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23));
  q.y = __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23));
  return q;
}

__device__ __forceinline__ void named_bar_sync(int id, int n) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory");
}

template <int D, int BLK>
__global__ void __maxnreg__(96)
    attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmP,
                    const AttnParams p) {
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
  float* sMax = reinterpret_cast<float*>(smem + C::kOffMax);
  int32_t* sSlot = reinterpret_cast<int32_t*>(smem + C::kOffSlot);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
  uint64_t* bar_q = bars;
  uint64_t* k_full = bars + 1;
  uint64_t* k_empty = k_full + S;
  uint64_t* v_full = k_empty + S;
  uint64_t* v_empty = v_full + S;
  uint64_t* s_full = v_empty + S;  // [2] S_s written by Q K^T
  uint64_t* p_full = s_full + 2;   // [2] P_s written by the stream's 8 softmax warps (one arrival each)
  uint64_t* o_full = p_full + 2;   // [2] a P V of stream s has completed
  uint64_t* s_free = o_full + 2;   // [2] S_s has been read into registers (decoupled-P layout only)
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  int* s_nent = reinterpret_cast<int*>(smem + C::kOffMisc + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  PROF_T(t_cta0);
  const int bh = blockIdx.y;
  const int batch = bh / p.H, head = bh % p.H;
  // the CTA's two query blocks (any two blocks of the head: a pairing pass picks partners whose kept
  // lists overlap); blk[1] < 0 means the CTA has a single block
  const int32_t* pr = p.pairs + ((int64_t)bh * gridDim.x + blockIdx.x) * 2;
  const int blk[2] = {pr[0], pr[1]};

  // ---- setup ------------------------------------------------------------------------------
  if (tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(bar_q, 1);
    for (int s = 0; s < S; ++s) {
      mbar_init(k_full + s, 1);
      mbar_init(k_empty + s, 2);
      mbar_init(v_full + s, 1);
      mbar_init(v_empty + s, 2);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(s_full + s, 1);
      mbar_init(p_full + s, 8);
      mbar_init(o_full + s, 1);
      mbar_init(s_free + s, 8);
    }
    mbar_init_fence();
    *s_abort = 0;
  }
  if (warp == 1) {
    tmem_alloc(s_tmem, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0) {
    // union of the two mask rows -> ascending entry list; flag bit q = kept by query block blk[q]
    const uint32_t* mrow0 = p.mask + ((int64_t)bh * p.NB + max(blk[0], 0)) * p.Wd;
    const uint32_t* mrow1 = p.mask + ((int64_t)bh * p.NB + max(blk[1], 0)) * p.Wd;
    int running = 0;
    for (int w0 = 0; w0 < p.Wd; w0 += 32) {
      const int w = w0 + lane;
      uint32_t rb[2];
      rb[0] = (w < p.Wd && blk[0] >= 0) ? mrow0[w] : 0u;
      rb[1] = (w < p.Wd && blk[1] >= 0) ? mrow1[w] : 0u;
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
        if (p.slot) sSlot[pos] = p.slot[(int64_t)bh * p.NB + w * 32 + t];
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
      // a Q tile is 128 rows: one 128-token block, or two 64-token blocks stacked (an absent second
      // block re-reads the first: finite data whose rows are never used)
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int tok = max(blk[q] >= 0 ? blk[q] : blk[0], 0) * BLK;
        unsigned char* dst = C::kSplitKV ? sQ + q * (BLK * 128) : sQ + q * C::kQBytes;
#pragma unroll
        for (int c = 0; c < D / 64; ++c) tma_load_4d(dst + c * 16384, &tmQ, bar_q, c * 64, tok, head, batch);
      }
      const int tile_base = p.slot ? (int)p.tile_base[batch] : 0;
      auto load_tile = [&](unsigned char* dst, const CUtensorMap* tm, uint64_t* bar, int n) {
#ifdef SPARSP_ATTN_NOLOAD  // tuning builds only: reuse stale tiles to take TMA traffic out of the picture
        if (n >= S) {
          mbar_arrive(bar);
          return;
        }
#endif
        mbar_expect_tx(bar, C::kTileBytes);
#pragma unroll
        for (int e = 0; e < C::kEPT; ++e) {
          const int ent = min(n * C::kEPT + e, n_ent - 1);  // an absent second half re-reads the last entry
          const int j = sEntJ[ent];
          const int slot = p.slot ? sSlot[ent] : -1;
          if (slot < 0) {
#pragma unroll
            for (int c = 0; c < D / 64; ++c)
              tma_load_4d(dst + c * 16384 + e * (BLK * 128), tm, bar, c * 64, j * BLK, head, batch);
          } else {
            // remote block: its K tile and V tile are consecutive tiles of the consumer's packed buffer
            const int tile = tile_base + 2 * slot + (tm == &tmV ? 1 : 0);
#pragma unroll
            for (int c = 0; c < D / 64; ++c)
              tma_load_4d(dst + c * 16384 + e * (BLK * 128), &tmP, bar, c * 64, 0, tile, 0);
          }
        }
      };
      int kn = 0, vn = 0;
      const long long t0 = clock64();
      while ((kn < n_tiles || vn < n_tiles) && !*s_abort) {
        bool progressed = false;
        if (kn < n_tiles && mbar_test_wait(k_empty + kn % S, ((kn / S) & 1) ^ 1)) {
          load_tile(sK + (kn % S) * C::kTileBytes, &tmK, k_full + kn % S, kn);
          ++kn;
          progressed = true;
        }
        if (vn < n_tiles && mbar_test_wait(v_empty + vn % S, ((vn / S) & 1) ^ 1)) {
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
  } else if (warp == 1 || warp == kIssuer1Warp) {
    // ================================ MMA issuers (one thread per stream) =================
    // Each issuer walks ALL KV tiles in order and, for every tile, first observes the tile's "full"
    // barrier and then arrives once on its "empty" barrier (count 2: one arrival per issuer) --
    // through tcgen05.commit after its MMAs if its stream uses the tile, directly otherwise.  The
    // two streams therefore never wait on each other's softmax, only on the shared K/V rings.
    // The whole warp runs the loop (uniform control flow and uniform operands, so descriptors and
    // addresses can live in uniform registers); one elected lane issues the tcgen05 instructions.
    if (n_tiles > 0) {
      const int s = (warp == 1) ? 0 : 1;
      const bool leader = elect_one();
      constexpr uint32_t kIdescQK = make_idesc_bf16(128, 128, 0, 0);
      constexpr uint32_t kIdescPV = make_idesc_bf16(128, D, 0, 1);
      const uint32_t tSs = tmem_base + s * 128;
      const uint32_t tPs = C::kDecoupledP ? tmem_base + C::kColP + s * 64 : tSs;  // bf16 P (A operand of P V)
      const uint32_t tOs = tmem_base + C::kColO + s * D;
      int qcnt = 0;  // Q K^T tiles issued
      constexpr int kVLag = (S >= 4) ? S - 2 : 1;
      const uint64_t descQ = make_smem_desc(smem_u32(sQ + (C::kSplitKV ? 0 : s) * C::kQBytes), 16, 1024);
      const uint64_t descK = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint64_t descV = make_smem_desc(smem_u32(sV), 16384, 1024);
      // low words of the descriptors per K step (stage 0); a stage adds kTileBytes/16 to the low word
      const uint32_t hiQK = (uint32_t)(descK >> 32), hiV = (uint32_t)(descV >> 32);
      uint32_t qlo[D / 16], klo[D / 16], vlo[8];
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (uint32_t)(((kk / 4) * 16384 + (kk % 4) * 32) >> 4);
        qlo[kk] = (uint32_t)descQ + off;
        klo[kk] = (uint32_t)descK + off;
      }
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) vlo[kk] = (uint32_t)descV + (uint32_t)((kk * 2048) >> 4);
      int vdone = 0;       // tiles whose V obligation (P V or plain release) has been handled
      int last_kept = -1;  // last tile whose Q K^T this stream has issued
      int pcnt = 0;        // P tiles consumed
      uint32_t started = 0;

      auto handle_v = [&](int m) {
        const bool keep = (stream_mask(m) >> s) & 1;
        if (keep) {
          PROF_T(t_p0);
          mbar_wait_bounded(p_full + s, pcnt & 1, s_abort, p.status, 20 + s, p.wait_limit);
          ++pcnt;
          PROF_T(t_p1);
          PROF_ADD(8, t_p0, t_p1);  // issuer waiting for P
        }
        PROF_T(t_v0);
        mbar_wait_bounded(v_full + m % S, (m / S) & 1, s_abort, p.status, 22, p.wait_limit);
        PROF_T(t_v1);
        PROF_ADD(10, t_v0, t_v1);  // issuer waiting for V
        if (keep) {
          tc_fence_after();
          const uint32_t stage_off = (uint32_t)(((m % S) * C::kTileBytes) >> 4);
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              mma_ts_lohi(tOs, tPs + kk * 8, vlo[kk] + stage_off, hiV, kIdescPV, (kk > 0) ? 1u : started);
            mma_commit(o_full + s);
            mma_commit(v_empty + m % S);
          }
          started = 1u;
          PROF_T(t_v2);
          PROF_ADD(6, t_v1, t_v2);  // issuer issuing P V
        } else if (leader) {
          mbar_arrive(v_empty + m % S);
        }
        __syncwarp();
      };

      mbar_wait_bounded(bar_q, 0, s_abort, p.status, 11, p.wait_limit);
      for (int n = 0; n < n_tiles; ++n) {
        const bool keep = (stream_mask(n) >> s) & 1;
        // a V stage is released at most kVLag + 1 steps after its fill (always fewer than the ring has stages)
        while (vdone < n - kVLag) handle_v(vdone++);
        PROF_T(t_k0);
        mbar_wait_bounded(k_full + n % S, (n / S) & 1, s_abort, p.status, 12, p.wait_limit);
        PROF_T(t_k1);
        PROF_ADD(9, t_k0, t_k1);  // issuer waiting for K
        if (keep) {
          if (C::kDecoupledP) {
            // S_s is free once the softmax warps have loaded the previous tile's scores
            if (qcnt > 0) mbar_wait_bounded(s_free + s, (qcnt - 1) & 1, s_abort, p.status, 24 + s, p.wait_limit);
          } else {
            while (vdone <= last_kept) handle_v(vdone++);  // P V of the previous kept tile frees S_s
          }
          PROF_T(t_k3);
          tc_fence_after();
          const uint32_t stage_off = (uint32_t)(((n % S) * C::kTileBytes) >> 4);
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk)
              mma_ss_lohi(tSs, qlo[kk], hiQK, klo[kk] + stage_off, hiQK, kIdescQK, kk > 0 ? 1u : 0u);
            mma_commit(s_full + s);
            mma_commit(k_empty + n % S);
          }
          ++qcnt;
          PROF_T(t_k2);
          PROF_ADD(7, t_k3, t_k2);  // issuer issuing Q K^T
          if (C::kDecoupledP)
            while (vdone <= last_kept) handle_v(vdone++);  // P V of the previous kept tile, after this Q K^T
          last_kept = n;
        } else if (leader) {
          mbar_arrive(k_empty + n % S);
        }
        __syncwarp();
      }
      while (vdone < n_tiles) handle_v(vdone++);
    }
  } else if (warp >= 2 && warp < 18) {
    // ================================ softmax warps =======================================
    const int sidx = (warp - 2) >> 3;       // stream
    const int half = ((warp - 2) >> 2) & 1;  // which 64 key columns of a tile this thread owns
    const int rgrp = warp & 3;               // tensor-memory lane group this warp may access
    const int row = rgrp * 32 + lane;
    const int rh = row >> 6;                 // which query block of a stacked Q tile the row belongs to
    const int pair_bar = 1 + sidx * 4 + rgrp;  // named barrier shared with the row's other thread
    const uint32_t lane_off = (uint32_t)(rgrp * 32) << 16;
    const uint32_t tS = tmem_base + sidx * 128 + lane_off;
    const uint32_t tP = (C::kDecoupledP ? tmem_base + C::kColP + sidx * 64 : tmem_base + sidx * 128) + lane_off;
    const uint32_t tO = tmem_base + C::kColO + sidx * D + lane_off;
    float m_used = -INFINITY;  // reference maximum (log2 domain) of the row's exponentials
    float l_run = 0.0f;        // this thread's share of the row sum
    int cnt = 0;

    PROF_T(t_loop0);
    PROF_ADD(11, t_cta0, t_loop0);  // prologue up to the softmax loop
    for (int n = 0; n < n_tiles; ++n) {
      if (!((stream_mask(n) >> sidx) & 1)) continue;
      // kept / valid columns of my 64-column half (warp-uniform)
      int nv;
      if (C::kSplitKV) {
        const int ent = n * 2 + half;
        nv = 0;
        if (ent < n_ent && ((sEntF[ent] >> rh) & 1)) nv = (int)min((int64_t)64, p.N - (int64_t)sEntJ[ent] * 64);
      } else {
        nv = (int)min((int64_t)128, p.N - (int64_t)sEntJ[n] * 128) - 64 * half;
        nv = max(0, min(64, nv));
      }
      const int valid[2] = {min(nv, 32), max(nv - 32, 0)};

      PROF_T(t_a);
      mbar_wait_bounded(s_full + sidx, cnt & 1, s_abort, p.status, 30 + sidx, p.wait_limit);
      tc_fence_after();
      PROF_T(t_b);
#ifdef SPARSP_ATTN_NOSOFTMAX  // tuning builds only: measure the MMA / TMA pipeline alone
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full + sidx);
      ++cnt;
      continue;
#endif
      float sv[64];
      tmem_ld32(tS + half * 64, reinterpret_cast<uint32_t*>(sv));
      tmem_ld32(tS + half * 64 + 32, reinterpret_cast<uint32_t*>(sv) + 32);
      tmem_ld_wait();
      if (C::kDecoupledP) {
        // S is in registers: let the issuer start the next Q K^T
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_free + sidx);
      }
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (valid[c] == 32) {
#pragma unroll
          for (int e = 0; e < 32; e += 2) mx = fmaxf(mx, fmaxf(sv[c * 32 + e], sv[c * 32 + e + 1]));
        } else if (valid[c] > 0) {
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, e < valid[c] ? sv[c * 32 + e] : -INFINITY);
        }
      }
      // exchange the two halves' maxima (double-buffered by tile parity); the barrier also orders
      // my partner's reads of S before my writes of P into the columns it read
      float* mslot = sMax + (((cnt & 1) * 2 + sidx) * 2) * 128;
      mslot[half * 128 + row] = mx;
      named_bar_sync(pair_bar, 64);
      mx = fmaxf(mx, mslot[(1 - half) * 128 + row]) * p.scale_log2;
      PROF_T(t_c);
      if (C::kDecoupledP && cnt > 0) {
        // the previous P V must have finished reading P (and updating O) before either is touched
        mbar_wait_bounded(o_full + sidx, (cnt - 1) & 1, s_abort, p.status, 34 + sidx, p.wait_limit);
        tc_fence_after();
      }
      const float m_new = fmaxf(m_used, mx);
      const bool grow = m_new > m_used + kGrowThreshold || (m_used == -INFINITY && m_new > -INFINITY);
      if (__any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? ex2(m_used - m_new) : 1.0f;  // m_used = -inf -> 0
        if (cnt > 0) {  // S_s of this tile is complete, hence so is every earlier P V of the stream
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {  // my half of the accumulator's columns, 16 at a time
            uint32_t o[16];
            tmem_ld16(tO + half * (D / 2) + c * 16, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st16(tO + half * (D / 2) + c * 16, o);
          }
        }
        l_run *= alpha;
        if (grow) m_used = m_new;
      }
      PROF_T(t_d);

      // exponentials; bf16 P overwrites S in place: my keys [64*half, 64*half+64) go to columns
      // [32*half, 32*half+32)
      float lsum = 0.0f;
      float2 lsum2 = make_float2(0.0f, 0.0f);
      const float neg_m = -m_used;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t pk[16];
        const float* svc = sv + c * 32;
        if (valid[c] == 32) {
#if SPARSP_TUNE_F32X2
          const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float2 x = ffma2(make_float2(svc[2 * e], svc[2 * e + 1]), sc2, nm2);
            const float2 pp = (SPARSP_TUNE_POLY > 0 && (e % (SPARSP_TUNE_POLY > 0 ? SPARSP_TUNE_POLY : 1)) == 1)
                                  ? exp2_poly2(x)
                                  : make_float2(ex2(x.x), ex2(x.y));
            lsum2 = fadd2(lsum2, pp);
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(pp.x, pp.y);
            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
#else
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = ex2(fmaf(svc[2 * e], p.scale_log2, neg_m));
            const float p1 = ex2(fmaf(svc[2 * e + 1], p.scale_log2, neg_m));
            lsum += p0 + p1;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
#endif
        } else if (valid[c] > 0) {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = 2 * e < valid[c] ? ex2(fmaf(svc[2 * e], p.scale_log2, neg_m)) : 0.0f;
            const float p1 = 2 * e + 1 < valid[c] ? ex2(fmaf(svc[2 * e + 1], p.scale_log2, neg_m)) : 0.0f;
            lsum += p0 + p1;
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) pk[e] = 0u;
        }
        tmem_st16(tP + half * 32 + c * 16, pk);
      }
      l_run += lsum + (lsum2.x + lsum2.y);
      PROF_T(t_e);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full + sidx);
      ++cnt;
      PROF_T(t_f);
      PROF_ADD(0, t_a, t_b);  // wait for S
      PROF_ADD(1, t_b, t_c);  // load + max + exchange
      PROF_ADD(2, t_c, t_d);  // rescale decision
      PROF_ADD(3, t_d, t_e);  // exponentials + P store
      PROF_ADD(4, t_e, t_f);  // store wait + arrive
      PROF_ADD(5, t_a, t_a + 1);  // tile count
    }

    // ---- epilogue -------------------------------------------------------------------------
    PROF_T(t_ep0);
    if (cnt > 0) {
      mbar_wait_bounded(o_full + sidx, (cnt - 1) & 1, s_abort, p.status, 40 + sidx, p.wait_limit);
      tc_fence_after();
    }
    PROF_T(t_ep1);
    PROF_ADD(12, t_ep0, t_ep1);  // wait for the last P V
    sStat[(sidx * 2 + half) * 128 + row] = make_float2(m_used, l_run);
    if (!C::kSplitKV) {
      // the row's two threads add their partial sums; each writes its half of the columns
      named_bar_sync(pair_bar, 64);
      const float l = l_run + sStat[(sidx * 2 + 1 - half) * 128 + row].y;
      const int64_t tok = blk[sidx] >= 0 ? (int64_t)blk[sidx] * BLK + row : p.N;
      const float inv_l = l > 0.0f ? 1.0f / l : 0.0f;
      __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT + half * (D / 2);
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        uint32_t o[32];
        if (cnt > 0) {  // warp-uniform: tensor-memory loads are warp-collective
          tmem_ld32(tO + half * (D / 2) + c * 32, o);
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
      if (p.lse && half == 0 && tok < p.N)
        p.lse[(int64_t)bh * p.N + tok] = l > 0.0f ? (m_used + log2f(l)) * 0.6931471805599453f : -INFINITY;
    } else {
      // merge the two streams' partial results.  Thread (stream s, half h) finalises the column
      // quarter 2s+h; it hands the other stream's thread of the same half the quarter that one
      // finalises, scaled to the common reference maximum.
      constexpr int QW = D / 4;
      float* mbuf = reinterpret_cast<float*>(sK);  // K/V rings are idle once both streams are done
      named_bar_sync(9, 512);
      const float l_me = l_run + sStat[(sidx * 2 + 1 - half) * 128 + row].y;
      const float2 o0 = sStat[((1 - sidx) * 2) * 128 + row];
      const float2 o1 = sStat[((1 - sidx) * 2 + 1) * 128 + row];
      const float m_ot = o0.x, l_ot = o0.y + o1.y;
      const float m = fmaxf(m_used, m_ot);
      const float a_me = m_used > -INFINITY ? ex2(m_used - m) : 0.0f;
      const float a_ot = m_ot > -INFINITY ? ex2(m_ot - m) : 0.0f;
      const float l = l_me * a_me + l_ot * a_ot;
      const float inv_l = l > 0.0f ? 1.0f / l : 0.0f;
      const int give_q = 2 * (1 - sidx) + half, keep_q = 2 * sidx + half;
      float* give = mbuf + ((size_t)(sidx * 2 + half) * 128 + row) * C::kMergeStride;
      {
        uint32_t o[QW];
        if (cnt > 0) {
          if constexpr (QW == 32) tmem_ld32(tO + give_q * QW, o); else tmem_ld16(tO + give_q * QW, o);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < QW; ++e) o[e] = 0u;
        }
#pragma unroll
        for (int v = 0; v < QW / 4; ++v)
          *reinterpret_cast<float4*>(give + v * 4) =
              make_float4(__uint_as_float(o[v * 4]) * a_me, __uint_as_float(o[v * 4 + 1]) * a_me,
                          __uint_as_float(o[v * 4 + 2]) * a_me, __uint_as_float(o[v * 4 + 3]) * a_me);
      }
      named_bar_sync(9, 512);
      const int64_t tok = blk[rh] >= 0 ? (int64_t)blk[rh] * BLK + (row & 63) : p.N;
      const float* take = mbuf + ((size_t)((1 - sidx) * 2 + half) * 128 + row) * C::kMergeStride;
      __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT + keep_q * QW;
      {
        uint32_t o[QW];
        if (cnt > 0) {
          if constexpr (QW == 32) tmem_ld32(tO + keep_q * QW, o); else tmem_ld16(tO + keep_q * QW, o);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < QW; ++e) o[e] = 0u;
        }
        if (tok < p.N) {
#pragma unroll
          for (int v = 0; v < QW / 8; ++v) {
            const float4 t0 = *reinterpret_cast<const float4*>(take + v * 8);
            const float4 t1 = *reinterpret_cast<const float4*>(take + v * 8 + 4);
            const float tt[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float x0 = (__uint_as_float(o[v * 8 + 2 * e]) * a_me + tt[2 * e]) * inv_l;
              const float x1 = (__uint_as_float(o[v * 8 + 2 * e + 1]) * a_me + tt[2 * e + 1]) * inv_l;
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
              w[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(orow + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
      if (p.lse && sidx == 0 && half == 0 && tok < p.N)
        p.lse[(int64_t)bh * p.N + tok] = l > 0.0f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }

  PROF_T(t_cta1);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
  PROF_T(t_cta2);
  PROF_ADD(13, t_cta0, t_cta1);  // CTA lifetime of the sampled lanes up to the final barrier
  PROF_ADD(14, t_cta1, t_cta2);  // final barrier + dealloc
  PROF_ADD(15, t_cta0, t_cta0 + 1);
}

// ------------------------------------------------------------------------------------------------
// Pairing pass: which two query blocks of a head share a CTA.  Blocks i and i+D are paired in
// stripes (i mod 2D < D), leftovers pair up consecutively.  With `search` the offset D in 1..NB/2 that
// maximises the summed overlap |M[i] & M[i+D]| of the kept lists is chosen per (batch, head) --
// video attention is multi-diagonal, so the best partner of a block is typically the same position a
// fixed number of blocks away; the more two stacked blocks share, the less of a 128-row tile's work
// is masked away.  Without `search`, D = 1 (neighbours).  One CTA per (batch, head).
// ------------------------------------------------------------------------------------------------
constexpr int kPairThreads = 256;
constexpr int kPairSample = 4;

__global__ void __launch_bounds__(kPairThreads) pair_kernel(const uint32_t* __restrict__ mask, int NB, int Wd,
                                                            int search, int32_t* __restrict__ pairs) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* m = reinterpret_cast<uint32_t*>(smem_raw);  // [NB][Wd]
  __shared__ unsigned int s_best;                        // (score << 10) | (1023 - D): max = best score, smallest D
  const int bh = blockIdx.x;
  if (threadIdx.x == 0) s_best = (0u << 10) | (1023u - 1u);  // default D = 1
  if (search) {
    const uint32_t* src = mask + (int64_t)bh * NB * Wd;
    for (int idx = threadIdx.x; idx < NB * Wd; idx += kPairThreads) m[idx] = src[idx];
    __syncthreads();
    for (int d = 1 + threadIdx.x; d <= NB / 2; d += kPairThreads) {
      unsigned int score = 0;
      for (int i = 0; i + d < NB; i += kPairSample)  // every kPairSample-th row is enough to rank offsets
        for (int w = 0; w < Wd; ++w) score += __popc(m[i * Wd + w] & m[(i + d) * Wd + w]);
      atomicMax(&s_best, (score << 10) | (unsigned int)(1023 - d));
    }
  }
  __syncthreads();
  const int D = 1023 - (int)(s_best & 1023u);
  // stripes: rows with (i mod 2D) < D pair with i + D; the rows of the last partial stripe that have
  // no partner form one consecutive run and pair up as neighbours
  const int full = NB / (2 * D), R = NB % (2 * D);
  const int np_last = max(R - D, 0), lo_end = min(R, D);
  int32_t* out = pairs + (int64_t)bh * ((NB + 1) / 2) * 2;
  for (int i = threadIdx.x; i < NB; i += kPairThreads) {
    const int st = i / (2 * D), pos = i % (2 * D);
    if (st < full) {
      if (pos < D) {
        out[2 * (st * D + pos)] = i;
        out[2 * (st * D + pos) + 1] = i + D;
      }
    } else if (pos < np_last) {
      out[2 * (full * D + pos)] = i;
      out[2 * (full * D + pos) + 1] = i + D;
    } else if (pos < lo_end) {
      const int k = pos - np_last, n_left = lo_end - np_last;
      if ((k & 1) == 0) {
        const int c = full * D + np_last + k / 2;
        out[2 * c] = i;
        out[2 * c + 1] = (k + 1 < n_left) ? i + 1 : -1;
      }
    }
  }
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

// Packed buffer viewed as a sequence of (block x d) bf16 tiles: dims (d, block, n_tiles, 1).
static int make_packed_tmap(CUtensorMap* out, const void* packed, int64_t capacity_bytes, const Geometry& g) {
  EncodeTiledFn enc = get_encode_fn();
  if (!enc) {
    set_error("cuTensorMapEncodeTiled is not available from the driver");
    return SPARSP_ERR_CUDA;
  }
  const int64_t tile_bytes = (int64_t)g.b * g.d * 2;
  const int64_t n_tiles = capacity_bytes / tile_bytes;
  if (n_tiles < 1 || n_tiles > 0x7fffffff) {
    set_error("packed buffer holds %lld tiles: outside 1..2^31-1", (long long)n_tiles);
    return SPARSP_ERR_INVALID_ARG;
  }
  cuuint64_t dims[4] = {(cuuint64_t)g.d, (cuuint64_t)g.b, (cuuint64_t)n_tiles, 1};
  cuuint64_t strides[3] = {(cuuint64_t)g.d * 2, (cuuint64_t)tile_bytes, (cuuint64_t)(tile_bytes * n_tiles)};
  cuuint32_t box[4] = {64, (cuuint32_t)g.b, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(packed), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_error("cuTensorMapEncodeTiled (packed) failed with %d", (int)r);
    return SPARSP_ERR_CUDA;
  }
  return SPARSP_OK;
}

template <int D, int BLK>
static int launch_attn_t(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                         const void* packed, int64_t packed_capacity, const AttnParams& p, cudaStream_t st) {
  CUtensorMap tq, tk, tv, tp;
  int rc;
  if ((rc = make_tmap(&tq, Q, s, g, BLK)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tk, K, s, g, BLK)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tv, V, s, g, BLK)) != SPARSP_OK) return rc;
  if (packed) {
    if ((rc = make_packed_tmap(&tp, packed, packed_capacity, g)) != SPARSP_OK) return rc;
  } else {
    tp = tk;  // never used without a slot table
  }
  auto kern = attn_fwd_kernel<D, BLK>;
  const int smem = AttnCfg<D, BLK>::kDynamic;
  SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)kern, smem));
  dim3 grid((unsigned)((g.NB + 1) / 2), (unsigned)(g.B * g.H));
  kern<<<grid, kAttnThreads, smem, st>>>(tq, tk, tv, tp, p);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

static int launch_attn_common(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                              const void* packed, int64_t packed_capacity, AttnParams p, float scale, void* O,
                              float* lse, char* ws, const WsLayout& L, cudaStream_t st) {
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
  if (g.d == 64 && g.b == 64) return launch_attn_t<64, 64>(s, g, Q, K, V, packed, packed_capacity, p, st);
  if (g.d == 64 && g.b == 128) return launch_attn_t<64, 128>(s, g, Q, K, V, packed, packed_capacity, p, st);
  if (g.d == 128 && g.b == 64) return launch_attn_t<128, 64>(s, g, Q, K, V, packed, packed_capacity, p, st);
  return launch_attn_t<128, 128>(s, g, Q, K, V, packed, packed_capacity, p, st);
}

int launch_attn(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                const uint32_t* mask, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                cudaStream_t st) {
  int32_t* pairs = (int32_t*)(ws + L.pairs);
  {
    const size_t smem = (size_t)g.NB * g.Wd * 4;
    SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)pair_kernel, (int)smem));
    pair_kernel<<<g.B * g.H, kPairThreads, smem, st>>>(mask, g.NB, g.Wd, g.b == 64 ? 1 : 0, pairs);
    count_launch();
  }
  AttnParams p;
  p.mask = mask;
  p.pairs = pairs;
  p.slot = nullptr;
  p.tile_base = nullptr;
  return launch_attn_common(s, g, Q, K, V, nullptr, 0, p, scale, O, lse, ws, L, st);
}

// ------------------------------------------------------------------------------------------------
// Packed-source attention for one consumer rank: pairs are formed among the consumer's own query
// blocks, and every kept KV block the consumer does not own is read from the consumer's packed buffer.
// ------------------------------------------------------------------------------------------------
// pairs of the consumer's blocks (ascending, neighbours in that order); the rest of the table is (-1, -1)
__global__ void pair_rank_kernel(const int32_t* __restrict__ rank, int NB, int consumer, int32_t* __restrict__ pairs) {
  const int n_pairs = (NB + 1) / 2;
  int32_t* out = pairs + (int64_t)blockIdx.x * n_pairs * 2;
  for (int i = threadIdx.x; i < 2 * n_pairs; i += blockDim.x) out[i] = -1;
  __syncthreads();
  if (threadIdx.x == 0) {
    int k = 0;
    for (int i = 0; i < NB; ++i)
      if (rank[i] == consumer) out[k++] = i;  // pair c = entries 2c and 2c+1
  }
}

// slot[bh][j] = entry index of block j inside the consumer's packed buffer (pack order: producer ascending,
// head ascending, block ascending), for every block of the consumer's union that another rank owns.  One warp
// per (batch, producer, head).  The table must have been filled with -1.  Also writes tile_base[b].
__global__ void slot_kernel(const uint32_t* __restrict__ U, const int32_t* __restrict__ rank,
                            const int64_t* __restrict__ seg_off, const int64_t* __restrict__ seg_total,
                            const int64_t* __restrict__ dst_base, int B, int H, int NB, int Wd, int P, int consumer,
                            int64_t tile_bytes, int32_t* __restrict__ slot, int64_t* __restrict__ tile_base) {
  const int64_t wid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (wid < B && lane == 0) {  // first tile of the consumer's buffer for batch item wid
    const int64_t br = wid * P + consumer;
    int64_t base;
    if (dst_base) {
      base = dst_base[br];
    } else {
      base = 0;
      for (int64_t t = 0; t < br; ++t) base += seg_total[t] * 2 * tile_bytes;
    }
    tile_base[wid] = base / tile_bytes;
  }
  const int64_t n_seg = (int64_t)B * P * H;
  if (wid >= n_seg) return;
  const int h = (int)(wid % H);
  const int prod = (int)((wid / H) % P);
  const int bb = (int)(wid / ((int64_t)H * P));
  if (prod == consumer) return;
  const uint32_t* u = U + ((int64_t)(bb * P + consumer) * H + h) * Wd;
  const int64_t first = seg_off[((int64_t)(bb * P + consumer) * P + prod) * H + h];
  int32_t* out = slot + (int64_t)(bb * H + h) * NB;
  int running = 0;
  for (int w0 = 0; w0 < Wd; w0 += 32) {
    const int w = w0 + lane;
    uint32_t bits = 0;
    if (w < Wd) {
      uint32_t own = 0;
      for (int t = 0; t < 32; ++t) {
        const int j = w * 32 + t;
        if (j < NB && rank[j] == prod) own |= 1u << t;
      }
      bits = u[w] & own;
    }
    const int mine = __popc(bits);
    int incl = mine;
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, sft);
      if (lane >= sft) incl += v;
    }
    int pos = running + incl - mine;
    while (bits) {
      const int t = __ffs(bits) - 1;
      bits &= bits - 1;
      out[w * 32 + t] = (int32_t)(first + pos);
      ++pos;
    }
    running += __shfl_sync(0xffffffffu, incl, 31);
  }
}

int launch_attn_packed(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                       const uint32_t* mask, const int32_t* rank, int P, int consumer, const uint32_t* U,
                       const int64_t* seg_off, const int64_t* seg_total, const void* packed, int64_t capacity,
                       const int64_t* dst_base, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                       cudaStream_t st) {
  int32_t* pairs = (int32_t*)(ws + L.pairs);
  int32_t* slot = (int32_t*)(ws + L.slot);
  int64_t* tile_base = (int64_t*)(ws + L.tile_base);
  const int64_t tile_bytes = (int64_t)g.b * g.d * 2;
  SPARSP_CUDA_OK(cudaMemsetAsync(slot, 0xFF, (size_t)g.B * g.H * g.NB * 4, st));
  pair_rank_kernel<<<g.B * g.H, 128, 0, st>>>(rank, g.NB, consumer, pairs);
  const int64_t n_warps = std::max<int64_t>((int64_t)g.B * P * g.H, g.B);
  slot_kernel<<<(unsigned)((n_warps * 32 + 255) / 256), 256, 0, st>>>(U, rank, seg_off, seg_total, dst_base, g.B, g.H,
                                                                    g.NB, g.Wd, P, consumer, tile_bytes, slot,
                                                                    tile_base);
  count_launch(2);
  AttnParams p;
  p.mask = mask;
  p.pairs = pairs;
  p.slot = slot;
  p.tile_base = tile_base;
  return launch_attn_common(s, g, Q, K, V, packed, capacity, p, scale, O, lse, ws, L, st);
}

#ifdef SPARSP_ATTN_PROFILE
extern "C" __attribute__((visibility("default"))) int sparsp_debug_attn_profile(unsigned long long* out16, int reset) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(out16, g_attn_prof, sizeof(g_attn_prof));
  if (reset) {
    unsigned long long z[16] = {0};
    cudaMemcpyToSymbol(g_attn_prof, z, sizeof z);
  }
  return 0;
}
#endif

}  // namespace sparsp
