// Step 3: block-sparse FlashAttention forward on tcgen05 tensor cores (sm_100a).
//
// Work item = ONE 128-row Q tile of one (batch, head) with one fp32 accumulator O in tensor memory:
//   block = 128: the Q tile is one query block; the item walks that block's kept KV blocks.
//   block = 64 : two query blocks (chosen by a pairing pass so that their kept lists overlap) are stacked
//                into the Q tile (full-rate M = 128 MMAs); a KV tile is two entries of the UNION of their
//                kept lists (128 keys, full-rate N = 128); each 64x64 quadrant the mask does not keep is
//                zeroed in P.
// The kernel is persistent: one CTA per SM takes items from a global counter; the next item's kept
// list, Q tile and first K/V tiles overlap the current item's last tiles, its first Q K^T the epilogue.
// The scores S = Q K^T are double-buffered in tensor memory (S: 2 x 128 fp32 columns; P: 64 columns of packed bf16,
// two buffers at d = 64, one at d = 128 where 16 columns hold the row sums instead; O: d columns), so that the tensor pipe always has the next
// tiles' MMAs queued while the softmax of the current tile runs: Q K^T of tile g+2 starts as soon as the
// scores of tile g have been READ, and P V of tile g is issued as soon as P_g is written.  Tiles are
// numbered g = 0, 1, 2, ... across the CTA's items; every ring, buffer and barrier phase follows g.
// Warp roles (512 threads = 4 warpgroups; the first two hand most of their registers to the other two):
//   warp 0      TMA producer of Q (per item) and of the K ring
//   warp 1      issues every Q K^T          warp 2      issues every P V
//   warp 3      TMA producer of the V ring
//   warp 4      builds the kept / union list of the NEXT items (two list buffers; warps 5-7 idle)
//   warps 8-11  softmax of the even tiles   warps 12-15 softmax of the odd tiles
// (A producer is one thread running a chain of dependent instructions next to busy softmax warps: it gets
// an instruction issued every ~8 cycles, so K and V loads have a warp each and keep per-tile work minimal.)
// A softmax thread owns one query row of its tile: the whole 128-column row of S sits in registers.  The
// two threads that own the same row (one per warpgroup) share the row's reference maximum through shared
// memory and take their decisions strictly in tile order (a pair of 64-thread named barriers per row
// group hands the turn back and forth); each keeps its own partial row sum.
// Online softmax is base-2 in fp32; O is rescaled lazily, only when a row's maximum has grown by more
// than 2^8 since the reference last moved -- the thread that decides so first waits for every P V
// issued so far, then rescales the row of O.
// Norm bounds shorten most tiles: |q_row| * (largest key norm of a block) * scale bounds the block's scores, so
// a tile whose bound stays within 2^64 of the row's reference skips its row-maximum pass, and once the bound
// with the item's largest key norm holds, the reference is final and the two warps of a row group stop taking
// turns for the rest of the item (load scores -> exponentials -> store P).
// And if that bound is at most 2^80 in absolute terms -- ordinary inputs -- the item needs no reference at all: every
// softmax thread takes its row's norm from the Q tile while the first Q K^T runs, and an item whose bounds hold runs
// on the fixed reference 0 from its first tile on.
// The block-64 pairing and the order of a head's items (longest list first) come from attn_prep_kernel,
// which also takes the key norms.
// Every mbarrier wait is bounded; a wait that runs out sets SPARSP_ERR_TIMEOUT in the status word
// and raises a CTA-wide flag that makes all later waits fall through, so the CTA still drains.
#include <algorithm>
#include <type_traits>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace sparsp {

using namespace ptx;

struct AttnParams {
  const uint32_t* mask;
  // block 64: [B*H][ceil(NB/2)][2] query blocks of each item (second may be -1); block 128:
  // [B*H][2*ceil(NB/2)] query block of each item (-1 = none), or NULL (item x handles block x)
  const int32_t* pairs;
  // packed-source mode (NULL = every tile comes from K / V): slot[bh][j] = entry index of KV block j in
  // the consumer's packed buffer, or -1 if the consumer owns the block; tile_base = index of the
  // consumer's first tile in the packed tensor map (a device scalar)
  const int32_t* slot;
  const int64_t* tile_base;
  // largest key norm (L2) of every KV block, [B*H][NB], or NULL: lets a softmax row skip the row-maximum pass
  // of a tile whose scores provably stay within 2^kSkipMargin of the row's reference maximum
  const float* knorm;
  __nv_bfloat16* O;
  float* lse;
  int32_t* status;
  int32_t* work_counter;  // next work item to hand out; zeroed by the preparatory launch
  // packed-source mode: number of work items per (batch, head) that can have rows at all (the consumer's query
  // blocks come first in the pairs table), a device scalar; NULL = all per_bh items
  const int32_t* active_per_bh;
  int64_t N;
  int64_t sB, sH, sT;
  int H, NB, Wd;
  int per_bh;   // work items per (batch, head): NB (block 128) or ceil(NB/2) (block 64)
  int n_items;  // B * H * per_bh
  float scale_log2;  // softmax scale * log2(e)
  long long wait_limit;
};

constexpr int kAttnThreads = 512;  // four warpgroups: two of utility warps, softmax of the even tiles, softmax of the odd tiles
// register budget per thread after the warpgroups re-balance (128*48 + 128*32 + 256*216 = 512*128)
#ifndef SPARSP_REGS_UTILITY
#define SPARSP_REGS_UTILITY 48
#define SPARSP_REGS_UTILITY2 32
#define SPARSP_REGS_SOFTMAX 216
#endif
constexpr int kTmemCols = 512;
constexpr int kWorkCounterWord = 8;  // word of the workspace header that holds the attention work counter
constexpr float kGrowThreshold = 8.0f;
constexpr float kSkipMargin = 64.0f;  // 2^64 * (keys of a sequence) * |V| stays far inside fp32
// If |q_row| * (largest key norm of the item) * scale * log2(e) <= kStaticBound for all rows of a warp, every score of
// the item lies in [-kStaticBound, kStaticBound] (log2 domain) and the fixed reference 0 serves the whole item:
// exponentials between 2^-80 and 2^80 are normal numbers in fp32 and bf16 with full relative precision, and
// 2^80 * (keys of a sequence) * |V| stays inside fp32.
constexpr float kStaticBound = 80.0f;
// Tuning switch (compile-time): how many of the exponentials go to the FMA pipe instead of the
// special-function unit (every n-th pair; 0 = none).
#ifndef SPARSP_TUNE_POLY
#define SPARSP_TUNE_POLY 3
#endif
// d = 128: take the row sum on the tensor pipe as well (an extra N = 16 MMA per 16 keys against a small block of
// ones), at the price of the second P buffer, whose tensor-memory columns the 16 sum columns need (1 = on)
#ifndef SPARSP_SUM_MMA_128
#define SPARSP_SUM_MMA_128 1
#endif
// ... at d = 64 (measured there: every 3rd pair is 3 % faster than every 4th, every 2nd 4 % slower; at d = 128, with the
// row sum on the tensor pipe, every 3rd is 1-2 % faster than every 4th and every 2nd 2 % slower)
#ifndef SPARSP_TUNE_POLY_D64
#define SPARSP_TUNE_POLY_D64 3
#endif

template <int D, int BLK>
struct AttnCfg {
  static constexpr bool kStacked = (BLK == 64);  // Q tile = two 64-token query blocks
  static constexpr int kEPT = 128 / BLK;         // kept-list entries per 128-key KV tile
  static constexpr int kStagesK = (D == 64) ? 4 : 3;
  static constexpr int kStagesV = (D == 64) ? 4 : 2;
  static constexpr int kQBytes = 128 * D * 2;
  static constexpr int kTileBytes = 128 * D * 2;  // one K or V tile
  static constexpr int kOffQ = 0;
  static constexpr int kOffK = kOffQ + kQBytes;
  static constexpr int kOffV = kOffK + kStagesK * kTileBytes;
  // d = 64 leaves room in tensor memory for 16 more accumulator columns: P V then runs with N = 80, its B
  // operand continuing, 64 columns on, into a constant [128 keys][column 64 = 1, the rest 0] block in shared
  // memory, so that accumulator column 64 is the row sum of P -- taken by the tensor pipe from the very
  // bf16 values it multiplies with V, instead of one more packed add per pair of scores in the softmax warps
  static constexpr bool kOnes = (D == 64);
  static constexpr int kAccCols = D + (kOnes ? 16 : 0);
  // d = 128: the row sum also comes from the tensor pipe, through a separate N = 16 MMA per 16
  // keys against a [16 keys][column 0 = 1] block (2 KB, 128-byte swizzle like a V box), into 16 tensor-memory columns
  // of its own -- which exist only if P keeps ONE buffer instead of two (tensor memory is full otherwise)
  static constexpr bool kSum128 = (D == 128 && SPARSP_SUM_MMA_128 != 0);
  static constexpr bool kSumMma = kOnes || kSum128;  // the softmax warps keep no row sums
  static constexpr int kNumP = kSum128 ? 1 : 2;
  static constexpr int kOffOnes = kOffV + kStagesV * kTileBytes;  // bf16 [128][64], 128-byte swizzle like a V box
  static constexpr int kOffEntJ = kOffOnes + (kOnes ? 128 * 128 : (kSum128 ? 2048 : 0));  // uint16 [2][1024] kept / union list
  static constexpr int kOffEntV = kOffEntJ + 2 * 2 * kMaxBlocks;  // uint8 [2][1024][2] keys of the entry valid for query block q (0 = not kept)
  static constexpr int kOffSlot = kOffEntV + 2 * 2 * kMaxBlocks;  // int32 [2][1024] packed-buffer slot per entry
  static constexpr int kOffEntN = kOffSlot + 2 * 4 * kMaxBlocks;  // float [2][1024] largest key norm of the entry's block
  static constexpr int kOffStat = kOffEntN + 2 * 4 * kMaxBlocks;  // float2 [2 items][2 warpgroups][128]
  static constexpr int kOffRef = kOffStat + 2 * 2 * 128 * 8;      // float [3 items][128] reference maximum per row
  static constexpr int kOffBars = kOffRef + 3 * 128 * 4;
  static constexpr int kNumBars = 2 + 2 * (kStagesK + kStagesV) + 10 + 1 + 4;
  static constexpr int kColS = 0;    // S buffers: columns [0, 256)
  static constexpr int kColP = 256;  // P: two buffers in columns [256, 384), or one in [256, 320) with the row sums in [320, 336)
  static constexpr int kColO = 384;  // accumulator: columns [384, 384 + d)
  static constexpr int kColL = kOnes ? kColO + D : 320;  // row sums (column 0 of 16), where the tensor pipe takes them
  static constexpr int kOffMisc = kOffBars + 8 * kNumBars;
  static constexpr int kTotal = kOffMisc + 80;
  static constexpr int kDynamic = kTotal + 1024;  // slack for the 1024-byte alignment of the base
  static_assert(kDynamic <= 232448, "shared memory budget");
};

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
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmP,
                    const AttnParams p) {
  using C = AttnCfg<D, BLK>;
  constexpr int SK = C::kStagesK, SV = C::kStagesV;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem + C::kOffQ;
  unsigned char* sK = smem + C::kOffK;
  unsigned char* sV = smem + C::kOffV;
  uint16_t* sEntJ = reinterpret_cast<uint16_t*>(smem + C::kOffEntJ);  // [2][kMaxBlocks]
  uint8_t* sEntV = smem + C::kOffEntV;                                // [2][kMaxBlocks][2]
  int32_t* sSlot = reinterpret_cast<int32_t*>(smem + C::kOffSlot);    // [2][kMaxBlocks]
  float* sEntN = reinterpret_cast<float*>(smem + C::kOffEntN);        // [2][kMaxBlocks]
  float2* sStat = reinterpret_cast<float2*>(smem + C::kOffStat);      // [2][2][128]
  volatile float* sRef = reinterpret_cast<volatile float*>(smem + C::kOffRef);  // [3][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kOffBars);
  uint64_t* q_full = bars;          // the item's Q tile has landed
  uint64_t* q_free = bars + 1;      // every Q K^T of the item has completed: Q may be overwritten
  uint64_t* k_full = bars + 2;
  uint64_t* k_empty = k_full + SK;
  uint64_t* v_full = k_empty + SK;
  uint64_t* v_empty = v_full + SV;
  uint64_t* s_full = v_empty + SV;  // [2] S buffer written by a Q K^T
  uint64_t* s_free = s_full + 2;    // [2] S buffer read into registers by its 4 softmax warps
  uint64_t* p_full = s_free + 2;    // [2] P of an even / odd tile written by its 4 softmax warps
  // [4] the P V of tile g arrives on o_full[g % 4].  Four barriers, because a parity wait can only tell the
  // phase a barrier is in from the one before: a softmax thread that wants P V g-1 or g-2 has itself seen
  // P V g-4 complete, and P V g+2 cannot complete before that thread has stored P_g.
  uint64_t* o_full = p_full + 2;
  uint64_t* o_drained = o_full + 4;      // the item's accumulator has been read out by all 8 softmax warps
  uint64_t* list_ready = o_drained + 1;  // [2] list buffer filled
  uint64_t* list_free = list_ready + 2;  // [2] list buffer no longer needed by its 11 readers
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + C::kOffMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 4);
  int* s_nent = reinterpret_cast<int*>(smem + C::kOffMisc + 8);   // [2]
  int* s_blk = reinterpret_cast<int*>(smem + C::kOffMisc + 16);   // [2][2] the item's query block(s); < 0 = absent
  int* s_item = reinterpret_cast<int*>(smem + C::kOffMisc + 32);  // [2] the work item of each list buffer; < 0 = no more
  int* s_rag = reinterpret_cast<int*>(smem + C::kOffMisc + 40);   // [2] the item's last tile reaches past the end of the sequence
  volatile int* s_frz = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 56);  // [4] per row group: reference frozen
  volatile int* s_pv_items = reinterpret_cast<volatile int*>(smem + C::kOffMisc + 72);  // items whose P V are all issued
  float* s_knmax = reinterpret_cast<float*>(smem + C::kOffMisc + 48);  // [2] largest key norm bound among the item's entries
  constexpr int kListReaders = 12;  // two producers, two issuers, eight softmax warps

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- setup ------------------------------------------------------------------------------
  if (tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(q_full, 1);
    mbar_init(q_free, 1);
    for (int s = 0; s < SK; ++s) {
      mbar_init(k_full + s, 1);
      mbar_init(k_empty + s, 1);
    }
    for (int s = 0; s < SV; ++s) {
      mbar_init(v_full + s, 1);
      mbar_init(v_empty + s, 1);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(s_full + s, 1);
      mbar_init(s_free + s, 4);
      mbar_init(p_full + s, 4);
      mbar_init(list_ready + s, 1);
      mbar_init(list_free + s, kListReaders);
    }
    for (int s = 0; s < 4; ++s) mbar_init(o_full + s, 1);
    mbar_init(o_drained, 8);
    mbar_init_fence();
    *s_abort = 0;
    *s_pv_items = 0;
    for (int r = 0; r < 4; ++r) s_frz[r] = 0;
  }
  if (tid < 384) sRef[tid] = -INFINITY;  // 3 x 128 entries
  if (C::kSumMma) {
    // key row r holds column 64 + c at byte r*128 + ((c/8 ^ (r & 7)) << 4) + (c%8)*2 (the swizzle of a TMA box);
    // 128 key rows at d = 64 (one block for a whole tile), 16 at d = 128 (every group of 16 keys uses the same)
    uint4* ones = reinterpret_cast<uint4*>(smem + C::kOffOnes);
    for (int idx = tid; idx < (C::kOnes ? 128 : 16) * 8; idx += kAttnThreads) {
      const int r = idx >> 3, chunk = idx & 7;
      ones[idx] = make_uint4(chunk == (r & 7) ? 0x3F80u : 0u, 0u, 0u, 0u);  // bf16 1.0 in element 0 of logical chunk 0
    }
    fence_proxy_async_smem();  // read by the tensor pipe
  }
  if (warp == 1) {
    tmem_alloc(s_tmem, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  // the utility warpgroup hands most of its registers to the two softmax warpgroups (the re-balancing
  // instruction sits inside each role's branch so that the register allocator sees which code runs
  // under which limit)
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SPARSP_REGS_UTILITY));
    if (warp == 3) {
      // ================================ TMA producer: V =====================================
      if (lane == 0) {
        int vn = 0;  // V tiles loaded so far
        for (int i = 0;; ++i) {
          const int buf = i & 1;
          mbar_wait_bounded_inline(list_ready + buf, (i >> 1) & 1, s_abort, 58, p.wait_limit);
          const int it = s_item[buf];
          if (it < 0) break;  // (only the list builder decides when to stop, so that all roles stop at the same item)
          const int n_ent = s_nent[buf];
          const int n_tiles = (n_ent + C::kEPT - 1) / C::kEPT;
          if (n_tiles > 0) {
            const int bh = it / p.per_bh;
            const int batch = bh / p.H, head = bh % p.H;
            const uint16_t* entJ = sEntJ + buf * kMaxBlocks;
            const int32_t* entS = sSlot + buf * kMaxBlocks;
            const int tile_base = p.slot ? (int)p.tile_base[batch] : 0;
            for (int n = 0; n < n_tiles; ++n, ++vn) {
              const int st = vn % SV;
              mbar_wait_bounded_inline(v_empty + st, ((vn / SV) & 1) ^ 1, s_abort, 59, p.wait_limit);
              unsigned char* dst = sV + st * C::kTileBytes;
              mbar_expect_tx(v_full + st, C::kTileBytes);
  #pragma unroll
              for (int e = 0; e < C::kEPT; ++e) {
                const int ent = min(n * C::kEPT + e, n_ent - 1);
                const int slot = p.slot ? entS[ent] : -1;
                if (slot < 0) {
                  const int tok = (int)entJ[ent] * BLK;
  #pragma unroll
                  for (int c = 0; c < D / 64; ++c)
                    tma_load_4d(dst + c * 16384 + e * (BLK * 128), &tmV, v_full + st, c * 64, tok, head, batch);
                } else {
  #pragma unroll
                  for (int c = 0; c < D / 64; ++c)
                    tma_load_4d(dst + c * 16384 + e * (BLK * 128), &tmP, v_full + st, c * 64, 0, tile_base + 2 * slot + 1, 0);
                }
              }
            }
          }
          mbar_arrive(list_free + buf);
        }
      }
    } else if (warp == 0) {
      // ================================ TMA producer: Q and K ===============================
      if (lane == 0) {
        int kn = 0, qc = 0;  // K tiles loaded so far; items that had tiles
        for (int i = 0;; ++i) {
          const int buf = i & 1;
          mbar_wait_bounded_inline(list_ready + buf, (i >> 1) & 1, s_abort, 51, p.wait_limit);
          const int it = s_item[buf];
          if (it < 0) break;  // (only the list builder decides when to stop, so that all roles stop at the same item)
          const int n_ent = s_nent[buf];
          const int n_tiles = (n_ent + C::kEPT - 1) / C::kEPT;
          if (n_tiles > 0) {
            const int bh = it / p.per_bh;
            const int batch = bh / p.H, head = bh % p.H;
            const uint16_t* entJ = sEntJ + buf * kMaxBlocks;
            const int32_t* entS = sSlot + buf * kMaxBlocks;
            const int tile_base = p.slot ? (int)p.tile_base[batch] : 0;
            for (int n = 0; n < n_tiles; ++n, ++kn) {
              const int st = kn % SK;
              mbar_wait_bounded_inline(k_empty + st, ((kn / SK) & 1) ^ 1, s_abort, 57, p.wait_limit);
              unsigned char* dst = sK + st * C::kTileBytes;
              mbar_expect_tx(k_full + st, C::kTileBytes);
#pragma unroll
              for (int e = 0; e < C::kEPT; ++e) {
                const int ent = min(n * C::kEPT + e, n_ent - 1);  // an absent second half re-reads the last entry
                const int slot = p.slot ? entS[ent] : -1;
                if (slot < 0) {
                  const int tok = (int)entJ[ent] * BLK;
#pragma unroll
                  for (int c = 0; c < D / 64; ++c)
                    tma_load_4d(dst + c * 16384 + e * (BLK * 128), &tmK, k_full + st, c * 64, tok, head, batch);
                } else {
                  // remote block: its K tile and V tile are consecutive tiles of the consumer's packed buffer
#pragma unroll
                  for (int c = 0; c < D / 64; ++c)
                    tma_load_4d(dst + c * 16384 + e * (BLK * 128), &tmP, k_full + st, c * 64, 0, tile_base + 2 * slot, 0);
                }
              }
              if (n == 0) {
                // the item's first K tile is on its way; now the Q tile, which may be overwritten once every
                // Q K^T of the previous item has completed
                if (qc > 0) mbar_wait_bounded_inline(q_free, (qc - 1) & 1, s_abort, 52, p.wait_limit);
                ++qc;
                mbar_expect_tx(q_full, C::kQBytes);
                // a Q tile is 128 rows: one 128-token block, or two 64-token blocks stacked (an absent second
                // block re-reads the first: finite data whose rows are never used)
#pragma unroll
                for (int q = 0; q < C::kEPT; ++q) {
                  const int bq = s_blk[buf * 2 + q] >= 0 ? s_blk[buf * 2 + q] : s_blk[buf * 2];
                  const int tok = max(bq, 0) * BLK;
#pragma unroll
                  for (int c = 0; c < D / 64; ++c)
                    tma_load_4d(sQ + c * 16384 + q * (BLK * 128), &tmQ, q_full, c * 64, tok, head, batch);
                }
              }
            }
          }
          mbar_arrive(list_free + buf);
        }
      }
    } else if (warp == 1) {
      // ================================ Q K^T issuer ========================================
      // The whole warp runs the loop (uniform control flow and operands); one elected lane issues.
      const bool leader = elect_one();
      constexpr uint32_t kIdescQK = make_idesc_bf16(128, 128, 0, 0);
      const uint64_t descQ = make_smem_desc(smem_u32(sQ), 16, 1024);
      const uint64_t descK = make_smem_desc(smem_u32(sK), 16, 1024);
      const uint32_t hiQK = (uint32_t)(descK >> 32);
      uint32_t qlo[D / 16], klo[D / 16];
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (uint32_t)(((kk / 4) * 16384 + (kk % 4) * 32) >> 4);
        qlo[kk] = (uint32_t)descQ + off;
        klo[kk] = (uint32_t)descK + off;
      }
      int g = 0, qc = 0;
      for (int i = 0;; ++i) {
        const int buf = i & 1;
        mbar_wait_bounded_inline(list_ready + buf, (i >> 1) & 1, s_abort, 53, p.wait_limit);
        if (s_item[buf] < 0) break;
        const int n_tiles = (s_nent[buf] + C::kEPT - 1) / C::kEPT;
        if (n_tiles > 0) {
          // The tensor pipe works in issue order.  The first Q K^T of an item could be issued a tile or two
          // before the previous item ends, ahead of that item's last P V, and the epilogue (which waits for
          // that P V) would start ~1000 cycles later for nothing: the scores are not needed before the
          // epilogue is over.  So they wait until the previous item's P V are all issued.
          if (i > 0) {
            const long long t0 = clock64();
            while (*s_pv_items < i) {
              if (*s_abort) break;
              if (clock64() - t0 > p.wait_limit) {
                *s_abort = 14;
                break;
              }
            }
          }
          mbar_wait_bounded_inline(q_full, qc & 1, s_abort, 11, p.wait_limit);
          ++qc;
          for (int n = 0; n < n_tiles; ++n, ++g) {
            mbar_wait_bounded_inline(k_full + g % SK, (g / SK) & 1, s_abort, 12, p.wait_limit);
            // S buffer g%2 is free once the softmax warps have loaded the scores of tile g-2
            if (g >= 2) mbar_wait_bounded_inline(s_free + (g & 1), ((g - 2) >> 1) & 1, s_abort, 24, p.wait_limit);
            tc_fence_after();
            const uint32_t stage_off = (uint32_t)(((g % SK) * C::kTileBytes) >> 4);
            const uint32_t tS = tmem_base + C::kColS + (g & 1) * 128;
            if (leader) {
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk)
                mma_ss_lohi(tS, qlo[kk], hiQK, klo[kk] + stage_off, hiQK, kIdescQK, kk > 0 ? 1u : 0u);
              mma_commit(s_full + (g & 1));
              mma_commit(k_empty + g % SK);
              if (n == n_tiles - 1) mma_commit(q_free);
            }
            __syncwarp();
          }
        }
        if (lane == 0) mbar_arrive(list_free + buf);
        __syncwarp();
      }
    } else {
      // ================================ P V issuer ==========================================
      const bool leader = elect_one();
      constexpr uint32_t kIdescPV = make_idesc_bf16(128, C::kAccCols, 0, 1);
      // second 64-column group of the B operand: the other half of a d = 128 tile, or the block of ones, which
      // lies kOffOnes - kOffV behind the FIRST stage (the stage offset is taken off again below)
      const uint64_t descV = make_smem_desc(smem_u32(sV), C::kOnes ? (uint32_t)(C::kOffOnes - C::kOffV) : 16384u, 1024);
      const uint32_t hiV = (uint32_t)(descV >> 32);
      uint32_t vlo[8];
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) vlo[kk] = (uint32_t)descV + (uint32_t)((kk * 2048) >> 4);
      const uint32_t tO = tmem_base + C::kColO;
      constexpr uint32_t kIdescSum = make_idesc_bf16(128, 16, 0, 1);
      const uint64_t descOnes = make_smem_desc(smem_u32(smem + C::kOffOnes), 16384u, 1024);
      const uint32_t tL = tmem_base + C::kColL;
      int g = 0;
      for (int i = 0;; ++i) {
        const int buf = i & 1;
        mbar_wait_bounded_inline(list_ready + buf, (i >> 1) & 1, s_abort, 54, p.wait_limit);
        if (s_item[buf] < 0) break;
        const int n_tiles = (s_nent[buf] + C::kEPT - 1) / C::kEPT;
        // the previous item's accumulator must have been read out before this item's first P V overwrites it
        if (i > 0) mbar_wait_bounded_inline(o_drained, (i - 1) & 1, s_abort, 55, p.wait_limit);
        for (int n = 0; n < n_tiles; ++n, ++g) {
          mbar_wait_bounded_inline(p_full + (g & 1), (g >> 1) & 1, s_abort, 20, p.wait_limit);
          mbar_wait_bounded_inline(v_full + g % SV, (g / SV) & 1, s_abort, 22, p.wait_limit);
          tc_fence_after();
          uint32_t stage_off = (uint32_t)(((g % SV) * C::kTileBytes) >> 4);
          if (C::kOnes) stage_off -= stage_off << 16;  // start address up, distance to the ones block down
          const uint32_t tP = tmem_base + C::kColP + (C::kNumP == 2 ? (g & 1) * 64 : 0);
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              mma_ts_lohi(tO, tP + kk * 8, vlo[kk] + stage_off, hiV, kIdescPV, (kk > 0 || n > 0) ? 1u : 0u);
              if (C::kSum128)
                mma_ts_lohi(tL, tP + kk * 8, (uint32_t)descOnes, (uint32_t)(descOnes >> 32), kIdescSum,
                            (kk > 0 || n > 0) ? 1u : 0u);
            }
            mma_commit(o_full + (g & 3));
            mma_commit(v_empty + g % SV);
          }
          __syncwarp();
        }
        if (lane == 0) {
          *s_pv_items = i + 1;
          mbar_arrive(list_free + buf);
        }
        __syncwarp();
      }
    }
  } else if (warp < 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(SPARSP_REGS_UTILITY2));
    // ================================ list builder ========================================
    if (warp == 4) {
      // union of the item's (up to) two mask rows -> ascending entry list; flag bit q = kept by query
      // block blk[q].  Runs up to two items ahead of the consumers.
      // Work items are handed out by a global counter (first come, first served), so CTAs whose items are
      // short simply take more of them; the item number travels to the other roles with the list.
      for (int i = 0;; ++i) {
        const int buf = i & 1;
        if (i >= 2) mbar_wait_bounded_inline(list_free + buf, ((i - 2) >> 1) & 1, s_abort, 50, p.wait_limit);
        int it = 0;
        if (lane == 0) it = atomicAdd(p.work_counter, 1);
        it = __shfl_sync(0xffffffffu, it, 0);
        // one consumer's call walks only the items of its own query blocks (the first `active` of every head)
        const int active = p.active_per_bh ? *p.active_per_bh : p.per_bh;
        if (it >= active * (p.n_items / p.per_bh) || *s_abort) {
          if (lane == 0) {
            s_item[buf] = -1;
            mbar_arrive(list_ready + buf);
          }
          break;
        }
        const int bh = it / active, x = it - bh * active;
        it = bh * p.per_bh + x;  // the item's number in the full table, which the other roles derive the head from
        int blk[2];
        if (C::kStacked) {
          const int32_t* pr = p.pairs + ((int64_t)bh * p.per_bh + x) * 2;
          blk[0] = pr[0];
          blk[1] = pr[1];
        } else {
          blk[0] = p.pairs ? p.pairs[(int64_t)bh * (2 * ((p.NB + 1) / 2)) + x] : x;
          blk[1] = -1;
        }
        uint16_t* entJ = sEntJ + buf * kMaxBlocks;
        uint8_t* entV = sEntV + buf * kMaxBlocks * 2;
        int32_t* entS = sSlot + buf * kMaxBlocks;
        float* entN = sEntN + buf * kMaxBlocks;
        // NB <= 1024, so a mask row is at most 32 words: one word per lane
        const uint32_t rb0 = (lane < p.Wd && blk[0] >= 0) ? p.mask[((int64_t)bh * p.NB + blk[0]) * p.Wd + lane] : 0u;
        const uint32_t rb1 = (lane < p.Wd && blk[1] >= 0) ? p.mask[((int64_t)bh * p.NB + blk[1]) * p.Wd + lane] : 0u;
        // Entry order (any order gives the same attention).  Blocks BOTH query blocks keep make full tiles; a
        // block only the first keeps is put next to a block only the second keeps, so that such a tile costs
        // every softmax row one 64-key half instead of costing half of the rows two.  A full tile is bound by
        // the softmax warps, a half-work tile by the tensor pipe (its MMAs cost the same), so the two kinds
        // alternate in groups of two tiles (one of each per softmax warpgroup) while both last; then the rest
        // of the full tiles, the rest of the paired one-sided blocks and what is left of the longer one-sided
        // list.  With a single query block this is plain ascending order.
        uint32_t cls[3] = {rb0 & rb1, rb0 & ~rb1, rb1 & ~rb0};
        int before[3], total[3];
#pragma unroll
        for (int c = 0; c < 3; ++c) {
          const int mine = __popc(cls[c]);
          int incl = mine;
#pragma unroll
          for (int s = 1; s < 32; s <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, s);
            if (lane >= s) incl += v;
          }
          before[c] = incl - mine;
          total[c] = __shfl_sync(0xffffffffu, incl, 31);
        }
        const int n_both = total[0], n_mix = min(total[1], total[2]);
        // two full tiles (four blocks both keep), then two half-work tiles (two one-sided pairs), and so on
        const int n_grp = min(n_both >> 2, n_mix >> 1);
        const int running = total[0] + total[1] + total[2];
        float kn_max = 0.0f;
#pragma unroll
        for (int c = 0; c < 3; ++c) {
          uint32_t u = cls[c];
          int idx = before[c];  // rank of the entry inside its class
          while (u) {
            const int t = __ffs(u) - 1;
            u &= u - 1;
            int pos;
            if (c == 0) pos = idx < 4 * n_grp ? 8 * (idx >> 2) + (idx & 3) : 4 * n_grp + idx;
            else if (idx < 2 * n_grp) pos = 8 * (idx >> 1) + 4 + 2 * (idx & 1) + (c - 1);
            else if (idx < n_mix) pos = n_both + 2 * idx + (c - 1);
            else pos = n_both + n_mix + idx;  // tail of the longer class
            entJ[pos] = (uint16_t)(lane * 32 + t);
            const int jb = lane * 32 + t;
            const int nvalid = (int)min((int64_t)BLK, p.N - (int64_t)jb * BLK);
            entV[pos * 2] = (uint8_t)(c != 2 ? nvalid : 0);      // keys valid for the first query block's rows
            entV[pos * 2 + 1] = (uint8_t)(c != 1 ? nvalid : 0);  // ... for the second's
            if (p.slot) entS[pos] = p.slot[(int64_t)bh * p.NB + lane * 32 + t];
            if (p.knorm) {
              const float kn = p.knorm[(int64_t)bh * p.NB + lane * 32 + t];
              entN[pos] = kn;
              kn_max = fmaxf(kn_max, kn);
            }
            ++idx;
          }
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) kn_max = fmaxf(kn_max, __shfl_xor_sync(0xffffffffu, kn_max, s));
        __syncwarp();
        // the softmax code lets only the LAST tile reach past the end of the sequence: if the last block of
        // the sequence is ragged and in the list, it trades places with the last entry
        bool last_ragged = false;
        if ((int64_t)p.NB * BLK > p.N && running > 0) {
          const int lw = (p.NB - 1) >> 5, lb = (p.NB - 1) & 31;
          const uint32_t have = __shfl_sync(0xffffffffu, rb0 | rb1, lw);
          if ((have >> lb) & 1u) {
            last_ragged = true;
            if (lane == 0) {
              int r = 0;
              while (r < running - 1 && entJ[r] != (uint16_t)(p.NB - 1)) ++r;
              const int e = running - 1;
              const uint16_t tj = entJ[r]; entJ[r] = entJ[e]; entJ[e] = tj;
              for (int q = 0; q < 2; ++q) { const uint8_t tv = entV[r * 2 + q]; entV[r * 2 + q] = entV[e * 2 + q]; entV[e * 2 + q] = tv; }
              if (p.slot) { const int32_t ts = entS[r]; entS[r] = entS[e]; entS[e] = ts; }
              if (p.knorm) { const float tn = entN[r]; entN[r] = entN[e]; entN[e] = tn; }
            }
            __syncwarp();
          }
        }
        if (lane == 0) {
          s_item[buf] = it;
          s_rag[buf] = last_ragged ? 1 : 0;
          s_nent[buf] = running;
          s_knmax[buf] = kn_max;
          s_blk[buf * 2] = blk[0];
          s_blk[buf * 2 + 1] = blk[1];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(list_ready + buf);
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(SPARSP_REGS_SOFTMAX));
    // ================================ softmax warpgroups ==================================
    const int wg = (warp >> 2) - 2;  // 0: even tiles g, 1: odd tiles; also the S (and, where there are two, P) buffer this warpgroup uses
    const int rgrp = warp & 3;       // tensor-memory lane group this warp may access
    const int row = rgrp * 32 + lane;
    const int rh = row >> 6;         // which query block of a stacked Q tile the row belongs to
    const uint32_t lane_off = (uint32_t)(rgrp * 32) << 16;
    const uint32_t tS = tmem_base + C::kColS + wg * 128 + lane_off;
    const uint32_t tP = tmem_base + C::kColP + (C::kNumP == 2 ? wg * 64 : 0) + lane_off;
    const uint32_t tO = tmem_base + C::kColO + lane_off;
    const int bar_mine = 1 + wg * 4 + rgrp;         // I arrive here after my decision
    const int bar_other = 1 + (1 - wg) * 4 + rgrp;  // the row group's other warp arrives here after its decision
    volatile int* frz = s_frz + rgrp;               // set by the warp that freezes the reference, cleared by the other

    int g0 = 0;  // number of the item's first tile
    int qn = 0;  // items that had tiles (the phase of the Q barrier)
    for (int i = 0;; ++i) {
      const int buf = i & 1;
      volatile float* ref = sRef + (i % 3) * 128;
      mbar_wait_bounded_inline(list_ready + buf, (i >> 1) & 1, s_abort, 56, p.wait_limit);
      const int it = s_item[buf];
      if (it < 0) break;
      const int n_ent = s_nent[buf];
      const int n_tiles = (n_ent + C::kEPT - 1) / C::kEPT;
      const uint8_t* entV = sEntV + buf * kMaxBlocks * 2 + (C::kStacked ? rh : 0);  // my query block's column
      const bool item_ragged = s_rag[buf] != 0;
      const float* entN = sEntN + buf * kMaxBlocks;
      const float kn_item = s_knmax[buf];
      const int bh = it / p.per_bh;
      const int batch = bh / p.H, head = bh % p.H;
      // Once no score of any remaining tile of the item can exceed the row's reference maximum by more than
      // 2^kSkipMargin (Cauchy-Schwarz with the item's largest key norm), the reference is final: both warps of
      // the row group stop taking turns and the rest of the item is load -> exponentials -> store.
      bool frozen = false;
      float q_bound = INFINITY;  // |q_row| * softmax scale * log2(e) (+0.1 %), once known
      float m_ref = -INFINITY;  // the row's reference maximum (log2 domain) as this thread last saw it
      float l_run = 0.0f;       // this thread's partial row sum, relative to m_ref
      if (n_tiles > 0) {
        if (p.knorm != nullptr && n_tiles >= 4) {
          // The norm of my query row, read from the Q tile in shared memory while the item's first Q K^T runs (any
          // order of its 16-byte units will do, so the swizzle does not matter).  Q stays there until the item's
          // last Q K^T has completed; with four or more tiles that one cannot be issued before both warpgroups
          // have released a score buffer, which they do after this.
          mbar_wait_bounded_inline(q_full, qn & 1, s_abort, 42, p.wait_limit);
          float ss[4] = {0.0f, 0.0f, 0.0f, 0.0f};  // four chains, so that the additions do not wait for each other
#pragma unroll
          for (int c = 0; c < D / 64; ++c) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint4 v = *reinterpret_cast<const uint4*>(sQ + c * 16384 + row * 128 + (((k + lane) & 7) << 4));
              const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
                ss[e] = fmaf(lo, lo, ss[e]);
                ss[e] = fmaf(hi, hi, ss[e]);
              }
            }
          }
          q_bound = sqrtf((ss[0] + ss[1]) + (ss[2] + ss[3])) * p.scale_log2 * 1.001f;
          // Both threads of a row compute the same bound from the same data, so both warps of a row group take this
          // decision alike without talking to each other: the item runs on the fixed reference 0 from its first
          // tile on -- no row maximum, no turns, no named barrier (neither warp arrives, neither waits).
          if (__all_sync(0xffffffffu, q_bound * kn_item <= kStaticBound)) {
            frozen = true;
            m_ref = 0.0f;
            ref[row] = 0.0f;  // (both threads of the row write the same value; the epilogue reads it)
          }
        }
        ++qn;
      }

      // One tile of this warpgroup.  kRagged = the sequence ends inside the tile (possible only for the item's
      // last tile): that variant carries the column masking, the common one stays small.
      auto do_tile = [&](auto ragged_tag, const int n) {
        constexpr bool kRagged = decltype(ragged_tag)::value;
        const int g = g0 + n;
        // kept / valid key columns of each 64-column half of the tile (warp-uniform), as the list builder left them
        int vh[2];
        if (C::kStacked) {
          vh[0] = entV[(n * 2) * 2];
          vh[1] = n * 2 + 1 < n_ent ? entV[(n * 2 + 1) * 2] : 0;
        } else {
          const int nv = entV[n * 2];
          vh[0] = min(nv, 64);
          vh[1] = max(nv - 64, 0);
        }

        mbar_wait_bounded_inline(s_full + wg, (g >> 1) & 1, s_abort, 30 + wg, p.wait_limit);
        tc_fence_after();
        float sv[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, reinterpret_cast<uint32_t*>(sv) + c * 32);
        tmem_ld_wait();
        // S is in registers: the Q K^T of tile g+2 may overwrite the buffer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(s_free + wg);

        if (kRagged) {
          // the sequence ends inside this tile: columns past the end count as -inf
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            if (vh[h] > 0 && vh[h] < 64) {
#pragma unroll
              for (int e = 0; e < 64; ++e) sv[h * 64 + e] = e < vh[h] ? sv[h * 64 + e] : -INFINITY;
            }
          }
        }
        if (!frozen) {
          // Cauchy-Schwarz: no score of this tile exceeds |q| * max |k| * scale.  If that bound stays within
          // 2^kSkipMargin of the row's reference maximum (which only grows, so the value this thread saw last
          // will do) for all 32 rows of the warp, the reference need not move and the row-maximum pass is
          // skipped: the exponentials stay below 2^kSkipMargin, harmless in fp32 / bf16, and the result does
          // not depend on the reference.
          bool skip = false;
          if (!kRagged && p.knorm != nullptr) {
            float kn = entN[n * C::kEPT];
            if (C::kStacked) kn = fmaxf(kn, entN[min(n * 2 + 1, n_ent - 1)]);
            skip = __all_sync(0xffffffffu, q_bound * kn <= m_ref + kSkipMargin);
          }

          // one flat instruction stream per 64-key half; an absent half (not kept by this row's query block)
          // is skipped
          float mx = -INFINITY;
          if (!skip)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float* svh = sv + h * 64;
            if (vh[h] > 0) {
              float m0 = svh[0], m1 = svh[1], m2 = svh[2], m3 = svh[3];
#pragma unroll
              for (int e = 4; e < 64; e += 4) {
                m0 = fmaxf(m0, svh[e]);
                m1 = fmaxf(m1, svh[e + 1]);
                m2 = fmaxf(m2, svh[e + 2]);
                m3 = fmaxf(m3, svh[e + 3]);
              }
              mx = fmaxf(mx, fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)));
            }
          }
          mx *= p.scale_log2;

          // ---- my turn to look at / move the row's reference maximum (strictly in tile order) ----
          if (n > 0) named_bar_sync(bar_other, 64);
          const float m_cur = ref[row];
          const int told = n > 0 ? *frz : 0;  // the row group's other warp froze the reference in its last turn
          if (m_cur != m_ref) {  // the other thread moved it since my last tile
            l_run *= ex2(m_ref - m_cur);  // m_ref = -inf: l_run is 0 and stays 0
            m_ref = m_cur;
          }
          if (told) {
            frozen = true;
            __syncwarp();
            if (lane == 0) *frz = 0;  // nobody looks at it again before the next item's turns
          } else {
            // the first of the two warps to see the bound hold for the whole item says so, takes its last turn
            // without moving the reference (no score can make that necessary) and releases the other one more time
            if (n + 1 < n_tiles && p.knorm != nullptr &&
                __all_sync(0xffffffffu, q_bound * kn_item <= m_ref + kSkipMargin)) {
              frozen = true;
              if (lane == 0) *frz = 1;
            }
            const float m_new = fmaxf(m_ref, mx);
            const bool grow = !frozen && (m_new > m_ref + kGrowThreshold || (m_ref == -INFINITY && m_new > -INFINITY));
            if (!skip && __any_sync(0xffffffffu, grow)) {
              const float alpha = grow ? ex2(m_ref - m_new) : 1.0f;  // m_ref = -inf -> 0
              if (n > 0) {
                // every P V of the item issued so far must have landed in O before the row is rescaled; they
                // complete in order, so the one of tile g-1 suffices
                mbar_wait_bounded_inline(o_full + ((g - 1) & 3), ((g - 1) >> 2) & 1, s_abort, 38, p.wait_limit);
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < C::kAccCols / 16; ++c) {  // the row's accumulator, 16 columns at a time (rare: kept small)
                  uint32_t o[16];
                  tmem_ld16(tO + c * 16, o);
                  tmem_ld_wait();
#pragma unroll
                  for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                  tmem_st16(tO + c * 16, o);
                }
                if (C::kSum128) {  // the row sums live in columns of their own
                  uint32_t o[16];
                  tmem_ld16(tmem_base + C::kColL + lane_off, o);
                  tmem_ld_wait();
#pragma unroll
                  for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
                  tmem_st16(tmem_base + C::kColL + lane_off, o);
                }
                tmem_st_wait();
                tc_fence_before();
              }
              l_run *= alpha;
              if (grow) {
                m_ref = m_new;
                ref[row] = m_new;
              }
            }
            if (n + 1 < n_tiles) {
              asm volatile("bar.arrive %0, %1;" ::"r"(bar_mine), "r"(64) : "memory");
            }
          }
        }

        // exponentials of keys [64h, 64h+64) -> packed bf16 columns [32h, 32h+32) of the P buffer
        float2 lsum2 = make_float2(0.0f, 0.0f);
        const float neg_m = -m_ref;
        uint32_t pk[64];
        const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(neg_m, neg_m);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float* svh = sv + h * 64;
          uint32_t* pkh = pk + h * 32;
          if (vh[h] > 0) {  // then the row has a finite reference maximum
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float2 x = ffma2(make_float2(svh[2 * e], svh[2 * e + 1]), sc2, nm2);
              constexpr int kPoly = C::kOnes ? SPARSP_TUNE_POLY_D64 : SPARSP_TUNE_POLY;
              const float2 pp = (kPoly > 0 && (e % (kPoly > 0 ? kPoly : 1)) == 1)
                                    ? exp2_poly2(x)
                                    : make_float2(ex2(x.x), ex2(x.y));
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(pp.x, pp.y);
              pkh[e] = *reinterpret_cast<const uint32_t*>(&h2);
              if (!C::kSumMma) {
                // the row sum adds the bf16 values that P V multiplies, not the unrounded exponentials: with a
                // reference that is not the row's maximum the largest term is an arbitrary 2^x, and a sum of
                // unrounded terms would differ from the numerator's weights by up to 2^-9 of a peaked row
                asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
                    : "+f"(lsum2.x), "+f"(lsum2.y)
                    : "r"(pkh[e]));
              }
            }
            if (kRagged && vh[h] < 64) {
              // columns past the end of the sequence: exactly zero in P (the polynomial path returns
              // 2^-126 for them, which the row sum may keep)
#pragma unroll
              for (int e = 0; e < 32; ++e) pkh[e] = 2 * e + 1 < vh[h] ? pkh[e] : (2 * e < vh[h] ? (pkh[e] & 0xffffu) : 0u);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) pkh[e] = 0u;
          }
        }
        l_run += lsum2.x + lsum2.y;
        // my P buffer was last read by the P V of tile g-2; a single P buffer by that of tile g-1
        constexpr int kBack = C::kNumP == 2 ? 2 : 1;
        if (g >= kBack) {
          mbar_wait_bounded_inline(o_full + ((g - kBack) & 3), ((g - kBack) >> 2) & 1, s_abort, 34 + wg, p.wait_limit);
          tc_fence_after();
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st16(tP + c * 16, pk + c * 16);
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full + wg);
      };
      for (int n = (wg - g0) & 1; n < n_tiles; n += 2) {
        // the list builder puts the sequence's last block (the only one that can be ragged) into the last tile
        const bool ragged = item_ragged && n == n_tiles - 1;
        if (ragged) {
          do_tile(std::true_type{}, n);
        } else {
          do_tile(std::false_type{}, n);
        }
      }

      // ---- item epilogue: warpgroup x writes the column half x of every row -------------------------
      sStat[(buf * 2 + wg) * 128 + row] = make_float2(m_ref, l_run);
      named_bar_sync(9, 256);  // all of the item's decisions and P stores are done
      if (n_tiles > 0) {
        const int last = g0 + n_tiles - 1;
        mbar_wait_bounded_inline(o_full + (last & 3), (last >> 2) & 1, s_abort, 40, p.wait_limit);
        tc_fence_after();
      }
      {
        constexpr int HW = D / 2;
        const float m_fin = ref[row];
        const float2 st0 = sStat[(buf * 2) * 128 + row], st1 = sStat[(buf * 2 + 1) * 128 + row];
        // this reference buffer serves the item after next: no warp can be there before every warp has passed
        // the barrier above, and the item before this one (its last user) is finished for all of them
        sRef[((i + 2) % 3) * 128 + row] = -INFINITY;
        float l = (st0.y > 0.0f ? st0.y * ex2(st0.x - m_fin) : 0.0f) + (st1.y > 0.0f ? st1.y * ex2(st1.x - m_fin) : 0.0f);
        if (C::kSumMma) {  // the row sum is a tensor-memory column (CTA-uniform branch: the load is warp-collective)
          l = 0.0f;
          if (n_tiles > 0) {
            uint32_t sums[16];
            tmem_ld16(tmem_base + C::kColL + lane_off, sums);
            tmem_ld_wait();
            l = __uint_as_float(sums[0]);
          }
        }
        const float inv_l = l > 0.0f ? 1.0f / l : 0.0f;
        const int qb = C::kStacked ? s_blk[buf * 2 + rh] : s_blk[buf * 2];
        const int64_t tok = qb >= 0 ? (int64_t)qb * BLK + (C::kStacked ? (row & 63) : row) : p.N;
        __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT + wg * HW;
        uint32_t o[HW];
        if (n_tiles > 0) {  // CTA-uniform: tensor-memory loads are warp-collective
#pragma unroll
          for (int c = 0; c < HW / 32; ++c) tmem_ld32(tO + wg * HW + c * 32, o + c * 32);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int e = 0; e < HW; ++e) o[e] = 0u;
        }
        // the accumulator is in registers: the next item's first P V may overwrite it
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(o_drained);
          mbar_arrive(list_free + buf);
        }
        if (tok < p.N) {
          // a thread's row segment is 2 HW contiguous bytes but the rows of a warp are sT elements apart, so every
          // store instruction touches 32 lines: 32-byte stores (when the layout allows) halve their number
          const bool wide = ((reinterpret_cast<uintptr_t>(orow) | (uintptr_t)(p.sT * 2)) & 31) == 0;
#pragma unroll
          for (int v = 0; v < HW / 16; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(o[v * 16 + 2 * e]) * inv_l,
                                                              __uint_as_float(o[v * 16 + 2 * e + 1]) * inv_l);
              w[e] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            if (wide) {
              asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(orow + v * 16), "r"(w[0]),
                           "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                           : "memory");
            } else {
              *reinterpret_cast<uint4*>(orow + v * 16) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(orow + v * 16 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
            }
          }
        }
        if (p.lse && wg == 0 && tok < p.N)
          p.lse[(int64_t)bh * p.N + tok] = l > 0.0f ? (m_fin + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
      g0 += n_tiles;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
  if (tid == 0) report_abort(s_abort, p.status);
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
constexpr int kPairSample = 8;

// Sorts n keys (n a power of two, <= 1024) in shared memory into descending order; all kPairThreads threads call it.
__device__ __forceinline__ void sort_keys_descending(uint32_t* keys, int n) {
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < n; t += kPairThreads) {
        const int u = t ^ j;
        if (u > t) {
          const uint32_t a = keys[t], b = keys[u];
          if (((t & k) == 0) ? a < b : a > b) {
            keys[t] = b;
            keys[u] = a;
          }
        }
      }
      __syncthreads();
    }
  }
}

// Work items of one (batch, head) are handed out longest list first: the items still running when the queue
// runs dry are then the short ones, which matters when list lengths vary (threshold selection, unions of two
// stacked blocks).  Key = (list length << 10) | (1023 - index): equal lengths keep their index order.
__device__ __forceinline__ int next_pow2(int n) {
  int v = 1;
  while (v < n) v <<= 1;
  return v;
}

// block 128: order[x] = the query block that item x of this (batch, head) handles
__device__ __forceinline__ void order_body(const uint32_t* __restrict__ mask, int NB, int Wd,
                                           int32_t* __restrict__ pairs, int bh) {
  __shared__ uint32_t s_keys[1024];
  const int n2 = next_pow2(NB);
  const uint32_t* rows = mask + (int64_t)bh * NB * Wd;
  for (int i = threadIdx.x; i < n2; i += kPairThreads) {
    uint32_t key = 0;
    if (i < NB) {
      int len = 0;
      for (int w = 0; w < Wd; ++w) len += __popc(rows[(int64_t)i * Wd + w]);
      key = ((uint32_t)len << 10) | (uint32_t)(1023 - i);
    }
    s_keys[i] = key;
  }
  __syncthreads();
  sort_keys_descending(s_keys, n2);
  int32_t* out = pairs + (int64_t)bh * ((NB + 1) / 2) * 2;
  for (int x = threadIdx.x; x < NB; x += kPairThreads) out[x] = 1023 - (int)(s_keys[x] & 1023u);
}

__device__ __forceinline__ void pair_body(const uint32_t* __restrict__ mask, int NB, int Wd, int search,
                                          int32_t* __restrict__ pairs, int bh, unsigned char* smem_raw) {
  uint32_t* m = reinterpret_cast<uint32_t*>(smem_raw);  // [NB][Wd]
  __shared__ unsigned int s_best;                        // (score << 10) | (1023 - D): max = best score, smallest D
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
  // longest union first
  __shared__ uint32_t s_keys[512];
  const int n_pairs = (NB + 1) / 2, n2 = next_pow2(n_pairs);
  const uint32_t* rows = mask + (int64_t)bh * NB * Wd;
  __syncthreads();  // the pairs written above are visible to the whole block
  for (int c = threadIdx.x; c < n2; c += kPairThreads) {
    uint32_t key = 0;
    if (c < n_pairs) {
      const int a = out[2 * c], b = out[2 * c + 1];
      int len = 0;
      for (int w = 0; w < Wd; ++w)
        len += __popc(rows[(int64_t)a * Wd + w] | (b >= 0 ? rows[(int64_t)b * Wd + w] : 0u));
      key = ((uint32_t)len << 10) | (uint32_t)(1023 - c);
    }
    s_keys[c] = key;
  }
  __syncthreads();
  sort_keys_descending(s_keys, n2);
  int pa[2], pb[2];  // at most 512 pairs for 256 threads
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int x = threadIdx.x + r * kPairThreads;
    if (x < n_pairs) {
      const int c = 1023 - (int)(s_keys[x] & 1023u);
      pa[r] = out[2 * c];
      pb[r] = out[2 * c + 1];
    }
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int x = threadIdx.x + r * kPairThreads;
    if (x < n_pairs) {
      out[2 * x] = pa[r];
      out[2 * x + 1] = pb[r];
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
  // work item = one 128-row Q tile (a 128-token block, or a pair of 64-token blocks); one persistent CTA per SM
  AttnParams pp = p;
  pp.per_bh = BLK == 128 ? g.NB : (g.NB + 1) / 2;
  pp.n_items = g.B * g.H * pp.per_bh;
  int dev = 0, sms = 0;
  SPARSP_CUDA_OK(cudaGetDevice(&dev));
  SPARSP_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  dim3 grid((unsigned)std::min(pp.n_items, sms));
  kern<<<grid, kAttnThreads, smem, st>>>(tq, tk, tv, tp, pp);
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
  p.work_counter = p.status + kWorkCounterWord;
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

// Largest L2 norm of the keys of every KV block (times 1.001), fp32 [B*H][NB]: with the norm of a query row it
// bounds the scores of a tile.  One warp per (batch, head, block); d/8 lanes read one token (16 bytes each).
template <int D>
__device__ __forceinline__ void knorm_body(const __nv_bfloat16* __restrict__ K, int64_t sB, int64_t sH, int64_t sT,
                                           int H, int NB, int b, int64_t N, int64_t n_units, float* __restrict__ out,
                                           int64_t unit) {
  constexpr int LPT = D / 8;       // lanes per token
  constexpr int TPW = 32 / LPT;    // tokens per warp pass
  if (unit >= n_units) return;
  const int lane = threadIdx.x & 31;
  const int j = (int)(unit % NB);
  const int64_t bh = unit / NB;
  const int64_t batch = bh / H, head = bh % H;
  const __nv_bfloat16* base = K + batch * sB + head * sH;
  float best = 0.0f;
#pragma unroll 8
  for (int t0 = 0; t0 < b; t0 += TPW) {
    const int64_t tok = (int64_t)j * b + t0 + lane / LPT;
    float ss = 0.0f;
    if (tok < N && t0 + lane / LPT < b) {
      const uint4 v = *reinterpret_cast<const uint4*>(base + tok * sT + (lane % LPT) * 8);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
        ss = fmaf(lo, lo, ss);
        ss = fmaf(hi, hi, ss);
      }
    }
#pragma unroll
    for (int sft = 1; sft < LPT; sft <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, sft);
    best = fmaxf(best, ss);
  }
#pragma unroll
  for (int sft = LPT; sft < 32; sft <<= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, sft));
  if (lane == 0) out[unit] = sqrtf(best) * 1.001f;
}

// One launch for the two passes that precede the attention kernel and do not depend on each other: blocks
// [0, n_pair) fix the work items of one (batch, head) each (block 64: which query blocks are stacked; both block
// sizes: longest list first), the rest take the largest
// key norm of every KV block (times 1.001), fp32 [B*H][NB], one warp per block and d/8 lanes per token: with the
// norm of a query row it bounds the scores of a tile.
template <int D>
__global__ void __launch_bounds__(kPairThreads) attn_prep_kernel(const uint32_t* __restrict__ mask, int NB, int Wd,
                                                                 int32_t* __restrict__ pairs, int n_pair,
                                                                 const __nv_bfloat16* __restrict__ K, int64_t sB,
                                                                 int64_t sH, int64_t sT, int H, int b, int64_t N,
                                                                 int64_t n_units, float* __restrict__ knorm,
                                                                 int32_t* __restrict__ work_counter) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (blockIdx.x == 0 && threadIdx.x == 0) *work_counter = 0;  // the attention kernel's work queue
  if ((int)blockIdx.x < n_pair) {
    if (b == 64) pair_body(mask, NB, Wd, 1, pairs, (int)blockIdx.x, smem_raw);
    else order_body(mask, NB, Wd, pairs, (int)blockIdx.x);
  } else {
    const int64_t unit = ((int64_t)(blockIdx.x - n_pair) * kPairThreads + threadIdx.x) >> 5;
    knorm_body<D>(K, sB, sH, sT, H, NB, b, N, n_units, knorm, unit);
  }
}

int launch_attn(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                const uint32_t* mask, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                cudaStream_t st) {
  int32_t* pairs = (int32_t*)(ws + L.pairs);  // block 64: the two stacked blocks of each item; block 128: its block
  float* knorm = (float*)(ws + L.knorm);
  {
    const int n_pair = g.B * g.H;
    const size_t smem = g.b == 64 ? (size_t)g.NB * g.Wd * 4 : 0;
    const int64_t n_units = (int64_t)g.B * g.H * g.NB;
    const unsigned blocks = (unsigned)(n_pair + (n_units * 32 + kPairThreads - 1) / kPairThreads);
    const int64_t sB = s.stride_batch > 0 ? s.stride_batch : 0;
    if (g.d == 64) {
      SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)attn_prep_kernel<64>, (int)smem));
      attn_prep_kernel<64><<<blocks, kPairThreads, smem, st>>>(mask, g.NB, g.Wd, pairs, n_pair, (const __nv_bfloat16*)K, sB,
                                                             s.stride_head, s.stride_token, g.H, g.b, g.N, n_units, knorm,
                                                             (int32_t*)(ws + L.status) + kWorkCounterWord);
    } else {
      SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)attn_prep_kernel<128>, (int)smem));
      attn_prep_kernel<128><<<blocks, kPairThreads, smem, st>>>(mask, g.NB, g.Wd, pairs, n_pair, (const __nv_bfloat16*)K, sB,
                                                              s.stride_head, s.stride_token, g.H, g.b, g.N, n_units, knorm,
                                                             (int32_t*)(ws + L.status) + kWorkCounterWord);
    }
    count_launch();
  }
  AttnParams p;
  p.mask = mask;
  p.pairs = pairs;
  p.slot = nullptr;
  p.tile_base = nullptr;
  p.active_per_bh = nullptr;
  p.knorm = knorm;
  return launch_attn_common(s, g, Q, K, V, nullptr, 0, p, scale, O, lse, ws, L, st);
}

// ------------------------------------------------------------------------------------------------
// Packed-source attention for one consumer rank: pairs are formed among the consumer's own query
// blocks, and every kept KV block the consumer does not own is read from the consumer's packed buffer.
// ------------------------------------------------------------------------------------------------
// pairs of the consumer's blocks (ascending, neighbours in that order); the rest of the table is (-1, -1)
// Also leaves the number of work items per (batch, head) that hold any of the consumer's blocks.
__global__ void pair_rank_kernel(const int32_t* __restrict__ rank, int NB, int consumer, int stacked,
                                 int32_t* __restrict__ pairs, int32_t* __restrict__ active_per_bh) {
  const int n_pairs = (NB + 1) / 2;
  int32_t* out = pairs + (int64_t)blockIdx.x * n_pairs * 2;
  for (int i = threadIdx.x; i < 2 * n_pairs; i += blockDim.x) out[i] = -1;
  __syncthreads();
  if (threadIdx.x == 0) {
    int k = 0;
    for (int i = 0; i < NB; ++i)
      if (rank[i] == consumer) out[k++] = i;  // pair c = entries 2c and 2c+1
    if (blockIdx.x == 0) *active_per_bh = stacked ? (k + 1) / 2 : k;
  }
}

// slot[bh][j] = entry index of block j inside the consumer's packed buffer (pack order: producer ascending,
// head ascending, block ascending), for every block of the consumer's union that another rank owns.  One warp
// per (batch, producer, head).  The table must have been filled with -1.  Also writes tile_base[b].
__global__ void slot_kernel(const uint32_t* __restrict__ U, const int32_t* __restrict__ rank,
                            const int64_t* __restrict__ seg_off, const int64_t* __restrict__ seg_total,
                            const int64_t* __restrict__ dst_base, int B, int H, int NB, int Wd, int P, int consumer,
                            int64_t tile_bytes, int32_t* __restrict__ slot, int64_t* __restrict__ tile_base,
                            int32_t* __restrict__ work_counter) {
  if (blockIdx.x == 0 && threadIdx.x == 0) *work_counter = 0;  // the attention kernel's work queue
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
  int32_t* active = (int32_t*)(ws + L.status) + kWorkCounterWord + 1;
  pair_rank_kernel<<<g.B * g.H, 128, 0, st>>>(rank, g.NB, consumer, g.b == 64 ? 1 : 0, pairs, active);
  const int64_t n_warps = std::max<int64_t>((int64_t)g.B * P * g.H, g.B);
  slot_kernel<<<(unsigned)((n_warps * 32 + 255) / 256), 256, 0, st>>>(U, rank, seg_off, seg_total, dst_base, g.B, g.H,
                                                                    g.NB, g.Wd, P, consumer, tile_bytes, slot,
                                                                    tile_base, (int32_t*)(ws + L.status) + kWorkCounterWord);
  count_launch(2);
  AttnParams p;
  p.mask = mask;
  p.pairs = pairs;
  p.slot = slot;
  p.tile_base = tile_base;
  p.active_per_bh = active;
  p.knorm = nullptr;  // remote keys live in the packed buffer: every tile takes its row maximum
  return launch_attn_common(s, g, Q, K, V, packed, capacity, p, scale, O, lse, ws, L, st);
}

}  // namespace sparsp
