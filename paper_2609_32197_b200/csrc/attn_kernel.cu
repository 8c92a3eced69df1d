// Step 3: block-sparse FlashAttention forward on tcgen05 tensor cores.
//
// One CTA owns a 128-row query tile of one (batch, head): one query block when block = 128, two
// adjacent query blocks when block = 64 (the tile then walks the UNION of the two rows' kept KV
// blocks and each half masks out the blocks its own row does not keep, so the MMAs always run at
// the full M = 128 rate).  Per kept KV block j:
//     TMA   K_j, V_j -> shared memory (128-byte swizzle, 2-stage ring)
//     MMA   S = Q K_j^T            (tcgen05.mma, fp32 accumulator in tensor memory)
//     all   thread r reads row r of S from tensor memory, online softmax in fp32 (base-2
//           exponentials, lazy rescale of O only when a row's max grows by more than 2^8),
//           writes P (bf16) to shared memory in the swizzled K-major operand layout
//     MMA   O += P V_j             (V consumed in place as an MN-major operand)
// Epilogue: O / l -> bf16 -> global, optional log-sum-exp.
// Every mbarrier wait is bounded; a wait that runs out sets SPARSP_ERR_TIMEOUT in the status word.
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

constexpr int kAttnThreads = 128;
constexpr int kTileM = 128;
constexpr int kStages = 2;
constexpr int kTmemCols = 256;

template <int D, int BLK>
struct AttnSmem {
  static constexpr int kQBytes = kTileM * D * 2;
  static constexpr int kKVBytes = BLK * D * 2;
  static constexpr int kPBytes = kTileM * BLK * 2;
  static constexpr int kOffQ = 0;
  static constexpr int kOffK = kOffQ + kQBytes;
  static constexpr int kOffV = kOffK + kStages * kKVBytes;
  static constexpr int kOffP = kOffV + kStages * kKVBytes;
  static constexpr int kOffList = kOffP + kPBytes;            // uint16 [1024] kept KV blocks of the tile
  static constexpr int kOffFlags = kOffList + 2 * kMaxBlocks;  // uint8 [1024] which tile halves keep it
  static constexpr int kOffBars = kOffFlags + kMaxBlocks;      // mbarriers
  static constexpr int kOffMisc = kOffBars + 64;
  static constexpr int kTotal = kOffMisc + 64;
  static constexpr int kDynamic = kTotal + 1024;  // slack for the 1024-byte alignment of the base
};

template <int D, int BLK>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  using L = AttnSmem<D, BLK>;
  constexpr int QB = kTileM / BLK;  // query blocks per tile
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem + L::kOffQ;
  unsigned char* sK = smem + L::kOffK;
  unsigned char* sV = smem + L::kOffV;
  unsigned char* sP = smem + L::kOffP;
  uint16_t* sList = reinterpret_cast<uint16_t*>(smem + L::kOffList);
  uint8_t* sFlags = smem + L::kOffFlags;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kOffBars);
  uint64_t* bar_q = bars + 0;
  uint64_t* bar_full = bars + 1;  // [kStages]
  uint64_t* bar_s = bars + 3;
  uint64_t* bar_o = bars + 4;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + L::kOffMisc);
  int* s_ntiles = reinterpret_cast<int*>(smem + L::kOffMisc + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::kOffMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x;
  const int bh = blockIdx.y;
  const int batch = bh / p.H, head = bh % p.H;
  const int64_t q0 = (int64_t)tile * kTileM;
  const int my_qb = tid / BLK;  // which of the tile's query blocks this row belongs to
  const int i0 = tile * QB;

  // ---- setup ------------------------------------------------------------------------------
  if (tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    mbar_init(bar_q, 1);
    for (int s = 0; s < kStages; ++s) mbar_init(bar_full + s, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    mbar_init_fence();
    *s_abort = 0;
  }
  if (warp == 0) {
    // union of the tile's mask rows -> ascending list of KV blocks + per-block "kept by half q" flags
    const uint32_t* mrow = p.mask + ((int64_t)bh * p.NB + i0) * p.Wd;
    int running = 0;
    for (int w0 = 0; w0 < p.Wd; w0 += 32) {
      const int w = w0 + lane;
      uint32_t rowbits[QB];
      uint32_t u = 0;
#pragma unroll
      for (int q = 0; q < QB; ++q) {
        rowbits[q] = (w < p.Wd && i0 + q < p.NB) ? mrow[(int64_t)q * p.Wd + w] : 0u;
        u |= rowbits[q];
      }
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
        const int j = w * 32 + t;
        if (j < p.NB) {
          uint8_t f = 0;
#pragma unroll
          for (int q = 0; q < QB; ++q) f |= ((rowbits[q] >> t) & 1u) << q;
          sList[pos] = (uint16_t)j;
          sFlags[pos] = f;
          ++pos;
        }
      }
      running += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) *s_ntiles = running;
    tmem_alloc(s_tmem, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int n_tiles = *s_ntiles;
  const uint32_t tmem_S = tmem_base;        // columns [0, BLK)
  const uint32_t tmem_O = tmem_base + BLK;  // columns [BLK, BLK + D)
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;

  constexpr uint32_t kIdescQK = make_idesc_bf16(kTileM, BLK, 0, 0);
  constexpr uint32_t kIdescPV = make_idesc_bf16(kTileM, D, 0, 1);
  constexpr uint32_t kStageTx = 2u * L::kKVBytes;

  auto load_kv = [&](int n) {
    const int s = n % kStages;
    const int j = sList[n];
    mbar_expect_tx(bar_full + s, kStageTx);
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
      tma_load_4d(sK + s * L::kKVBytes + c * (BLK * 128), &tmK, bar_full + s, c * 64, j * BLK, head, batch);
      tma_load_4d(sV + s * L::kKVBytes + c * (BLK * 128), &tmV, bar_full + s, c * 64, j * BLK, head, batch);
    }
  };
  auto issue_qk = [&](int n) {
    const int s = n % kStages;
    const uint32_t a0 = smem_u32(sQ), b0 = smem_u32(sK + s * L::kKVBytes);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
      const uint64_t da = make_smem_desc(a0 + (kk / 4) * (kTileM * 128) + (kk % 4) * 32, 16, 1024);
      const uint64_t db = make_smem_desc(b0 + (kk / 4) * (BLK * 128) + (kk % 4) * 32, 16, 1024);
      mma_ss(tmem_S, da, db, kIdescQK, kk > 0 ? 1u : 0u);
    }
    mma_commit(bar_s);
  };
  auto issue_pv = [&](int n) {
    const int s = n % kStages;
    const uint32_t a0 = smem_u32(sP), b0 = smem_u32(sV + s * L::kKVBytes);
#pragma unroll
    for (int kk = 0; kk < BLK / 16; ++kk) {
      const uint64_t da = make_smem_desc(a0 + (kk / 4) * (kTileM * 128) + (kk % 4) * 32, 16, 1024);
      const uint64_t db = make_smem_desc(b0 + kk * 2048, BLK * 128, 1024);
      mma_ss(tmem_O, da, db, kIdescPV, (n > 0 || kk > 0) ? 1u : 0u);
    }
    mma_commit(bar_o);
  };

  float m_used = -INFINITY;  // running reference max (log2 domain) the row's exponentials use
  float l_run = 0.0f;

  if (n_tiles > 0) {
    if (tid == 0) {
      mbar_expect_tx(bar_q, L::kQBytes);
#pragma unroll
      for (int c = 0; c < D / 64; ++c)
        tma_load_4d(sQ + c * (kTileM * 128), &tmQ, bar_q, c * 64, (int)q0, head, batch);
      load_kv(0);
      mbar_wait_bounded(bar_q, 0, s_abort, p.status, 1, p.wait_limit);
    }

    for (int n = 0; n < n_tiles; ++n) {
      const int s = n % kStages;
      if (tid == 0) {
        mbar_wait_bounded(bar_full + s, (n / kStages) & 1, s_abort, p.status, 2, p.wait_limit);
        tc_fence_after();
        issue_qk(n);
        if (n > 0) mbar_wait_bounded(bar_o, (n - 1) & 1, s_abort, p.status, 3, p.wait_limit);
        if (n + 1 < n_tiles) load_kv(n + 1);  // stage (n+1)%2 was last read by P V of tile n-1
      }
      __syncwarp();
      mbar_wait_bounded(bar_s, n & 1, s_abort, p.status, 4, p.wait_limit);
      tc_fence_after();

      float sv[BLK];
#pragma unroll
      for (int c = 0; c < BLK / 32; ++c)
        tmem_ld32(tmem_S + lane_off + c * 32, reinterpret_cast<uint32_t*>(sv) + c * 32);
      tmem_ld_wait();

      const int j = sList[n];
      const bool kept = (sFlags[n] >> my_qb) & 1;  // warp-uniform (BLK >= 64 rows per half)
      const int ncols = (int)min((int64_t)BLK, p.N - (int64_t)j * BLK);
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < BLK; ++c) mx = fmaxf(mx, c < ncols ? sv[c] : -INFINITY);
      mx *= p.scale_log2;
      const float m_new = fmaxf(m_used, mx);
      const bool grow = kept && (m_new > m_used + 8.0f || m_used == -INFINITY);
      const bool any_grow = __any_sync(0xffffffffu, grow);

      // P V of the previous tile must be done before P is overwritten or O is rescaled
      if (n > 0) mbar_wait_bounded(bar_o, (n - 1) & 1, s_abort, p.status, 5, p.wait_limit);
      tc_fence_after();
      if (any_grow) {
        const float alpha = grow ? ex2(m_used - m_new) : 1.0f;  // m_used = -inf -> 0
        if (n > 0) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_O + lane_off + c * 32, o);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_O + lane_off + c * 32, o);
          }
          tmem_st_wait();
        }
        l_run *= alpha;
        if (grow) m_used = m_new;
      }

      float lsum = 0.0f;
      const int row = tid;
#pragma unroll
      for (int c8 = 0; c8 < BLK / 8; ++c8) {
        uint32_t packed[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = c8 * 8 + 2 * e;
          float p0 = 0.0f, p1 = 0.0f;
          if (kept) {
            if (c < ncols) p0 = ex2(fmaf(sv[c], p.scale_log2, -m_used));
            if (c + 1 < ncols) p1 = ex2(fmaf(sv[c + 1], p.scale_log2, -m_used));
          }
          lsum += p0 + p1;
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
          packed[e] = *reinterpret_cast<const uint32_t*>(&h2);
        }
        // K-major operand, 128-byte swizzle: 16-byte chunk cc of row r sits at chunk (cc ^ (r & 7))
        const int sub = c8 / 8, cc = c8 % 8;
        unsigned char* dst = sP + sub * (kTileM * 128) + row * 128 + ((cc ^ (row & 7)) * 16);
        *reinterpret_cast<uint4*>(dst) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
      }
      l_run += lsum;

      fence_proxy_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        issue_pv(n);
      }
    }
    mbar_wait_bounded(bar_o, (n_tiles - 1) & 1, s_abort, p.status, 6, p.wait_limit);
    tc_fence_after();
  }

  // ---- epilogue ---------------------------------------------------------------------------
  const int64_t tok = q0 + tid;
  const float inv_l = l_run > 0.0f ? 1.0f / l_run : 0.0f;
  __nv_bfloat16* orow = p.O + (int64_t)batch * p.sB + (int64_t)head * p.sH + tok * p.sT;
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
    uint32_t o[32];
    if (n_tiles > 0) {
      tmem_ld32(tmem_O + lane_off + c * 32, o);
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

  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, kTmemCols);
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
  if ((rc = make_tmap(&tq, Q, s, g, kTileM)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tk, K, s, g, BLK)) != SPARSP_OK) return rc;
  if ((rc = make_tmap(&tv, V, s, g, BLK)) != SPARSP_OK) return rc;
  auto kern = attn_fwd_kernel<D, BLK>;
  const int smem = AttnSmem<D, BLK>::kDynamic;
  SPARSP_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  dim3 grid((unsigned)((g.N + kTileM - 1) / kTileM), (unsigned)(g.B * g.H));
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
  p.wait_limit = 2000000000LL;  // ~1 s of SM clocks
  if (g.d == 64 && g.b == 64) return launch_attn_t<64, 64>(s, g, Q, K, V, p, st);
  if (g.d == 64 && g.b == 128) return launch_attn_t<64, 128>(s, g, Q, K, V, p, st);
  if (g.d == 128 && g.b == 64) return launch_attn_t<128, 64>(s, g, Q, K, V, p, st);
  return launch_attn_t<128, 128>(s, g, Q, K, V, p, st);
}

}  // namespace sparsp
