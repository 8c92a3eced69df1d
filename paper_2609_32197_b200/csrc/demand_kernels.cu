// Step 2: per-rank per-head unions of required KV blocks, demand counts, exchange volume,
// pack-order offsets, the entry table, and the gather of K/V tiles into per-consumer buffers.
// Everything before the gather is small integer work on bit words; the gather is the HBM-bound part.
#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace sparsp {

// One CTA per (batch, head) computes, for that head,
//   own[p][w]     : bit j set iff rank_of_block[j] == p                      (CTA 0 also writes it out)
//   U[b][r][h][w] = OR over the query blocks i of rank r of M[b][h][i][w]
//   cnt[b][r][p][h] = popcount(U[b][r][h] & own[p])
// The head's mask rows are read once, coalesced, and OR-ed into a [P][Wd] table in shared memory (at most
// 64 ranks x 32 words = 8 KiB; OR does not depend on the order, so the bits are well defined); the ownership
// words are rebuilt per CTA from the rank table (a few thousand compares) rather than fetched from an earlier
// launch.  A rank value outside [0, P) is ignored.
constexpr int kUnionThreads = 1024;
static_assert(2 * kMaxRanks * (kMaxBlocks / 32) * 4 <= 48 * 1024, "union and ownership tables must fit shared memory");

__global__ void __launch_bounds__(kUnionThreads) union_count_kernel(const uint32_t* __restrict__ mask,
                                                                    const int32_t* __restrict__ rank, int H, int NB,
                                                                    int Wd, int P, uint32_t* __restrict__ own,
                                                                    uint32_t* __restrict__ U,
                                                                    int32_t* __restrict__ cnt) {
  extern __shared__ uint32_t tab[];
  uint32_t* u_s = tab;             // [P][Wd]
  uint32_t* own_s = tab + P * Wd;  // [P][Wd]
  const int bh = blockIdx.x, bb = bh / H, h = bh % H;
  for (int idx = threadIdx.x; idx < P * Wd; idx += kUnionThreads) {
    const int p = idx / Wd, w = idx - p * Wd;
    uint32_t bits = 0;
    for (int t = 0; t < 32; ++t) {
      const int j = w * 32 + t;
      if (j < NB && rank[j] == p) bits |= 1u << t;
    }
    own_s[idx] = bits;
    u_s[idx] = 0u;
    if (bh == 0) own[idx] = bits;
  }
  __syncthreads();
  const uint32_t* m = mask + (int64_t)bh * NB * Wd;
  for (int idx = threadIdx.x; idx < NB * Wd; idx += kUnionThreads) {
    const int i = idx / Wd, w = idx - i * Wd;
    const uint32_t v = m[idx];
    const int r = rank[i];
    if (v != 0u && (unsigned)r < (unsigned)P) atomicOr(&u_s[r * Wd + w], v);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < P * Wd; idx += kUnionThreads) {
    const int r = idx / Wd, w = idx - r * Wd;
    U[((int64_t)(bb * P + r) * H + h) * Wd + w] = u_s[idx];
  }
  for (int idx = threadIdx.x; idx < P * P; idx += kUnionThreads) {
    const int r = idx / P, p = idx - r * P;
    int c = 0;
    for (int w = 0; w < Wd; ++w) c += __popc(u_s[r * Wd + w] & own_s[p * Wd + w]);
    cnt[((int64_t)(bb * P + r) * P + p) * H + h] = c;
  }
}

static void launch_union_count(const uint32_t* mask, const int32_t* rank, const Geometry& g, int P, uint32_t* own,
                               uint32_t* U, int32_t* cnt, cudaStream_t st) {
  union_count_kernel<<<g.B * g.H, kUnionThreads, (size_t)2 * P * g.Wd * 4, st>>>(mask, rank, g.H, g.NB, g.Wd, P, own,
                                                                                 U, cnt);
}

// One thread per (b, r): exclusive scan of cnt over (p, h) in pack order, totals and volume; then
// thread 0 turns the totals into table bases.  Sizes are tiny (P*H values per thread).
__global__ void scan_kernel(const int32_t* __restrict__ cnt, int B, int H, int P, int include_local,
                            int64_t entry_bytes, int64_t* __restrict__ seg_off,
                            int64_t* __restrict__ seg_total, int64_t* __restrict__ volume,
                            int64_t* __restrict__ ent_base, int64_t* __restrict__ n_entries) {
  const int idx = threadIdx.x;
  if (idx < B * P) {
    const int r = idx % P;
    int64_t cursor = 0, remote = 0;
    for (int p = 0; p < P; ++p) {
      for (int h = 0; h < H; ++h) {
        const int64_t o = ((int64_t)idx * P + p) * H + h;
        const int c = cnt[o];
        seg_off[o] = cursor;
        if (p != r) remote += c;
        if (p != r || include_local) cursor += c;
      }
    }
    seg_total[idx] = cursor;
    volume[idx] = entry_bytes * remote;
  }
  __syncthreads();
  if (idx == 0) {
    int64_t base = 0;
    for (int t = 0; t < B * P; ++t) {
      ent_base[t] = base;
      base += seg_total[t];
    }
    *n_entries = base;
  }
}

// Entry table: one warp per (b, r, p, h) segment enumerates the set bits of U & own[p] in ascending
// order and writes entry records at table index ent_base[b,r] + seg_off + t.
__global__ void entries_kernel(const uint32_t* __restrict__ U, const uint32_t* __restrict__ own, int B,
                               int H, int Wd, int P, int include_local, int64_t entry_bytes,
                               const int64_t* __restrict__ seg_off, const int64_t* __restrict__ ent_base,
                               const int64_t* __restrict__ dst_base, int64_t capacity,
                               PackEntry* __restrict__ entries, int32_t* __restrict__ status) {
  const int64_t seg = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t n_seg = (int64_t)B * P * P * H;
  if (seg >= n_seg) return;
  const int h = (int)(seg % H);
  const int p = (int)((seg / H) % P);
  const int r = (int)((seg / ((int64_t)H * P)) % P);
  const int bb = (int)(seg / ((int64_t)H * P * P));
  if (p == r && !include_local) return;
  const uint32_t* u = U + ((int64_t)(bb * P + r) * H + h) * Wd;
  const uint32_t* o = own + (int64_t)p * Wd;
  const int64_t br = (int64_t)bb * P + r;
  const int64_t first = seg_off[seg];
  const int64_t base_byte = dst_base ? dst_base[br] : ent_base[br] * entry_bytes;
  PackEntry* out = entries + ent_base[br] + first;
  int running = 0;
  for (int w0 = 0; w0 < Wd; w0 += 32) {
    const int w = w0 + lane;
    uint32_t bits = w < Wd ? (u[w] & o[w]) : 0u;
    const int mine = __popc(bits);
    int incl = mine;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, s);
      if (lane >= s) incl += v;
    }
    int pos = running + incl - mine;
    while (bits) {
      const int t = __ffs(bits) - 1;
      bits &= bits - 1;
      PackEntry e;
      e.dst_byte = base_byte + (first + pos) * entry_bytes;
      e.bh = bb * H + h;
      e.j = w * 32 + t;
      if (capacity >= 0 && e.dst_byte + entry_bytes > capacity) {
        e.j = -1;  // would overflow: skipped by the gather
        atomicExch(status, SPARSP_ERR_CAPACITY);
      }
      out[pos] = e;
      ++pos;
    }
    running += __shfl_sync(0xffffffffu, incl, 31);
  }
}

int launch_demand(const Geometry& g, const uint32_t* mask, const int32_t* rank_of_block, int P,
                  int flags, uint32_t* U, int32_t* cnt, int64_t* seg_off, int64_t* seg_total,
                  int64_t* volume, const int64_t* dst_base, int64_t capacity, char* ws,
                  const WsLayout& L, cudaStream_t st) {
  uint32_t* own = (uint32_t*)(ws + L.own);
  int64_t* ent_base = (int64_t*)(ws + L.ent_base);
  int64_t* n_entries = (int64_t*)(ws + L.n_entries);
  PackEntry* entries = (PackEntry*)(ws + L.entries);
  int32_t* status = (int32_t*)(ws + L.status);
  const int include_local = (flags & SPARSP_INCLUDE_LOCAL) ? 1 : 0;
  const int64_t entry_bytes = 2LL * g.b * g.d * 2;
  if (g.B * P > 1024) {
    set_error("batch * n_ranks = %d exceeds 1024", g.B * P);
    return SPARSP_ERR_UNSUPPORTED;
  }
  launch_union_count(mask, rank_of_block, g, P, own, U, cnt, st);
  const int64_t n_c = (int64_t)g.B * P * P * g.H;
  scan_kernel<<<1, 1024, 0, st>>>(cnt, g.B, g.H, P, include_local, entry_bytes, seg_off, seg_total,
                                  volume, ent_base, n_entries);
  entries_kernel<<<(int)((n_c * 32 + 255) / 256), 256, 0, st>>>(U, own, g.B, g.H, g.Wd, P,
                                                               include_local, entry_bytes, seg_off,
                                                               ent_base, dst_base, capacity, entries,
                                                               status);
  count_launch(3);
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

// ------------------------------------------------------------------------------------------------
// Gather.  All K and V tiles of all entries form one flat sequence of 16-byte vectors (tile t of the
// sequence = K or V tile of entry t/2).  Persistent CTAs take chunks of kPackThreads * kPackUnroll
// consecutive vectors, so the bytes in flight per SM do not depend on the tile size (8..32 KiB); loads
// and stores are fully coalesced when a tile's rows are adjacent in memory.  Rows at or beyond N are
// written as zeros.
// ------------------------------------------------------------------------------------------------
constexpr int kPackThreads = 256;
constexpr int kPackUnroll = 8;

template <int D>
__global__ void __launch_bounds__(kPackThreads) pack_kernel(
    const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
    const PackEntry* __restrict__ entries, const int64_t* __restrict__ n_entries_p, int H, int b,
    int64_t N, int64_t sB, int64_t sH, int64_t sT, unsigned char* __restrict__ packed) {
  constexpr int VPR = D / 8;                // 16-byte vectors per row
  const int vpt = b * VPR;                  // vectors per tile (a power of two)
  const int vpt_shift = 31 - __clz(vpt);
  const int64_t n_vec = 2 * (*n_entries_p) * (int64_t)vpt;
  constexpr int64_t kChunk = (int64_t)kPackThreads * kPackUnroll;
  for (int64_t base = (int64_t)blockIdx.x * kChunk; base < n_vec; base += (int64_t)gridDim.x * kChunk) {
    uint4 buf[kPackUnroll];
    uint4* dst[kPackUnroll];
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u) {
      const int64_t g = base + u * kPackThreads + threadIdx.x;
      buf[u] = make_uint4(0u, 0u, 0u, 0u);
      dst[u] = nullptr;
      if (g < n_vec) {
        const int64_t tile = g >> vpt_shift;
        const int v = (int)(g & (vpt - 1));
        const int4 raw = __ldg(reinterpret_cast<const int4*>(entries) + (tile >> 1));
        PackEntry e;
        e.dst_byte = (int64_t)(((uint64_t)(uint32_t)raw.y << 32) | (uint32_t)raw.x);
        e.bh = raw.z;
        e.j = raw.w;
        if (e.j >= 0) {
          const int which = (int)(tile & 1);
          const int row = v / VPR, col = v % VPR;
          const int64_t tok = (int64_t)e.j * b + row;
          dst[u] = reinterpret_cast<uint4*>(packed + e.dst_byte + (int64_t)which * vpt * 16) + v;
          if (tok < N) {
            const int64_t batch = e.bh / H, head = e.bh % H;
            const __nv_bfloat16* src = (which ? V : K) + batch * sB + head * sH + tok * sT;
            buf[u] = __ldcs(reinterpret_cast<const uint4*>(src) + col);
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kPackUnroll; ++u)
      if (dst[u]) __stcs(dst[u], buf[u]);
  }
}

// Per-tile variant for large tiles (>= 16 KiB): one K or V tile per CTA step, the entry record is read
// once per tile.  Measured faster than the flat variant when a tile alone fills a CTA's loads in flight.
template <int D>
__global__ void __launch_bounds__(kPackThreads) pack_tile_kernel(
    const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
    const PackEntry* __restrict__ entries, const int64_t* __restrict__ n_entries_p, int H, int b,
    int64_t N, int64_t sB, int64_t sH, int64_t sT, unsigned char* __restrict__ packed) {
  constexpr int VPR = D / 8;  // 16-byte vectors per row
  const int64_t n_items = 2 * (*n_entries_p);
  const int vec_per_tile = b * VPR;
  const int64_t tile_bytes = (int64_t)b * D * 2;
  for (int64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const PackEntry e = entries[item >> 1];
    if (e.j < 0) continue;
    const int which = (int)(item & 1);
    const int64_t batch = e.bh / H, head = e.bh % H;
    const int64_t tok0 = (int64_t)e.j * b;
    const int n_valid = (int)min((int64_t)b, N - tok0);
    const __nv_bfloat16* src = (which ? V : K) + batch * sB + head * sH + tok0 * sT;
    uint4* dst = reinterpret_cast<uint4*>(packed + e.dst_byte + which * tile_bytes);
    for (int v0 = threadIdx.x; v0 < vec_per_tile; v0 += kPackThreads * kPackUnroll) {
      uint4 buf[kPackUnroll];
#pragma unroll
      for (int u = 0; u < kPackUnroll; ++u) {
        const int v = v0 + u * kPackThreads;
        const int row = v / VPR, col = v % VPR;
        buf[u] = make_uint4(0u, 0u, 0u, 0u);
        if (v < vec_per_tile && row < n_valid)
          buf[u] = __ldcs(reinterpret_cast<const uint4*>(src + (int64_t)row * sT) + col);
      }
#pragma unroll
      for (int u = 0; u < kPackUnroll; ++u) {
        const int v = v0 + u * kPackThreads;
        if (v < vec_per_tile) __stcs(dst + v, buf[u]);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Bulk-copy gather for layouts in which a tile's rows are adjacent in memory ([B][H][N][d]): one warp
// per CTA streams whole tiles global -> shared -> global with the TMA bulk engine (cp.async.bulk), a
// ring of n_stages tile buffers per warp (1, 2 or 4 warps per CTA for 32, 16, 8 KiB tiles, so that the
// bytes in flight per SM do not depend on the tile size), loads running n_stages-1 tiles ahead of the
// stores.
// No thread touches the data, except to zero the missing rows of a ragged last block.
// ------------------------------------------------------------------------------------------------
constexpr int kBulkMaxStages = 8;
#ifndef SPARSP_TUNE_PACK_BULK
#define SPARSP_TUNE_PACK_BULK 1
#endif
constexpr bool kPackUseBulk = SPARSP_TUNE_PACK_BULK != 0;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   ptx::smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
               "r"(ptx::smem_u32(smem_src)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <int D>
__global__ void __launch_bounds__(128) pack_bulk_kernel(const __nv_bfloat16* __restrict__ K,
                                                       const __nv_bfloat16* __restrict__ V,
                                                       const PackEntry* __restrict__ entries,
                                                       const int64_t* __restrict__ n_entries_p, int H, int b,
                                                       int64_t N, int64_t sB, int64_t sH, int n_stages,
                                                       unsigned char* __restrict__ packed,
                                                       int32_t* __restrict__ status) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ uint64_t full_all[4 * kBulkMaxStages];
  __shared__ int s_abort;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_warps = blockDim.x >> 5;
  const uint32_t tile_bytes = (uint32_t)b * D * 2;
  uint64_t* full = full_all + warp * kBulkMaxStages;
  unsigned char* ring = smem_raw + (size_t)warp * n_stages * tile_bytes;  // this warp's buffers
  const int64_t unit = (int64_t)blockIdx.x * n_warps + warp, n_units = (int64_t)gridDim.x * n_warps;
  const int64_t n_items = 2 * (*n_entries_p);
  const int64_t n_local = n_items > unit ? (n_items - unit + n_units - 1) / n_units : 0;
  if (threadIdx.x == 0) s_abort = 0;
  if (lane == 0) {
    for (int st = 0; st < n_stages; ++st) ptx::mbar_init(full + st, 1);
    ptx::mbar_init_fence();
  }
  __syncthreads();

  // source address and valid byte count of local item q (0 valid bytes = entry skipped for capacity)
  auto locate = [&](int64_t q, const unsigned char*& src, unsigned char*& dst, uint32_t& valid) {
    const int64_t item = unit + q * n_units;
    const int4 raw = __ldg(reinterpret_cast<const int4*>(entries) + (item >> 1));
    const int64_t dst_byte = (int64_t)(((uint64_t)(uint32_t)raw.y << 32) | (uint32_t)raw.x);
    const int bh = raw.z, j = raw.w;
    const int which = (int)(item & 1);
    if (j < 0) {
      valid = 0;
      src = nullptr;
      dst = nullptr;
      return;
    }
    const int64_t batch = bh / H, head = bh % H, tok0 = (int64_t)j * b;
    const int64_t n_valid = min((int64_t)b, N - tok0);
    valid = (uint32_t)(n_valid * D * 2);
    src = reinterpret_cast<const unsigned char*>((which ? V : K) + batch * sB + head * sH + tok0 * D);
    dst = packed + dst_byte + (int64_t)which * tile_bytes;
  };
  auto issue_load = [&](int64_t q) {
    const unsigned char* src;
    unsigned char* dst;
    uint32_t valid;
    locate(q, src, dst, valid);
    uint64_t* bar = full + q % n_stages;
    if (valid == 0) {
      ptx::mbar_arrive(bar);  // nothing to move: complete the phase directly
    } else {
      ptx::mbar_expect_tx(bar, valid);
      bulk_load(ring + (size_t)(q % n_stages) * tile_bytes, src, valid, bar);
    }
  };

  if (lane == 0)
    for (int64_t q = 0; q < n_stages - 1 && q < n_local; ++q) issue_load(q);
  for (int64_t q = 0; q < n_local; ++q) {
    const unsigned char* src;
    unsigned char* dst;
    uint32_t valid;
    locate(q, src, dst, valid);  // same values in every lane
    unsigned char* buf = ring + (size_t)(q % n_stages) * tile_bytes;
    ptx::mbar_wait_bounded(full + q % n_stages, (uint32_t)((q / n_stages) & 1), &s_abort, status, 50, 200000000LL);
    if (valid != 0 && valid < tile_bytes) {  // ragged last block: zero the missing rows
      for (uint32_t o = valid + lane * 16; o < tile_bytes; o += 32 * 16)
        *reinterpret_cast<uint4*>(buf + o) = make_uint4(0u, 0u, 0u, 0u);
      ptx::fence_proxy_async_smem();
    }
    __syncwarp();
    if (lane == 0) {
      if (valid != 0) bulk_store(dst, buf, tile_bytes);
      // the buffer of item q-1 may be refilled once its store has read it
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      if (q + n_stages - 1 < n_local) issue_load(q + n_stages - 1);
    }
    __syncwarp();
  }
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

int launch_pack(const sparsp_shape& s, const Geometry& g, const void* K, const void* V, void* packed,
                int64_t capacity, int P, char* ws, const WsLayout& L, cudaStream_t st) {
  (void)capacity;
  (void)P;
  const PackEntry* entries = (const PackEntry*)(ws + L.entries);
  const int64_t* n_entries = (const int64_t*)(ws + L.n_entries);
  int dev = 0, sms = 148;
  SPARSP_CUDA_OK(cudaGetDevice(&dev));
  SPARSP_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int grid = sms * 8;
  auto k = (const __nv_bfloat16*)K;
  auto v = (const __nv_bfloat16*)V;
  const bool small_tiles = g.b * g.d / 8 < 1024;  // 8 KiB tiles: several tiles per CTA step
  unsigned char* out = (unsigned char*)packed;
  const bool rows_adjacent = s.stride_token == g.d;
  if (rows_adjacent && kPackUseBulk) {
    // TMA bulk path: a ring of whole-tile buffers per CTA, one CTA per SM
    const int tile_bytes = g.b * g.d * 2;
    const int n_warps = std::max(1, std::min(4, (32 * 1024) / tile_bytes));
    const int n_stages = 5;  // per warp: 160 KiB of tile buffers per CTA whatever the tile size
    const int smem = n_warps * n_stages * tile_bytes;
    int32_t* status = (int32_t*)(ws + L.status);
    if (g.d == 64) {
      SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)pack_bulk_kernel<64>, smem));
      pack_bulk_kernel<64><<<sms, 32 * n_warps, smem, st>>>(k, v, entries, n_entries, g.H, g.b, g.N,
                                                            s.stride_batch, s.stride_head, n_stages, out, status);
    } else {
      SPARSP_CUDA_OK(ensure_dynamic_smem((const void*)pack_bulk_kernel<128>, smem));
      pack_bulk_kernel<128><<<sms, 32 * n_warps, smem, st>>>(k, v, entries, n_entries, g.H, g.b, g.N,
                                                             s.stride_batch, s.stride_head, n_stages, out, status);
    }
  } else if (small_tiles) {
    if (g.d == 64)
      pack_kernel<64><<<grid, kPackThreads, 0, st>>>(k, v, entries, n_entries, g.H, g.b, g.N, s.stride_batch,
                                                     s.stride_head, s.stride_token, out);
    else
      pack_kernel<128><<<grid, kPackThreads, 0, st>>>(k, v, entries, n_entries, g.H, g.b, g.N, s.stride_batch,
                                                      s.stride_head, s.stride_token, out);
  } else {
    if (g.d == 64)
      pack_tile_kernel<64><<<grid, kPackThreads, 0, st>>>(k, v, entries, n_entries, g.H, g.b, g.N,
                                                          s.stride_batch, s.stride_head, s.stride_token, out);
    else
      pack_tile_kernel<128><<<grid, kPackThreads, 0, st>>>(k, v, entries, n_entries, g.H, g.b, g.N,
                                                           s.stride_batch, s.stride_head, s.stride_token, out);
  }
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}

// ------------------------------------------------------------------------------------------------
// Pack of ONE (consumer, producer) segment (Section 6.1: the producer packs the payload of one consumer into
// the slot designated for that pair).  The entry table holds that segment alone, with destinations relative
// to the start of the slot: entry (h, j) sits where it sits inside the consumer's buffer, minus the segment's
// first entry, so that consumer and producer derive the same byte ranges from the demand counts.
// One warp per head enumerates U[consumer][h] & own[producer] in ascending block order.
// ------------------------------------------------------------------------------------------------
__global__ void segment_entries_kernel(const uint32_t* __restrict__ U, const int32_t* __restrict__ rank, int H, int NB,
                                       int Wd, int P, int consumer, int producer,
                                       const int64_t* __restrict__ seg_off, const int32_t* __restrict__ cnt,
                                       int64_t entry_bytes, int64_t capacity, PackEntry* __restrict__ entries,
                                       int64_t* __restrict__ n_entries, int32_t* __restrict__ status) {
  const int h = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  const int lane = threadIdx.x & 31;
  if (h >= H) return;
  const int64_t seg0 = ((int64_t)consumer * P + producer) * H;  // batch item 0
  const int64_t first_of_segment = seg_off[seg0];
  if (h == 0 && lane == 0) *n_entries = seg_off[seg0 + H - 1] + cnt[seg0 + H - 1] - first_of_segment;
  const uint32_t* u = U + ((int64_t)consumer * H + h) * Wd;
  const int64_t first = seg_off[seg0 + h] - first_of_segment;
  int running = 0;
  for (int w0 = 0; w0 < Wd; w0 += 32) {
    const int w = w0 + lane;
    uint32_t bits = 0;
    if (w < Wd) {
      uint32_t own = 0;
      for (int t = 0; t < 32; ++t) {
        const int j = w * 32 + t;
        if (j < NB && rank[j] == producer) own |= 1u << t;
      }
      bits = u[w] & own;
    }
    const int mine = __popc(bits);
    int incl = mine;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, s);
      if (lane >= s) incl += v;
    }
    int pos = running + incl - mine;
    while (bits) {
      const int t = __ffs(bits) - 1;
      bits &= bits - 1;
      PackEntry e;
      e.dst_byte = (first + pos) * entry_bytes;
      e.bh = h;
      e.j = w * 32 + t;
      if (e.dst_byte + entry_bytes > capacity) {
        e.j = -1;  // would not fit the slot: skipped by the gather
        atomicExch(status, SPARSP_ERR_CAPACITY);
      }
      entries[first + pos] = e;
      ++pos;
    }
    running += __shfl_sync(0xffffffffu, incl, 31);
  }
}

int launch_pack_segment(const sparsp_shape& s, const Geometry& g, const uint32_t* U, const int32_t* rank, int P,
                        int consumer, int producer, const int64_t* seg_off, const int32_t* cnt, const void* K,
                        const void* V, void* dst, int64_t capacity, char* ws, const WsLayout& L, cudaStream_t st) {
  PackEntry* entries = (PackEntry*)(ws + L.entries);
  int64_t* n_entries = (int64_t*)(ws + L.n_entries);
  int32_t* status = (int32_t*)(ws + L.status);
  const int64_t entry_bytes = 2LL * g.b * g.d * 2;
  segment_entries_kernel<<<(g.H * 32 + 255) / 256, 256, 0, st>>>(U, rank, g.H, g.NB, g.Wd, P, consumer, producer, seg_off,
                                                                cnt, entry_bytes, capacity, entries, n_entries, status);
  count_launch();
  SPARSP_CUDA_OK(cudaGetLastError());
  return launch_pack(s, g, K, V, dst, capacity, P, ws, L, st);
}

// ------------------------------------------------------------------------------------------------
// Allocation-free planning call.  Its scratch (the per-rank ownership bit words and the per-consumer
// table bases) lives in one file-scope device array instead of a caller-provided workspace, so a
// caller that cannot allocate device memory at all can still obtain unions, counts, offsets and
// volumes.  Every GPU that loads the library carries the array (kPlanScratchBytes) until exit.
// ------------------------------------------------------------------------------------------------
constexpr int kPlanMaxRanks = 64;         // n_ranks limit of the allocation-free call
constexpr int kPlanMaxBatchRanks = 1024;  // batch * n_ranks limit
constexpr int kPlanOwnWords = kPlanMaxRanks * (kMaxBlocks / 32);
constexpr size_t kPlanScratchBytes = kPlanOwnWords * sizeof(uint32_t) + (kPlanMaxBatchRanks + 1) * sizeof(int64_t);

static __device__ __align__(256) unsigned char g_plan_scratch[kPlanScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_plan_mutex;
static void* g_plan_scratch_addr[kMaxDevices] = {nullptr};

// Device address of g_plan_scratch on the current device.  In host code the array's name is only a
// handle, so the address is resolved once per device with that device current.
static int plan_scratch_address(void** out) {
  int dev = 0;
  SPARSP_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    set_error("device ordinal %d outside 0..%d", dev, kMaxDevices - 1);
    return SPARSP_ERR_UNSUPPORTED;
  }
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  if (!g_plan_scratch_addr[dev]) {
    void* ptr = nullptr;
    SPARSP_CUDA_OK(cudaGetSymbolAddress(&ptr, g_plan_scratch));
    g_plan_scratch_addr[dev] = ptr;
  }
  *out = g_plan_scratch_addr[dev];
  return SPARSP_OK;
}

}  // namespace sparsp

using namespace sparsp;

extern "C" SPARSP_API int sparsp_demand_plan_noalloc(const sparsp_shape* shape, const uint32_t* mask,
                                                     const int32_t* rank_of_block, int32_t n_ranks,
                                                     int32_t flags, uint32_t* union_mask, int32_t* cnt,
                                                     int64_t* seg_offset, int64_t* seg_total,
                                                     int64_t* volume_bytes, void* stream) {
  Geometry g;
  int rc = make_geometry(shape, &g);
  if (rc != SPARSP_OK) return rc;
  if (n_ranks < 1 || n_ranks > kPlanMaxRanks || (int64_t)g.B * n_ranks > kPlanMaxBatchRanks) {
    set_error("sparsp_demand_plan_noalloc supports n_ranks <= %d and batch * n_ranks <= %d (got %d, %lld)",
              kPlanMaxRanks, kPlanMaxBatchRanks, n_ranks, (long long)g.B * n_ranks);
    return SPARSP_ERR_CAPACITY;
  }
  if (flags & ~SPARSP_INCLUDE_LOCAL) {
    set_error("sparsp_demand_plan_noalloc accepts only SPARSP_INCLUDE_LOCAL (got 0x%x)", flags);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (!mask || !rank_of_block || !union_mask || !cnt || !seg_offset || !seg_total || !volume_bytes) {
    set_error("sparsp_demand_plan_noalloc: NULL argument");
    return SPARSP_ERR_INVALID_ARG;
  }
  if ((uintptr_t)seg_offset % 8 || (uintptr_t)seg_total % 8 || (uintptr_t)volume_bytes % 8 ||
      (uintptr_t)mask % 4 || (uintptr_t)union_mask % 4 || (uintptr_t)cnt % 4 || (uintptr_t)rank_of_block % 4) {
    set_error("sparsp_demand_plan_noalloc: misaligned argument");
    return SPARSP_ERR_INVALID_ARG;
  }
  void* scratch = nullptr;
  if ((rc = plan_scratch_address(&scratch)) != SPARSP_OK) return rc;
  uint32_t* own = (uint32_t*)scratch;                                       // [P][Wd], fully rewritten
  int64_t* ent_base = (int64_t*)((char*)scratch + kPlanOwnWords * sizeof(uint32_t));  // [B*P] + total
  int64_t* n_entries = ent_base + kPlanMaxBatchRanks;
  const int P = n_ranks;
  const int include_local = (flags & SPARSP_INCLUDE_LOCAL) ? 1 : 0;
  const int64_t entry_bytes = 2LL * g.b * g.d * 2;
  cudaStream_t st = (cudaStream_t)stream;
  launch_union_count(mask, rank_of_block, g, P, own, union_mask, cnt, st);
  scan_kernel<<<1, 1024, 0, st>>>(cnt, g.B, g.H, P, include_local, entry_bytes, seg_offset, seg_total,
                                  volume_bytes, ent_base, n_entries);
  count_launch(2);
  SPARSP_CUDA_OK(cudaGetLastError());
  return SPARSP_OK;
}
