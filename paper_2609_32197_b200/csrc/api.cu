// extern "C" entry points of the SparSP library: argument checking, workspace carving, launch order.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>

#include "common.cuh"

namespace sparsp {

static thread_local char tl_error[512] = "";
std::atomic<int64_t> g_launches{0};

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(tl_error, sizeof tl_error, fmt, ap);
  va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what) {
  set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
  return SPARSP_ERR_CUDA;
}

cudaError_t ensure_dynamic_smem(const void* func, int bytes) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, int> limit;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  int& cur = limit[std::make_pair(func, dev)];
  if (bytes > cur) {
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    cur = bytes;
  }
  return cudaSuccess;
}

int make_geometry(const sparsp_shape* s, Geometry* g) {
  if (!s) {
    set_error("shape is NULL");
    return SPARSP_ERR_INVALID_ARG;
  }
  if (s->batch < 1 || s->heads < 1 || s->head_dim < 1 || s->grid_t < 1 || s->grid_h < 1 ||
      s->grid_w < 1 || s->n_text < 0 || s->block < 1) {
    set_error("shape has a non-positive dimension");
    return SPARSP_ERR_INVALID_ARG;
  }
  g->B = s->batch;
  g->H = s->heads;
  g->d = s->head_dim;
  g->b = s->block;
  g->n_video = (int64_t)s->grid_t * s->grid_h * s->grid_w;
  g->N = g->n_video + s->n_text;
  int64_t nb = (g->N + s->block - 1) / s->block;
  if (nb > kMaxBlocks) {
    set_error("NB = %lld exceeds the supported %d blocks", (long long)nb, kMaxBlocks);
    return SPARSP_ERR_UNSUPPORTED;
  }
  g->NB = (int32_t)nb;
  g->Wd = (g->NB + 31) / 32;
  g->nb_cand = s->n_text > 0 ? (int32_t)(g->n_video / s->block) : g->NB;
  return SPARSP_OK;
}

static int check_supported(const Geometry& g) {
  if (g.d != 64 && g.d != 128) {
    set_error("head_dim %d unsupported (64 or 128)", g.d);
    return SPARSP_ERR_UNSUPPORTED;
  }
  if (g.b != 64 && g.b != 128) {
    set_error("block %d unsupported (64 or 128)", g.b);
    return SPARSP_ERR_UNSUPPORTED;
  }
  return SPARSP_OK;
}

int check_strides(const sparsp_shape* s, const Geometry& g) {
  if (s->stride_token < g.d || s->stride_token % 8 || s->stride_head % 8 || s->stride_batch % 8 ||
      s->stride_head < 1 || (g.B > 1 && s->stride_batch < 1)) {
    set_error("strides must be positive multiples of 8 elements with stride_token >= head_dim");
    return SPARSP_ERR_INVALID_ARG;
  }
  return SPARSP_OK;
}

static int check_ptr(const void* p, const char* name, size_t align = 16) {
  if (!p) {
    set_error("%s is NULL", name);
    return SPARSP_ERR_INVALID_ARG;
  }
  if ((uintptr_t)p % align) {
    set_error("%s must be %zu-byte aligned", name, align);
    return SPARSP_ERR_INVALID_ARG;
  }
  return SPARSP_OK;
}

WsLayout make_layout(const Geometry& g, int P) {
  WsLayout L;
  int64_t off = 0;
  L.status = off;
  off += align_up(kStatusWords * 4, 256);
  const int64_t pooled = (int64_t)g.B * g.H * g.NB * g.d * 4;
  L.pooled_q = off;
  off += align_up(pooled, 256);
  L.pooled_k = off;
  off += align_up(pooled, 256);
  L.scores = off;  // pooled-Q x pooled-K^T, fp32 [B][H][NB][NB]
  off += align_up((int64_t)g.B * g.H * g.NB * g.NB * 4, 256);
  L.pairs = off;  // query-block pairs of the attention CTAs, int32 [B][H][ceil(NB/2)][2]
  off += align_up((int64_t)g.B * g.H * ((g.NB + 1) / 2) * 2 * 4, 256);
  L.slot = off;  // packed-buffer slot of every KV block for one consumer, int32 [B][H][NB]
  off += align_up((int64_t)g.B * g.H * g.NB * 4, 256);
  L.tile_base = off;  // first packed tile of that consumer per batch item, int64 [B]
  off += align_up((int64_t)g.B * 8, 256);
  L.knorm = off;  // largest key norm of every KV block, fp32 [B][H][NB] (attention: bound on the scores of a tile)
  off += align_up((int64_t)g.B * g.H * g.NB * 4, 256);
  L.own = off;
  off += align_up((int64_t)P * g.Wd * 4, 256);
  L.ent_base = off;
  off += align_up((int64_t)g.B * P * 8, 256);
  L.n_entries = off;
  off += 256;
  L.entries = off;
  off += align_up((int64_t)g.B * P * g.H * g.NB * (int64_t)sizeof(PackEntry), 256);
  L.total = off;
  return L;
}

}  // namespace sparsp

using namespace sparsp;

#define SPARSP_TRY(x)             \
  do {                            \
    int rc__ = (x);               \
    if (rc__ != SPARSP_OK) return rc__; \
  } while (0)

extern "C" {

const char* sparsp_last_error(void) { return tl_error; }

int64_t sparsp_launch_count(void) { return g_launches.load(); }

int sparsp_geometry(const sparsp_shape* shape, int64_t* n_tokens, int32_t* n_blocks, int32_t* n_words,
                    int32_t* n_video_blocks) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_tokens) *n_tokens = g.N;
  if (n_blocks) *n_blocks = g.NB;
  if (n_words) *n_words = g.Wd;
  if (n_video_blocks) *n_video_blocks = g.nb_cand;
  return SPARSP_OK;
}

int32_t sparsp_resolve_topk(int32_t pct, int32_t n_video_blocks) {
  int64_t k = ((int64_t)pct * n_video_blocks + 99) / 100;
  if (k < 1) k = 1;
  if (k > n_video_blocks) k = n_video_blocks;
  return (int32_t)k;
}

int sparsp_placement_contiguous(const sparsp_shape* shape, int32_t n_ranks, int32_t* rank_of_block) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || !rank_of_block) {
    set_error("bad n_ranks or NULL output");
    return SPARSP_ERR_INVALID_ARG;
  }
  for (int32_t j = 0; j < g.NB; ++j) rank_of_block[j] = (int32_t)(((int64_t)j * n_ranks) / g.NB);
  return SPARSP_OK;
}

int sparsp_placement_periodic(const sparsp_shape* shape, int32_t n_ranks, int32_t* rank_of_block) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || !rank_of_block) {
    set_error("bad n_ranks or NULL output");
    return SPARSP_ERR_INVALID_ARG;
  }
  const int64_t F = (int64_t)shape->grid_h * shape->grid_w;
  for (int32_t j = 0; j < g.NB; ++j) {
    const int64_t first = (int64_t)j * g.b;
    rank_of_block[j] = first >= g.n_video ? j % n_ranks : (int32_t)((n_ranks * (first % F)) / F);
  }
  return SPARSP_OK;
}

int sparsp_placement_permutation(const sparsp_shape* shape, int32_t n_ranks, const int32_t* rank_of_block,
                                 int32_t* block_of_slot, int64_t* token_offset_of_slot, int32_t* first_slot_of_rank) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || !rank_of_block || !block_of_slot || !token_offset_of_slot) {
    set_error("bad n_ranks or NULL argument");
    return SPARSP_ERR_INVALID_ARG;
  }
  for (int32_t j = 0; j < g.NB; ++j)
    if (rank_of_block[j] < 0 || rank_of_block[j] >= n_ranks) {
      set_error("rank_of_block[%d] = %d outside 0..%d", j, rank_of_block[j], n_ranks - 1);
      return SPARSP_ERR_INVALID_ARG;
    }
  int32_t slot = 0;
  int64_t tok = 0;
  for (int32_t r = 0; r < n_ranks; ++r) {
    if (first_slot_of_rank) first_slot_of_rank[r] = slot;
    for (int32_t j = 0; j < g.NB; ++j)
      if (rank_of_block[j] == r) {
        block_of_slot[slot] = j;
        token_offset_of_slot[slot] = tok;
        tok += std::min<int64_t>(g.b, g.N - (int64_t)j * g.b);
        ++slot;
      }
  }
  token_offset_of_slot[g.NB] = tok;
  if (first_slot_of_rank) first_slot_of_rank[n_ranks] = slot;
  return SPARSP_OK;
}

int sparsp_permute_tokens(const sparsp_shape* shape, const void* X, void* Y, const int32_t* block_of_slot,
                          const int64_t* token_offset_of_slot, int32_t inverse, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(X, "X"));
  SPARSP_TRY(check_ptr(Y, "Y"));
  SPARSP_TRY(check_ptr(block_of_slot, "block_of_slot", 4));
  SPARSP_TRY(check_ptr(token_offset_of_slot, "token_offset_of_slot", 8));
  if (X == Y) {
    set_error("X and Y must be different buffers");
    return SPARSP_ERR_INVALID_ARG;
  }
  return launch_permute_tokens(*shape, g, X, Y, block_of_slot, token_offset_of_slot, inverse != 0,
                               (cudaStream_t)stream);
}

int sparsp_sharing_histogram(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                             int32_t n_ranks, int64_t* hist, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks) {
    set_error("n_ranks %d outside 1..%d", n_ranks, kMaxRanks);
    return SPARSP_ERR_INVALID_ARG;
  }
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  SPARSP_TRY(check_ptr(hist, "hist", 8));
  return launch_sharing(g, mask, rank_of_block, n_ranks, hist, (cudaStream_t)stream);
}

int sparsp_exchange_plan(const sparsp_shape* shape, int32_t n_ranks, const int32_t* cnt, const int64_t* seg_offset,
                         int32_t steady_chunks, int32_t tail_chunks, sparsp_transfer* transfers, int64_t capacity,
                         int64_t* n_transfers) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || !cnt || !seg_offset || !n_transfers || capacity < 0 ||
      (capacity > 0 && !transfers) || steady_chunks < 1 || tail_chunks < 1) {
    set_error("bad n_ranks, chunk count, capacity or NULL argument");
    return SPARSP_ERR_INVALID_ARG;
  }
  const int P = n_ranks, H = g.H;
  const int c_steady = std::min(steady_chunks, H), c_tail = std::min(tail_chunks, H);
  const int64_t per_consumer = P > 1 ? (int64_t)(P - 2) * c_steady + c_tail : 0;
  *n_transfers = (int64_t)g.B * P * per_consumer;
  if (*n_transfers > capacity) {
    set_error("transfer list needs %lld records, capacity %lld", (long long)*n_transfers, (long long)capacity);
    return SPARSP_ERR_CAPACITY;
  }
  const int64_t entry_bytes = 2LL * g.b * g.d * 2;
  sparsp_transfer* out = transfers;
  for (int bb = 0; bb < g.B; ++bb)
    for (int r = 0; r < P; ++r)
      for (int k = 0; k + 1 < P; ++k) {
        const int p = ((r - (k + 1)) % P + P) % P;
        const int C = k == P - 2 ? c_tail : c_steady;
        const int32_t* c_row = cnt + (((int64_t)bb * P + r) * P + p) * H;
        const int64_t* o_row = seg_offset + (((int64_t)bb * P + r) * P + p) * H;
        sparsp_transfer* hop = out;
        for (int c = 0; c < C; ++c) {
          const int h0 = (int)(((int64_t)c * H) / C), h1 = (int)(((int64_t)(c + 1) * H) / C);
          int64_t n = 0;
          for (int h = h0; h < h1; ++h) n += c_row[h];
          sparsp_transfer t;
          t.batch = bb; t.consumer = r; t.producer = p; t.round = k; t.order = 0;
          t.head_begin = h0; t.head_end = h1; t.reserved = 0;
          t.entry_begin = o_row[h0]; t.n_entries = n;
          t.byte_offset = t.entry_begin * entry_bytes; t.n_bytes = n * entry_bytes;
          *out++ = t;
        }
        // most blocks first, lower head first among equals (the chunks were produced in head order)
        std::stable_sort(hop, out, [](const sparsp_transfer& a, const sparsp_transfer& b) { return a.n_entries > b.n_entries; });
        for (int c = 0; c < C; ++c) hop[c].order = c;
      }
  return SPARSP_OK;
}

int sparsp_workspace_bytes(const sparsp_shape* shape, int32_t n_ranks, int64_t* bytes) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || !bytes) {
    set_error("bad n_ranks or NULL output");
    return SPARSP_ERR_INVALID_ARG;
  }
  *bytes = make_layout(g, n_ranks).total;
  return SPARSP_OK;
}

int sparsp_block_mask(const sparsp_shape* shape, const void* Q, const void* K, int32_t topk_video,
                      uint32_t* mask, int32_t* kv_list, int32_t* kv_count, float* pooled_q,
                      float* pooled_k, void* workspace, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(Q, "Q"));
  SPARSP_TRY(check_ptr(K, "K"));
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (topk_video < 1 || topk_video > g.nb_cand) {
    set_error("topk_video %d outside 1..%d", topk_video, g.nb_cand);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (pooled_q && (uintptr_t)pooled_q % 16) return check_ptr((void*)1, "pooled_q");
  if (pooled_k && (uintptr_t)pooled_k % 16) return check_ptr((void*)1, "pooled_k");
  char* ws = (char*)workspace;
  const WsLayout L = make_layout(g, 1);
  float* pq = pooled_q ? pooled_q : (float*)(ws + L.pooled_q);
  float* pk = pooled_k ? pooled_k : (float*)(ws + L.pooled_k);
  cudaStream_t st = (cudaStream_t)stream;
  SPARSP_TRY(launch_pool(*shape, g, Q, K, pq, pk, st));
  SPARSP_TRY(launch_score_topk(g, pq, pk, (float*)(ws + L.scores), topk_video, mask, kv_list, kv_count, st));
  return SPARSP_OK;
}

int sparsp_block_mask_cdf(const sparsp_shape* shape, const void* Q, const void* K, float tau, float score_scale,
                          uint32_t* mask, int32_t* kv_count, float* pooled_q, float* pooled_k, void* workspace,
                          void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(Q, "Q"));
  SPARSP_TRY(check_ptr(K, "K"));
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (!(tau > 0.0f && tau <= 1.0f)) {
    set_error("tau %g outside (0, 1]", (double)tau);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (!(score_scale >= 0.0f) || score_scale > 1e6f) {
    set_error("score_scale %g must be 0 (meaning 1/sqrt(d)) or a positive finite number", (double)score_scale);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (g.nb_cand < 1) {
    set_error("the sequence has no video block to choose from");
    return SPARSP_ERR_INVALID_ARG;
  }
  if (pooled_q && (uintptr_t)pooled_q % 16) return check_ptr((void*)1, "pooled_q");
  if (pooled_k && (uintptr_t)pooled_k % 16) return check_ptr((void*)1, "pooled_k");
  char* ws = (char*)workspace;
  const WsLayout L = make_layout(g, 1);
  float* pq = pooled_q ? pooled_q : (float*)(ws + L.pooled_q);
  float* pk = pooled_k ? pooled_k : (float*)(ws + L.pooled_k);
  cudaStream_t st = (cudaStream_t)stream;
  const float scale = score_scale > 0.0f ? score_scale : 1.0f / sqrtf((float)g.d);
  SPARSP_TRY(launch_pool(*shape, g, Q, K, pq, pk, st));
  SPARSP_TRY(launch_score_cdf(g, pq, pk, (float*)(ws + L.scores), tau, scale, mask, kv_count, st));
  return SPARSP_OK;
}

int sparsp_demand_pack(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                       int32_t n_ranks, int32_t flags, const void* K, const void* V,
                       uint32_t* union_mask, int32_t* cnt, int64_t* seg_offset, int64_t* seg_total,
                       int64_t* volume_bytes, void* packed, int64_t packed_capacity_bytes,
                       const int64_t* dst_base_bytes, void* workspace, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  if (n_ranks < 1 || n_ranks > kMaxRanks) {
    set_error("n_ranks %d outside 1..%d", n_ranks, kMaxRanks);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (flags & ~(SPARSP_PLAN_ONLY | SPARSP_INCLUDE_LOCAL)) {
    set_error("unknown flag bits 0x%x", flags);
    return SPARSP_ERR_INVALID_ARG;
  }
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  SPARSP_TRY(check_ptr(union_mask, "union_mask", 4));
  SPARSP_TRY(check_ptr(cnt, "cnt", 4));
  SPARSP_TRY(check_ptr(seg_offset, "seg_offset", 8));
  SPARSP_TRY(check_ptr(seg_total, "seg_total", 8));
  SPARSP_TRY(check_ptr(volume_bytes, "volume_bytes", 8));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  const bool plan_only = flags & SPARSP_PLAN_ONLY;
  if (!plan_only) {
    SPARSP_TRY(check_strides(shape, g));
    SPARSP_TRY(check_ptr(K, "K"));
    SPARSP_TRY(check_ptr(V, "V"));
    SPARSP_TRY(check_ptr(packed, "packed"));
    if (packed_capacity_bytes < 0) {
      set_error("negative packed_capacity_bytes");
      return SPARSP_ERR_INVALID_ARG;
    }
  }
  if (dst_base_bytes && (uintptr_t)dst_base_bytes % 8) return check_ptr((void*)1, "dst_base_bytes", 8);
  char* ws = (char*)workspace;
  const WsLayout L = make_layout(g, n_ranks);
  cudaStream_t st = (cudaStream_t)stream;
  SPARSP_TRY(launch_demand(g, mask, rank_of_block, n_ranks, flags, union_mask, cnt, seg_offset,
                           seg_total, volume_bytes, dst_base_bytes,
                           plan_only ? (int64_t)-1 : packed_capacity_bytes, ws, L, st));
  if (!plan_only) SPARSP_TRY(launch_pack(*shape, g, K, V, packed, packed_capacity_bytes, n_ranks, ws, L, st));
  return SPARSP_OK;
}

int sparsp_pack_segment(const sparsp_shape* shape, const uint32_t* union_mask, const int32_t* rank_of_block,
                        int32_t n_ranks, int32_t consumer, int32_t producer, const int32_t* cnt,
                        const int64_t* seg_offset, const void* K, const void* V, void* dst, int64_t dst_capacity_bytes,
                        void* workspace, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  if (g.B != 1) {
    set_error("sparsp_pack_segment handles one batch item per call (batch = %d)", g.B);
    return SPARSP_ERR_UNSUPPORTED;
  }
  if (n_ranks < 1 || n_ranks > kMaxRanks || consumer < 0 || consumer >= n_ranks || producer < 0 ||
      producer >= n_ranks || consumer == producer) {
    set_error("consumer / producer %d / %d must be two different ranks of 0..%d", consumer, producer, n_ranks - 1);
    return SPARSP_ERR_INVALID_ARG;
  }
  SPARSP_TRY(check_ptr(union_mask, "union_mask", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  SPARSP_TRY(check_ptr(cnt, "cnt", 4));
  SPARSP_TRY(check_ptr(seg_offset, "seg_offset", 8));
  SPARSP_TRY(check_ptr(K, "K"));
  SPARSP_TRY(check_ptr(V, "V"));
  SPARSP_TRY(check_ptr(dst, "dst"));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (dst_capacity_bytes < 0) {
    set_error("negative dst_capacity_bytes");
    return SPARSP_ERR_INVALID_ARG;
  }
  const WsLayout L = make_layout(g, n_ranks);
  return launch_pack_segment(*shape, g, union_mask, rank_of_block, n_ranks, consumer, producer, seg_offset, cnt, K, V,
                             dst, dst_capacity_bytes, (char*)workspace, L, (cudaStream_t)stream);
}

int sparsp_sparse_attn_fwd(const sparsp_shape* shape, const void* Q, const void* K, const void* V,
                           const uint32_t* mask, float softmax_scale, void* O, float* lse,
                           void* workspace, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(Q, "Q"));
  SPARSP_TRY(check_ptr(K, "K"));
  SPARSP_TRY(check_ptr(V, "V"));
  SPARSP_TRY(check_ptr(O, "O"));
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (lse && (uintptr_t)lse % 4) return check_ptr((void*)1, "lse", 4);
  if (!(softmax_scale >= 0.0f)) {
    set_error("softmax_scale must be >= 0");
    return SPARSP_ERR_INVALID_ARG;
  }
  const WsLayout L = make_layout(g, 1);
  return launch_attn(*shape, g, Q, K, V, mask, softmax_scale, O, lse, (char*)workspace, L,
                     (cudaStream_t)stream);
}

int sparsp_sparse_attn_fwd_packed(const sparsp_shape* shape, const void* Q, const void* K, const void* V,
                                  const uint32_t* mask, const int32_t* rank_of_block, int32_t n_ranks,
                                  int32_t consumer, const uint32_t* union_mask, const int64_t* seg_offset,
                                  const int64_t* seg_total, const void* packed, int64_t packed_capacity_bytes,
                                  const int64_t* dst_base_bytes, float softmax_scale, void* O, float* lse,
                                  void* workspace, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || consumer < 0 || consumer >= n_ranks) {
    set_error("consumer %d outside 0..%d", consumer, n_ranks - 1);
    return SPARSP_ERR_INVALID_ARG;
  }
  SPARSP_TRY(check_ptr(Q, "Q"));
  SPARSP_TRY(check_ptr(K, "K"));
  SPARSP_TRY(check_ptr(V, "V"));
  SPARSP_TRY(check_ptr(O, "O"));
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  SPARSP_TRY(check_ptr(union_mask, "union_mask", 4));
  SPARSP_TRY(check_ptr(seg_offset, "seg_offset", 8));
  SPARSP_TRY(check_ptr(seg_total, "seg_total", 8));
  SPARSP_TRY(check_ptr(packed, "packed", 16));
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (lse && (uintptr_t)lse % 4) return check_ptr((void*)1, "lse", 4);
  if (dst_base_bytes && (uintptr_t)dst_base_bytes % 8) return check_ptr((void*)1, "dst_base_bytes", 8);
  if (!(softmax_scale >= 0.0f)) {
    set_error("softmax_scale must be >= 0");
    return SPARSP_ERR_INVALID_ARG;
  }
  if (packed_capacity_bytes < (int64_t)g.b * g.d * 2) {
    set_error("packed_capacity_bytes is smaller than one tile");
    return SPARSP_ERR_INVALID_ARG;
  }
  const WsLayout L = make_layout(g, 1);
  return launch_attn_packed(*shape, g, Q, K, V, mask, rank_of_block, n_ranks, consumer, union_mask, seg_offset,
                            seg_total, packed, packed_capacity_bytes, dst_base_bytes, softmax_scale, O, lse,
                            (char*)workspace, L, (cudaStream_t)stream);
}

int sparsp_hop_chunk_mask(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                          int32_t n_ranks, int32_t consumer, int32_t producer, int32_t head_begin, int32_t head_end,
                          uint32_t* hop_mask, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  if (n_ranks < 1 || n_ranks > kMaxRanks || consumer < 0 || consumer >= n_ranks || producer < 0 ||
      producer >= n_ranks) {
    set_error("consumer/producer %d/%d outside 0..%d", consumer, producer, n_ranks - 1);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (head_begin < 0 || head_end > g.H || head_begin > head_end) {
    set_error("head range [%d, %d) outside [0, %d)", head_begin, head_end, g.H);
    return SPARSP_ERR_INVALID_ARG;
  }
  SPARSP_TRY(check_ptr(mask, "mask", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  SPARSP_TRY(check_ptr(hop_mask, "hop_mask", 4));
  return launch_hop_mask(g, mask, rank_of_block, consumer, producer, head_begin, head_end, hop_mask,
                         (cudaStream_t)stream);
}

int sparsp_hop_mask(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block, int32_t n_ranks,
                    int32_t consumer, int32_t producer, uint32_t* hop_mask, void* stream) {
  if (!shape) return sparsp_hop_chunk_mask(shape, mask, rank_of_block, n_ranks, consumer, producer, 0, 0, hop_mask, stream);
  return sparsp_hop_chunk_mask(shape, mask, rank_of_block, n_ranks, consumer, producer, 0, shape->heads, hop_mask,
                               stream);
}

int sparsp_attn_merge(const sparsp_shape* shape, const void* O_a, const float* lse_a, const void* O_b,
                      const float* lse_b, void* O, float* lse, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(O_a, "O_a"));
  SPARSP_TRY(check_ptr(O_b, "O_b"));
  SPARSP_TRY(check_ptr(O, "O"));
  SPARSP_TRY(check_ptr(lse_a, "lse_a", 4));
  SPARSP_TRY(check_ptr(lse_b, "lse_b", 4));
  SPARSP_TRY(check_ptr(lse, "lse", 4));
  return launch_attn_merge(*shape, g, O_a, lse_a, O_b, lse_b, O, lse, nullptr, 0, 0, g.H, (cudaStream_t)stream);
}

int sparsp_attn_merge_rows(const sparsp_shape* shape, const void* O_a, const float* lse_a, const void* O_b,
                           const float* lse_b, void* O, float* lse, const int32_t* rank_of_block, int32_t n_ranks,
                           int32_t consumer, int32_t head_begin, int32_t head_end, void* stream) {
  Geometry g;
  SPARSP_TRY(make_geometry(shape, &g));
  SPARSP_TRY(check_supported(g));
  SPARSP_TRY(check_strides(shape, g));
  SPARSP_TRY(check_ptr(O_a, "O_a"));
  SPARSP_TRY(check_ptr(O_b, "O_b"));
  SPARSP_TRY(check_ptr(O, "O"));
  SPARSP_TRY(check_ptr(lse_a, "lse_a", 4));
  SPARSP_TRY(check_ptr(lse_b, "lse_b", 4));
  SPARSP_TRY(check_ptr(lse, "lse", 4));
  SPARSP_TRY(check_ptr(rank_of_block, "rank_of_block", 4));
  if (n_ranks < 1 || n_ranks > kMaxRanks || consumer < 0 || consumer >= n_ranks || head_begin < 0 ||
      head_end > g.H || head_begin > head_end) {
    set_error("consumer %d outside 0..%d or head range [%d, %d) outside [0, %d)", consumer, n_ranks - 1, head_begin,
              head_end, g.H);
    return SPARSP_ERR_INVALID_ARG;
  }
  return launch_attn_merge(*shape, g, O_a, lse_a, O_b, lse_b, O, lse, rank_of_block, consumer, head_begin, head_end,
                           (cudaStream_t)stream);
}

int sparsp_selftest_wait_timeout(void* workspace, int64_t limit_cycles, void* stream) {
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (limit_cycles < 1 || limit_cycles > 100000000LL) {
    set_error("limit_cycles %lld outside 1..1e8", (long long)limit_cycles);
    return SPARSP_ERR_INVALID_ARG;
  }
  WsLayout L;
  L.status = 0;  // the status words open the workspace whatever the shape
  return launch_wait_timeout((char*)workspace, L, limit_cycles, (cudaStream_t)stream);
}

int sparsp_status(void* workspace, void* stream, int32_t* code) {
  SPARSP_TRY(check_ptr(workspace, "workspace", 256));
  if (!code) {
    set_error("code is NULL");
    return SPARSP_ERR_INVALID_ARG;
  }
  cudaStream_t st = (cudaStream_t)stream;
  int32_t words[4] = {0, 0, 0, 0};
  SPARSP_CUDA_OK(cudaMemcpyAsync(words, workspace, sizeof words, cudaMemcpyDeviceToHost, st));
  SPARSP_CUDA_OK(cudaStreamSynchronize(st));
  *code = words[0];
  if (words[0] != SPARSP_OK) {
    set_error("device status %d (detail %d %d %d)", words[0], words[1], words[2], words[3]);
    SPARSP_CUDA_OK(cudaMemsetAsync(workspace, 0, kStatusWords * 4, st));
    SPARSP_CUDA_OK(cudaStreamSynchronize(st));
  }
  return SPARSP_OK;
}

}  // extern "C"
