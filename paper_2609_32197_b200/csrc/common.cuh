// Shared host-side plumbing of the SparSP library: geometry, error reporting, workspace layout.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdarg>
#include <cstdio>

#include "../../include/sparsp.h"

namespace sparsp {

constexpr int kMaxBlocks = 1024;  // NB limit (score rows are held in shared memory)
constexpr int kMaxRanks = 64;
constexpr int kStatusWords = 64;  // workspace header: word 0 = status code, 1.. = detail

struct Geometry {
  int64_t N;         // tokens
  int64_t n_video;   // video tokens
  int32_t NB;        // blocks
  int32_t Wd;        // mask words per row
  int32_t nb_cand;   // text-free blocks (top-k candidates); text blocks are NB - nb_cand tail blocks
  int32_t B, H, d, b;
};

// One 16-byte record per packed entry, in pack order.
struct PackEntry {
  int64_t dst_byte;  // byte offset of the entry's K tile inside `packed`
  int32_t bh;        // batch * H + head
  int32_t j;         // KV block
};

struct WsLayout {
  int64_t status, pooled_q, pooled_k, scores, pairs, slot, tile_base, knorm, own, ent_base, n_entries, entries, total;
};

void set_error(const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);
extern std::atomic<int64_t> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int make_geometry(const sparsp_shape* s, Geometry* g);
int check_strides(const sparsp_shape* s, const Geometry& g);
WsLayout make_layout(const Geometry& g, int n_ranks);

// Raises a kernel's dynamic shared-memory limit to at least `bytes` on the current device; remembers
// what was set per (kernel, device) so that the driver call is made only when the limit must grow.
cudaError_t ensure_dynamic_smem(const void* func, int bytes);

inline int64_t align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

#define SPARSP_CUDA_OK(call)                              \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
  } while (0)

// launchers implemented in the kernel files -------------------------------------------------
int launch_pool(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, float* pq,
                float* pk, cudaStream_t st);
int launch_permute_tokens(const sparsp_shape& s, const Geometry& g, const void* X, void* Y,
                          const int32_t* block_of_slot, const int64_t* token_offset_of_slot, int inverse,
                          cudaStream_t st);
int launch_sharing(const Geometry& g, const uint32_t* mask, const int32_t* rank, int P, int64_t* hist,
                   cudaStream_t st);
int launch_score_cdf(const Geometry& g, const float* pq, const float* pk, float* scores, float tau, float scale,
                     uint32_t* mask, int32_t* kv_count, cudaStream_t st);
int launch_score_topk(const Geometry& g, const float* pq, const float* pk, float* scores, int topk,
                      uint32_t* mask, int32_t* kv_list, int32_t* kv_count, cudaStream_t st);
int launch_demand(const Geometry& g, const uint32_t* mask, const int32_t* rank_of_block, int P,
                  int flags, uint32_t* U, int32_t* cnt, int64_t* seg_off, int64_t* seg_total,
                  int64_t* volume, const int64_t* dst_base, int64_t capacity, char* ws,
                  const WsLayout& L, cudaStream_t st);
int launch_pack(const sparsp_shape& s, const Geometry& g, const void* K, const void* V, void* packed,
                int64_t capacity, int P, char* ws, const WsLayout& L, cudaStream_t st);
int launch_pack_segment(const sparsp_shape& s, const Geometry& g, const uint32_t* U, const int32_t* rank, int P,
                        int consumer, int producer, const int64_t* seg_off, const int32_t* cnt, const void* K,
                        const void* V, void* dst, int64_t capacity, char* ws, const WsLayout& L, cudaStream_t st);
int launch_attn(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                const uint32_t* mask, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                cudaStream_t st);

int launch_attn_packed(const sparsp_shape& s, const Geometry& g, const void* Q, const void* K, const void* V,
                       const uint32_t* mask, const int32_t* rank, int P, int consumer, const uint32_t* U,
                       const int64_t* seg_off, const int64_t* seg_total, const void* packed, int64_t capacity,
                       const int64_t* dst_base, float scale, void* O, float* lse, char* ws, const WsLayout& L,
                       cudaStream_t st);
int launch_hop_mask(const Geometry& g, const uint32_t* mask, const int32_t* rank, int consumer, int producer,
                    int head_begin, int head_end, uint32_t* hop, cudaStream_t st);
int launch_wait_timeout(char* ws, const WsLayout& L, long long limit_cycles, cudaStream_t st);
int launch_attn_merge(const sparsp_shape& s, const Geometry& g, const void* Oa, const float* la, const void* Ob,
                      const float* lb, void* O, float* lse, const int32_t* rank, int consumer, int head_begin,
                      int head_end, cudaStream_t st);

}  // namespace sparsp
