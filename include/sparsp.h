/*
 * sparsp.h -- C ABI of the SparSP single-device hot path on B200 (sm_100a).
 *
 * Three calls make one sparse sequence-parallel attention layer for P *virtual* ranks that all live
 * on one GPU (nothing crosses devices):
 *
 *   sparsp_block_mask       block mask M[h,i,j] from mean-pooled query / key tiles
 *   sparsp_demand_pack      receiver demand D[r,h,p], exchange volume V_r, row-major packing
 *   sparsp_sparse_attn_fwd  block-sparse softmax(QK^T/sqrt(d))V over M
 *
 * Conventions shared by every call
 *   - Return value: SPARSP_OK (0) or a negative SPARSP_ERR_* code.  Argument errors are detected
 *     on the host before anything is launched; sparsp_last_error() returns a text for the calling
 *     thread's most recent failure.
 *   - Unless a parameter says "host", every data pointer is a DEVICE pointer owned by the caller.
 *     The library never allocates, frees or keeps caller memory; scratch lives in a caller-provided
 *     device workspace of sparsp_workspace_bytes() bytes (256-byte aligned).  Calls that share a
 *     workspace must be ordered on one stream.
 *   - `stream` is a cudaStream_t passed as void*; all work is enqueued on it asynchronously.
 *     Conditions only the device can detect (packed buffer too small, a bounded wait inside a
 *     kernel running out) are written to a status word in the workspace; sparsp_status()
 *     synchronises the stream and returns it.  No kernel traps or asserts.
 *   - Q, K, V, O are bf16 with the head_dim axis contiguous; element strides for batch, head and
 *     token are given in sparsp_shape, so both [B][H][N][d] and [B][N][H][d] work.  Base pointers
 *     and strides must be multiples of 8 elements (16 bytes).
 *   - Tokens: the grid_t*grid_h*grid_w video tokens in row-major (t, h, w) order, then n_text text
 *     tokens.  N = their sum.  Blocks are flat runs of `block` tokens, NB = ceil(N/block); the last
 *     block may be ragged.  A block is a *text block* iff it holds at least one text token.
 *   - Masks are uint32 words: KV block j of row (b, h, i) is bit (j & 31) of word (j >> 5);
 *     Wd = ceil(NB/32) words per row; bits at and beyond NB are zero.
 *   - Supported: head_dim in {64, 128}, block in {64, 128}, NB <= 1024, n_ranks <= 64.
 */
#ifndef SPARSP_H_
#define SPARSP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SPARSP_API __attribute__((visibility("default")))
#else
#define SPARSP_API
#endif

#define SPARSP_OK 0
#define SPARSP_ERR_INVALID_ARG (-1)
#define SPARSP_ERR_UNSUPPORTED (-2)
#define SPARSP_ERR_CAPACITY (-3)
#define SPARSP_ERR_CUDA (-4)
#define SPARSP_ERR_TIMEOUT (-5)

/* flags of sparsp_demand_pack */
#define SPARSP_PLAN_ONLY 1     /* compute union/cnt/offsets/volume, copy nothing */
#define SPARSP_INCLUDE_LOCAL 2 /* also pack the p == r segment (in its ascending-p position) */

typedef struct sparsp_shape {
  int32_t batch, heads, head_dim;         /* B, H, d */
  int32_t grid_t, grid_h, grid_w, n_text; /* latent grid T x H x W, text tokens appended */
  int32_t block;                          /* b: tokens per query / KV block */
  int64_t stride_batch, stride_head, stride_token; /* in elements, for Q, K, V and O alike */
} sparsp_shape;

/* Host helpers (no GPU work). ---------------------------------------------------------------- */

/* N, NB, Wd and the number of candidate (text-free) blocks for a shape.  Any out pointer may be
 * NULL.  Returns SPARSP_ERR_INVALID_ARG for non-positive dimensions. */
SPARSP_API int sparsp_geometry(const sparsp_shape* shape, int64_t* n_tokens, int32_t* n_blocks,
                    int32_t* n_words, int32_t* n_video_blocks);

/* "top-k = pct % of the blocks": ceil(pct * n_video_blocks / 100) clamped to [1, n_video_blocks]. */
SPARSP_API int32_t sparsp_resolve_topk(int32_t pct, int32_t n_video_blocks);

/* Naive contiguous partition of the sequence (Section 3.2): rank(j) = floor(j * n_ranks / NB).
 * rank_of_block: HOST array of NB int32. */
SPARSP_API int sparsp_placement_contiguous(const sparsp_shape* shape, int32_t n_ranks, int32_t* rank_of_block);

/* Interval-periodic layout (Section 4.3, Eq. "periodic-placement"): each frame is cut into
 * n_ranks contiguous spatial intervals and the same interval goes to the same rank in every frame.
 * For block j whose first token lies in the video part, rank = floor(G * ((j*b) mod F) / F) with
 * F = grid_h * grid_w tokens per frame, which is floor(G*s/B) when frames are whole blocks; blocks
 * starting in the text tail get j mod G.  rank_of_block: HOST array of NB int32. */
SPARSP_API int sparsp_placement_periodic(const sparsp_shape* shape, int32_t n_ranks, int32_t* rank_of_block);

/* The placement as a permutation of whole KV blocks (Section 4.3: a deterministic permutation from logical
 * block coordinates to (rank, offset) pairs, computed once per geometry and rank count, undone by its
 * inverse).  Slots are ordered by rank and, inside a rank, by logical block index.
 *   rank_of_block           in   HOST int32 [NB], values 0 .. n_ranks-1
 *   block_of_slot           out  HOST int32 [NB]: the logical block held by slot s
 *   token_offset_of_slot    out  HOST int64 [NB+1]: first token of slot s in the permuted sequence (the
 *                                sequence's last block may be shorter than `block`); entry NB = N
 *   first_slot_of_rank      out  HOST int32 [n_ranks+1]; may be NULL */
SPARSP_API int sparsp_placement_permutation(const sparsp_shape* shape, int32_t n_ranks, const int32_t* rank_of_block,
                                 int32_t* block_of_slot, int64_t* token_offset_of_slot,
                                 int32_t* first_slot_of_rank);

/* Applies that permutation (inverse = 0: logical order -> permuted order) or undoes it (inverse != 0) on a
 * bf16 tensor strided as in `shape`; block membership is unchanged, tokens inside a block keep their order.
 *   X in, Y out: DEVICE, different buffers;  block_of_slot, token_offset_of_slot: DEVICE copies of the above */
SPARSP_API int sparsp_permute_tokens(const sparsp_shape* shape, const void* X, void* Y, const int32_t* block_of_slot,
                          const int64_t* token_offset_of_slot, int32_t inverse, void* stream);

/* How widely received K blocks are shared (Section 3.2): for every remote KV block j that consumer r
 * receives for head h (some query block of r keeps it), the fraction of r's query blocks that keep it.
 *   hist  out  DEVICE int64 [B][n_ranks][101]: hist[b][r][q] = number of such (h, j) pairs whose fraction,
 *              in whole percent rounded down, is q
 *   mask  uint32 [B][H][NB][Wd];  rank_of_block  DEVICE int32 [NB] */
SPARSP_API int sparsp_sharing_histogram(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                             int32_t n_ranks, int64_t* hist, void* stream);

/* Bytes of device workspace the three calls need for this shape and rank count. */
SPARSP_API int sparsp_workspace_bytes(const sparsp_shape* shape, int32_t n_ranks, int64_t* bytes);

/* Step 1 -- block-importance estimation (Section 4.2: masks are materialised from pooled query
 * and key tiles; selection rule: top-k per query block).
 *   pooled[b,h,i,:] = mean over the valid tokens of block i (fp32, ascending-token sum, one division)
 *   S[b,h,i,j]      = sum_c pooledQ[i,c] * pooledK[j,c]   (fp32 fused multiply-add chain, c ascending)
 *   per row keep the topk_video highest-scoring text-free blocks (equal scores: lower j first,
 *   -0 == +0), then every text block.
 * Q, K        in   bf16, strided as in `shape`
 * topk_video  in   1 .. n_video_blocks
 * mask        out  uint32 [B][H][NB][Wd]
 * kv_list     out  int32 [B][H][NB][kept] ascending kept blocks, kept = topk_video + #text blocks; may be NULL
 * kv_count    out  int32 [B][H][NB]; may be NULL
 * pooled_q/k  out  fp32 [B][H][NB][d]; may be NULL (kept in the workspace then)
 */
SPARSP_API int sparsp_block_mask(const sparsp_shape* shape, const void* Q, const void* K, int32_t topk_video,
                      uint32_t* mask, int32_t* kv_list, int32_t* kv_count, float* pooled_q,
                      float* pooled_k, void* workspace, void* stream);

/* Step 1, CDF-threshold selection (Section 8.1: for each query, keep the key blocks with the highest
 * scores until their cumulative attention mass reaches the threshold).  Same pooling and scores as
 * sparsp_block_mask; per row, over the text-free blocks:
 *   p_j = exp(score_scale * (S_j - max S)),  Z = sum_j p_j,
 *   keep the smallest set { j : S_j >= v } (v one of the row's scores) whose mass reaches tau * Z --
 *   blocks with equal scores (-0 == +0) are kept or dropped together -- then every text block.
 * The arithmetic is fixed: x_j = (S_j - max S) * (score_scale * log2 e) in fp32, one subtraction and
 * one multiplication; p_j = 2^x_j in fp32 by clamping x at -125, splitting off the nearest integer (ties to
 * even) and a degree-5 Horner polynomial of the remainder with fused multiply-adds (coefficients
 * 0.0013400432653725147, 0.009676037356257439, 0.05550327152013779, 0.2402210682630539,
 * 0.6931471824645996, 1.0000001192092896), the integer part added into the exponent field.  The mass is
 * counted in integers, so that no order of additions is part of the definition: w_j = floor(p_j * 2^26),
 * Z = sum_j w_j, and a set reaches the threshold when its sum of w_j is >= ceil(tau * Z), that product
 * taken once in fp64.
 *   tau          in   (0, 1]
 *   score_scale  in   0 means 1/sqrt(d)
 *   mask         out  uint32 [B][H][NB][Wd]   (rows keep different numbers of blocks)
 *   kv_count     out  int32 [B][H][NB]; may be NULL
 *   pooled_q/k   out  fp32 [B][H][NB][d]; may be NULL
 */
SPARSP_API int sparsp_block_mask_cdf(const sparsp_shape* shape, const void* Q, const void* K, float tau,
                          float score_scale, uint32_t* mask, int32_t* kv_count, float* pooled_q,
                          float* pooled_k, void* workspace, void* stream);

/* Step 2 -- demand and packing for n_ranks virtual ranks (Section 4.1, Eq. "receiver-demand" and
 * Eq. "sparse-exchange-volume"; Section 5.2: head-preserving demand, row-major packing with
 * locally derived offsets; Section 6: one slot per (producer, consumer) pair).
 *   Q_r = { i : rank_of_block[i] = r },  P(j) = rank_of_block[j]
 *   union_mask[b,r,h]  = OR_{i in Q_r} M[b,h,i]
 *   cnt[b,r,p,h]       = | { j in union_mask[b,r,h] : P(j) = p } |         (p == r: local reuse)
 *   volume_bytes[b,r]  = 2*block*d*2 * sum_h sum_{p != r} cnt[b,r,p,h]
 *   seg_offset[b,r,p,h]= entry index in consumer r's buffer of the first block of (producer p, head h):
 *                        exclusive scan of cnt over p ascending (p == r skipped unless
 *                        SPARSP_INCLUDE_LOCAL) then h ascending
 *   seg_total[b,r]     = number of entries in consumer r's buffer
 *   packed             = for every (b, r): at byte dst_base_bytes[b,r], the entries in that order, each
 *                        entry = K tile (block x d bf16) then V tile of (h, j), j ascending inside a head;
 *                        rows at or beyond N are zero.
 * mask            in   uint32 [B][H][NB][Wd]
 * rank_of_block   in   DEVICE int32 [NB], values 0 .. n_ranks-1
 * K, V            in   bf16 (ignored with SPARSP_PLAN_ONLY)
 * union_mask      out  uint32 [B][P][H][Wd]
 * cnt             out  int32 [B][P][P][H]
 * seg_offset      out  int64 [B][P][P][H]
 * seg_total       out  int64 [B][P]
 * volume_bytes    out  int64 [B][P]
 * packed          out  bytes; 16-byte aligned (ignored with SPARSP_PLAN_ONLY)
 * packed_capacity_bytes  size of `packed`
 * dst_base_bytes  in   DEVICE int64 [B][P], multiples of 16, or NULL = consumers back to back in
 *                      (b, r) order starting at byte 0
 * If an entry would end beyond packed_capacity_bytes it is not written and the status word becomes
 * SPARSP_ERR_CAPACITY.
 */
SPARSP_API int sparsp_demand_pack(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                       int32_t n_ranks, int32_t flags, const void* K, const void* V,
                       uint32_t* union_mask, int32_t* cnt, int64_t* seg_offset, int64_t* seg_total,
                       int64_t* volume_bytes, void* packed, int64_t packed_capacity_bytes,
                       const int64_t* dst_base_bytes, void* workspace, void* stream);

/* Step 3 -- block-sparse attention forward (Section 2.2, Eq. "attention", restricted to the kept
 * blocks of M): for every valid query token q of block i,
 *   O[q,:] = sum_t p_t V[t,:] / sum_t p_t,   p_t = exp(s_t - max s),   s_t = scale * Q[q,:].K[t,:]
 * over the tokens t < N of the KV blocks kept in row (b,h,i).  bf16 tensor-core products, fp32
 * accumulation and fp32 online softmax.  Every row must keep at least one block.
 *   mask           in   uint32 [B][H][NB][Wd]
 *   softmax_scale  in   0 means 1/sqrt(d)
 *   O              out  bf16, strided like Q; rows of tokens >= N are not written
 *   lse            out  fp32 [B][H][N], natural-log sum-exp of the scaled logits; may be NULL
 */
SPARSP_API int sparsp_sparse_attn_fwd(const sparsp_shape* shape, const void* Q, const void* K, const void* V,
                           const uint32_t* mask, float softmax_scale, void* O, float* lse,
                           void* workspace, void* stream);

/* Consumer side of the demand-routed exchange (Section 5.1: in round k a rank receives from the
 * producer at ring distance k exactly the blocks it selected; Section 7: the attention over each
 * arriving part is merged with the running result by online softmax).
 *
 * sparsp_hop_mask: the mask of ONE hop,
 *   hop_mask[b,h,i,:] = (rank_of_block[i] == consumer) ? mask[b,h,i,:] AND own[producer,:] : 0,
 * i.e. the consumer rank's query blocks restricted to the KV blocks the producer owns.  Feeding it to
 * sparsp_sparse_attn_fwd (with lse) gives that hop's partial result; rows without any kept key come
 * out as zeros with lse = -inf.
 *   mask, hop_mask  uint32 [B][H][NB][Wd];  rank_of_block  DEVICE int32 [NB]
 *
 * sparsp_attn_merge: log-sum-exp merge of two partial results over disjoint key sets,
 *   lse = log(exp(lse_a) + exp(lse_b)),  O = O_a * exp(lse_a - lse) + O_b * exp(lse_b - lse),
 * computed in fp32, O rounded to bf16.  O may alias O_a or O_b (and lse alias lse_a or lse_b).
 *   O_a, O_b, O  bf16, strided as in `shape`;  lse_a, lse_b, lse  fp32 [B][H][N] */
/* sparsp_sparse_attn_fwd_packed: step 3 as the CONSUMER rank sees it after the exchange (Section 6: packed
 * blocks arrive in the consumer's slot; here they are read in place, through the locally derived offsets of
 * Section 5.2, instead of being scattered back first).  Computes the rows of the consumer's query blocks
 * only; a kept KV block the consumer owns is read from K / V, every other kept block from the consumer's
 * packed buffer as written by sparsp_demand_pack WITHOUT SPARSP_INCLUDE_LOCAL -- K and V of blocks owned by
 * other ranks are never touched.  Rows of other ranks' query blocks are left unwritten.
 *   mask, rank_of_block, union_mask, seg_offset, seg_total   as for / from sparsp_demand_pack
 *   consumer         0 .. n_ranks-1
 *   packed, packed_capacity_bytes, dst_base_bytes             the buffer sparsp_demand_pack filled, with the
 *                    same bases (NULL = dense); bases must be multiples of the tile size block*d*2
 *   O, lse           as for sparsp_sparse_attn_fwd */
SPARSP_API int sparsp_sparse_attn_fwd_packed(const sparsp_shape* shape, const void* Q, const void* K, const void* V,
                                             const uint32_t* mask, const int32_t* rank_of_block, int32_t n_ranks,
                                             int32_t consumer, const uint32_t* union_mask,
                                             const int64_t* seg_offset, const int64_t* seg_total, const void* packed,
                                             int64_t packed_capacity_bytes, const int64_t* dst_base_bytes,
                                             float softmax_scale, void* O, float* lse, void* workspace,
                                             void* stream);
SPARSP_API int sparsp_hop_mask(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                               int32_t n_ranks, int32_t consumer, int32_t producer, uint32_t* hop_mask,
                               void* stream);
/* One chunk of a hop (Section 7.1: a hop is cut into chunks of heads so that attention on a chunk can start as
 * soon as it has arrived): sparsp_hop_mask with the rows of heads outside [head_begin, head_end) zeroed as well. */
SPARSP_API int sparsp_hop_chunk_mask(const sparsp_shape* shape, const uint32_t* mask, const int32_t* rank_of_block,
                                     int32_t n_ranks, int32_t consumer, int32_t producer, int32_t head_begin,
                                     int32_t head_end, uint32_t* hop_mask, void* stream);
SPARSP_API int sparsp_attn_merge(const sparsp_shape* shape, const void* O_a, const float* lse_a, const void* O_b,
                                 const float* lse_b, void* O, float* lse, void* stream);
/* The same merge restricted to what one chunk of one hop produced (Section 7.1): only the rows of the query blocks
 * of `consumer` in heads [head_begin, head_end) are merged; every other row of O / lse is left untouched.
 *   rank_of_block  DEVICE int32 [NB] */
SPARSP_API int sparsp_attn_merge_rows(const sparsp_shape* shape, const void* O_a, const float* lse_a, const void* O_b,
                                      const float* lse_b, void* O, float* lse, const int32_t* rank_of_block,
                                      int32_t n_ranks, int32_t consumer, int32_t head_begin, int32_t head_end,
                                      void* stream);

/* The transfer list of the demand-routed exchange, derived from the demand counts alone (host arithmetic, no
 * GPU work).  Section 5.1: in round k = 0 .. P-2 consumer r receives from the producer at ring distance
 * k+1, p = (r - (k+1)) mod P, exactly the blocks it selected there.  Sections 5.2 / 6: those blocks are one
 * contiguous run of the consumer's buffer (heads ascending), so producer and consumer compute the same byte
 * ranges without exchanging any descriptor.  Section 7.1: a hop is cut into chunks of contiguous heads,
 * `steady_chunks` in every round but the last and `tail_chunks` in the last (never more than heads; chunk c
 * of C starts at head c*H/C).  Section 7.2: the chunks of a hop are listed in descending order of their
 * number of kept blocks (ties: lower head first), the sparsest last.
 *   cnt, seg_offset   in   HOST copies of sparsp_demand_pack's outputs (made WITHOUT SPARSP_INCLUDE_LOCAL),
 *                          int32 / int64 [B][P][P][H]
 *   transfers         out  HOST [capacity]; sorted by batch, consumer, round, order; a chunk without blocks is
 *                          listed with n_bytes = 0.  Offsets are relative to the consumer's buffer.
 *   n_transfers       out  B * P * sum over rounds of that round's chunk count (written even if the list does
 *                          not fit, in which case the call returns SPARSP_ERR_CAPACITY and writes nothing else) */
typedef struct sparsp_transfer {
  int32_t batch, consumer, producer, round; /* round = ring distance - 1 */
  int32_t order;                            /* position inside its hop */
  int32_t head_begin, head_end;             /* heads [head_begin, head_end) */
  int32_t reserved;
  int64_t entry_begin, n_entries;           /* entries (K tile + V tile of one block) of the consumer's buffer */
  int64_t byte_offset, n_bytes;             /* the same run in bytes */
} sparsp_transfer;
SPARSP_API int sparsp_exchange_plan(const sparsp_shape* shape, int32_t n_ranks, const int32_t* cnt,
                                    const int64_t* seg_offset, int32_t steady_chunks, int32_t tail_chunks,
                                    sparsp_transfer* transfers, int64_t capacity, int64_t* n_transfers);

/* Transfer runtime of the demand-routed exchange (Section 6.1: the five primitives Export, Publish, Fetch,
 * Release, Fence; Section 6.2: raw asynchronous peer copies of receiver-derived byte ranges; Section 6.3: a
 * bounded window of reusable slots whose dependencies are Publish and Release alone).
 *
 * One endpoint (`sparsp_xchg`) per rank.  A rank is a GPU of the node or, on one device, a virtual rank driven by
 * its own host thread with its own streams.  In round k = 0 .. P-2 rank p packs what consumer (p + k + 1) mod P
 * selected from it into slot (k mod window) of its own window (`use` = k below), and consumer r fetches from
 * producer (r - (k + 1)) mod P.  A slot holds the whole payload of one (consumer, producer) pair, laid out like that
 * pair's run of the consumer's buffer (heads ascending, blocks ascending), so a consumer derives any chunk's byte
 * range inside the slot from the demand counts: chunk.byte_offset - seg_offset[r][p][0] * entry bytes.
 *
 * Flags: 4-byte sequence numbers, one (publish, release) pair per (rank, slot), in a page of
 * sparsp_xchg_flag_bytes() bytes of HOST memory that every rank can read and write (pinned memory for the ranks of
 * one process, inter-process shared memory for one process per GPU); zero-filled by whoever creates it.  Publish and
 * Release store them from a host function enqueued on the given stream, i.e. in stream order after the pack
 * (Publish) or after the copies (Release); no kernel is launched and no kernel ever waits for another rank.  Every
 * wait -- sparsp_xchg_acquire for the release of the slot's previous content, sparsp_xchg_fetch for the
 * publication -- polls on the host for at most `wait_limit_us` and then fails with SPARSP_ERR_TIMEOUT (text in
 * sparsp_last_error()); the endpoint stays usable.
 *
 *   sparsp_xchg_export   Export: registers this rank's window (`slots`: `window` slots of `slot_bytes` each, DEVICE
 *                        memory the caller owns, 16-byte aligned) and the shared flag page; *out is the endpoint.
 *                        flags: 0, or SPARSP_XCHG_HOST_MEMORY -- slots and destinations are HOST memory, copies
 *                        are memcpy and flag stores happen at once (for multi-process tests of the protocol on
 *                        machines without a GPU; never chosen by the library itself).
 *   sparsp_xchg_connect  address under which this rank reaches `peer`'s window (the same pointer on one device; a
 *                        peer mapping of the other GPU's window on a node).
 *   sparsp_xchg_fence    Fence: call once per attention call on every rank, AFTER the caller's barrier across
 *                        ranks (and after this rank's copies of the previous call have completed).  Moves the
 *                        endpoint to the next epoch: flags of the previous call no longer satisfy any wait.
 *   sparsp_xchg_acquire  producer: slot of packing number `use` (use mod window) and its address; for use >= window
 *                        waits until the consumer of packing use - window has released it.
 *   sparsp_xchg_publish  producer: marks packing `use` as ready once the work enqueued on `stream` so far is done.
 *   sparsp_xchg_fetch    consumer: waits for producer's packing `use`, then enqueues ONE asynchronous copy of
 *                        [src_offset, src_offset + n_bytes) of that slot to `dst` (device memory of this rank) on
 *                        `copy_stream` (copy engines; no SM).  n_bytes = 0 only waits.
 *   sparsp_xchg_release  consumer: returns producer's slot of packing `use` once the copies enqueued on
 *                        `copy_stream` so far are done.
 *   sparsp_xchg_stats    out[8] (HOST): publications, fetches, releases, acquisitions that found the slot still in
 *                        use, bytes fetched, microseconds waited for releases, for publications, timeouts.
 *   sparsp_xchg_destroy  frees the endpoint (not the slots or the flag page).
 * `use` is 0 .. 65534.  Calls on one endpoint come from one host thread. */
#define SPARSP_XCHG_HOST_MEMORY 1
typedef struct sparsp_xchg sparsp_xchg;
SPARSP_API int sparsp_xchg_flag_bytes(int32_t n_ranks, int32_t window, int64_t* bytes);
SPARSP_API int sparsp_xchg_export(int32_t n_ranks, int32_t rank, int32_t window, int64_t slot_bytes, void* slots,
                                  void* flag_page, int64_t wait_limit_us, int32_t flags, sparsp_xchg** out);
SPARSP_API int sparsp_xchg_connect(sparsp_xchg* x, int32_t peer, void* peer_slots);
SPARSP_API int sparsp_xchg_fence(sparsp_xchg* x);
SPARSP_API int sparsp_xchg_acquire(sparsp_xchg* x, int64_t use, int32_t* slot, void** slot_ptr);
SPARSP_API int sparsp_xchg_publish(sparsp_xchg* x, int64_t use, void* stream);
SPARSP_API int sparsp_xchg_fetch(sparsp_xchg* x, int32_t producer, int64_t use, int64_t src_offset, void* dst,
                                 int64_t n_bytes, void* copy_stream);
SPARSP_API int sparsp_xchg_release(sparsp_xchg* x, int32_t producer, int64_t use, void* copy_stream);
SPARSP_API int sparsp_xchg_stats(sparsp_xchg* x, int64_t* out);
SPARSP_API int sparsp_xchg_destroy(sparsp_xchg* x);

/* The producer's pack of ONE hop (Section 6.1: for each producer-consumer pair the producer packs the payload into
 * the slot designated for it).  Writes, starting at `dst`, the K and V tiles of every block that `consumer` selected
 * from `producer` -- the entries seg_offset[consumer][producer][0] .. of the consumer's buffer, in that order (heads
 * ascending, blocks ascending; entry = K tile then V tile; rows at or beyond N are zero).  Only blocks `producer`
 * owns are read from K / V.  An entry that would end beyond dst_capacity_bytes is not written and the status word
 * becomes SPARSP_ERR_CAPACITY.  One batch item.
 *   union_mask, cnt, seg_offset   outputs of sparsp_demand_pack / sparsp_demand_plan_noalloc made WITHOUT
 *                                 SPARSP_INCLUDE_LOCAL (DEVICE)
 *   dst                           DEVICE, 16-byte aligned (a slot of the producer's window)
 *   workspace                     this rank's own (the call rewrites the workspace's entry table) */
SPARSP_API int sparsp_pack_segment(const sparsp_shape* shape, const uint32_t* union_mask, const int32_t* rank_of_block,
                                   int32_t n_ranks, int32_t consumer, int32_t producer, const int32_t* cnt,
                                   const int64_t* seg_offset, const void* K, const void* V, void* dst,
                                   int64_t dst_capacity_bytes, void* workspace, void* stream);

/* Planning without any allocation.  (No counterpart in the paper: an engineering variant of the
 * planning half of sparsp_demand_pack.)
 * For callers that are not allowed to allocate device memory -- for example a plug-in running inside a
 * host application that has handed all GPU memory to its own pool, or a latency-critical loop that
 * must never enter the driver's allocator -- and so cannot provide the workspace the other calls need.
 * Computes exactly what sparsp_demand_pack computes with SPARSP_PLAN_ONLY (same definitions, layouts
 * and argument meaning for union_mask, cnt, seg_offset, seg_total, volume_bytes; `flags` may only carry
 * SPARSP_INCLUDE_LOCAL) but keeps its scratch (per-rank ownership bit words and table bases) in a
 * 16.4 KB array that is part of the library image; every GPU that loads the library holds that array
 * until the process exits.  The call itself allocates and frees nothing, on the host or on the device.
 * Limits: n_ranks <= 64 and batch * n_ranks <= 1024, else SPARSP_ERR_CAPACITY (nothing is launched).
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call before any stream capture begins.  All calls on a device share the one array: it
 * keeps the previous call's contents, every word a call reads is rewritten by that call first (nothing
 * needs to start at zero), and two calls whose kernels may overlap on the GPU (different streams
 * without ordering) race on it -- serialise them. */
SPARSP_API int sparsp_demand_plan_noalloc(const sparsp_shape* shape, const uint32_t* mask,
                                          const int32_t* rank_of_block, int32_t n_ranks, int32_t flags,
                                          uint32_t* union_mask, int32_t* cnt, int64_t* seg_offset,
                                          int64_t* seg_total, int64_t* volume_bytes, void* stream);

/* Synchronises `stream` and returns the workspace's status word in *code (SPARSP_OK if no kernel
 * reported a problem since the last reset), then resets it. */
SPARSP_API int sparsp_status(void* workspace, void* stream, int32_t* code);

/* Diagnostic (no counterpart in the paper): launches one tiny kernel whose only wait is on a barrier nobody
 * arrives on, bounded by `limit_cycles` SM clock cycles (1 .. 1e8) -- the same bounded wait every kernel of the
 * library uses.  The wait runs out, the kernel writes SPARSP_ERR_TIMEOUT and the detail words (where = 99, CTA 0)
 * to the workspace's status words and returns normally; the next sparsp_status() reports it (and resets it), and
 * the context stays usable.  Nothing else is in flight in that kernel (no copy, no MMA).  For testing the
 * error path of bounded waits without any kernel actually being stuck; any workspace of >= 256 bytes will do. */
SPARSP_API int sparsp_selftest_wait_timeout(void* workspace, int64_t limit_cycles, void* stream);

/* Text of the calling thread's most recent error ("" if none). */
SPARSP_API const char* sparsp_last_error(void);

/* Number of kernels this library has launched in the calling process (for benchmarks). */
SPARSP_API int64_t sparsp_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPARSP_H_ */
