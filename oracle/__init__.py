"""CPU oracle for the SparSP single-device hot path -- TEST INFRASTRUCTURE, not product code.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline legs of ``bench.py`` may import
this package.  It shares nothing with the CUDA path: the arithmetic lives in ``sparsp_oracle.c``
(plain C, compiled by gcc) and in the few pure-Python definitions below.

Pins (see tests/test_oracle_*.py): every function here is checked against closed forms, brute
force, textbook special cases or library routines.  The one example of the paper that cannot be
pinned is the re-placement figure (23 -> 16 transferred blocks, Section 4.3): its mask exists only
as a picture, so nothing here reproduces it -- "parity unpinned" for that example alone.

Layouts are canonical and dense: Q/K/V ``[H][N][d]`` bf16, masks ``[H][NB][Wd]`` uint32 with KV
block ``j`` at bit ``j & 31`` of word ``j >> 5``.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparsp_oracle.c")
_LIB = os.path.join(_HERE, "libsparsp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


# ---------------------------------------------------------------------------------------------
# marshalling helpers
# ---------------------------------------------------------------------------------------------
def _u16(x) -> np.ndarray:
    """bf16 torch tensor (CPU) or uint16 array -> contiguous uint16 numpy array."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return np.ascontiguousarray(x.contiguous().view(torch.int16).numpy().view(np.uint16))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(v) -> ctypes.c_int64:
    return ctypes.c_int64(int(v))


def n_blocks(N: int, b: int) -> int:
    return (N + b - 1) // b


def n_words(NB: int) -> int:
    return (NB + 31) // 32


# ---------------------------------------------------------------------------------------------
# pure-Python definitions (host-side readings)
# ---------------------------------------------------------------------------------------------
def text_block_flags(n_video: int, n_text: int, b: int) -> np.ndarray:
    """is_text[j] = 1 iff block j holds at least one text token; tokens are ordered video first,
    then text, and blocks are flat runs of ``b`` tokens."""
    N = n_video + n_text
    NB = n_blocks(N, b)
    flags = np.zeros(NB, dtype=np.uint8)
    for j in range(NB):
        last = min((j + 1) * b, N) - 1
        if n_text > 0 and last >= n_video:
            flags[j] = 1
    return flags


def resolve_topk(pct: int, nb_video: int) -> int:
    """"top-k = pct % of blocks": integer ceiling of pct*nb_video/100, clamped to [1, nb_video]."""
    k = -(-pct * nb_video // 100)
    return max(1, min(nb_video, k))


def placement_contiguous(NB: int, P: int) -> np.ndarray:
    """Naive contiguous sequence partition: rank(j) = floor(j*P/NB)."""
    return np.array([(j * P) // NB for j in range(NB)], dtype=np.int32)


def placement_periodic(NB: int, P: int, b: int, frame_tokens: int, n_video: int) -> np.ndarray:
    """Interval-periodic layout (Eq. "periodic-placement"): each frame is cut into P contiguous
    spatial intervals and interval g belongs to rank g in every frame.  With B = frame_tokens/b
    blocks per frame and s the in-frame block index this is floor(P*s/B); for frames that are not a
    whole number of blocks the block's first token decides: floor(P*((j*b) mod F)/F).  Blocks that
    start in the text tail are dealt round-robin (j mod P)."""
    out = np.zeros(NB, dtype=np.int32)
    for j in range(NB):
        first = j * b
        if first >= n_video:
            out[j] = j % P
        else:
            out[j] = (P * (first % frame_tokens)) // frame_tokens
    return out


def placement_permutation(rank_of_block: np.ndarray, P: int, N: int, b: int):
    """Section 4.3: the placement as a deterministic permutation from logical block coordinates to
    (rank, offset) pairs, at the granularity of whole KV blocks.  Slots are ordered by rank, and inside a rank
    by logical block index.  Returns (block_of_slot [NB], token_offset_of_slot [NB+1], first_slot_of_rank
    [P+1]): slot s holds logical block block_of_slot[s], whose tokens start at token_offset_of_slot[s] in the
    permuted sequence (the sequence's last block may be shorter than b)."""
    NB = len(rank_of_block)
    block_of_slot, first = [], [0]
    for r in range(P):
        block_of_slot += [j for j in range(NB) if rank_of_block[j] == r]
        first.append(len(block_of_slot))
    off = [0]
    for j in block_of_slot:
        off.append(off[-1] + min(b, N - j * b))
    return (np.array(block_of_slot, np.int32), np.array(off, np.int64), np.array(first, np.int32))


def permute_tokens(X, block_of_slot, token_offset_of_slot, b: int, inverse: bool = False):
    """X [H][N][d] -> the same tokens in permuted order (or back, with inverse=True)."""
    H, N, d = X.shape
    Y = X.clone()
    for s, j in enumerate(block_of_slot):
        n_j = min(b, N - int(j) * b)
        lo_new, lo_old = int(token_offset_of_slot[s]), int(j) * b
        if inverse:
            Y[:, lo_old:lo_old + n_j] = X[:, lo_new:lo_new + n_j]
        else:
            Y[:, lo_new:lo_new + n_j] = X[:, lo_old:lo_old + n_j]
    return Y


def sharing_histogram(mask: np.ndarray, rank_of_block: np.ndarray, P: int) -> np.ndarray:
    """Section 3.2: for each remote K block a rank receives (per head), the fraction of that rank's local Q
    blocks that access it.  hist[r][q], q = 0..100, counts the (head, remote block) pairs of consumer r whose
    fraction, in whole percent rounded down, is q (a received block is accessed by at least one local Q block,
    so a fraction below 1 % lands in bin 0)."""
    H, NB, _ = mask.shape
    hist = np.zeros((P, 101), np.int64)
    for r in range(P):
        local = [i for i in range(NB) if rank_of_block[i] == r]
        for h in range(H):
            for j in range(NB):
                if rank_of_block[j] == r:
                    continue
                c = sum((int(mask[h, i, j >> 5]) >> (j & 31)) & 1 for i in local)
                if c > 0:
                    hist[r, (100 * c) // len(local)] += 1
    return hist


# ---------------------------------------------------------------------------------------------
# step 1
# ---------------------------------------------------------------------------------------------
def pool(x, b: int) -> np.ndarray:
    xs = _u16(x)
    H, N, d = xs.shape
    NB = n_blocks(N, b)
    out = np.empty((H, NB, d), dtype=np.float32)
    lib().oracle_pool(_p(xs), _i64(H), _i64(N), _i64(d), _i64(b), _p(out))
    return out


def scores(pq: np.ndarray, pk: np.ndarray) -> np.ndarray:
    pq = np.ascontiguousarray(pq, dtype=np.float32)
    pk = np.ascontiguousarray(pk, dtype=np.float32)
    H, NB, d = pq.shape
    out = np.empty((H, NB, NB), dtype=np.float32)
    lib().oracle_scores(_p(pq), _p(pk), _i64(H), _i64(NB), _i64(d), _p(out))
    return out


def scores_f64(pq: np.ndarray, pk: np.ndarray) -> np.ndarray:
    pq = np.ascontiguousarray(pq, dtype=np.float32)
    pk = np.ascontiguousarray(pk, dtype=np.float32)
    H, NB, d = pq.shape
    out = np.empty((H, NB, NB), dtype=np.float64)
    lib().oracle_scores_f64(_p(pq), _p(pk), _i64(H), _i64(NB), _i64(d), _p(out))
    return out


def topk_mask(sc: np.ndarray, is_text: np.ndarray, k: int):
    """-> (mask [H][NB][Wd] uint32, kv_list [H][NB][kept] int32 ascending, kv_count [H][NB])."""
    sc = np.ascontiguousarray(sc, dtype=np.float32)
    is_text = np.ascontiguousarray(is_text, dtype=np.uint8)
    H, NB, _ = sc.shape
    Wd = n_words(NB)
    kept_cap = min(k, int((is_text == 0).sum())) + int(is_text.sum())
    mask = np.empty((H, NB, Wd), dtype=np.uint32)
    kv_list = np.empty((H, NB, kept_cap), dtype=np.int32)
    kv_count = np.empty((H, NB), dtype=np.int32)
    lib().oracle_topk_mask(_p(sc), _p(is_text), _i64(H), _i64(NB), _i64(k), _p(mask), _p(kv_list),
                           _i64(kept_cap), _p(kv_count))
    return mask, kv_list, kv_count


def exp2c(x: np.ndarray) -> np.ndarray:
    """The fixed-arithmetic 2^x of the CDF-threshold mode (fp32)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    y = np.empty_like(x)
    lib().oracle_exp2c_array(_p(x), _i64(x.size), _p(y))
    return y


def cdf_mask(sc: np.ndarray, is_text: np.ndarray, tau: float, scale: float):
    """CDF-threshold selection -> (mask [H][NB][Wd] uint32, kv_count [H][NB])."""
    sc = np.ascontiguousarray(sc, dtype=np.float32)
    is_text = np.ascontiguousarray(is_text, dtype=np.uint8)
    H, NB, _ = sc.shape
    mask = np.empty((H, NB, n_words(NB)), dtype=np.uint32)
    kv_count = np.empty((H, NB), dtype=np.int32)
    lib().oracle_cdf_mask(_p(sc), _p(is_text), _i64(H), _i64(NB), ctypes.c_float(tau), ctypes.c_float(scale),
                          _p(mask), _p(kv_count))
    return mask, kv_count


def block_mask_cdf(Q, K, b: int, tau: float, n_text: int = 0, scale: float = 0.0):
    """Whole step 1 in CDF-threshold mode (scale 0 means 1/sqrt(d))."""
    H, N, d = Q.shape
    pq, pk = pool(Q, b), pool(K, b)
    sc = scores(pq, pk)
    is_text = text_block_flags(N - n_text, n_text, b)
    sc_scale = np.float32(scale) if scale > 0 else np.float32(1.0) / np.sqrt(np.float32(d))
    mask, kv_count = cdf_mask(sc, is_text, tau, float(sc_scale))
    return dict(mask=mask, kv_count=kv_count, pq=pq, pk=pk, scores=sc, is_text=is_text, scale=float(sc_scale))


def block_mask(Q, K, b: int, k: int, n_text: int = 0):
    """Whole step 1: pool -> scores -> top-k.  Returns dict with mask, kv_list, kv_count, pq, pk."""
    H, N, d = Q.shape
    pq, pk = pool(Q, b), pool(K, b)
    sc = scores(pq, pk)
    is_text = text_block_flags(N - n_text, n_text, b)
    mask, kv_list, kv_count = topk_mask(sc, is_text, k)
    return dict(mask=mask, kv_list=kv_list, kv_count=kv_count, pq=pq, pk=pk, scores=sc,
                is_text=is_text)


# ---------------------------------------------------------------------------------------------
# step 2
# ---------------------------------------------------------------------------------------------
def demand(mask: np.ndarray, rank_of_block: np.ndarray, P: int, b: int, d: int,
           include_local: bool = False, w_bytes: int = 2):
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    rank_of_block = np.ascontiguousarray(rank_of_block, dtype=np.int32)
    H, NB, Wd = mask.shape
    U = np.empty((P, H, Wd), dtype=np.uint32)
    cnt = np.empty((P, P, H), dtype=np.int32)
    seg_off = np.empty((P, P, H), dtype=np.int64)
    total = np.empty((P,), dtype=np.int64)
    volume = np.empty((P,), dtype=np.int64)
    lib().oracle_demand(_p(mask), _p(rank_of_block), _i64(H), _i64(NB), _i64(P), _i64(b), _i64(d),
                        _i64(w_bytes), ctypes.c_int(int(include_local)), _p(U), _p(cnt),
                        _p(seg_off), _p(total), _p(volume))
    return dict(U=U, cnt=cnt, seg_off=seg_off, total=total, volume=volume)


def pack(K, V, U: np.ndarray, rank_of_block: np.ndarray, b: int, P: int, total: np.ndarray,
         include_local: bool = False, dst_base: np.ndarray | None = None) -> np.ndarray:
    """-> packed bytes (uint8).  Default destination bases are the dense prefix of ``total``."""
    Ks, Vs = _u16(K), _u16(V)
    H, N, d = Ks.shape
    entry = 2 * b * d * 2
    if dst_base is None:
        dst_base = np.concatenate([[0], np.cumsum(total)[:-1]]).astype(np.int64) * entry
    dst_base = np.ascontiguousarray(dst_base, dtype=np.int64)
    size = int(max(dst_base[r] + total[r] * entry for r in range(P))) if P else 0
    out = np.zeros(size, dtype=np.uint8)
    U = np.ascontiguousarray(U, dtype=np.uint32)
    rank_of_block = np.ascontiguousarray(rank_of_block, dtype=np.int32)
    lib().oracle_pack(_p(Ks), _p(Vs), _p(U), _p(rank_of_block), _i64(H), _i64(N), _i64(d), _i64(b),
                      _i64(P), ctypes.c_int(int(include_local)), _p(dst_base), _p(out))
    return out


def exchange_plan(cnt: np.ndarray, seg_off: np.ndarray, b: int, d: int, steady_chunks: int = 1,
                  tail_chunks: int = 1, w_bytes: int = 2):
    """The transfer list of the demand-routed exchange for one batch item, written out from the paper's
    description (plain loops; cnt and seg_off as returned by demand() without include_local):
      * Section 5.1: in round k = 0 .. P-2 every consumer r receives from the producer at ring distance k+1,
        p = (r - (k+1)) mod P, exactly the blocks it selected from that producer;
      * Section 5.2 / 6: the blocks of one (consumer, producer) pair are one contiguous run of the consumer's
        buffer, heads ascending, so both ends derive every byte range from the demand counts alone;
      * Section 7.1: a hop is cut into chunks of contiguous heads, `steady_chunks` of them in every round but
        the last, `tail_chunks` in the last (never more chunks than heads; chunk c starts at head c*H // C);
      * Section 7.2: the chunks of a hop go in descending order of their number of kept blocks (ties: lower
        head first), so that the sparsest chunk, whose attention is the shortest, comes last.
    -> list of dicts (consumer, producer, round, order, head_begin, head_end, entry_begin, n_entries,
       byte_offset, n_bytes), sorted by consumer, round, order; offsets relative to the consumer's buffer."""
    P, _, H = cnt.shape
    entry = 2 * b * d * w_bytes
    out = []
    for r in range(P):
        for k in range(P - 1):
            p = (r - (k + 1)) % P
            C = tail_chunks if k == P - 2 else steady_chunks
            C = max(1, min(C, H))
            chunks = []
            for c in range(C):
                h0, h1 = (c * H) // C, ((c + 1) * H) // C
                n = int(sum(int(cnt[r, p, h]) for h in range(h0, h1)))
                chunks.append((h0, h1, n))
            chunks.sort(key=lambda t: (-t[2], t[0]))
            for order, (h0, h1, n) in enumerate(chunks):
                e0 = int(seg_off[r, p, h0])
                out.append(dict(consumer=r, producer=p, round=k, order=order, head_begin=h0, head_end=h1,
                                entry_begin=e0, n_entries=n, byte_offset=e0 * entry, n_bytes=n * entry))
    return out


# ---------------------------------------------------------------------------------------------
# step 3
# ---------------------------------------------------------------------------------------------
def attn_rows(Q, K, V, mask: np.ndarray, b: int, units, scale: float | None = None):
    """Attention for the listed (head, query block) units.  -> (out [U][b][d] fp32, lse [U][b])."""
    Qs, Ks, Vs = _u16(Q), _u16(K), _u16(V)
    H, N, d = Qs.shape
    units = np.asarray(units, dtype=np.int32).reshape(-1, 2)
    uh = np.ascontiguousarray(units[:, 0])
    ub = np.ascontiguousarray(units[:, 1])
    n = len(uh)
    out = np.zeros((n, b, d), dtype=np.float32)
    lse = np.zeros((n, b), dtype=np.float32)
    sc = (1.0 / math.sqrt(d)) if scale is None else float(scale)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    lib().oracle_attn_rows(_p(Qs), _p(Ks), _p(Vs), _p(mask), _i64(H), _i64(N), _i64(d), _i64(b),
                           ctypes.c_double(sc), _p(uh), _p(ub), _i64(n), _p(out), _p(lse))
    return out, lse


def attn_all(Q, K, V, mask: np.ndarray, b: int, scale: float | None = None):
    """Attention for every (head, query block); -> out [H][N][d] fp32, lse [H][N]."""
    H, N, d = Q.shape
    NB = n_blocks(N, b)
    units = [(h, i) for h in range(H) for i in range(NB)]
    out, lse = attn_rows(Q, K, V, mask, b, units, scale)
    out = out.reshape(H, NB * b, d)[:, :N]
    lse = lse.reshape(H, NB * b)[:, :N]
    return np.ascontiguousarray(out), np.ascontiguousarray(lse)


def attn_dense_masked(Q, K, V, mask: np.ndarray, b: int, scale: float | None = None):
    """Textbook masked-row form (tiny inputs).  -> (out [H][N][d] fp32, rowsum [H][N] fp64)."""
    Qs, Ks, Vs = _u16(Q), _u16(K), _u16(V)
    H, N, d = Qs.shape
    out = np.zeros((H, N, d), dtype=np.float32)
    rowsum = np.zeros((H, N), dtype=np.float64)
    sc = (1.0 / math.sqrt(d)) if scale is None else float(scale)
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    lib().oracle_attn_dense_masked(_p(Qs), _p(Ks), _p(Vs), _p(mask), _i64(H), _i64(N), _i64(d),
                                   _i64(b), ctypes.c_double(sc), _p(out), _p(rowsum))
    return out, rowsum


# ---------------------------------------------------------------------------------------------
# consumer-side pipeline ("next" rows): per-hop masks and log-sum-exp merging of partial results
# ---------------------------------------------------------------------------------------------
def hop_mask(mask: np.ndarray, rank_of_block: np.ndarray, consumer: int, producer: int,
             head_begin: int = 0, head_end: int | None = None) -> np.ndarray:
    """Rows of the consumer rank's query blocks, restricted to the KV blocks the producer owns
    (the blocks that travel in one hop of the demand-routed exchange, Section 5.1); all else zero.
    With a head range: one chunk of that hop (Section 7.1), i.e. the other heads are zero as well."""
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    H, NB, Wd = mask.shape
    head_end = H if head_end is None else head_end
    own = np.zeros(Wd, dtype=np.uint32)
    for j in range(NB):
        if rank_of_block[j] == producer:
            own[j >> 5] |= np.uint32(1 << (j & 31))
    out = np.zeros_like(mask)
    for i in range(NB):
        if rank_of_block[i] == consumer:
            for h in range(head_begin, head_end):
                out[h, i, :] = mask[h, i, :] & own
    return out


def attn_merge(oa: np.ndarray, la: np.ndarray, ob: np.ndarray, lb: np.ndarray):
    """Log-sum-exp merge of two partial results over disjoint key sets. oa/ob [..., d] fp32, la/lb [...]."""
    oa = np.ascontiguousarray(oa, dtype=np.float32)
    ob = np.ascontiguousarray(ob, dtype=np.float32)
    la = np.ascontiguousarray(la, dtype=np.float32)
    lb = np.ascontiguousarray(lb, dtype=np.float32)
    d = oa.shape[-1]
    rows = oa.size // d
    out = np.empty_like(oa)
    lse = np.empty_like(la)
    lib().oracle_attn_merge(_p(oa), _p(la), _p(ob), _p(lb), _i64(rows), _i64(d), _p(out), _p(lse))
    return out, lse


def consumer_view(K, V, packed: np.ndarray, dem: dict, rank_of_block: np.ndarray, b: int, consumer: int,
                  dst_base: np.ndarray | None = None):
    """What consumer rank r can see after the exchange: its own K/V blocks from the original tensors,
    the blocks it demanded from other ranks out of ITS packed buffer (entry order: producer ascending,
    head ascending, block ascending; entry = K tile then V tile), and NaN everywhere else -- so that an
    attention over this view proves that nothing but local blocks and packed entries is needed.
    -> (K_r, V_r) fp32 [H][NB*b][d]."""
    Ks, Vs = _u16(K), _u16(V)
    H, N, d = Ks.shape
    NB = n_blocks(N, b)
    P = dem["cnt"].shape[0]
    entry = 2 * b * d * 2
    if dst_base is None:
        dst_base = np.concatenate([[0], np.cumsum(dem["total"])[:-1]]).astype(np.int64) * entry

    def bf16_to_f32(u16):
        return (u16.astype(np.uint32) << 16).view(np.float32)

    Kr = np.full((H, NB * b, d), np.nan, dtype=np.float32)
    Vr = np.full((H, NB * b, d), np.nan, dtype=np.float32)
    for j in range(NB):
        if rank_of_block[j] == consumer:
            n_j = min(b, N - j * b)
            Kr[:, j * b:j * b + n_j] = bf16_to_f32(Ks[:, j * b:j * b + n_j])
            Vr[:, j * b:j * b + n_j] = bf16_to_f32(Vs[:, j * b:j * b + n_j])
    for p in range(P):
        if p == consumer:
            continue
        for h in range(H):
            words = dem["U"][consumer, h]
            pos = int(dem["seg_off"][consumer, p, h])
            for j in range(NB):
                if rank_of_block[j] == p and (int(words[j >> 5]) >> (j & 31)) & 1:
                    off = int(dst_base[consumer]) + pos * entry
                    tile = packed[off:off + entry].view(np.uint16).reshape(2, b, d)
                    Kr[h, j * b:(j + 1) * b] = bf16_to_f32(tile[0])
                    Vr[h, j * b:(j + 1) * b] = bf16_to_f32(tile[1])
                    pos += 1
    return Kr, Vr
