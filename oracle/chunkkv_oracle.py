"""CPU oracle for ChunkKV prefill-time KV-cache compression (fp64, numpy).

THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH. It is a plain, slow, step-by-step
statement of what the method computes, used only to check the CUDA kernels and to
serve as the timed CPU baseline. It shares no code with the CUDA path and must never
be imported by the library or its Python binding.

What it follows (ChunkKV paper):
  * Algorithm 3 ("ChunkKV Implementation", appendix "Implementation Details") is the
    primary text: observe-window scores, per-chunk sums over queries and chunk tokens,
    k = min(floor((L_max - w) / c), C), top-k chunks, whole chunks kept, the last w
    tokens always kept, kept indices in ascending order, index_select on K and V.
  * Algorithm 1 and the paragraph after it (section "Chunk Based KV Compression") for
    the notation (w, c, L_max) and "indices ... preserve the original sequence order".
  * Algorithm 2 (section "Layer-Wise Index Reuse") for which layers compute indices and
    which reuse them.

Readings taken where the paper is silent (each is a choice, not something the paper
prints; parity on these choices is UNPINNED by the paper itself):
  * "Attention scores" are the softmax attention probabilities of the window queries,
    softmax(q k^T / sqrt(d)) over the keys each window query can see in a causal model
    (all prefix keys, plus window keys at or before its own position).
  * With grouped-query attention, the scores of the G query heads that share one KV head
    are summed, and chunks are selected independently per KV head.
  * The chunk grid covers the prefix [0, L-w) only (origin 0, stride c, last chunk
    clipped); the window is appended separately, so it never consumes chunk budget.
  * Ties between chunk scores go to the lower chunk index.

What pins it (tests/test_oracle_*.py): brute-force enumeration of chunk subsets, softmax
row sums, mass conservation, the uniform-attention closed form (q = 0), a dominant-key
limit, an e-ratio logit case that fixes the 1/sqrt(d) scale, an independent library
softmax, library top-k for c = 1, the budget/ordering/window invariants, reuse identity;
for Algorithm 1's budget rule (select_alg1): hand-worked cases, brute-force enumeration of
chunk subsets followed by the cut, and the exact output length; for the prefill-tail adapters
(rope, window_queries, gather_paged; tests/test_oracle_adapters.py): norm preservation, identity
at angle 0, relative-position dependence, complex multiplication, un-paging to the dense gather.

Layouts (numpy arrays; bf16 tensors arrive as uint16 bit patterns):
  q_obs [Hq, w, d]   K, V [Hkv, L, d]   token scores [Hkv, P]   chunk scores [Hkv, C]
  idx [Hkv, n_max] int32 (padding -1)   out_K, out_V [Hkv, n_max, d] uint16 (padding 0)
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------- helpers
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    u32 = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def num_chunks(L: int, w: int, c: int) -> int:
    """C = ceil(P / c) with P = L - w (Algorithm 3, "Number of chunks", prefix grid)."""
    P = L - w
    return -(-P // c) if P > 0 else 0


def num_kept_chunks(L: int, w: int, c: int, budget: int) -> int:
    """k = min(floor((L_max - w) / c), C)  (Algorithm 3, "Limit k to available chunks")."""
    return min((budget - w) // c, num_chunks(L, w, c))


def out_len(L: int, w: int, c: int, budget: int) -> int:
    """n_max = k * c + w: row stride of the compacted outputs."""
    return num_kept_chunks(L, w, c, budget) * c + w


def _check(L: int, w: int, c: int, budget: int) -> None:
    if w < 1 or c < 1 or L < w or budget < w:
        raise ValueError("need w >= 1, c >= 1, L >= w, budget >= w")


# --------------------------------------------------------------------------- step 1: scores
def attention_probs(q_obs_head: np.ndarray, K_head: np.ndarray, w: int) -> np.ndarray:
    """Softmax attention of one KV head's window queries over the keys they can see.

    q_obs_head [R, d] fp64, rows ordered (g, r) -> g * w + r; K_head [L, d] fp64.
    Row (g, r) sits at absolute position P + r and sees key j iff j <= P + r.
    Returns p [R, L] (zeros on keys a row cannot see).
    (Algorithm 3: "A <- q_observe K^T"; softmax and 1/sqrt(d) are this oracle's reading.)
    """
    R, d = q_obs_head.shape
    L = K_head.shape[0]
    P = L - w
    S = (q_obs_head @ K_head.T) / math.sqrt(d)                   # [R, L]
    r = np.arange(R) % w                                         # window position of each row
    visible = np.arange(L)[None, :] <= (P + r)[:, None]
    S = np.where(visible, S, -np.inf)
    m = S.max(axis=1, keepdims=True)
    E = np.exp(S - m)                                            # exp(-inf) = 0 on hidden keys
    return E / E.sum(axis=1, keepdims=True)


def token_scores(q_obs: np.ndarray, K: np.ndarray, Hq: int, Hkv: int, w: int) -> np.ndarray:
    """t[h, j] = sum over the R = w * G rows of KV head h of p[i, j], for prefix keys j < P.

    (Algorithm 3: the inner sum over q of A[q, j]; the sum over the G grouped query heads
    is this oracle's GQA reading.)  q_obs, K: bf16 bit patterns.
    """
    G = Hq // Hkv
    if G * Hkv != Hq:
        raise ValueError("Hq must be a multiple of Hkv")
    L, d = K.shape[1], K.shape[2]
    P = L - w
    q = bf16_bits_to_f64(q_obs).reshape(Hkv, G * w, d)
    out = np.zeros((Hkv, P), dtype=np.float64)
    for h in range(Hkv):
        p = attention_probs(q[h], bf16_bits_to_f64(K[h]), w)
        out[h] = p[:, :P].sum(axis=0)
    return out


# --------------------------------------------------------------------------- step 2: chunk sums
def chunk_scores(t: np.ndarray, c: int) -> np.ndarray:
    """score[h, ch] = sum of t[h, j] for j in [ch*c, min((ch+1)*c, P)).

    (Algorithm 3, "Vectorized Chunk Score Calculation"; Algorithm 1, "Chunk Attention
    Score Calculation".)
    """
    Hkv, P = t.shape
    C = -(-P // c) if P > 0 else 0
    out = np.zeros((Hkv, C), dtype=np.float64)
    for ch in range(C):
        start, end = ch * c, min((ch + 1) * c, P)
        out[:, ch] = t[:, start:end].sum(axis=1)
    return out


# --------------------------------------------------------------------------- step 3: select
def select_chunks(scores_head: np.ndarray, k: int) -> np.ndarray:
    """Ids of the k highest-scoring chunks of one head, ascending; ties -> lower id.

    (Algorithm 3, "kept_chunks <- Top-K(chunk_scores, k)".)
    """
    if k <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(-np.asarray(scores_head, dtype=np.float64), kind="stable")
    return np.sort(order[:k])


def kept_indices(kept: Sequence[int], L: int, w: int, c: int, n_max: int) -> np.ndarray:
    """Ascending token indices of the kept chunks, then the window P..L-1, padded with -1.

    (Algorithm 3, "Build selection mask" / "Always keep most recent tokens" /
    "indices <- nonzero(mask)".)
    """
    P = L - w
    mask = np.zeros(L, dtype=bool)
    for ch in kept:
        mask[ch * c:min((ch + 1) * c, P)] = True
    mask[P:L] = True
    idx = np.nonzero(mask)[0].astype(np.int32)
    out = np.full(n_max, -1, dtype=np.int32)
    out[:idx.size] = idx
    return out


def select(scores: np.ndarray, L: int, w: int, c: int, budget: int) -> np.ndarray:
    """idx [Hkv, n_max] from chunk scores [Hkv, C]."""
    _check(L, w, c, budget)
    k = num_kept_chunks(L, w, c, budget)
    n_max = k * c + w
    Hkv = scores.shape[0]
    out = np.empty((Hkv, n_max), dtype=np.int32)
    for h in range(Hkv):
        out[h] = kept_indices(select_chunks(scores[h], k), L, w, c, n_max)
    return out


# --------------------------------------------------------------------------- Algorithm 1's budget rule
# The alternative selection policy printed in Algorithm 1 (section "Chunk Based KV Compression")
# and the paragraph after it: k = floor(L_max / c) chunks are selected, their tokens are taken in
# the original order, only the first L_max - w of them are kept, and the observe window takes the
# last w places. Compression-ratio budgets (the 10 % / 20 % / 30 % settings of the experiments)
# are L_max = floor(ratio * L). Same readings as above for everything the algorithm leaves open
# (chunk grid over the prefix, ties to the lower chunk id).
def budget_from_ratio(L: int, ratio: float) -> int:
    """L_max for a compression ratio (fraction of the L tokens that is kept)."""
    if not (0.0 <= ratio <= 1.0):
        raise ValueError("ratio must lie in [0, 1]")
    return int(math.floor(ratio * L))


def num_kept_chunks_alg1(L: int, w: int, c: int, budget: int) -> int:
    """k = floor(L_max / c), limited to the chunks that exist. (Algorithm 1, "Top-K Chunk Selection".)"""
    _check(L, w, c, budget)
    return min(budget // c, num_chunks(L, w, c))


def out_len_alg1(L: int, w: int, c: int, budget: int) -> int:
    """Row count of the outputs: at most L_max - w selected tokens, then the window."""
    return min(num_kept_chunks_alg1(L, w, c, budget) * c, budget - w) + w


def kept_indices_alg1(kept: Sequence[int], L: int, w: int, c: int, budget: int, n_max: int) -> np.ndarray:
    """Tokens of the kept chunks in ascending order, cut to the first L_max - w, then the window.

    (Algorithm 1, "Compression" and "Concatenation": K' <- concat(K'[0 : L_max - w], K[T_k - w : T_k]).)
    """
    P = L - w
    sel: List[int] = []
    for ch in sorted(int(v) for v in kept):
        sel.extend(range(ch * c, min((ch + 1) * c, P)))
    sel = sel[:budget - w]
    idx = np.asarray(sel + list(range(P, L)), dtype=np.int32)
    out = np.full(n_max, -1, dtype=np.int32)
    out[:idx.size] = idx
    return out


def select_alg1(scores: np.ndarray, L: int, w: int, c: int, budget: int) -> np.ndarray:
    """idx [Hkv, n_max] from chunk scores [Hkv, C] under Algorithm 1's budget rule."""
    k = num_kept_chunks_alg1(L, w, c, budget)
    n_max = out_len_alg1(L, w, c, budget)
    Hkv = scores.shape[0]
    out = np.empty((Hkv, n_max), dtype=np.int32)
    for h in range(Hkv):
        out[h] = kept_indices_alg1(select_chunks(scores[h], k), L, w, c, budget, n_max)
    return out


# --------------------------------------------------------------------------- step 4: gather
def gather(K: np.ndarray, V: np.ndarray, idx: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """out_K[h, n] = K[h, idx[h, n]] (bit copies), zero rows where idx is -1.

    (Algorithm 3, "K' <- index_select(K, indices)"; Algorithm 2, the two index_select lines.)
    """
    Hkv, n_max = idx.shape
    d = K.shape[2]
    out_K = np.zeros((Hkv, n_max, d), dtype=K.dtype)
    out_V = np.zeros((Hkv, n_max, d), dtype=V.dtype)
    for h in range(Hkv):
        for n in range(n_max):
            j = int(idx[h, n])
            if j >= 0:
                out_K[h, n] = K[h, j]
                out_V[h, n] = V[h, j]
    return out_K, out_V


# --------------------------------------------------------------------------- one layer
def compress_layer(q_obs: np.ndarray, K: np.ndarray, V: np.ndarray, Hq: int, Hkv: int,
                   w: int, c: int, budget: int, reuse_idx: Optional[np.ndarray] = None,
                   ) -> Dict[str, np.ndarray]:
    """Score -> chunk-sum -> top-k -> gather for one layer (all KV heads).

    With ``reuse_idx`` the scoring and selection are skipped and the given indices are used
    (Algorithm 2, the else-branch). Returns out_K, out_V, idx and, when computed, the
    token and chunk scores.
    """
    L = K.shape[1]
    _check(L, w, c, budget)
    res: Dict[str, np.ndarray] = {}
    if reuse_idx is None:
        t = token_scores(q_obs, K, Hq, Hkv, w)
        s = chunk_scores(t, c)
        idx = select(s, L, w, c, budget)
        res["token_scores"], res["chunk_scores"] = t, s
    else:
        idx = np.array(reuse_idx, dtype=np.int32, copy=True)
    out_K, out_V = gather(K, V, idx)
    res.update(out_K=out_K, out_V=out_V, idx=idx)
    return res


def compress_layer_alg1(q_obs: np.ndarray, K: np.ndarray, V: np.ndarray, Hq: int, Hkv: int,
                        w: int, c: int, budget: int) -> Dict[str, np.ndarray]:
    """One layer under Algorithm 1's budget rule: same scores, select_alg1, same gather."""
    L = K.shape[1]
    t = token_scores(q_obs, K, Hq, Hkv, w)
    s = chunk_scores(t, c)
    idx = select_alg1(s, L, w, c, budget)
    out_K, out_V = gather(K, V, idx)
    return dict(token_scores=t, chunk_scores=s, idx=idx, out_K=out_K, out_V=out_V)


# --------------------------------------------------------------------------- many layers
def compress_model(layers: Sequence[Tuple[np.ndarray, np.ndarray, np.ndarray]], Hq: int,
                   Hkv: int, w: int, c, budget: int, n_reuse: int = 1,
                   ) -> List[Dict[str, np.ndarray]]:
    """Layer-wise index reuse (Algorithm 2).

    Layer l computes its own indices iff l mod n_reuse == 0; otherwise it takes the
    indices stored for layer floor(l / n_reuse) * n_reuse. Every layer gathers.
    ``layers`` is a sequence of (q_obs, K, V).

    ``c`` is one chunk size for all layers or one per layer (the hybrid of the paper's section on
    chunk- and token-level layers: chunks in the first layers, c = 1 in the rest). A layer that
    reuses indices has no chunk size of its own: it takes its source layer's.
    """
    cs = [int(c)] * len(layers) if np.isscalar(c) else [int(v) for v in c]
    if len(cs) != len(layers):
        raise ValueError("one chunk size per layer expected")
    store: Dict[int, np.ndarray] = {}
    out = []
    for l, (q_obs, K, V) in enumerate(layers):
        if l % n_reuse == 0:
            res = compress_layer(q_obs, K, V, Hq, Hkv, w, cs[l], budget)
            store[l] = res["idx"]
        else:
            src = (l // n_reuse) * n_reuse
            res = compress_layer(q_obs, K, V, Hq, Hkv, w, cs[src], budget, reuse_idx=store[src])
        out.append(res)
    return out


# --------------------------------------------------------------------------- diagnostics
def jaccard(idx_a: np.ndarray, idx_b: np.ndarray) -> float:
    """|A n B| / |A u B| of two kept-index lists (padding -1 ignored).

    (Section "Layer-Wise Index Reuse": adjacent-layer similarity of preserved indices.)
    """
    a = set(int(v) for v in np.asarray(idx_a).ravel() if v >= 0)
    b = set(int(v) for v in np.asarray(idx_b).ravel() if v >= 0)
    u = len(a | b)
    return (len(a & b) / u) if u else 1.0


# --------------------------------------------------------------------------- prefill-tail inputs and paged outputs
# The paper runs the compression at the end of prefill, on the queries of the last w positions
# ("q_observe <- Q[T_q - w : T_q]", Algorithm 3; section "Efficiency Analysis": compression happens
# once, after prefill, and the compacted cache then serves decoding). In a model those queries sit
# in the layer's fused QKV projection output, before the rotary position embedding, and the
# compacted rows go to the decode cache, which serving systems keep in pages. The three functions
# below state those two adapters; nothing in them changes what is selected.
def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to bf16 (round to nearest even, through fp32) and return the bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotary position embedding in the rotate-half convention, fp64.

    x [..., d]; cos, sin [..., d/2] (broadcast against x's leading dims): the pair (x[i], x[i + d/2])
    is rotated by the angle whose cosine / sine are cos[i] / sin[i].
    """
    d = x.shape[-1]
    h = d // 2
    x1, x2 = x[..., :h], x[..., h:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def window_queries(qkv: np.ndarray, Hq: int, Hkv: int, d: int, w: int, cos: np.ndarray,
                   sin: np.ndarray) -> np.ndarray:
    """q_obs [Hq, w, d] (bf16 bits) from a fused QKV activation.

    qkv [T, (Hq + 2 Hkv) * d] bf16 bits, token-major, query heads first, before RoPE; the window is
    its last w rows; cos, sin [w, d/2] are the table rows of the window's positions. The rotation
    runs in fp64 on the exactly widened inputs and the result is rounded once to bf16.
    """
    T = qkv.shape[0]
    q = bf16_bits_to_f64(qkv[T - w:, :Hq * d]).reshape(w, Hq, d)
    out = rope(q, np.asarray(cos, dtype=np.float64)[:, None, :], np.asarray(sin, dtype=np.float64)[:, None, :])
    return f64_to_bf16_bits(np.transpose(out, (1, 0, 2)))


def gather_paged(K: np.ndarray, V: np.ndarray, idx: np.ndarray, block_table: np.ndarray, page_size: int,
                 cache_K: np.ndarray, cache_V: np.ndarray) -> None:
    """Scatter the kept rows into a paged cache, in place.

    cache_K, cache_V [num_pages, page_size, Hkv, d]; compacted position n of every head goes to page
    block_table[n // page_size], slot n % page_size (zero rows where idx is -1). Pages not named
    by the block table, and slots past n_max in the last page, are left as they are.
    (Algorithm 3's two index_select lines, written to where a paged decode cache keeps its rows.)
    """
    Hkv, n_max = idx.shape
    for h in range(Hkv):
        for n in range(n_max):
            page, slot = int(block_table[n // page_size]), n % page_size
            j = int(idx[h, n])
            cache_K[page, slot, h] = K[h, j] if j >= 0 else 0
            cache_V[page, slot, h] = V[h, j] if j >= 0 else 0
