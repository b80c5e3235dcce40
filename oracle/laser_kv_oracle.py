"""fp64 CPU oracle for LASER-KV's prefill-time token selection (TEST INFRASTRUCTURE ONLY).

This module is the slow, plain statement of what the CUDA path must compute. It is used by
the tests, by the smoke check and by the benchmark's CPU-baseline leg, and by nothing else:
the product path never imports it, and it imports nothing from the product path. It shares
no code, table or helper with the CUDA kernels.

Everything is numpy in float64 on the exact values of the bf16 input bits (decoded here by
this module's own routine). A library matmul serves as the inner-product step; there is no
blocking, fusion or reordering beyond what the paper's definitions state.

What each function follows:

* ``budget``            - Appendix B, Eq. 1 (effective budget from block size and context length).
* ``partition``         - Section 3.1 (protection divisor n: anchors B/n, local window B/n,
                          recall budget B - 2B/n) and Algorithm 1 lines 4 and 7 (alpha split).
* ``window_scores``     - Section 3.3 "Precision" and Algorithm 1 line 3, per layer and per
                          KV head: attention probabilities of the window queries over the
                          block's keys, summed over the queries of the KV head's GQA group.
* ``simhash_buckets``   - Section 3.3 "Recall" and Algorithm 1's hash functions h_r, taken as
                          K-bit SimHash (sign of Gaussian hyperplane projections) per table.
* ``collision_counts``  - Algorithm 1 line 6: number of (query, table) pairs whose bucket equals
                          the key's bucket (S_lsh is this count divided by R * number of queries).
* ``collision_probability`` - Section 3.3 "Recall" as worded (tokens ranked by the theoretical hash
                          collision probability with the query): the expectation of the
                          collision fraction over the hyperplane draw, (1 - theta/pi)^K per query.
* ``topk_lower_index``  - the TopK of Algorithm 1 lines 4 and 7, ties to the lower index.
* ``select_indices``    - Algorithm 1 lines 3-8 on the candidate set left by Section 3.1.
* ``select_block`` / ``AppendOnlyCache`` - Section 3 (only selected tokens are kept) and the
                          introduction's append-only accumulative memory.
* ``decode_attention``  - Section 3 (the kept tokens serve the decoding phase): softmax attention
                          of one decode query over the cache entries of its KV head.
* ``tail_budget``       - a last block with fewer tokens than a block (not covered by the paper,
                          whose contexts are whole numbers of blocks): the same rule with
                          B_t = min(B, tokens).
* ``lookback_partition`` / ``select_block_lookback`` / ``LookbackPrefill`` - Section 3.2 (block
                          processing and boundary smoothing): the scoring window of block t also
                          covers the tail of block t-1, whose tokens are pruned only then.

Readings taken where the paper is silent (rounding of B/n and alpha*B_long, per-block anchors,
softmax over the block's own keys, bit = [projection >= 0], tie rule) are listed in the design
notes of the repository and restated at each function.

Parity status: every function is pinned in the CPU test suite by something other than itself:
budget and partition by tables evaluated by hand as exact fractions at the paper's settings; the softmax
scores and the decode attention by library routines (scipy's softmax, torch's
scaled_dot_product_attention in float64), hand cases and scalar loops; SimHash bits by hand
cases and the (1 - theta/pi)^K collision rate; collision counts by a scalar triple loop; the
closed-form recall score by special angles and by the empirical collision fraction it is the
expectation of; top-k by exhaustive subset search; the consensus sums and the append-only cache
by their invariants; the look-back rule by its reduction to the plain rule when the local window
is empty, by exhaustive subset search over its candidate set, by a hand case and by the keep-count
and append-only invariants. The paper prints no numeric example of scores or chosen sets, so there is
no golden vector of that kind.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "bf16_bits_to_f64", "budget", "partition", "window_scores", "simhash_projections",
    "simhash_buckets", "collision_counts", "topk_lower_index", "select_indices",
    "group_queries", "select_block", "AppendOnlyCache", "BlockResult",
    "lookback_partition", "select_block_lookback", "LookbackPrefill", "LookbackResult", "tail_budget",
]


# ----------------------------------------------------------------------------------------------
# input decoding
# ----------------------------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bfloat16 bit patterns (uint16) as float64.

    A bfloat16 is the upper half of an IEEE binary32, so widening is exact.
    """
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    f32 = (b.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(np.float64)


# ----------------------------------------------------------------------------------------------
# budget arithmetic
# ----------------------------------------------------------------------------------------------
def budget(context_len: int, block_size: int, ratio: float = 0.25) -> int:
    """Eq. 1 (Appendix B): B = floor(2 r S_block L / (S_block + L)), in IEEE double."""
    if context_len <= 0 or block_size <= 0 or not (ratio > 0.0):
        raise ValueError("context_len, block_size and ratio must be positive")
    num = 2.0 * float(ratio) * float(block_size) * float(context_len)
    return int(math.floor(num / (float(block_size) + float(context_len))))


def partition(B: int, n: int, alpha: float = 0.75):
    """Section 3.1 + Algorithm 1 lines 4/7.

    Returns (anchors, local, B_long, k_exact, k_lsh) with
      anchors = local = floor(B / n)      (the syntactic set 2B/n, each half rounded down)
      B_long  = B - 2*floor(B/n)          (recall budget; absorbs the rounding remainder so the
                                           keep count is exactly B)
      k_exact = floor(alpha * B_long)     (IEEE double product, then floor)
      k_lsh   = B_long - k_exact
    n = 2 gives B_long = 0 (only anchors and the local window are kept).
    """
    if B < 0 or n < 2 or not (0.0 <= alpha <= 1.0):
        raise ValueError("need B >= 0, n >= 2, 0 <= alpha <= 1")
    a = B // n
    b_long = B - 2 * a
    k_e = int(math.floor(float(alpha) * float(b_long)))
    k_e = max(0, min(k_e, b_long))
    return a, a, b_long, k_e, b_long - k_e


# ----------------------------------------------------------------------------------------------
# step 1: observation-window attention scores (Section 3.3 "Precision", Algorithm 1 line 3)
# ----------------------------------------------------------------------------------------------
def window_scores(q_bits: np.ndarray, k_bits: np.ndarray, scale: float | None = None) -> np.ndarray:
    """S_exact[j] = sum over the group's window queries of softmax_j(<q, k_j> * scale).

    q_bits: uint16 [n_queries, d]  - every window query of every query head in the KV head's
                                     GQA group (G*W rows).
    k_bits: uint16 [S, d]          - the block's keys for this KV head.
    The softmax is over all S keys of the block (no causal mask, no pooling); scale defaults
    to 1/sqrt(d). Returns float64 [S]; each query contributes a row that sums to 1.
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    d = k.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    s = (q @ k.T) * float(scale)                      # [n_queries, S] logits
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=1, keepdims=True)              # attention probabilities per query
    return p.sum(axis=0)


# ----------------------------------------------------------------------------------------------
# step 2: SimHash signatures and collision counts (Section 3.3 "Recall", Algorithm 1 line 6)
# ----------------------------------------------------------------------------------------------
def simhash_projections(x_bits: np.ndarray, p_bits: np.ndarray) -> np.ndarray:
    """<p_m, x> for every vector x and every hyperplane p_m, float64 [N, L*K]."""
    return bf16_bits_to_f64(x_bits) @ bf16_bits_to_f64(p_bits).T


def simhash_buckets(x_bits: np.ndarray, p_bits: np.ndarray, n_bits: int, n_tables: int):
    """K-bit SimHash bucket of every vector in every table.

    Hyperplane m = r*K + b is bit b of table r; bit = 1 iff the projection is >= 0; the bucket
    id is sum_b bit_b * 2**b. Returns (buckets int64 [N, L], min_abs float64 [N, L]) where
    min_abs is the smallest |projection| among the table's K bits (used by comparisons that
    exempt signs decided by a projection smaller than 1e-6 in magnitude).
    """
    proj = simhash_projections(x_bits, p_bits)
    n = proj.shape[0]
    if proj.shape[1] != n_bits * n_tables:
        raise ValueError("hyperplane count must be n_bits * n_tables")
    proj = proj.reshape(n, n_tables, n_bits)
    bits = (proj >= 0.0).astype(np.int64)
    weights = (1 << np.arange(n_bits, dtype=np.int64))
    return (bits * weights).sum(axis=2), np.abs(proj).min(axis=2)


def collision_counts(q_buckets: np.ndarray, k_buckets: np.ndarray) -> np.ndarray:
    """count[j] = sum over queries and tables of 1[h_r(q) = h_r(k_j)]  (Algorithm 1 line 6,
    before the division by R and by the number of queries).

    q_buckets int [n_queries, L], k_buckets int [S, L] -> int64 [S]. Written as the plain loop
    over queries (each step compares one query's L buckets with every key's).
    """
    q_buckets = np.asarray(q_buckets)
    k_buckets = np.asarray(k_buckets)
    counts = np.zeros(k_buckets.shape[0], dtype=np.int64)
    for qi in range(q_buckets.shape[0]):
        counts += (k_buckets == q_buckets[qi][None, :]).sum(axis=1)
    return counts


# ----------------------------------------------------------------------------------------------
# step 3: two-stage top-k (Algorithm 1 lines 4-8)
# ----------------------------------------------------------------------------------------------
def topk_lower_index(candidates: np.ndarray, score: np.ndarray, k: int) -> np.ndarray:
    """The k candidates with the largest score; among equal scores the lower index wins.

    candidates: ascending int array of indices into ``score``. Returns the picks in ascending
    index order. Implemented as a full stable sort by descending score.
    """
    candidates = np.asarray(candidates, dtype=np.int64)
    if k <= 0 or candidates.size == 0:
        return np.zeros(0, dtype=np.int64)
    k = min(k, candidates.size)
    vals = np.asarray(score)[candidates]
    order = np.argsort(-vals, kind="stable")          # stable: ties keep ascending index order
    return np.sort(candidates[order[:k]])


def select_indices(s_exact: np.ndarray, counts: np.ndarray, S: int, anchors: int,
                   k_exact: int, k_lsh: int):
    """Algorithm 1 on the candidate set C = [anchors, S - anchors).

    Returns (K_exact, K_lsh, idx): the exact-stage picks, the LSH-stage picks from the residual
    C \\ K_exact, and the kept indices of the block in ascending order: anchors [0, a), the
    picks, and the local window [S - a, S).
    """
    cand = np.arange(anchors, S - anchors, dtype=np.int64)
    k_ex = topk_lower_index(cand, s_exact, k_exact)
    residual = np.setdiff1d(cand, k_ex, assume_unique=True)
    k_ls = topk_lower_index(residual, counts, k_lsh)
    idx = np.concatenate([np.arange(0, anchors, dtype=np.int64), k_ex, k_ls,
                          np.arange(S - anchors, S, dtype=np.int64)])
    return k_ex, k_ls, np.sort(idx)


# ----------------------------------------------------------------------------------------------
# the whole per-block path for one (layer, sequence)
# ----------------------------------------------------------------------------------------------
def group_queries(q_bits: np.ndarray, n_kv_heads: int, h: int) -> np.ndarray:
    """The window queries that score KV head h's keys: query heads h*G, h*G+1, ..., h*G+G-1
    (G = H_q / H_kv consecutive query heads share one KV head - grouped-query attention), each
    with its W window queries, as rows [G*W, d] in (head, window position) order.

    q_bits uint16 [H_q, W, d].
    """
    h_q, W, d = q_bits.shape
    if h_q % n_kv_heads:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    G = h_q // n_kv_heads
    heads = [h * G + g for g in range(G)]
    return np.concatenate([q_bits[i] for i in heads], axis=0)


@dataclass
class BlockResult:
    s_exact: np.ndarray          # float64 [H_kv, S]
    counts: np.ndarray           # int64   [H_kv, S]
    key_buckets: np.ndarray      # int64   [H_kv, S, L]
    key_min_abs: np.ndarray      # float64 [H_kv, S, L]
    query_buckets: np.ndarray    # int64   [H_kv, G*W, L]
    query_min_abs: np.ndarray    # float64 [H_kv, G*W, L]
    k_exact: list                # per KV head: ascending picks of the exact stage
    k_lsh: list                  # per KV head: ascending picks of the LSH stage
    idx: np.ndarray              # int64   [H_kv, B] kept block-local indices, ascending


def select_block(k_bits: np.ndarray, q_bits: np.ndarray, p_bits: np.ndarray, *, n_bits: int,
                 n_tables: int, B: int, n: int, alpha: float = 0.75,
                 scale: float | None = None) -> BlockResult:
    """Steps 1-3 for one block of one (layer, sequence).

    k_bits uint16 [H_kv, S, d]; q_bits uint16 [H_q, W, d] (query head h*G+g belongs to KV head
    h); p_bits uint16 [L*K, d]. Each KV head selects independently.
    """
    h_kv, S, d = k_bits.shape
    h_q, W, _ = q_bits.shape
    if h_q % h_kv:
        raise ValueError("n_q_heads must be a multiple of n_kv_heads")
    G = h_q // h_kv
    a, _, _b_long, k_e, k_l = partition(B, n, alpha)
    if 2 * a > S or B > S:
        raise ValueError("budget does not fit the block")
    out = BlockResult(np.zeros((h_kv, S)), np.zeros((h_kv, S), np.int64),
                      np.zeros((h_kv, S, n_tables), np.int64), np.zeros((h_kv, S, n_tables)),
                      np.zeros((h_kv, G * W, n_tables), np.int64),
                      np.zeros((h_kv, G * W, n_tables)), [], [], np.zeros((h_kv, B), np.int64))
    for h in range(h_kv):
        qg = group_queries(q_bits, h_kv, h)
        out.s_exact[h] = window_scores(qg, k_bits[h], scale)
        out.key_buckets[h], out.key_min_abs[h] = simhash_buckets(k_bits[h], p_bits, n_bits, n_tables)
        out.query_buckets[h], out.query_min_abs[h] = simhash_buckets(qg, p_bits, n_bits, n_tables)
        out.counts[h] = collision_counts(out.query_buckets[h], out.key_buckets[h])
        k_ex, k_ls, idx = select_indices(out.s_exact[h], out.counts[h], S, a, k_e, k_l)
        out.k_exact.append(k_ex)
        out.k_lsh.append(k_ls)
        out.idx[h] = idx
    return out


def select_block_consensus(k_layers, q_layers, p_bits: np.ndarray, *, n_bits: int, n_tables: int, B: int,
                           n: int, alpha: float = 0.75, scale: float | None = None):
    """Consensus form of steps 1-3 for one block of one sequence (Section 3.3 "Precision" as printed:
    a candidate's exact score is the attention it receives from the query summed over all layers
    and heads; Algorithm 1 then picks one index set that every head keeps).

    k_layers[l] uint16 [H_kv, S, d] and q_layers[l] uint16 [H_q, W, d] for every layer l. The exact
    scores and the collision counts of all (layer, KV head) pairs are added up; the two-stage
    top-k runs once on the sums. Returns (s_sum float64 [S], c_sum int64 [S], k_exact, k_lsh, idx).
    """
    s_sum = None
    c_sum = None
    for k_bits, q_bits in zip(k_layers, q_layers):
        r = select_block(k_bits, q_bits, p_bits, n_bits=n_bits, n_tables=n_tables, B=B, n=n, alpha=alpha, scale=scale)
        for h in range(k_bits.shape[0]):
            s_sum = r.s_exact[h].copy() if s_sum is None else s_sum + r.s_exact[h]
            c_sum = r.counts[h].copy() if c_sum is None else c_sum + r.counts[h]
    S = s_sum.shape[0]
    a, _, _b_long, k_e, k_l = partition(B, n, alpha)
    k_ex, k_ls, idx = select_indices(s_sum, c_sum, S, a, k_e, k_l)
    return s_sum, c_sum, k_ex, k_ls, idx


@dataclass
class AppendOnlyCache:
    """Accumulative cache of one (layer, sequence): entries are only ever appended.

    K, V hold raw bf16 bit patterns [H_kv, capacity, d]; pos holds absolute token positions
    [H_kv, capacity]; length is the same for every KV head (B per block).
    """
    n_kv_heads: int
    head_dim: int
    capacity: int
    K: np.ndarray = field(init=False)
    V: np.ndarray = field(init=False)
    pos: np.ndarray = field(init=False)
    length: int = 0

    def __post_init__(self):
        self.K = np.zeros((self.n_kv_heads, self.capacity, self.head_dim), np.uint16)
        self.V = np.zeros((self.n_kv_heads, self.capacity, self.head_dim), np.uint16)
        self.pos = np.full((self.n_kv_heads, self.capacity), -1, np.int32)

    def append(self, k_bits: np.ndarray, v_bits: np.ndarray, idx: np.ndarray, block_start: int):
        """Copy rows idx[h] of the block into [length, length + B) and advance length by B."""
        B = idx.shape[1]
        if self.length + B > self.capacity:
            raise ValueError("cache capacity exceeded")
        for h in range(self.n_kv_heads):
            sl = slice(self.length, self.length + B)
            self.K[h, sl] = k_bits[h, idx[h]]
            self.V[h, sl] = v_bits[h, idx[h]]
            self.pos[h, sl] = (block_start + idx[h]).astype(np.int32)
        self.length += B


# ----------------------------------------------------------------------------------------------
# recall score in closed form (Section 3.3 "Recall": ranking by the theoretical collision probability)
# ----------------------------------------------------------------------------------------------
def collision_probability(q_bits: np.ndarray, k_bits: np.ndarray, n_bits: int) -> np.ndarray:
    """S_theory[j] = (1/n_queries) * sum_q (1 - theta(q, k_j)/pi)^K.

    A K-bit SimHash table puts q and k in the same bucket exactly when none of K independent
    Gaussian hyperplanes separates them; one hyperplane separates them with probability
    theta/pi, theta the angle between them. This is the expectation over the hyperplane draw
    of Algorithm 1's collision fraction (``collision_counts`` divided by tables * queries).
    q_bits uint16 [n_queries, d], k_bits uint16 [S, d] -> float64 [S]. A zero vector has no angle:
    its cosine is taken as 0 (theta = pi/2), the value the hashes give it against any hyperplane
    draw in expectation.
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    qn = np.sqrt((q * q).sum(axis=1))
    kn = np.sqrt((k * k).sum(axis=1))
    dots = q @ k.T                                        # [n_queries, S]
    denom = qn[:, None] * kn[None, :]
    cos = np.divide(dots, denom, out=np.zeros_like(dots), where=denom > 0)
    theta = np.arccos(np.clip(cos, -1.0, 1.0))
    return ((1.0 - theta / math.pi) ** int(n_bits)).mean(axis=0)


# ----------------------------------------------------------------------------------------------
# decoding over the kept tokens (Section 3: only the selected tokens stay in the cache and are
# used for the decoding phase)
# ----------------------------------------------------------------------------------------------
def decode_attention(q_bits: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray,
                     scale: float | None = None) -> np.ndarray:
    """out[g] = sum_i softmax_i(<q_g, k_i> * scale) * v_i over the cache entries of one KV head.

    q_bits: uint16 [G, d]   - the decode-step queries of the KV head's query heads.
    k_bits, v_bits: uint16 [len, d] - the head's cache entries (len >= 1).
    Plain softmax attention, no mask (every cache entry precedes the decode position); scale
    defaults to 1/sqrt(d). Returns float64 [G, d].
    """
    q = bf16_bits_to_f64(q_bits)
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    if k.shape[0] < 1:
        raise ValueError("decode_attention needs at least one cache entry")
    if scale is None:
        scale = 1.0 / math.sqrt(k.shape[1])
    s = (q @ k.T) * float(scale)                      # [G, len]
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v


# ----------------------------------------------------------------------------------------------
# look-back boundary smoothing (Section 3.2)
# ----------------------------------------------------------------------------------------------
# Reading taken (the text says only that the scoring window of block t is expanded to include the
# tail of block t-1, so that tokens at a block's edge are evaluated with the context that follows
# them before they are pruned): the "tail" is the block's local sliding window, its last
# a = floor(B/n) tokens. Without look-back those tokens are kept unconditionally by their own
# block. With look-back the window slides: block t-1 does not decide about them; they are scored
# together with block t's keys against block t's window queries (one softmax over a + S keys) and
# compete with block t's candidates. Per block (index g in the sequence):
#   g = 0 : scored keys = the block; kept = anchors [0, a) + Algorithm 1 on C = [a, S - a) with
#           B_long = B - 2a; the tail [S - a, S) is held back. B - a entries appended.
#   g >= 1: scored keys = held-back tail of block g-1 (a keys) followed by the block (S keys);
#           kept = anchors of the block + Algorithm 1 on C = tail(g-1) + [a, S - a) of the block
#           with B_long = (B - 2a) + a = B - a (the recall budget plus the a entries the slid window released);
#           the block's own tail is held back. B entries appended, in position order.
#   close : the tail of the last block is appended as it is (nothing follows it). a entries.
# After m blocks and the close the cache holds m * B entries per head, as without look-back.
def lookback_partition(B: int, n: int, alpha: float, released: int):
    """(anchors, held_back, B_long, k_exact, k_lsh) of one look-back step; see the rule above.
    `released` is the number of held-back tokens of the previous block that this step decides about
    (0 for the first block of a sequence): the recall budget is the block's own B - 2a plus those
    entries, which the previous block's local window no longer occupies."""
    a, _, b_long0, _, _ = partition(B, n, alpha)
    b_long = b_long0 + released
    k_e = int(math.floor(float(alpha) * float(b_long)))
    k_e = max(0, min(k_e, b_long))
    return a, a, b_long, k_e, b_long - k_e


def tail_budget(B: int, n_tokens: int) -> int:
    """Budget of a last block that has fewer tokens than a block (the paper's contexts are whole
    numbers of blocks; reading taken: the same rule on the tokens there are): B_t = min(B, S_t).
    The partition of B_t by the protection divisor and alpha is the usual one, so a tail block with
    at least B tokens keeps B of them and a shorter one keeps all of its tokens."""
    if n_tokens < 1:
        raise ValueError("a block has at least one token")
    return min(B, n_tokens)


@dataclass
class LookbackResult:
    s_exact: np.ndarray          # float64 [H_kv, n_scored]   n_scored = S (first block) or a + S
    counts: np.ndarray           # int64   [H_kv, n_scored]
    k_exact: list                # per KV head: picks of the exact stage, scored-key indices, ascending
    k_lsh: list                  # per KV head: picks of the LSH stage
    idx: np.ndarray              # int64   [H_kv, n_kept] kept scored-key indices, ascending
    offset: int                  # position of scored key 0 relative to the block's first token (0 or -a)


def select_block_lookback(k_prev_tail, k_bits: np.ndarray, q_bits: np.ndarray, p_bits: np.ndarray, *,
                          n_bits: int, n_tables: int, B: int, n: int, alpha: float = 0.75,
                          scale: float | None = None) -> LookbackResult:
    """One look-back step for one block of one (layer, sequence).

    k_prev_tail: uint16 [H_kv, a, d], the held-back tail of the previous block, or None for the
    first block of the sequence. k_bits uint16 [H_kv, S, d]; q_bits uint16 [H_q, W, d]; p_bits
    uint16 [L*K, d]. Indices in the result count the scored keys: the previous tail first
    (when there is one), then the block.
    """
    h_kv, S, d = k_bits.shape
    first = k_prev_tail is None
    a, _, b_long, k_e, k_l = lookback_partition(B, n, alpha, 0 if first else k_prev_tail.shape[1])
    if 2 * a > S or B > S:
        raise ValueError("budget does not fit the block")
    if first:
        scored = k_bits
        off = 0
    else:
        # the previous block's tail has that block's own floor(B/n) rows (a shorter last block, see
        # tail_budget, has a smaller budget than the blocks before it)
        if k_prev_tail.shape[0] != h_kv or k_prev_tail.shape[2] != d:
            raise ValueError("the held-back tail must be [H_kv, rows, d]")
        scored = np.concatenate([k_prev_tail, k_bits], axis=1)
        off = k_prev_tail.shape[1]
    n_scored = scored.shape[1]
    # candidates: the previous tail, and the block without its anchors and without its own tail
    cand = np.concatenate([np.arange(0, off, dtype=np.int64),
                           np.arange(off + a, off + S - a, dtype=np.int64)])
    anchors = np.arange(off, off + a, dtype=np.int64)
    n_kept = a + b_long
    if b_long > cand.size:
        raise ValueError("recall budget exceeds the candidate set")
    out = LookbackResult(np.zeros((h_kv, n_scored)), np.zeros((h_kv, n_scored), np.int64), [], [],
                         np.zeros((h_kv, n_kept), np.int64), -off)
    for h in range(h_kv):
        qg = group_queries(q_bits, h_kv, h)
        out.s_exact[h] = window_scores(qg, scored[h], scale)          # one softmax over all scored keys
        kb, _ = simhash_buckets(scored[h], p_bits, n_bits, n_tables)
        qb, _ = simhash_buckets(qg, p_bits, n_bits, n_tables)
        out.counts[h] = collision_counts(qb, kb)
        k_ex = topk_lower_index(cand, out.s_exact[h], k_e)
        residual = np.setdiff1d(cand, k_ex, assume_unique=True)
        k_ls = topk_lower_index(residual, out.counts[h], k_l)
        out.k_exact.append(k_ex)
        out.k_lsh.append(k_ls)
        out.idx[h] = np.sort(np.concatenate([anchors, k_ex, k_ls]))
    return out


class LookbackPrefill:
    """Block-by-block prefill of one (layer, sequence) with look-back: owns the append-only cache
    and the held-back tail between steps."""

    def __init__(self, n_kv_heads: int, head_dim: int, capacity: int, *, n_bits: int, n_tables: int,
                 B: int, n: int, alpha: float = 0.75, scale: float | None = None):
        self.cache = AppendOnlyCache(n_kv_heads, head_dim, capacity)
        self.kw = dict(n_bits=n_bits, n_tables=n_tables, B=B, n=n, alpha=alpha, scale=scale)
        self.a = B // n
        self.tail = None             # (k, v, first position) of the held-back tokens
        self.blocks = 0
        self.tokens = 0
        self.block_size = None
        self.short = False
        self.closed = False

    def step(self, k_bits, v_bits, q_bits, p_bits) -> LookbackResult:
        """One block. A block with fewer tokens than the ones before it (the last one) runs with
        tail_budget(B, tokens); nothing may follow it but close()."""
        if self.closed or self.short:
            raise ValueError("the sequence was closed or has had its short last block")
        S = k_bits.shape[1]
        if self.block_size is None:
            self.block_size = S
        start = self.tokens
        kw = dict(self.kw)
        if S < self.block_size:
            kw["B"] = tail_budget(kw["B"], S)
            self.short = True
        elif S != self.block_size:
            raise ValueError("only the last block may differ in length, and only by being shorter")
        prev = None if self.tail is None else self.tail[0]
        r = select_block_lookback(prev, k_bits, q_bits, p_bits, **kw)
        if self.tail is None:
            ks, vs = k_bits, v_bits
        else:
            ks = np.concatenate([self.tail[0], k_bits], axis=1)
            vs = np.concatenate([self.tail[1], v_bits], axis=1)
        self.cache.append(ks, vs, r.idx, start + r.offset)
        a = kw["B"] // kw["n"]
        self.tail = (k_bits[:, S - a:].copy(), v_bits[:, S - a:].copy(), start + S - a)
        self.blocks += 1
        self.tokens += S
        return r

    def close(self):
        """Appends the last block's held-back tail: nothing follows it, so nothing can prune it."""
        if self.closed or self.tail is None:
            raise ValueError("nothing to close")
        k, v, pos0 = self.tail
        a = k.shape[1]
        idx = np.tile(np.arange(a, dtype=np.int64), (k.shape[0], 1))
        self.cache.append(k, v, idx, pos0)
        self.closed = True
