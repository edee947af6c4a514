"""CPU oracle for the Focus-dLLM per-step sparse-attention path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 restatement of what the paper defines, used to judge the
CUDA library.  Only tests, the smoke check and the benchmark's CPU-baseline leg
may import this module; the product path never does, and this module imports
nothing from the product package (no shared kernels, helpers or tables).

Positions are 0-indexed here (the paper counts from 1): prompt [0, M), response
(gen region) [M, L).  Prompt block b covers [b*B, min((b+1)*B, M)).  Query head h
reads KV head g(h) = h // (H // Hkv).  Every sort is a brute-force stable sort on
(-score, index): ties go to the lower index, NaN scores rank last.

Functions and the passages they follow
  select_queries   Section "Past Confidence-Guided Indicator", Eq. 4 (I_focus) and Eq. 5 (I_active);
                   Algorithm 1, the two lines of the non-block-entry branch.
  sink_scores      Section "Sink-Aware Sparse Attention", Eq. 6 (S_j).
  find_sinks       same section: I_sink = Top-N_sink(S_j).
  pool_keys        "Block-wise token pruning": K-bar_b = mean of the block's keys.
  score_blocks     Eq. 7 (R_b).
  select_blocks    B_relevant = Top-C(R_b) and Eq. 8 (I_p).
  sparse_attn      K_attn = concat(K_Ip, K_resp) and Eq. 9.
  dense_attn       "FullAttn" of Algorithm 1: plain bidirectional softmax attention.
  confidence       Section "Diffusion LLM inference", Eq. 2: predicted token and confidence of a position.
  update_kv        "Approximate KV cache in dLLMs", Eq. 3: refreshed rows replace the cached ones.
  commit_step      Algorithm 1, the state update that ends a step, with the unmasking rule stated right after Eq. 2:
                   the most confident masked positions receive their predicted tokens, the rest stay masked.

Readings where the paper leaves a choice (parity unpinned by the paper for these):
  * Eq. 6 writes one softmax over an "aggregated query representation"; here every
    active query row has its own softmax over all L keys and S_j is the mean of the
    probabilities over rows and heads (column-summed attention mass).
  * Top-N_sink candidates are the prompt positions handed in by the caller
    ([cand_lo, cand_hi)); response tokens are always attended anyway.
  * I_active is clipped to a caller range; K_resp is every response position [M, L).
Everything else is pinned by the tests in tests/test_oracle_pins.py.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

PER_KV_GROUP = 0   # one block set per KV head (scores averaged over the query heads of the group)
ALL_HEADS = 1      # one block set for the layer (Eq. 7 as printed: average over all H heads)

SINK_TOKENS = 0    # sinks join the key set as single tokens (Eq. 8 as printed)
SINK_BLOCKS = 1    # variant: the whole block around each sink token is kept


def _rank_desc(scores: Sequence[float], idx: Sequence[int]) -> List[int]:
    """Indices ordered by score descending, ties by lower index, NaN last."""
    def key(t):
        s, i = t
        s = float(s)
        if math.isnan(s):
            s = -math.inf
        return (-s, i)
    return [i for _, i in sorted(zip(scores, idx), key=key)]


# ----------------------------------------------------------------------------- Eq. 4, Eq. 5
def select_queries(conf_prev: np.ndarray, masked: np.ndarray, blk_lo: int, blk_hi: int,
                   k: int, w: int, clip_lo: int, clip_hi: int) -> Tuple[np.ndarray, np.ndarray]:
    """I_focus: the k still-masked positions of the current decoding block with the highest
    previous-step confidence (Eq. 4).  I_active: union of the windows
    [i - floor(w/2), i + floor(w/2)] around them (Eq. 5), clipped to [clip_lo, clip_hi).
    Both are returned ascending."""
    cand = [i for i in range(blk_lo, blk_hi) if masked[i] != 0]
    order = _rank_desc([conf_prev[i] for i in cand], cand)
    focus = sorted(order[:max(0, min(k, len(cand)))])
    hw = w // 2
    active = set()
    for i in focus:
        for l in range(i - hw, i + hw + 1):
            if clip_lo <= l < clip_hi:
                active.add(l)
    return np.array(focus, dtype=np.int64), np.array(sorted(active), dtype=np.int64)


# ----------------------------------------------------------------------------- Eq. 6
def _softmax_rows(s: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return e / z, (m + np.log(z))[:, 0]


def sink_scores(Qa: np.ndarray, K: np.ndarray, scale: float) -> np.ndarray:
    """S_j = (1/(H*n)) sum_h sum_i softmax_j(scale * q_i^h . k_j^{g(h)}) over all L keys (Eq. 6).
    Qa: [n, H, d] rows of the active queries; K: [Hkv, L, d]."""
    Qa = np.asarray(Qa, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    n, H, _ = Qa.shape
    Hkv, L, _ = K.shape
    if n == 0:
        raise ValueError("I_active is empty")
    hpg = H // Hkv
    S = np.zeros(L, dtype=np.float64)
    for h in range(H):
        p, _ = _softmax_rows(scale * (Qa[:, h, :] @ K[h // hpg].T))
        S += p.sum(axis=0)
    return S / (H * n)


def find_sinks(S: np.ndarray, n_sink: int, cand_lo: int, cand_hi: int) -> np.ndarray:
    """I_sink = Top-N_sink(S_j) over j in [cand_lo, cand_hi), ascending."""
    cand = list(range(cand_lo, cand_hi))
    order = _rank_desc([S[j] for j in cand], cand)
    return np.array(sorted(order[:max(0, min(n_sink, len(cand)))]), dtype=np.int64)


# ----------------------------------------------------------------------------- K-bar, Eq. 7
def pool_keys(K: np.ndarray, M: int, B: int) -> np.ndarray:
    """K-bar[g, b, :] = mean of K[g, j, :] over the prompt block b (the last block may be short)."""
    K = np.asarray(K, dtype=np.float64)
    Hkv, _, d = K.shape
    nb = (M + B - 1) // B
    out = np.zeros((Hkv, nb, d), dtype=np.float64)
    for b in range(nb):
        lo, hi = b * B, min((b + 1) * B, M)
        out[:, b, :] = K[:, lo:hi, :].mean(axis=1)
    return out


def score_blocks(Qf: np.ndarray, Kbar: np.ndarray, head_reduce: int) -> np.ndarray:
    """Block relevance (Eq. 7).  Qf: [n_focus, H, d] rows of the focus queries.
    ALL_HEADS:     R[0, b] = (1/H) sum_h mean_i q_i^h . K-bar_b^{g(h)}   (as printed)
    PER_KV_GROUP:  R[g, b] = mean over the heads h of group g and over i of the same product.
    No softmax and no 1/sqrt(d)."""
    Qf = np.asarray(Qf, dtype=np.float64)
    Kbar = np.asarray(Kbar, dtype=np.float64)
    nf, H, _ = Qf.shape
    Hkv, nb, _ = Kbar.shape
    if nf == 0:
        raise ValueError("I_focus is empty")
    hpg = H // Hkv
    per_head = np.zeros((H, nb), dtype=np.float64)
    for h in range(H):
        per_head[h] = (Qf[:, h, :] @ Kbar[h // hpg].T).mean(axis=0)
    if head_reduce == ALL_HEADS:
        return per_head.mean(axis=0, keepdims=True)
    return per_head.reshape(Hkv, hpg, nb).mean(axis=1)


# ----------------------------------------------------------------------------- Top-C, Eq. 8
def select_blocks(R: np.ndarray, C: int, sink_idx: np.ndarray, B: int,
                  sink_mode: int = SINK_TOKENS) -> Tuple[List[np.ndarray], np.ndarray]:
    """Per row of R (one per group): the C highest-scoring prompt blocks, ascending.
    SINK_TOKENS: sink_keep[g, s] = 1 iff sink token s lies outside every selected block of
    group g (it must then be attended as a single token; inside a block it is already there).
    SINK_BLOCKS: the block containing each sink token is added to the group's list."""
    R = np.asarray(R, dtype=np.float64)
    G, nb = R.shape
    sink_idx = np.asarray(sink_idx, dtype=np.int64)
    blocks: List[np.ndarray] = []
    keep = np.zeros((G, len(sink_idx)), dtype=np.uint8)
    for g in range(G):
        order = _rank_desc(list(R[g]), list(range(nb)))
        sel = set(order[:max(0, min(C, nb))])
        if sink_mode == SINK_BLOCKS:
            sel |= {int(j) // B for j in sink_idx}
        else:
            for s, j in enumerate(sink_idx):
                keep[g, s] = 0 if (int(j) // B) in sel else 1
        blocks.append(np.array(sorted(sel), dtype=np.int64))
    return blocks, keep


# ----------------------------------------------------------------------------- Eq. 9
def key_set(M: int, L: int, B: int, blocks: np.ndarray, sink_idx: np.ndarray) -> np.ndarray:
    """I_p (Eq. 8) joined with every response position [M, L): sorted, without duplicates."""
    ks = set(range(M, L))
    for b in blocks:
        ks.update(range(int(b) * B, min((int(b) + 1) * B, M)))
    ks.update(int(j) for j in sink_idx)
    return np.array(sorted(ks), dtype=np.int64)


def _attend(q: np.ndarray, Kh: np.ndarray, Vh: np.ndarray, keys: Optional[np.ndarray], scale: float):
    if keys is not None:
        Kh, Vh = Kh[keys], Vh[keys]
    p, lse = _softmax_rows(scale * (q @ Kh.T))
    return p @ Vh, lse


def sparse_attn(Q: np.ndarray, K: np.ndarray, V: np.ndarray, M: int, B: int,
                blocks: List[np.ndarray], sink_idx: np.ndarray, scale: float,
                heads: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """o_i^h = sum over the key set of head h of softmax(scale * q_i^h . k_j) v_j  (Eq. 9), with the
    key set = tokens of the selected blocks of the head's group, the sink tokens, and all
    response tokens, taken as a set.  Q: [n, H, d]; K, V: [Hkv, L, d]; blocks: one list per
    group (len 1 = shared by all heads).  Returns O [n, H, d] and lse [H, n]
    (natural log of the softmax denominator).  `heads` restricts the work to some heads
    (other outputs stay zero)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    n, H, d = Q.shape
    Hkv, L, _ = K.shape
    hpg = H // Hkv
    O = np.zeros((n, H, d), dtype=np.float64)
    lse = np.zeros((H, n), dtype=np.float64)
    for h in (range(H) if heads is None else heads):
        g = h // hpg
        ks = key_set(M, L, B, blocks[g if len(blocks) > 1 else 0], sink_idx)
        O[:, h, :], lse[h] = _attend(Q[:, h, :], K[g], V[g], ks, scale)
    return O, lse


def dense_attn(Q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float,
               heads: Optional[Sequence[int]] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Bidirectional softmax attention of the given query rows over all L keys (no mask)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    n, H, d = Q.shape
    Hkv = K.shape[0]
    hpg = H // Hkv
    O = np.zeros((n, H, d), dtype=np.float64)
    lse = np.zeros((H, n), dtype=np.float64)
    for h in (range(H) if heads is None else heads):
        O[:, h, :], lse[h] = _attend(Q[:, h, :], K[h // hpg], V[h // hpg], None, scale)
    return O, lse


# ----------------------------------------------------------------------------- Eq. 2
def confidence(logits: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 2 for each row of `logits` [n, V]: the predicted token argmax_v p(v) (lowest v on ties) and its
    confidence c = max_v p(v), with p = softmax(logits) over the vocabulary.  NaN logits count as -inf."""
    x = np.asarray(logits, dtype=np.float64).copy()
    x[np.isnan(x)] = -np.inf
    tok = np.zeros(x.shape[0], dtype=np.int64)
    conf = np.zeros(x.shape[0], dtype=np.float64)
    for r in range(x.shape[0]):
        row = x[r]
        m = row.max()
        p = np.exp(row - m)
        p = p / p.sum()
        tok[r] = int(np.argmax(p))          # first occurrence = lowest index
        conf[r] = p[tok[r]]
    return conf, tok


# ----------------------------------------------------------------------------- Eq. 3
def update_kv(K_cache: np.ndarray, V_cache: np.ndarray, K_new: np.ndarray, V_new: np.ndarray,
              rows: Sequence[int]) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 3: K_i = f_K(x)_i for i in the refreshed set U (here `rows`, with the new states K_new[r] for rows[r]),
    the cached state otherwise; same for V.  Caches are [Hkv, L, d], new states [n, Hkv, d].  Returns new arrays."""
    K, V = np.array(K_cache, copy=True), np.array(V_cache, copy=True)
    for r, pos in enumerate(rows):
        K[:, int(pos), :] = K_new[r]
        V[:, int(pos), :] = V_new[r]
    return K, V


# ----------------------------------------------------------------------------- end of a step (after Eq. 2; Algorithm 1)
def commit_step(conf: np.ndarray, masked: np.ndarray, x: np.ndarray, pos: Sequence[int], conf_new: Sequence[float],
                token_new: Sequence[int], blk_lo: int, blk_hi: int, n: int):
    """x^(t) -> x^(t+1) and c^(t) -> c^(t+1) for the positions `pos` evaluated this step (conf_new[r], token_new[r]
    belong to pos[r]; Eq. 2).  Every evaluated position takes its new confidence.  Among the evaluated positions
    that are still masked and lie in the decoding block [blk_lo, blk_hi), the n with the highest new confidence
    (ties: lower position, NaN last) are unmasked: they receive their predicted token and leave the masked set;
    everything else stays as it was.  Returns new (conf, masked, x) and the unmasked positions, ascending."""
    conf, masked, x = np.array(conf, copy=True), np.array(masked, copy=True), np.array(x, copy=True)
    row_of = {int(p): r for r, p in enumerate(pos)}
    cand = [int(p) for p in pos if masked[int(p)] != 0 and blk_lo <= int(p) < blk_hi]
    order = _rank_desc([conf_new[row_of[p]] for p in cand], cand)
    picks = sorted(order[:max(0, min(n, len(cand)))])
    for p, r in row_of.items():
        conf[p] = conf_new[r]
    for p in picks:
        x[p] = token_new[row_of[p]]
        masked[p] = 0
    return conf, masked, x, picks
