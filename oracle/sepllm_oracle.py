"""CPU oracle for the SepLLM attention path (TEST INFRASTRUCTURE, not product code).

A plain, slow, fp64 restatement of what the paper defines, written to be checked
against the paper by eye.  Only tests, the smoke check and the CPU-baseline leg
of the benchmark may import it; the CUDA path shares no code with it.

Notation follows the paper: sequence length m is called ``L`` here, ``a`` is
the number of initial tokens, ``n`` the number of neighbouring tokens, and for
the streaming cache ``s``, ``w``, ``c`` are the separator-cache, local-window
and total capacities.

Pins (see tests/test_oracle_*.py): brute-force loops on tiny inputs, the
dense-causal / sliding-window special cases, row sums, finite differences,
the closed forms of Eq. 3 and Eq. 4 with the runtime-KV values the paper
prints, the attention-map ratio of Table 3, and for the cache a prompt leaves
behind the description of its content that does not run the state machine
(newest separators before a contiguous neighbour run).

Parity unpinned (the paper gives no value that separates the alternatives):
  * the order in which separators leave a full Separator Cache (taken: oldest
    first), and
  * whether a streaming step attends before or after compaction (taken:
    append, compact if full, then attend), and
  * the rotary formula behind "positions within the cache" (Section 3.3 names
    none; taken: rotate-half pairs (i, i + d/2), theta_i = base^(-2i/d), cache
    entry r at position r, query at the last position).  rope_rotate itself is
    pinned to the mathematics (complex-multiplication form, shift invariance,
    norm preservation), and
  * where the intervals of the fixed-interval variant start (taken: position 0), and
  * rows that pack several documents (the paper does not treat them; taken:
    Eq. 2 inside each document, nothing across a boundary).  Given that
    reading, packed_mask_matrix, the packed attention and build_index_packed
    are pinned to the per-document functions.
"""
from __future__ import annotations

import math
from typing import Iterable, List, Sequence

import numpy as np


# ----------------------------------------------------------------------------
# Mask (Section 3.1; Eq. 2)
# ----------------------------------------------------------------------------

def separator_flags(token_ids: np.ndarray, sep_ids: Iterable[int]) -> np.ndarray:
    """f[j] = True iff token j is one of the separator ids (Section 4.1 lists
    the nine separator strings; here they arrive as ids)."""
    sep = set(int(x) for x in sep_ids)
    return np.array([int(t) in sep for t in token_ids], dtype=bool)


def fixed_interval_flags(L: int, interval: int) -> np.ndarray:
    """Flags of the fixed-interval variant (Section 4.7 and the appendix
    "Fixed-Interval Variant"): one token every ``interval`` positions takes the
    separators' place.  The paper does not say where the intervals start; here
    they start at position 0."""
    return (np.arange(L) % int(interval)) == 0


def mask_matrix(f: np.ndarray, a: int, n: int) -> np.ndarray:
    """Binary mask M of Eq. 2 for one sequence.

    Query i sees key j (j <= i) iff j is one of the first ``a`` tokens, or j is
    a separator, or j is among the ``n`` closest tokens, the query's own
    position counted as the closest (Section 3.1).
    """
    L = f.shape[0]
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    causal = j <= i
    initial = j < a
    separator = f[None, :]
    neighbour = (i - j) < n
    return causal & (initial | separator | neighbour)


def mask_rows(f: np.ndarray, a: int, n: int, rows: np.ndarray, cols: np.ndarray | None = None) -> np.ndarray:
    """Rows ``rows`` (and, if given, only columns ``cols``) of the mask of Eq. 2: the same
    predicate on fewer entries."""
    L = f.shape[0]
    i = np.asarray(rows)[:, None]
    j = (np.arange(L) if cols is None else np.asarray(cols))[None, :]
    return (j <= i) & ((j < a) | f[j] | ((i - j) < n))


def document_bounds(doc_first: np.ndarray, length: int | None = None):
    """start[j], end[j] of the document position j belongs to, for a row that
    holds several documents one after the other: a document begins at position
    0 and at every j with doc_first[j] != 0 and ends where the next one begins
    (or at ``length``, the number of tokens in the row).  Positions from
    ``length`` on are padding: start = end = j (no document)."""
    doc_first = np.asarray(doc_first)
    L = doc_first.shape[0]
    Lv = L if length is None else int(length)
    start = np.zeros(L, dtype=np.int64)
    end = np.zeros(L, dtype=np.int64)
    s = 0
    for j in range(L):
        if j >= Lv:
            start[j] = j
            continue
        if j == 0 or doc_first[j]:
            s = j
        start[j] = s
    e = Lv
    for j in range(L - 1, -1, -1):
        if j >= Lv:
            end[j] = j
            continue
        end[j] = e
        if j == 0 or doc_first[j]:
            e = j
    return start, end


def packed_mask_matrix(f: np.ndarray, doc_first: np.ndarray, a: int, n: int) -> np.ndarray:
    """Mask of a row that packs several documents.  The paper trains on full
    rows and does not treat packing; the reading taken: Eq. 2 holds inside each
    document and nothing is seen across a boundary, so the initial tokens are
    the first ``a`` tokens of the query's own document and the neighbour window
    stops at the document's first token."""
    L = f.shape[0]
    start, _ = document_bounds(doc_first)
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    same_doc = start[None, :] == start[:, None]
    initial = (j - start[None, :]) < a
    return (j <= i) & same_doc & (initial | f[None, :] | ((i - j) < n))


def kept_pairs(f: np.ndarray, a: int, n: int) -> int:
    """Number of ones in M, counted row by row from the predicate."""
    L = f.shape[0]
    total = 0
    side = (np.arange(L) < a) | f
    prefix = np.concatenate([[0], np.cumsum(side)])  # prefix[j] = #side in [0, j)
    for i in range(L):
        lo = max(0, i - n + 1)          # first position of the neighbour window
        total += (i - lo + 1) + int(prefix[lo])
    return total


def attention_map_ratio(f: np.ndarray, a: int, n: int) -> float:
    """Share of ones in the lower triangle of the mask (Table 3, 'Atten. (%)')."""
    L = f.shape[0]
    return kept_pairs(f, a, n) / (L * (L + 1) / 2)


# ----------------------------------------------------------------------------
# Forward (Eq. 1, Eq. 2)
# ----------------------------------------------------------------------------

def attn_fwd_rows(Q: np.ndarray, K: np.ndarray, V: np.ndarray, M: np.ndarray,
                  scale: float | None = None):
    """Masked softmax attention for one head.

    Q: [R][d] (the R query rows that M's rows describe), K, V: [L][d], M: [R][L].
    Lambda = Q K^T * scale where M = 1 and -inf elsewhere; A = softmax(Lambda);
    O = A V.  Returns O [R][d], LSE [R] (natural log), A [R][L].
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    d = Q.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    Lam = (Q @ K.T) * scale
    Lam = np.where(M, Lam, -np.inf)
    mx = Lam.max(axis=1, keepdims=True)
    E = np.exp(Lam - mx)
    Z = E.sum(axis=1, keepdims=True)
    A = E / Z
    O = A @ V
    LSE = (mx + np.log(Z))[:, 0]
    return O, LSE, A


def _batch_mask(flags, a, n, b, doc_first):
    """Mask of sequence b: Eq. 2, or its packed form when document boundaries are given."""
    if doc_first is None:
        return mask_matrix(flags[b], a, n)
    return packed_mask_matrix(flags[b], np.asarray(doc_first)[b], a, n)


def attn_fwd(Q: np.ndarray, K: np.ndarray, V: np.ndarray, flags: np.ndarray,
             a: int, n: int, scale: float | None = None, doc_first=None):
    """Forward for a batch.  Q [B][Hq][L][d], K,V [B][Hkv][L][d], flags [B][L].

    Query head h reads KV head h // (Hq // Hkv).  The mask is the same for all
    heads (Section 3.2, after Eq. 2).  Returns O [B][Hq][L][d], LSE [B][Hq][L].
    doc_first [B][L] (optional): rows that pack several documents, see
    packed_mask_matrix.
    """
    B, Hq, L, d = Q.shape
    G = Hq // K.shape[1]
    O = np.zeros((B, Hq, L, d))
    LSE = np.zeros((B, Hq, L))
    for b in range(B):
        M = _batch_mask(flags, a, n, b, doc_first)
        for h in range(Hq):
            O[b, h], LSE[b, h], _ = attn_fwd_rows(Q[b, h], K[b, h // G], V[b, h // G], M, scale)
    return O, LSE


# ----------------------------------------------------------------------------
# Backward (gradient of Eq. 1 under the mask of Eq. 2)
# ----------------------------------------------------------------------------

def attn_bwd_head(Q, K, V, dO, M, scale: float | None = None):
    """Gradients of sum(O * dO) for one head, all rows.

    With A = softmax(Lambda): dV = A^T dO; dA = dO V^T;
    dLambda = A * (dA - rowsum(dA * A)); dQ = dLambda K * scale;
    dK = dLambda^T Q * scale.  rowsum(dA * A) equals rowsum(dO * O).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    d = Q.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    O, _, A = attn_fwd_rows(Q, K, V, M, scale)
    dV = A.T @ dO
    dA = dO @ V.T
    delta = (dO * O).sum(axis=1, keepdims=True)
    dLam = A * (dA - delta)
    dQ = (dLam @ K) * scale
    dK = (dLam.T @ Q) * scale
    return dQ, dK, dV


def attn_bwd(Q, K, V, dO, flags, a: int, n: int, scale: float | None = None, doc_first=None):
    """Backward for a batch; dK and dV are summed over the query heads that
    share a KV head.  doc_first: as in attn_fwd."""
    B, Hq, L, d = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    dQ = np.zeros((B, Hq, L, d))
    dK = np.zeros((B, Hkv, L, d))
    dV = np.zeros((B, Hkv, L, d))
    for b in range(B):
        M = _batch_mask(flags, a, n, b, doc_first)
        for h in range(Hq):
            q, k, v = attn_bwd_head(Q[b, h], K[b, h // G], V[b, h // G], dO[b, h], M, scale)
            dQ[b, h] = q
            dK[b, h // G] += k
            dV[b, h // G] += v
    return dQ, dK, dV


def attn_rows_fwd_bwd(Q, K, V, dO, f, a: int, n: int, rows, scale: float | None = None):
    """O, LSE and dQ for selected rows of one head (each is a function of its
    own row only).  Q, dO: [L][d]; rows: indices.  Used where L is too long to
    evaluate every row."""
    rows = np.asarray(rows)
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    d = Q.shape[1]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    M = mask_rows(f, a, n, rows)
    O, LSE, A = attn_fwd_rows(Q[rows], K, V, M, scale)
    dA = dO[rows] @ V.T
    delta = (dO[rows] * O).sum(axis=1, keepdims=True)
    dLam = A * (dA - delta)
    dQ = (dLam @ K) * scale
    return O, LSE, dQ


def attn_keys_bwd(Q, K, V, dO, f, a: int, n: int, keys, scale: float | None = None):
    """dK and dV of selected key positions for one query head (the caller sums
    over the query heads that share the KV head).  Q, dO, K, V: [L][d].

    A key's gradient gathers every query row that keeps it, so the rows that
    keep at least one selected key are evaluated in full (same formulas as
    attn_bwd_head) and only the selected columns are summed.  Used where L is
    too long to evaluate every row; pick keys that few rows keep."""
    keys = np.asarray(keys)
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    L, d = Q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    first = int(keys.min())
    cand = np.arange(first, L)
    Mc = mask_rows(f, a, n, cand)
    rows = cand[Mc[:, keys].any(axis=1)]
    M = mask_rows(f, a, n, rows)
    O, _, A = attn_fwd_rows(Q[rows], K, V, M, scale)
    dA = dO[rows] @ V.T
    delta = (dO[rows] * O).sum(axis=1, keepdims=True)
    dLam = A * (dA - delta)
    dK = (dLam[:, keys].T @ Q[rows]) * scale
    dV = A[:, keys].T @ dO[rows]
    return dK, dV


def attn_keys_bwd_blocked(Q, K, V, dO, f, a: int, n: int, keys, scale: float | None = None,
                          block_rows: int = 1024, with_term_scale: bool = False):
    """Same result as :func:`attn_keys_bwd` for keys that many rows keep (an
    initial token or an early separator of a long sequence is kept by every
    later row, and a dense [rows][L] evaluation of all of them at once does not
    fit in memory).

    The rows from the first selected key to the end are taken ``block_rows`` at
    a time.  Within a block only the columns that some row of the block keeps
    are evaluated: a column that no row of the block keeps has Lambda = -inf,
    hence weight 0, in every one of those rows, so leaving it out changes
    nothing.  Each row still sees every key it keeps, so its softmax is the
    full one of Eq. 1 under the mask of Eq. 2.  The formulas are those of
    :func:`attn_bwd_head`.  with_term_scale: also return the squares that
    :func:`attn_bwd_term_scale` sums, for the selected keys (dK, dV, sK2, sV2;
    the caller adds the squares over the query heads of a group and takes the
    root).
    """
    keys = np.asarray(keys)
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    L, d = Q.shape
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    dK = np.zeros((keys.size, d))
    dV = np.zeros((keys.size, d))
    sK2 = np.zeros((keys.size, d))
    sV2 = np.zeros((keys.size, d))
    for r0 in range(int(keys.min()), L, block_rows):
        rows = np.arange(r0, min(L, r0 + block_rows))
        # columns a row of this block can keep: initial tokens, separators, and the positions
        # within n of the block; the predicate of Eq. 2 is then evaluated on those columns only
        j = np.arange(int(rows[-1]) + 1)
        cols = np.flatnonzero((j < a) | f[j] | (j > r0 - n))
        M = mask_rows(f, a, n, rows, cols)
        rows_used = M[:, np.isin(cols, keys)].any(axis=1)
        if not rows_used.any():
            continue
        rows, M = rows[rows_used], M[rows_used]
        used = M.any(axis=0)                            # every selected key a row keeps is among them
        cols, M = cols[used], M[:, used]
        O, _, A = attn_fwd_rows(Q[rows], K[cols], V[cols], M, scale)
        dA = dO[rows] @ V[cols].T
        delta = (dO[rows] * O).sum(axis=1, keepdims=True)
        dLam = A * (dA - delta)
        where = np.searchsorted(cols, keys)             # column of each selected key inside the block
        present = (where < cols.size) & (cols[np.minimum(where, cols.size - 1)] == keys)
        w = where[present]
        dK[present] += (dLam[:, w].T @ Q[rows]) * scale
        dV[present] += A[:, w].T @ dO[rows]
        if with_term_scale:
            s_delta = np.sqrt(((dO[rows] * O) ** 2).sum(axis=1, keepdims=True))
            sK2[present] += ((dLam[:, w] ** 2 + (A[:, w] * s_delta) ** 2).T @ (Q[rows] ** 2)) * scale ** 2
            sV2[present] += (A[:, w] ** 2).T @ (dO[rows] ** 2)
    if with_term_scale:
        return dK, dV, sK2, sV2
    return dK, dV


def attn_bwd_term_scale(Q, K, V, dO, flags, a: int, n: int, scale: float | None = None, doc_first=None):
    """Size of the terms behind every gradient entry, for error bounds in tests.

    Each entry of dV, dK, dQ is a sum of products (A_ij dO_i, dLambda_ij Q_i,
    dLambda_ij K_j).  An implementation that rounds A and dLambda to bf16
    before its matrix products perturbs every term by up to 2^-9 of its size,
    independently from term to term, so the error of an entry grows like the
    root of the sum of its squared terms, not like the entry's own value (which
    may be small through cancellation).  The backward is also handed O as the
    bf16 tensor the forward wrote, and rowsum(dO * O) computed from it is off
    by up to 2^-9 of each product dO_ie O_ie; that error s_i enters dLambda_ij
    as A_ij s_i, whatever the size of dLambda_ij itself.  Returns the root of
    the sum of squares of both kinds of terms for dQ [B][Hq][L][d], dK and dV
    [B][Hkv][L][d] (summed over the query heads that share a KV head, as the
    gradients are; dV has no term of the second kind)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    B, Hq, L, d = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    sQ = np.zeros((B, Hq, L, d))
    sK = np.zeros((B, Hkv, L, d))
    sV = np.zeros((B, Hkv, L, d))
    for b in range(B):
        M = _batch_mask(flags, a, n, b, doc_first)
        for h in range(Hq):
            hk = h // G
            O, _, A = attn_fwd_rows(Q[b, h], K[b, hk], V[b, hk], M, scale)
            dA = dO[b, h] @ V[b, hk].T
            delta = (dO[b, h] * O).sum(axis=1, keepdims=True)
            dLam = A * (dA - delta)
            s_delta = np.sqrt(((dO[b, h] * O) ** 2).sum(axis=1, keepdims=True))
            both = dLam ** 2 + (A * s_delta) ** 2
            sQ[b, h] = both @ (K[b, hk] ** 2) * scale ** 2
            sK[b, hk] += both.T @ (Q[b, h] ** 2) * scale ** 2
            sV[b, hk] += (A ** 2).T @ (dO[b, h] ** 2)
    return np.sqrt(sQ), np.sqrt(sK), np.sqrt(sV)


def attn_fwd_term_scale(Q, K, V, flags, a: int, n: int, scale: float | None = None, doc_first=None):
    """Size of the terms behind every entry of O, for error bounds in tests: O_ie
    is the sum over kept keys j of A_ij V_je, and an implementation that rounds
    A to bf16 before the product perturbs every term by up to 2^-9 of its size.
    Returns the root of the sum of the squared terms, [B][Hq][L][d].  (A row
    that keeps one key has a single term, V itself.)"""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    B, Hq, L, d = Q.shape
    G = Hq // K.shape[1]
    out = np.zeros((B, Hq, L, d))
    for b in range(B):
        M = _batch_mask(flags, a, n, b, doc_first)
        for h in range(Hq):
            _, _, A = attn_fwd_rows(Q[b, h], K[b, h // G], V[b, h // G], M, scale)
            out[b, h] = np.sqrt((A ** 2) @ (V[b, h // G] ** 2))
    return out


# ----------------------------------------------------------------------------
# Index (the data the kernels consume; integers, compared bit for bit)
# ----------------------------------------------------------------------------

def build_index(token_ids: np.ndarray, sep_ids, a: int, n: int, BM: int, BN: int,
                side_cap: int, seq_len=None):
    """Canonical index arrays for a batch of sequences.

    seq_len (optional, one length per sequence): sequence b holds seq_len[b]
    tokens, the rest of its row is padding.  The paper does not treat batches
    of unequal lengths; the reading taken here is the obvious one: a padded
    position is no token (no initial token, no separator), a query tile whose
    first row is padding has no work (all eight metadata words 0), the last
    valid tile ends at the last valid row, and ``pairs`` counts valid rows only.
    cnt and lim keep their formulas on every position of the row.

    side member g[j] = (j < a) or f[j]            (initial tokens and separators)
    cnt[j]  = number of side members at positions < j, j = 0..L
    side_pos = ascending positions of side members, n_side = cnt[L]
    lim[i]  = cnt[max(0, i-n+1)]: side members at distance >= n from query i,
              i.e. those row i keeps that its neighbour window does not cover
    tile_meta[t] for the query tile of rows [t*BM, min(L,(t+1)*BM)):
      0 side_full  = floor(lim[first row] / BN)   side tiles every row sees in full
      1 side_last  = ceil(lim[last row] / BN)     side tiles some row sees
      2 win_lo     = max(0, first row - n + 1)    first key of the tile's window
      3 win_hi     = last row + 1                 one past its last key
      4 win_tile_lo = win_lo // BN
      5 win_tile_hi = ceil(win_hi / BN)
      6 pairs      = kept (query, key) pairs in the tile
      7 reserved (0)
    """
    token_ids = np.asarray(token_ids)
    B, L = token_ids.shape
    T = (L + BM - 1) // BM
    cnt = np.zeros((B, L + 1), dtype=np.int32)
    lim = np.zeros((B, L), dtype=np.int32)
    side_pos = np.full((B, side_cap), -1, dtype=np.int32)
    n_side = np.zeros((B,), dtype=np.int32)
    tile_meta = np.zeros((B, T, 8), dtype=np.int32)
    sep = set(int(x) for x in sep_ids)
    lens = np.full((B,), L, dtype=np.int32) if seq_len is None else np.asarray(seq_len, dtype=np.int32)
    for b in range(B):
        Lv = int(lens[b])
        k = 0
        for j in range(L):
            cnt[b, j] = k
            if j < Lv and (j < a or int(token_ids[b, j]) in sep):
                if k < side_cap:
                    side_pos[b, k] = j
                k += 1
        cnt[b, L] = k
        n_side[b] = k
        for i in range(L):
            lim[b, i] = cnt[b, max(0, i - n + 1)]
        for t in range(T):
            r0 = t * BM
            if r0 >= Lv:
                continue                      # a tile of padding: all words stay 0
            r1 = min(Lv, (t + 1) * BM) - 1
            pairs = 0
            for i in range(r0, r1 + 1):
                pairs += int(lim[b, i]) + min(i + 1, n)
            win_lo = max(0, r0 - n + 1)
            win_hi = r1 + 1
            tile_meta[b, t] = [int(lim[b, r0]) // BN, -(-int(lim[b, r1]) // BN), win_lo, win_hi,
                               win_lo // BN, -(-win_hi // BN), pairs, 0]
    return dict(cnt=cnt, lim=lim, side_pos=side_pos, n_side=n_side, tile_meta=tile_meta, seq_len=lens)


def build_index_fast(token_ids: np.ndarray, sep_ids, a: int, n: int, BM: int, BN: int,
                     side_cap: int, seq_len=None):
    """Same arrays as :func:`build_index`, with numpy prefix sums in place of
    the Python loops, for sequences too long to loop over.  Tests check the two
    against each other."""
    token_ids = np.asarray(token_ids)
    B, L = token_ids.shape
    T = (L + BM - 1) // BM
    lens = np.full((B,), L, dtype=np.int32) if seq_len is None else np.asarray(seq_len, dtype=np.int32)
    g = np.isin(token_ids, np.asarray(list(sep_ids))) | (np.arange(L)[None, :] < a)
    g &= np.arange(L)[None, :] < lens[:, None]
    cnt = np.zeros((B, L + 1), dtype=np.int64)
    cnt[:, 1:] = np.cumsum(g, axis=1)
    i = np.arange(L)
    lim = cnt[:, np.maximum(0, i - n + 1)]
    side_pos = np.full((B, side_cap), -1, dtype=np.int32)
    for b in range(B):
        p = np.nonzero(g[b])[0][:side_cap]
        side_pos[b, :p.size] = p
    per_row = lim + np.minimum(i + 1, n)[None, :]
    tile_meta = np.zeros((B, T, 8), dtype=np.int32)
    for b in range(B):
        Lv = int(lens[b])
        for t in range(T):
            r0 = t * BM
            if r0 >= Lv:
                break
            r1 = min(Lv, (t + 1) * BM) - 1
            win_lo = max(0, r0 - n + 1)
            win_hi = r1 + 1
            tile_meta[b, t] = [lim[b, r0] // BN, -(-lim[b, r1] // BN), win_lo, win_hi, win_lo // BN,
                               -(-win_hi // BN), per_row[b, r0:r1 + 1].sum(), 0]
    return dict(cnt=cnt.astype(np.int32), lim=lim.astype(np.int32), side_pos=side_pos,
                n_side=cnt[:, L].astype(np.int32), tile_meta=tile_meta, seq_len=lens)


def build_index_packed(token_ids: np.ndarray, doc_first: np.ndarray, sep_ids, a: int, n: int,
                       BM: int, BN: int, side_cap: int, seq_len=None):
    """Index arrays for rows that pack several documents (packed_mask_matrix).

    Side members are the separators and the first ``a`` tokens of every
    document; cnt, side_pos, n_side are as in build_index.  With start[i] /
    end[i] the bounds of row i's document (document_bounds):
      win_start[i] = max(i-n+1, start[i])   first key of the row's window
      lim[i]       = cnt[win_start[i]]      side members before the window ...
      side_lo[i]   = cnt[start[i]]          ... from the document's first one on:
                                            row i keeps side entries [side_lo, lim)
    doc_start = start, doc_end = end are part of the index (a key j is kept by
    queries up to end[j] - 1 only).  tile_meta as in build_index with
      0 side_full = floor(lim[first row] / BN), 1 side_last = ceil(lim[last row] / BN)
      2 win_lo = win_start[first row], 3 win_hi = last row + 1, 4, 5 their tiles
      6 pairs = sum over the tile's valid rows of (lim - side_lo) + (i - win_start + 1)
      7 side_first = floor(side_lo[first row] / BN)   first side tile any row sees
    """
    token_ids = np.asarray(token_ids)
    doc_first = np.asarray(doc_first)
    B, L = token_ids.shape
    T = (L + BM - 1) // BM
    cnt = np.zeros((B, L + 1), dtype=np.int32)
    lim = np.zeros((B, L), dtype=np.int32)
    doc_start = np.zeros((B, L), dtype=np.int32)
    doc_end = np.zeros((B, L), dtype=np.int32)
    side_pos = np.full((B, side_cap), -1, dtype=np.int32)
    n_side = np.zeros((B,), dtype=np.int32)
    tile_meta = np.zeros((B, T, 8), dtype=np.int32)
    sep = set(int(x) for x in sep_ids)
    lens = np.full((B,), L, dtype=np.int32) if seq_len is None else np.asarray(seq_len, dtype=np.int32)
    for b in range(B):
        Lv = int(lens[b])
        start, end = document_bounds(doc_first[b], Lv)
        doc_start[b], doc_end[b] = start, end
        k = 0
        for j in range(L):
            cnt[b, j] = k
            if j < Lv and (j - start[j] < a or int(token_ids[b, j]) in sep):
                if k < side_cap:
                    side_pos[b, k] = j
                k += 1
        cnt[b, L] = k
        n_side[b] = k
        win_start = [max(i - n + 1, int(start[i])) for i in range(L)]
        side_lo = [int(cnt[b, int(start[i])]) for i in range(L)]
        for i in range(L):
            lim[b, i] = cnt[b, win_start[i]]
        for t in range(T):
            r0 = t * BM
            if r0 >= Lv:
                continue
            r1 = min(Lv, (t + 1) * BM) - 1
            pairs = 0
            for i in range(r0, r1 + 1):
                pairs += int(lim[b, i]) - side_lo[i] + (i - win_start[i] + 1)
            win_lo, win_hi = win_start[r0], r1 + 1
            tile_meta[b, t] = [int(lim[b, r0]) // BN, -(-int(lim[b, r1]) // BN), win_lo, win_hi,
                               win_lo // BN, -(-win_hi // BN), pairs, side_lo[r0] // BN]
    return dict(cnt=cnt, lim=lim, side_pos=side_pos, n_side=n_side, tile_meta=tile_meta, seq_len=lens,
                doc_start=doc_start, doc_end=doc_end)


# ----------------------------------------------------------------------------
# Streaming cache (Section 3.3, "Tailored Streaming Design")
# ----------------------------------------------------------------------------

class StreamingCache:
    """The four cache blocks as lists of token positions.

    Initial Cache fills first and is never changed.  Every later token enters
    the neighbour run, whose newest ``w`` entries are the Local Window Cache and
    whose older entries are the Past Window Cache.  When the runtime size
    reaches ``c`` the separators of the Past Window Cache move to the Separator
    Cache in position order and the other Past Window entries are dropped; a
    Separator Cache holding more than ``s`` entries drops its oldest.
    """

    def __init__(self, a: int, s: int, w: int, c: int):
        if not (a + s + w < c):
            raise ValueError("the paper requires a + s + w < c")
        self.a, self.s, self.w, self.c = a, s, w, c
        self.init: List[int] = []
        self.sep: List[int] = []
        self.window: List[int] = []      # past window followed by local window
        self.window_is_sep: List[bool] = []
        self.next_pos = 0
        self.compactions = 0

    # sizes in the paper's names
    @property
    def size_init(self):
        return len(self.init)

    @property
    def size_sep(self):
        return len(self.sep)

    @property
    def size_local_w(self):
        return min(len(self.window), self.w)

    @property
    def size_past_w(self):
        return len(self.window) - self.size_local_w

    @property
    def n(self):
        return len(self.window)

    @property
    def size_run(self):
        return len(self.init) + len(self.sep) + len(self.window)

    def update(self, is_sep: bool) -> None:
        """Take in the next token of the stream."""
        pos = self.next_pos
        self.next_pos += 1
        if len(self.init) < self.a:
            self.init.append(pos)
            return
        self.window.append(pos)
        self.window_is_sep.append(bool(is_sep))
        if self.size_run == self.c:
            n_past = len(self.window) - self.w
            moved = [p for p, f in zip(self.window[:n_past], self.window_is_sep[:n_past]) if f]
            self.sep.extend(moved)
            if len(self.sep) > self.s:
                self.sep = self.sep[len(self.sep) - self.s:]
            self.window = self.window[n_past:]
            self.window_is_sep = self.window_is_sep[n_past:]
            self.compactions += 1

    def retained(self) -> List[int]:
        """Positions whose K/V the next decode step attends to."""
        return self.init + self.sep + self.window


class FundamentalCache:
    """Generation in the fundamental design (Section 3.2, "Generation"): after every token the KV
    kept are those of the initial tokens, of every separator seen so far and of the ``n`` most
    recent tokens; Section 4.2 runs this setting with all separator KV kept.  There is no
    capacity and nothing is ever evicted from the separator list.  A token that falls out of the
    window of the ``n`` most recent ones is kept on if it is a separator and dropped otherwise.
    Same attribute names as :class:`StreamingCache` (``compactions`` counts the steps at which a
    token left the window)."""

    def __init__(self, a: int, n: int):
        if n < 1:
            raise ValueError("n >= 1: the current token always attends to itself")
        self.a, self.n = a, n
        self.init: List[int] = []
        self.sep: List[int] = []
        self.window: List[int] = []
        self.window_is_sep: List[bool] = []
        self.next_pos = 0
        self.compactions = 0

    @property
    def size_run(self):
        return len(self.init) + len(self.sep) + len(self.window)

    def update(self, is_sep: bool) -> None:
        pos = self.next_pos
        self.next_pos += 1
        if len(self.init) < self.a:
            self.init.append(pos)
            return
        self.window.append(pos)
        self.window_is_sep.append(bool(is_sep))
        if len(self.window) > self.n:
            left, was_sep = self.window.pop(0), self.window_is_sep.pop(0)
            if was_sep:
                self.sep.append(left)
            self.compactions += 1

    def retained(self) -> List[int]:
        return self.init + self.sep + self.window


def cache_after_prompt(flags: Sequence[bool], a: int, s: int, w: int, c: int) -> StreamingCache:
    """The cache a prompt leaves behind for generation (Section 3.2 "Generation",
    Section 3.3): the state the machine above reaches after taking in the
    prompt's tokens one by one.  The paper describes no other way of going from
    a pre-filled prompt to the four blocks, so this is the definition the
    hand-off from pre-filling is held to."""
    cache = StreamingCache(a, s, w, c)
    for fl in flags:
        cache.update(bool(fl))
    return cache


def avg_neighbour_limit(w: int, c: int, a: int, s: int) -> float:
    """Eq. 3: long-run mean of n."""
    return (w + c - a - s) / 2.0


def avg_runtime_kv_limit(w: int, c: int, a: int, s: int) -> float:
    """Eq. 4: long-run mean of Size_run."""
    return (w + c + a + s) / 2.0


def decode_attention(q: np.ndarray, Kc: np.ndarray, Vc: np.ndarray, scale: float | None = None):
    """One query over a retained set: q [d], Kc, Vc [R][d].  Returns o [d], lse."""
    q = np.asarray(q, dtype=np.float64)
    Kc = np.asarray(Kc, dtype=np.float64)
    Vc = np.asarray(Vc, dtype=np.float64)
    d = q.shape[0]
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    lam = (Kc @ q) * scale
    mx = lam.max()
    e = np.exp(lam - mx)
    Z = e.sum()
    return (e / Z) @ Vc, mx + math.log(Z)


# ----------------------------------------------------------------------------
# Decode with positions inside the cache (Section 3.3, "Positional Encoding")
# ----------------------------------------------------------------------------

def rope_rotate(x: np.ndarray, pos, base: float) -> np.ndarray:
    """Rotary encoding, rotate-half form (the paper names no formula; this is
    the library's stated reading).  x [..., d]; pos broadcastable to x[..., 0].
    theta_i = base^(-2i/d); (x_i, x_{i+d/2}) turns by the angle pos * theta_i."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    h = d // 2
    theta = base ** (-2.0 * np.arange(h) / d)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta
    c, s = np.cos(ang), np.sin(ang)
    lo, hi = x[..., :h], x[..., h:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def decode_attention_rope(q, Kc, Vc, base: float, q_pos=None, k_pos=None, scale: float | None = None):
    """One un-rotated query over un-rotated retained keys given in cache order:
    key r sits at position r and the query at position R-1 (positions within
    the cache, not in the text), unless positions are passed explicitly."""
    Kc = np.asarray(Kc, dtype=np.float64)
    R = Kc.shape[0]
    k_pos = np.arange(R) if k_pos is None else np.asarray(k_pos)
    q_pos = R - 1 if q_pos is None else q_pos
    return decode_attention(rope_rotate(q, np.asarray(q_pos), base), rope_rotate(Kc, k_pos, base), Vc, scale)
