"""Pins that hold the CPU oracle to the paper and to textbook routines.

None of these retype the oracle's own formula: they use Python-loop brute
force built from the paper's wording, torch's dense attention and autograd,
closed forms and values the paper prints.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(seed, L, d, p):
    g = np.random.default_rng(seed)
    f = g.random(L) < p
    Q = g.standard_normal((L, d))
    K = g.standard_normal((L, d))
    V = g.standard_normal((L, d))
    dO = g.standard_normal((L, d))
    return f, Q, K, V, dO


def _kept_set_from_words(f, a, n, i):
    """Section 3.1 in words: the first a tokens, every separator before the
    current token, the n closest tokens (the current one included)."""
    kept = set(range(min(a, i + 1)))
    kept |= {j for j in range(i + 1) if f[j]}
    kept |= {j for j in range(i, max(-1, i - n), -1)}
    return kept


@pytest.mark.parametrize("a,n", [(0, 1), (0, 3), (2, 1), (3, 5), (4, 64), (1, 200)])
def test_mask_matches_set_construction(a, n):
    f, *_ = _rand_case(a * 100 + n, 96, 4, 0.15)
    M = orc.mask_matrix(f, a, n)
    for i in range(96):
        assert set(np.nonzero(M[i])[0].tolist()) == _kept_set_from_words(f, a, n, i)
    rows = np.array([0, 5, 50, 95])
    assert (orc.mask_rows(f, a, n, rows) == M[rows]).all()
    cols = np.array([0, 1, 4, 49, 50, 51, 94, 95])
    assert (orc.mask_rows(f, a, n, rows, cols) == M[np.ix_(rows, cols)]).all()


def test_mask_regression_golden_ten_tokens():
    """Not a value of the paper (its mask figure is an image, only the caption's input "ABC,DE.FG\\n"
    is text): the mask of that input as written out by tests/golden/make_mask_golden.py, read back
    and checked by hand against Section 3.1 (row 9, the newline, keeps token 0, the separators 3
    and 6, and tokens 8, 9; row 7 keeps 0, 3 and the window 6, 7)."""
    sys_path = os.path.join(GOLD, "mask_10_tokens.txt")
    rows = [l.strip() for l in open(sys_path) if l.strip() and not l.startswith("#")]
    f = np.array([ch in ",.\n" for ch in "ABC,DE.FG\n"], dtype=bool)
    assert np.flatnonzero(f).tolist() == [3, 6, 9]
    M = orc.mask_matrix(f, 1, 2)
    assert ["".join("1" if x else "." for x in r) for r in M] == rows
    assert rows[9] == "1..1..1.11" and rows[7] == "1..1..11.." and rows[4] == "1..11....." and rows[0] == "1........."


def test_fixed_interval_variant_mask():
    """The appendix "Fixed-Interval Variant" in words: the initial tokens, one token every `interval`
    positions, the n closest tokens.  interval = 1 keeps everything (dense
    causal); an interval beyond the length keeps only position 0 besides the
    initial and neighbouring tokens (the StreamingLLM pattern when a >= 1)."""
    L, a, n = 90, 3, 7
    for interval in (1, 2, 5, 16, 200):
        f = orc.fixed_interval_flags(L, interval)
        assert f.sum() == (L + interval - 1) // interval and f[0]
        M = orc.mask_matrix(f, a, n)
        for i in range(L):
            kept = set(range(min(a, i + 1))) | set(range(0, i + 1, interval)) | set(range(max(0, i - n + 1), i + 1))
            assert set(np.nonzero(M[i])[0].tolist()) == kept
    assert (orc.mask_matrix(orc.fixed_interval_flags(L, 1), a, n) == np.tril(np.ones((L, L), bool))).all()
    assert (orc.mask_matrix(orc.fixed_interval_flags(L, 200), a, n)
            == orc.mask_matrix(np.zeros(L, bool), a, n)).all()


@pytest.mark.parametrize("a,n", [(0, 1), (2, 4), (4, 16)])
def test_forward_matches_python_loops(a, n):
    L, d = 40, 8
    f, Q, K, V, _ = _rand_case(7 + a + n, L, d, 0.2)
    O, LSE, A = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(f, a, n))
    for i in range(L):
        kept = sorted(_kept_set_from_words(f, a, n, i))
        lam = [sum(Q[i][t] * K[j][t] for t in range(d)) / math.sqrt(d) for j in kept]
        mx = max(lam)
        e = [math.exp(x - mx) for x in lam]
        Z = sum(e)
        o = [sum(e[k] / Z * V[j][t] for k, j in enumerate(kept)) for t in range(d)]
        assert np.allclose(O[i], o, rtol=1e-12, atol=1e-13)
        assert abs(LSE[i] - (mx + math.log(Z))) < 1e-12
        assert abs(A[i].sum() - 1.0) < 1e-12
        assert all(A[i][j] == 0.0 for j in range(L) if j not in kept)


def _torch_dense(Q, K, V, mask=None, causal=False):
    q, k, v = (torch.from_numpy(x)[None, None] for x in (Q, K, V))
    m = None if mask is None else torch.from_numpy(mask)[None, None]
    return torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=m, is_causal=causal)[0, 0].numpy()


def test_dense_causal_special_cases():
    L, d = 128, 16
    f, Q, K, V, _ = _rand_case(3, L, d, 0.1)
    ref = _torch_dense(Q, K, V, causal=True)
    # n >= L: every earlier token is a neighbour
    O1, _, _ = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(f, 2, L))
    # every token a separator
    O2, _, _ = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(np.ones(L, bool), 0, 1))
    assert np.allclose(O1, ref, atol=1e-12)
    assert np.allclose(O2, ref, atol=1e-12)


def test_sliding_window_and_streaming_special_cases():
    L, d, n = 96, 8, 7
    _, Q, K, V, _ = _rand_case(5, L, d, 0.0)
    none = np.zeros(L, bool)
    band = torch.ones(L, L, dtype=torch.bool).tril().triu(-(n - 1)).numpy()
    O, _, _ = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(none, 0, n))
    assert np.allclose(O, _torch_dense(Q, K, V, mask=band), atol=1e-12)
    # initial + neighbouring tokens only (the StreamingLLM mask)
    a = 3
    sink = band.copy()
    sink[:, :a] = True
    sink &= np.tril(np.ones((L, L), bool))
    O, _, _ = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(none, a, n))
    assert np.allclose(O, _torch_dense(Q, K, V, mask=sink), atol=1e-12)


def test_backward_matches_autograd_and_gqa_sum():
    B, Hq, Hkv, L, d, a, n = 2, 4, 2, 48, 8, 2, 5
    g = np.random.default_rng(11)
    flags = g.random((B, L)) < 0.2
    Q = g.standard_normal((B, Hq, L, d))
    K = g.standard_normal((B, Hkv, L, d))
    V = g.standard_normal((B, Hkv, L, d))
    dO = g.standard_normal((B, Hq, L, d))
    dQ, dK, dV = orc.attn_bwd(Q, K, V, dO, flags, a, n)
    O, LSE = orc.attn_fwd(Q, K, V, flags, a, n)
    q, k, v = (torch.tensor(x, requires_grad=True) for x in (Q, K, V))
    G = Hq // Hkv
    kk = k.repeat_interleave(G, dim=1)
    vv = v.repeat_interleave(G, dim=1)
    M = torch.stack([torch.from_numpy(orc.mask_matrix(flags[b], a, n)) for b in range(B)])[:, None]
    lam = (q @ kk.transpose(-1, -2)) / math.sqrt(d)
    lam = lam.masked_fill(~M, float("-inf"))
    o = torch.softmax(lam, dim=-1) @ vv
    (o * torch.tensor(dO)).sum().backward()
    assert np.allclose(O, o.detach().numpy(), atol=1e-12)
    assert np.allclose(LSE, torch.logsumexp(lam, dim=-1).detach().numpy(), atol=1e-12)
    assert np.allclose(dQ, q.grad.numpy(), atol=1e-11)
    assert np.allclose(dK, k.grad.numpy(), atol=1e-11)
    assert np.allclose(dV, v.grad.numpy(), atol=1e-11)


def test_backward_matches_finite_differences():
    L, d, a, n = 24, 4, 1, 3
    f, Q, K, V, dO = _rand_case(21, L, d, 0.25)
    M = orc.mask_matrix(f, a, n)
    dQ, dK, dV = orc.attn_bwd_head(Q, K, V, dO, M)

    def loss(q, k, v):
        return float((orc.attn_fwd_rows(q, k, v, M)[0] * dO).sum())

    h = 1e-6
    g = np.random.default_rng(0)
    for X, dX, which in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2)):
        for _ in range(12):
            i, t = int(g.integers(L)), int(g.integers(d))
            Xp, Xm = X.copy(), X.copy()
            Xp[i, t] += h
            Xm[i, t] -= h
            args_p = [Q, K, V]
            args_m = [Q, K, V]
            args_p[which] = Xp
            args_m[which] = Xm
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - dX[i, t]) <= 1e-6 * max(1.0, abs(fd))


def test_rows_variant_matches_full():
    L, d, a, n = 80, 8, 2, 6
    f, Q, K, V, dO = _rand_case(33, L, d, 0.2)
    M = orc.mask_matrix(f, a, n)
    O, LSE, _ = orc.attn_fwd_rows(Q, K, V, M)
    dQ, _, _ = orc.attn_bwd_head(Q, K, V, dO, M)
    rows = np.array([0, 1, 17, 79])
    o, lse, dq = orc.attn_rows_fwd_bwd(Q, K, V, dO, f, a, n, rows)
    assert np.allclose(o, O[rows]) and np.allclose(lse, LSE[rows]) and np.allclose(dq, dQ[rows])


# ---------------------------------------------------------------- Table 3
def test_attention_map_ratio_table3():
    for line in open(os.path.join(GOLD, "attention_map_ratio.txt")):
        if line.startswith("#") or not line.strip():
            continue
        L, a, n, printed = line.split()
        r = 100.0 * orc.attention_map_ratio(np.zeros(int(L), bool), int(a), int(n))
        assert f"{r:.2f}" == printed
    # brute-force count equals the row-wise count
    f, *_ = _rand_case(2, 200, 2, 0.12)
    assert orc.kept_pairs(f, 4, 16) == int(orc.mask_matrix(f, 4, 16).sum())


# ---------------------------------------------------------------- Eq. 3 / Eq. 4
def _golden_rkv():
    rows = []
    for line in open(os.path.join(GOLD, "runtime_kv_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        a, s, w, c, r = (int(x) for x in line.split()[:5])
        rows.append((a, s, w, c, r))
    return rows


def test_eq4_reproduces_printed_runtime_kv():
    rows = _golden_rkv()
    assert len(rows) == 10
    for a, s, w, c, printed in rows:
        assert orc.avg_runtime_kv_limit(w, c, a, s) == printed
        assert orc.avg_neighbour_limit(w, c, a, s) + a + s == printed


@pytest.mark.parametrize("a,s,w,c,printed", _golden_rkv()[:4] + _golden_rkv()[6:7])
def test_streaming_cache_simulation_meets_eq3_eq4(a, s, w, c, printed):
    g = np.random.default_rng(c + s)
    cache = orc.StreamingCache(a, s, w, c)
    period = c - a - s - w
    T = 60 * period + 4 * c
    sizes, ns = [], []
    first_full = None
    for t in range(T):
        cache.update(bool(g.random() < 0.3))
        assert cache.size_run <= c
        assert cache.size_run == cache.size_init + cache.size_sep + cache.size_past_w + cache.size_local_w
        assert cache.size_local_w <= w and cache.size_sep <= s and cache.size_init <= a
        if first_full is None and cache.size_sep == s and cache.compactions > 0:
            first_full = t
        if first_full is not None and t >= first_full + period:
            sizes.append(cache.size_run)
            ns.append(cache.n)
            assert w <= cache.n <= c - a - s
    assert min(ns) == w
    k = (len(ns) // period) * period      # whole periods
    assert abs(np.mean(sizes[:k]) - printed) <= 0.5
    assert abs(np.mean(ns[:k]) - orc.avg_neighbour_limit(w, c, a, s)) <= 0.5


def test_streaming_cache_keeps_what_the_mask_keeps():
    """With room for every separator, the retained set at step t is row t of
    the mask with n = the current length of the neighbour run."""
    a, s, w = 3, 100, 8
    g = np.random.default_rng(4)
    f = g.random(600) < 0.2
    cache = orc.StreamingCache(a, s, w, a + s + w + 13)
    checked_after_compaction = 0
    for t in range(600):
        cache.update(bool(f[t]))
        if cache.size_sep < s:        # nothing evicted yet
            row = orc.mask_rows(f, a, cache.n, np.array([t]))[0]
            assert sorted(cache.retained()) == np.nonzero(row)[0].tolist()
            checked_after_compaction += cache.compactions > 0
    assert cache.compactions >= 3 and checked_after_compaction > 50


def test_streaming_cache_fifo_and_order():
    cache = orc.StreamingCache(1, 2, 2, 8)
    flags = [0, 1, 1, 0, 1, 1, 1, 1, 0, 0, 1, 0, 0, 0]
    for fl in flags:
        cache.update(bool(fl))
    # step by step by hand: init=[0]; window fills 1..7 -> size 8 == c at pos 7:
    # past = [1..5], separators there 1,2,4,5 -> sep keeps the newest two [4,5]
    # window = [6,7]; then 8,9,10 appended (size 1+2+5 = 8 at pos 10):
    # past = [6,7,8], separators 6,7 -> sep = [6,7]; window = [9,10]; then 11,12,13
    # size = 1+2+5 = 8 at pos 13: past = [9,10,11], separator 10 -> sep = [7,10]
    assert cache.init == [0]
    assert cache.sep == [7, 10]
    assert cache.window == [12, 13]


def test_cache_after_prompt_has_the_content_the_blocks_are_defined_by():
    """Without running the state machine: the neighbour run is a contiguous
    stretch of positions ending at the prompt's last token, at least w and at
    most c - a - Size_sep - 1 long; the Separator Cache is the newest (at most
    s) separators between the initial tokens and that run.  Where the run
    starts (when the compactions happened) is pinned by the hand-worked stream
    at the end."""
    g = np.random.default_rng(12)
    for a, s, w, c in [(1, 2, 2, 8), (3, 4, 5, 20), (0, 3, 2, 9), (2, 0, 4, 11), (4, 16, 8, 40)]:
        for T in [0, 1, a, a + 1, c - 1, c, c + 1, 3 * c + 2, 11 * c + 5]:
            f = g.random(T) < 0.35
            cache = orc.cache_after_prompt(f, a, s, w, c)
            assert cache.init == list(range(min(T, a))) and cache.next_pos == T
            if T <= a:
                assert cache.sep == [] and cache.window == []
                continue
            lo = cache.window[0]
            assert cache.window == list(range(lo, T))
            seps = [j for j in range(a, lo) if f[j]]
            assert cache.sep == seps[max(0, len(seps) - s):]
            assert cache.window_is_sep == [bool(x) for x in f[lo:]]
            assert cache.size_run < c
            if cache.compactions == 0:
                assert lo == a and T < c
            else:
                assert w <= len(cache.window) <= c - a - cache.size_sep - 1
    # the worked example of the test above, cut at three prompt lengths
    flags = [0, 1, 1, 0, 1, 1, 1, 1, 0, 0, 1, 0, 0, 0]
    c7 = orc.cache_after_prompt(flags[:7], 1, 2, 2, 8)
    assert (c7.init, c7.sep, c7.window, c7.compactions) == ([0], [], [1, 2, 3, 4, 5, 6], 0)
    c8 = orc.cache_after_prompt(flags[:8], 1, 2, 2, 8)
    assert (c8.init, c8.sep, c8.window, c8.compactions) == ([0], [4, 5], [6, 7], 1)
    c12 = orc.cache_after_prompt(flags[:12], 1, 2, 2, 8)
    assert (c12.init, c12.sep, c12.window, c12.compactions) == ([0], [6, 7], [9, 10, 11], 2)


# ---------------------------------------------------------------- decode
def test_fundamental_cache_retains_exactly_the_mask_row():
    """Section 3.2: in generation the KV kept after token t are those row t of the mask keeps.
    FundamentalCache against mask_matrix (pinned above to the section's wording) after every
    token, for windows shorter and longer than the stream, with and without initial tokens."""
    rng = np.random.default_rng(12)
    for a, n, p in [(0, 1, 0.3), (2, 3, 0.3), (4, 9, 0.1), (3, 200, 0.2), (5, 4, 0.0), (1, 2, 1.0)]:
        L = 70
        f = rng.random(L) < p
        M = orc.mask_matrix(f, a, n)
        cache = orc.FundamentalCache(a, n)
        for t in range(L):
            cache.update(bool(f[t]))
            assert sorted(cache.retained()) == np.flatnonzero(M[t]).tolist(), (a, n, t)
            assert cache.retained() == sorted(cache.retained())          # position order
            assert len(cache.window) == min(n, max(0, t + 1 - a))
        assert cache.compactions == max(0, L - a - n)


def test_decode_equals_last_prefill_row():
    L, d, a, n = 70, 8, 2, 9
    f, Q, K, V, _ = _rand_case(9, L, d, 0.2)
    O, LSE, _ = orc.attn_fwd_rows(Q, K, V, orc.mask_matrix(f, a, n))
    t = L - 1
    kept = sorted(_kept_set_from_words(f, a, n, t))
    o, lse = orc.decode_attention(Q[t], K[kept], V[kept])
    assert np.allclose(o, O[t], atol=1e-13) and abs(lse - LSE[t]) < 1e-12
    o1, lse1 = orc.decode_attention(Q[t], K[5:6], V[5:6])
    assert np.allclose(o1, V[5])


# ---------------------------------------------------------------- index
@pytest.mark.parametrize("L,a,n,BM,BN", [(300, 4, 64, 128, 128), (129, 0, 1, 128, 128), (64, 3, 500, 32, 16)])
def test_index_invariants(L, a, n, BM, BN):
    g = np.random.default_rng(L)
    sep_ids = [5, 7, 9]
    ids = g.integers(0, 40, size=(2, L)).astype(np.int32)
    idx = orc.build_index(ids, sep_ids, a, n, BM, BN, side_cap=L)
    fast = orc.build_index_fast(ids, sep_ids, a, n, BM, BN, side_cap=L)
    for k in idx:
        assert idx[k].dtype == fast[k].dtype and (idx[k] == fast[k]).all(), k
    for b in range(2):
        f = orc.separator_flags(ids[b], sep_ids)
        M = orc.mask_matrix(f, a, n)
        cnt, lim, sp, ns = idx["cnt"][b], idx["lim"][b], idx["side_pos"][b], int(idx["n_side"][b])
        assert (np.diff(cnt) >= 0).all() and cnt[L] == ns
        assert (np.diff(sp[:ns]) > 0).all() and (sp[ns:] == -1).all()
        assert (np.diff(lim) >= 0).all() and (lim <= cnt[1:]).all()
        # row i keeps exactly side entries [0, lim[i]) plus its window
        for i in range(L):
            kept = set(sp[:lim[i]].tolist()) | set(range(max(0, i - n + 1), i + 1))
            assert kept == set(np.nonzero(M[i])[0].tolist())
            assert len(kept) == lim[i] + min(i + 1, n)      # the two parts are disjoint
        assert idx["tile_meta"][b, :, 6].sum() == M.sum() == orc.kept_pairs(f, a, n)
        T = (L + BM - 1) // BM
        for t in range(T):
            sf, sl, wl, wh, tl, th, _, z = idx["tile_meta"][b, t]
            rows = range(t * BM, min(L, (t + 1) * BM))
            assert sf * BN <= min(lim[i] for i in rows) < (sf + 1) * BN
            assert (sl - 1) * BN < max(lim[i] for i in rows) <= sl * BN or (sl == 0 and max(lim[i] for i in rows) == 0)
            assert wl == max(0, rows[0] - n + 1) and wh == rows[-1] + 1
            assert tl * BN <= wl < (tl + 1) * BN and (th - 1) * BN < wh <= th * BN and z == 0


def test_index_with_lengths_is_the_index_of_the_truncated_sequences():
    """A batch padded to a common length, with its lengths given, must index every sequence as if
    it stood alone at its own length (valid positions, valid tiles), leave tiles of padding empty,
    and count nothing behind the end; the prefix-sum version agrees with the loops."""
    rng = np.random.default_rng(21)
    B, L, a, n, BM, BN = 5, 300, 3, 17, 32, 16
    ids = rng.integers(0, 12, size=(B, L)).astype(np.int32)
    sep = [2, 7]
    lens = np.array([300, 299, 97, 1, 0], dtype=np.int32)
    full = orc.build_index(ids, sep, a, n, BM, BN, L, seq_len=lens)
    fast = orc.build_index_fast(ids, sep, a, n, BM, BN, L, seq_len=lens)
    for k in ("cnt", "lim", "side_pos", "n_side", "tile_meta", "seq_len"):
        assert np.array_equal(full[k], fast[k]), k
    for b in range(B):
        Lv = int(lens[b])
        if Lv == 0:
            assert full["n_side"][b] == 0 and not full["tile_meta"][b].any() and not full["cnt"][b].any()
            continue
        alone = orc.build_index(ids[b:b + 1, :Lv], sep, a, n, BM, BN, L)
        Tv = (Lv + BM - 1) // BM
        assert np.array_equal(full["cnt"][b, :Lv + 1], alone["cnt"][0])
        assert (full["cnt"][b, Lv:] == alone["n_side"][0]).all()          # nothing is counted behind the end
        assert np.array_equal(full["lim"][b, :Lv], alone["lim"][0])
        assert np.array_equal(full["side_pos"][b], alone["side_pos"][0]) and full["n_side"][b] == alone["n_side"][0]
        assert np.array_equal(full["tile_meta"][b, :Tv], alone["tile_meta"][0])
        assert not full["tile_meta"][b, Tv:].any()
    # without lengths nothing changes
    plain = orc.build_index(ids, sep, a, n, BM, BN, L)
    same = orc.build_index(ids, sep, a, n, BM, BN, L, seq_len=np.full(B, L))
    for k in ("cnt", "lim", "side_pos", "n_side", "tile_meta"):
        assert np.array_equal(plain[k], same[k])


def test_selected_key_gradients_equal_the_all_rows_backward():
    """attn_keys_bwd (used at sizes where not every row can be evaluated) against attn_bwd_head,
    which is pinned above by autograd and finite differences."""
    rng = np.random.default_rng(5)
    L, d, a, n = 90, 8, 2, 7
    f = rng.random(L) < 0.2
    Q, K, V, dO = (rng.standard_normal((L, d)) for _ in range(4))
    M = orc.mask_matrix(f, a, n)
    _, dK, dV = orc.attn_bwd_head(Q, K, V, dO, M)
    keys = np.array([40, 41, 55, 70, 88, 89])
    keys = np.concatenate([keys, np.flatnonzero(f)[-2:]])
    gk, gv = orc.attn_keys_bwd(Q, K, V, dO, f, a, n, keys)
    assert np.allclose(gk, dK[keys], rtol=1e-12, atol=1e-12)
    assert np.allclose(gv, dV[keys], rtol=1e-12, atol=1e-12)


def test_blocked_key_gradients_equal_the_all_rows_backward():
    """attn_keys_bwd_blocked (keys that nearly every row keeps, rows taken in blocks, columns no
    row of a block keeps left out) against attn_bwd_head; block sizes that split the rows
    unevenly, keys of every class (initial token, separators, plain tokens near and far)."""
    rng = np.random.default_rng(6)
    L, d, a, n = 150, 8, 2, 9
    f = rng.random(L) < 0.15
    Q, K, V, dO = (rng.standard_normal((L, d)) for _ in range(4))
    M = orc.mask_matrix(f, a, n)
    _, dK, dV = orc.attn_bwd_head(Q, K, V, dO, M)
    seps = np.flatnonzero(f)
    keys = np.unique(np.concatenate([[0, 1, 2, 60, 149], seps[:3], seps[-2:]]))
    for block in (7, 64, 1000):
        gk, gv = orc.attn_keys_bwd_blocked(Q, K, V, dO, f, a, n, keys, block_rows=block)
        assert np.allclose(gk, dK[keys], rtol=1e-12, atol=1e-12)
        assert np.allclose(gv, dV[keys], rtol=1e-12, atol=1e-12)
    # the squared term sizes of the same keys against the all-rows version
    flags2 = f[None, :]
    _, sK, sV = orc.attn_bwd_term_scale(Q[None, None], K[None, None], V[None, None], dO[None, None], flags2, a, n)
    _, _, k2, v2 = orc.attn_keys_bwd_blocked(Q, K, V, dO, f, a, n, keys, block_rows=13, with_term_scale=True)
    assert np.allclose(np.sqrt(k2), sK[0, 0][keys], rtol=1e-10) and np.allclose(np.sqrt(v2), sV[0, 0][keys], rtol=1e-10)
    # unsorted key list, custom scale
    perm = keys[::-1]
    gk, gv = orc.attn_keys_bwd_blocked(Q, K, V, dO, f, a, n, perm, scale=0.3, block_rows=11)
    _, dK3, dV3 = orc.attn_bwd_head(Q, K, V, dO, M, 0.3)
    assert np.allclose(gk, dK3[perm], atol=1e-12) and np.allclose(gv, dV3[perm], atol=1e-12)


def test_term_scale_is_the_root_sum_square_of_the_gradient_terms():
    """attn_bwd_term_scale against the terms written out one by one with torch (softmax over an
    explicitly built kept set), including the sum over the query heads of a group; and the two
    inequalities any root-sum-square obeys against the gradient itself."""
    rng = np.random.default_rng(8)
    B, Hq, Hkv, L, d, a, n = 1, 4, 2, 40, 4, 1, 5
    G = Hq // Hkv
    f = rng.random((B, L)) < 0.2
    Q = rng.standard_normal((B, Hq, L, d))
    K = rng.standard_normal((B, Hkv, L, d))
    V = rng.standard_normal((B, Hkv, L, d))
    dO = rng.standard_normal((B, Hq, L, d))
    sQ, sK, sV = orc.attn_bwd_term_scale(Q, K, V, dO, f, a, n)
    keep = torch.zeros((L, L), dtype=torch.bool)
    for i in range(L):
        keep[i, sorted(_kept_set_from_words(f[0], a, n, i))] = True
    tK = torch.zeros((Hkv, L, d), dtype=torch.float64)
    tV = torch.zeros((Hkv, L, d), dtype=torch.float64)
    for h in range(Hq):
        q, k, v, g = (torch.from_numpy(x) for x in (Q[0, h], K[0, h // G], V[0, h // G], dO[0, h]))
        lam = (q @ k.T) / math.sqrt(d)
        A = torch.softmax(lam.masked_fill(~keep, float("-inf")), dim=1)
        o = A @ v
        dlam = A * (g @ v.T - (g * o).sum(dim=1, keepdim=True))
        s_row = ((g * o) ** 2).sum(dim=1).sqrt()                       # size of the products behind rowsum(dO * O)
        terms_v = A[:, :, None] * g[:, None, :]                       # [i][j][e]
        terms_k = dlam[:, :, None] * q[:, None, :] / math.sqrt(d)
        terms_q = dlam[:, :, None] * k[None, :, :] / math.sqrt(d)     # [i][j][e]
        extra_k = (A * s_row[:, None])[:, :, None] * q[:, None, :] / math.sqrt(d)
        extra_q = (A * s_row[:, None])[:, :, None] * k[None, :, :] / math.sqrt(d)
        tV[h // G] += (terms_v ** 2).sum(dim=0)
        tK[h // G] += (terms_k ** 2).sum(dim=0) + (extra_k ** 2).sum(dim=0)
        assert np.allclose(sQ[0, h], ((terms_q ** 2).sum(dim=1) + (extra_q ** 2).sum(dim=1)).sqrt().numpy(),
                           rtol=1e-10, atol=1e-14)
    assert np.allclose(sK[0], tK.sqrt().numpy(), rtol=1e-10, atol=1e-14)
    assert np.allclose(sV[0], tV.sqrt().numpy(), rtol=1e-10, atol=1e-14)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, dO, f, a, n)
    for grad, s, terms in ((dQ, sQ, L), (dK, sK, L * G), (dV, sV, L * G)):
        assert (np.abs(grad) <= math.sqrt(terms) * s + 1e-12).all()      # Cauchy-Schwarz


def test_rope_decode_pins():
    """The rotary decode of the oracle against what the mathematics fixes: rotation as complex
    multiplication (an independent formulation), norm preservation, dependence on position
    differences only, and no rotation at all when every position is the same."""
    rng = np.random.default_rng(9)
    d, R, base = 16, 23, 10000.0
    q = rng.standard_normal(d)
    K = rng.standard_normal((R, d))
    V = rng.standard_normal((R, d))
    h = d // 2
    theta = base ** (-2.0 * np.arange(h) / d)
    # complex form: z_i = x_i + 1j x_{i+h}, rotated by exp(1j p theta_i); score = Re sum zq conj(zk)
    zq = (q[:h] + 1j * q[h:]) * np.exp(1j * (R - 1) * theta)
    zk = (K[:, :h] + 1j * K[:, h:]) * np.exp(1j * np.arange(R)[:, None] * theta)
    lam = np.real((zk.conj() * zq).sum(axis=1)) / math.sqrt(d)
    e = np.exp(lam - lam.max())
    o_ref = (e / e.sum()) @ V
    o, lse = orc.decode_attention_rope(q, K, V, base)
    assert np.allclose(o, o_ref, rtol=1e-12, atol=1e-12)
    assert abs(lse - (lam.max() + math.log(e.sum()))) < 1e-12
    assert np.allclose(np.linalg.norm(orc.rope_rotate(K, np.arange(R), base), axis=1), np.linalg.norm(K, axis=1))
    o_shift, _ = orc.decode_attention_rope(q, K, V, base, q_pos=R - 1 + 37, k_pos=np.arange(R) + 37)
    assert np.allclose(o_shift, o, rtol=1e-9, atol=1e-11)
    o_same, l_same = orc.decode_attention_rope(q, K, V, base, q_pos=5, k_pos=np.full(R, 5))
    o_plain, l_plain = orc.decode_attention(q, K, V)
    assert np.allclose(o_same, o_plain, rtol=1e-10, atol=1e-12) and abs(l_same - l_plain) < 1e-10


# ----------------------------------------------------------------------------
# Rows that pack several documents
# ----------------------------------------------------------------------------

def _docs_of(df):
    """[(start, end)] of the documents of one row, from the boundary marks alone."""
    cuts = [0] + [int(j) for j in np.nonzero(df)[0] if j > 0] + [len(df)]
    return [(cuts[k], cuts[k + 1]) for k in range(len(cuts) - 1) if cuts[k + 1] > cuts[k]]


def test_packed_mask_is_the_per_document_mask_on_the_diagonal_blocks():
    """The packed mask restricted to a document equals Eq. 2's mask of that document alone, and
    everything outside the diagonal blocks is 0."""
    for seed, (L, a, n, mean) in enumerate([(60, 2, 5, 9.0), (97, 0, 3, 20.0), (40, 4, 64, 6.0), (33, 1, 1, 1.5)]):
        ids = inputs.token_ids(40 + seed, 1, L, 0.2)[0]
        f = orc.separator_flags(ids, inputs.SEP_IDS)
        df = inputs.doc_first(40 + seed, 1, L, mean)[0]
        M = orc.packed_mask_matrix(f, df, a, n)
        expect = np.zeros((L, L), dtype=bool)
        for s, e in _docs_of(df):
            expect[s:e, s:e] = orc.mask_matrix(f[s:e], a, n)
        assert np.array_equal(M, expect)
    # no boundary marks: the plain mask
    f = orc.separator_flags(inputs.token_ids(3, 1, 50, 0.2)[0], inputs.SEP_IDS)
    assert np.array_equal(orc.packed_mask_matrix(f, np.zeros(50, dtype=np.int32), 3, 7), orc.mask_matrix(f, 3, 7))


def test_packed_attention_is_attention_on_every_document_by_itself():
    B, Hq, Hkv, L, d, a, n = 2, 4, 2, 90, 8, 2, 6
    ids = inputs.token_ids(51, B, L, 0.2)
    f = np.stack([orc.separator_flags(ids[b], inputs.SEP_IDS) for b in range(B)])
    df = inputs.doc_first(51, B, L, 14.0)
    Q, K, V, dO = (t.double().numpy() for t in inputs.qkv_do(51, B, Hq, Hkv, L, d))
    O, LSE = orc.attn_fwd(Q, K, V, f, a, n, doc_first=df)
    dQ, dK, dV = orc.attn_bwd(Q, K, V, dO, f, a, n, doc_first=df)
    for b in range(B):
        for s, e in _docs_of(df[b]):
            sl = (slice(b, b + 1), slice(None), slice(s, e))
            o, lse = orc.attn_fwd(Q[sl], K[sl], V[sl], f[b:b + 1, s:e], a, n, scale=1.0 / np.sqrt(d))
            assert np.allclose(O[sl], o, atol=1e-12) and np.allclose(LSE[sl], lse, atol=1e-12)
            q, k, v = orc.attn_bwd(Q[sl], K[sl], V[sl], dO[sl], f[b:b + 1, s:e], a, n, scale=1.0 / np.sqrt(d))
            assert np.allclose(dQ[sl], q, atol=1e-12) and np.allclose(dK[sl], k, atol=1e-12)
            assert np.allclose(dV[sl], v, atol=1e-12)


def test_packed_index_encodes_the_packed_mask_row_by_row():
    """Row i of the packed mask is exactly: side entries [cnt[doc_start[i]], lim[i]) plus the keys
    from max(i-n+1, doc_start[i]) to i; a key j is kept by no query at or after doc_end[j]; the tile
    words follow from the row values; pairs is the mask's row sum over the tile."""
    BM = BN = 16
    for seed, (L, a, n, mean, lens) in enumerate([(150, 2, 7, 23.0, None), (130, 0, 20, 40.0, [101, 130]),
                                                  (64, 3, 1, 5.0, [64, 17]), (100, 1, 200, 30.0, None)]):
        B = 2
        ids = inputs.token_ids(60 + seed, B, L, 0.15)
        df = inputs.doc_first(60 + seed, B, L, mean)
        idx = orc.build_index_packed(ids, df, inputs.SEP_IDS, a, n, BM, BN, L, seq_len=lens)
        for b in range(B):
            Lv = L if lens is None else lens[b]
            f = orc.separator_flags(ids[b], inputs.SEP_IDS)
            M = orc.packed_mask_matrix(f[:Lv], df[b, :Lv], a, n)
            sp, cnt, lim = idx["side_pos"][b], idx["cnt"][b], idx["lim"][b]
            ds, de = idx["doc_start"][b], idx["doc_end"][b]
            for i in range(Lv):
                ws = max(i - n + 1, int(ds[i]))
                kept = set(int(x) for x in sp[cnt[ds[i]]:lim[i]]) | set(range(ws, i + 1))
                assert kept == set(np.nonzero(M[i])[0].tolist()), (seed, b, i)
                assert len(kept) == (lim[i] - cnt[ds[i]]) + (i - ws + 1)      # the two parts do not overlap
            for j in range(Lv):
                assert not M[de[j]:, j].any() and (de[j] == Lv or df[b, de[j]])
                assert ds[j] == 0 or df[b, ds[j]]
            for t in range((L + BM - 1) // BM):
                m = idx["tile_meta"][b, t]
                r0, r1 = t * BM, min(Lv, (t + 1) * BM) - 1
                if r0 >= Lv:
                    assert not m.any()
                    continue
                assert m[6] == M[r0:r1 + 1].sum()
                assert m[0] == lim[r0] // BN and m[1] == -(-lim[r1] // BN) and m[7] == cnt[ds[r0]] // BN
                assert m[2] == max(r0 - n + 1, ds[r0]) and m[3] == r1 + 1
                assert m[4] == m[2] // BN and m[5] == -(-m[3] // BN)


def test_packed_index_without_boundaries_is_the_plain_index():
    ids = inputs.token_ids(70, 2, 200, 0.1)
    plain = orc.build_index(ids, inputs.SEP_IDS, 3, 11, 16, 16, 200, seq_len=[200, 77])
    packed = orc.build_index_packed(ids, np.zeros_like(ids), inputs.SEP_IDS, 3, 11, 16, 16, 200, seq_len=[200, 77])
    for k in ("cnt", "side_pos", "n_side", "tile_meta", "seq_len"):
        assert np.array_equal(plain[k], packed[k]), k
    # lim differs only on rows of padding, where the packed builder takes cnt at the row itself
    assert np.array_equal(plain["lim"][0], packed["lim"][0]) and np.array_equal(plain["lim"][1, :77], packed["lim"][1, :77])


def test_forward_term_scale_is_the_root_sum_square_of_the_terms_of_O():
    B, Hq, Hkv, L, d, a, n = 1, 2, 1, 40, 6, 2, 5
    ids = inputs.token_ids(90, B, L, 0.2)
    f = np.stack([orc.separator_flags(ids[b], inputs.SEP_IDS) for b in range(B)])
    Q, K, V, _ = (t.double() for t in inputs.qkv_do(90, B, Hq, Hkv, L, d))
    rss = orc.attn_fwd_term_scale(Q.numpy(), K.numpy(), V.numpy(), f, a, n)
    M = torch.from_numpy(orc.mask_matrix(f[0], a, n))
    for h in range(Hq):
        S = (Q[0, h] @ K[0, 0].T) / math.sqrt(d)
        A = torch.softmax(S.masked_fill(~M, float("-inf")), dim=-1)
        terms = A[:, :, None] * V[0, 0][None, :, :]          # [i][j][e]
        assert np.allclose(rss[0, h], terms.pow(2).sum(1).sqrt().numpy(), rtol=1e-12, atol=1e-15)
        assert np.allclose(terms.sum(1).numpy(), orc.attn_fwd(Q.numpy(), K.numpy(), V.numpy(), f, a, n)[0][0, h])
    # a row with one key: the single term is V itself
    assert np.allclose(rss[0, :, 0], np.abs(V[0, 0, 0].numpy())[None, :])
