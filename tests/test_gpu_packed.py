"""Rows that pack several documents: sepllm_build_index_packed against the oracle's packed index
(bit for bit), and the attention calls on such an index against the oracle's packed attention
(Eq. 2 inside each document, nothing across a boundary)."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import (TOL_GRAD, TOL_LSE, TOL_O, assert_close, assert_grad_close,
                             assert_o_close, attn_bwd, attn_fwd, errors, flags_of)

pytestmark = pytest.mark.gpu
KEYS = ("cnt", "lim", "side_pos", "n_side", "tile_meta", "seq_len", "doc_start", "doc_end")


def _index(ids, df, lens, a, n, side_cap=None, BM=128, BN=128):
    B, L = ids.shape
    side_cap = L if side_cap is None else side_cap
    desc = api.IndexDesc(B, L, a, n, len(inputs.SEP_IDS), BM, BN, side_cap)
    ib, _ = api.sepllm_index_bytes(desc)
    index = api.alloc_bytes(ib)
    lens_d = None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda")
    api.sepllm_build_index_packed(desc, torch.from_numpy(np.ascontiguousarray(ids)).cuda(),
                                  torch.from_numpy(np.ascontiguousarray(df)).cuda(), lens_d, inputs.SEP_IDS, index)
    torch.cuda.synchronize()
    return desc, index


@pytest.mark.parametrize("L,a,n,mean,BM,BN", [(1000, 4, 64, 150.0, 128, 128), (5000, 3, 300, 700.0, 128, 128),
                                              (4097, 30, 17, 50.0, 64, 32), (3000, 0, 1, 3.0, 128, 128),
                                              (2048, 2, 4000, 400.0, 128, 128), (1024, 1, 8, 1.0, 128, 128)])
def test_packed_index_matches_oracle(L, a, n, mean, BM, BN):
    B = 4
    ids = inputs.token_ids(500 + L, B, L, 0.2)
    df = inputs.doc_first(500 + L, B, L, mean)
    for lens in (None, [L, L // 2 + 3, 129, 0]):
        desc, index = _index(ids, df, lens, a, n, BM=BM, BN=BN)
        got = api.read_index(index)
        ref = orc.build_index_packed(ids, df, inputs.SEP_IDS, a, n, BM, BN, L, seq_len=lens)
        for k in KEYS:
            assert np.array_equal(got[k], ref[k]), (k, lens)
        assert got["header"].status == 0 and got["header"].packed == 1


def test_packed_index_without_boundaries_equals_the_plain_index():
    L, B = 3000, 3
    ids = inputs.token_ids(43, B, L, 0.15)
    desc, a = _index(ids, np.zeros_like(ids), None, 4, 100)
    ib, sb = api.sepllm_index_bytes(desc)
    b = api.alloc_bytes(ib)
    api.sepllm_build_index(desc, torch.from_numpy(ids).cuda(), inputs.SEP_IDS, b, api.alloc_bytes(sb))
    torch.cuda.synchronize()
    ga, gb = api.read_index(a), api.read_index(b)
    for k in ("cnt", "lim", "side_pos", "n_side", "tile_meta", "seq_len"):
        assert np.array_equal(ga[k], gb[k]), k
    assert gb["header"].packed == 0


def test_packed_index_capacity_exceeded_is_reported():
    L = 600
    ids = inputs.token_ids(44, 1, L, 0.3)
    df = inputs.doc_first(44, 1, L, 20.0)
    desc, index = _index(ids, df, None, 2, 16, side_cap=40)
    got = api.read_index(index)
    ref = orc.build_index_packed(ids, df, inputs.SEP_IDS, 2, 16, 128, 128, 40)
    assert got["header"].status == api.CAPACITY_EXCEEDED
    assert np.array_equal(got["side_pos"], ref["side_pos"]) and np.array_equal(got["cnt"], ref["cnt"])


def _attention_case(B, Hq, Hkv, L, d, a, n, mean, rho, seed, grad_dtype=0, lens=None):
    ids = inputs.token_ids(seed, B, L, rho)
    df = inputs.doc_first(seed, B, L, mean)
    Q, K, V, dO = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    if lens is not None:
        for b in range(B):
            dO[b, :, lens[b]:] = 0
    idesc, index = _index(ids, df, lens, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype)
    f = flags_of(ids, inputs.SEP_IDS)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    O, LSE = O.float().cpu().numpy(), LSE.cpu().numpy()
    grads = [g.float().cpu().numpy() for g in (dQ, dK, dV)]
    for b in range(B):
        Lv = L if lens is None else lens[b]
        if Lv == 0:
            continue
        sl = (slice(b, b + 1), slice(None), slice(0, Lv))
        fb, dfb = f[b:b + 1, :Lv], df[b:b + 1, :Lv]
        Oref, LSEref = orc.attn_fwd(Qn[sl], Kn[sl], Vn[sl], fb, a, n, doc_first=dfb)
        assert_o_close(O[sl], Oref, orc.attn_fwd_term_scale(Qn[sl], Kn[sl], Vn[sl], fb, a, n, doc_first=dfb), f"O[{b}]")
        assert np.abs(LSE[b, :, :Lv] - LSEref[0]).max() <= TOL_LSE
        refs = orc.attn_bwd(Qn[sl], Kn[sl], Vn[sl], dOn[sl], fb, a, n, doc_first=dfb)
        scales = orc.attn_bwd_term_scale(Qn[sl], Kn[sl], Vn[sl], dOn[sl], fb, a, n, doc_first=dfb)
        for got, ref, rss, what in zip(grads, refs, scales, ("dQ", "dK", "dV")):
            assert_grad_close(got[sl], ref, rss, f"{what}[{b}]", bf16_out=(grad_dtype == 0))
            assert errors(got[sl], ref)[1] <= TOL_GRAD["rel_fro"], (what, b, errors(got[sl], ref))
        # keys of padding take no gradient
        assert not grads[1][b, :, Lv:].any() and not grads[2][b, :, Lv:].any()


@pytest.mark.parametrize("d,Hq,Hkv,grad_dtype", [(128, 4, 1, 0), (64, 2, 2, 0), (128, 3, 1, 1), (64, 4, 2, 0)])
@pytest.mark.parametrize("L,a,n,mean", [(1000, 3, 64, 170.0), (900, 2, 200, 60.0), (1100, 4, 16, 400.0)])
def test_attention_on_packed_rows(d, Hq, Hkv, grad_dtype, L, a, n, mean):
    _attention_case(2, Hq, Hkv, L, d, a, n, mean, 0.2, 520 + d + Hq + L, grad_dtype)


def test_attention_on_packed_rows_many_side_tiles():
    """Long documents with many separators: rows of a later document start their side tiles far
    from tile 0 and tiles in the middle of a document are kept in full."""
    _attention_case(1, 4, 1, 4096, 128, 4, 128, 1500.0, 0.3, 77)
    _attention_case(1, 2, 2, 4096, 64, 4, 128, 1500.0, 0.3, 78)


def test_attention_on_packed_rows_of_unequal_lengths():
    _attention_case(4, 4, 2, 1000, 128, 3, 100, 120.0, 0.2, 79, lens=[1000, 437, 130, 0])


def test_attention_with_documents_of_one_token():
    """Every token its own document: each row keeps only itself."""
    L = 300
    ids = inputs.token_ids(80, 1, L, 0.2)
    df = np.ones((1, L), dtype=np.int32)
    Q, K, V, dO = inputs.qkv_do(80, 1, 2, 1, L, 64)
    idesc, index = _index(ids, df, None, 4, 32)
    O, LSE = attn_fwd(Q.cuda(), K.cuda(), V.cuda(), idesc, index)
    # softmax over one key: O is that key's V row, LSE its score
    assert_close(O.float().cpu().numpy(), V.float().numpy().repeat(2, axis=1), TOL_O, "O")
    s = (Q.double().numpy() * K.double().numpy().repeat(2, axis=1)).sum(-1) / 8.0
    assert np.abs(LSE.cpu().numpy() - s).max() <= TOL_LSE


def test_prompt_hand_off_refuses_a_packed_index():
    L, B, Hkv, Hq, d = 512, 1, 1, 2, 64
    ids = inputs.token_ids(81, B, L, 0.2)
    idesc, index = _index(ids, inputs.doc_first(81, B, L, 100.0), None, 4, 64)
    cdesc = api.CacheDesc(B, Hkv, Hq, d, 4, 16, 32, 128, 0)
    sb, kvb = api.sepllm_cache_bytes(cdesc)
    state, Kc, Vc = api.alloc_bytes(sb), api.alloc_bytes(kvb), api.alloc_bytes(kvb)
    K = torch.zeros((B, Hkv, L, d), dtype=torch.bfloat16, device="cuda")
    api.sepllm_cache_from_prompt(cdesc, idesc, index, None, K, K, state, Kc, Vc)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(state) == api.INVALID_ARG
