"""Batches of unequal lengths: sepllm_build_index_varlen against the oracle's index with lengths,
and attention on such an index against the oracle run on every sequence cut to its own length.
Query tiles that hold only padding are skipped: their rows of O, LSE and dQ keep what the buffers
held, their rows of dK and dV are written as 0."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_GRAD, TOL_LSE, TOL_O, assert_close, assert_grad_close, errors, flags_of

pytestmark = pytest.mark.gpu
KEYS = ("cnt", "lim", "side_pos", "n_side", "tile_meta", "seq_len")


def _index(ids, lens, a, n, side_cap=None, BM=128, BN=128):
    B, L = ids.shape
    side_cap = L if side_cap is None else side_cap
    desc = api.IndexDesc(B, L, a, n, len(inputs.SEP_IDS), BM, BN, side_cap)
    ib, sb = api.sepllm_index_bytes(desc)
    index, scratch = api.alloc_bytes(ib), api.alloc_bytes(sb)
    api.sepllm_build_index_varlen(desc, torch.from_numpy(np.ascontiguousarray(ids)).cuda(),
                                  torch.tensor(lens, dtype=torch.int32, device="cuda"), inputs.SEP_IDS, index,
                                  scratch)
    torch.cuda.synchronize()
    return desc, index


@pytest.mark.parametrize("L,a,n,BM,BN", [(1000, 4, 64, 128, 128), (5000, 3, 300, 128, 128), (4097, 300, 17, 64, 32),
                                         (9000, 0, 1, 128, 128)])
def test_index_with_lengths_matches_oracle(L, a, n, BM, BN):
    B = 7
    ids = inputs.token_ids(400 + L, B, L, 0.2)
    lens = [L, L - 1, (L // 128) * 128, L // 2 + 3, 129, 1, 0]
    desc, index = _index(ids, lens, a, n, BM=BM, BN=BN)
    got = api.read_index(index)
    ref = orc.build_index_fast(ids, inputs.SEP_IDS, a, n, BM, BN, L, seq_len=np.array(lens))
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k
    assert got["header"].status == 0
    # lengths outside [0, L] are clamped
    desc, index = _index(ids, [L + 50, -3] + lens[2:], a, n, BM=BM, BN=BN)
    got = api.read_index(index)
    ref = orc.build_index_fast(ids, inputs.SEP_IDS, a, n, BM, BN, L, seq_len=np.array([L, 0] + lens[2:]))
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k


def test_index_with_full_lengths_equals_the_plain_index():
    L, B = 3000, 3
    ids = inputs.token_ids(41, B, L, 0.15)
    desc, a = _index(ids, [L] * B, 4, 100)
    ib, sb = api.sepllm_index_bytes(desc)
    b = api.alloc_bytes(ib)
    api.sepllm_build_index(desc, torch.from_numpy(ids).cuda(), inputs.SEP_IDS, b, api.alloc_bytes(sb))
    torch.cuda.synchronize()
    ga, gb = api.read_index(a), api.read_index(b)
    for k in KEYS:
        assert np.array_equal(ga[k], gb[k]), k


@pytest.mark.parametrize("d,Hq,Hkv,grad_dtype", [(128, 4, 1, 0), (64, 2, 2, 0), (128, 3, 1, 1)])
def test_attention_on_sequences_of_unequal_lengths(d, Hq, Hkv, grad_dtype):
    """d = 128 with four heads per group runs the CTA-pair forward, the others the single-CTA
    forward with two adjacent tiles (or two heads) per CTA; all of them the same backward."""
    L, a, n = 1000, 4, 100
    lens = [1000, 437, 384, 130, 77, 0]
    B = len(lens)
    seed = 420 + d + Hq
    ids = inputs.token_ids(seed, B, L, 0.2)
    Q, K, V, dO = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    for b in range(B):
        dO[b, :, lens[b]:] = 0            # the caller's part of the contract for padded rows
    idesc, index = _index(ids, lens, a, n)
    desc = api.AttnDesc(B, Hq, Hkv, d, L, 0.0, grad_dtype)
    _, bb = api.sepllm_attn_workspace_bytes(desc, idesc)
    ws = api.alloc_bytes(bb)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    gdt = torch.bfloat16 if grad_dtype == 0 else torch.float32
    sentinel = 7.0
    O = torch.full_like(Qd, sentinel)
    LSE = torch.full((B, Hq, L), sentinel, dtype=torch.float32, device="cuda")
    dQ = torch.full(Q.shape, sentinel, dtype=gdt, device="cuda")
    dK = torch.full(K.shape, sentinel, dtype=gdt, device="cuda")
    dV = torch.full(V.shape, sentinel, dtype=gdt, device="cuda")
    api.sepllm_attn_fwd(desc, idesc, Qd, Kd, Vd, index, O, LSE, ws)
    # rows the forward did not write must not feed the backward with garbage: give it zeros there
    Ob = O.clone()
    for b in range(B):
        first_skipped = -(-lens[b] // 128) * 128
        Ob[b, :, first_skipped:] = 0
    LSEb = torch.where(LSE == sentinel, torch.zeros_like(LSE), LSE)
    api.sepllm_attn_bwd(desc, idesc, dOd, Qd, Kd, Vd, Ob, LSEb, index, dQ, dK, dV, ws)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(ws) == 0
    G = Hq // Hkv
    f = flags_of(ids, inputs.SEP_IDS)
    On, Ln = O.float().cpu().numpy(), LSE.cpu().numpy()
    dQn, dKn, dVn = dQ.float().cpu().numpy(), dK.float().cpu().numpy(), dV.float().cpu().numpy()
    for b in range(B):
        Lv = lens[b]
        first_skipped = -(-Lv // 128) * 128
        # skipped tiles: untouched O / LSE / dQ, zero dK / dV; padded keys of the last valid tile: zero
        assert (On[b, :, first_skipped:] == sentinel).all() and (Ln[b, :, first_skipped:] == sentinel).all()
        assert (dQn[b, :, first_skipped:] == sentinel).all()
        assert (dKn[b, :, Lv:] == 0).all() and (dVn[b, :, Lv:] == 0).all()
        if Lv == 0:
            continue
        cut = lambda t: t[b:b + 1, :, :Lv].double().numpy()
        Oref, LSEref = orc.attn_fwd(cut(Q), cut(K), cut(V), f[b:b + 1, :Lv], a, n)
        assert_close(On[b:b + 1, :, :Lv], Oref, TOL_O, f"O[{b}]")
        assert np.abs(Ln[b:b + 1, :, :Lv] - LSEref).max() <= TOL_LSE
        refs = orc.attn_bwd(cut(Q), cut(K), cut(V), cut(dO), f[b:b + 1, :Lv], a, n)
        scales = orc.attn_bwd_term_scale(cut(Q), cut(K), cut(V), cut(dO), f[b:b + 1, :Lv], a, n)
        for got, ref, rss, what in zip((dQn, dKn, dVn), refs, scales, ("dQ", "dK", "dV")):
            g = got[b:b + 1, :, :Lv]
            assert_grad_close(g, ref, rss, f"{what}[{b}]", bf16_out=(grad_dtype == 0))
            assert errors(g, ref)[1] <= TOL_GRAD["rel_fro"], (what, b)
