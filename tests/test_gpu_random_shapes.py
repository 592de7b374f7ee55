"""Seeded random shapes through index, forward and backward (lengths that are no tile multiple,
neighbour counts from 1 to beyond L, separator rates from none to all, odd head groups)."""
import numpy as np
import pytest

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import (TOL_GRAD, TOL_LSE, TOL_O, assert_close, assert_grad_close, attn_bwd, attn_fwd,
                             build_index, errors, flags_of)

pytestmark = pytest.mark.gpu


def _case(seed):
    g = np.random.default_rng(seed)
    d = int(g.choice([64, 128]))
    Hkv = int(g.choice([1, 2, 3]))
    G = int(g.choice([1, 2, 3, 4, 5, 8]))
    return dict(d=d, Hkv=Hkv, Hq=Hkv * G, B=int(g.choice([1, 2, 3])), L=int(g.integers(1, 1400)),
                a=int(g.choice([0, 1, 4, 7, 130])), n=int(g.choice([1, 2, 17, 64, 128, 129, 300, 2000])),
                rho=float(g.choice([0.0, 0.02, 0.1, 0.3, 0.9, 1.0])), gd=int(g.choice([0, 1])))


@pytest.mark.parametrize("seed", range(24))
def test_random_shape(seed):
    c = _case(7000 + seed)
    B, Hq, Hkv, L, d, a, n = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"], c["a"], c["n"]
    if c["rho"] < 1.0:
        ids = inputs.token_ids(7000 + seed, B, L, c["rho"])
    else:
        ids = np.full((B, L), inputs.SEP_IDS[2], np.int32)
    f = flags_of(ids, inputs.SEP_IDS)
    Q, K, V, dO = inputs.qkv_do(7000 + seed, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    got = api.read_index(index)
    ref = orc.build_index_fast(ids, inputs.SEP_IDS, a, n, 128, 128, L)
    for k in ("cnt", "lim", "side_pos", "n_side", "tile_meta"):
        assert np.array_equal(got[k], ref[k]), (k, c)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    Oref, LSEref = orc.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(), f, a, n)
    # n = 1 or 2: rows that keep one or two keys copy V rows, whose entries reach 4 and more, where
    # a bf16 output is 0.016 off by rounding alone; only there is the bound taken relative
    assert_close(O.float().cpu().numpy(), Oref, TOL_O, f"O {c}", scaled=(n <= 2))
    assert np.abs(LSE.cpu().numpy() - LSEref).max() <= TOL_LSE, c
    grads = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype=c["gd"])
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    refs = orc.attn_bwd(Qn, Kn, Vn, dOn, f, a, n)
    scales = orc.attn_bwd_term_scale(Qn, Kn, Vn, dOn, f, a, n)
    for got_g, ref_g, rss, what in zip(grads, refs, scales, ("dQ", "dK", "dV")):
        got_g = got_g.float().cpu().numpy()
        # Plain absolute bound, except for entries whose own terms are large enough for the bf16
        # rounding of P / dS to exceed it: where a handful of keys collect thousands of weights
        # (tiny n, hardly any side entries, or a wide query group) single entries reach 10 and more.
        assert_grad_close(got_g, ref_g, rss, f"{what} {c}", bf16_out=(c["gd"] == 0))
        if np.linalg.norm(ref_g) > 1e-6:      # n = 1 without side entries: every dQ and dK is exactly 0
            assert errors(got_g, ref_g)[1] <= TOL_GRAD["rel_fro"], (what, errors(got_g, ref_g), c)
        else:
            assert np.abs(got_g - ref_g).max() <= 1e-4, (what, c)


def _variant_case(seed):
    g = np.random.default_rng(seed)
    Hkv = int(g.choice([1, 2]))
    G = int(g.choice([1, 2, 3, 4, 8]))
    B, L = int(g.choice([1, 2, 3])), int(g.integers(1, 1500))
    mode = str(g.choice(["packed", "packed+len", "varlen"]))
    return dict(d=int(g.choice([64, 80, 96, 112, 128])), Hkv=Hkv, Hq=Hkv * G, B=B, L=L,
                a=int(g.choice([0, 1, 4, 7, 130])), n=int(g.choice([3, 5, 17, 64, 128, 129, 300, 2000])),
                rho=float(g.choice([0.0, 0.02, 0.1, 0.3, 0.9])), gd=int(g.choice([0, 1])),
                mean=float(g.choice([1.0, 3.0, 40.0, 200.0, 700.0, 1e9])), mode=mode,
                lens=None if mode == "packed" else [int(g.integers(0, L + 1)) for _ in range(B)])


@pytest.mark.parametrize("seed", range(16))
def test_random_shape_packed_rows_lengths_and_head_sizes(seed):
    """The same sweep over the index variants (several documents per row, per-row lengths, both)
    and the head sizes between the kernel widths; each sequence is compared on its own tokens."""
    import torch
    from tests._gpu_util import assert_o_close
    c = _variant_case(7100 + seed)
    B, Hq, Hkv, L, d, a, n, lens = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"], c["a"], c["n"], c["lens"]
    ids = inputs.token_ids(7100 + seed, B, L, c["rho"])
    df = inputs.doc_first(7100 + seed, B, L, c["mean"]) if c["mode"] != "varlen" else None
    Q, K, V, dO = inputs.qkv_do(7100 + seed, B, Hq, Hkv, L, d)
    if lens is not None:
        for b in range(B):
            dO[b, :, lens[b]:] = 0
    idesc = api.IndexDesc(B, L, a, n, len(inputs.SEP_IDS), 128, 128, L)
    ib, sb = api.sepllm_index_bytes(idesc)
    index = api.alloc_bytes(ib)
    ids_d = torch.from_numpy(np.ascontiguousarray(ids)).cuda()
    lens_d = None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda")
    if df is None:
        api.sepllm_build_index_varlen(idesc, ids_d, lens_d, inputs.SEP_IDS, index, api.alloc_bytes(sb))
        ref = orc.build_index_fast(ids, inputs.SEP_IDS, a, n, 128, 128, L, seq_len=np.array(lens))
    else:
        api.sepllm_build_index_packed(idesc, ids_d, torch.from_numpy(df).cuda(), lens_d, inputs.SEP_IDS, index)
        ref = orc.build_index_packed(ids, df, inputs.SEP_IDS, a, n, 128, 128, L, seq_len=lens)
    torch.cuda.synchronize()
    got = api.read_index(index)
    for k in ref:
        assert np.array_equal(got[k], ref[k]), (k, c)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    grads = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype=c["gd"])
    O, LSE = O.float().cpu().numpy(), LSE.cpu().numpy()
    grads = [t.float().cpu().numpy() for t in grads]
    f = flags_of(ids, inputs.SEP_IDS)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    for b in range(B):
        Lv = L if lens is None else lens[b]
        if Lv == 0:
            continue
        sl = (slice(b, b + 1), slice(None), slice(0, Lv))
        fb = f[b:b + 1, :Lv]
        dfb = None if df is None else df[b:b + 1, :Lv]
        Oref, LSEref = orc.attn_fwd(Qn[sl], Kn[sl], Vn[sl], fb, a, n, doc_first=dfb)
        assert_o_close(O[sl], Oref, orc.attn_fwd_term_scale(Qn[sl], Kn[sl], Vn[sl], fb, a, n, doc_first=dfb), f"O {c}")
        assert np.abs(LSE[b, :, :Lv] - LSEref[0]).max() <= TOL_LSE, c
        refs = orc.attn_bwd(Qn[sl], Kn[sl], Vn[sl], dOn[sl], fb, a, n, doc_first=dfb)
        scales = orc.attn_bwd_term_scale(Qn[sl], Kn[sl], Vn[sl], dOn[sl], fb, a, n, doc_first=dfb)
        for got_g, ref_g, rss, what in zip(grads, refs, scales, ("dQ", "dK", "dV")):
            assert_grad_close(got_g[sl], ref_g, rss, f"{what} {c}", bf16_out=(c["gd"] == 0))
            if np.linalg.norm(ref_g) > 1e-2:
                assert errors(got_g[sl], ref_g)[1] <= TOL_GRAD["rel_fro"], (what, errors(got_g[sl], ref_g), c)
            else:      # one-token documents: every dQ and dK is exactly 0
                assert np.abs(got_g[sl] - ref_g).max() <= 1e-4, (what, c)
        assert not grads[1][b, :, Lv:].any() and not grads[2][b, :, Lv:].any(), c
