"""Parity at the full benchmark sizes, in the launch configuration bench.py times, on sampled
outputs the oracle can compute one by one: whole query rows (O, LSE, dQ are functions of their own
row) and key positions near the end of the sequence (few rows keep them, so dK / dV are cheap)."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import (TOL_GRAD, TOL_LSE, TOL_O, assert_close, assert_grad_close, attn_bwd, attn_fwd,
                             build_index, errors, flags_of)

pytestmark = pytest.mark.gpu


def _sample_rows(L, n, rng):
    fixed = [0, 1, n - 1, n, n + 1, 127, 128, L // 2, L - 129, L - 128, L - 1]
    return np.unique(np.concatenate([np.array(fixed), rng.integers(0, L, 40)]))


def test_prefill_llama_shape_sampled_rows():
    c = inputs.CONFIGS["llama8b_prefill"]
    B, Hq, Hkv, L, d = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"]
    G = Hq // Hkv
    ids = inputs.token_ids(c["seed"], B, L, c["rho"], c["structure"])
    Q, K, V, dO = inputs.qkv_do(c["seed"], B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, c["n_init"], c["n_neighbor"])
    O, LSE = attn_fwd(Q.cuda(), K.cuda(), V.cuda(), idesc, index)
    O = O.float().cpu().numpy()
    LSE = LSE.cpu().numpy()
    f = flags_of(ids, inputs.SEP_IDS)[0]
    rows = _sample_rows(L, c["n_neighbor"], np.random.default_rng(3))
    for h in (0, 5, 14, 31):
        o, lse, _ = orc.attn_rows_fwd_bwd(Q[0, h].double().numpy(), K[0, h // G].double().numpy(),
                                          V[0, h // G].double().numpy(), dO[0, h].double().numpy(),
                                          f, c["n_init"], c["n_neighbor"], rows)
        assert_close(O[0, h][rows], o, TOL_O, f"O[head {h}]")
        assert np.abs(LSE[0, h][rows] - lse).max() <= TOL_LSE


@pytest.mark.parametrize("name", ["llama8b_long_r05", "llama8b_long_r10", "llama8b_long_r20"])
def test_long_context_training_sampled_rows_and_keys(name):
    c = inputs.CONFIGS[name]
    B, Hq, Hkv, L, d = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"]
    G = Hq // Hkv
    a, n = c["n_init"], c["n_neighbor"]
    ids = inputs.token_ids(c["seed"], B, L, c["rho"], c["structure"])
    Q, K, V, dO = inputs.qkv_do(c["seed"], B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, 0)
    f = flags_of(ids, inputs.SEP_IDS)[0]
    rng = np.random.default_rng(4)
    rows = _sample_rows(L, n, rng)
    On, LSEn, dQn = O.float().cpu().numpy(), LSE.cpu().numpy(), dQ.float().cpu().numpy()
    for h in (2, 29):
        o, lse, dq = orc.attn_rows_fwd_bwd(Q[0, h].double().numpy(), K[0, h // G].double().numpy(),
                                           V[0, h // G].double().numpy(), dO[0, h].double().numpy(),
                                           f, a, n, rows)
        assert_close(On[0, h][rows], o, TOL_O, f"O[head {h}]")
        assert np.abs(LSEn[0, h][rows] - lse).max() <= TOL_LSE
        assert_close(dQn[0, h][rows], dq, TOL_GRAD, f"dQ[head {h}]")
    # keys near the end: the last positions (window only) and the last separators (side + window)
    seps = np.flatnonzero(f)
    keys = np.unique(np.concatenate([np.arange(L - 24, L), seps[seps >= L - 700][-6:],
                                     np.array([L - 300, L - 513, L - 640])]))
    hk = 3
    gk = np.zeros((len(keys), d))
    gv = np.zeros((len(keys), d))
    for g in range(G):
        h = hk * G + g
        k_, v_ = orc.attn_keys_bwd(Q[0, h].double().numpy(), K[0, hk].double().numpy(),
                                   V[0, hk].double().numpy(), dO[0, h].double().numpy(), f, a, n, keys)
        gk += k_
        gv += v_
    assert_close(dK.float().cpu().numpy()[0, hk][keys], gk, TOL_GRAD, "dK")
    assert_close(dV.float().cpu().numpy()[0, hk][keys], gv, TOL_GRAD, "dV")
    # Separator keys far from the end: the first one behind the initial tokens (r10 only: every one
    # of the 65 536 rows keeps it), one in the middle and one three quarters along.  These are the
    # keys whose gradients the key-stationary side pass sums over hundreds of query tiles x G heads.
    far = [seps[seps >= L // 2][0], seps[seps >= 3 * L // 4][0]]
    if name == "llama8b_long_r10":
        far = [0, a - 1, seps[seps >= a][0]] + far
    far = np.array(sorted(set(int(x) for x in far)))
    fk = np.zeros((len(far), d))
    fv = np.zeros((len(far), d))
    for g in range(G):
        h = hk * G + g
        k_, v_ = orc.attn_keys_bwd_blocked(Q[0, h].double().numpy(), K[0, hk].double().numpy(),
                                           V[0, hk].double().numpy(), dO[0, h].double().numpy(), f, a, n, far)
        fk += k_
        fv += v_
    assert_close(dK.float().cpu().numpy()[0, hk][far], fk, TOL_GRAD, "dK of far separator keys")
    assert_close(dV.float().cpu().numpy()[0, hk][far], fv, TOL_GRAD, "dV of far separator keys")
    # a property that holds at any size: rows of A sum to one, so the column sums of dV over all
    # keys equal the sum of dO over the queries of the group (an extra check, not the parity bar)
    lhs = dV.double().sum(dim=2)[0, hk].cpu().numpy()
    rhs = dOd.double()[0, hk * G:(hk + 1) * G].sum(dim=(0, 1)).cpu().numpy()
    assert np.allclose(lhs, rhs, atol=2.0, rtol=2e-2)


def test_long_context_16k_copy_first_side_tile_keys():
    """The 16 384-token copy of the long-context workload (the shape the profiler captures use):
    dK and dV of keys of side tile 0 -- the initial tokens, the first separators -- and of a
    mid-sequence separator, each summed by the side pass over every later query tile of the four
    heads of the group, plus sampled rows for O, LSE and dQ."""
    c = inputs.CONFIGS["llama8b_L16k_r10"]
    B, Hq, Hkv, L, d = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"]
    G = Hq // Hkv
    a, n = c["n_init"], c["n_neighbor"]
    ids = inputs.token_ids(c["seed"], B, L, c["rho"], c["structure"])
    Q, K, V, dO = inputs.qkv_do(c["seed"], B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, 0)
    f = flags_of(ids, inputs.SEP_IDS)[0]
    seps = np.flatnonzero(f)
    seps = seps[seps >= a]
    keys = np.unique(np.concatenate([np.arange(a), seps[:6], seps[120:123], [seps[len(seps) // 2]], seps[-3:]]))
    for hk in (0, 6):
        gk, gv, k2, v2 = (np.zeros((len(keys), d)) for _ in range(4))
        for g in range(G):
            h = hk * G + g
            parts = orc.attn_keys_bwd_blocked(Q[0, h].double().numpy(), K[0, hk].double().numpy(),
                                              V[0, hk].double().numpy(), dO[0, h].double().numpy(), f, a, n, keys,
                                              with_term_scale=True)
            for acc, part in zip((gk, gv, k2, v2), parts):
                acc += part
        # The initial tokens take weights near 1 from the first rows of all four heads: entries of
        # 4 and more, whose bf16 rounding alone is 0.016, so an entry may exceed the absolute bound
        # as far as its own rounding floor does (none of the other keys comes near it).
        for got, ref, s2, what in ((dK, gk, k2, "dK"), (dV, gv, v2, "dV")):
            got = got.float().cpu().numpy()[0, hk][keys]
            assert_grad_close(got, ref, np.sqrt(s2), f"{what}[kv head {hk}]")
            assert errors(got, ref)[1] <= TOL_GRAD["rel_fro"]
            assert_close(got[a:], ref[a:], TOL_GRAD, f"{what}[kv head {hk}] of the separator keys")
    rows = _sample_rows(L, n, np.random.default_rng(5))
    On, LSEn, dQn = O.float().cpu().numpy(), LSE.cpu().numpy(), dQ.float().cpu().numpy()
    for h in (1, 30):
        o, lse, dq = orc.attn_rows_fwd_bwd(Q[0, h].double().numpy(), K[0, h // G].double().numpy(),
                                           V[0, h // G].double().numpy(), dO[0, h].double().numpy(),
                                           f, a, n, rows)
        assert_close(On[0, h][rows], o, TOL_O, f"O[head {h}]")
        assert np.abs(LSEn[0, h][rows] - lse).max() <= TOL_LSE
        assert_close(dQn[0, h][rows], dq, TOL_GRAD, f"dQ[head {h}]")
