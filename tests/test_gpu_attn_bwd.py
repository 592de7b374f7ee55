"""sepllm_attn_bwd against the fp64 oracle's analytic gradients."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_GRAD, assert_close, assert_grad_close, attn_bwd, attn_fwd, build_index, errors, flags_of

pytestmark = pytest.mark.gpu


def _run(B, Hq, Hkv, L, d, a, n, rho, seed, grad_dtype=0, ids=None, sep_ids=inputs.SEP_IDS, plain=False):
    """plain: the absolute bound as it stands (the workload configurations).  Otherwise an entry
    may exceed it only as far as its own rounding floor does (key 0 of a short sequence collects
    weights near 1 from the first rows of every head of the group: entries of 4 and more, where a
    bf16 result is 0.016 off by rounding alone)."""
    if ids is None:
        ids = inputs.token_ids(seed, B, L, rho, "iid")
    Q, K, V, dO = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, sep_ids, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    f = flags_of(ids, sep_ids)
    refs = orc.attn_bwd(Qn, Kn, Vn, dOn, f, a, n)
    scales = None if plain else orc.attn_bwd_term_scale(Qn, Kn, Vn, dOn, f, a, n)
    for i, (got, what) in enumerate(((dQ, "dQ"), (dK, "dK"), (dV, "dV"))):
        got = got.float().cpu().numpy()
        if plain:
            assert_close(got, refs[i], TOL_GRAD, what)
        else:
            assert_grad_close(got, refs[i], scales[i], what, bf16_out=(grad_dtype == 0))
            assert errors(got, refs[i])[1] <= TOL_GRAD["rel_fro"], (what, errors(got, refs[i]))
    return (Qd, Kd, Vd, dOd, O, LSE, idesc, index), (dQ, dK, dV)


def test_bwd_tiny_config():
    c = inputs.CONFIGS["tiny"]
    _run(c["B"], c["Hq"], c["Hkv"], c["L"], c["d"], c["n_init"], c["n_neighbor"], c["rho"], c["seed"], plain=True)


def test_bwd_pythia_shape_sampled_heads():
    """The Pythia-160m-shaped training configuration (B8 H12 d64 L2048 n256) at full size: every
    row of dQ, dK and dV of three (sequence, head) pairs (12 heads, no grouping: a head's dK and dV
    are its own)."""
    c = inputs.CONFIGS["pythia160m"]
    B, Hq, Hkv, L, d, a, n = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"], c["n_init"], c["n_neighbor"]
    ids = inputs.token_ids(c["seed"], B, L, c["rho"], c["structure"])
    Q, K, V, dO = inputs.qkv_do(c["seed"], B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, 0)
    f = flags_of(ids, inputs.SEP_IDS)
    for b, h in [(0, 0), (3, 7), (7, 11)]:
        M = orc.mask_matrix(f[b], a, n)
        rq, rk, rv = orc.attn_bwd_head(Q[b, h].double().numpy(), K[b, h].double().numpy(),
                                       V[b, h].double().numpy(), dO[b, h].double().numpy(), M)
        assert_close(dQ[b, h].float().cpu().numpy(), rq, TOL_GRAD, f"dQ[{b},{h}]")
        assert_close(dK[b, h].float().cpu().numpy(), rk, TOL_GRAD, f"dK[{b},{h}]")
        assert_close(dV[b, h].float().cpu().numpy(), rv, TOL_GRAD, f"dV[{b},{h}]")


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 4, 1), (128, 2, 2), (64, 4, 2)])
@pytest.mark.parametrize("L,a,n", [(512, 4, 64), (300, 4, 64), (777, 3, 200), (129, 2, 128), (1000, 4, 1000)])
def test_bwd_shapes(d, Hq, Hkv, L, a, n):
    _run(2, Hq, Hkv, L, d, a, n, 0.15, 200 + L + d)


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 16, 1), (128, 12, 2), (64, 3, 1)])
def test_bwd_wide_and_odd_query_groups(d, Hq, Hkv):
    """16 query heads per kv head (Falcon-40B's ratio), 6, and an odd group of 3 (no head pairing);
    the forward is checked on the way through the backward's inputs."""
    (Qd, Kd, Vd, dOd, O, LSE, idesc, index), _ = _run(1, Hq, Hkv, 700, d, 3, 96, 0.2, 230 + Hq)
    f = flags_of(inputs.token_ids(230 + Hq, 1, 700, 0.2, "iid"), inputs.SEP_IDS)
    Oref, _ = orc.attn_fwd(Qd.double().cpu().numpy(), Kd.double().cpu().numpy(), Vd.double().cpu().numpy(), f, 3, 96)
    assert_close(O.float().cpu().numpy(), Oref, dict(max_abs=1e-2, rel_fro=5e-3), "O")


def test_bwd_fp32_gradients_and_determinism():
    args, (dQ, dK, dV) = _run(1, 4, 2, 900, 128, 4, 100, 0.2, 71, grad_dtype=1)
    assert dQ.dtype == torch.float32
    Qd, Kd, Vd, dOd, O, LSE, idesc, index = args
    dQ2, dK2, dV2 = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, 1)
    assert torch.equal(dQ, dQ2) and torch.equal(dK, dK2) and torch.equal(dV, dV2)


def test_bwd_special_masks():
    L = 640
    _run(1, 2, 1, L, 128, 0, L, 0.1, 81)                      # dense causal
    _run(1, 2, 1, L, 64, 0, 100, 0.0, 82)                     # sliding window, empty side list
    ids = np.full((1, L), inputs.SEP_IDS[0], dtype=np.int32)
    _run(1, 2, 2, L, 64, 0, 1, 0.0, 83, ids=ids)              # every token a separator, n = 1
    _run(1, 2, 2, 256, 64, 0, 1, 0.3, 84)                     # n = 1 with sparse separators


def test_bwd_many_side_tiles():
    _run(1, 4, 2, 3000, 128, 4, 300, 0.3, 91)
    _run(1, 2, 2, 2500, 64, 4, 77, 0.4, 92)


def test_bwd_dv_column_sums_property():
    """Rows of A sum to one, so sum_j dV[j] equals the sum of dO over the queries of the group."""
    args, (dQ, dK, dV) = _run(1, 4, 2, 1100, 64, 4, 128, 0.12, 93, grad_dtype=1)
    dOd = args[3]
    lhs = dV.double().sum(dim=2)                                  # [B][Hkv][d]
    rhs = dOd.double().view(1, 2, 2, 1100, 64).sum(dim=(2, 3))
    # bf16 rounding of P leaves each row sum of A off by ~1e-4; over 2200 rows that is ~1e-2 here
    assert torch.allclose(lhs, rhs, atol=0.1, rtol=1e-3)
